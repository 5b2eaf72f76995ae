/* ccr.h — C ABI of the sorted-search edge-feature join for NVIDIA B200 (sm_100a).
 *
 * The library implements one operation of the paper "Connected Content Retriever": the join of a
 * viewer's dense edge features onto a request's candidate documents at scoring time
 * (Section 3.1, Eq. 1 and Algorithm 1), fused with the gather of the candidates' document features
 * from the GPU-resident index (Section 6.3, "Feat. gather"; Section 6.3.1, "Batching and Padding")
 * and with the broadcast of the request-level features (Section 3), for a ragged batch of requests
 * in one kernel launch.
 *
 * Conventions
 *   - Plain C.  Every call returns a ccr_status; nothing throws across the boundary.
 *   - Pointers are marked HOST or DEVICE.  DEVICE pointers must belong to the store's device.
 *   - The caller owns every buffer it passes; the library keeps none of them after a call returns
 *     (asynchronous work enqueued on `stream` still reads/writes them until the stream reaches it).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Feature, key and output buffers must be 16-byte aligned; section widths (dim * element size)
 *     must be multiples of 16 bytes.
 *   - There is no CPU fallback: without a CUDA device every compute entry returns CCR_ERR_CUDA.
 *   - Host threads: the join entries (ccr_join_batch, _padded, _ex, _host with a workspace of its own) may be
 *     called on one store from several host threads at once, each on its own stream: the launch counter is
 *     atomic and every launch draws its own pair of scheduling words.  Everything that changes a store or reads
 *     its status (upload, upsert, set_tuning, set_cosine, CCR_FLAG_VALIDATE, device_status, selftest_wait, free)
 *     and ccr_join_payload_static (one shared block) must be serialised by the caller.
 *   - Handles are looked up in a table of live handles before they are used: a freed, NULL or foreign pointer
 *     gives CCR_ERR_BAD_HANDLE without being dereferenced.
 */
#ifndef CCR_H_
#define CCR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ccr_docstore ccr_docstore;   /* opaque; owns its device memory */
typedef struct ccr_workspace ccr_workspace; /* opaque; device staging for the host-buffer entry */
typedef struct ccr_idindex ccr_idindex;     /* opaque; sorted document ids + sampled search levels on the device */

typedef enum {
  CCR_OK = 0,
  CCR_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, negative size, misaligned buffer   */
  CCR_ERR_UNSUPPORTED = 2, /* a width, dtype or size outside what the kernels handle               */
  CCR_ERR_OOM = 3,         /* device (or pinned host) allocation failed or would not fit           */
  CCR_ERR_CUDA = 4,        /* a CUDA runtime call failed, or no usable device                      */
  CCR_ERR_BAD_HANDLE = 5,  /* handle is NULL, freed or not one of ours                             */
  CCR_ERR_VALIDATION = 6,  /* CCR_FLAG_VALIDATE found a broken precondition                        */
  CCR_ERR_DEVICE_WAIT = 7, /* a bounded device-side wait ran out (reported by device_status)       */
  CCR_ERR_BOUNDS = 8       /* bounds-checked build only (-DCCR_DEBUG_BOUNDS): a kernel computed an address outside the
                              buffers of its launch; the access was skipped (joins: reported by device_status; sort,
                              resolve, compaction and upsert calls wait for their kernels and return it themselves)   */
} ccr_status;

typedef enum { CCR_F16 = 0, CCR_F32 = 1 } ccr_dtype;

/* Store schema.  One store is one GPU's shard of the document index (Section 6.3, Eq. 5):
 * per-document feature rows addressed by position, plus the ids the join needs.                    */
typedef struct {
  int64_t  n_docs;          /* capacity in rows; valid positions are 0 .. n_docs-1                  */
  int32_t  doc_dim;         /* document features per row                                            */
  int32_t  doc_dtype;       /* ccr_dtype                                                            */
  int32_t  edge_dim;        /* D of Eq. 1: features per viewer-author affinity record               */
  int32_t  edge_dtype;      /* ccr_dtype (second-degree reduction needs CCR_F16)                    */
  int32_t  req_dim;         /* request-level features per request, 0 = none                         */
  int32_t  req_dtype;       /* ccr_dtype                                                            */
  int32_t  max_actors;      /* engager slots per document: 0 = first-degree store, else 1..4        */
  int32_t  device;          /* CUDA device ordinal                                                  */
  uint64_t reduce_sum_mask; /* second-degree: bit d set = edge dim d is summed over the found
                               engagers, clear = elementwise max (edge_dim <= 64 when max_actors>0) */
} ccr_docstore_desc;

/* Flags of ccr_join_batch. */
enum {
  CCR_FLAG_FORCE_SMEM        = 1u << 0, /* stage every request's full key list in shared memory
                                           (CCR_ERR_UNSUPPORTED if max_edge_len does not fit)       */
  CCR_FLAG_FORCE_GLOBAL      = 1u << 1, /* never stage keys: search them in global memory / L2      */
  CCR_FLAG_CANDS_SORTED      = 1u << 2, /* caller promises that, inside each request, the author ids of the
                                           resolved candidates are non-decreasing (a position outside
                                           [0, n_docs) has no author and may sit anywhere: a sub-tile that holds
                                           one is searched candidate by candidate).  Together with CCR_FLAG_TWO_PHASE
                                           this selects the merge-path kernel; the default kernel does not
                                           need the promise (sorted candidates still help its locality)    */
  CCR_FLAG_VALIDATE          = 1u << 3, /* check offsets, key order (and candidate order) on the
                                           device first; synchronises the stream                     */
  CCR_FLAG_FIRST_DEGREE_ONLY = 1u << 4, /* ignore engager slots of a second-degree store: no edge2
                                           section, mask is 0/1                                      */
  CCR_FLAG_FORCE_SAMPLED     = 1u << 5, /* stage only every s-th key (a sampled top of the search
                                           tree) even when the list would fit; testing aid          */
  CCR_FLAG_STATIC_SPLIT      = 1u << 6, /* warp-specialised kernel: give every block one equal contiguous
                                           slice instead of drawing chunks from a device-side counter */
  CCR_FLAG_TWO_PHASE         = 1u << 7, /* use the two-phase kernel (every warp alternates search and
                                           row streaming) instead of the warp-specialised kernel      */
  CCR_FLAG_COSINE            = 1u << 8, /* append the derived cosine section (ccr_docstore_set_cosine,
                                           ccr_join_batch_ex); adds 32 bytes to the row                */
  CCR_FLAG_NO_REBALANCE      = 1u << 10, /* second-degree joins: keep the 16-warp form of the warp-specialised kernel
                                           instead of its 20-warp form with registers moved from the search warps to
                                           the row-streaming warps (comparison aid)                                  */
  CCR_FLAG_NO_OVERLAP        = 1u << 11, /* do not let this launch move in behind a join that is still draining on the same
                                           stream (see "Back-to-back joins" at ccr_join_batch)                       */
  CCR_FLAG_WARP_SEARCH       = 1u << 12, /* lists that are searched in global memory (CCR_FLAG_FORCE_GLOBAL, key capacity 0)
                                           use the warp-cooperative 32-ary search: one id at a time, 32 pivots per round
                                           picked by ballot (comparison aid: the lane-per-id binary search is faster)     */
  CCR_FLAG_WARP_SPECIALISED  = 1u << 9  /* take the warp-specialised kernel whatever the launch size (by default a
                                           ragged launch of at most 131,072 candidates — a single request —
                                           runs on the two-phase kernel, which has the shorter start-up)      */
};

/* Create an empty store on desc->device.  Allocates doc_feats [n_docs, doc_dim] and author ids
 * int64[n_docs]; when max_actors > 0 the ids of a document (author, engagers, types) are kept in one
 * 64-byte record instead, plus a 16 MiB staging block for uploads.  Rows are uninitialised until uploaded.  The required bytes are compared
 * with the device's free memory before anything is allocated (CCR_ERR_OOM).  HOST call.            */
ccr_status ccr_docstore_create(const ccr_docstore_desc* desc, ccr_docstore** out);

/* Write rows [first_doc, first_doc + n) of the store (Section 6.2: features are written into the GPU
 * index by position).  Sources are HOST pointers when src_on_device == 0, DEVICE pointers otherwise;
 * doc_feats is [n, doc_dim] in doc_dtype, author_ids int64[n]; actor_ids int64[n, max_actors] and
 * actor_types uint8[n, max_actors] (engagement type 0 reacted, 1 commented, 2 reshared; values are
 * taken modulo 3) are required when max_actors > 0, an empty slot is any negative id.  A NULL source
 * leaves that array untouched.  Copies are enqueued on `stream`; the store must not be joined
 * against concurrently with an upload (the paper's index read/write lock, Section 6.3.1, is the
 * caller's job).                                                                                   */
ccr_status ccr_docstore_upload(ccr_docstore* store, int64_t first_doc, int64_t n,
                               const void* doc_feats, const int64_t* author_ids,
                               const int64_t* actor_ids, const uint8_t* actor_types,
                               int src_on_device, void* stream);

/* Write a batch of rows by position: the device-side write of step 3 of the per-batch bootstrap protocol of
 * Section 6.2 (features go to the positions the host assigned in step 2), also used for the steady-state
 * updates.  Row i of the batch replaces row positions[i] of the store:
 * doc_feats [n, doc_dim], author_ids int64[n], and for second-degree stores actor_ids int64[n, max_actors] /
 * actor_types uint8[n, max_actors], with the meaning they have in ccr_docstore_upload.  A NULL source leaves that
 * array untouched (an engagement update that only rewrites the engager slots passes only those).  A position
 * outside [0, n_docs) skips its row.  The positions of one call must be distinct: rows are written by many
 * threads, so two batch rows aimed at one position would leave a mixture (the paper's host-side hash map hands
 * out one position per document; coalescing repeated updates of a document inside a batch is the caller's job).
 * All pointers are DEVICE pointers (the caller brings the batch over on its ingestion stream).  One kernel on
 * `stream`, nothing allocated, no synchronisation.
 * Concurrency: a join may run at the same time on another stream as long as none of its candidates points at
 * a row this call writes — new documents go to positions no request can name before the host publishes their
 * ids, which is the order the paper's protocol prescribes (step 4 after step 3); rewriting rows that in-flight
 * requests may read needs the paper's index-level read-write lock, which stays with the caller.            */
ccr_status ccr_docstore_upsert(ccr_docstore* store, int64_t n,
                               const int32_t* positions,   /* DEVICE [n]                                  */
                               const void*    doc_feats,   /* DEVICE [n, doc_dim] or NULL                 */
                               const int64_t* author_ids,  /* DEVICE [n] or NULL                          */
                               const int64_t* actor_ids,   /* DEVICE [n, max_actors] or NULL              */
                               const uint8_t* actor_types, /* DEVICE [n, max_actors] or NULL              */
                               void* stream);

/* Free the store and its device memory.  A second free of the same handle returns CCR_ERR_BAD_HANDLE
 * (the handle is no longer in the table of live handles; the freed memory is not read).              */
ccr_status ccr_docstore_free(ccr_docstore* store);

/* Bytes of one output row for this store and these flags:
 * doc_dim*sizeof(doc) + edge_dim*sizeof(edge) [+ edge_dim*sizeof(edge) if max_actors > 0 and not
 * FIRST_DEGREE_ONLY] + req_dim*sizeof(req).  0 for a bad handle.                                    */
size_t ccr_out_row_bytes(const ccr_docstore* store, uint32_t flags);

/* The join (Eq. 1 / Algorithm 1 steps 2-4, fused with the document gather and request broadcast).
 *
 * For request r = 0 .. n_req-1, with keys = edge_keys[edge_offsets[r] .. edge_offsets[r+1]) (K of
 * them, ascending, unique and non-negative: ids are signed 64-bit and a negative id means "no id" — an empty
 * engager slot — so a negative key can never be matched) and candidates j in [cand_offsets[r], cand_offsets[r+1]):
 *     p   = cand_idx[j]                       position in the store
 *     d   = author_id[p]                      Algorithm 1's d_j
 *     pos = lower bound of d in keys;  found = pos < K and keys[pos] == d
 *     out_rows[j] = [ doc_feats[p] | found ? edge_feats[edge_offsets[r]+pos] : 0
 *                   | edge2 (second-degree stores) | req_feats[r] ]
 *     out_mask[j] = bit0 found; bits1-4 engager slot 0-3 found; bits5-7 OR of 1<<type over found slots
 * edge2[dim] reduces, over the found engager slots in ascending slot order, the matched edge rows:
 * max (strict > on the fp32 values, earlier slot wins ties, the winner's bits are kept) or sum (fp32
 * accumulator from +0, one rounded add per slot, rounded once to fp16 with ties to even; NaN is stored
 * as 0x7fff); all zero when no slot is found.  A position p < 0 or p >= n_docs gives zero doc/edge/
 * edge2 sections and mask 0 (the request section is still written).  Values are moved bit for bit.
 *
 * All array arguments are DEVICE pointers.  n_req, total_cands (= cand_offsets[n_req]) and
 * max_edge_len (>= every request's K) are HOST scalars: the offsets live on the device and the call
 * never synchronises.  cand_offsets[0] must be 0 and both offset arrays non-decreasing; they and the
 * key order are trusted unless CCR_FLAG_VALIDATE is given.  With unsorted keys or an untruthful
 * CCR_FLAG_CANDS_SORTED the values are unspecified but every access stays in bounds.
 * The call allocates nothing, clears nothing and is asynchronous: one kernel on `stream`.
 *
 * Back-to-back joins.  The warp-specialised kernel is launched with programmatic stream serialization: when the
 * work in front of it on `stream` is another join of this library, its blocks take over each SM as soon as that
 * join's block there has retired and read their own inputs (offsets, keys, candidate positions, ids) while the
 * earlier join drains; they write nothing — rows, mask — before the earlier join has completed, so reusing the
 * output buffers of the previous call is safe, and any other kernel, copy or event on the stream orders the
 * launch as usual.  What is NOT ordered is a join that reads, as an input, memory the join directly in front of
 * it writes (its rows or mask reinterpreted as keys or positions): give such a call CCR_FLAG_NO_OVERLAP.          */
ccr_status ccr_join_batch(const ccr_docstore* store,
                          int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                          const int64_t* edge_keys,    /* DEVICE [E]                               */
                          const void*    edge_feats,   /* DEVICE [E, edge_dim]                     */
                          const int64_t* edge_offsets, /* DEVICE [n_req + 1]                       */
                          const int32_t* cand_idx,     /* DEVICE [total_cands]                     */
                          const int64_t* cand_offsets, /* DEVICE [n_req + 1]                       */
                          const void*    req_feats,    /* DEVICE [n_req, req_dim]; NULL if req_dim == 0 */
                          void*          out_rows,     /* DEVICE [total_cands, out_row_bytes]      */
                          uint8_t*       out_mask,     /* DEVICE [total_cands]                     */
                          uint32_t       flags,
                          void*          stream);

/* Batching and padding of variable-length requests (Section 6.3.1, "Batching and Padding for Variable-Length
 * Requests").  The section pads a batch of b requests with n_i valid candidates each to n_max = max n_i in
 * three steps: scatter indices (batch_idx, pos_idx) from the valid-position masks; the valid positions
 * flattened across the batch for a single gather; a scatter of the gathered rows into T[b, n_max, features].
 * The two entries below are those steps.
 *
 * ccr_compact_valid is the first two: a candidate is valid when 0 <= cand_idx[j] < n_docs (the resolver writes
 * -1 for an unknown id).  For every request r its valid positions are copied, in their input order, to
 * idx_out[offsets_out[r] .. offsets_out[r+1]); offsets_out[0] = 0 and offsets_out[r+1] - offsets_out[r] = n_r.
 * The scatter index of kept candidate k of request r is therefore (r, k - offsets_out[r]).  src_out (optional,
 * int32[>= number of valid candidates]) receives the flat input index j of every kept candidate, so that
 * scores can be carried back to the caller's candidate order (CCR_ERR_UNSUPPORTED when total_cands exceeds
 * 2^31 - 1, the range of those indices).  idx_out needs room for cand_offsets[n_req]
 * entries (all candidates may be valid); idx_out / offsets_out must not alias the inputs.  All pointers are
 * DEVICE pointers; three small kernels on `stream`, nothing allocated, no synchronisation.  total_cands only
 * chooses how many blocks share a request (from the mean request length); the count pass uses one block per
 * request, so the cost grows with the longest request rather than with the batch.
 *
 * ccr_join_batch_padded is the gather and the scatter in one kernel: the join of ccr_join_batch with the
 * same arguments, flags and kernels, except that the row and mask of candidate j of request r are written at
 * slot r * n_max + (j - cand_offsets[r]) of out_rows [n_req * n_max, out_row_bytes] / out_mask
 * [n_req * n_max] instead of at j, so every gathered row is written once, at its place in T.  Slots behind a
 * request's last candidate (pads) are all-zero rows — request section included — with mask 0; the caller
 * masks their scores using n_r from the offsets.  n_max (HOST scalar, > 0) is normally the longest request;
 * with a smaller n_max the candidates of a request behind its n_max-th are dropped.  Because the compacted
 * offsets live on the device, total_cands may here be any upper bound of cand_offsets[n_req] (for instance
 * the candidate count before compaction): flat indices at or above cand_offsets[n_req] belong to no request
 * and are skipped.  CCR_FLAG_VALIDATE is not supported (CCR_ERR_UNSUPPORTED): validate with ccr_join_batch
 * semantics first.  Two kernels on `stream` (pad fill, join); nothing allocated.                          */
ccr_status ccr_compact_valid(const ccr_docstore* store, int32_t n_req,
                             int64_t        total_cands,  /* HOST: cand_offsets[n_req] (sizes the launch only) */
                             const int32_t* cand_idx,     /* DEVICE [cand_offsets[n_req]]               */
                             const int64_t* cand_offsets, /* DEVICE [n_req + 1]                         */
                             int32_t*       idx_out,      /* DEVICE [cand_offsets[n_req]]               */
                             int64_t*       offsets_out,  /* DEVICE [n_req + 1]                         */
                             int32_t*       src_out,      /* DEVICE [cand_offsets[n_req]] or NULL       */
                             void*          stream);

ccr_status ccr_join_batch_padded(const ccr_docstore* store,
                                 int32_t n_req, int64_t total_cands, int64_t max_edge_len, int64_t n_max,
                                 const int64_t* edge_keys, const void* edge_feats, const int64_t* edge_offsets,
                                 const int32_t* cand_idx, const int64_t* cand_offsets, const void* req_feats,
                                 void*          out_rows,  /* DEVICE [n_req * n_max, out_row_bytes]       */
                                 uint8_t*       out_mask,  /* DEVICE [n_req * n_max]                      */
                                 uint32_t       flags,
                                 void*          stream);

/* Derived features (Section 4.1.2 "Derived Features"): the member representation is n_chunks medoid embeddings
 * of `dim` values each (3 x 50 in the paper), the item embedding has `dim` values; per chunk the cosine
 * similarity is computed in float32 and stored as float16.  Here the item embedding is elements
 * [item_first, item_first + dim) of the document row (float16 stores only; item_first a multiple of 8; the
 * 16-byte piece holding the last element must lie inside the row), and the member embeddings arrive per
 * request through ccr_join_io::member_emb.  With CCR_FLAG_COSINE every output row gets a last 32-byte section
 * [cos_0 .. cos_{n_chunks-1}, 0 ...] of float16 values (one whole 32-byte sector, so that rows whose other
 * sections are multiples of 32 bytes stay sector-aligned), computed by the join kernel from the row it streams:
 *     dot_k = sum_e x[e] m_k[e],  |x|^2 = sum_e x[e]^2,  |m_k|^2 = sum_e m_k[e]^2
 *             each a float32 fused-multiply-add chain from +0 over e = 0 .. dim-1 in ascending order;
 *     den_k = sqrtf(|x|^2) * sqrtf(|m_k|^2), replaced by 1e-8 unless den_k > 1e-8 (zero vectors give 0);
 *     cos_k = float16(dot_k / den_k), round to nearest even; NaN is stored as 0x7fff.
 * A candidate whose position is outside [0, n_docs) has x = 0.  dim <= 64, n_chunks <= 4
 * (CCR_ERR_UNSUPPORTED above).  spec == NULL switches the section off.  HOST call, no device work.      */
typedef struct {
  int32_t item_first; /* first element of the item embedding in a document row            */
  int32_t dim;        /* elements per chunk                                                 */
  int32_t n_chunks;   /* medoid chunks of the member representation                         */
  int32_t reserved;   /* 0                                                                  */
} ccr_cosine_spec;
ccr_status ccr_docstore_set_cosine(ccr_docstore* store, const ccr_cosine_spec* spec);

/* The join with every optional input in one argument block: ccr_join_batch (n_max == 0) or
 * ccr_join_batch_padded (n_max > 0) with the same meaning of every field, plus member_emb for
 * CCR_FLAG_COSINE: DEVICE float16 [n_req, n_chunks * dim], chunk k of request r at
 * member_emb[(r * n_chunks + k) * dim], 2-byte aligned; ignored without the flag.  struct_bytes must be
 * sizeof(ccr_join_io).  The derived section is computed by the warp-specialised kernel only: with
 * CCR_FLAG_TWO_PHASE the call returns CCR_ERR_UNSUPPORTED.                                                 */
typedef struct {
  uint32_t       struct_bytes;
  int32_t        n_req;
  int64_t        total_cands, max_edge_len;
  int64_t        n_max;          /* 0 = ragged output                                       */
  const int64_t* edge_keys;
  const void*    edge_feats;
  const int64_t* edge_offsets;
  const int32_t* cand_idx;
  const int64_t* cand_offsets;
  const void*    req_feats;
  const void*    member_emb;     /* DEVICE float16 [n_req, n_chunks * dim] or NULL          */
  void*          out_rows;
  uint8_t*       out_mask;
} ccr_join_io;
ccr_status ccr_join_batch_ex(const ccr_docstore* store, const ccr_join_io* io, uint32_t flags, void* stream);

/* Algorithm 1 step 1 for request payloads whose affinity records arrive unsorted: for every request r the
 * records [edge_offsets[r], edge_offsets[r+1]) — key int64 + feature row of the store's edge width — are put
 * in ascending key order (records with equal keys keep their input order) into keys_out / feats_out, which
 * use the same offsets and must not alias the inputs.  perm_out (optional, int32[E]) receives for every
 * output record the index of its source record inside the request.  Without perm_out every list is sorted by
 * one 1024-thread block in shared memory (one kernel); lists of more than 19,000 records then have no place to
 * be sorted in and the call returns CCR_ERR_INVALID_ARG.  With perm_out, and max_edge_len above 4,096, lists
 * whose keys leave room for the record index in one 64-bit word (non-negative, below 2^(63 - index bits): every
 * realistic id) are sorted in chunks of 4,096 records by one block each and the sorted chunks merged pairwise,
 * one grid-wide launch per doubling of the run length (the merged words alternate between keys_out and the
 * list's own part of feats_out, which therefore holds scratch data until the end of the call), so that a long
 * list is spread over many SMs instead of one, and the rows of all lists are moved by one grid-wide gather:
 * 3 + ceil(log2(max_edge_len / 4096)) small kernels on `stream` (CCR_ERR_UNSUPPORTED if n_req x the tiles of
 * max_edge_len records exceed the 2^31 - 1 blocks of a grid).
 * A batch in which some key does not leave that room is sorted list by list by the one-block kernel inside the same
 * call (a device-side flag word of the store, taken in turn from 64 such words: at most 64 calls with perm_out may be
 * in flight on one store at once, on any streams).
 * max_edge_len (HOST) must be at least the longest list; a longer list is cut there (its first max_edge_len
 * records are sorted among themselves, the rest of its output is left unwritten) and no access leaves the arrays.
 * All pointers DEVICE; no allocation, no synchronisation.
 * The output is what ccr_join_batch expects as edge_keys / edge_feats.                                    */
ccr_status ccr_sort_edges(const ccr_docstore* store, int32_t n_req, int64_t max_edge_len,
                          const int64_t* edge_keys_in, const void* edge_feats_in, const int64_t* edge_offsets,
                          int64_t* edge_keys_out, void* edge_feats_out, int32_t* perm_out, void* stream);

/* Document-id resolution on the GPU (Section 6.3.1 "Document ID Resolution", Eq. 6): pos(q) = position of
 * document id q in the index, or -1 when q is not indexed.
 *
 * ccr_idindex_create copies n_ids ascending, unique ids (HOST or DEVICE source per src_on_device) into device
 * memory and builds the sampled search levels above them (every 8th key, repeatedly, until at most 2,048
 * keys remain).  `positions` (optional, int32[n_ids], same source side) gives the store position of each id;
 * NULL means the position of an id is its rank.  Synchronous; allocates 9.2 bytes per id (+4 with positions).
 * ccr_resolve_ids writes out_pos[i] = position of query_ids[i] or -1 for n_queries DEVICE queries: one kernel
 * on `stream`, no allocation, no sync.  Ids that break the ascending order give unspecified positions but
 * every access stays in bounds.  The output is what ccr_join_batch takes as cand_idx (-1 = unresolved).      */
ccr_status ccr_idindex_create(int32_t device, int64_t n_ids, const int64_t* sorted_ids, const int32_t* positions,
                              int src_on_device, ccr_idindex** out);
ccr_status ccr_idindex_free(ccr_idindex* index);
ccr_status ccr_resolve_ids(const ccr_idindex* index, int64_t n_queries, const int64_t* query_ids,
                           int32_t* out_pos, void* stream);

/* Device staging buffers for ccr_join_batch_host, sized for the largest batch the caller will pass.
 * HOST calls; allocation happens here, never inside the join.                                      */
ccr_status ccr_workspace_create(const ccr_docstore* store, int32_t max_req, int64_t max_cands,
                                int64_t max_edges, ccr_workspace** out);
ccr_status ccr_workspace_free(ccr_workspace* ws);
/* DEVICE pointers of the workspace's output buffers: rows [max_cands, out_row_bytes], mask [max_cands]. */
ccr_status ccr_workspace_outputs(const ccr_workspace* ws, void** rows, uint8_t** mask);

/* The same join with HOST buffers (the request payload of Section 6.1.3 arrives in host memory):
 * copies the inputs to the workspace, runs ccr_join_batch, copies rows and mask back — all enqueued
 * on `stream`, nothing synchronised.  Pinned host memory makes the copies asynchronous.
 * total_edges = edge_offsets[n_req].  Sizes beyond the workspace give CCR_ERR_INVALID_ARG.
 * A batch of at least three requests and 786,432 candidates is pipelined: the requests are cut into three
 * groups of about equal candidate counts, and a group's payload crosses PCIe on a stream the workspace owns while
 * the groups already on the device are joined on `stream` (events order the two; results are those of one
 * ccr_join_batch over the whole batch).  For that the rebased offsets of the groups pass through a small pinned
 * block of the workspace with three rotation slots; a call only ever waits on the host when the copy of the call
 * three calls back has not yet run.  One workspace serves one stream at a time.
 * out_rows may be NULL: the rows then stay in the workspace's device buffer, where the ranking model reads them
 * (ccr_workspace_outputs gives the DEVICE pointers; valid until the next call on this workspace), and only the
 * mask travels back — the serving case, in which the rows never leave the GPU.                      */
ccr_status ccr_join_batch_host(const ccr_docstore* store, ccr_workspace* ws,
                               int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                               int64_t total_edges,
                               const int64_t* edge_keys, const void* edge_feats,
                               const int64_t* edge_offsets, const int32_t* cand_idx,
                               const int64_t* cand_offsets, const void* req_feats,
                               void* out_rows, uint8_t* out_mask, /* HOST */
                               uint32_t flags, void* stream);

/* The join for callers that cannot allocate device memory.  (The paper has no counterpart: this entry exists
 * for embedding the library, not for the method.)
 *
 * Who that is: code that runs after a serving process has handed all of its device memory to its own pool
 * and must not touch the CUDA allocator again — the paper's server keeps only a few hundred MB of headroom
 * beside the index and saw allocations fail under fragmentation (Section 6.3.1) — and request handlers on a
 * latency budget, for which cudaMalloc / cudaFree mean a device-wide synchronisation and an unbounded
 * stall.  Such a caller creates the store once at start-up (that does allocate) and then uses this call
 * per request batch: it takes the request payload from HOST memory (pinned memory makes the copies
 * asynchronous), writes rows and mask to the caller's DEVICE buffers, and calls neither cudaMalloc nor
 * cudaFree nor any allocating library routine.
 *
 * What it uses instead: one fixed 16 MiB block of device memory that belongs to the library image (every GPU
 * that loads the library holds it until the process exits).  The block carries the kernel's
 * scheduling words and the device copy of the payload (keys, edge rows, offsets, candidate positions, request
 * rows, each rounded up to 256 bytes).  ccr_static_payload_capacity() returns the bytes available to the
 * payload; a batch that needs more is refused with CCR_ERR_UNSUPPORTED before anything is enqueued.
 * CCR_FLAG_VALIDATE is not accepted here (CCR_ERR_UNSUPPORTED).  Because the offsets are host-readable in this
 * entry, they are checked before anything is enqueued (CCR_ERR_INVALID_ARG): cand_offsets[0] == 0, both arrays
 * non-decreasing, no request longer than max_edge_len, edge_offsets[n_req] <= total_edges and
 * cand_offsets[n_req] == total_cands.  Only the scheduling words live in the block; a bounded device-side wait
 * that runs out is recorded in the store's own status word and reported by ccr_docstore_device_status as usual.
 *
 * Sharing: all calls in a process use the same block on a device and it keeps the previous call's contents.
 * Each call re-clears the control words on `stream` before use and overwrites the payload area, so calls on
 * ONE stream are safe back to back; calls that can overlap on the GPU (different streams, or another
 * thread) race on the block and must be serialised by the caller.  Results, flags and row layout are
 * those of ccr_join_batch on the same inputs.
 *
 * First use on a device looks up the block's device address (once per device, with that device current);
 * make that first call outside any stream capture.                                                       */
size_t     ccr_static_payload_capacity(void);
ccr_status ccr_join_payload_static(const ccr_docstore* store,
                                   int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                                   int64_t total_edges,          /* = edge_offsets[n_req]                   */
                                   const int64_t* edge_keys,     /* HOST [total_edges]                      */
                                   const void*    edge_feats,    /* HOST [total_edges, edge_dim]            */
                                   const int64_t* edge_offsets,  /* HOST [n_req + 1]                        */
                                   const int32_t* cand_idx,      /* HOST [total_cands]                      */
                                   const int64_t* cand_offsets,  /* HOST [n_req + 1]                        */
                                   const void*    req_feats,     /* HOST [n_req, req_dim] or NULL           */
                                   void*          out_rows,      /* DEVICE [total_cands, out_row_bytes]     */
                                   uint8_t*       out_mask,      /* DEVICE [total_cands]                    */
                                   uint32_t flags, void* stream);

/* Synchronise `stream` and report the store's device-side status word: CCR_OK, or
 * CCR_ERR_DEVICE_WAIT if a kernel gave up a bounded wait for a shared-memory bulk copy since the
 * last call (the affected rows of that launch were not written).  Clears the word.
 * The bounds-checked build of the library (compiled with -DCCR_DEBUG_BOUNDS; `python -m paper_2609_22441_b200.build
 * --debug-bounds` writes it next to the release build) checks every global address the join, sort, resolve,
 * compaction and upsert kernels compute against the extents of the launch's buffers and leaves out an access that
 * falls outside (never a trap).  A join reports CCR_ERR_BOUNDS here; the other calls wait for their kernels and
 * return it as their own status.  The build synchronises in every call and is meant for tests, not for serving.   */
ccr_status ccr_docstore_device_status(ccr_docstore* store, void* stream);

/* Self-test of the failure-reporting path (no fault, trap or hang is involved): enqueues a one-block kernel
 * that waits, with the kernels' bounded wait cut down to a few thousand polls, on a barrier that nothing will
 * ever complete.  The wait runs out, the kernel records it and returns; the next ccr_docstore_device_status
 * reports CCR_ERR_DEVICE_WAIT (and clears the word), and the store and the context stay usable.            */
ccr_status ccr_docstore_selftest_wait(ccr_docstore* store, void* stream);

/* Tuning knobs of the join kernels; a field that is 0 keeps the store's current value.              */
typedef struct {
  int32_t tile_cands;         /* candidates per ring slot / search-copy phase pair: multiple of 256, <= 4096;
                                 unset = 256 (warp-specialised kernel; 128 in its 20-warp second-degree form, which
                                 a configured value switches off) / 1024 (two-phase kernel)                    */
  int32_t key_capacity;       /* longest list a block stages in full in shared memory (next to its hash table
                                 while both fit; longer lists keep a table only, or a sampled top of the tree);
                                 unset = what fits a 160 KB shared-memory budget per block (warp-specialised
                                 kernel) or 4096 (the others)                                                */
  int32_t ws_streamers;       /* warp-specialised kernel: row-streaming warps per block (1..14)              */
  int32_t ws_resolvers;       /* warp-specialised kernel: search warps per block (1..8); sum <= 16; set both
                                 or neither (unset = 12 + 4; one warp moves to the resolvers over a store whose author
                                 ids — 8 bytes per document, 64 with engager slots — exceed 64 MB and do not stay in
                                 L2, one to the streamers for a first-degree join with the cosine section; second-degree joins: 12 + 8 in the 20-warp form with
                                 registers moved from the search warps to the streaming warps, which a configured
                                 split switches off)                                                           */
  int32_t blocks_per_sm;      /* two-phase kernel: cap on resident blocks per SM (1..8)                      */
} ccr_tuning;
ccr_status ccr_docstore_set_tuning(ccr_docstore* store, const ccr_tuning* tuning);

/* Number of kernels the library has launched on behalf of this store since creation.               */
int64_t ccr_docstore_launch_count(const ccr_docstore* store);

const char* ccr_status_str(ccr_status s);
int         ccr_version(void);
/* 1 in the bounds-checked build, 0 in the release build. */
int         ccr_debug_bounds_enabled(void);
/* Bounds-checked build only (no-op otherwise): pretend that the output rows of the following joins and sorts on this
 * store (and the store's own rows, for upserts) end `rows` rows early, so that the mechanism itself can be tested without a real out-of-range access.   */
ccr_status  ccr_debug_shrink_outputs(ccr_docstore* store, int64_t rows);

#ifdef __cplusplus
}
#endif
#endif /* CCR_H_ */
