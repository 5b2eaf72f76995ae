// Device-side building blocks of the join kernels (sm_100a): bulk-copy + mbarrier wrappers,
// cache-hinted 128-bit loads/stores and the branch-free lower-bound searches.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace ccr {

constexpr int kThreads = 256;            // threads per block of every join kernel
constexpr int kWarps = kThreads / 32;
constexpr int kSmemHeader = 16;          // one mbarrier (8 B) + padding so that keys start 16-B aligned
constexpr unsigned kFull = 0xffffffffu;

// Device status word values (written to JoinArgs::status[0]).
constexpr int kDevOk = 0;
constexpr int kDevWaitExpired = 1;

// Ids of one document of a second-degree store, packed so that one 64-byte aligned access (two sectors)
// brings everything a lookup needs: a random 8-byte read costs HBM about as much as 100+ streamed bytes,
// and author, engagers and types in three arrays would be three such reads per candidate.
struct __align__(64) IdRec {
  long long author;
  long long actor[4];   // empty slot = negative
  uint8_t type[4];
  uint8_t pad[20];
};
static_assert(sizeof(IdRec) == 64, "one record per 64-byte line");

// Everything a join launch needs, passed by value as the kernel argument.
constexpr int kCosMaxDim = 64;     // most elements per medoid chunk
constexpr int kCosMaxChunks = 4;   // most medoid chunks
constexpr int kCosSectionBytes = 32;  // derived section of a row: fp16 cosines, zero-filled to one 32-byte sector
constexpr int kCosSlotFloat4 = kCosMaxDim + 1;  // per ring slot: element e -> (m_0[e] .. m_3[e]), then the squared norms

struct JoinArgs {
  // store
  const uint8_t* doc_feats;
  const int64_t* author_ids;  // first-degree stores: int64[n_docs]; null when id_recs is used
  const IdRec* id_recs;       // second-degree stores: one packed record per document; else null
  long long n_docs;
  int max_actors;
  unsigned long long reduce_sum_mask;
  // section widths in 16-byte chunks
  int doc_ch, edge_ch, req_ch;
  // batch
  int n_req;
  long long total;            // candidates in the launch
  int max_edge_len;           // host-promised bound on every request's key count
  const int64_t* edge_keys;
  const uint8_t* edge_feats;
  const int64_t* edge_offsets;
  const int32_t* cand_idx;
  const int64_t* cand_offsets;
  const uint8_t* req_feats;
  uint8_t* out_rows;
  uint8_t* out_mask;
  // derived features (Section 4.1.2): per-chunk cosine of the request's medoid embeddings and the candidate's
  // item embedding, appended to the row as a 32-byte section of fp16 values (zero-filled)
  const uint16_t* member_emb;  // fp16 [n_req, cos_chunks * cos_dim]; unused when cos_chunks == 0
  int cos_first;               // first element of the item embedding inside a document row (multiple of 8)
  int cos_dim;                 // elements per chunk (<= kCosMaxDim)
  int cos_chunks;              // chunks (<= kCosMaxChunks); 0 = no derived section
  int cos_stage;               // bytes of embedding staging per streamer warp: 32 rows x (pieces | 1) x 16
  long long n_max;            // 0: ragged output (row j); > 0: padded output, row r * n_max + (j - cand_offsets[r])
  // launch shape
  int tile;                   // candidates per block
  int key_cap;                // longest list a block may stage in full per request; 0 = search global memory
  int search_area;            // bytes of shared memory the search may use for keys, tables or sampled keys
  int min_stride_log2;        // >0 forces sampling with at least this stride (testing aid)
  int warp_search;            // searches that run in global memory use the warp-cooperative 32-ary search (comparison aid)
  int* status;                // device status words
  int* sched;                 // two scheduling words (next tile, finished blocks), zero between launches; or null
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Make generic-proxy writes to shared memory (the barrier's initial state) visible to the async proxy.
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// 1-D bulk copy global -> this block's shared memory through the TMA engine; completion is signalled
// on `bar` as `bytes` of transaction count.  Both addresses 16-B aligned, bytes a multiple of 16.
// The copy has a single destination: the issuing block.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait: gives up after kWaitTries polls (each poll may itself suspend for a short, hardware-defined
// time) or after kWaitNanos of wall time, whichever comes first.  Returns false when the phase never completed.
constexpr int kWaitTries = 1 << 22;
constexpr unsigned long long kWaitNanos = 2000000000ull;  // two seconds: far beyond any launch of this library
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, int tries = kWaitTries) {
  unsigned long long t0 = 0;
  for (int i = 0; i < tries; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023) == 1023) {  // the clock is read rarely: the common wait ends within a few polls
      const unsigned long long t = global_timer_ns();
      if (t0 == 0) t0 = t;
      else if (t - t0 > kWaitNanos) return false;
    }
  }
  return false;
}

// Programmatic dependent launch.  A join launched right behind another join on the same stream may become resident
// while the earlier one drains (as its blocks leave their SMs) and run everything that only reads its own inputs;
// pdl_wait() returns once the earlier grid has completed and its writes are visible, and comes before the first
// global store.  pdl_trigger() tells the runtime that this block no longer needs to hold back a dependent launch.
// Both are no-ops for a launch without the attribute or without a predecessor that triggers.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// First statement of the kernels that run as a chain of small launches (sort, compaction).  This kernel touches
// memory only after the launch in front of it has completed; when another kernel of the same chain follows
// (more_follow), that launch may be set up right away and will wait in the same way, so the launch gaps inside the
// chain overlap.  The LAST kernel of a chain never lets its successor in early: whatever is launched behind the chain
// (a join, whose resolver warps read their inputs without waiting) starts only after the whole chain has completed.
__device__ __forceinline__ void chain_enter(bool more_follow) {
  if (more_follow) pdl_trigger();
  pdl_wait();
}

// ---- bounds-checked build (-DCCR_DEBUG_BOUNDS) ------------------------------------------------------------------
// Every global load and store of the kernels goes through gload / gstore / ldg128 / st128_stream and their kin.  In the
// checked build the host registers the extent of every buffer of the launch in g_dbg; an access that does not lie
// inside one of them is not made (loads give zero), and a code is left in the store's third status word, which
// ccr_docstore_device_status reports as CCR_ERR_BOUNDS.  Nothing traps.  The release build compiles the checks away.
#ifdef CCR_DEBUG_BOUNDS
struct DbgRange {
  unsigned long long lo, hi;
};
struct DbgTable {
  DbgRange r[16];
  int n;
  int* word;
};
__device__ DbgTable g_dbg;
__device__ __noinline__ bool dbg_in_bounds(const void* p, int bytes) {
  const unsigned long long q = reinterpret_cast<unsigned long long>(p);
  for (int i = 0; i < g_dbg.n; ++i)
    if (q >= g_dbg.r[i].lo && q + static_cast<unsigned long long>(bytes) <= g_dbg.r[i].hi) return true;
  if (g_dbg.word != nullptr) atomicCAS(g_dbg.word, 0, 1);
  return false;
}
#define CCR_CHK(p, bytes) ::ccr::dbg_in_bounds((p), (bytes))
#else
#define CCR_CHK(p, bytes) true
#endif

template <typename T>
__device__ __forceinline__ T gload(const T* p) {
  if (!CCR_CHK(p, static_cast<int>(sizeof(T)))) return T{};
  return __ldg(p);
}
template <typename T, typename V>
__device__ __forceinline__ void gstore(T* p, V v) {
  if (CCR_CHK(p, static_cast<int>(sizeof(T)))) *p = static_cast<T>(v);
}
// load of data that an earlier part of the same kernel may have written (no read-only path)
template <typename T>
__device__ __forceinline__ T gload_rw(const T* p) {
  if (!CCR_CHK(p, static_cast<int>(sizeof(T)))) return T{};
  return *p;
}
__device__ __forceinline__ void gatomic_or(int* p, int v) {
  if (CCR_CHK(p, 4)) atomicOr(p, v);
}
__device__ __forceinline__ uint4 ldg128(const void* p) {
  if (!CCR_CHK(p, 16)) return make_uint4(0u, 0u, 0u, 0u);
  return __ldg(reinterpret_cast<const uint4*>(p));
}

// 128-bit load of data that is read once and whole (document rows: the 16 lanes of a row fetch its two lines in one
// instruction): not kept in L1, so the lines that are re-read there (request rows, edge rows, id records) are not
// pushed out by it.  Config 1: 207.0 -> 202.9 us.
__device__ __forceinline__ uint4 ldg128_once(const void* p) {
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (!CCR_CHK(p, 16)) return v;
#ifdef CCR_NO_L1_BYPASS
  return __ldg(reinterpret_cast<const uint4*>(p));
#else
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
#endif
}

// Author id of the document at position idx (0 <= idx < n_docs).
__device__ __forceinline__ long long load_author(const JoinArgs& a, int idx) {
  // (through L1: four ids share a sector, and bypassing L1 for these and for the candidate positions cost 6 % on
  // the batched configuration)
  return a.id_recs != nullptr ? gload(&a.id_recs[idx].author) : gload(a.author_ids + idx);
}
// 256-bit load (one whole 32-byte sector per lane), optionally past L1.
struct U32x8 {
  unsigned v[8];
};
__device__ __forceinline__ U32x8 ldg256(const void* p) {
  U32x8 r;
#pragma unroll
  for (int i = 0; i < 8; ++i) r.v[i] = 0u;
  if (!CCR_CHK(p, 32)) return r;
#ifdef CCR_IDREC_L1
  asm volatile("ld.global.nc.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
#else
  asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
#endif
               : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]), "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
               : "l"(p));
  return r;
}

// Author, engager ids and types (one byte per slot, packed little-endian) of the document at position idx: the
// 64-byte record as two 256-bit loads, each exactly one sector, read once (three 128-bit reads of the line had to go
// through L1 to be merged).
__device__ __forceinline__ void load_record(const JoinArgs& a, int idx, long long& author, long long (&act)[4], unsigned& types) {
  const unsigned char* r = reinterpret_cast<const unsigned char*>(a.id_recs + idx);
  const U32x8 lo = ldg256(r), hi = ldg256(r + 32);  // author|a0|a1|a2, a3|types|pad
  author = static_cast<long long>(lo.v[0] | (static_cast<unsigned long long>(lo.v[1]) << 32));
  act[0] = static_cast<long long>(lo.v[2] | (static_cast<unsigned long long>(lo.v[3]) << 32));
  act[1] = static_cast<long long>(lo.v[4] | (static_cast<unsigned long long>(lo.v[5]) << 32));
  act[2] = static_cast<long long>(lo.v[6] | (static_cast<unsigned long long>(lo.v[7]) << 32));
  act[3] = static_cast<long long>(hi.v[0] | (static_cast<unsigned long long>(hi.v[1]) << 32));
  types = hi.v[2];
}
// Engager ids and types only (callers that already hold the author id).
__device__ __forceinline__ void load_actors(const JoinArgs& a, int idx, long long (&act)[4], unsigned& types) {
  long long author;
  load_record(a, idx, author, act, types);
}

// Output rows are written once and never read back by the kernel: streaming (evict-first) stores keep
// them from displacing the keys, edge tables and id arrays that live in L2.
__device__ __forceinline__ void st128_stream(void* p, uint4 v) {
  if (CCR_CHK(p, 16)) __stcs(reinterpret_cast<uint4*>(p), v);
}

// Branch-free lower bound over n ascending keys: number of keys < id.  Every lane of a warp runs the
// same trip count when n is warp-uniform.
__device__ __forceinline__ int lower_bound_smem(const int64_t* s, int n, int64_t id) {
  int lo = 0;
  while (n > 1) {
    const int half = n >> 1;
    lo = (s[lo + half - 1] < id) ? lo + half : lo;
    n -= half;
  }
  if (n == 1) lo += (s[lo] < id) ? 1 : 0;
  return lo;
}

__device__ __forceinline__ int lower_bound_global(const int64_t* g, int n, int64_t id) {
  int lo = 0;
  while (n > 1) {
    const int half = n >> 1;
    lo = (gload(g + lo + half - 1) < id) ? lo + half : lo;
    n -= half;
  }
  if (n == 1) lo += (gload(g + lo) < id) ? 1 : 0;
  return lo;
}

}  // namespace ccr
