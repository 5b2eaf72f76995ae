// Host side of the C ABI declared in include/ccr.h: handles, argument checks, kernel selection, launches.
// No CPU fallback exists: when CUDA is unavailable every compute entry fails with CCR_ERR_CUDA.
#include "../../include/ccr.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <unordered_set>

#include "ccr_join.cuh"
#include "ccr_pad.cuh"
#include "ccr_resolve.cuh"
#include "ccr_sort.cuh"
#include "ccr_upsert.cuh"
#include "ccr_ws.cuh"

namespace {

constexpr uint64_t kStoreMagic = 0x43435253544f5245ull;  // "CCRSTORE"
constexpr uint64_t kWsMagic = 0x4343525753504143ull;     // "CCRWSPAC"
constexpr uint64_t kIxMagic = 0x4343524944494e44ull;     // "CCRIDIND"
constexpr int kMaxSmemBytes = 227 * 1024;
constexpr int kDefaultTileWs = 256;        // candidates per ring slot of the warp-specialised kernel
constexpr int kDefaultTileWsRebal = 128;   // ... of its register-rebalanced form (a ring twice as deep)
constexpr int kDefaultTileTwoPhase = 1024; // candidates per search/copy phase pair of the two-phase kernel
constexpr int kSmemPerSm = 228 * 1024;
constexpr int kDefaultKeyCap = 4096;
constexpr long long kSmallLaunchCands = 131072;  // plain launches up to this size default to the two-phase kernel
constexpr int kAutoSmemBudget = 160 * 1024;  // shared memory the warp-specialised kernel takes by default
constexpr long long kIdsInL2Bytes = 64LL << 20;  // an author-id array up to this size is taken to stay in the 126 MB L2
constexpr int kMaxTile = ccr::kMaxTileCands;
constexpr size_t kStageBytes = 16u << 20;  // staging block of second-degree stores (ids uploaded from the host)
#ifndef CCR_HOST_GROUPS
#define CCR_HOST_GROUPS 3  // config 1, rows staying on the device: 1 group 0.514 ms, 2 0.431, 3 0.413, 4 0.437, 6 0.456, 8 0.495
#endif
#ifndef CCR_HOST_GROUP_CANDS
#define CCR_HOST_GROUP_CANDS (2 * kSmallLaunchCands)
#endif
constexpr int kHostGroups = CCR_HOST_GROUPS;         // most request groups of a pipelined host-buffer join
constexpr int kSchedRegions = 64;                    // launches of one store that may be in flight at once
constexpr int kStatusHead = 4;                       // [0] wait expiry, [1] validation code; then the scheduling words:
                                                     // kSchedRegions regions of sched_stride ints

inline size_t dtype_size(int32_t dt) { return dt == CCR_F16 ? 2 : (dt == CCR_F32 ? 4 : 0); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Sets the store's device for the scope of a call and restores the caller's device afterwards.
struct DeviceScope {
  int prev = -1;
  bool ok = false;
  explicit DeviceScope(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    if (prev == dev) prev = -1;
  }
  ~DeviceScope() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

}  // namespace

struct ccr_docstore {
  uint64_t magic;
  ccr_docstore_desc desc;
  int doc_b, edge_b, req_b;  // section widths in bytes
  uint8_t* doc_feats;
  int64_t* author_ids;     // first-degree stores
  ccr::IdRec* id_recs;     // second-degree stores: author, engagers and types of a doc in one 64-byte record
  uint8_t* stage;          // second-degree stores: device staging for host-sourced id uploads (kStageBytes)
  int* status;        // device: [0] wait expiry, [1] validation code
  int* status_host;   // pinned host copy
  int tile;
  int key_cap;
  int blocks_per_sm;  // cap on resident blocks per SM of the two-phase kernel (0 = as many as fit)
  int ws_streamers, ws_resolvers;  // warp split of the warp-specialised kernel
  int n_sms;
  int sched_stride;   // ints per scheduling region (next tile, finished blocks; a region has a 128-byte line to itself)
  int cos_first, cos_dim, cos_chunks;  // derived cosine section (cos_chunks == 0: not configured)
  int64_t dbg_shrink_rows;             // bounds-checked build: rows cut off the registered output extents
  std::atomic<int64_t> launches;  // kernels launched for this store; also hands out the scheduling-word pairs
  std::atomic<int64_t> sort_calls;  // chunked ccr_sort_edges calls; hands out their flag words
};

struct ccr_workspace {
  uint64_t magic;
  int device;
  int32_t max_req;
  int64_t max_cands, max_edges;
  size_t out_b_max, edge_b, req_b;
  int64_t* edge_keys;
  uint8_t* edge_feats;
  int64_t* edge_offsets;
  int32_t* cand_idx;
  int64_t* cand_offsets;
  uint8_t* req_feats;
  uint8_t* out_rows;
  uint8_t* out_mask;
  // Pipelined host entry: the payload of a large batch crosses PCIe in groups of requests on a stream of the
  // workspace's own while the groups already there are being joined on the caller's stream.
  cudaStream_t copy_stream;
  cudaEvent_t ev_begin;                  // caller's stream -> copy stream: everything queued before the call
  cudaEvent_t ev_group[kHostGroups];               // copy stream -> caller's stream: group g has arrived
  cudaEvent_t ev_offsets[kHostGroups];             // the pinned offset block of rotation slot k has been read by its copy
  int64_t* host_offsets;                 // pinned: 4 rotation slots of (max_req + 1 + 4) rebased candidate offsets
  int64_t calls;
};

struct ccr_idindex {
  uint64_t magic;
  int device;
  int n_sms;
  int64_t n_ids;
  int n_levels;
  int64_t* level[ccr::kResolveMaxLevels];  // level[0] = sorted ids (owned copy)
  long long count[ccr::kResolveMaxLevels];
  int32_t* positions;                      // owned copy, or null
  int* dbg_word;                           // bounds-checked build: set by a kernel whose access left the registered buffers
  int64_t launches;
};

namespace {

// Live handles of every kind.  A handle is looked up here before it is dereferenced, so a freed (or never
// created) pointer is refused without reading the memory behind it.
std::mutex g_handles_mutex;
std::unordered_set<const void*>& live_handles() {
  static std::unordered_set<const void*>* h = new std::unordered_set<const void*>();  // never destroyed: no exit-order hazard
  return *h;
}
inline void handle_add(const void* p) {
  std::lock_guard<std::mutex> lock(g_handles_mutex);
  live_handles().insert(p);
}
inline bool handle_remove(const void* p) {  // true if it was live
  std::lock_guard<std::mutex> lock(g_handles_mutex);
  return live_handles().erase(p) != 0;
}
inline bool handle_live(const void* p) {
  if (p == nullptr) return false;
  std::lock_guard<std::mutex> lock(g_handles_mutex);
  return live_handles().count(p) != 0;
}

inline bool good(const ccr_docstore* s) { return handle_live(s) && s->magic == kStoreMagic; }
inline bool good(const ccr_workspace* w) { return handle_live(w) && w->magic == kWsMagic; }
inline bool good(const ccr_idindex* ix) { return handle_live(ix) && ix->magic == kIxMagic; }

// ---------------------------------------------------------------------------------------------------
// Precondition check behind CCR_FLAG_VALIDATE: one block per request.
//   code 1: cand_offsets malformed   2: edge_offsets malformed / longer than max_edge_len
//   code 3: keys not strictly ascending or negative   4: candidates not sorted by author (CANDS_SORTED)
__global__ void validate_kernel(const ccr::JoinArgs a, int check_sorted, int* code) {
  const int r = blockIdx.x;
  const int64_t c0 = a.cand_offsets[r], c1 = a.cand_offsets[r + 1];
  const int64_t e0 = a.edge_offsets[r], e1 = a.edge_offsets[r + 1];
  int bad = 0;
  if (threadIdx.x == 0) {
    if (c0 > c1 || c0 < 0 || (r == 0 && c0 != 0) || (r == a.n_req - 1 && c1 != a.total)) bad = 1;
    else if (e0 > e1 || e0 < 0 || e1 - e0 > a.max_edge_len) bad = 2;
  }
  bad = __syncthreads_or(bad) ? (bad ? bad : -1) : 0;
  if (bad != 0) {
    if (bad > 0) atomicCAS(code, 0, bad);
    return;
  }
  for (int64_t i = e0 + threadIdx.x; i < e1; i += blockDim.x) {
    const int64_t k = a.edge_keys[i];
    if (k < 0 || (i > e0 && a.edge_keys[i - 1] >= k)) atomicCAS(code, 0, 3);
  }
  if (check_sorted) {
    // the promise is over author ids, so it binds resolved candidates only: each one is compared with the
    // nearest resolved candidate before it (unresolved / out-of-range positions may sit anywhere)
    for (int64_t j = c0 + 1 + threadIdx.x; j < c1; j += blockDim.x) {
      const int q = a.cand_idx[j];
      if (q < 0 || q >= a.n_docs) continue;
      int64_t i = j - 1;
      while (i >= c0 && (a.cand_idx[i] < 0 || a.cand_idx[i] >= a.n_docs)) --i;
      if (i >= c0 && ccr::load_author(a, a.cand_idx[i]) > ccr::load_author(a, q)) atomicCAS(code, 0, 4);
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// Self-test of the failure-reporting path: one block waits, with the kernels' bounded wait, on a barrier that
// nothing will ever complete.  The wait must run out, the status word must be set, the kernel must return.
__global__ void selftest_wait_kernel(int* status, int tries) {
  __shared__ __align__(8) unsigned long long bar_storage;
  const uint32_t bar = ccr::smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    ccr::mbar_init(bar, 1);
    ccr::fence_proxy_async_smem();
  }
  __syncthreads();
  const bool completed = ccr::mbar_wait_bounded(bar, 0, tries);
  if (!completed && threadIdx.x == 0) atomicExch(status, ccr::kDevWaitExpired);
}

// ---------------------------------------------------------------------------------------------------
// Upload path of second-degree stores: scatter the caller's separate id arrays into the packed records.
// A null source leaves its fields untouched.
__global__ void pack_ids_kernel(ccr::IdRec* recs, long long n, int max_actors, const int64_t* author_ids,
                                const int64_t* actor_ids, const uint8_t* actor_types) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    ccr::IdRec& r = recs[i];
    if (author_ids) r.author = author_ids[i];
    if (actor_ids) {
      for (int s = 0; s < 4; ++s) r.actor[s] = s < max_actors ? actor_ids[i * max_actors + s] : -1;
    }
    if (actor_types) {
      for (int s = 0; s < 4; ++s) r.type[s] = s < max_actors ? actor_types[i * max_actors + s] : 0;
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// Kernel variants: section widths fixed at compile time for the layouts the benchmark configurations
// use (256-byte doc rows; 64- or 128-byte edge rows; 0 or 64 bytes of request features), and a generic
// variant with run-time widths for everything else.
using KernelFn = void (*)(const ccr::JoinArgs);
using WsKernelFn = void (*)(const ccr::JoinArgs, int);

// The tuned variants compute the derived cosine section for an item embedding of exactly this many 16-byte
// pieces (the paper's 50 values span 7); any other shape runs on the generic variant.
constexpr int kTunedCosPieces = 7;

// The bounds-checked build leaves the register-rebalanced form out: its checks do not fit the fixed register split.
#ifdef CCR_DEBUG_BOUNDS
constexpr bool kRebalBuilt = false;
#else
constexpr bool kRebalBuilt = true;
#endif

struct Variant {
  int doc_ch, edge_ch, req_ch;
  KernelFn first, second, merge;
  WsKernelFn ws_first, ws_second, ws_first_cos, ws_second_cos, ws_second_rebal;
};

#define CCR_VARIANT(D, E, R)                                                                                      \
  Variant {                                                                                                       \
    D, E, R, ccr::join_kernel<D, E, R, false, false>, ccr::join_kernel<D, E, R, true, false>,                     \
        ccr::join_kernel<D, E, R, false, true>,                                                                   \
        ccr::join_ws_kernel<D, E, R, false>, ccr::join_ws_kernel<D, E, R, true>,                                  \
        ccr::join_ws_kernel<D, E, R, false, (D > 0 ? kTunedCosPieces : -1)>,                                      \
        ccr::join_ws_kernel<D, E, R, true, (D > 0 ? kTunedCosPieces : -1)>,                                       \
        ccr::join_ws_kernel<D, E, R, true, 0, kRebalBuilt>                                                        \
  }

const Variant kVariants[] = {
    CCR_VARIANT(16, 4, 0),
    CCR_VARIANT(16, 4, 4),
    CCR_VARIANT(16, 8, 0),
    CCR_VARIANT(16, 8, 4),
    CCR_VARIANT(0, 0, 0),  // generic: must stay last
};
constexpr int kNumVariants = sizeof(kVariants) / sizeof(kVariants[0]);

// The padded output layout on the two-phase kernels (CCR_FLAG_TWO_PHASE, merge path): generic widths only.
const KernelFn kPaddedFirst = ccr::join_kernel<0, 0, 0, false, false, true>;
const KernelFn kPaddedSecond = ccr::join_kernel<0, 0, 0, true, false, true>;
const KernelFn kPaddedMerge = ccr::join_kernel<0, 0, 0, false, true, true>;

const Variant& pick_variant(int doc_ch, int edge_ch, int req_ch) {
  for (int i = 0; i < kNumVariants - 1; ++i) {
    const Variant& v = kVariants[i];
    if (v.doc_ch == doc_ch && v.edge_ch == edge_ch && v.req_ch == req_ch) return v;
  }
  return kVariants[kNumVariants - 1];
}

ccr_status allow_large_smem() {
  for (int i = 0; i < kNumVariants; ++i) {
    const KernelFn fns[6] = {kVariants[i].first, kVariants[i].second, kVariants[i].merge,
                             kPaddedFirst,       kPaddedSecond,      kPaddedMerge};
    for (KernelFn f : fns) {
      if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return CCR_ERR_CUDA;
      }
    }
    if (i == 0 && cudaFuncSetAttribute(ccr::sort_edges_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kMaxSmemBytes) != cudaSuccess) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    const WsKernelFn ws[5] = {kVariants[i].ws_first, kVariants[i].ws_second, kVariants[i].ws_first_cos,
                              kVariants[i].ws_second_cos, kVariants[i].ws_second_rebal};
    for (WsKernelFn f : ws) {
      if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return CCR_ERR_CUDA;
      }
    }
  }
  return CCR_OK;
}

#ifdef CCR_DEBUG_BOUNDS
// Bounds-checked build: the extents of every buffer a join launch may touch, registered before the launch.
struct DbgRegistrar {
  ccr::DbgTable t;
  DbgRegistrar() { std::memset(&t, 0, sizeof(t)); }
  void add(const void* p, size_t bytes) {
    if (p == nullptr || bytes == 0 || t.n >= 16) return;
    t.r[t.n].lo = reinterpret_cast<unsigned long long>(p);
    t.r[t.n].hi = t.r[t.n].lo + bytes;
    ++t.n;
  }
  bool commit(int* word) {
    t.word = word;
    return cudaMemcpyToSymbol(ccr::g_dbg, &t, sizeof(t)) == cudaSuccess;
  }
};
// End of a checked call outside the joins: wait for its kernels and report a flagged address as the call's status
// (the joins leave that to ccr_docstore_device_status).
ccr_status dbg_finish(int* word, cudaStream_t st) {
  int v = 0;
  if (cudaStreamSynchronize(st) != cudaSuccess || cudaMemcpy(&v, word, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return CCR_ERR_CUDA;
  }
  if (v != 0) {
    cudaMemset(word, 0, 4);
    return CCR_ERR_BOUNDS;
  }
  return CCR_OK;
}
#endif

// Launch of a kernel that belongs to a chain of small launches (its first statement is chain_enter()): with
// programmatic stream serialization the launch is set up while the kernel in front of it still runs.
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*fn)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, fn, static_cast<KArgs>(args)...);
}

size_t out_row_bytes(const ccr_docstore* s, uint32_t flags) {
  const bool second = s->desc.max_actors > 0 && !(flags & CCR_FLAG_FIRST_DEGREE_ONLY);
  return static_cast<size_t>(s->doc_b) + s->edge_b * (second ? 2 : 1) + s->req_b + ((flags & CCR_FLAG_COSINE) ? ccr::kCosSectionBytes : 0);
}

}  // namespace

extern "C" {

int ccr_version(void) { return 100; }

int ccr_debug_bounds_enabled(void) {
#ifdef CCR_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

ccr_status ccr_debug_shrink_outputs(ccr_docstore* s, int64_t rows) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  s->dbg_shrink_rows = rows < 0 ? 0 : rows;
  return CCR_OK;
}

const char* ccr_status_str(ccr_status s) {
  switch (s) {
    case CCR_OK: return "ok";
    case CCR_ERR_INVALID_ARG: return "invalid argument";
    case CCR_ERR_UNSUPPORTED: return "unsupported width, dtype or size";
    case CCR_ERR_OOM: return "out of device memory";
    case CCR_ERR_CUDA: return "CUDA runtime error or no usable device";
    case CCR_ERR_BAD_HANDLE: return "bad handle";
    case CCR_ERR_VALIDATION: return "input validation failed";
    case CCR_ERR_DEVICE_WAIT: return "a bounded device-side wait expired";
    case CCR_ERR_BOUNDS: return "bounds-checked build: an address outside the launch's buffers was skipped";
  }
  return "unknown status";
}

ccr_status ccr_docstore_create(const ccr_docstore_desc* d, ccr_docstore** out) {
  if (out == nullptr) return CCR_ERR_INVALID_ARG;
  *out = nullptr;
  if (d == nullptr) return CCR_ERR_INVALID_ARG;
  if (d->n_docs < 0 || d->doc_dim <= 0 || d->edge_dim <= 0 || d->req_dim < 0 || d->max_actors < 0 || d->device < 0)
    return CCR_ERR_INVALID_ARG;
  const size_t dsz = dtype_size(d->doc_dtype), esz = dtype_size(d->edge_dtype), rsz = dtype_size(d->req_dtype);
  if (dsz == 0 || esz == 0 || (d->req_dim > 0 && rsz == 0)) return CCR_ERR_INVALID_ARG;
  const size_t doc_b = d->doc_dim * dsz, edge_b = d->edge_dim * esz, req_b = d->req_dim * rsz;
  if (doc_b % 16 || edge_b % 16 || req_b % 16) return CCR_ERR_UNSUPPORTED;
  if (doc_b > (1u << 20) || edge_b > (1u << 20) || req_b > (1u << 20)) return CCR_ERR_UNSUPPORTED;
  if (d->n_docs > 0x7fffffffLL) return CCR_ERR_UNSUPPORTED;  // positions are int32
  if (d->max_actors > 4) return CCR_ERR_UNSUPPORTED;
  if (d->max_actors > 0 && (d->edge_dtype != CCR_F16 || d->edge_dim > 64)) return CCR_ERR_UNSUPPORTED;

  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || d->device >= n_dev) {
    cudaGetLastError();
    return CCR_ERR_CUDA;
  }
  DeviceScope scope(d->device);
  if (!scope.ok) return CCR_ERR_CUDA;

  const size_t n = static_cast<size_t>(d->n_docs);
  const size_t need = n * doc_b + (d->max_actors ? n * sizeof(ccr::IdRec) + kStageBytes : n * 8) + 4096;
  size_t free_b = 0, total_b = 0;
  if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) return CCR_ERR_CUDA;
  if (need > free_b) return CCR_ERR_OOM;

  ccr_docstore* s = new (std::nothrow) ccr_docstore();  // value-initialised: every field zero
  if (s == nullptr) return CCR_ERR_OOM;
  s->launches.store(0);
  s->sort_calls.store(0);
  s->desc = *d;
  s->doc_b = static_cast<int>(doc_b);
  s->edge_b = static_cast<int>(edge_b);
  s->req_b = static_cast<int>(req_b);
  s->tile = 0;  // automatic: kDefaultTileWs / kDefaultTileTwoPhase
  s->key_cap = 0;  // automatic
  s->ws_streamers = 0;  // automatic: 12 streamer + 4 resolver warps
  s->ws_resolvers = 0;
  if (cudaDeviceGetAttribute(&s->n_sms, cudaDevAttrMultiProcessorCount, d->device) != cudaSuccess || s->n_sms <= 0) {
    cudaGetLastError();
    delete s;
    return CCR_ERR_CUDA;
  }
  bool ok = true;
  // n == 0 still allocates a token block so that every pointer is valid and aligned
  ok = ok && cudaMalloc(&s->doc_feats, n * doc_b + 256) == cudaSuccess;
  if (d->max_actors > 0) {
    ok = ok && cudaMalloc(&s->id_recs, n * sizeof(ccr::IdRec) + 256) == cudaSuccess;
    ok = ok && cudaMalloc(&s->stage, kStageBytes) == cudaSuccess;
  } else {
    ok = ok && cudaMalloc(&s->author_ids, n * 8 + 256) == cudaSuccess;
  }
  s->sched_stride = 32;
  const size_t status_ints = kStatusHead + static_cast<size_t>(kSchedRegions) * s->sched_stride;
  ok = ok && cudaMalloc(&s->status, status_ints * sizeof(int)) == cudaSuccess;
  ok = ok && cudaMemset(s->status, 0, status_ints * sizeof(int)) == cudaSuccess;
  ok = ok && cudaHostAlloc(&s->status_host, 4 * sizeof(int), cudaHostAllocDefault) == cudaSuccess;
  ccr_status st = ok ? allow_large_smem() : CCR_ERR_OOM;
  if (st != CCR_OK) {
    cudaGetLastError();
    cudaFree(s->doc_feats);
    cudaFree(s->author_ids);
    cudaFree(s->id_recs);
    cudaFree(s->stage);
    cudaFree(s->status);
    if (s->status_host) cudaFreeHost(s->status_host);
    delete s;
    return st;
  }
  s->magic = kStoreMagic;
  handle_add(s);
  *out = s;
  return CCR_OK;
}

ccr_status ccr_docstore_free(ccr_docstore* s) {
  if (!good(s) || !handle_remove(s)) return CCR_ERR_BAD_HANDLE;  // of two racing frees only one gets past this
  DeviceScope scope(s->desc.device);
  s->magic = 0;
  cudaFree(s->doc_feats);
  cudaFree(s->author_ids);
  cudaFree(s->id_recs);
  cudaFree(s->stage);
  cudaFree(s->status);
  cudaFreeHost(s->status_host);
  delete s;
  return CCR_OK;
}

ccr_status ccr_docstore_upload(ccr_docstore* s, int64_t first_doc, int64_t n, const void* doc_feats,
                               const int64_t* author_ids, const int64_t* actor_ids, const uint8_t* actor_types,
                               int src_on_device, void* stream) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  if (first_doc < 0 || n < 0 || first_doc + n > s->desc.n_docs) return CCR_ERR_INVALID_ARG;
  if (n == 0) return CCR_OK;
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const cudaMemcpyKind kind = src_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  const size_t un = static_cast<size_t>(n), uf = static_cast<size_t>(first_doc);
  const int ma = s->desc.max_actors;
  bool ok = true;
  if (doc_feats) ok = ok && cudaMemcpyAsync(s->doc_feats + uf * s->doc_b, doc_feats, un * s->doc_b, kind, st) == cudaSuccess;
  if (ma == 0) {
    if (author_ids) ok = ok && cudaMemcpyAsync(s->author_ids + uf, author_ids, un * 8, kind, st) == cudaSuccess;
  } else if (author_ids || actor_ids || actor_types) {
    // second-degree store: the ids go into the packed records.  Device sources are packed in place; host
    // sources pass through the store's staging block, a chunk at a time (stream order keeps the block safe).
    const size_t per_row = 8 + static_cast<size_t>(ma) * 9;
    const size_t chunk = src_on_device ? un : (kStageBytes - 4096) / per_row;
    for (size_t o = 0; o < un && ok; o += chunk) {
      const size_t m = un - o < chunk ? un - o : chunk;
      const int64_t* d_auth = author_ids ? author_ids + o : nullptr;
      const int64_t* d_act = actor_ids ? actor_ids + o * ma : nullptr;
      const uint8_t* d_typ = actor_types ? actor_types + o * ma : nullptr;
      if (!src_on_device) {
        uint8_t* p = s->stage;
        if (author_ids) {
          ok = ok && cudaMemcpyAsync(p, d_auth, m * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
          d_auth = reinterpret_cast<const int64_t*>(p);
          p += (m * 8 + 255) & ~static_cast<size_t>(255);
        }
        if (actor_ids) {
          ok = ok && cudaMemcpyAsync(p, d_act, m * ma * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
          d_act = reinterpret_cast<const int64_t*>(p);
          p += (m * ma * 8 + 255) & ~static_cast<size_t>(255);
        }
        if (actor_types) {
          ok = ok && cudaMemcpyAsync(p, d_typ, m * ma, cudaMemcpyHostToDevice, st) == cudaSuccess;
          d_typ = p;
        }
      }
      const unsigned blocks = static_cast<unsigned>((m + 255) / 256 < 4096 ? (m + 255) / 256 : 4096);
      pack_ids_kernel<<<blocks, 256, 0, st>>>(s->id_recs + uf + o, static_cast<long long>(m), ma, d_auth, d_act, d_typ);
      s->launches++;
      ok = ok && cudaGetLastError() == cudaSuccess;
    }
  }
  if (!ok) {
    cudaGetLastError();
    return CCR_ERR_CUDA;
  }
  return CCR_OK;
}

ccr_status ccr_docstore_upsert(ccr_docstore* s, int64_t n, const int32_t* positions, const void* doc_feats,
                               const int64_t* author_ids, const int64_t* actor_ids, const uint8_t* actor_types,
                               void* stream) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  if (n < 0) return CCR_ERR_INVALID_ARG;
  if (n == 0) return CCR_OK;
  if (!positions) return CCR_ERR_INVALID_ARG;
  if (!aligned16(doc_feats) || (reinterpret_cast<uintptr_t>(positions) & 3u) ||
      (reinterpret_cast<uintptr_t>(author_ids) & 7u) || (reinterpret_cast<uintptr_t>(actor_ids) & 7u))
    return CCR_ERR_INVALID_ARG;
  const int ma = s->desc.max_actors;
  if (ma == 0 && (actor_ids || actor_types)) return CCR_ERR_INVALID_ARG;  // a first-degree store has no engager slots
  if (!doc_feats && !author_ids && !actor_ids && !actor_types) return CCR_OK;
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  ccr::UpsertArgs a;
  a.n = n;
  a.n_docs = s->desc.n_docs;
  a.positions = positions;
  a.src_rows = static_cast<const uint8_t*>(doc_feats);
  a.dst_rows = s->doc_feats;
  a.row_ch = s->doc_b / 16;
  a.src_author = author_ids;
  a.src_actor = actor_ids;
  a.src_type = actor_types;
  a.dst_author = s->author_ids;
  a.dst_recs = ma > 0 ? s->id_recs : nullptr;
  a.max_actors = ma;
#ifdef CCR_DEBUG_BOUNDS
  {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    const int64_t rows = s->desc.n_docs > s->dbg_shrink_rows ? s->desc.n_docs - s->dbg_shrink_rows : 0;
    DbgRegistrar reg;
    reg.add(positions, static_cast<size_t>(n) * 4);
    reg.add(doc_feats, static_cast<size_t>(n) * s->doc_b);
    reg.add(author_ids, static_cast<size_t>(n) * 8);
    reg.add(actor_ids, static_cast<size_t>(n) * ma * 8);
    reg.add(actor_types, static_cast<size_t>(n) * ma);
    reg.add(s->doc_feats, static_cast<size_t>(rows) * s->doc_b);
    reg.add(s->author_ids, static_cast<size_t>(rows) * 8);
    reg.add(s->id_recs, static_cast<size_t>(rows) * sizeof(ccr::IdRec));
    if (!reg.commit(s->status + 2)) return CCR_ERR_CUDA;
  }
#endif
  const long long work = doc_feats ? n * a.row_ch : n;
  const long long per_block = static_cast<long long>(ccr::kUpsertThreads) * ccr::kUpsertUnroll;
  long long blocks = (work + per_block - 1) / per_block;
  const long long cap = static_cast<long long>(s->n_sms) * 8;
  blocks = blocks < 1 ? 1 : (blocks > cap ? cap : blocks);
  ccr::upsert_kernel<<<static_cast<unsigned>(blocks), ccr::kUpsertThreads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  s->launches++;
  if (cudaGetLastError() != cudaSuccess) return CCR_ERR_CUDA;
#ifdef CCR_DEBUG_BOUNDS
  return dbg_finish(s->status + 2, static_cast<cudaStream_t>(stream));
#else
  return CCR_OK;
#endif
}

size_t ccr_out_row_bytes(const ccr_docstore* s, uint32_t flags) { return good(s) ? out_row_bytes(s, flags) : 0; }

ccr_status ccr_docstore_set_tuning(ccr_docstore* s, const ccr_tuning* t) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  if (t == nullptr) return CCR_ERR_INVALID_ARG;
  if (t->tile_cands < 0 || t->key_capacity < 0 || t->ws_streamers < 0 || t->ws_resolvers < 0 || t->blocks_per_sm < 0)
    return CCR_ERR_INVALID_ARG;
  if (t->tile_cands % 256 || t->tile_cands > kMaxTile) return CCR_ERR_INVALID_ARG;
  if (t->key_capacity > 0 &&
      static_cast<size_t>(ccr::search_keys_bytes(t->key_capacity)) + ccr::kSmemHeader > static_cast<size_t>(kMaxSmemBytes))
    return CCR_ERR_INVALID_ARG;
  const int st = t->ws_streamers > 0 ? t->ws_streamers : s->ws_streamers;
  const int rs = t->ws_resolvers > 0 ? t->ws_resolvers : s->ws_resolvers;
  if ((st > 0) != (rs > 0)) return CCR_ERR_INVALID_ARG;  // the warp split is set as a pair
  if (st > 14 || rs > 8 || (st + rs) * 32 > ccr::kWsMaxThreads) return CCR_ERR_INVALID_ARG;
  if (t->blocks_per_sm > 8) return CCR_ERR_INVALID_ARG;
  if (t->tile_cands > 0) s->tile = t->tile_cands;
  if (t->key_capacity > 0) s->key_cap = t->key_capacity;
  s->ws_streamers = st;
  s->ws_resolvers = rs;
  if (t->blocks_per_sm > 0) s->blocks_per_sm = t->blocks_per_sm;
  return CCR_OK;
}

int64_t ccr_docstore_launch_count(const ccr_docstore* s) { return good(s) ? s->launches.load() : -1; }

ccr_status ccr_docstore_device_status(ccr_docstore* s, void* stream) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool ok = cudaMemcpyAsync(s->status_host, s->status, 4 * sizeof(int), cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok = ok && cudaMemsetAsync(s->status, 0, 4 * sizeof(int), st) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return CCR_ERR_CUDA;
  }
  if (s->status_host[2] != 0) return CCR_ERR_BOUNDS;  // only the bounds-checked build ever sets this word
  return s->status_host[0] == ccr::kDevWaitExpired ? CCR_ERR_DEVICE_WAIT : CCR_OK;
}

ccr_status ccr_idindex_free(ccr_idindex* ix) {
  if (!good(ix) || !handle_remove(ix)) return CCR_ERR_BAD_HANDLE;
  DeviceScope scope(ix->device);
  ix->magic = 0;
  for (int l = 0; l < ccr::kResolveMaxLevels; ++l) cudaFree(ix->level[l]);
  cudaFree(ix->positions);
  cudaFree(ix->dbg_word);
  delete ix;
  return CCR_OK;
}

ccr_status ccr_idindex_create(int32_t device, int64_t n_ids, const int64_t* sorted_ids, const int32_t* positions,
                              int src_on_device, ccr_idindex** out) {
  if (out == nullptr) return CCR_ERR_INVALID_ARG;
  *out = nullptr;
  if (device < 0 || n_ids < 0 || (n_ids > 0 && sorted_ids == nullptr)) return CCR_ERR_INVALID_ARG;
  if (n_ids > 0x7fffffffLL) return CCR_ERR_UNSUPPORTED;  // positions are int32
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device >= n_dev) {
    cudaGetLastError();
    return CCR_ERR_CUDA;
  }
  DeviceScope scope(device);
  if (!scope.ok) return CCR_ERR_CUDA;
  // level sizes: sample every 8th key until the top level is small enough to stage per block
  long long count[ccr::kResolveMaxLevels];
  int n_levels = 1;
  count[0] = n_ids;
  while (count[n_levels - 1] > ccr::kResolveTopMax) {
    if (n_levels == ccr::kResolveMaxLevels) return CCR_ERR_UNSUPPORTED;
    count[n_levels] = count[n_levels - 1] >> ccr::kResolveFanLog2;
    ++n_levels;
  }
  if (n_levels == 1) {  // a tiny index still gets a (possibly empty) top level of its own
    count[1] = count[0] >> ccr::kResolveFanLog2;
    n_levels = 2;
  }
  size_t need = 4096 + (positions ? static_cast<size_t>(n_ids) * 4 : 0);
  for (int l = 0; l < n_levels; ++l) need += static_cast<size_t>(count[l]) * 8 + 256;
  size_t free_b = 0, total_b = 0;
  if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) return CCR_ERR_CUDA;
  if (need > free_b) return CCR_ERR_OOM;
  ccr_idindex* ix = new (std::nothrow) ccr_idindex();
  if (ix == nullptr) return CCR_ERR_OOM;
  std::memset(ix, 0, sizeof(*ix));
  ix->device = device;
  ix->n_ids = n_ids;
  ix->n_levels = n_levels;
  bool ok = cudaDeviceGetAttribute(&ix->n_sms, cudaDevAttrMultiProcessorCount, device) == cudaSuccess;
  for (int l = 0; l < n_levels && ok; ++l) {
    ix->count[l] = count[l];
    ok = cudaMalloc(&ix->level[l], static_cast<size_t>(count[l]) * 8 + 256) == cudaSuccess;
  }
  const cudaMemcpyKind kind = src_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  if (ok && n_ids > 0) ok = cudaMemcpy(ix->level[0], sorted_ids, static_cast<size_t>(n_ids) * 8, kind) == cudaSuccess;
  if (ok && positions && n_ids > 0) {
    ok = cudaMalloc(&ix->positions, static_cast<size_t>(n_ids) * 4) == cudaSuccess;
    ok = ok && cudaMemcpy(ix->positions, positions, static_cast<size_t>(n_ids) * 4, kind) == cudaSuccess;
  }
  for (int l = 1; l < n_levels && ok; ++l) {
    if (count[l] == 0) continue;
    const unsigned blocks = static_cast<unsigned>((count[l] + 255) / 256 < 8192 ? (count[l] + 255) / 256 : 8192);
    ccr::build_level_kernel<<<blocks, 256>>>(ix->level[l - 1], count[l - 1], ix->level[l], count[l]);
    ix->launches++;
    ok = cudaGetLastError() == cudaSuccess;
  }
  for (int l = 0; l < n_levels && ok; ++l) {  // the +infinity keys behind every level (the allocation has room)
    ccr::pad_level_kernel<<<1, 32>>>(ix->level[l], count[l]);
    ix->launches++;
    ok = cudaGetLastError() == cudaSuccess;
  }
#ifdef CCR_DEBUG_BOUNDS
  ok = ok && cudaMalloc(&ix->dbg_word, 256) == cudaSuccess && cudaMemset(ix->dbg_word, 0, 256) == cudaSuccess;
#endif
  ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(ccr::resolve_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  ccr::kResolveTopMax * 8 + 256) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(ccr::resolve_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  ccr::kResolveTopMax * 8 + 256) == cudaSuccess;
  ix->magic = kIxMagic;
  handle_add(ix);
  if (!ok) {
    cudaGetLastError();
    ccr_idindex_free(ix);
    return CCR_ERR_CUDA;
  }
  *out = ix;
  return CCR_OK;
}

ccr_status ccr_resolve_ids(const ccr_idindex* cix, int64_t n_queries, const int64_t* query_ids, int32_t* out_pos,
                           void* stream) {
  if (!good(cix)) return CCR_ERR_BAD_HANDLE;
  ccr_idindex* ix = const_cast<ccr_idindex*>(cix);  // only the launch counter changes
  if (n_queries < 0) return CCR_ERR_INVALID_ARG;
  if (n_queries == 0) return CCR_OK;
  if (!query_ids || !out_pos) return CCR_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(query_ids) & 7u) || (reinterpret_cast<uintptr_t>(out_pos) & 3u)) return CCR_ERR_INVALID_ARG;
  DeviceScope scope(ix->device);
  if (!scope.ok) return CCR_ERR_CUDA;
  ccr::ResolveArgs a;
  for (int l = 0; l < ccr::kResolveMaxLevels; ++l) {
    a.level[l] = ix->level[l];
    a.count[l] = ix->count[l];
  }
  a.n_levels = ix->n_levels;
  a.positions = ix->positions;
  a.n_queries = n_queries;
  a.queries = query_ids;
  a.out_pos = out_pos;
#ifdef CCR_DEBUG_BOUNDS
  {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    DbgRegistrar reg;
    for (int l = 0; l < ix->n_levels; ++l) reg.add(ix->level[l], static_cast<size_t>(ix->count[l] + ccr::kResolvePad) * 8);
    reg.add(ix->positions, static_cast<size_t>(ix->n_ids) * 4);
    reg.add(query_ids, static_cast<size_t>(n_queries) * 8);
    reg.add(out_pos, static_cast<size_t>(n_queries) * 4);
    if (!reg.commit(ix->dbg_word)) return CCR_ERR_CUDA;
  }
#endif
  const long long per_block = static_cast<long long>(ccr::kResolveThreads);
  const long long lanes = 1LL << (ccr::kResolveFanLog2 - 1);  // lanes that share a query
  long long blocks = (n_queries * lanes + per_block - 1) / per_block;
  const long long cap = static_cast<long long>(ix->n_sms) * ccr::kResolveBlocksPerSm;  // the top level is re-read by every block
  if (blocks > cap) blocks = cap;
  const size_t smem = static_cast<size_t>(ix->count[ix->n_levels - 1]) * 8 + 16;
  if (n_queries >= ccr::kResolveWarpMin)
    ccr::resolve_kernel<true><<<static_cast<unsigned>(blocks), ccr::kResolveThreads, smem, static_cast<cudaStream_t>(stream)>>>(a);
  else
    ccr::resolve_kernel<false><<<static_cast<unsigned>(blocks), ccr::kResolveThreads, smem, static_cast<cudaStream_t>(stream)>>>(a);
  ix->launches++;
  if (cudaGetLastError() != cudaSuccess) return CCR_ERR_CUDA;
#ifdef CCR_DEBUG_BOUNDS
  return dbg_finish(ix->dbg_word, static_cast<cudaStream_t>(stream));  // an index has no status call of its own
#else
  return CCR_OK;
#endif
}

ccr_status ccr_sort_edges(const ccr_docstore* cs, int32_t n_req, int64_t max_edge_len, const int64_t* keys_in,
                          const void* feats_in, const int64_t* edge_offsets, int64_t* keys_out, void* feats_out,
                          int32_t* perm_out, void* stream) {
  if (!good(cs)) return CCR_ERR_BAD_HANDLE;
  ccr_docstore* s = const_cast<ccr_docstore*>(cs);  // only the launch counter changes
  if (n_req < 0 || max_edge_len < 0) return CCR_ERR_INVALID_ARG;
  if (max_edge_len > 0x7fffffffLL) return CCR_ERR_UNSUPPORTED;
  if (n_req == 0 || max_edge_len == 0) return CCR_OK;
  if (!keys_in || !feats_in || !edge_offsets || !keys_out || !feats_out) return CCR_ERR_INVALID_ARG;
  if (keys_in == keys_out || feats_in == feats_out) return CCR_ERR_INVALID_ARG;  // not in place
  if (!aligned16(feats_in) || !aligned16(feats_out) || (reinterpret_cast<uintptr_t>(keys_in) & 7u) ||
      (reinterpret_cast<uintptr_t>(keys_out) & 7u) || (reinterpret_cast<uintptr_t>(perm_out) & 3u))
    return CCR_ERR_INVALID_ARG;
  if (max_edge_len > ccr::kSortSmemMaxKeys && perm_out == nullptr) return CCR_ERR_INVALID_ARG;  // long lists sort in perm_out
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  ccr::SortArgs a;
  a.n_req = n_req;
  a.keys_in = keys_in;
  a.feats_in = static_cast<const uint8_t*>(feats_in);
  a.edge_offsets = edge_offsets;
  a.row_ch = s->edge_b / 16;
  a.keys_out = keys_out;
  a.feats_out = static_cast<uint8_t*>(feats_out);
  a.perm_out = perm_out;
  a.max_len = static_cast<int>(max_edge_len);
  a.smem_keys = static_cast<int>(max_edge_len < ccr::kSortSmemMaxKeys ? max_edge_len : ccr::kSortSmemMaxKeys);
  a.smem_keys = (a.smem_keys + 1) & ~1;  // keeps the index array 8-byte aligned behind the keys
  const size_t smem = static_cast<size_t>(a.smem_keys) * 12;
  a.smem_words = static_cast<int>(smem / 8);  // packed key|index words fit half as many bytes again
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Lists longer than one chunk are spread over many blocks when the caller provides perm_out (the row gather
  // of that path reads the source indices from it).
  a.multi = (perm_out != nullptr && max_edge_len > ccr::kSortChunk) ? 1 : 0;
  // the call's flag word: word 8 of a scheduling region (the joins use words 0 and 1), regions taken in turn, so up
  // to kSchedRegions chunked sorts of one store may be in flight at once
  a.call_flag = a.multi ? s->status + kStatusHead + s->sched_stride * static_cast<int>(s->sort_calls.fetch_add(1) % kSchedRegions) + 8 : nullptr;
#ifdef CCR_DEBUG_BOUNDS
  {
    // the record count is on the device: read it back (this build synchronises anyway)
    int64_t E = 0;
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaMemcpy(&E, edge_offsets + n_req, 8, cudaMemcpyDeviceToHost) != cudaSuccess) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    const size_t row_b = static_cast<size_t>(a.row_ch) * 16;
    const int64_t out_rows_n = E > s->dbg_shrink_rows ? E - s->dbg_shrink_rows : 0;
    DbgRegistrar reg;
    reg.add(keys_in, static_cast<size_t>(E) * 8);
    reg.add(feats_in, static_cast<size_t>(E) * row_b);
    reg.add(edge_offsets, static_cast<size_t>(n_req + 1) * 8);
    reg.add(keys_out, static_cast<size_t>(E) * 8);
    reg.add(feats_out, static_cast<size_t>(out_rows_n) * row_b);
    reg.add(perm_out, static_cast<size_t>(E) * 4);
    reg.add(a.call_flag, 4);
    if (!reg.commit(s->status + 2)) return CCR_ERR_CUDA;
  }
#endif
  // grids of the chunked path: one block per tile of every list, sized for the longest list, folded into one
  // dimension; the row gather takes lists x tiles when the tiles fit a grid's second dimension (x = 0: too many blocks)
  auto tiles_grid = [&](long long per_list_units, long long tile, bool two_d) -> dim3 {
    const long long tiles = (per_list_units + tile - 1) / tile;
    if (two_d && tiles <= 65535) return dim3(static_cast<unsigned>(n_req), static_cast<unsigned>(tiles));
    const long long blocks = static_cast<long long>(n_req) * tiles;
    return dim3(blocks <= 0x7fffffffLL ? static_cast<unsigned>(blocks) : 0u);
  };
  const dim3 g_chunk = tiles_grid(max_edge_len, ccr::kSortChunk, false), g_merge = tiles_grid(max_edge_len, ccr::kSortMergeTile, false);
  const dim3 g_gather = tiles_grid(max_edge_len * a.row_ch, ccr::kSortGatherTile, true);
  if (a.multi) {
    if (g_chunk.x == 0 || g_merge.x == 0 || g_gather.x == 0) return CCR_ERR_UNSUPPORTED;
    a.more_follow = 1;  // every kernel of the call but the last lets the next one be set up early
    launch_chained(ccr::sort_chunks_kernel, g_chunk, dim3(ccr::kSortChunkThreads), 0, st, a);
    s->launches++;
    for (int phase = 1; phase <= ccr::sort_merge_phases(max_edge_len); ++phase) {
      launch_chained(ccr::sort_merge_kernel, g_merge, dim3(ccr::kSortMergeThreads), 0, st, a, phase);
      s->launches++;
    }
  }
  // short or unpackable lists (all lists without perm_out): one block per list
  a.more_follow = a.multi ? 1 : 0;
  launch_chained(ccr::sort_edges_kernel, dim3(static_cast<unsigned>(n_req)), dim3(ccr::kSortThreads), smem, st, a);
  s->launches++;
  if (a.multi) {
    a.more_follow = 0;
    launch_chained(ccr::gather_all_kernel, g_gather, dim3(ccr::kSortGatherThreads), 0, st, a);
    s->launches++;
  }
  if (cudaGetLastError() != cudaSuccess) return CCR_ERR_CUDA;
#ifdef CCR_DEBUG_BOUNDS
  return dbg_finish(s->status + 2, st);
#else
  return CCR_OK;
#endif
}

ccr_status ccr_docstore_selftest_wait(ccr_docstore* s, void* stream) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  selftest_wait_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(s->status, 2000);
  s->launches++;
  if (cudaGetLastError() != cudaSuccess) return CCR_ERR_CUDA;
  return CCR_OK;
}

}  // extern "C"

namespace {
// ccr_join_batch (n_max == 0, ragged output) and ccr_join_batch_padded (n_max > 0) share everything but the
// output addressing.
ccr_status join_impl(const ccr_docstore* cs, int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                     const int64_t* edge_keys, const void* edge_feats, const int64_t* edge_offsets,
                     const int32_t* cand_idx, const int64_t* cand_offsets, const void* req_feats,
                     void* out_rows, uint8_t* out_mask, uint32_t flags, void* stream, int64_t n_max,
                     const void* member_emb, int* sched_override = nullptr) {
  if (!good(cs)) return CCR_ERR_BAD_HANDLE;
  ccr_docstore* s = const_cast<ccr_docstore*>(cs);  // only the launch counter and status words change
  if (n_req < 0 || total_cands < 0 || max_edge_len < 0) return CCR_ERR_INVALID_ARG;
  if (max_edge_len > 0x7fffffffLL) return CCR_ERR_UNSUPPORTED;
  const uint32_t path = flags & (CCR_FLAG_FORCE_SMEM | CCR_FLAG_FORCE_GLOBAL | CCR_FLAG_FORCE_SAMPLED);
  if (path & (path - 1)) return CCR_ERR_INVALID_ARG;  // at most one forced path
  if (n_req == 0 || total_cands == 0) return (n_req == 0 && total_cands != 0) ? CCR_ERR_INVALID_ARG : CCR_OK;
  if (!edge_offsets || !cand_offsets || !cand_idx || !out_rows || !out_mask) return CCR_ERR_INVALID_ARG;
  if (max_edge_len > 0 && (!edge_keys || !edge_feats)) return CCR_ERR_INVALID_ARG;
  if (s->req_b > 0 && !req_feats) return CCR_ERR_INVALID_ARG;
  if (!aligned16(edge_keys) || !aligned16(edge_feats) || !aligned16(req_feats) || !aligned16(out_rows))
    return CCR_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(edge_offsets) & 7u) || (reinterpret_cast<uintptr_t>(cand_offsets) & 7u) ||
      (reinterpret_cast<uintptr_t>(cand_idx) & 3u))
    return CCR_ERR_INVALID_ARG;

  const bool second = s->desc.max_actors > 0 && !(flags & CCR_FLAG_FIRST_DEGREE_ONLY);
  // engager ids are not sorted, so the merge path serves first-degree joins only; a second-degree join
  // on sorted candidates takes the binary-search kernel (same result by definition)
  // (and only when the two-phase kernel is asked for: the warp-specialised kernel is the faster one on sorted
  // candidates too — 212 against 262 us on the batched configuration, 1631 against 1780 us at production scale)
  const bool merge = (flags & CCR_FLAG_CANDS_SORTED) && (flags & CCR_FLAG_TWO_PHASE) && !second;

  // which kernel: the merge path and CCR_FLAG_TWO_PHASE take the two-phase kernel, and so does a small plain
  // launch (a single request: the latency case), where the two-phase kernel's shorter start-up wins — measured
  // on one request of 30,000 candidates 16.4 against 18.4 us, 100,000 candidates x 20,000 keys 38 against 56 us;
  // from about 200,000 candidates on the warp-specialised kernel is ahead (240,000: 43 against 48 us).  The
  // same holds for second-degree joins (one request: 20.5 against 28.7 us; 240,000 candidates: equal).
  const bool cos = (flags & CCR_FLAG_COSINE) != 0;
  const bool small = total_cands <= kSmallLaunchCands && !cos && n_max == 0 &&
                     !(flags & (CCR_FLAG_WARP_SPECIALISED | CCR_FLAG_STATIC_SPLIT));
  const bool use_ws = !merge && !(flags & CCR_FLAG_TWO_PHASE) && !small;
  if (cos) {
    if (s->cos_chunks == 0 || !member_emb) return CCR_ERR_INVALID_ARG;  // not configured / no member embeddings
    if (!use_ws) return CCR_ERR_UNSUPPORTED;  // the derived section is computed by the warp-specialised kernel only
    if (reinterpret_cast<uintptr_t>(member_emb) & 1u) return CCR_ERR_INVALID_ARG;
  }
  // second-degree joins on the default warp split take the register-rebalanced form (12 + 8 warps); a configured
  // split, a configured sub-tile and the cosine section keep the 16-warp kernel
  const bool rebal = kRebalBuilt && use_ws && second && !cos && s->ws_streamers == 0 && s->tile == 0 && !(flags & CCR_FLAG_NO_REBALANCE);
  // Default split of the 16-warp kernel: 12 streamers + 4 resolvers; over a store whose author ids do not stay in L2
  // (the id array, or the 64-byte id records of a store with engagers, beyond kIdsInL2Bytes) every candidate's id is a trip to HBM and a fifth resolver pays for the
  // streamer it replaces (50M documents: 1666 -> 1639 us, sorted candidates 1643 -> 1615 us; 10 + 6: 1643 us; on the
  // 1M-document store 11 + 5 costs 2 %: 207.0 against 202.9 us).
  const long long id_bytes = s->id_recs != nullptr ? static_cast<long long>(sizeof(ccr::IdRec)) : 8;  // what holds a document's author id
  const bool ids_beyond_l2 = !second && static_cast<long long>(s->desc.n_docs) * id_bytes > kIdsInL2Bytes;
  // With the cosine section the streamers carry the arithmetic tail of every group as well, and a first-degree join
  // over a store whose ids stay in L2 does better with one resolver less (config 1: 13 + 3 242 us, 12 + 4 251 us,
  // 11 + 5 265 us, 14 + 2 269 us).
  // Over a store whose ids do not stay in L2 the two shifts cancel (50M documents with the section: 12 + 4 1950 us,
  // 11 + 5 1968 us, 13 + 3 2021 us).
  const int shift = ((cos && !second) ? 1 : 0) - (ids_beyond_l2 ? 1 : 0);  // streamers gained from the resolvers
  const int n_str = rebal ? ccr::kRebalStreamers : (s->ws_streamers > 0 ? s->ws_streamers : 12 + shift);
  const int n_res = rebal ? ccr::kRebalResolvers : (s->ws_resolvers > 0 ? s->ws_resolvers : 4 - shift);
  const int cos_stage = cos ? 32 * (((s->cos_dim + 7) / 8) | 1) * 16 : 0;
  const int cos_bytes = cos ? ccr::ws_cos_bytes(n_str, cos_stage) : 0;
  // Shared memory of a block: the kernel's own arrays for a sub-tile of t candidates plus `area` bytes for the search
  // (staged keys, hash tables, sampled keys; ccr_search.cuh).
  auto smem_for = [&](int t, int area) -> size_t {
    return use_ws ? static_cast<size_t>(ccr::WsLayout(t, second, area, n_req <= ccr::kWsMaxCachedReq ? n_req : 0, cos_bytes, n_res,
                                                      rebal ? ccr::kRebalSlots : ccr::kWsSlots,
                                                      rebal ? ccr::kRebalInFlight * 128 : ccr::kWsWorkItems).bytes)
                  : static_cast<size_t>(ccr::TileLayout(t, second, merge, area).bytes);
  };
  // bytes that hold a list of K keys in its best form: staged next to its table (the merge path builds no table)
  auto best_area = [&](long long K) -> long long {
    return K <= 0 ? 0 : ccr::search_bytes(static_cast<int>(K), !merge);
  };
  // key_cap = the longest list a block stages in full; the area is sized so that a list of key_cap keys has its
  // best form, capped by the budget.  The warp-specialised kernel runs one block per SM, so by default it serves
  // whole lists up to a shared-memory budget; the kernels that keep several blocks per SM default to
  // kDefaultKeyCap.  A configured key_capacity overrides both.
  const int tile_cfg = s->tile > 0 ? s->tile : (use_ws ? (rebal ? kDefaultTileWsRebal : kDefaultTileWs) : kDefaultTileTwoPhase);
  int tile = tile_cfg;
  long long budget = kMaxSmemBytes;  // for the whole block
  int key_cap;
  if (flags & CCR_FLAG_FORCE_GLOBAL) {
    key_cap = 0;
  } else if (flags & CCR_FLAG_FORCE_SMEM) {
    key_cap = static_cast<int>(max_edge_len);
  } else if (s->key_cap > 0 || !use_ws) {
    const long long cap = s->key_cap > 0 ? s->key_cap : kDefaultKeyCap;
    key_cap = static_cast<int>(max_edge_len < cap ? max_edge_len : cap);
  } else {
    // What the block takes from the SM's 228 KB is taken from the L1 that the streamers' loads pass through: the
    // production-scale join (lists up to 20,000 keys) ran a third slower with ~205 KB per block than with
    // 100-150 KB, hence kAutoSmemBudget for launches that are bound by streaming.  A launch of a few tiles per
    // block (a single request: the latency case) is bound by the searches and may take all of it.
    key_cap = static_cast<int>(max_edge_len);
    const long long tiles = (total_cands + tile - 1) / tile;
    const bool streaming_bound = tiles >= 2LL * s->n_sms * n_res;
    if (streaming_bound) budget = kAutoSmemBudget;
  }
  // sub-tile size: the configured one, shrunk (in steps of 256) until the kernel's arrays leave room for the keys
  // of the longest list an explicit capacity promises to stage (the automatic capacity adapts to the room instead)
  const bool explicit_cap = (flags & CCR_FLAG_FORCE_SMEM) || s->key_cap > 0;
  const int must_fit = explicit_cap ? ccr::search_keys_bytes(key_cap) : 0;
  while (tile > 256 && static_cast<long long>(smem_for(tile, must_fit)) > kMaxSmemBytes) tile -= 256;
  const long long fixed = static_cast<long long>(smem_for(tile, 0));
  long long area = best_area(key_cap);
  if (fixed + area > budget) area = budget - fixed;
  if (area < 0) area = 0;
  area &= ~15LL;
  if (explicit_cap) {
    // an explicit capacity is honoured as long as the bare keys fit in the block at all
    const long long need = ccr::search_keys_bytes(key_cap);
    if (area < need) area = need;
    if (fixed + area > kMaxSmemBytes) return CCR_ERR_UNSUPPORTED;
  } else if (key_cap > 0) {
    // automatic: lists longer than what fits in full (next to a table where one is built) are not staged
    while (key_cap > 1 && best_area(key_cap) > area) key_cap -= std::max(1, key_cap / 64);
  }
  const size_t smem = smem_for(tile, static_cast<int>(area));
  if (smem > static_cast<size_t>(kMaxSmemBytes)) return CCR_ERR_UNSUPPORTED;

  ccr::JoinArgs a;
  a.doc_feats = s->doc_feats;
  a.author_ids = s->author_ids;
  a.id_recs = s->id_recs;
  a.n_docs = s->desc.n_docs;
  a.max_actors = s->desc.max_actors;
  a.reduce_sum_mask = s->desc.reduce_sum_mask;
  a.doc_ch = s->doc_b / 16;
  a.edge_ch = s->edge_b / 16;
  a.req_ch = s->req_b / 16;
  a.n_req = n_req;
  a.total = total_cands;
  a.max_edge_len = static_cast<int>(max_edge_len);
  a.edge_keys = edge_keys;
  a.edge_feats = static_cast<const uint8_t*>(edge_feats);
  a.edge_offsets = edge_offsets;
  a.cand_idx = cand_idx;
  a.cand_offsets = cand_offsets;
  a.req_feats = static_cast<const uint8_t*>(req_feats);
  a.out_rows = static_cast<uint8_t*>(out_rows);
  a.out_mask = out_mask;
  a.n_max = n_max;
  a.member_emb = static_cast<const uint16_t*>(member_emb);
  a.cos_first = s->cos_first;
  a.cos_dim = s->cos_dim;
  a.cos_chunks = cos ? s->cos_chunks : 0;
  a.cos_stage = cos_stage;
  a.tile = tile;
  a.key_cap = key_cap;
  a.search_area = static_cast<int>(area);
  a.min_stride_log2 = (flags & CCR_FLAG_FORCE_SAMPLED) ? 2 : 0;
  a.warp_search = ((flags & CCR_FLAG_WARP_SEARCH) && use_ws) ? 1 : 0;  // its callers there are converged warps
  a.status = s->status;
  a.sched = nullptr;

  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#ifdef CCR_DEBUG_BOUNDS
  {
    // the true sizes of the ragged arrays are on the device: read them back (this build synchronises anyway)
    int64_t C = 0, E = 0;
    if (cudaStreamSynchronize(st) != cudaSuccess ||
        cudaMemcpy(&C, cand_offsets + n_req, 8, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(&E, edge_offsets + n_req, 8, cudaMemcpyDeviceToHost) != cudaSuccess) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    const size_t out_b = out_row_bytes(s, flags);
    int64_t rows = n_max > 0 ? static_cast<int64_t>(n_req) * n_max : C;
    rows = rows > s->dbg_shrink_rows ? rows - s->dbg_shrink_rows : 0;
    DbgRegistrar reg;
    reg.add(s->doc_feats, static_cast<size_t>(s->desc.n_docs) * s->doc_b);
    reg.add(s->author_ids, static_cast<size_t>(s->desc.n_docs) * 8);
    reg.add(s->id_recs, static_cast<size_t>(s->desc.n_docs) * sizeof(ccr::IdRec));
    reg.add(edge_keys, static_cast<size_t>(E) * 8);
    reg.add(edge_feats, static_cast<size_t>(E) * s->edge_b);
    reg.add(edge_offsets, static_cast<size_t>(n_req + 1) * 8);
    reg.add(cand_idx, static_cast<size_t>(C) * 4);
    reg.add(cand_offsets, static_cast<size_t>(n_req + 1) * 8);
    reg.add(req_feats, static_cast<size_t>(n_req) * s->req_b);
    if (cos) reg.add(member_emb, static_cast<size_t>(n_req) * s->cos_chunks * s->cos_dim * 2);
    reg.add(out_rows, static_cast<size_t>(rows) * out_b);
    reg.add(out_mask, static_cast<size_t>(rows));
    if (!reg.commit(s->status + 2)) return CCR_ERR_CUDA;
  }
#endif

  if (flags & CCR_FLAG_VALIDATE) {
    validate_kernel<<<n_req, 256, 0, st>>>(a, (flags & CCR_FLAG_CANDS_SORTED) ? 1 : 0, s->status + 1);
    s->launches++;
    bool ok = cudaMemcpyAsync(s->status_host + 1, s->status + 1, sizeof(int), cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemsetAsync(s->status + 1, 0, sizeof(int), st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    if (s->status_host[1] != 0) return CCR_ERR_VALIDATION;
  }

  const bool cos_tuned = cos && (s->cos_dim + 7) / 8 == kTunedCosPieces;
  const Variant& v = (cos && !cos_tuned) ? kVariants[kNumVariants - 1] : pick_variant(a.doc_ch, a.edge_ch, a.req_ch);
  const long long groups = (total_cands + 31) / 32;
  if (use_ws) {
    // one persistent warp-specialised block per SM (fewer when there are fewer 32-row groups than SMs)
    long long blocks = s->n_sms;
    if (blocks > groups) blocks = groups;
    const WsKernelFn fn = cos ? (second ? v.ws_second_cos : v.ws_first_cos) : (second ? (rebal ? v.ws_second_rebal : v.ws_second) : v.ws_first);
    // dynamic chunk scheduling through a pair of device words; each launch takes the next pair in turn, so
    // up to kSchedRegions launches of one store may be in flight at once (on any streams)
    // Small launches (fewer tiles than two rounds per block) are split evenly instead: drawing whole rounds
    // from the counter would leave most SMs without work, and a single request is the latency-critical case.
    const int n_res_auto = n_res;
    const long long n_tiles = (total_cands + a.tile - 1) / a.tile;
    const bool dynamic = !(flags & CCR_FLAG_STATIC_SPLIT) && n_tiles >= 2LL * blocks * n_res_auto;
    // (the pair is drawn from the atomic launch counter, so host threads that join against one store at the
    // same time never share a pair)
    const int64_t seq = s->launches.fetch_add(1);
    if (dynamic) a.sched = sched_override ? sched_override : s->status + kStatusHead + s->sched_stride * static_cast<int>(seq % kSchedRegions);
    // Launched with programmatic stream serialization: behind another join on the same stream the blocks become
    // resident as that join's blocks leave their SMs and prepare (barriers, offsets, first keys, first ids and
    // searches) while it drains; they store nothing before it has completed (griddepcontrol.wait in the kernel).
    // Behind any other kernel, copy or event the launch is ordered as usual.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(static_cast<unsigned>((n_str + n_res) * 32));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (flags & CCR_FLAG_NO_OVERLAP) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, fn, a, n_str) != cudaSuccess) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
  } else {
    // persistent two-phase kernel: as many blocks as stay resident, each with at least 64 candidates (a single
    // small request is spread over many SMs: 21.6 against 23.4 us for 1,000 candidates with 256 per block)
    const KernelFn fn = n_max > 0 ? (merge ? kPaddedMerge : (second ? kPaddedSecond : kPaddedFirst))
                                  : (merge ? v.merge : (second ? v.second : v.first));
    const int by_regs = ccr::kJoinMinBlocks;  // matches the kernel's __launch_bounds__
    int per_sm = static_cast<int>(kSmemPerSm / (smem + 1024));
    if (per_sm > by_regs) per_sm = by_regs;
    if (s->blocks_per_sm > 0 && per_sm > s->blocks_per_sm) per_sm = s->blocks_per_sm;
    if (per_sm < 1) per_sm = 1;
    long long blocks = static_cast<long long>(s->n_sms) * per_sm;
    const long long most = (groups + 1) / 2;
    if (blocks > most) blocks = most;
    fn<<<static_cast<unsigned>(blocks), ccr::kThreads, smem, st>>>(a);
    s->launches++;
  }
  if (cudaGetLastError() != cudaSuccess) return CCR_ERR_CUDA;
#ifdef CCR_DEBUG_BOUNDS
  if (cudaStreamSynchronize(st) != cudaSuccess) return CCR_ERR_CUDA;  // the table is one per process: no overlap
#endif
  return CCR_OK;
}

}  // namespace

extern "C" {

ccr_status ccr_join_batch(const ccr_docstore* cs, int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                          const int64_t* edge_keys, const void* edge_feats, const int64_t* edge_offsets,
                          const int32_t* cand_idx, const int64_t* cand_offsets, const void* req_feats,
                          void* out_rows, uint8_t* out_mask, uint32_t flags, void* stream) {
  if (flags & CCR_FLAG_COSINE) return CCR_ERR_INVALID_ARG;  // the member embeddings come through ccr_join_batch_ex
  return join_impl(cs, n_req, total_cands, max_edge_len, edge_keys, edge_feats, edge_offsets, cand_idx, cand_offsets,
                   req_feats, out_rows, out_mask, flags, stream, 0, nullptr);
}

}  // extern "C"

namespace {
ccr_status padded_impl(const ccr_docstore* cs, int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                       int64_t n_max, const int64_t* edge_keys, const void* edge_feats,
                       const int64_t* edge_offsets, const int32_t* cand_idx, const int64_t* cand_offsets,
                       const void* req_feats, void* out_rows, uint8_t* out_mask, uint32_t flags,
                       void* stream, const void* member_emb) {
  if (!good(cs)) return CCR_ERR_BAD_HANDLE;
  if (n_max <= 0 || n_req < 0) return CCR_ERR_INVALID_ARG;
  if (flags & CCR_FLAG_VALIDATE) return CCR_ERR_UNSUPPORTED;  // validate with ccr_join_batch semantics first
  if (n_req == 0) return CCR_OK;
  if (!cand_offsets || !out_rows || !out_mask) return CCR_ERR_INVALID_ARG;
  ccr_docstore* s = const_cast<ccr_docstore*>(cs);
  {
    DeviceScope scope(s->desc.device);
    if (!scope.ok) return CCR_ERR_CUDA;
#ifdef CCR_DEBUG_BOUNDS
    {
      DbgRegistrar reg;
      const size_t out_b = out_row_bytes(s, flags);
      reg.add(cand_offsets, static_cast<size_t>(n_req + 1) * 8);
      reg.add(out_rows, static_cast<size_t>(n_req) * n_max * out_b);
      reg.add(out_mask, static_cast<size_t>(n_req) * n_max);
      if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess || !reg.commit(s->status + 2)) return CCR_ERR_CUDA;
    }
#endif
    // enough blocks to fill the device however few requests there are
    const unsigned slices = static_cast<unsigned>(std::max(1, std::min(64, (2 * s->n_sms + n_req - 1) / n_req)));
    ccr::pad_fill_kernel<<<dim3(static_cast<unsigned>(n_req), slices), ccr::kPadThreads, 0,
                           static_cast<cudaStream_t>(stream)>>>(
        cand_offsets, n_max, static_cast<long long>(out_row_bytes(s, flags)), static_cast<uint8_t*>(out_rows), out_mask);
    s->launches++;
    if (cudaGetLastError() != cudaSuccess) return CCR_ERR_CUDA;
  }
  if (total_cands == 0) return CCR_OK;
  return join_impl(cs, n_req, total_cands, max_edge_len, edge_keys, edge_feats, edge_offsets, cand_idx, cand_offsets,
                   req_feats, out_rows, out_mask, flags, stream, n_max, member_emb);
}
}  // namespace

extern "C" {

ccr_status ccr_join_batch_padded(const ccr_docstore* cs, int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                                 int64_t n_max, const int64_t* edge_keys, const void* edge_feats,
                                 const int64_t* edge_offsets, const int32_t* cand_idx, const int64_t* cand_offsets,
                                 const void* req_feats, void* out_rows, uint8_t* out_mask, uint32_t flags,
                                 void* stream) {
  if (flags & CCR_FLAG_COSINE) return CCR_ERR_INVALID_ARG;  // the member embeddings come through ccr_join_batch_ex
  return padded_impl(cs, n_req, total_cands, max_edge_len, n_max, edge_keys, edge_feats, edge_offsets, cand_idx,
                     cand_offsets, req_feats, out_rows, out_mask, flags, stream, nullptr);
}

ccr_status ccr_join_batch_ex(const ccr_docstore* cs, const ccr_join_io* io, uint32_t flags, void* stream) {
  if (!good(cs)) return CCR_ERR_BAD_HANDLE;
  if (io == nullptr || io->struct_bytes != sizeof(ccr_join_io) || io->n_max < 0) return CCR_ERR_INVALID_ARG;
  if (io->n_max > 0)
    return padded_impl(cs, io->n_req, io->total_cands, io->max_edge_len, io->n_max, io->edge_keys, io->edge_feats,
                       io->edge_offsets, io->cand_idx, io->cand_offsets, io->req_feats, io->out_rows, io->out_mask,
                       flags, stream, io->member_emb);
  return join_impl(cs, io->n_req, io->total_cands, io->max_edge_len, io->edge_keys, io->edge_feats, io->edge_offsets,
                   io->cand_idx, io->cand_offsets, io->req_feats, io->out_rows, io->out_mask, flags, stream, 0,
                   io->member_emb);
}

ccr_status ccr_docstore_set_cosine(ccr_docstore* s, const ccr_cosine_spec* spec) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  if (spec == nullptr) {
    s->cos_first = s->cos_dim = s->cos_chunks = 0;
    return CCR_OK;
  }
  if (spec->item_first < 0 || spec->dim <= 0 || spec->n_chunks <= 0 || (spec->item_first & 7)) return CCR_ERR_INVALID_ARG;
  if (s->desc.doc_dtype != CCR_F16) return CCR_ERR_UNSUPPORTED;  // the item embedding is float16
  if (spec->dim > ccr::kCosMaxDim || spec->n_chunks > ccr::kCosMaxChunks) return CCR_ERR_UNSUPPORTED;
  // the embedding is read in 16-byte pieces: the last piece must end inside the row
  if ((spec->item_first + ((spec->dim + 7) & ~7)) * 2 > s->doc_b) return CCR_ERR_INVALID_ARG;
  s->cos_first = spec->item_first;
  s->cos_dim = spec->dim;
  s->cos_chunks = spec->n_chunks;
  return CCR_OK;
}

ccr_status ccr_compact_valid(const ccr_docstore* cs, int32_t n_req, int64_t total_cands, const int32_t* cand_idx, const int64_t* cand_offsets,
                             int32_t* idx_out, int64_t* offsets_out, int32_t* src_out, void* stream) {
  if (!good(cs)) return CCR_ERR_BAD_HANDLE;
  ccr_docstore* s = const_cast<ccr_docstore*>(cs);  // only the launch counter changes
  if (n_req < 0 || total_cands < 0) return CCR_ERR_INVALID_ARG;
  if (n_req == 0) return CCR_OK;
  if (!cand_offsets || !offsets_out || (total_cands > 0 && (!cand_idx || !idx_out))) return CCR_ERR_INVALID_ARG;
  if (src_out != nullptr && total_cands > 0x7fffffffLL) return CCR_ERR_UNSUPPORTED;  // source indices are int32
  if (cand_idx == idx_out || static_cast<const void*>(cand_offsets) == static_cast<const void*>(offsets_out))
    return CCR_ERR_INVALID_ARG;  // not in place
  if ((reinterpret_cast<uintptr_t>(cand_idx) & 3u) || (reinterpret_cast<uintptr_t>(idx_out) & 3u) ||
      (reinterpret_cast<uintptr_t>(src_out) & 3u) || (reinterpret_cast<uintptr_t>(cand_offsets) & 7u) ||
      (reinterpret_cast<uintptr_t>(offsets_out) & 7u))
    return CCR_ERR_INVALID_ARG;
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const long long n_docs = s->desc.n_docs;
#ifdef CCR_DEBUG_BOUNDS
  {
    if (cudaStreamSynchronize(st) != cudaSuccess) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    DbgRegistrar reg;
    reg.add(cand_idx, static_cast<size_t>(total_cands) * 4);
    reg.add(cand_offsets, static_cast<size_t>(n_req + 1) * 8);
    reg.add(offsets_out, static_cast<size_t>(n_req + 1) * 8);
    reg.add(idx_out, static_cast<size_t>(total_cands) * 4);
    reg.add(src_out, static_cast<size_t>(total_cands) * 4);
    if (!reg.commit(s->status + 2)) return CCR_ERR_CUDA;
  }
#endif
  launch_chained(ccr::count_valid_kernel, dim3(static_cast<unsigned>(n_req)), dim3(ccr::kPadThreads), 0, st, cand_idx, cand_offsets,
                 n_docs, offsets_out);
  launch_chained(ccr::scan_counts_kernel, dim3(1), dim3(ccr::kPadThreads), 0, st, offsets_out, n_req);
  // slices per request: about one round of the compaction each, bounded so that the re-count stays small
  const long long per_round = static_cast<long long>(ccr::kPadThreads) * ccr::kPadItems;
  const long long avg = (total_cands + n_req - 1) / n_req;
  const unsigned slices = static_cast<unsigned>(std::max(1LL, std::min(8LL, (avg + per_round - 1) / per_round)));
  launch_chained(ccr::compact_valid_kernel, dim3(static_cast<unsigned>(n_req), slices), dim3(ccr::kPadThreads), 0, st,
      cand_idx, cand_offsets, n_docs, offsets_out, idx_out, src_out);
  s->launches += 3;
  if (cudaGetLastError() != cudaSuccess) return CCR_ERR_CUDA;
#ifdef CCR_DEBUG_BOUNDS
  return dbg_finish(s->status + 2, st);
#else
  return CCR_OK;
#endif
}

ccr_status ccr_workspace_create(const ccr_docstore* s, int32_t max_req, int64_t max_cands, int64_t max_edges,
                                ccr_workspace** out) {
  if (out == nullptr) return CCR_ERR_INVALID_ARG;
  *out = nullptr;
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  if (max_req <= 0 || max_cands <= 0 || max_edges < 0) return CCR_ERR_INVALID_ARG;
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  ccr_workspace* w = new (std::nothrow) ccr_workspace();
  if (w == nullptr) return CCR_ERR_OOM;
  std::memset(w, 0, sizeof(*w));
  w->device = s->desc.device;
  w->max_req = max_req;
  w->max_cands = max_cands;
  w->max_edges = max_edges;
  w->out_b_max = out_row_bytes(s, 0);
  w->edge_b = s->edge_b;
  w->req_b = s->req_b;
  const size_t need = (max_edges + 2) * (8 + w->edge_b) + (max_req + 1) * (16 + w->req_b) + max_cands * (5 + w->out_b_max);
  size_t free_b = 0, total_b = 0;
  if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess || need + (64u << 20) > free_b) {
    cudaGetLastError();
    delete w;
    return CCR_ERR_OOM;
  }
  bool ok = true;
  ok = ok && cudaMalloc(&w->edge_keys, (max_edges + 2) * 8) == cudaSuccess;
  ok = ok && cudaMalloc(&w->edge_feats, (max_edges + 2) * w->edge_b) == cudaSuccess;
  ok = ok && cudaMalloc(&w->edge_offsets, (max_req + 1) * 8) == cudaSuccess;
  ok = ok && cudaMalloc(&w->cand_idx, max_cands * 4) == cudaSuccess;
  ok = ok && cudaMalloc(&w->cand_offsets, (max_req + 1 + kHostGroups) * 8) == cudaSuccess;
  ok = ok && cudaMalloc(&w->req_feats, (max_req + 1) * (w->req_b ? w->req_b : 16)) == cudaSuccess;
  ok = ok && cudaMalloc(&w->out_rows, max_cands * w->out_b_max) == cudaSuccess;
  ok = ok && cudaMalloc(&w->out_mask, max_cands) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&w->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&w->ev_begin, cudaEventDisableTiming) == cudaSuccess;
  for (int g = 0; g < kHostGroups; ++g) {
    ok = ok && cudaEventCreateWithFlags(&w->ev_group[g], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&w->ev_offsets[g], cudaEventDisableTiming) == cudaSuccess;
  }
  ok = ok && cudaHostAlloc(&w->host_offsets, static_cast<size_t>(kHostGroups) * (max_req + 1 + kHostGroups) * 8,
                           cudaHostAllocDefault) == cudaSuccess;
  w->magic = kWsMagic;
  handle_add(w);
  if (!ok) {
    cudaGetLastError();
    ccr_workspace_free(w);
    return CCR_ERR_OOM;
  }
  *out = w;
  return CCR_OK;
}

ccr_status ccr_workspace_free(ccr_workspace* w) {
  if (!good(w) || !handle_remove(w)) return CCR_ERR_BAD_HANDLE;
  DeviceScope scope(w->device);
  w->magic = 0;
  cudaFree(w->edge_keys);
  cudaFree(w->edge_feats);
  cudaFree(w->edge_offsets);
  cudaFree(w->cand_idx);
  cudaFree(w->cand_offsets);
  cudaFree(w->req_feats);
  cudaFree(w->out_rows);
  cudaFree(w->out_mask);
  if (w->copy_stream) cudaStreamDestroy(w->copy_stream);
  if (w->ev_begin) cudaEventDestroy(w->ev_begin);
  for (int g = 0; g < kHostGroups; ++g) {
    if (w->ev_group[g]) cudaEventDestroy(w->ev_group[g]);
    if (w->ev_offsets[g]) cudaEventDestroy(w->ev_offsets[g]);
  }
  if (w->host_offsets) cudaFreeHost(w->host_offsets);
  delete w;
  return CCR_OK;
}

ccr_status ccr_workspace_outputs(const ccr_workspace* w, void** rows, uint8_t** mask) {
  if (!good(w)) return CCR_ERR_BAD_HANDLE;
  if (rows) *rows = w->out_rows;
  if (mask) *mask = w->out_mask;
  return CCR_OK;
}

ccr_status ccr_join_batch_host(const ccr_docstore* s, ccr_workspace* w, int32_t n_req, int64_t total_cands,
                               int64_t max_edge_len, int64_t total_edges, const int64_t* edge_keys,
                               const void* edge_feats, const int64_t* edge_offsets, const int32_t* cand_idx,
                               const int64_t* cand_offsets, const void* req_feats, void* out_rows,
                               uint8_t* out_mask, uint32_t flags, void* stream) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  if (!good(w) || w->device != s->desc.device) return CCR_ERR_BAD_HANDLE;
  if (n_req < 0 || total_cands < 0 || total_edges < 0 || max_edge_len < 0) return CCR_ERR_INVALID_ARG;
  if (n_req > w->max_req || total_cands > w->max_cands || total_edges > w->max_edges) return CCR_ERR_INVALID_ARG;
  if (n_req == 0 || total_cands == 0) return (n_req == 0 && total_cands != 0) ? CCR_ERR_INVALID_ARG : CCR_OK;
  if (!edge_offsets || !cand_offsets || !cand_idx || !out_mask) return CCR_ERR_INVALID_ARG;  // out_rows may be NULL
  if (total_edges > 0 && (!edge_keys || !edge_feats)) return CCR_ERR_INVALID_ARG;
  if (s->req_b > 0 && !req_feats) return CCR_ERR_INVALID_ARG;
  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t out_b = out_row_bytes(s, flags);
  bool ok = true;
  // A batch of several large requests is pipelined: its requests are cut into up to kHostGroups groups of about
  // equal candidate counts; group g + 1 crosses PCIe on the workspace's copy stream while group g is joined on the
  // caller's stream (each group is an ordinary ccr_join_batch over its own requests, candidates renumbered from 0).
  int n_groups = 1;
  if (!(flags & CCR_FLAG_VALIDATE)) {
    const int64_t by_size = total_cands / (CCR_HOST_GROUP_CANDS);
    n_groups = static_cast<int>(by_size < kHostGroups ? by_size : kHostGroups);
    if (n_groups > n_req) n_groups = n_req;
    if (n_groups < kHostGroups) n_groups = 1;
  }
  if (n_groups == 1) {
    if (total_edges > 0) {
      ok = ok && cudaMemcpyAsync(w->edge_keys, edge_keys, total_edges * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
      ok = ok && cudaMemcpyAsync(w->edge_feats, edge_feats, total_edges * w->edge_b, cudaMemcpyHostToDevice, st) == cudaSuccess;
    }
    ok = ok && cudaMemcpyAsync(w->edge_offsets, edge_offsets, (n_req + 1) * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(w->cand_idx, cand_idx, total_cands * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(w->cand_offsets, cand_offsets, (n_req + 1) * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (s->req_b > 0)
      ok = ok && cudaMemcpyAsync(w->req_feats, req_feats, static_cast<size_t>(n_req) * w->req_b, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    const ccr_status js = ccr_join_batch(s, n_req, total_cands, max_edge_len, w->edge_keys, w->edge_feats, w->edge_offsets,
                                         w->cand_idx, w->cand_offsets, s->req_b ? w->req_feats : nullptr, w->out_rows,
                                         w->out_mask, flags, stream);
    if (js != CCR_OK) return js;
  } else {
    // group boundaries: request ranges [first[g], first[g + 1]) with about total_cands / n_groups candidates each
    int32_t first[kHostGroups + 1];
    first[0] = 0;
    int32_t r = 0;
    for (int g = 1; g < n_groups; ++g) {
      const int64_t want = total_cands * g / n_groups;
      while (r < n_req && cand_offsets[r] < want) ++r;
      if (r > n_req - (n_groups - g)) r = n_req - (n_groups - g);  // leave a request for every later group
      if (r <= first[g - 1]) r = first[g - 1] + 1;
      first[g] = r;
    }
    first[n_groups] = n_req;
    // rebased candidate offsets of every group, in a pinned block of this call's rotation slot (a slot is reused
    // kHostGroups calls later; should its copy still be pending then, the host waits for it)
    const int slot = static_cast<int>(w->calls++ % kHostGroups);
    int64_t* h_off = w->host_offsets + static_cast<size_t>(slot) * (w->max_req + 1 + kHostGroups);
    ok = ok && cudaEventSynchronize(w->ev_offsets[slot]) == cudaSuccess;
    size_t k = 0;
    size_t group_off[kHostGroups];
    for (int g = 0; g < n_groups; ++g) {
      group_off[g] = k;
      for (int32_t q = first[g]; q <= first[g + 1]; ++q) h_off[k++] = cand_offsets[q] - cand_offsets[first[g]];
    }
    // the copy stream starts behind everything already queued on the caller's stream (earlier calls may still
    // be reading the workspace)
    ok = ok && cudaEventRecord(w->ev_begin, st) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(w->copy_stream, w->ev_begin, 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(w->cand_offsets, h_off, k * 8, cudaMemcpyHostToDevice, w->copy_stream) == cudaSuccess;
    ok = ok && cudaEventRecord(w->ev_offsets[slot], w->copy_stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(w->edge_offsets, edge_offsets, (n_req + 1) * 8, cudaMemcpyHostToDevice, w->copy_stream) == cudaSuccess;
    for (int g = 0; g < n_groups && ok; ++g) {
      const int32_t r0 = first[g], r1 = first[g + 1];
      const int64_t c0 = cand_offsets[r0], c1 = cand_offsets[r1], e0 = edge_offsets[r0], e1 = edge_offsets[r1];
      if (e1 > e0) {
        ok = ok && cudaMemcpyAsync(w->edge_keys + e0, edge_keys + e0, (e1 - e0) * 8, cudaMemcpyHostToDevice, w->copy_stream) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(w->edge_feats + e0 * w->edge_b, static_cast<const uint8_t*>(edge_feats) + e0 * w->edge_b,
                                   (e1 - e0) * w->edge_b, cudaMemcpyHostToDevice, w->copy_stream) == cudaSuccess;
      }
      if (c1 > c0)
        ok = ok && cudaMemcpyAsync(w->cand_idx + c0, cand_idx + c0, (c1 - c0) * 4, cudaMemcpyHostToDevice, w->copy_stream) == cudaSuccess;
      if (s->req_b > 0)
        ok = ok && cudaMemcpyAsync(w->req_feats + static_cast<size_t>(r0) * w->req_b,
                                   static_cast<const uint8_t*>(req_feats) + static_cast<size_t>(r0) * w->req_b,
                                   static_cast<size_t>(r1 - r0) * w->req_b, cudaMemcpyHostToDevice, w->copy_stream) == cudaSuccess;
      ok = ok && cudaEventRecord(w->ev_group[g], w->copy_stream) == cudaSuccess;
      ok = ok && cudaStreamWaitEvent(st, w->ev_group[g], 0) == cudaSuccess;
      if (!ok) break;
      if (c1 > c0) {
        const ccr_status js = ccr_join_batch(s, r1 - r0, c1 - c0, max_edge_len, w->edge_keys, w->edge_feats, w->edge_offsets + r0,
                                             w->cand_idx + c0, w->cand_offsets + group_off[g],
                                             s->req_b ? w->req_feats + static_cast<size_t>(r0) * w->req_b : nullptr,
                                             w->out_rows + static_cast<size_t>(c0) * out_b, w->out_mask + c0, flags, stream);
        if (js != CCR_OK) return js;
      }
    }
    if (!ok) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
  }
  if (out_rows != nullptr)  // NULL: the rows stay in the workspace for a consumer on the device (ccr_workspace_outputs)
    ok = ok && cudaMemcpyAsync(out_rows, w->out_rows, total_cands * out_b, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(out_mask, w->out_mask, total_cands, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return CCR_ERR_CUDA;
  }
  return CCR_OK;
}

// ---------------------------------------------------------------------------------------------------
// ccr_join_payload_static: the join for callers that must not allocate (declared in ccr.h).
//
// Everything the call needs beyond the caller's buffers lives in one fixed block of device memory that is
// part of the library image: the kernel's status and scheduling words and the device copy of the request
// payload.  In host code the array's name is only a stand-in for the device symbol, so its device address
// is looked up once per device with cudaGetSymbolAddress and that pointer is what kernels and copies get.
constexpr size_t kStaticScratchBytes = 16u << 20;  // 16 MiB, held by every GPU that loads the library
constexpr size_t kStaticControlBytes = 256;        // scheduling words in front of the payload
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
unsigned char* g_static_ptr[kMaxDevices] = {};
std::mutex g_static_mutex;

// Device address of the scratch block on `device` (which must be current); resolved on first use.
ccr_status static_scratch(int device, unsigned char** out) {
  if (device < 0 || device >= kMaxDevices) return CCR_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[device] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return CCR_ERR_CUDA;
    }
    g_static_ptr[device] = static_cast<unsigned char*>(p);
  }
  *out = g_static_ptr[device];
  return CCR_OK;
}

inline size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }
}  // namespace

size_t ccr_static_payload_capacity(void) { return kStaticScratchBytes - kStaticControlBytes; }

ccr_status ccr_join_payload_static(const ccr_docstore* s, int32_t n_req, int64_t total_cands, int64_t max_edge_len,
                                   int64_t total_edges, const int64_t* edge_keys, const void* edge_feats,
                                   const int64_t* edge_offsets, const int32_t* cand_idx, const int64_t* cand_offsets,
                                   const void* req_feats, void* out_rows, uint8_t* out_mask, uint32_t flags,
                                   void* stream) {
  if (!good(s)) return CCR_ERR_BAD_HANDLE;
  if (n_req < 0 || total_cands < 0 || total_edges < 0 || max_edge_len < 0) return CCR_ERR_INVALID_ARG;
  if (n_req == 0 || total_cands == 0) return (n_req == 0 && total_cands != 0) ? CCR_ERR_INVALID_ARG : CCR_OK;
  if (!edge_offsets || !cand_offsets || !cand_idx || !out_rows || !out_mask) return CCR_ERR_INVALID_ARG;
  if (total_edges > 0 && (!edge_keys || !edge_feats)) return CCR_ERR_INVALID_ARG;
  if (s->req_b > 0 && !req_feats) return CCR_ERR_INVALID_ARG;
  if (flags & CCR_FLAG_VALIDATE) return CCR_ERR_UNSUPPORTED;  // validation synchronises the stream
  if (flags & CCR_FLAG_COSINE) return CCR_ERR_INVALID_ARG;    // the member embeddings come through ccr_join_batch_ex
  // the offsets are host-readable here, so the scalars that size the copies are checked against them
  if (edge_offsets[0] < 0 || cand_offsets[0] != 0) return CCR_ERR_INVALID_ARG;
  for (int32_t r = 0; r < n_req; ++r) {
    if (edge_offsets[r + 1] < edge_offsets[r] || cand_offsets[r + 1] < cand_offsets[r]) return CCR_ERR_INVALID_ARG;
    if (edge_offsets[r + 1] - edge_offsets[r] > max_edge_len) return CCR_ERR_INVALID_ARG;
  }
  if (edge_offsets[n_req] > total_edges || cand_offsets[n_req] != total_cands) return CCR_ERR_INVALID_ARG;

  // device copy of the payload, every piece on a 256-byte boundary behind the control words
  const size_t n_off = static_cast<size_t>(n_req) + 1;
  const size_t sz_keys = static_cast<size_t>(total_edges) * 8, sz_feats = static_cast<size_t>(total_edges) * s->edge_b;
  const size_t sz_off = n_off * 8, sz_idx = static_cast<size_t>(total_cands) * 4;
  const size_t sz_req = static_cast<size_t>(n_req) * s->req_b;
  const size_t o_keys = kStaticControlBytes, o_feats = o_keys + round256(sz_keys), o_eo = o_feats + round256(sz_feats);
  const size_t o_idx = o_eo + round256(sz_off), o_co = o_idx + round256(sz_idx), o_req = o_co + round256(sz_off);
  const size_t need = o_req + round256(sz_req);
  if (need > kStaticScratchBytes) return CCR_ERR_UNSUPPORTED;  // payload larger than the fixed block

  DeviceScope scope(s->desc.device);
  if (!scope.ok) return CCR_ERR_CUDA;
  unsigned char* base = nullptr;
  const ccr_status rs = static_scratch(s->desc.device, &base);
  if (rs != CCR_OK) return rs;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool ok = cudaMemsetAsync(base, 0, kStaticControlBytes, st) == cudaSuccess;  // the words must start at zero
  if (total_edges > 0) {
    ok = ok && cudaMemcpyAsync(base + o_keys, edge_keys, sz_keys, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(base + o_feats, edge_feats, sz_feats, cudaMemcpyHostToDevice, st) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(base + o_eo, edge_offsets, sz_off, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(base + o_idx, cand_idx, sz_idx, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(base + o_co, cand_offsets, sz_off, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (sz_req > 0) ok = ok && cudaMemcpyAsync(base + o_req, req_feats, sz_req, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return CCR_ERR_CUDA;
  }
  // The kernel's scheduling words are the ones at the head of the fixed block; its status word stays the store's
  // own (allocated when the store was created), so a bounded wait that runs out in this launch is reported by
  // ccr_docstore_device_status like any other.
  const ccr_status js = join_impl(s, n_req, total_cands, max_edge_len, reinterpret_cast<const int64_t*>(base + o_keys),
                                  base + o_feats, reinterpret_cast<const int64_t*>(base + o_eo),
                                  reinterpret_cast<const int32_t*>(base + o_idx),
                                  reinterpret_cast<const int64_t*>(base + o_co), s->req_b > 0 ? base + o_req : nullptr,
                                  out_rows, out_mask, flags, stream, 0, nullptr, reinterpret_cast<int*>(base));
  return js;
}

}  // extern "C"
