// Algorithm 1 step 1 of the paper on the device: per request, sort the viewer's affinity records by author
// id (a_sorted, idx = sort(a); F_sorted = gather(F, idx)) so that unsorted request payloads can be joined.
//
// One 1024-thread block per request.  Keys and record indices are sorted together in shared memory with a
// bitonic network written for arbitrary n (flip + disperse steps, every compare-exchange ascending, partners
// beyond n skipped — equivalent to padding with +infinity); the order is on (key, index), which makes the
// result the stable sort.  Keys that leave room for the index in the same 64-bit word (the usual case) take 8
// bytes per record, so lists of up to ~29,000 records are sorted in shared memory; other keys take 12 bytes
// (~19,000 records).  Longer lists are sorted by the same network directly on the output arrays in global memory (L2).  The rows then follow their keys in 16-byte chunks.
#pragma once

#include "ccr_device.cuh"

namespace ccr {

constexpr int kSortThreads = 1024;
constexpr int kSortSmemMaxKeys = 19000;  // 12 bytes per record (int64 key + int32 index) within 227 KB

// One pass structure for both element types: for partner mask j, the pairs (i, i ^ j) with i < i ^ j are
// exactly the i whose bit `top(j)` is clear; pair number p (0 .. n/2) maps to i by inserting a zero there.
__device__ __forceinline__ int pair_low_index(int p, int top_bit) {
  const int low = p & ((1 << top_bit) - 1);
  return ((p >> top_bit) << (top_bit + 1)) | low;
}

// (key, index) records in two arrays, ordered by key then index.
__device__ __forceinline__ void sort_pairs_bitonic(long long* keys, int* idx, int n) {
  if (n < 2) return;
  for (int k = 2;; k <<= 1) {
    // flip: i pairs with its mirror inside the block of k; then disperse at distances k/4, k/8, ..., 1
    for (int j = k - 1;;) {
      const int top = 31 - __clz(j);
      for (int p = threadIdx.x;; p += blockDim.x) {
        const int i = pair_low_index(p, top), l = i ^ j;
        if (i >= n) break;  // i grows with p
        if (l < n) {
          const long long ki = keys[i], kl = keys[l];
          const int ii = idx[i], il = idx[l];
          if (ki > kl || (ki == kl && ii > il)) {
            keys[i] = kl;
            keys[l] = ki;
            idx[i] = il;
            idx[l] = ii;
          }
        }
      }
      __syncthreads();
      if (j == k - 1) j = k >> 2; else j >>= 1;
      if (j == 0) break;
    }
    if (k >= n) break;
  }
}

// M consecutive disperse steps of the network (partner distances 2^b, 2^(b-1), ..., 2^(b-M+1)) in one pass:
// the 2^M elements whose indices differ only in those M bits form a closed group, so a thread loads the group,
// runs the M rounds of compare-exchanges in registers and stores it — one barrier and one trip through shared
// memory instead of M.  Elements at or beyond n count as +infinity (every real word is below 2^63).
template <int M>
__device__ __forceinline__ void disperse_fused(unsigned long long* w, int n, int b) {
  const int sh = b - M + 1;
  for (int g = threadIdx.x;; g += blockDim.x) {
    const int base = ((g >> sh) << (b + 1)) | (g & ((1 << sh) - 1));
    if (base >= n) break;  // base grows with g
    unsigned long long v[1 << M];
#pragma unroll
    for (int m = 0; m < (1 << M); ++m) {
      const int i = base + (m << sh);
      v[m] = i < n ? w[i] : ~0ull;
    }
#pragma unroll
    for (int s = M - 1; s >= 0; --s) {
#pragma unroll
      for (int m = 0; m < (1 << M); ++m) {
        if ((m & (1 << s)) == 0) {
          const int p = m | (1 << s);
          const unsigned long long lo = min(v[m], v[p]), hi = max(v[m], v[p]);
          v[m] = lo;
          v[p] = hi;
        }
      }
    }
#pragma unroll
    for (int m = 0; m < (1 << M); ++m) {
      const int i = base + (m << sh);
      if (i < n) w[i] = v[m];
    }
  }
  __syncthreads();
}

// Every step whose partner distance is below 32 stays inside 32 consecutive elements, so a warp holding one
// element per lane runs those steps with shuffles: no shared-memory traffic, no bank conflicts, no barriers.
// FIRST: the whole network up to blocks of 32 (flip and disperse steps of k = 2 .. 32); otherwise the last five
// disperse steps (distances 16 .. 1) of a larger block.  The lane with the lower index keeps the minimum.
template <bool FIRST>
__device__ __forceinline__ void warp_steps(unsigned long long* w, int n) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int c = warp; c * 32 < n; c += n_warps) {
    const int i = c * 32 + lane;
    unsigned long long v = i < n ? w[i] : ~0ull;
    if (FIRST) {
#pragma unroll
      for (int L = 1; L <= 5; ++L) {
        const unsigned long long pf = __shfl_xor_sync(0xffffffffu, v, (1 << L) - 1);  // flip: mirror inside the block
        v = (lane & (1 << (L - 1))) == 0 ? min(v, pf) : max(v, pf);
#pragma unroll
        for (int d = (1 << L) >> 2; d >= 1; d >>= 1) {
          const unsigned long long pv = __shfl_xor_sync(0xffffffffu, v, d);
          v = (lane & d) == 0 ? min(v, pv) : max(v, pv);
        }
      }
    } else {
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) {
        const unsigned long long pv = __shfl_xor_sync(0xffffffffu, v, d);
        v = (lane & d) == 0 ? min(v, pv) : max(v, pv);
      }
    }
    if (i < n) w[i] = v;
  }
  __syncthreads();
}

// The same network on single 64-bit words (key << shift | index): half the shared-memory traffic; steps at
// distances below 32 run in registers (warp_steps), the others are fused up to three at a time
// (disperse_fused, always at strides of 32 words or more, which keeps them free of bank conflicts).
__device__ __forceinline__ void sort_words_bitonic(unsigned long long* w, int n) {
  if (n < 2) return;
  warp_steps<true>(w, n);  // blocks of 32 are sorted
  for (int k = 64, log_k = 6; (k >> 1) < n; k <<= 1, ++log_k) {
    {  // flip: i pairs with its mirror inside the block of k
      const int j = k - 1, top = log_k - 1;
      for (int p = threadIdx.x;; p += blockDim.x) {
        const int i = pair_low_index(p, top), l = i ^ j;
        if (i >= n) break;  // i grows with p
        if (l < n) {
          const unsigned long long wi = w[i], wl = w[l];
          if (wi > wl) {
            w[i] = wl;
            w[l] = wi;
          }
        }
      }
      __syncthreads();
    }
    // disperse at distances k/4 ... 32 in shared memory, 16 ... 1 in registers
    for (int b = log_k - 2; b >= 5;) {
      const int m = b - 4 >= 3 ? 3 : b - 4;
      if (m == 3) disperse_fused<3>(w, n, b);
      else if (m == 2) disperse_fused<2>(w, n, b);
      else disperse_fused<1>(w, n, b);
      b -= m;
    }
    warp_steps<false>(w, n);
  }
}

// Rows follow their keys: output chunk c (16 bytes) comes from row source_of(c / row_ch) of the input.  One block
// moves a whole list, so every thread keeps kSortGatherUnroll loads in flight.
constexpr int kSortGatherUnroll = 8;
template <typename SourceOf>
__device__ __forceinline__ void gather_rows(const uint4* src, uint4* dst, long long chunks, int row_ch, SourceOf source_of) {
  for (long long c0 = threadIdx.x; c0 < chunks; c0 += static_cast<long long>(blockDim.x) * kSortGatherUnroll) {
    uint4 v[kSortGatherUnroll];
#pragma unroll
    for (int u = 0; u < kSortGatherUnroll; ++u) {
      const long long c = c0 + static_cast<long long>(u) * blockDim.x;
      if (c < chunks) {
        const int row = static_cast<int>(c / row_ch), piece = static_cast<int>(c - static_cast<long long>(row) * row_ch);
        v[u] = __ldg(src + source_of(row) * row_ch + piece);
      }
    }
#pragma unroll
    for (int u = 0; u < kSortGatherUnroll; ++u) {
      const long long c = c0 + static_cast<long long>(u) * blockDim.x;
      if (c < chunks) dst[c] = v[u];
    }
  }
}

struct SortArgs {
  int more_follow;           // another kernel of the same ccr_sort_edges call is launched behind this one
  int n_req;
  const int64_t* keys_in;
  const uint8_t* feats_in;
  const int64_t* edge_offsets;
  int row_ch;            // 16-byte chunks per feature row
  int64_t* keys_out;
  uint8_t* feats_out;
  int* perm_out;         // may be null when every list fits shared memory
  int smem_keys;         // (key, index) records the dynamic shared memory can hold: 12 bytes each
  int smem_words;        // packed key|index words it can hold: 8 bytes each
  int max_len;           // the host's bound on the list length: longer lists are cut there (their tail is left alone)
  int multi;             // 1: packable lists longer than kSortChunk are sorted by the multi-block kernels, and the
                         //    rows of every list are moved by gather_all_kernel (perm_out is then required)
};

constexpr int kSortChunkLog = 12;
constexpr int kSortChunk = 1 << kSortChunkLog;  // records one block of the multi-block path sorts in shared memory
constexpr int kSortMultiBalance = 64;  // long lists are spread over blocks while their total length is at most this many times the longest
constexpr int kSortMultiFlag = 0x5a17ed01;      // "this list is on the multi-block path", kept in the list's first output row

__device__ __forceinline__ int sort_index_bits(int K) {
  int idx_bits = 1;
  while ((1 << idx_bits) < K) ++idx_bits;
  return idx_bits;
}

// Block-wide: do the K keys leave room for the record index in one 64-bit word (non-negative, below
// 2^(63 - idx_bits))?  All threads of the block must call.
__device__ __forceinline__ bool list_is_packable(const int64_t* keys, int K, int idx_bits) {
  long long kmax = 0;
  int negative = 0;
  for (int i = threadIdx.x; i < K; i += blockDim.x) {
    const long long k = __ldg(keys + i);
    kmax = max(kmax, k);
    negative |= (k < 0);
  }
  return __syncthreads_or(negative || (kmax >> (63 - idx_bits)) != 0) == 0;
}

__global__ void __launch_bounds__(kSortThreads, 1) sort_edges_kernel(const SortArgs a) {
  chain_enter(a.more_follow != 0);
  extern __shared__ __align__(16) unsigned char smem_sort[];
  const int r = blockIdx.x;
  const long long e0 = __ldg(a.edge_offsets + r);
  const long long Kl = min(static_cast<long long>(__ldg(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len));
  if (Kl <= 0) return;
  const int K = static_cast<int>(Kl);
  // keys that leave room for the record index in one 64-bit word (non-negative, below 2^(63 - index bits)) are
  // sorted as single words: key << shift | index orders like (key, index), needs 8 bytes per record and no
  // index array at all (the word's low bits are the index)
  if (a.multi && *reinterpret_cast<const volatile int*>(a.feats_out + e0 * a.row_ch * 16) == kSortMultiFlag)
    return;  // the chunked kernels have sorted this list
  const int idx_bits = sort_index_bits(K);
  const bool packable = list_is_packable(a.keys_in + e0, K, idx_bits);
  const long long chunks = a.multi ? 0 : static_cast<long long>(K) * a.row_ch;  // multi: rows move in gather_all_kernel
  const uint4* src = reinterpret_cast<const uint4*>(a.feats_in) + e0 * a.row_ch;
  uint4* dst = reinterpret_cast<uint4*>(a.feats_out) + e0 * a.row_ch;

  if (packable && K <= a.smem_words) {
    unsigned long long* w = reinterpret_cast<unsigned long long*>(smem_sort);
    for (int i = threadIdx.x; i < K; i += blockDim.x)
      w[i] = (static_cast<unsigned long long>(__ldg(a.keys_in + e0 + i)) << idx_bits) | static_cast<unsigned>(i);
    __syncthreads();
    sort_words_bitonic(w, K);
    const unsigned long long low = (1ull << idx_bits) - 1;
    for (int i = threadIdx.x; i < K; i += blockDim.x) {
      const unsigned long long v = w[i];
      a.keys_out[e0 + i] = static_cast<long long>(v >> idx_bits);
      if (a.perm_out) a.perm_out[e0 + i] = static_cast<int>(v & low);
    }
    gather_rows(src, dst, chunks, a.row_ch, [&](int row) { return static_cast<long long>(w[row] & low); });
    return;
  }

  const bool in_smem = K <= a.smem_keys;
  if (!in_smem && a.perm_out == nullptr) return;  // refused on the host; never reached
  long long* keys = in_smem ? reinterpret_cast<long long*>(smem_sort) : reinterpret_cast<long long*>(a.keys_out + e0);
  int* idx = in_smem ? reinterpret_cast<int*>(smem_sort + static_cast<size_t>(a.smem_keys) * 8) : a.perm_out + e0;
  if (packable) {  // only reached by lists too long for shared memory: the words live in the key output array
    unsigned long long* w = reinterpret_cast<unsigned long long*>(keys);
    for (int i = threadIdx.x; i < K; i += blockDim.x)
      w[i] = (static_cast<unsigned long long>(__ldg(a.keys_in + e0 + i)) << idx_bits) | static_cast<unsigned>(i);
    __syncthreads();
    sort_words_bitonic(w, K);
    const unsigned long long low = (1ull << idx_bits) - 1;
    for (int i = threadIdx.x; i < K; i += blockDim.x) {  // unpack; each thread rewrites only its own slots
      const unsigned long long v = w[i];
      idx[i] = static_cast<int>(v & low);
      keys[i] = static_cast<long long>(v >> idx_bits);
    }
    __syncthreads();
  } else {
    for (int i = threadIdx.x; i < K; i += blockDim.x) {
      keys[i] = __ldg(a.keys_in + e0 + i);
      idx[i] = i;
    }
    __syncthreads();
    sort_pairs_bitonic(keys, idx, K);
  }
  if (in_smem) {
    for (int i = threadIdx.x; i < K; i += blockDim.x) {
      a.keys_out[e0 + i] = keys[i];
      if (a.perm_out) a.perm_out[e0 + i] = idx[i];
    }
  }
  gather_rows(src, dst, chunks, a.row_ch, [&](int row) { return static_cast<long long>(idx[row]); });
}


// ---------------------------------------------------------------------------------------------------
// Multi-block path for long lists.  One block per list leaves a 19,000-record list to a single SM (264 us,
// instruction-bound) while the others idle.  Here the same network runs over the packed words in global
// memory (the key output array): chunks of kSortChunk records are sorted in shared memory by one block each;
// then, for every larger block size k, the steps whose partner distance reaches across chunks (the flip, and
// disperse steps at distances >= kSortChunk) run as grid-wide passes, one launch each, and the remaining steps
// of the phase run per chunk in shared memory again.  A flag in the list's first output row (written by the
// chunk kernel, overwritten by the final row gather) tells the later kernels that the list is packable.

__device__ __forceinline__ bool list_on_multi_path(const SortArgs& a, int r, long long& e0, int& K) {
  e0 = __ldg(a.edge_offsets + r);
  const long long Kl = min(static_cast<long long>(__ldg(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len));
  K = Kl > 0 ? static_cast<int>(Kl) : 0;
  if (K == 0) return false;
  return *reinterpret_cast<const volatile int*>(a.feats_out + e0 * a.row_ch * 16) == kSortMultiFlag;
}

// grid (n_req, chunks of the longest list): sort chunk blockIdx.y of list blockIdx.x
__global__ void __launch_bounds__(kSortThreads, 1) sort_chunks_kernel(const SortArgs a) {
  chain_enter(a.more_follow != 0);
  __shared__ unsigned long long w[kSortChunk];
  const int r = blockIdx.x;
  const long long e0 = __ldg(a.edge_offsets + r);
  const int K = static_cast<int>(min(static_cast<long long>(__ldg(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len)));
  const int c0 = blockIdx.y * kSortChunk;
  if (c0 >= K) return;  // also K <= 0
  const int idx_bits = sort_index_bits(K);
  bool take = list_is_packable(a.keys_in + e0, K, idx_bits);
  if (K > kSortChunk) {
    // Spreading a long list over many blocks costs more SM time than sorting it in one block, so it pays only
    // while the batch's long lists would not keep the SMs busy one list each.
    // every block sizes up the batch's long lists for itself (the same numbers in all of them): their total
    // length against the longest one — one block per list takes about 14 ns per record of the longest list,
    // the chunked path about 0.2 ns per record of all long lists (measured)
    __shared__ unsigned long long sum_long_s;
    __shared__ int max_long_s;
    if (threadIdx.x == 0) {
      sum_long_s = 0;
      max_long_s = 0;
    }
    __syncthreads();
    unsigned long long sum = 0;
    int longest = 0;
    for (int q = threadIdx.x; q < a.n_req; q += blockDim.x) {
      const long long len = min(static_cast<long long>(__ldg(a.edge_offsets + q + 1) - __ldg(a.edge_offsets + q)), static_cast<long long>(a.max_len));
      if (len > kSortChunk) {
        sum += static_cast<unsigned long long>(len);
        longest = max(longest, static_cast<int>(min(len, 0x7fffffffLL)));
      }
    }
    if (sum) {
      atomicAdd(&sum_long_s, sum);
      atomicMax(&max_long_s, longest);
    }
    __syncthreads();
    take = take && sum_long_s <= static_cast<unsigned long long>(kSortMultiBalance) * max_long_s;
  }
  if (blockIdx.y == 0 && threadIdx.x == 0)
    *reinterpret_cast<int*>(a.feats_out + e0 * a.row_ch * 16) = take ? kSortMultiFlag : 0;
  if (!take) return;
  const int n = min(kSortChunk, K - c0);
  for (int t = threadIdx.x; t < n; t += blockDim.x)
    w[t] = (static_cast<unsigned long long>(__ldg(a.keys_in + e0 + c0 + t)) << idx_bits) | static_cast<unsigned>(c0 + t);
  __syncthreads();
  sort_words_bitonic(w, n);
  unsigned long long* W = reinterpret_cast<unsigned long long*>(a.keys_out + e0);
  for (int t = threadIdx.x; t < n; t += blockDim.x) W[c0 + t] = w[t];
}

// grid (n_req, pair blocks): one step of the network across chunks — partner mask j = k - 1 (flip) or a
// power of two >= kSortChunk (disperse) — for the lists that have a block of size k to sort.
constexpr int kSortPairsPerThread = 4;
__global__ void __launch_bounds__(kSortThreads) sort_global_step_kernel(const SortArgs a, int k, int j) {
  chain_enter(a.more_follow != 0);
  long long e0;
  int K;
  if (!list_on_multi_path(a, blockIdx.x, e0, K) || (k >> 1) >= K) return;
  unsigned long long* W = reinterpret_cast<unsigned long long*>(a.keys_out + e0);
  const int top = 31 - __clz(j);
#pragma unroll
  for (int u = 0; u < kSortPairsPerThread; ++u) {
    const int p = (blockIdx.y * kSortPairsPerThread + u) * kSortThreads + threadIdx.x;
    const int i = pair_low_index(p, top), l = i ^ j;
    if (i < K && l < K) {
      const unsigned long long wi = W[i], wl = W[l];
      if (wi > wl) {
        W[i] = wl;
        W[l] = wi;
      }
    }
  }
}

// grid (n_req, chunks): the disperse steps at distances kSortChunk / 2 ... 1 of phase k, per chunk in shared memory
__global__ void __launch_bounds__(kSortThreads, 1) sort_chunk_finish_kernel(const SortArgs a, int k) {
  chain_enter(a.more_follow != 0);
  __shared__ unsigned long long w[kSortChunk];
  long long e0;
  int K;
  const int c0 = blockIdx.y * kSortChunk;
  if (!list_on_multi_path(a, blockIdx.x, e0, K) || (k >> 1) >= K || c0 >= K) return;
  unsigned long long* W = reinterpret_cast<unsigned long long*>(a.keys_out + e0);
  const int n = min(kSortChunk, K - c0);
  for (int t = threadIdx.x; t < n; t += blockDim.x) w[t] = W[c0 + t];
  __syncthreads();
  for (int b = kSortChunkLog - 1; b >= 5;) {
    const int m = b - 4 >= 3 ? 3 : b - 4;
    if (m == 3) disperse_fused<3>(w, n, b);
    else if (m == 2) disperse_fused<2>(w, n, b);
    else disperse_fused<1>(w, n, b);
    b -= m;
  }
  warp_steps<false>(w, n);
  for (int t = threadIdx.x; t < n; t += blockDim.x) W[c0 + t] = w[t];
}

// grid (n_req, chunks): words -> keys (in place) and source indices
__global__ void __launch_bounds__(kSortThreads) sort_unpack_kernel(const SortArgs a) {
  chain_enter(a.more_follow != 0);
  long long e0;
  int K;
  const int c0 = blockIdx.y * kSortChunk;
  if (!list_on_multi_path(a, blockIdx.x, e0, K) || c0 >= K) return;
  const int idx_bits = sort_index_bits(K);
  const unsigned long long low = (1ull << idx_bits) - 1;
  const int n = min(kSortChunk, K - c0);
  for (int t = threadIdx.x; t < n; t += blockDim.x) {
    const unsigned long long v = reinterpret_cast<const unsigned long long*>(a.keys_out + e0)[c0 + t];
    a.keys_out[e0 + c0 + t] = static_cast<long long>(v >> idx_bits);
    a.perm_out[e0 + c0 + t] = static_cast<int>(v & low);
  }
}

// grid (n_req, row blocks): rows follow their keys, for every list of the batch, kSortGatherUnroll 16-byte chunks
// per thread in flight
__global__ void __launch_bounds__(kSortThreads) gather_all_kernel(const SortArgs a) {
  chain_enter(a.more_follow != 0);
  const int r = blockIdx.x;
  const long long e0 = __ldg(a.edge_offsets + r);
  const long long K = min(static_cast<long long>(__ldg(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len));
  const long long chunks = K * a.row_ch;
  const long long first = static_cast<long long>(blockIdx.y) * kSortThreads * kSortGatherUnroll;
  if (first >= chunks) return;
  const uint4* src = reinterpret_cast<const uint4*>(a.feats_in) + e0 * a.row_ch;
  uint4* dst = reinterpret_cast<uint4*>(a.feats_out) + e0 * a.row_ch;
  const int* perm = a.perm_out + e0;
  uint4 v[kSortGatherUnroll];
#pragma unroll
  for (int u = 0; u < kSortGatherUnroll; ++u) {
    const long long c = first + static_cast<long long>(u) * kSortThreads + threadIdx.x;
    if (c < chunks) {
      const int row = static_cast<int>(c / a.row_ch), piece = static_cast<int>(c - static_cast<long long>(row) * a.row_ch);
      v[u] = __ldg(src + static_cast<long long>(__ldg(perm + row)) * a.row_ch + piece);
    }
  }
#pragma unroll
  for (int u = 0; u < kSortGatherUnroll; ++u) {
    const long long c = first + static_cast<long long>(u) * kSortThreads + threadIdx.x;
    if (c < chunks) dst[c] = v[u];
  }
}

}  // namespace ccr
