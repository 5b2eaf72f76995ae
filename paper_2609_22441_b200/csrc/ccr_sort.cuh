// Algorithm 1 step 1 of the paper on the device: per request, sort the viewer's affinity records by author
// id (a_sorted, idx = sort(a); F_sorted = gather(F, idx)) so that unsorted request payloads can be joined.
//
// The order is on (key, index of the record in its list), which makes the result the stable sort.  Keys that leave
// room for the index in the same 64-bit word (the usual case) are sorted as single words, key << bits | index.
// With a permutation output the lists are cut into chunks of 4,096 records, one block sorts a chunk in shared
// memory (a merge sort: four words per thread in registers, then runs doubled per pass along merge paths), the
// sorted chunks are merged pairwise by grid-wide launches (merge path again, one output tile per block), and the
// rows follow their keys in one grid-wide gather.  Without a permutation output, or for keys that do not leave
// room for the index, one 1024-thread block sorts a whole list in shared memory (merge sort up to 16,384 packed
// words, a bitonic network written for arbitrary n beyond that and for the 12-byte (key, index) records of
// unpackable keys; lists that do not fit shared memory are sorted by the network on the output arrays in L2) and
// moves its rows itself.
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

// Merge passes over sorted runs of `run` words in shared memory (n <= IPT * blockDim.x distinct words): runs are
// merged pairwise, doubling per pass; in a pass a thread produces IPT consecutive output words, from the point of
// its pair of runs that the merge path (a binary search along its diagonal) assigns to it, into registers, and
// writes them back after a barrier.  Two barriers per pass.
template <int IPT>
__device__ __forceinline__ void merge_passes(unsigned long long* w, int n, int run) {
  const int t0 = static_cast<int>(threadIdx.x) * IPT;
  unsigned long long v[IPT];
  for (; run < n; run <<= 1) {
    const int pb = (t0 / (2 * run)) * (2 * run);
    const int lenA = max(0, min(run, n - pb)), lenB = max(0, min(run, n - pb - run));
    const unsigned long long* A = w + pb;
    const unsigned long long* B = A + run;
    const int d = min(t0 - pb, lenA + lenB);
    int lo = max(0, d - lenB), hi = min(d, lenA);
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (A[mid] < B[d - 1 - mid]) lo = mid + 1; else hi = mid;
    }
    int i = lo, j = d - lo;
#pragma unroll
    for (int u = 0; u < IPT; ++u) {
      const bool has_a = i < lenA, has_b = j < lenB;
      const unsigned long long va = has_a ? A[i] : ~0ull, vb = has_b ? B[j] : ~0ull;
      const bool take_a = has_a && (!has_b || va < vb);
      v[u] = take_a ? va : vb;
      i += take_a ? 1 : 0;
      j += take_a ? 0 : 1;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < IPT; ++u)
      if (t0 + u < n) w[t0 + u] = v[u];
    __syncthreads();
  }
}

// Merge sort of n <= IPT * blockDim.x distinct words in shared memory: every thread sorts IPT consecutive words in
// registers (odd-even transposition), then log2(n / IPT) merge passes.
template <int IPT>
__device__ __forceinline__ void sort_words_merge(unsigned long long* w, int n) {
  const int t0 = static_cast<int>(threadIdx.x) * IPT;
  unsigned long long v[IPT];
#pragma unroll
  for (int u = 0; u < IPT; ++u) v[u] = t0 + u < n ? w[t0 + u] : ~0ull;
#pragma unroll
  for (int rd = 0; rd < IPT; ++rd) {
#pragma unroll
    for (int u = rd & 1; u + 1 < IPT; u += 2) {
      const unsigned long long lo = min(v[u], v[u + 1]), hi = max(v[u], v[u + 1]);
      v[u] = lo;
      v[u + 1] = hi;
    }
  }
#pragma unroll
  for (int u = 0; u < IPT; ++u)
    if (t0 + u < n) w[t0 + u] = v[u];
  __syncthreads();
  merge_passes<IPT>(w, n, IPT);
}

// The same for n <= 4 * blockDim.x with the first seven doublings in registers: a warp holds 128 consecutive words,
// lane-strided (word e in register e / 32 of lane e % 32, so its loads and stores are to consecutive words), and
// sorts them with a bitonic network whose steps at distances 32 and 64 pair registers of one lane and the others
// lanes (shuffles): no shared memory, no barriers.  Measured per 4,096-word chunk (two blocks resident per SM):
// 8 us for this start + 13 us for the five merge passes behind it, against 30 us for ten merge passes from runs of
// four, and 23 us with the merge passes done warp-wise on strided registers as well (bitonic merges of 128).
template <int J, typename Up>
__device__ __forceinline__ void warp128_step(unsigned long long (&v)[4], int lane, Up up) {
  if constexpr (J >= 32) {
    constexpr int dr = J >> 5;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      if ((r & dr) == 0) {
        const unsigned long long lo = min(v[r], v[r | dr]), hi = max(v[r], v[r | dr]);
        const bool u = up((r << 5) | lane);  // the pair holding word e goes in ascending order
        v[r] = u ? lo : hi;
        v[r | dr] = u ? hi : lo;
      }
    }
  } else {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const unsigned long long pv = __shfl_xor_sync(0xffffffffu, v[r], J);
      const bool keep_min = ((lane & J) == 0) == up((r << 5) | lane);
      v[r] = keep_min ? min(v[r], pv) : max(v[r], pv);
    }
  }
}
// the steps of one block size K of the network: partner distances K/2 ... 1
template <int K, typename Up>
__device__ __forceinline__ void warp128_block(unsigned long long (&v)[4], int lane, Up up) {
  if constexpr (K >= 128) warp128_step<64>(v, lane, up);
  if constexpr (K >= 64) warp128_step<32>(v, lane, up);
  if constexpr (K >= 32) warp128_step<16>(v, lane, up);
  if constexpr (K >= 16) warp128_step<8>(v, lane, up);
  if constexpr (K >= 8) warp128_step<4>(v, lane, up);
  if constexpr (K >= 4) warp128_step<2>(v, lane, up);
  warp128_step<1>(v, lane, up);
}
__device__ __forceinline__ void sort_words_merge128(unsigned long long* w, int n) {
  const int lane = threadIdx.x & 31, o = (static_cast<int>(threadIdx.x) >> 5) * 128;
  unsigned long long v[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = o + (r << 5) + lane;
    v[r] = i < n ? w[i] : ~0ull;  // padding sorts last
  }
  // blocks of K words alternate in direction until the last, which is ascending
  warp128_block<2>(v, lane, [](int e) { return (e & 2) == 0; });
  warp128_block<4>(v, lane, [](int e) { return (e & 4) == 0; });
  warp128_block<8>(v, lane, [](int e) { return (e & 8) == 0; });
  warp128_block<16>(v, lane, [](int e) { return (e & 16) == 0; });
  warp128_block<32>(v, lane, [](int e) { return (e & 32) == 0; });
  warp128_block<64>(v, lane, [](int e) { return (e & 64) == 0; });
  warp128_block<128>(v, lane, [](int) { return true; });
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = o + (r << 5) + lane;
    if (i < n) w[i] = v[r];
  }
  __syncthreads();
  merge_passes<4>(w, n, 128);
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
        v[u] = ldg128(src + source_of(row) * row_ch + piece);
      }
    }
#pragma unroll
    for (int u = 0; u < kSortGatherUnroll; ++u) {
      const long long c = c0 + static_cast<long long>(u) * blockDim.x;
      if (c < chunks) st128_stream(dst + c, v[u]);
    }
  }
}

struct SortArgs {
  int* call_flag;          // multi: device word, zero between calls; set when a key of the batch cannot share a word with its index
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
  int multi;             // 1: the chunked kernels sort every list (sort_edges_kernel only when a key of the batch cannot be
                         //    packed), and the rows of every list are moved by gather_all_kernel (perm_out is then required)
};

#ifndef CCR_SORT_CHUNK_LOG
#define CCR_SORT_CHUNK_LOG 12
#endif
#ifndef CCR_SORT_CHUNK_THREADS
#define CCR_SORT_CHUNK_THREADS 1024
#endif
#ifndef CCR_SORT_CHUNK_BLOCKS
#define CCR_SORT_CHUNK_BLOCKS 2  // resident per SM: one block's loads hide behind the other's merging (32 registers, no spill)
#endif
constexpr int kSortChunkLog = CCR_SORT_CHUNK_LOG;
constexpr int kSortChunk = 1 << kSortChunkLog;  // records one block of the multi-block path sorts in shared memory
constexpr int kSortChunkThreads = CCR_SORT_CHUNK_THREADS;

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
#pragma unroll 8
  for (int i = threadIdx.x; i < K; i += blockDim.x) {
    const long long k = gload(keys + i);
    kmax = max(kmax, k);
    negative |= (k < 0);
  }
  return __syncthreads_or(negative || (kmax >> (63 - idx_bits)) != 0) == 0;
}

__global__ void __launch_bounds__(kSortThreads, 1) sort_edges_kernel(const SortArgs a) {
  chain_enter(a.more_follow != 0);
  extern __shared__ __align__(16) unsigned char smem_sort[];
  const int r = blockIdx.x;
  const long long e0 = gload(a.edge_offsets + r);
  const long long Kl = min(static_cast<long long>(gload(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len));
  if (Kl <= 0) return;
  const int K = static_cast<int>(Kl);
  // keys that leave room for the record index in one 64-bit word (non-negative, below 2^(63 - index bits)) are
  // sorted as single words: key << shift | index orders like (key, index), needs 8 bytes per record and no
  // index array at all (the word's low bits are the index)
  if (a.multi && gload(a.call_flag) == 0) return;  // the chunked kernels have sorted every list
  const int idx_bits = sort_index_bits(K);
  const bool packable = list_is_packable(a.keys_in + e0, K, idx_bits);
  const long long chunks = a.multi ? 0 : static_cast<long long>(K) * a.row_ch;  // multi: rows move in gather_all_kernel
  const uint4* src = reinterpret_cast<const uint4*>(a.feats_in) + e0 * a.row_ch;
  uint4* dst = reinterpret_cast<uint4*>(a.feats_out) + e0 * a.row_ch;

  if (packable && K <= a.smem_words) {
    unsigned long long* w = reinterpret_cast<unsigned long long*>(smem_sort);
    for (int i = threadIdx.x; i < K; i += blockDim.x)
      w[i] = (static_cast<unsigned long long>(gload(a.keys_in + e0 + i)) << idx_bits) | static_cast<unsigned>(i);
    __syncthreads();
    // merge sort while a thread's share of the list fits its registers, the network beyond
    if (K <= 4 * kSortThreads) sort_words_merge128(w, K);
    else if (K <= 8 * kSortThreads) sort_words_merge<8>(w, K);
    else if (K <= 16 * kSortThreads) sort_words_merge<16>(w, K);
    else sort_words_bitonic(w, K);
    const unsigned long long low = (1ull << idx_bits) - 1;
    for (int i = threadIdx.x; i < K; i += blockDim.x) {
      const unsigned long long v = w[i];
      gstore(a.keys_out + e0 + i, v >> idx_bits);
      if (a.perm_out) gstore(a.perm_out + e0 + i, v & low);
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
      w[i] = (static_cast<unsigned long long>(gload(a.keys_in + e0 + i)) << idx_bits) | static_cast<unsigned>(i);
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
      keys[i] = gload(a.keys_in + e0 + i);
      idx[i] = i;
    }
    __syncthreads();
    sort_pairs_bitonic(keys, idx, K);
  }
  if (in_smem) {
    for (int i = threadIdx.x; i < K; i += blockDim.x) {
      gstore(a.keys_out + e0 + i, keys[i]);
      if (a.perm_out) gstore(a.perm_out + e0 + i, idx[i]);
    }
  }
  gather_rows(src, dst, chunks, a.row_ch, [&](int row) { return static_cast<long long>(idx[row]); });
}


// ---------------------------------------------------------------------------------------------------
// Multi-block path.  One block per list leaves a 19,000-record list to a single SM while the others idle.  Here
// chunks of kSortChunk records are sorted in shared memory by one block each (packed words) and the sorted chunks
// are then merged pairwise, one launch per doubling of the run length, every block producing kSortMergeTile
// consecutive output words from the two stretches of its pair of runs that the merge path assigns to them.
// Packing needs keys that leave room for the index (non-negative, below 2^(63 - index bits)).  Every chunk block
// checks the keys it loads; one that cannot be packed sets the call's flag word, and the batch is then sorted
// list by list by sort_edges_kernel instead (what the chunked kernels wrote is overwritten).  The row gather at the
// end of the call puts the word back to zero.

__device__ __forceinline__ bool list_on_multi_path(const SortArgs& a, int r, long long& e0, int& K) {
  e0 = gload(a.edge_offsets + r);
  const long long Kl = min(static_cast<long long>(gload(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len));
  K = Kl > 0 ? static_cast<int>(Kl) : 0;
  // (read-only in every kernel that tests it, so the load may be cached: ten thousand blocks reading one word
  // past L1 queue up at a single L2 slice — 15 us on a 256-list batch)
  return K > 0 && gload(a.call_flag) == 0;
}

// The grids of this path have one block per (list, tile of the longest list), either folded into x with lists
// varying fastest, or lists along x and tiles along y.  Either way the blocks that have work (every list has a
// first tile, few have a twentieth) come first and the ones that leave at once are the tail of the launch.  Which
// form a kernel gets is a measurement on a 256-list batch: the row gather was 9 us faster on the two-dimensional
// grid (it falls back to the folded one when a list has more tiles than a grid has rows), the chunk and merge kernels
// together 6 us faster on the folded one.
__device__ __forceinline__ void sort_block_item(const SortArgs& a, int& r, long long& y) {
  if (gridDim.y > 1) {
    r = static_cast<int>(blockIdx.x);
    y = blockIdx.y;
  } else {
    y = blockIdx.x / static_cast<unsigned>(a.n_req);
    r = static_cast<int>(blockIdx.x - static_cast<unsigned>(y) * static_cast<unsigned>(a.n_req));
  }
}

// Merging the sorted chunks.  Phase p = 1, 2, ... merges neighbouring runs of kSortChunk << (p - 1) words into
// runs of twice that length, out of place: the words alternate between the key output array and a scratch area
// inside the list's own output rows (8 bytes per record; a row has at least 16), which
// nothing else uses until the rows are gathered at the end.  A list takes part in a phase while it is longer than
// the phase's input runs, so a list of K records goes through P = sort_merge_phases(K) phases.  Its last phase
// writes keys and source indices instead of words (a single-chunk list gets them from the chunk kernel), and so
// that this never overwrites words another block still has to read, the last phase must read from the scratch
// area: phase p reads it when P - p is even, and the chunk kernel writes there when P is odd.
__device__ __host__ __forceinline__ int sort_merge_phases(long long K) {
  int p = 0;
  while ((static_cast<long long>(kSortChunk) << p) < K) ++p;
  return p;
}
__device__ __forceinline__ unsigned long long* sort_words_at(const SortArgs& a, long long e0, bool scratch) {
  return scratch ? reinterpret_cast<unsigned long long*>(a.feats_out + e0 * a.row_ch * 16)
                 : reinterpret_cast<unsigned long long*>(a.keys_out + e0);
}

// One block per chunk of kSortChunk records of a list: the chunk sorted in shared memory, as packed words
__global__ void __launch_bounds__(kSortChunkThreads, CCR_SORT_CHUNK_BLOCKS) sort_chunks_kernel(const SortArgs a) {
  chain_enter(a.more_follow != 0);
  __shared__ unsigned long long w[kSortChunk];
  int r;
  long long y;
  sort_block_item(a, r, y);
  const long long e0 = gload(a.edge_offsets + r);
  const int K = static_cast<int>(min(static_cast<long long>(gload(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len)));
  if (y * kSortChunk >= K) return;  // also K <= 0
  const int c0 = static_cast<int>(y) * kSortChunk;
  const int idx_bits = sort_index_bits(K);
  const int n = min(kSortChunk, K - c0);
  int bad = 0;
  for (int t = threadIdx.x; t < n; t += blockDim.x) {
    const long long k = gload(a.keys_in + e0 + c0 + t);
    bad |= (k < 0 || (k >> (63 - idx_bits)) != 0) ? 1 : 0;
    w[t] = (static_cast<unsigned long long>(k) << idx_bits) | static_cast<unsigned>(c0 + t);
  }
  if (__syncthreads_or(bad)) {  // a key that cannot share a word with its index: the batch goes to the one-block path
    if (threadIdx.x == 0) gatomic_or(a.call_flag, 1);
    return;
  }
  static_assert(kSortChunk == 4 * kSortChunkThreads, "a warp of a chunk block owns 128 words");
  sort_words_merge128(w, n);
  const int P = sort_merge_phases(K);
  if (P == 0) {  // the whole list: done
    const unsigned long long low = (1ull << idx_bits) - 1;
    for (int t = threadIdx.x; t < n; t += blockDim.x) {
      gstore(a.keys_out + e0 + t, w[t] >> idx_bits);
      gstore(a.perm_out + e0 + t, w[t] & low);
    }
    return;
  }
  unsigned long long* W = sort_words_at(a, e0, (P & 1) != 0);
  for (int t = threadIdx.x; t < n; t += blockDim.x) gstore(W + c0 + t, w[t]);
}

// Merge path, warp-cooperative: how many of the first d words of merge(A, B) come from A.  All words are distinct
// (the record index is part of the word).  A[i] is among the first d exactly when A[i] < B[d - 1 - i]; that holds for
// i below the answer and fails from it on, so the warp probes the last element of up to 32 equal sub-ranges at once
// and narrows the range by a factor of 32 per round trip to memory (three rounds for runs of 16,384).
__device__ __forceinline__ int merge_path_warp(const unsigned long long* A, int lenA, const unsigned long long* B, int lenB,
                                               int d, int lane) {
  int lo = max(0, d - lenB), hi = min(d, lenA);
  while (lo < hi) {
    const int span = hi - lo, s = (span + 31) >> 5;
    const int i = lo + lane * s + s - 1;
    const bool before = i < hi && gload(A + i) < gload(B + d - 1 - i);
    const int cnt = __popc(__ballot_sync(0xffffffffu, before));  // the predicate is monotone: the first cnt probes hold
    const int first_fail = lo + cnt * s + s - 1;                 // probe number cnt failed or lies beyond the range
    lo += cnt * s;
    hi = min(hi, first_fail);
  }
  return lo;
}

// One block per kSortMergeTile consecutive output words of phase `phase` of a list.  Small blocks, several per
// SM: the grid is sized for the longest list, and the blocks beyond the end of a shorter one leave after reading
// the offsets — side by side rather than one after the other.
constexpr int kSortMergeThreads = 256;
constexpr int kSortMergePerThread = 4;
constexpr int kSortMergeTile = kSortMergeThreads * kSortMergePerThread;
__global__ void __launch_bounds__(kSortMergeThreads) sort_merge_kernel(const SortArgs a, int phase) {
  chain_enter(a.more_follow != 0);
  __shared__ unsigned long long w[kSortMergeTile];
  __shared__ int split[2];
  long long e0, y;
  int K, r;
  sort_block_item(a, r, y);
  const long long run = static_cast<long long>(kSortChunk) << (phase - 1);
  if (!list_on_multi_path(a, r, e0, K) || run >= K || y * kSortMergeTile >= K) return;
  const int o0 = static_cast<int>(y) * kSortMergeTile;  // first output word of this block, within the list
  const int P = sort_merge_phases(K);
  const unsigned long long* src = sort_words_at(a, e0, ((P - phase) & 1) == 0);
  unsigned long long* dst = sort_words_at(a, e0, ((P - phase) & 1) != 0);
  const int pb = static_cast<int>((o0 / (2 * run)) * (2 * run));  // the pair of runs this block's words belong to
  const int lenA = static_cast<int>(min(run, static_cast<long long>(K - pb)));
  const int lenB = static_cast<int>(min(run, static_cast<long long>(K - pb - lenA)));
  const unsigned long long* A = src + pb;
  const unsigned long long* B = A + lenA;
  const int d0 = o0 - pb, d1 = min(d0 + kSortMergeTile, lenA + lenB);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < 2) {
    const int ia = merge_path_warp(A, lenA, B, lenB, warp == 0 ? d0 : d1, lane);
    if (lane == 0) split[warp] = ia;
  }
  __syncthreads();
  const int ia0 = split[0], ia1 = split[1], ib0 = d0 - ia0, ib1 = d1 - ia1;
  const int nA = ia1 - ia0, nB = ib1 - ib0, n = nA + nB;
  if (nA < 0 || nB < 0 || n > kSortMergeTile) return;  // only if the runs were not sorted: touch nothing out of range
  for (int t = threadIdx.x; t < n; t += kSortMergeThreads) w[t] = t < nA ? gload(A + ia0 + t) : gload(B + ib0 + t - nA);
  __syncthreads();
  // every thread merges kSortMergePerThread consecutive output words: its own split of the tile by binary search
  const unsigned long long* sa = w;
  const unsigned long long* sb = w + nA;
  const int d = min(static_cast<int>(threadIdx.x) * kSortMergePerThread, n);
  int lo = max(0, d - nB), hi = min(d, nA);
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (sa[mid] < sb[d - 1 - mid]) lo = mid + 1; else hi = mid;
  }
  int i = lo, j = d - lo;
  unsigned long long out[kSortMergePerThread];
#pragma unroll
  for (int u = 0; u < kSortMergePerThread; ++u) {
    const bool has_a = i < nA, has_b = j < nB;
    const unsigned long long va = has_a ? sa[i] : ~0ull, vb = has_b ? sb[j] : ~0ull;
    const bool take_a = has_a && (!has_b || va < vb);
    out[u] = take_a ? va : vb;
    i += take_a ? 1 : 0;
    j += take_a ? 0 : 1;
  }
  if (phase == P) {  // the list's last merge: keys and source indices (src is the scratch area here)
    const int idx_bits = sort_index_bits(K);
    const unsigned long long low = (1ull << idx_bits) - 1;
#pragma unroll
    for (int u = 0; u < kSortMergePerThread; ++u) {
      if (d + u < n) {
        gstore(a.keys_out + e0 + o0 + d + u, out[u] >> idx_bits);
        gstore(a.perm_out + e0 + o0 + d + u, out[u] & low);
      }
    }
    return;
  }
#pragma unroll
  for (int u = 0; u < kSortMergePerThread; ++u)
    if (d + u < n) gstore(dst + o0 + d + u, out[u]);
}

// One block per kSortGatherTile 16-byte chunks of a list's rows: rows follow their keys, for every list of the
// batch, kSortGatherUnroll chunks per thread in flight; small blocks for the same reason as in the merge kernel
constexpr int kSortGatherThreads = 256;
constexpr int kSortGatherTile = kSortGatherThreads * kSortGatherUnroll;
__global__ void __launch_bounds__(kSortGatherThreads) gather_all_kernel(const SortArgs a) {
  chain_enter(a.more_follow != 0);
  int r;
  long long y;
  sort_block_item(a, r, y);
  if (r == 0 && y == 0 && threadIdx.x == 0) gstore(a.call_flag, 0);  // every reader of the word has finished: ready for the next call
  const long long e0 = gload(a.edge_offsets + r);
  const long long K = min(static_cast<long long>(gload(a.edge_offsets + r + 1) - e0), static_cast<long long>(a.max_len));
  const long long chunks = K * a.row_ch;
  const long long first = y * kSortGatherTile;
  if (first >= chunks) return;
  const uint4* src = reinterpret_cast<const uint4*>(a.feats_in) + e0 * a.row_ch;
  uint4* dst = reinterpret_cast<uint4*>(a.feats_out) + e0 * a.row_ch;
  const int* perm = a.perm_out + e0;
  uint4 v[kSortGatherUnroll];
#pragma unroll
  for (int u = 0; u < kSortGatherUnroll; ++u) {
    const long long c = first + static_cast<long long>(u) * kSortGatherThreads + threadIdx.x;
    if (c < chunks) {
      const int row = static_cast<int>(c / a.row_ch), piece = static_cast<int>(c - static_cast<long long>(row) * a.row_ch);
      v[u] = ldg128(src + static_cast<long long>(gload(perm + row)) * a.row_ch + piece);
    }
  }
#pragma unroll
  for (int u = 0; u < kSortGatherUnroll; ++u) {
    const long long c = first + static_cast<long long>(u) * kSortGatherThreads + threadIdx.x;
    if (c < chunks) st128_stream(dst + c, v[u]);  // written once, read by a later kernel at the earliest
  }
}

}  // namespace ccr
