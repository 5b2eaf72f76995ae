// Batching and padding of variable-length requests (Section 6.3.1, "Batching and Padding for Variable-Length
// Requests").  The paper's three steps are: (1) scatter indices (batch_idx, pos_idx) from the valid-position
// masks, (2) the valid positions flattened across the batch for one gather from the index, (3) a scatter of the
// gathered rows into T[b, n_max, features].  Here step 1 is a stable per-request compaction of the resolved
// positions (the kept candidate's pos_idx is its rank among the request's valid candidates, its batch_idx the
// request), step 2 is the join itself over the compacted list, and step 3 is folded into the join's store
// addressing (row r * n_max + pos_idx), so the gathered rows are written once, straight into T.  The slots
// behind a request's last valid candidate are filled by pad_fill_kernel.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "ccr_device.cuh"

namespace ccr {

constexpr int kPadThreads = 1024;
constexpr int kPadItems = 8;  // consecutive candidates per thread and round of the compaction

__device__ __forceinline__ bool position_valid(int p, long long n_docs) { return p >= 0 && p < n_docs; }

// Block-wide inclusive scan of one int per thread (kPadThreads threads); returns the inclusive prefix and
// the block total.  `warp_sums` is kPadThreads / 32 ints of shared memory; the caller syncs before reuse.
__device__ __forceinline__ int block_scan_inclusive(int v, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, v, d);
    if (lane >= d) v += t;
  }
  if (lane == 31) warp_sums[warp] = v;
  __syncthreads();
  int before = 0;
  total = 0;
#pragma unroll
  for (int w = 0; w < kPadThreads / 32; ++w) {
    const int s = warp_sums[w];
    if (w < warp) before += s;
    total += s;
  }
  return v + before;
}

// Valid candidates among [j0, j1), counted by the whole block with kPadItems loads in flight per thread.
__device__ __forceinline__ int block_count_valid(const int32_t* cand_idx, long long j0, long long j1, long long n_docs,
                                                 int* warp_sums) {
  int c = 0;
  for (long long base = j0 + threadIdx.x; base < j1; base += static_cast<long long>(kPadThreads) * kPadItems) {
    int p[kPadItems];
#pragma unroll
    for (int k = 0; k < kPadItems; ++k) {
      const long long j = base + static_cast<long long>(k) * kPadThreads;
      p[k] = j < j1 ? gload(cand_idx + j) : -1;
    }
#pragma unroll
    for (int k = 0; k < kPadItems; ++k) c += position_valid(p[k], n_docs) ? 1 : 0;
  }
  int total;
  block_scan_inclusive(c, warp_sums, total);
  __syncthreads();  // warp_sums may be reused at once
  return total;
}

// Step 1a: valid candidates per request -> counts[r + 1] (counts[0] = 0).  One block per request.
__global__ void __launch_bounds__(kPadThreads)
count_valid_kernel(const int32_t* cand_idx, const int64_t* cand_offsets, long long n_docs, int64_t* counts) {
  chain_enter(true);
  __shared__ int warp_sums[kPadThreads / 32];
  const int r = blockIdx.x;
  const int total = block_count_valid(cand_idx, gload(cand_offsets + r), gload(cand_offsets + r + 1), n_docs, warp_sums);
  if (threadIdx.x == 0) {
    gstore(counts + r + 1, total);
    if (r == 0) gstore(counts, 0);
  }
}

// Step 1b: in-place inclusive scan of counts[1 .. n_req] (one block; n_req is a batch size, a few hundred).
__global__ void __launch_bounds__(kPadThreads) scan_counts_kernel(int64_t* counts, int n_req) {
  chain_enter(true);
  __shared__ int warp_sums[kPadThreads / 32];
  __shared__ long long carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < n_req; base += kPadThreads) {
    const int r = base + threadIdx.x;
    const int v = r < n_req ? static_cast<int>(gload_rw(counts + r + 1)) : 0;
    int total;
    const int inc = block_scan_inclusive(v, warp_sums, total);
    const long long carry = carry_s;
    if (r < n_req) gstore(counts + r + 1, carry + inc);
    __syncthreads();
    if (threadIdx.x == 0) carry_s = carry + total;
    __syncthreads();
  }
}

// Step 1c + 2: the request's valid positions, in their input order, at [offsets_out[r], offsets_out[r + 1]);
// src_out[k] (optional) is the flat input index of kept candidate k, so scores can be carried back.
// Blocks (r, 0 .. gridDim.y) each take one slice of request r; a block first counts the valid candidates in
// the slices before its own (a re-read of at most the request's positions, which sit in L2), then walks its
// slice in rounds of kPadThreads * kPadItems candidates.  In a round warp w owns the kPadItems consecutive
// groups of 32 candidates from w * 32 * kPadItems: a ballot per group ranks its valid lanes, so loads and
// stores are both contiguous per warp instruction and the order is kept without a second pass.
__global__ void __launch_bounds__(kPadThreads)
compact_valid_kernel(const int32_t* cand_idx, const int64_t* cand_offsets, long long n_docs, const int64_t* offsets_out,
                     int32_t* idx_out, int32_t* src_out) {
  chain_enter(false);
  __shared__ int warp_sums[kPadThreads / 32];
  const int r = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long j0 = gload(cand_offsets + r), j1 = gload(cand_offsets + r + 1);
  const long long slice = (((j1 - j0) + gridDim.y - 1) / gridDim.y + 31) / 32 * 32;
  const long long s0 = min(j1, j0 + blockIdx.y * slice), s1 = min(j1, s0 + slice);
  if (s0 >= s1) return;
  long long out = gload(offsets_out + r) + block_count_valid(cand_idx, j0, s0, n_docs, warp_sums);
  for (long long base = s0; base < s1; base += kPadThreads * kPadItems) {
    const long long jw = base + static_cast<long long>(warp) * (32 * kPadItems) + lane;
    int p[kPadItems];
#pragma unroll
    for (int k = 0; k < kPadItems; ++k) p[k] = jw + 32 * k < s1 ? gload(cand_idx + jw + 32 * k) : -1;
    unsigned votes[kPadItems];
    int warp_total = 0;
#pragma unroll
    for (int k = 0; k < kPadItems; ++k) {
      votes[k] = __ballot_sync(0xffffffffu, position_valid(p[k], n_docs));
      warp_total += __popc(votes[k]);
    }
    if (lane == 0) warp_sums[warp] = warp_total;
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kPadThreads / 32; ++w) {
      const int c = warp_sums[w];
      if (w < warp) before += c;
      total += c;
    }
    long long w0 = out + before;
#pragma unroll
    for (int k = 0; k < kPadItems; ++k) {
      if ((votes[k] >> lane) & 1u) {
        const long long w = w0 + __popc(votes[k] & ((1u << lane) - 1u));
        gstore(idx_out + w, p[k]);
        if (src_out != nullptr) gstore(src_out + w, jw + 32 * k);
      }
      w0 += __popc(votes[k]);
    }
    out += total;
    __syncthreads();  // warp_sums is rewritten by the next round
  }
}

// Step 3's pads: rows [n_r, n_max) of request r are zero rows with mask 0.  Blocks (r, 0 .. gridDim.y) share
// request r's pad range; 16-byte streaming stores (out_b is a multiple of 16).
__global__ void __launch_bounds__(kPadThreads)
pad_fill_kernel(const int64_t* cand_offsets, long long n_max, long long out_b, uint8_t* out_rows, uint8_t* out_mask) {
  const int r = blockIdx.x;
  long long n_r = gload(cand_offsets + r + 1) - gload(cand_offsets + r);
  n_r = n_r < 0 ? 0 : (n_r > n_max ? n_max : n_r);
  const long long first = r * n_max + n_r, pads = n_max - n_r;
  uint4* rows = reinterpret_cast<uint4*>(out_rows + first * out_b);
  const long long chunks = pads * (out_b / 16);
  const long long t = static_cast<long long>(blockIdx.y) * kPadThreads + threadIdx.x;
  const long long stride = static_cast<long long>(gridDim.y) * kPadThreads;
  for (long long c = t; c < chunks; c += stride) st128_stream(rows + c, make_uint4(0u, 0u, 0u, 0u));
  for (long long i = t; i < pads; i += stride) gstore(out_mask + first + i, 0);
}

}  // namespace ccr
