// Document-id resolution on the GPU (Section 6.3.1 of the paper, "Document ID Resolution", Eq. 6):
// pos(q) = position of id q in the index, or -1.  The paper stored the id -> position map as a sorted array
// in HBM, resolved queries with a binary-search kernel (~5 ms per request over a few hundred million ids,
// ~47 ms at batch 8, every probe a dependent HBM access) and then moved the step to a CPU hash map.
//
// Here the sorted array gets a static search tree of sampled levels, fan-out 32: level l+1 holds the last
// key of every full block of 32 keys of level l.  The top level (<= 16,384 keys) is staged in shared
// memory; below it a query touches one 256-byte window (two cache lines) per level, inside which a lane
// needs two dependent rounds of loads (octant, then position): the ~2 MB level stays in L2, the larger ones come
// from HBM.  A query over 300M ids makes 6 dependent rounds instead of 29 dependent probes across the whole
// array; eight queries per lane are in flight at once.
#pragma once

#include "ccr_device.cuh"

namespace ccr {

constexpr int kResolveFanLog2 = 5;                 // 32 keys = one 256-byte window per level
constexpr int kResolveMaxLevels = 8;
constexpr int kResolveTopMax = 16384;              // keys of the top level (128 KB of shared memory)
constexpr int kResolveThreads = 256;
constexpr int kResolveUnroll = 8;                 // queries a lane keeps in flight
#ifndef CCR_RESOLVE_ROUND2
#define CCR_RESOLVE_ROUND2 2
#endif
constexpr int kResolveRound2 = CCR_RESOLVE_ROUND2;  // queries of a lane whose octants are in flight together
constexpr long long kResolveInf = 0x7fffffffffffffffLL;  // stands for the keys beyond the end of a level

struct ResolveArgs {
  const int64_t* level[kResolveMaxLevels];         // level[0] = the sorted ids, level[n_levels-1] = top
  long long count[kResolveMaxLevels];
  int n_levels;
  const int32_t* positions;                        // position of id i, or null: the rank i itself
  long long n_queries;
  const int64_t* queries;
  int32_t* out_pos;
};

__global__ void build_level_kernel(const int64_t* below, long long n_below, int64_t* above, long long n_above) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n_above;
       i += static_cast<long long>(gridDim.x) * blockDim.x)
    above[i] = below[((i + 1) << kResolveFanLog2) - 1];
}

__global__ void __launch_bounds__(kResolveThreads) resolve_kernel(const ResolveArgs a) {
  extern __shared__ __align__(16) unsigned char smem_res[];
  int64_t* top = reinterpret_cast<int64_t*>(smem_res);
  const int top_l = a.n_levels - 1;
  const int n_top = static_cast<int>(a.count[top_l]);
  for (int i = threadIdx.x; i < n_top; i += blockDim.x) top[i] = __ldg(a.level[top_l] + i);
  __syncthreads();

  // lane-per-query, kResolveUnroll queries of a lane in flight; inside a 32-key window the lane runs a
  // 5-step branch-free search (its sectors come from L2 / HBM on demand).  A warp-cooperative variant
  // (whole window per coalesced access, __ballot_sync rank) was measured and is slower at every batch size:
  // 886 vs 743 us for 1.92M queries, the extra shuffles and the lower number of independent accesses in
  // flight outweigh the saved sector fetches.
  // query u of a lane is `threads` apart from query u-1, so that a small launch still spreads over all blocks
  const long long threads = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long base = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; base < a.n_queries;
       base += threads * kResolveUnroll) {
    int64_t q[kResolveUnroll];
    long long c[kResolveUnroll];  // number of keys of the current level that are below q
#pragma unroll
    for (int u = 0; u < kResolveUnroll; ++u) {
      const long long j = base + static_cast<long long>(u) * threads;
      q[u] = j < a.n_queries ? __ldg(a.queries + j) : 0;
      c[u] = lower_bound_smem(top, n_top, q[u]);
    }
    // descend: c keys of level l+1 below q  =>  blocks 0..c-1 of level l are below q, the answer is in block c
    for (int l = top_l - 1; l >= 0; --l) {
      const int64_t* lev = a.level[l];
      const long long n = a.count[l];
      // Inside the 32-key window a query needs two dependent rounds instead of a six-probe binary search:
      // round 1 reads the last key of the first three octants (three independent loads; the fourth octant's last
      // key is not below q by construction of the level above) and picks the octant, round 2 reads the octant's
      // eight keys as four 16-byte loads and counts the ones below q.  Keys beyond the end of the level count as
      // +infinity.  All queries of the lane do round 1 together; round 2 runs for kResolveRound2 of them at a time, which
      // keeps the keys in flight within the register budget.
      long long lo[kResolveUnroll];
      int64_t r1[kResolveUnroll][3];
#pragma unroll
      for (int u = 0; u < kResolveUnroll; ++u) {
        lo[u] = c[u] << kResolveFanLog2;
#pragma unroll
        for (int o = 0; o < 3; ++o) {
          const long long i = lo[u] + 8 * o + 7;
          r1[u][o] = i < n ? __ldg(lev + i) : kResolveInf;
        }
      }
#pragma unroll
      for (int u = 0; u < kResolveUnroll; ++u)
        lo[u] += 8 * ((r1[u][0] < q[u] ? 1 : 0) + (r1[u][1] < q[u] ? 1 : 0) + (r1[u][2] < q[u] ? 1 : 0));
#pragma unroll
      for (int h = 0; h < kResolveUnroll; h += kResolveRound2) {
        longlong2 r2[kResolveRound2][4];
#pragma unroll
        for (int v = 0; v < kResolveRound2; ++v) {
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            const long long i = lo[h + v] + 2 * p;  // even, and the level's base is 16-byte aligned
            if (i + 1 < n) {
              r2[v][p] = __ldg(reinterpret_cast<const longlong2*>(lev + i));
            } else {
              r2[v][p].x = i < n ? __ldg(lev + i) : kResolveInf;
              r2[v][p].y = kResolveInf;
            }
          }
        }
#pragma unroll
        for (int v = 0; v < kResolveRound2; ++v) {
          int below = 0;
#pragma unroll
          for (int p = 0; p < 4; ++p) below += (r2[v][p].x < q[h + v] ? 1 : 0) + (r2[v][p].y < q[h + v] ? 1 : 0);
          c[h + v] = lo[h + v] + below;
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kResolveUnroll; ++u) {
      const long long j = base + static_cast<long long>(u) * threads;
      if (j >= a.n_queries) continue;
      int pos = -1;
      if (c[u] < a.count[0] && __ldg(a.level[0] + c[u]) == q[u])
        pos = a.positions ? __ldg(a.positions + c[u]) : static_cast<int>(c[u]);
      a.out_pos[j] = pos;
    }
  }
}

}  // namespace ccr
