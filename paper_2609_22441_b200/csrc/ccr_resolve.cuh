// Document-id resolution on the GPU (Section 6.3.1 of the paper, "Document ID Resolution", Eq. 6):
// pos(q) = position of id q in the index, or -1.  The paper stored the id -> position map as a sorted array
// in HBM, resolved queries with a binary-search kernel (~5 ms per request over a few hundred million ids,
// ~47 ms at batch 8, every probe a dependent HBM access) and then moved the step to a CPU hash map.
//
// Here the sorted array gets a static search tree of sampled levels, fan-out 8: level l+1 holds the last
// key of every full block of 8 keys of level l.  The top level (<= 2,048 keys, 16 KB) is staged in shared
// memory; below it a query reads one 64-byte window per level in one dependent round: the four lanes that share
// the query load 16 bytes each (one access for the load unit instead of four, which is what bounded the
// lane-per-query form: every scattered 16-byte load of a lane is a pass of its own through the L1), count the
// keys below the id and add the counts up with two shuffles; the leaf round also says whether the id is
// present.  The small levels stay in L2, the large ones come from HBM 64 bytes at a time.  A query over 300M ids
// makes 6 dependent rounds instead of 29 dependent probes across the whole array.  Two queries per group of
// lanes in flight, up to 2,048 threads per SM.  A batch of a million queries or more is bound by instruction
// issue rather than by the chain of rounds; there a warp takes 32 queries at a time, searches the top level a lane
// per query (the same instructions serve 32 queries instead of 8) and hands the queries to the lane groups by
// shuffles, four per group in flight (1.92M queries over 1M ids: 75 -> 62 us; on 240,000 queries over 300M ids
// that form was 13-20 % slower, hence the size rule).  Measured and slower: wider windows (128 bytes with eight lanes
// per query; 256 bytes in two rounds), a lane per query with 1-8 queries in flight, and a larger staged top
// level (it takes shared memory from the L1 and start-up time from every block).
#pragma once

#include "ccr_device.cuh"

namespace ccr {

constexpr int kResolveFanLog2 = 3;                 // 8 keys = one 64-byte window per level
constexpr int kResolveMaxLevels = 8;               // 2,048 x 8^7 ids: more than int32 positions can name
constexpr int kResolveTopMax = 2048;               // keys of the top level (16 KB of shared memory)
constexpr int kResolveThreads = 256;
constexpr int kResolveBlocksPerSm = 8;             // grid cap: the top level is staged by every block
constexpr int kResolveUnroll = 2;                  // queries a group of lanes keeps in flight
constexpr int kResolveWarpUnroll = 4;              // ... when a warp takes 32 queries at a time (all of them at once)
constexpr long long kResolveWarpMin = 1 << 20;     // batches from this size on search the top level a lane per query
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

// 16-byte window piece of a level that does not stay in any cache between queries (the three lowest levels of a
// large index): read past L1.
__device__ __forceinline__ longlong2 resolve_load(const longlong2* p, bool once) {
  if (!CCR_CHK(p, 16)) return make_longlong2(kResolveInf, kResolveInf);  // reads like the padding behind a level
#ifndef CCR_RESOLVE_L1
  if (once) {
    longlong2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.s64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p));
    return v;
  }
#endif
  return __ldg(p);
}

__global__ void build_level_kernel(const int64_t* below, long long n_below, int64_t* above, long long n_above) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n_above;
       i += static_cast<long long>(gridDim.x) * blockDim.x)
    above[i] = below[((i + 1) << kResolveFanLog2) - 1];
}

// Every level is followed by kResolvePad keys of +infinity, so that the window a query reads (window c of a level
// with n keys, c <= n / 8) needs no bounds checks; the allocation of a level leaves room for them.
constexpr int kResolvePad = 2 << kResolveFanLog2;
static_assert((1 << (kResolveFanLog2 - 1)) % kResolveWarpUnroll == 0, "the queries of a warp are handed out in whole rounds");
static_assert(kResolvePad <= 32 && kResolvePad * 8 <= 256, "one warp writes the padding; a level is allocated with 256 spare bytes");
__global__ void pad_level_kernel(int64_t* level, long long n) {
  if (threadIdx.x < kResolvePad) level[n + threadIdx.x] = kResolveInf;
}

// WARP_TOP: the top level searched a lane per query (large batches, bound by instruction issue); otherwise by the
// group of lanes that descends with the query (small batches, bound by the chain of dependent rounds).
template <bool WARP_TOP>
__global__ void __launch_bounds__(kResolveThreads) resolve_kernel(const ResolveArgs a) {
  extern __shared__ __align__(16) unsigned char smem_res[];
  int64_t* top = reinterpret_cast<int64_t*>(smem_res);
  const int top_l = a.n_levels - 1;
  const int n_top = static_cast<int>(a.count[top_l]);
  for (int i = threadIdx.x; i < n_top; i += blockDim.x) top[i] = gload(a.level[top_l] + i);
  __syncthreads();
  constexpr int G = 1 << (kResolveFanLog2 - 1);  // lanes that share a query: one 16-byte load each per window
  if constexpr (WARP_TOP) {
    constexpr int kPerRound = 32 / G;              // queries a warp descends with at a time
    const unsigned lane = threadIdx.x & 31, sub = lane & (G - 1);
    const long long n_warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
    const long long warp_id = (blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x) >> 5;
    // A warp takes 32 queries at a time.  The search of the top level runs a lane per query (the same instructions
    // serve 32 queries instead of the 8 that share the warp below); for the windows the queries are then handed,
    // kResolveWarpUnroll x 8 at a time, to groups of G lanes by shuffles.
    for (long long first = warp_id * 32; first < a.n_queries; first += n_warps * 32) {  // warp-uniform
      const long long mine = first + lane;
      const int64_t q_own = mine < a.n_queries ? gload(a.queries + mine) : 0;
      unsigned c_own = 0;  // number of keys of the current level that are below q (an index has < 2^31 ids)
      {
        int n = n_top;
        while (n > 1) {
          const int half = n >> 1;
          c_own = (top[c_own + half - 1] < q_own) ? c_own + half : c_own;
          n -= half;
        }
        if (n == 1) c_own += (top[c_own] < q_own) ? 1 : 0;
      }
      for (int part = 0; part < G / kResolveWarpUnroll; ++part) {
        int64_t q[kResolveWarpUnroll];
        unsigned c[kResolveWarpUnroll];
        int src[kResolveWarpUnroll];
  #pragma unroll
        for (int u = 0; u < kResolveWarpUnroll; ++u) {
          src[u] = (part * kResolveWarpUnroll + u) * kPerRound + static_cast<int>(lane / G);
          q[u] = __shfl_sync(kFull, q_own, src[u]);
          c[u] = __shfl_sync(kFull, c_own, src[u]);
        }
        // descend: c keys of level l+1 below q  =>  windows 0..c-1 of level l are below q, the answer is in window c
        for (int l = top_l - 1; l >= 1; --l) {
          const longlong2* lev = reinterpret_cast<const longlong2*>(a.level[l]);
          longlong2 k[kResolveWarpUnroll];
  #pragma unroll
          for (int u = 0; u < kResolveWarpUnroll; ++u) k[u] = resolve_load(lev + (static_cast<size_t>(c[u]) * G + sub), l <= 2);
  #pragma unroll
          for (int u = 0; u < kResolveWarpUnroll; ++u) {
            unsigned v = (k[u].x < q[u] ? 1u : 0u) + (k[u].y < q[u] ? 1u : 0u);
  #pragma unroll
            for (int d = 1; d < G; d <<= 1) v += __shfl_xor_sync(kFull, v, d);
            c[u] = (c[u] << kResolveFanLog2) + v;
          }
        }
        {  // the leaf round also tells whether the id is present (a match with the padding lands at c >= count[0])
          const longlong2* lev = reinterpret_cast<const longlong2*>(a.level[0]);
          longlong2 k[kResolveWarpUnroll];
  #pragma unroll
          for (int u = 0; u < kResolveWarpUnroll; ++u) k[u] = resolve_load(lev + (static_cast<size_t>(c[u]) * G + sub), true);
  #pragma unroll
          for (int u = 0; u < kResolveWarpUnroll; ++u) {
            unsigned v = (k[u].x < q[u] ? 1u : 0u) + (k[u].y < q[u] ? 1u : 0u) + ((k[u].x == q[u] || k[u].y == q[u]) ? 256u : 0u);
  #pragma unroll
            for (int d = 1; d < G; d <<= 1) v += __shfl_xor_sync(kFull, v, d);
            c[u] = (c[u] << kResolveFanLog2) + (v & 255u);
            const long long j = first + src[u];
            if (sub == 0 && j < a.n_queries) {
              int pos = -1;
              if (v >= 256u && c[u] < a.count[0]) pos = a.positions ? gload(a.positions + c[u]) : static_cast<int>(c[u]);
              gstore(a.out_pos + j, pos);
            }
          }
        }
      }
    }
    return;
  }
  const unsigned sub = threadIdx.x & (G - 1);
  const long long groups = (static_cast<long long>(gridDim.x) * blockDim.x) / G;
  const long long gid = (blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x) / G;
  const long long rounds = (a.n_queries + groups * kResolveUnroll - 1) / (groups * kResolveUnroll);
  for (long long it = 0; it < rounds; ++it) {  // warp-uniform trip count: the shuffles below need every lane
    const long long base = it * groups * kResolveUnroll + gid;
    int64_t q[kResolveUnroll];
    unsigned c[kResolveUnroll];  // number of keys of the current level that are below q (an index has < 2^31 ids)
#pragma unroll
    for (int u = 0; u < kResolveUnroll; ++u) {
      const long long j = base + static_cast<long long>(u) * groups;
      q[u] = j < a.n_queries ? gload(a.queries + j) : 0;
      c[u] = 0;
    }
    {  // the group's searches of the top level step together, so their shared-memory reads overlap
      int n = n_top;
      while (n > 1) {
        const int half = n >> 1;
#pragma unroll
        for (int u = 0; u < kResolveUnroll; ++u) c[u] = (top[c[u] + half - 1] < q[u]) ? c[u] + half : c[u];
        n -= half;
      }
      if (n == 1) {
#pragma unroll
        for (int u = 0; u < kResolveUnroll; ++u) c[u] += (top[c[u]] < q[u]) ? 1 : 0;
      }
    }
    // descend: c keys of level l+1 below q  =>  windows 0..c-1 of level l are below q, the answer is in window c
    for (int l = top_l - 1; l >= 1; --l) {
      const longlong2* lev = reinterpret_cast<const longlong2*>(a.level[l]);
      longlong2 k[kResolveUnroll];
#pragma unroll
      for (int u = 0; u < kResolveUnroll; ++u) k[u] = resolve_load(lev + (static_cast<size_t>(c[u]) * G + sub), l <= 2);
#pragma unroll
      for (int u = 0; u < kResolveUnroll; ++u) {
        unsigned v = (k[u].x < q[u] ? 1u : 0u) + (k[u].y < q[u] ? 1u : 0u);
#pragma unroll
        for (int d = 1; d < G; d <<= 1) v += __shfl_xor_sync(kFull, v, d);
        c[u] = (c[u] << kResolveFanLog2) + v;
      }
    }
    {  // the leaf round also tells whether the id is present (a match with the padding lands at c >= count[0])
      const longlong2* lev = reinterpret_cast<const longlong2*>(a.level[0]);
      longlong2 k[kResolveUnroll];
#pragma unroll
      for (int u = 0; u < kResolveUnroll; ++u) k[u] = resolve_load(lev + (static_cast<size_t>(c[u]) * G + sub), true);
#pragma unroll
      for (int u = 0; u < kResolveUnroll; ++u) {
        unsigned v = (k[u].x < q[u] ? 1u : 0u) + (k[u].y < q[u] ? 1u : 0u) + ((k[u].x == q[u] || k[u].y == q[u]) ? 256u : 0u);
#pragma unroll
        for (int d = 1; d < G; d <<= 1) v += __shfl_xor_sync(kFull, v, d);
        c[u] = (c[u] << kResolveFanLog2) + (v & 255u);
        const long long j = base + static_cast<long long>(u) * groups;
        if (sub == 0 && j < a.n_queries) {
          int pos = -1;
          if (v >= 256u && c[u] < a.count[0]) pos = a.positions ? gload(a.positions + c[u]) : static_cast<int>(c[u]);
          gstore(a.out_pos + j, pos);
        }
      }
    }
  }
}

}  // namespace ccr
