// Merge-path variant of the join for candidates whose author ids are non-decreasing inside each request.
// Same result as Algorithm 1 steps 2-3 of the paper (lower bound + equality test); the paper has no such
// variant, it is an addition for pre-sorted candidate lists.
//
// Per block and request segment (n candidates of the tile):
//   1. gather the candidates' author ids into shared memory (sa);
//   2. block-cooperative k-ary search (__syncthreads_count) for the lower bounds of sa[0] and sa[n-1]
//      in the request's keys: the only keys this tile can touch are the window [lo, hi);
//   3. stage that window in shared memory (TMA bulk copy), typically K*n/N keys instead of K;
//   4. merge path: thread t binary-searches its diagonal t*L of the (sa, window) merge grid, then walks L
//      steps of the merge sequentially; when a candidate is emitted, the number of window keys already
//      consumed is its lower bound.  O(n + w) comparisons instead of O(n log K);
//   5. rows are assembled exactly as in the binary-search kernel.
// If the window does not fit the staging budget the segment falls back to the binary-search path.
// With an untruthful promise (authors not sorted) every index stays clamped to the request's key range:
// values are then unspecified, accesses stay in bounds.
#pragma once

#include "ccr_join.cuh"

namespace ccr {

constexpr long long kNoAuthor = static_cast<long long>(0x8000000000000000ull);  // below every key (keys are >= 0)

// Block-wide lower bound of `id` in ascending g[0..K): every thread probes one pivot per round.
// All threads must call; returns the same value in every thread.  Result is always within [0, K].
__device__ __forceinline__ int block_lower_bound(const int64_t* g, int K, int64_t id) {
  int lo = 0, n = K;
  while (n > 0) {
    const int step = (n + kThreads - 1) / kThreads;
    const long long p = static_cast<long long>(lo) + static_cast<long long>(threadIdx.x + 1) * step - 1;
    const int below = (p < lo + n) && (__ldg(g + p) < id);
    const int c = __syncthreads_count(below);
    const int nlo = min(lo + c * step, lo + n);
    n = min(step - 1, lo + n - nlo);
    lo = nlo;
  }
  return lo;
}

template <int DOC_CH, int EDGE_CH, int REQ_CH>
__global__ void __launch_bounds__(kThreads, 2) join_merge_kernel(const JoinArgs a) {
  extern __shared__ __align__(16) unsigned char smem[];
  // layout: [mbarrier | sa int64[tile] | spos int32[tile] (padded to 16 B) | staged keys]
  int64_t* sa = reinterpret_cast<int64_t*>(smem + kSmemHeader);
  int* spos = reinterpret_cast<int*>(sa + a.tile);
  int64_t* skeys = reinterpret_cast<int64_t*>(spos + ((a.tile + 3) & ~3));
  const uint32_t bar = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const RowShape<DOC_CH, EDGE_CH, REQ_CH, false> sh(a);

  if (tid == 0) {
    mbar_init(bar, 1);
    fence_proxy_async_smem();
  }
  __syncthreads();
  uint32_t phase = 0;

  const long long j0 = static_cast<long long>(blockIdx.x) * a.tile;
  const long long j1 = min(j0 + a.tile, a.total);
  int r = request_of(a.cand_offsets, a.n_req, j0);

  long long seg = j0;
  while (seg < j1 && r < a.n_req) {
    const long long rend = __ldg(a.cand_offsets + r + 1);
    if (rend <= seg) {
      ++r;
      continue;
    }
    const long long seg_end = min(rend, j1);
    const int n = static_cast<int>(seg_end - seg);
    long long kb;
    const int K = request_keys(a, r, kb);
    const int64_t* gk = a.edge_keys + kb;

    // 1. author ids of the segment
    for (int i = tid; i < n; i += kThreads) {
      const int idx = __ldg(a.cand_idx + seg + i);
      sa[i] = (idx >= 0 && idx < a.n_docs) ? __ldg(a.author_ids + idx) : kNoAuthor;
    }
    __syncthreads();

    // 2. key window this segment can touch
    const int lo = block_lower_bound(gk, K, sa[0]);
    const int hi = min(K, block_lower_bound(gk, K, sa[n - 1]) + 1);
    const int w = max(hi - lo, 0);

    StagedKeys keys;
    const bool windowed = (a.key_cap > 0) && (w <= a.key_cap) && (a.min_stride_log2 == 0);
    // 3. stage the window (or, if it is too long, the request's keys as the binary-search kernel does)
    if (!stage_keys(a, skeys, bar, phase, windowed ? kb + lo : kb, windowed ? w : K, keys)) {
      give_up_wait(a, bar, phase);
      return;
    }

    if (windowed) {
      // 4. merge path over (sa[0..n), window[0..w)); a candidate goes before an equal key, so the keys
      //    consumed when it is emitted are exactly the keys below it
      const int64_t* B = keys.sk;
      const int total = n + w;
      const int L = (total + kThreads - 1) / kThreads;
      const int diag = min(tid * L, total);
      int ab = max(0, diag - w), ae = min(diag, n);
      while (ab < ae) {
        const int mid = (ab + ae) >> 1;
        if (sa[mid] <= B[diag - 1 - mid]) ab = mid + 1; else ae = mid;
      }
      int ai = ab, bi = diag - ab;
      for (int step = 0; step < L && (ai < n || bi < w); ++step) {
        if (ai < n && (bi >= w || sa[ai] <= B[bi])) {
          const bool hit = bi < w && B[bi] == sa[ai];
          spos[ai] = (lo + bi) | (hit ? static_cast<int>(0x80000000u) : 0);
          ++ai;
        } else {
          ++bi;
        }
      }
      __syncthreads();
    }

    // 5. rows
    for (int g = warp * 32; g < n; g += kWarps * 32) {
      const int cnt = min(32, n - g);
      if (windowed) {
        process_group<DOC_CH, EDGE_CH, REQ_CH, false>(
            a, sh, keys, r, kb, seg + g, cnt, lane, [&](bool inr, int64_t, int& pos) -> bool {
              const int packed = (lane < cnt) ? spos[g + lane] : 0;
              pos = packed & 0x7fffffff;
              return inr && (packed < 0) && pos < K;  // pos < K guards a stale slot under a broken promise
            });
      } else {
        process_group<DOC_CH, EDGE_CH, REQ_CH, false>(
            a, sh, keys, r, kb, seg + g, cnt, lane,
            [&](bool inr, int64_t auth, int& pos) -> bool { return inr && keys.find(auth, pos); });
      }
    }
    __syncthreads();
    seg = seg_end;
    ++r;
  }
}

}  // namespace ccr
