// The fused join kernel: Algorithm 1 steps 2-4 (search, validate, gather) of the paper fused with the
// document-row gather from the resident index (Section 6.3.1) and the request-feature broadcast
// (Section 3), for a ragged batch of requests in one launch.
//
// Work split.  The flat candidate range [0, total) is cut into tiles of `tile` candidates, one thread
// block each, so the grid is known on the host without reading the offsets.  A block walks the request
// segments that intersect its tile (usually one); per segment it stages that request's sorted keys in
// shared memory and its warps take groups of 32 consecutive candidates:
//   lane-per-candidate : position -> author id (8-B gather) -> branch-free lower bound in the staged keys
//   warp-cooperative   : rows are moved as 16-byte chunks, consecutive lanes on consecutive chunks of
//                        the same row, the owning lane's position / match broadcast with __shfl_sync;
//                        every output byte is written exactly once with full-sector streaming stores.
// Key staging.  K <= key_cap: the whole list, by one 1-D TMA bulk copy (plus at most one scalar key at
// either end when the request's first key is only 8-byte aligned).  K > key_cap: every 2^s-th key is
// staged as the top of the search tree and the last <= 2^s keys of a search are read from global
// memory (one 128-byte line at s = 4, L2 resident).  key_cap == 0: the whole search runs on global memory.
#pragma once

#include "ccr_device.cuh"

namespace ccr {

// Keys of the request a block is currently serving.
struct StagedKeys {
  const int64_t* sk;  // shared-memory copy (index i = key i when s_log == 0, sample i otherwise)
  const int64_t* gk;  // the request's keys in global memory
  int K;              // keys in the request
  int M;              // staged entries (0 = nothing staged)
  int s_log;          // log2 of the sampling stride

  // Algorithm 1 steps 2-3 for one id: pos = lower bound, found = pos < K and keys[pos] == id.
  __device__ __forceinline__ bool find(int64_t id, int& pos) const {
    if (K == 0) {
      pos = 0;
      return false;
    }
    if (M > 0 && s_log == 0) {
      pos = lower_bound_smem(sk, M, id);
      return pos < K && sk[pos] == id;
    }
    int lo = 0, n = K;
    if (M > 0) {
      // sample i is key (i+1)*2^s - 1: c samples below id means blocks 0..c-1 are entirely below it
      const int c = lower_bound_smem(sk, M, id);
      lo = c << s_log;
      n = min(1 << s_log, K - lo);
    }
    pos = lo + lower_bound_global(gk + lo, n, id);
    return pos < K && __ldg(gk + pos) == id;
  }
};

// Stage request keys [kb, kb+K) for the whole block.  Returns false if the bounded wait for the bulk
// copy expired (block-uniform).  Ends with a __syncthreads.
__device__ __forceinline__ bool stage_keys(const JoinArgs& a, int64_t* skeys, uint32_t bar, uint32_t& phase,
                                           long long kb, int K, StagedKeys& st) {
  const int tid = threadIdx.x;
  st.gk = a.edge_keys + kb;
  st.K = K;
  st.M = 0;
  st.s_log = 0;
  st.sk = skeys;
  int expired = 0;
  if (a.key_cap > 0 && K > 0) {
    if (K <= a.key_cap && a.min_stride_log2 == 0) {
      // slot of key i is i + shift, so that 16-byte aligned global addresses land on 16-byte aligned slots
      const int shift = static_cast<int>(kb & 1);
      const int i0 = shift;                       // first key whose address is 16-byte aligned
      const int nb = (K - i0) & ~1;               // keys moved by the bulk copy (even count)
      st.sk = skeys + shift;
      st.M = K;
      if (tid == 0 && nb > 0) {
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nb) * 8u);
        bulk_copy_g2s(smem_u32(skeys + i0 + shift), a.edge_keys + kb + i0, static_cast<uint32_t>(nb) * 8u, bar);
      }
      if (tid == 32 && shift) skeys[shift] = __ldg(a.edge_keys + kb);
      if (tid == 64 && ((K - i0) & 1)) skeys[K - 1 + shift] = __ldg(a.edge_keys + kb + K - 1);
      if (nb > 0) {
        expired = mbar_wait_bounded(bar, phase) ? 0 : 1;
        phase ^= 1u;
      }
    } else {
      int s_log = a.min_stride_log2;
      while ((K >> s_log) > a.key_cap) ++s_log;
      st.s_log = s_log;
      st.M = K >> s_log;
      for (int i = tid; i < st.M; i += kThreads)
        skeys[i] = __ldg(a.edge_keys + kb + ((static_cast<long long>(i) + 1) << s_log) - 1);
    }
  }
  return __syncthreads_or(expired) == 0;
}

// Copy one section of the 32 rows of a warp's group: `ch` 16-byte chunks per row, source row given by
// `src(row)` (nullptr = zeros), destination out + row*out_b.  Uniform trip count: safe for shuffles in src.
template <typename SrcFn>
__device__ __forceinline__ void copy_chunk(int i, int ch, int lane, int cnt, uint8_t* out, long long out_b, SrcFn& src) {
  const int c = i * 32 + lane;
  const int row = c / ch;
  const int piece = c - row * ch;
  const uint8_t* s = src(row);
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (s != nullptr) v = ldg128(s + piece * 16);
  if (row < cnt) st128_stream(out + row * out_b + piece * 16, v);
}

template <int CH, typename SrcFn>
__device__ __forceinline__ void copy_section(int ch_rt, int lane, int cnt, uint8_t* out, long long out_b, SrcFn src) {
  if constexpr (CH > 0) {
#pragma unroll
    for (int i = 0; i < CH; ++i) copy_chunk(i, CH, lane, cnt, out, out_b, src);
  } else {
    for (int i = 0; i < ch_rt; ++i) copy_chunk(i, ch_rt, lane, cnt, out, out_b, src);
  }
}

// Section widths of a launch, in 16-byte chunks and bytes (compile-time where the variant fixes them).
template <int DOC_CH, int EDGE_CH, int REQ_CH, bool SECOND>
struct RowShape {
  int doc_ch, edge_ch, req_ch, doc_b, edge_b, req_b;
  long long out_b;
  __device__ __forceinline__ explicit RowShape(const JoinArgs& a) {
    doc_ch = DOC_CH ? DOC_CH : a.doc_ch;
    edge_ch = EDGE_CH ? EDGE_CH : a.edge_ch;
    req_ch = (DOC_CH || EDGE_CH) ? REQ_CH : a.req_ch;  // REQ_CH == 0 is a real width in the tuned variants
    doc_b = doc_ch * 16;
    edge_b = edge_ch * 16;
    req_b = req_ch * 16;
    out_b = doc_b + edge_b * (SECOND ? 2 : 1) + req_b;
  }
};

// One warp, one group of up to 32 consecutive candidates [jg, jg+cnt) of request r.
// `lookup(inr, author, pos)` returns whether the author id is among the request's keys and its index.
template <int DOC_CH, int EDGE_CH, int REQ_CH, bool SECOND, typename Lookup>
__device__ __forceinline__ void process_group(const JoinArgs& a, const RowShape<DOC_CH, EDGE_CH, REQ_CH, SECOND>& sh,
                                              const StagedKeys& keys, int r, long long kb, long long jg, int cnt,
                                              int lane, Lookup lookup) {
  const int doc_b = sh.doc_b, edge_b = sh.edge_b;
  const long long out_b = sh.out_b;
  uint8_t* out = a.out_rows + jg * out_b;

  // ---- lane-per-candidate: position, ids
  const int idx = (lane < cnt) ? __ldg(a.cand_idx + jg + lane) : -1;
  const bool inr = idx >= 0 && idx < a.n_docs;
  const int64_t auth = inr ? __ldg(a.author_ids + idx) : -1;
  int64_t actor[4] = {-1, -1, -1, -1};
  unsigned types = 0;
  if (SECOND && inr) {
    if (a.max_actors == 4) {
      const longlong2* ap = reinterpret_cast<const longlong2*>(a.actor_ids + 4LL * idx);
      const longlong2 p0 = __ldg(ap);
      const longlong2 p1 = __ldg(ap + 1);
      actor[0] = p0.x;
      actor[1] = p0.y;
      actor[2] = p1.x;
      actor[3] = p1.y;
      types = __ldg(reinterpret_cast<const unsigned*>(a.actor_types + 4LL * idx));
    } else {
      for (int s = 0; s < a.max_actors; ++s) {
        actor[s] = __ldg(a.actor_ids + static_cast<long long>(a.max_actors) * idx + s);
        types |= static_cast<unsigned>(__ldg(a.actor_types + static_cast<long long>(a.max_actors) * idx + s)) << (8 * s);
      }
    }
  }

  // ---- document rows: issued before the search so that both latencies overlap
  auto doc_src = [&](int row) -> const uint8_t* {
    const int ridx = __shfl_sync(kFull, idx, row);
    return (ridx >= 0 && ridx < a.n_docs) ? a.doc_feats + static_cast<long long>(ridx) * doc_b : nullptr;
  };
  constexpr int kDocRegs = DOC_CH ? DOC_CH : 1;
  uint4 dv[kDocRegs];
  if constexpr (DOC_CH > 0) {
#pragma unroll
    for (int i = 0; i < DOC_CH; ++i) {
      const int c = i * 32 + lane;
      const int row = c / kDocRegs;
      const int piece = c - row * kDocRegs;
      const uint8_t* s = doc_src(row);
      dv[i] = make_uint4(0u, 0u, 0u, 0u);
      if (s != nullptr) dv[i] = ldg128(s + piece * 16);
    }
  }

  // ---- search (Algorithm 1 steps 2-3)
  int pos = 0;
  const bool found = lookup(inr, auth, pos);
  unsigned m = found ? 1u : 0u;
  int apos[4] = {0, 0, 0, 0};
  if (SECOND) {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      if (actor[s] >= 0 && keys.find(actor[s], apos[s])) {
        m |= 1u << (1 + s);
        m |= 1u << (5 + ((types >> (8 * s)) & 0xffu) % 3u);
      }
    }
  }

  // ---- doc section
  if constexpr (DOC_CH > 0) {
#pragma unroll
    for (int i = 0; i < DOC_CH; ++i) {
      const int c = i * 32 + lane;
      const int row = c / kDocRegs;
      const int piece = c - row * kDocRegs;
      if (row < cnt) st128_stream(out + row * out_b + piece * 16, dv[i]);
    }
  } else {
    copy_section<0>(sh.doc_ch, lane, cnt, out, out_b, doc_src);
  }

  // ---- edge section (Eq. 1: the matched row, or zeros)
  const uint8_t* edge_base = a.edge_feats + kb * edge_b;
  copy_section<EDGE_CH>(sh.edge_ch, lane, cnt, out + doc_b, out_b, [&](int row) -> const uint8_t* {
    const int rpos = __shfl_sync(kFull, pos, row);
    const unsigned rm = __shfl_sync(kFull, m, row);
    return (rm & 1u) ? edge_base + static_cast<long long>(rpos) * edge_b : nullptr;
  });

  // ---- edge2 section: the matched rows of the found engager slots, reduced per dim in slot order
  if (SECOND) {
    uint8_t* out2 = out + doc_b + edge_b;
    for (int ii = 0; ii < sh.edge_ch; ++ii) {
      const int c = ii * 32 + lane;
      const int row = c / sh.edge_ch;
      const int piece = c - row * sh.edge_ch;
      const unsigned rm = __shfl_sync(kFull, m, row);
      int rp[4];
#pragma unroll
      for (int s = 0; s < 4; ++s) rp[s] = __shfl_sync(kFull, apos[s], row);
      uint4 q[4];
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        q[s] = make_uint4(0u, 0u, 0u, 0u);
        if ((rm >> (1 + s)) & 1u) q[s] = ldg128(edge_base + static_cast<long long>(rp[s]) * edge_b + piece * 16);
      }
      float acc[8], bestf[8];
      unsigned short best[8];
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        acc[h] = 0.0f;
        bestf[h] = 0.0f;
        best[h] = 0;
      }
      bool any = false;
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        if ((rm >> (1 + s)) & 1u) {
          const unsigned w[4] = {q[s].x, q[s].y, q[s].z, q[s].w};
#pragma unroll
          for (int h = 0; h < 8; ++h) {
            const unsigned short bits = static_cast<unsigned short>((w[h >> 1] >> (16 * (h & 1))) & 0xffffu);
            const float f = __half2float(__ushort_as_half(bits));
            acc[h] = __fadd_rn(acc[h], f);  // one rounded fp32 add per found slot, never fused
            if (!any || f > bestf[h]) {     // strict >: the earlier slot keeps a tie
              bestf[h] = f;
              best[h] = bits;
            }
          }
          any = true;
        }
      }
      unsigned short res[8];
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        const int d = piece * 8 + h;
        const bool is_sum = (a.reduce_sum_mask >> (d & 63)) & 1ull;
        unsigned short sum_bits = __half_as_ushort(__float2half_rn(acc[h]));
        if (acc[h] != acc[h]) sum_bits = 0x7fffu;
        res[h] = any ? (is_sum ? sum_bits : best[h]) : static_cast<unsigned short>(0);
      }
      uint4 v;
      v.x = res[0] | (static_cast<unsigned>(res[1]) << 16);
      v.y = res[2] | (static_cast<unsigned>(res[3]) << 16);
      v.z = res[4] | (static_cast<unsigned>(res[5]) << 16);
      v.w = res[6] | (static_cast<unsigned>(res[7]) << 16);
      if (row < cnt) st128_stream(out2 + row * out_b + piece * 16, v);
    }
  }

  // ---- request section (one source row for the whole request)
  if (sh.req_ch) {
    const uint8_t* req_src = a.req_feats + static_cast<long long>(r) * sh.req_b;
    copy_section<((DOC_CH || EDGE_CH) ? REQ_CH : 0)>(sh.req_ch, lane, cnt, out + doc_b + edge_b * (SECOND ? 2 : 1), out_b,
                                                     [&](int) -> const uint8_t* { return req_src; });
  }

  if (lane < cnt) a.out_mask[jg + lane] = static_cast<uint8_t>(m);
}

// Index of the request that holds flat candidate j0 = number of requests that end at or before j0.
__device__ __forceinline__ int request_of(const int64_t* co, int n_req, long long j0) {
  int r = 0, n = n_req;
  while (n > 0) {
    const int half = n >> 1;
    if (__ldg(co + r + half + 1) <= j0) {
      r += half + 1;
      n -= half + 1;
    } else {
      n = half;
    }
  }
  return r;
}

// Key count of request r, clamped to what the host promised (so a malformed offset cannot widen a search).
__device__ __forceinline__ int request_keys(const JoinArgs& a, int r, long long& kb) {
  kb = __ldg(a.edge_offsets + r);
  long long K = __ldg(a.edge_offsets + r + 1) - kb;
  K = K < 0 ? 0 : (K > a.max_edge_len ? a.max_edge_len : K);
  return static_cast<int>(K);
}

// The bulk copy never signalled: record it, give the copy one more bounded chance to land so that the block
// does not retire with a transfer into its shared memory in flight, and let the block stop.
__device__ __forceinline__ void give_up_wait(const JoinArgs& a, uint32_t bar, uint32_t phase) {
  if (threadIdx.x == 0) {
    atomicExch(a.status, kDevWaitExpired);
    mbar_wait_bounded(bar, phase ^ 1u);
  }
  __syncthreads();
}

template <int DOC_CH, int EDGE_CH, int REQ_CH, bool SECOND>
__global__ void __launch_bounds__(kThreads, 2) join_kernel(const JoinArgs a) {
  extern __shared__ __align__(16) unsigned char smem[];
  int64_t* skeys = reinterpret_cast<int64_t*>(smem + kSmemHeader);
  const uint32_t bar = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const RowShape<DOC_CH, EDGE_CH, REQ_CH, SECOND> sh(a);

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
    if (rend <= seg) {  // request without candidates here
      ++r;
      continue;
    }
    const long long seg_end = min(rend, j1);
    long long kb;
    const int K = request_keys(a, r, kb);

    StagedKeys keys;
    if (!stage_keys(a, skeys, bar, phase, kb, K, keys)) {
      give_up_wait(a, bar, phase);
      return;
    }

    const long long nseg = seg_end - seg;
    for (long long g = static_cast<long long>(warp) * 32; g < nseg; g += kWarps * 32) {
      const int cnt = static_cast<int>(min(32LL, nseg - g));
      process_group<DOC_CH, EDGE_CH, REQ_CH, SECOND>(
          a, sh, keys, r, kb, seg + g, cnt, lane,
          [&](bool inr, int64_t auth, int& pos) -> bool { return inr && keys.find(auth, pos); });
    }
    __syncthreads();  // every warp is done with the staged keys before the next request overwrites them
    seg = seg_end;
    ++r;
  }
}

}  // namespace ccr
