// The fused join kernel: Algorithm 1 steps 2-4 (search, validate, gather) of the paper fused with the
// document-row gather from the resident index (Section 6.3.1) and the request-feature broadcast
// (Section 3), for a ragged batch of requests in one launch.
//
// Work split.  The kernel is persistent: the grid is a multiple of the SM count, every block owns one
// contiguous slice of the flat candidate range and walks the request segments inside it, so a request's
// keys are staged once per block.  Inside a segment the block alternates two phases over sub-tiles of
// `tile` candidates:
//   phase A, lane-per-candidate : position -> author id (8-byte gather) -> branch-free lower bound in the
//            staged keys -> (position, match index) into shared memory, mask byte to global memory.
//            Several candidates per thread are in flight at once, so the dependent chain
//            position -> id -> search is paid once per sub-tile, not once per row group.
//   phase B, warp-cooperative   : pure streaming.  Rows move as 16-byte chunks, consecutive lanes on
//            consecutive chunks of a row (the row's position / match index is a shared-memory broadcast);
//            all loads of a 32-row group are issued before its stores; every output byte is written
//            exactly once with full-sector streaming stores.
// Several blocks are resident per SM, so one block's phase A overlaps other blocks' phase B.
//
// Key staging and the search itself are in ccr_search.cuh (TMA bulk copy of the request's keys, bucket
// index, sampled top-of-tree for lists longer than the staging budget, global-memory search).
//
// Merge-path mode (MERGE = true; not in the paper) serves candidates whose author ids are non-decreasing
// inside each request: phase A gathers the sub-tile's author ids, finds with a block-cooperative k-ary
// search the window of keys the sub-tile can touch, stages only that window, and merges the two sorted
// runs along merge-path diagonals (O(n + w) comparisons instead of O(n log K)); phase B is unchanged.
#pragma once

#include "ccr_device.cuh"
#include "ccr_search.cuh"

namespace ccr {

constexpr long long kNoAuthor = static_cast<long long>(0x8000000000000000ull);  // below every key (keys are >= 0)

// One 16-byte chunk (8 fp16 dims, starting at dim piece*8) of the edge2 section of one candidate: the
// matched edge rows of its found engager slots (rp[s] >= 0 is the row index, < 0 = slot not found)
// reduced per dim in ascending slot order.  max: strict > on the fp32 values, the winner's 16 bits are
// kept.  sum: fp32 accumulator from +0, one rounded add per slot, one round-to-nearest-even conversion;
// a NaN sum is stored as 0x7fff.  Loading and reducing are separate so that a caller can put the loads of
// several chunks in flight before it reduces the first.
__device__ __forceinline__ void edge2_load(const uint8_t* edge_base, int edge_b, int piece, const int (&rp)[4],
                                           uint4 (&q)[4]) {
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    q[s] = make_uint4(0u, 0u, 0u, 0u);
    if (rp[s] >= 0) q[s] = ldg128(edge_base + static_cast<long long>(rp[s]) * edge_b + piece * 16);
  }
}

__device__ __forceinline__ uint4 edge2_reduce(unsigned long long reduce_sum_mask, int piece, const int (&rp)[4],
                                              const uint4 (&q)[4]) {
  // two fp16 dims per 32-bit word.  max: compare in fp16 (the same order as the fp32 values, conversions
  // being exact) and keep the winner's bits with a bit select; sum: fp32 accumulators.
  unsigned best[4] = {0u, 0u, 0u, 0u};
  float2 acc[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) acc[w] = make_float2(0.0f, 0.0f);
  bool any = false;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    if (rp[s] >= 0) {
      const unsigned v[4] = {q[s].x, q[s].y, q[s].z, q[s].w};
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const __half2 hv = *reinterpret_cast<const __half2*>(&v[w]);
        const float2 f = __half22float2(hv);
        acc[w].x = __fadd_rn(acc[w].x, f.x);  // one rounded fp32 add per found slot, never fused
        acc[w].y = __fadd_rn(acc[w].y, f.y);
        // strict >: the earlier slot keeps a tie; the first found slot always takes over
        const unsigned gt = any ? __hgt2_mask(hv, *reinterpret_cast<const __half2*>(&best[w])) : 0xffffffffu;
        best[w] = (v[w] & gt) | (best[w] & ~gt);
      }
      any = true;
    }
  }
  const unsigned sum8 = static_cast<unsigned>(reduce_sum_mask >> ((piece * 8) & 63)) & 0xffu;
  unsigned res[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const __half2 hs = __floats2half2_rn(acc[w].x, acc[w].y);
    unsigned sb = *reinterpret_cast<const unsigned*>(&hs);
    if (acc[w].x != acc[w].x) sb = (sb & 0xffff0000u) | 0x7fffu;
    if (acc[w].y != acc[w].y) sb = (sb & 0x0000ffffu) | 0x7fff0000u;
    const unsigned sel = (((sum8 >> (2 * w)) & 1u) ? 0x0000ffffu : 0u) | (((sum8 >> (2 * w + 1)) & 1u) ? 0xffff0000u : 0u);
    res[w] = any ? ((sb & sel) | (best[w] & ~sel)) : 0u;
  }
  return make_uint4(res[0], res[1], res[2], res[3]);
}

// Section widths of a launch, in 16-byte chunks and bytes (compile-time where the variant fixes them).
template <int DOC_CH, int EDGE_CH, int REQ_CH, bool SECOND, bool COS = false>
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
    out_b = doc_b + edge_b * (SECOND ? 2 : 1) + req_b + (COS ? kCosSectionBytes : 0);
  }
};

// Index of the request that holds flat candidate j0 = number of requests that end at or before j0.
__device__ __forceinline__ int request_of(const int64_t* co, int n_req, long long j0) {
  int r = 0, n = n_req;
  while (n > 0) {
    const int half = n >> 1;
    if (co[r + half + 1] <= j0) {
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
  kb = gload(a.edge_offsets + r);
  long long K = gload(a.edge_offsets + r + 1) - kb;
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

// Block-wide lower bound of `id` in ascending g[0..K): every thread probes one pivot per round.
// All threads must call; returns the same value in every thread.  Result is always within [0, K].
__device__ __forceinline__ int block_lower_bound(const int64_t* g, int K, int64_t id) {
  int lo = 0, n = K;
  while (n > 0) {
    const int step = (n + kThreads - 1) / kThreads;
    const long long p = static_cast<long long>(lo) + static_cast<long long>(threadIdx.x + 1) * step - 1;
    const int below = (p < lo + n) && (gload(g + p) < id);
    const int c = __syncthreads_count(below);
    const int nlo = min(lo + c * step, lo + n);
    n = min(step - 1, lo + n - nlo);
    lo = nlo;
  }
  return lo;
}

// Shared-memory layout of join_kernel, shared by host (sizing) and device (carving).
struct TileLayout {
  int off_idx, off_pos, off_apos, off_auth, off_keys, bytes;
  __host__ __device__ TileLayout(int tile, bool second, bool merge, int search_area) {
    off_idx = kSmemHeader;
    off_pos = off_idx + tile * 4;
    off_apos = off_pos + tile * 4;
    off_auth = off_apos + (second ? tile * 16 : 0);
    off_keys = off_auth + (merge ? tile * 8 : 0);
    off_keys = (off_keys + 15) & ~15;
    bytes = off_keys + search_area;
  }
};

// ---- phase B: 32 rows of one warp, everything already resolved in shared memory -------------------
// Derived section (Section 4.1.2) of the row held by this lane.  xv: the 16-byte pieces of the document row that
// hold the item embedding (element e of the embedding is half e of the pieces taken in order).  Dot product and
// squared norms are float32 fused-multiply-add chains over the elements in ascending order, exactly the order
// of the definition, so the result does not depend on how rows are spread over lanes.  cosM: element e ->
// (m_0[e], m_1[e], m_2[e], m_3[e]) as float32, cosM[kCosMaxDim] = the chunks' squared norms.
// TUNED: the embedding spans exactly NP pieces (cos_dim > 8 * (NP - 1)), so only the last piece needs the
// element bound; otherwise every piece is checked against the run-time width.  xrow: this lane's row in the
// warp's staging block.
template <int NP, bool TUNED>
__device__ __forceinline__ uint4 cosine_section(const JoinArgs& a, const uint4* xrow, const float4* cosM) {
  const int pieces = TUNED ? NP : (a.cos_dim + 7) >> 3;
  float nx = 0.0f, d[kCosMaxChunks] = {0.0f, 0.0f, 0.0f, 0.0f};
  uint4 xq[NP];  // the whole embedding is requested before the first element is used
#pragma unroll
  for (int q = 0; q < NP; ++q) xq[q] = q < pieces ? xrow[q] : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
  for (int q = 0; q < NP; ++q) {
    if (q >= pieces) break;  // warp-uniform
    // the eight medoid operands of the piece are requested together: one shared-memory latency per piece
    // instead of one per element in front of each group of dependent FMAs
    float4 m[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) m[t] = cosM[q * 8 + t];
    const unsigned w[4] = {xq[q].x, xq[q].y, xq[q].z, xq[q].w};
    float x[8];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[t]));
      x[2 * t] = f.x;
      x[2 * t + 1] = f.y;
    }
    const bool whole = TUNED && q < NP - 1;  // every element of the piece belongs to the embedding
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (whole || q * 8 + t < a.cos_dim) {
        nx = fmaf(x[t], x[t], nx);
        d[0] = fmaf(x[t], m[t].x, d[0]);
        d[1] = fmaf(x[t], m[t].y, d[1]);
        d[2] = fmaf(x[t], m[t].z, d[2]);
        d[3] = fmaf(x[t], m[t].w, d[3]);
      }
    }
  }
  const float4 nm4 = cosM[kCosMaxDim];
  const float nm[kCosMaxChunks] = {nm4.x, nm4.y, nm4.z, nm4.w};
  const float sx = sqrtf(nx);
  unsigned h[kCosMaxChunks];
#pragma unroll
  for (int k = 0; k < kCosMaxChunks; ++k) {
    float den = sx * sqrtf(nm[k]);
    if (!(den > 1e-8f)) den = 1e-8f;
    const float c = d[k] / den;
    h[k] = __half_as_ushort(__float2half_rn(c));
    if (c != c) h[k] = 0x7fffu;
    if (k >= a.cos_chunks) h[k] = 0u;
  }
  return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), 0u, 0u);
}

template <int DOC_CH, int EDGE_CH, int REQ_CH, bool SECOND, int CNP = 0>
__device__ __forceinline__ void emit_group(const JoinArgs& a, const RowShape<DOC_CH, EDGE_CH, REQ_CH, SECOND, CNP != 0>& sh,
                                           const int* s_idx, const int* s_pos, const int4* s_apos,
                                           const uint8_t* edge_base, const uint8_t* req_src, uint8_t* out, int cnt,
                                           int lane, const float4* cosM = nullptr, uint4* stage = nullptr,
                                           uint8_t* mask_out = nullptr, const unsigned* s_types = nullptr) {
  const long long out_b = sh.out_b;
  // mask bytes of the group (callers that resolved the candidates elsewhere and did not write them): lane = row;
  // bit 0 author found, bits 1-4 engager slot found, bits 5-7 engagement types of the found slots
  if (mask_out != nullptr && lane < cnt) {
    unsigned m = s_pos[lane] >= 0 ? 1u : 0u;
    if constexpr (SECOND) {
      const int4 ap4 = s_apos[lane];
      const int ap[4] = {ap4.x, ap4.y, ap4.z, ap4.w};
      const unsigned ty = s_types[lane];
#pragma unroll
      for (int sl = 0; sl < 4; ++sl)
        if (ap[sl] >= 0) m |= (1u << (1 + sl)) | (1u << (5 + ((ty >> (8 * sl)) & 0xffu) % 3u));
    }
    gstore(mask_out + lane, m);
  }
  // Derived section: the row streaming below is unchanged; the lanes that hold a piece of the item embedding
  // also drop it into this warp's staging block in shared memory (row-major, an odd number of 16-byte units
  // per row so that the read-back by lane = row is conflict-free), and once the group's stores are issued
  // every lane reads its row's embedding back and computes the cosines.
  constexpr bool kCos = CNP != 0;
  [[maybe_unused]] const int p0 = a.cos_first >> 3;
  [[maybe_unused]] const int np = CNP > 0 ? CNP : (a.cos_dim + 7) >> 3;
  [[maybe_unused]] const int sstride = np | 1;
  if constexpr (kCos) __syncwarp();  // the previous group's read-back is done before the block is rewritten
  if constexpr (DOC_CH > 0 && EDGE_CH > 0) {
    // every load of the group is issued before its first store
    uint4 dv[DOC_CH], ev[EDGE_CH];
#pragma unroll
    for (int i = 0; i < DOC_CH; ++i) {
      const int c = i * 32 + lane, row = c / DOC_CH, piece = c % DOC_CH;
      const int ridx = row < cnt ? s_idx[row] : -1;
      dv[i] = make_uint4(0u, 0u, 0u, 0u);
      if (ridx >= 0) dv[i] = ldg128_once(a.doc_feats + static_cast<long long>(ridx) * (DOC_CH * 16) + piece * 16);
    }
#pragma unroll
    for (int i = 0; i < EDGE_CH; ++i) {
      const int c = i * 32 + lane, row = c / EDGE_CH, piece = c % EDGE_CH;
      const int rpos = row < cnt ? s_pos[row] : -1;
      ev[i] = make_uint4(0u, 0u, 0u, 0u);
      if (rpos >= 0) ev[i] = ldg128(edge_base + static_cast<long long>(rpos) * (EDGE_CH * 16) + piece * 16);
    }
#pragma unroll
    for (int i = 0; i < DOC_CH; ++i) {
      const int c = i * 32 + lane, row = c / DOC_CH, piece = c % DOC_CH;
      if (row < cnt) st128_stream(out + row * out_b + piece * 16, dv[i]);
      if constexpr (kCos) {
        const int q = piece - p0;
        if (q >= 0 && q < np) stage[row * sstride + q] = dv[i];
      }
    }
#pragma unroll
    for (int i = 0; i < EDGE_CH; ++i) {
      const int c = i * 32 + lane, row = c / EDGE_CH, piece = c % EDGE_CH;
      if (row < cnt) st128_stream(out + row * out_b + DOC_CH * 16 + piece * 16, ev[i]);
    }
  } else {
    for (int i = 0; i < sh.doc_ch; ++i) {
      const int c = i * 32 + lane, row = c / sh.doc_ch, piece = c - row * sh.doc_ch;
      const int ridx = row < cnt ? s_idx[row] : -1;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (ridx >= 0) v = ldg128_once(a.doc_feats + static_cast<long long>(ridx) * sh.doc_b + piece * 16);
      if (row < cnt) st128_stream(out + row * out_b + piece * 16, v);
      if constexpr (kCos) {
        const int q = piece - p0;
        if (q >= 0 && q < np) stage[row * sstride + q] = v;
      }
    }
    for (int i = 0; i < sh.edge_ch; ++i) {
      const int c = i * 32 + lane, row = c / sh.edge_ch, piece = c - row * sh.edge_ch;
      const int rpos = row < cnt ? s_pos[row] : -1;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (rpos >= 0) v = ldg128(edge_base + static_cast<long long>(rpos) * sh.edge_b + piece * 16);
      if (row < cnt) st128_stream(out + row * out_b + sh.doc_b + piece * 16, v);
    }
  }
  // edge2 section: the matched rows of the found engager slots, reduced per dim in slot order
  if constexpr (SECOND) {
    auto slots_of = [&](int row, int (&rp)[4]) {
      rp[0] = rp[1] = rp[2] = rp[3] = -1;
      if (row < cnt) {
        const int4 p = s_apos[row];
        rp[0] = p.x;
        rp[1] = p.y;
        rp[2] = p.z;
        rp[3] = p.w;
      }
    };
    for (int i = 0; i < sh.edge_ch; ++i) {
      const int c = i * 32 + lane, row = c / sh.edge_ch, piece = c - row * sh.edge_ch;
      int rp[4];
      slots_of(row, rp);
      uint4 q[4];
      edge2_load(edge_base, sh.edge_b, piece, rp, q);
      const uint4 v = edge2_reduce(a.reduce_sum_mask, piece, rp, q);
      if (row < cnt) st128_stream(out + row * out_b + sh.doc_b + sh.edge_b + piece * 16, v);
    }
  }
  // request section: one source row for the whole request (L1/L2 hits)
  if (sh.req_ch) {
    const int off = sh.doc_b + sh.edge_b * (SECOND ? 2 : 1);
    for (int i = 0; i < sh.req_ch; ++i) {
      const int c = i * 32 + lane, row = c / sh.req_ch, piece = c - row * sh.req_ch;
      const uint4 v = ldg128(req_src + piece * 16);
      if (row < cnt) st128_stream(out + row * out_b + off + piece * 16, v);
    }
  }
  if constexpr (kCos) {
    constexpr int kPieces = CNP > 0 ? CNP : kCosMaxDim / 8;
    __syncwarp();
    const uint4 sec = cosine_section<kPieces, (CNP > 0)>(a, stage + lane * sstride, cosM);
    if (lane < cnt) {  // the section is one whole 32-byte sector: values, then zeros
      st128_stream(out + lane * out_b + out_b - kCosSectionBytes, sec);
      st128_stream(out + lane * out_b + out_b - kCosSectionBytes + 16, make_uint4(0u, 0u, 0u, 0u));
    }
  }
}

constexpr int kUnrollMax = 8;  // candidates a thread keeps in flight in phase A (4 in the variants that would spill with 8)
#ifndef CCR_JOIN_MIN_BLOCKS
#define CCR_JOIN_MIN_BLOCKS 2
#endif
constexpr int kJoinMinBlocks = CCR_JOIN_MIN_BLOCKS;  // resident blocks per SM the register budget is set for

// PADDED: rows go to slot r * n_max + (j - cand_offsets[r]) (JoinArgs::n_max > 0); a separate instantiation so
// that the ragged kernels carry no register for it.
template <int DOC_CH, int EDGE_CH, int REQ_CH, bool SECOND, bool MERGE, bool PADDED = false>
__global__ void __launch_bounds__(kThreads, kJoinMinBlocks) join_kernel(const JoinArgs a) {
  extern __shared__ __align__(16) unsigned char smem[];
  const TileLayout lay(a.tile, SECOND, MERGE, a.search_area);
  int* s_idx = reinterpret_cast<int*>(smem + lay.off_idx);
  int* s_pos = reinterpret_cast<int*>(smem + lay.off_pos);
  int4* s_apos = reinterpret_cast<int4*>(smem + lay.off_apos);
  int64_t* s_auth = reinterpret_cast<int64_t*>(smem + lay.off_auth);
  const SearchSmem ssm = carve_search(smem + lay.off_keys, a.search_area, !MERGE);
  const BlockGroup grp;
  const uint32_t bar = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const RowShape<DOC_CH, EDGE_CH, REQ_CH, SECOND> sh(a);
  // (the generic-width and the wide-row second-degree variants would spill with eight candidates of a thread in
  // flight in phase A)
  constexpr int kUnroll = (SECOND && (DOC_CH == 0 || EDGE_CH >= 8)) ? 4 : kUnrollMax;

  if (tid == 0) {
    mbar_init(bar, 1);
    fence_proxy_async_smem();
  }
  __syncthreads();
  uint32_t phase = 0;

  // this block's contiguous slice of the flat candidate range, in whole groups of 32
  const long long groups = (a.total + 31) >> 5;
  const long long per = (groups + gridDim.x - 1) / gridDim.x;
  const long long j0 = min(a.total, static_cast<long long>(blockIdx.x) * per * 32);
  const long long j1 = min(a.total, j0 + per * 32);
  if (j0 >= j1) return;
  int r = request_of(a.cand_offsets, a.n_req, j0);

  long long seg = j0;
  while (seg < j1 && r < a.n_req) {
    const long long rend = gload(a.cand_offsets + r + 1);
    if (rend <= seg) {  // request without candidates here
      ++r;
      continue;
    }
    const long long seg_end = min(rend, j1);
    long long kb;
    const int K = request_keys(a, r, kb);
    const uint8_t* edge_base = a.edge_feats + kb * sh.edge_b;
    const uint8_t* req_src = sh.req_ch ? a.req_feats + static_cast<long long>(r) * sh.req_b : nullptr;

    StagedKeys keys;
    if (!MERGE) {
      // lookups this block will make against the list: its candidates of the request (second degree: up to five ids each)
      if (!stage_keys(a, ssm, bar, phase, kb, K, true, (seg_end - seg) * (SECOND ? 3 : 1), keys, grp)) {
        give_up_wait(a, bar, phase);
        return;
      }
    }

    // padded output: a request's candidates behind its n_max-th have no slot and are dropped
    const long long r_first = PADDED ? gload(a.cand_offsets + r) : 0;
    const long long seg_lim = PADDED ? min(seg_end, r_first + a.n_max) : seg_end;
    for (long long sub = seg; sub < seg_lim; sub += a.tile) {
      const int n = static_cast<int>(min(static_cast<long long>(a.tile), seg_lim - sub));
      const long long out0 = PADDED ? r * a.n_max + (sub - r_first) : sub;

      // ================= phase A: resolve every candidate of the sub-tile =================
      if (!MERGE) {
        for (int base = 0; base < n; base += kThreads * kUnroll) {
          int idx[kUnroll];
          int64_t auth[kUnroll];
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int i = base + u * kThreads + tid;
            idx[u] = i < n ? gload(a.cand_idx + sub + i) : -1;
          }
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            if (idx[u] < 0 || idx[u] >= a.n_docs) idx[u] = -1;  // unresolved / out-of-range position
            auth[u] = idx[u] >= 0 ? load_author(a, idx[u]) : -1;
          }
          bool found[kUnroll];
          int pos[kUnroll];
          static_assert(kUnroll % 4 == 0, "lookups are interleaved four at a time");
#pragma unroll
          for (int h = 0; h < kUnroll; h += 4) {
            const int64_t id4[4] = {auth[h], auth[h + 1], auth[h + 2], auth[h + 3]};
            bool f4[4];
            int p4[4];
            keys.find_batch<4>(id4, f4, p4);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              found[h + q] = f4[q];
              pos[h + q] = p4[q];
            }
          }
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int i = base + u * kThreads + tid;
            if (i >= n) continue;
            unsigned m = found[u] ? 1u : 0u;
            if (SECOND) {
              int64_t act[4] = {-1, -1, -1, -1};
              unsigned types = 0;
              if (idx[u] >= 0) {
                long long rec[4];
                load_actors(a, idx[u], rec, types);
#pragma unroll
                for (int sl = 0; sl < 4; ++sl) act[sl] = sl < a.max_actors ? rec[sl] : -1;
              }
              bool af[4];
              int ap[4];
              keys.find_batch<4>(act, af, ap);
#pragma unroll
              for (int sl = 0; sl < 4; ++sl) {
                if (af[sl]) {
                  m |= 1u << (1 + sl);
                  m |= 1u << (5 + ((types >> (8 * sl)) & 0xffu) % 3u);
                } else {
                  ap[sl] = -1;
                }
              }
              s_apos[i] = make_int4(ap[0], ap[1], ap[2], ap[3]);
            }
            s_idx[i] = idx[u];
            s_pos[i] = found[u] ? pos[u] : -1;
            gstore(a.out_mask + out0 + i, m);
          }
        }
      } else {
        // 1. author ids of the sub-tile
        int bad = 0;
        for (int base = 0; base < n; base += kThreads * kUnroll) {
          int idx[kUnroll];
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int i = base + u * kThreads + tid;
            idx[u] = i < n ? gload(a.cand_idx + sub + i) : -1;
          }
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int i = base + u * kThreads + tid;
            if (idx[u] < 0 || idx[u] >= a.n_docs) idx[u] = -1;
            if (i < n) {
              bad |= idx[u] < 0;
              s_idx[i] = idx[u];
              s_auth[i] = idx[u] >= 0 ? load_author(a, idx[u]) : kNoAuthor;
            }
          }
        }
        // An unresolved / out-of-range position has no author, so a sub-tile that holds one is not a sorted run
        // (the sortedness promise is over author ids): it takes the per-candidate search below instead of the merge.
        const bool any_invalid = __syncthreads_or(bad);
        // 2. the only keys this sub-tile can touch: window [lo, hi)
        const int64_t* gk = a.edge_keys + kb;
        const int lo = block_lower_bound(gk, K, s_auth[0]);
        const int hi = min(K, block_lower_bound(gk, K, s_auth[n - 1]) + 1);
        const int w = max(hi - lo, 0);
        const bool windowed = (a.key_cap > 0) && (w <= a.key_cap) && (search_keys_bytes(w) <= a.search_area) &&
                              (a.min_stride_log2 == 0) && !any_invalid;
        // 3. stage the window (or, if it is too long, the request's keys as the binary-search mode does)
        if (!stage_keys(a, ssm, bar, phase, windowed ? kb + lo : kb, windowed ? w : K, false, 0, keys, grp)) {
          give_up_wait(a, bar, phase);
          return;
        }
        if (windowed) {
          // 4. merge path over (s_auth[0..n), window[0..w)); a candidate goes before an equal key, so the
          //    keys consumed when it is emitted are exactly the keys below it
          const int64_t* B = keys.sk;
          const int total = n + w;
          const int L = (total + kThreads - 1) / kThreads;
          const int diag = min(tid * L, total);
          int ab = max(0, diag - w), ae = min(diag, n);
          while (ab < ae) {
            const int mid = (ab + ae) >> 1;
            if (s_auth[mid] <= B[diag - 1 - mid]) ab = mid + 1; else ae = mid;
          }
          int ai = ab, bi = diag - ab;
          for (int step = 0; step < L && (ai < n || bi < w); ++step) {
            if (ai < n && (bi >= w || s_auth[ai] <= B[bi])) {
              const bool hit = bi < w && B[bi] == s_auth[ai] && s_idx[ai] >= 0;
              s_pos[ai] = hit ? lo + bi : -1;
              ++ai;
            } else {
              ++bi;
            }
          }
          __syncthreads();
          // under a broken sortedness promise a slot may not have been written by the merge: bound it
          for (int i = tid; i < n; i += kThreads) {
            int p = s_pos[i];
            if (p >= K) p = -1;
            s_pos[i] = p;
            gstore(a.out_mask + out0 + i, p >= 0 ? 1 : 0);
          }
        } else {
          for (int i = tid; i < n; i += kThreads) {
            int pos = 0;
            const bool found = s_idx[i] >= 0 && keys.find(s_auth[i], pos);
            s_pos[i] = found ? pos : -1;
            gstore(a.out_mask + out0 + i, found ? 1 : 0);
          }
        }
      }
      __syncthreads();

      // ================= phase B: stream the rows =================
      for (int g = warp * 32; g < n; g += kWarps * 32) {
        emit_group<DOC_CH, EDGE_CH, REQ_CH, SECOND>(a, sh, s_idx + g, s_pos + g, s_apos + g, edge_base, req_src,
                                                                       a.out_rows + (out0 + g) * sh.out_b, min(32, n - g), lane);
      }
      __syncthreads();  // phase A of the next sub-tile overwrites the resolved arrays (and, in merge mode, the keys)
    }
    seg = seg_end;
    ++r;
  }
}

}  // namespace ccr
