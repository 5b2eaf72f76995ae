// Warp-specialised variant of the fused join (same result as join_kernel).
//
// In join_kernel every warp alternates between resolving candidates (position -> author id -> search: two
// dependent memory accesses plus a shared-memory search) and streaming rows; while a block resolves, its
// share of the memory pipeline idles.  Here the two jobs run concurrently in one persistent block per SM:
//   resolver warps : take chunks of the flat candidate range, stage each request's keys (TMA bulk copy +
//                    mbarrier, waited on by the resolvers only), and fill a ring of sub-tile buffers in
//                    shared memory with (position, match index) per candidate; they write nothing to global
//                    memory.  Their latency (ids are 8-byte gathers, key staging) hides behind the streaming.
//   streamer warps : consume the ring; for every 32-row group the mask bytes are derived from the match
//                    indices, all loads are issued, then all stores — nothing else.  They never touch keys,
//                    ids or barriers other than the ring's.
// Ring slots are handed over with shared-memory mbarriers: full[slot] (one arrival, by the resolvers, once the
// slot is written) and empty[slot] (one arrival per streamer warp, once it has taken its last group of the
// slot).  Warps wait on them individually — a streamer warp that is done with a slot moves on to the next
// full slot without waiting for its siblings — and every wait is bounded: on expiry the warp records
// kDevWaitExpired and leaves.  A slot with n == 0 tells the streamers to stop.  Inside a slot the streamer
// warps take 32-row groups one at a time from a shared-memory counter.
//
// Work distribution.  With a scheduling word (JoinArgs::sched) the resolvers of all blocks draw chunks of
// consecutive tiles from one global counter; the chunk shrinks from kMaxRounds tiles per resolver warp to one
// as the launch drains (guided self-scheduling), so blocks on slower SMs or with costlier requests simply take
// fewer chunks and all blocks finish within about one tile of each other.  The last block to finish puts
// the two scheduling words back to zero for the next launch.  Without a scheduling word every block takes
// one equal contiguous slice.  (Contiguous slices with work stealing between them — fewer key stagings per block —
// were measured and lost 7-9 % on every configuration: all blocks walking one window of the candidate range
// together is what the memory system likes.)
#pragma once

#include "ccr_join.cuh"

namespace ccr {

constexpr int kWsSlots = 8;        // ring depth
constexpr int kWsMaxThreads = 512;
// Register-rebalanced form (second-degree joins, whose resolvers are the bottleneck): 12 streamer + 8 resolver
// warps = 640 threads.  The block is launched with 96 registers per thread (the most 640 threads can have); the
// resolver warpgroups then give registers back (setmaxnreg.dec) and the streamer warpgroups take them
// (setmaxnreg.inc).  Registers only move inside the block's own allocation, and an increase waits until they are
// there, so 384 x kRebalStreamerRegs + 256 x kRebalResolverRegs must not exceed 640 x 96 — more would never
// arrive.  Eight resolvers fill eight ring slots at a time, so the ring is twice as deep (of half-size slots).
#ifndef CCR_REBAL_STREAMERS
#define CCR_REBAL_STREAMERS 12
#endif
#ifndef CCR_REBAL_RESOLVERS
#define CCR_REBAL_RESOLVERS 8
#endif
constexpr int kRebalStreamers = CCR_REBAL_STREAMERS, kRebalResolvers = CCR_REBAL_RESOLVERS;
constexpr int kRebalThreads = (kRebalStreamers + kRebalResolvers) * 32;
#ifndef CCR_REBAL_STREAMER_REGS
#define CCR_REBAL_STREAMER_REGS 104
#endif
#ifndef CCR_REBAL_RESOLVER_REGS
#define CCR_REBAL_RESOLVER_REGS 80
#endif
constexpr int kRebalStreamerRegs = CCR_REBAL_STREAMER_REGS, kRebalResolverRegs = CCR_REBAL_RESOLVER_REGS;
constexpr int kRebalLaunchRegs = 96;  // 65,536 / 640 rounded down to the allocation unit of 8
static_assert(kRebalStreamers * 32 * kRebalStreamerRegs + kRebalResolvers * 32 * kRebalResolverRegs <= kRebalThreads * kRebalLaunchRegs,
              "the registers the streamers take must be the ones the resolvers give back");
static_assert(kRebalStreamerRegs >= kRebalLaunchRegs && kRebalResolverRegs <= kRebalLaunchRegs && kRebalStreamerRegs % 8 == 0 &&
              kRebalResolverRegs % 8 == 0, "inc raises, dec lowers, both in units of 8");
static_assert(kRebalStreamers % 4 == 0 && kRebalResolvers % 4 == 0, "setmaxnreg acts on whole warpgroups");
constexpr int kRebalSlots = 16;
constexpr int kRebalInFlight = 2;   // candidates a resolver lane keeps in flight (twice the warps, half the registers)
constexpr int kWsMaxCachedReq = 1024;  // batches up to this many requests keep their offsets in shared memory
#ifndef CCR_MAX_ROUNDS
#define CCR_MAX_ROUNDS 4
#endif
constexpr int kMaxRounds = CCR_MAX_ROUNDS;  // most tiles per resolver warp a block draws at once
constexpr int kMaxTileCands = 4096;  // largest sub-tile the host accepts
constexpr int kWsWorkItems = 4 * 32 * 4;  // engager slots of one resolver batch: 4 candidates per lane x 4 slots
constexpr int kWsWorkListBytes = kWsWorkItems * (8 + 2);  // ids (int64) + tags (uint16) per resolver warp

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

struct WsSlot {          // descriptor of one ring slot
  long long sub;         // first flat candidate of the sub-tile
  long long out0;        // output row of that candidate (= sub for the ragged layout)
  long long kb;          // first key / edge row of its request
  int n;                 // candidates in the sub-tile (0 = stop)
  int r;                 // request index
  int next;              // next 32-row group a streamer warp may take (reset by the resolvers)
  int pad;
  int cos_r;             // request whose member block the slot's cosine buffer holds (-1 = none)
  int pad2;
};

__host__ __device__ inline int ws_cos_bytes(int n_streamers, int stage_per_warp) {
  return kWsSlots * kCosSlotFloat4 * 16 + n_streamers * stage_per_warp;
}

struct WsLayout {
  int off_full, off_empty, off_slots, off_grab, off_offs, off_idx, off_pos, off_apos, off_types, off_cos, off_wl, off_keys, bytes;
  // n_req_cached: requests whose offsets are mirrored in shared memory (0 = read them from global memory)
  // cos_bytes: shared memory of the derived cosine section (0 = off): a block of member-embedding floats per
  // ring slot, then one embedding staging block per streamer warp
  // n_res: resolver warps (second-degree joins give each a work list of engager lookups)
  __host__ __device__ WsLayout(int tile, bool second, int search_area, int n_req_cached, int cos_bytes, int n_res,
                               int n_slots = kWsSlots, int wl_items = kWsWorkItems) {
    off_full = kSmemHeader;                 // after the key-staging mbarrier
    off_empty = off_full + n_slots * 8;
    off_slots = off_empty + n_slots * 8;
    off_grab = off_slots + n_slots * static_cast<int>(sizeof(WsSlot));
    off_offs = off_grab + 16;
    off_idx = off_offs + (n_req_cached > 0 ? 2 * (n_req_cached + 1) * 8 : 0);
    off_idx = (off_idx + 15) & ~15;
    off_pos = off_idx + n_slots * tile * 4;
    off_apos = off_pos + n_slots * tile * 4;
    off_types = off_apos + (second ? n_slots * tile * 16 : 0);
    off_cos = off_types + (second ? n_slots * tile * 4 : 0);
    off_wl = off_cos + cos_bytes;
    off_keys = off_wl + (second ? n_res * wl_items * (8 + 2) : 0);
    off_keys = (off_keys + 15) & ~15;
    bytes = off_keys + search_area;
  }
};

// CNP: 0 = no derived section; > 0 = the item embedding spans exactly CNP 16-byte pieces (tuned); < 0 = any shape
template <int DOC_CH, int EDGE_CH, int REQ_CH, bool SECOND, int CNP = 0, bool REBAL = false>
__global__ void __launch_bounds__(REBAL ? kRebalThreads : kWsMaxThreads, 1) join_ws_kernel(const JoinArgs a, int n_streamers) {
  extern __shared__ __align__(16) unsigned char smem_ws[];
  unsigned char* smem = smem_ws;
  constexpr bool COS = CNP != 0;
  constexpr int kSlots = REBAL ? kRebalSlots : kWsSlots;
  static_assert(!(REBAL && COS), "the rebalanced form carries no cosine section");
  const int n_req_cached = a.n_req <= kWsMaxCachedReq ? a.n_req : 0;
  const WsLayout lay(a.tile, SECOND, a.search_area, n_req_cached, COS ? ws_cos_bytes(n_streamers, a.cos_stage) : 0,
                     (static_cast<int>(blockDim.x) >> 5) - n_streamers, kSlots, REBAL ? kRebalInFlight * 128 : kWsWorkItems);
  WsSlot* slots = reinterpret_cast<WsSlot*>(smem + lay.off_slots);
  int* grab = reinterpret_cast<int*>(smem + lay.off_grab);
  int* s_idx = reinterpret_cast<int*>(smem + lay.off_idx);
  int* s_pos = reinterpret_cast<int*>(smem + lay.off_pos);
  int4* s_apos = reinterpret_cast<int4*>(smem + lay.off_apos);
  unsigned* s_types = reinterpret_cast<unsigned*>(smem + lay.off_types);
  float4* s_cos = reinterpret_cast<float4*>(smem + lay.off_cos);
  const SearchSmem ssm = carve_search(smem + lay.off_keys, a.search_area, true);
  const uint32_t bar = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_threads = blockDim.x;
  const RowShape<DOC_CH, EDGE_CH, REQ_CH, SECOND, COS> sh(a);
  const uint32_t full0 = smem_u32(smem + lay.off_full), empty0 = smem_u32(smem + lay.off_empty);
  const int kBarGroup = 1;  // named barrier of the resolver group

  // offsets of the batch, mirrored once per block: every chunk starts with a search over them
  const int64_t* co = a.cand_offsets;
  const int64_t* eo = a.edge_offsets;
  if (n_req_cached > 0) {
    int64_t* s_co = reinterpret_cast<int64_t*>(smem + lay.off_offs);
    int64_t* s_eo = s_co + (a.n_req + 1);
    for (int i = tid; i <= a.n_req; i += n_threads) {
      s_co[i] = gload(a.cand_offsets + i);
      s_eo[i] = gload(a.edge_offsets + i);
    }
    co = s_co;
    eo = s_eo;
  }
  if (tid == 0) {
    mbar_init(bar, 1);
    for (int s = 0; s < kSlots; ++s) {
      slots[s].cos_r = -1;
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, static_cast<uint32_t>(n_streamers));
    }
    fence_proxy_async_smem();
  }
  __syncthreads();

  // static split (no scheduling word): this block's contiguous slice, in whole groups of 32
  const long long groups = (a.total + 31) >> 5;
  const long long per = (groups + gridDim.x - 1) / gridDim.x;
  const long long slice0 = min(a.total, static_cast<long long>(blockIdx.x) * per * 32);
  const long long slice1 = min(a.total, slice0 + per * 32);
  if (a.sched == nullptr && slice0 >= slice1) return;  // block-uniform, before any named barrier

  const int n_res = (n_threads >> 5) - n_streamers;
  const int role_rank = (n_threads >> 5) - 1 - warp;  // resolvers are the last n_res warps
  if (role_rank >= n_res) {
    // ============================ streamers ============================
    if constexpr (REBAL) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRebalStreamerRegs));
    // this warp's embedding staging block (derived cosine section), behind the per-slot member blocks
    [[maybe_unused]] uint4* cos_stage = reinterpret_cast<uint4*>(
        smem + lay.off_cos + kWsSlots * kCosSlotFloat4 * 16 + (role_rank - n_res) * (COS ? a.cos_stage : 0));
    for (unsigned it = 0;; ++it) {
      const int s = it % kSlots;
      if (!mbar_wait_bounded(full0 + 8 * s, (it / kSlots) & 1u)) {
        if (lane == 0) atomicExch(a.status, kDevWaitExpired);
        return;
      }
      const WsSlot d = slots[s];
      if (d.n == 0) break;
      if (it == 0) pdl_wait();  // the first rows are about to be written: the launch before this one must be done
      const uint8_t* edge_base = a.edge_feats + d.kb * sh.edge_b;
      const uint8_t* req_src = sh.req_ch ? a.req_feats + static_cast<long long>(d.r) * sh.req_b : nullptr;
      const int* idx = s_idx + s * a.tile;
      const int* pos = s_pos + s * a.tile;
      const int4* apos = s_apos + s * a.tile;
      const unsigned* types = s_types + s * a.tile;
      // groups are handed out one at a time, so a warp that finishes early simply takes more
      for (;;) {
        int g = 0;
        if (lane == 0) g = atomicAdd(&slots[s].next, 1);
        g = __shfl_sync(kFull, g, 0) * 32;
        if (g >= d.n) break;
        emit_group<DOC_CH, EDGE_CH, REQ_CH, SECOND, CNP>(a, sh, idx + g, pos + g, apos + g, edge_base, req_src,
                                                         a.out_rows + (d.out0 + g) * sh.out_b, min(32, d.n - g), lane,
                                                         COS ? s_cos + s * kCosSlotFloat4 : nullptr,
                                                         COS ? cos_stage : nullptr, a.out_mask + d.out0 + g, types + g);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
    }
    return;
  }

  // ============================ resolvers ============================
  if constexpr (REBAL) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRebalResolverRegs));
  // All resolver warps walk the same sequence of sub-tiles; warp q fills every n_resolvers-th one on its own
  // (own bounded wait for the slot, own publish), so several sub-tiles are being resolved at any time.  They
  // meet on a named barrier only to draw the next chunk and to stage a new request's keys.
  const int gsize = n_res * 32;
  const int gtid = role_rank * 32 + lane;
  const int n_resolvers = gsize >> 5;
  const int rwarp = gtid >> 5;
  const NamedGroup grp(gtid, gsize, kBarGroup);
  uint32_t phase = 0;
  unsigned it = 0;       // sub-tiles walked so far (= ring slots handed out)
  bool failed = false;   // key staging gave up (group-uniform): stop drawing work
  bool dead = false;     // this warp's wait for a free slot expired: keep walking (barriers!), fill nothing
  int staged_r = -1;     // request whose keys are in shared memory
  StagedKeys keys;
  keys.declined = false;
  // this warp's work list of engager lookups (second-degree joins)
  constexpr int U = SECOND ? (REBAL ? kRebalInFlight : 4) : 8;  // candidates a lane keeps in flight
  constexpr int FB = U < 4 ? U : 4;                              // lookups interleaved in one find_batch
  constexpr int FBW = FB;                                        // ... of the engager work list (wider was slower)
  constexpr int kWlItems = U * 32 * 4;                           // every engager slot of one batch
  [[maybe_unused]] int64_t* wl_id = reinterpret_cast<int64_t*>(smem + lay.off_wl + (SECOND ? rwarp * kWlItems * (8 + 2) : 0));
  [[maybe_unused]] uint16_t* wl_tag = reinterpret_cast<uint16_t*>(wl_id + kWlItems);
  int cos_r = -1;        // request whose squared member norms lane k < kCosMaxChunks holds in cos_nm
  float cos_nm = 0.0f;
  const long long n_tiles = (a.total + a.tile - 1) / a.tile;
  static_assert(REBAL || !SECOND || kWlItems == kWsWorkItems, "the work list holds every engager slot of one batch");
  static_assert(kMaxTileCands * 4 <= 65536, "work-list tags are 16 bits: candidate index in the tile x 4 + slot");

  for (bool more = true; more && !failed;) {
    long long j0, j1;
    if (a.sched != nullptr) {
      if (gtid == 0) {
        // a chunk is a whole number of rounds (one tile per resolver warp), so the warps meet at the next
        // draw having done the same amount of work; rounds shrink from kMaxRounds to 1 as the launch drains
        const long long rem = n_tiles - *reinterpret_cast<volatile int*>(a.sched);
        long long m = rem / (2LL * gridDim.x * n_resolvers);
        m = m < 1 ? 1 : (m > kMaxRounds ? kMaxRounds : m);
        const long long c = m * n_resolvers;
        grab[0] = atomicAdd(a.sched, static_cast<int>(c));
        grab[1] = static_cast<int>(c);
      }
      grp.sync();
      const long long t = grab[0], c = grab[1];
      grp.sync();
      if (t >= n_tiles) break;
      j0 = t * a.tile;
      j1 = min(a.total, (t + c) * a.tile);
    } else {
      j0 = slice0;
      j1 = slice1;
      more = false;
    }

    int r = request_of(co, a.n_req, j0);
    long long seg = j0;
    while (seg < j1 && r < a.n_req && !failed) {
      const long long rend = co[r + 1];
      if (rend <= seg) {  // request without candidates here
        ++r;
        continue;
      }
      const long long seg_end = min(rend, j1);
      const long long kb = eo[r];
      const int K = static_cast<int>(min(max(eo[r + 1] - kb, 0LL), static_cast<long long>(a.max_edge_len)));
      const long long n_look = (seg_end - seg) * (SECOND ? 3 : 1);
      // (a list staged without a table for a short tail gets one when a longer run of the same request follows)
      if (r != staged_r || (keys.declined && n_look * kTableAmort >= K)) {
        // lookups the resolvers will make against the list before the next staging: this chunk's candidates of the
        // request (second degree: up to five ids each, about three on the benchmark stores)
        if (!stage_keys(a, ssm, bar, phase, kb, K, true, n_look, keys, grp)) {
          if (gtid == 0) {
            atomicExch(a.status, kDevWaitExpired);
            mbar_wait_bounded(bar, phase ^ 1u);
          }
          failed = true;
          break;
        }
        staged_r = r;
      }
      // padded output: a request's candidates behind its n_max-th have no slot and are dropped
      const long long seg_lim = a.n_max > 0 ? min(seg_end, co[r] + a.n_max) : seg_end;
      for (long long sub = seg; sub < seg_lim; sub += a.tile, ++it) {
        if (static_cast<int>(it % n_resolvers) != rwarp || dead) continue;
        const int n = static_cast<int>(min(static_cast<long long>(a.tile), seg_lim - sub));
        const int s = it % kSlots;
        if (it >= static_cast<unsigned>(kSlots) && !mbar_wait_bounded(empty0 + 8 * s, (it / kSlots - 1) & 1u)) {
          if (lane == 0) atomicExch(a.status, kDevWaitExpired);
          dead = true;  // the streamers are gone
          continue;
        }
        const long long out0 = a.n_max > 0 ? r * a.n_max + (sub - co[r]) : sub;
        int* out_idx = s_idx + s * a.tile;
        int* out_pos = s_pos + s * a.tile;
        int4* out_apos = s_apos + s * a.tile;
        [[maybe_unused]] unsigned* out_types = s_types + s * a.tile;
        for (int base = 0; base < n; base += 32 * U) {
          int idx[U];
          int64_t auth[U];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const int i = base + u * 32 + lane;
            idx[u] = i < n ? gload(a.cand_idx + sub + i) : -1;
          }
          // every id of the U candidates is requested before the first one is used
          int64_t act[SECOND ? U : 1][4];
          unsigned types[SECOND ? U : 1];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            if (idx[u] < 0 || idx[u] >= a.n_docs) idx[u] = -1;  // unresolved / out-of-range position
            if constexpr (SECOND) {
              auth[u] = -1;
              act[u][0] = act[u][1] = act[u][2] = act[u][3] = -1;
              types[u] = 0;
              if (idx[u] >= 0) {
                long long rec[4], au;
                load_record(a, idx[u], au, rec, types[u]);
                auth[u] = au;
#pragma unroll
                for (int sl = 0; sl < 4; ++sl) act[u][sl] = sl < a.max_actors ? rec[sl] : -1;
              }
            } else {
              auth[u] = idx[u] >= 0 ? load_author(a, idx[u]) : -1;
            }
          }
          bool found[U];
          int pos[U];
#pragma unroll
          for (int h = 0; h < U; h += FB) {
            int64_t idq[FB];
            bool fq[FB];
            int pq[FB];
#pragma unroll
            for (int q = 0; q < FB; ++q) idq[q] = auth[h + q];
            keys.find_batch<FB>(idq, fq, pq);
#pragma unroll
            for (int q = 0; q < FB; ++q) {
              found[h + q] = fq[q];
              pos[h + q] = pq[q];
            }
          }
          if constexpr (SECOND) {
            // Engager lookups.  Most slots are empty, and which ones differs from lane to lane, so looking up
            // "slot s of candidate u" in lock step would spend most of the warp's instructions on empty
            // slots.  The non-empty (candidate, slot) pairs of the batch are compacted into a work list in
            // shared memory (lane-major, so workers read consecutive entries) and the lanes share them out,
            // four interleaved lookups at a time; a hit writes its key index straight into the slot's
            // position array, which the owner lane has preset to -1.
            int* apos_i = reinterpret_cast<int*>(out_apos);
            int mine = 0;
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const int i = base + u * 32 + lane;
              if (i < n) out_apos[i] = make_int4(-1, -1, -1, -1);
#pragma unroll
              for (int sl = 0; sl < 4; ++sl) mine += act[u][sl] >= 0 ? 1 : 0;
            }
            int incl = mine;
#pragma unroll
            for (int dlt = 1; dlt < 32; dlt <<= 1) {
              const int t = __shfl_up_sync(kFull, incl, dlt);
              if (lane >= dlt) incl += t;
            }
            const int total = __shfl_sync(kFull, incl, 31);
            int w = incl - mine;
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
              for (int sl = 0; sl < 4; ++sl) {
                if (act[u][sl] >= 0) {
                  wl_id[w] = act[u][sl];
                  wl_tag[w] = static_cast<uint16_t>(((base + u * 32 + lane) << 2) | sl);
                  ++w;
                }
              }
            }
            __syncwarp();
            for (int w0 = 0; w0 < total; w0 += FBW * 32) {
              int64_t idq[FBW];
#pragma unroll
              for (int q = 0; q < FBW; ++q) {
                const int wi = w0 + q * 32 + lane;
                idq[q] = wi < total ? wl_id[wi] : -1;
              }
              bool fq[FBW];
              int pq[FBW];
              keys.find_batch<FBW>(idq, fq, pq);
#pragma unroll
              for (int q = 0; q < FBW; ++q) {
                const int wi = w0 + q * 32 + lane;
                if (wi < total && fq[q]) apos_i[wl_tag[wi]] = pq[q];
              }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const int i = base + u * 32 + lane;
              if (i < n) {
                out_idx[i] = idx[u];
                out_pos[i] = found[u] ? pos[u] : -1;
                out_types[i] = types[u];  // the streamers derive the mask byte from the match indices and these
              }
            }
          } else {
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const int i = base + u * 32 + lane;
              if (i < n) {
                out_idx[i] = idx[u];
                out_pos[i] = found[u] ? pos[u] : -1;
              }
            }
          }
        }
        if constexpr (COS) {
          // the request's medoid embeddings as float32, element-major, for the streamers of this slot; a slot
          // that already holds this request's block (tiles of one request follow each other) keeps it
          float4* M = s_cos + s * kCosSlotFloat4;
          if (slots[s].cos_r != r) {
            const uint16_t* mem = a.member_emb + static_cast<long long>(r) * a.cos_chunks * a.cos_dim;
            for (int e = lane; e < kCosMaxDim; e += 32) {
              float m[kCosMaxChunks] = {0.0f, 0.0f, 0.0f, 0.0f};
              if (e < a.cos_dim) {
#pragma unroll
                for (int k = 0; k < kCosMaxChunks; ++k)
                  if (k < a.cos_chunks) m[k] = __half2float(__ushort_as_half(gload(mem + k * a.cos_dim + e)));
              }
              M[e] = make_float4(m[0], m[1], m[2], m[3]);
            }
            if (r != cos_r) {  // squared norms: lane k sums chunk k in element order, once per request and warp
              cos_nm = 0.0f;
              if (lane < a.cos_chunks) {
                for (int e = 0; e < a.cos_dim; ++e) {
                  const float v = __half2float(__ushort_as_half(gload(mem + lane * a.cos_dim + e)));
                  cos_nm = fmaf(v, v, cos_nm);
                }
              }
              cos_r = r;
            }
            const float n0 = __shfl_sync(kFull, cos_nm, 0), n1 = __shfl_sync(kFull, cos_nm, 1);
            const float n2 = __shfl_sync(kFull, cos_nm, 2), n3 = __shfl_sync(kFull, cos_nm, 3);
            if (lane == 0) M[kCosMaxDim] = make_float4(n0, n1, n2, n3);
          }
        }
        __syncwarp();  // the whole warp's part of the slot is written
        if (lane == 0) {
          WsSlot d;
          d.sub = sub;
          d.out0 = out0;
          d.kb = kb;
          d.n = n;
          d.r = r;
          d.next = 0;
          d.pad = 0;
          d.cos_r = COS ? r : -1;
          d.pad2 = 0;
          slots[s] = d;
          mbar_arrive(full0 + 8 * s);
        }
      }
      seg = seg_end;
      ++r;
    }
  }

  // no more work will be drawn by this block: a join queued behind this one may start to move in
  if (gtid == 0) pdl_trigger();

  // stop slot: published by the warp whose turn it is
  if (static_cast<int>(it % n_resolvers) == rwarp && !dead) {
    const int s = it % kSlots;
    bool ok = true;
    if (it >= static_cast<unsigned>(kSlots)) ok = mbar_wait_bounded(empty0 + 8 * s, (it / kSlots - 1) & 1u);
    if (lane == 0) {
      if (!ok) atomicExch(a.status, kDevWaitExpired);
      WsSlot d;
      d.sub = 0;
      d.out0 = 0;
      d.kb = 0;
      d.n = 0;
      d.r = 0;
      d.next = 0;
      d.pad = 0;
      d.cos_r = -1;
      d.pad2 = 0;
      if (ok) {
        slots[s] = d;
        mbar_arrive(full0 + 8 * s);
      }
    }
  }
  // the last block to stop drawing tiles zeroes the scheduling words for the next launch
  if (a.sched != nullptr && gtid == 0) {
    __threadfence();
    if (atomicAdd(a.sched + 1, 1) == static_cast<int>(gridDim.x) - 1) {
      a.sched[0] = 0;
      a.sched[1] = 0;
      __threadfence();
    }
  }
}

}  // namespace ccr
