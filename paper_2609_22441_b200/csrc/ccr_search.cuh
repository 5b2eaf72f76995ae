// Key staging and the per-candidate sorted search (Algorithm 1 steps 2-3 of the paper).
//
// What a lookup has to decide is "does some key equal this id, and at which index" (Eq. 1); on sorted, unique keys
// that is exactly the lower bound + equality test of Algorithm 1.  A request's keys are served from this block's
// shared memory in one of four forms, chosen per request segment from the list's length K, the shared-memory area
// of the launch and the number of lookups the segment will make:
//
//   staged + table : the keys are brought in by one 1-D TMA bulk copy and a hash table over them is built beside
//                    them.  A lookup is two 16-byte table reads (two candidate buckets of four slots; a slot holds
//                    a 13-bit fingerprint of the key and the key's index) and, only when a fingerprint matches, one key
//                    read to verify: two dependent shared-memory accesses whatever K is and however the ids are
//                    spread over their range (a map of the key *range* to buckets degenerates for clustered ids:
//                    one far outlier puts a whole list into one bucket).
//   table only     : lists too long to stage next to their table keep only the table in shared memory; the
//                    verifying key read goes to global memory / L2 (hits only: a miss never leaves the SM).
//   staged         : segments with too few lookups to pay for building a table search the staged keys by a
//                    branch-free binary search.
//   sampled        : every 2^s-th key staged as the top of the search tree, the last <= 2^s keys of a search read
//                    from global memory / L2 (lists beyond everything above); key_cap == 0: the whole search runs
//                    in global memory.
//
// The table is filled with two-choice placement (a key goes to the emptier of its two buckets), at most one key per
// two slots.  A key that finds both buckets full is simply left out: a lookup that sees two full buckets and no
// verified match falls back to the binary search, so the table never has to be complete to be exact (simulated on
// uniform, consecutive and heavy-tailed ids: no key left out in most lists, both buckets full for 0.03 % of ids).
#pragma once

#include "ccr_device.cuh"

namespace ccr {

constexpr int kSlotPosBits = 18;                       // a slot = fingerprint tag (bits 18..31) | (key index + 1); 0 = empty
constexpr unsigned kSlotPosMask = (1u << kSlotPosBits) - 1u;
constexpr int kTableMaxKeys = (1 << kSlotPosBits) - 2;  // longer lists take the sampled search
#ifndef CCR_TABLE_AMORT
#define CCR_TABLE_AMORT 1
#endif
#ifndef CCR_BUILD_ILP
#define CCR_BUILD_ILP 2
#endif
constexpr int kTableAmort = CCR_TABLE_AMORT;  // a table over K keys is built for a segment of at least K / kTableAmort lookups

// Shared memory a search may use: one area that holds [table | keys], [table], [keys] or [sampled keys].
struct SearchSmem {
  unsigned char* base;
  int bytes;     // size of the area
  bool index;    // tables may be built
};

__host__ __device__ inline int pow2_ceil(int x) {
  int p = 1;
  while (p < x) p <<= 1;
  return p;
}
// buckets (of four 4-byte slots) of a table over K keys: two slots per key
__host__ __device__ inline int table_buckets(int K) { return K > 0 ? (K + 1) / 2 : 0; }
__host__ __device__ inline int search_keys_bytes(int K) { return K > 0 ? (((K + 2) + 1) & ~1) * 8 : 0; }  // K keys + 2, whole 16 bytes
// bytes that hold a list of K keys staged next to its table
__host__ __device__ inline int search_bytes(int K, bool want_index) {
  return search_keys_bytes(K) + (want_index ? table_buckets(K) * 16 : 0);
}
__device__ __forceinline__ SearchSmem carve_search(unsigned char* base, int bytes, bool want_index) {
  SearchSmem s;
  s.base = base;
  s.bytes = bytes;
  s.index = want_index;
  return s;
}

// Two bucket indices and the fingerprint tag of an id: 13 hash bits and a set top bit, placed above the index bits
// of a slot, so that (slot ^ tag) is the stored index + 1 for a slot that holds this fingerprint and at least
// 2^18 for every other slot, the empty one included.  Three 32-bit multiplies; the two bucket choices come from
// differently mixed words, so ids that collide in one rarely collide in the other.
__device__ __forceinline__ void key_hash(long long id, unsigned nbk, unsigned& b1, unsigned& b2, unsigned& tag) {
  const unsigned lo = static_cast<unsigned>(id), hi = static_cast<unsigned>(static_cast<unsigned long long>(id) >> 32);
  const unsigned u = lo * 0x9E3779B1u + hi * 0x85EBCA77u;
  const unsigned v = (u ^ (u >> 15)) * 0x2C1B3C6Du;
  b1 = __umulhi(u, nbk);
  b2 = __umulhi(v, nbk);
  tag = (v << kSlotPosBits) | 0x80000000u;
}

// Keys of the request a block is currently serving.
struct StagedKeys {
  const int64_t* sk;  // shared-memory copy (index i = key i when s_log == 0, sample i otherwise)
  const int64_t* gk;  // the request's keys in global memory
  const uint4* tab;   // hash table over the K keys (only when nbk > 0)
  int K;              // keys in the request
  int M;              // staged entries (0 = nothing staged)
  int s_log;          // log2 of the sampling stride
  unsigned nbk;       // buckets of the table (0 = none)
  bool warp_search;   // global-memory searches run warp-cooperatively (find_batch_warp)
  bool declined;      // no table only because the segment it was staged for had too few lookups to pay for one

  // Algorithm 1 steps 2-3 for one id by binary search: found = some key equals id; pos = its index (meaningful
  // when found).  Serves the segments without a table and the rare lookups the table cannot answer.
  __device__ __forceinline__ bool find(int64_t id, int& pos) const {
    pos = 0;
    if (K == 0) return false;
    if (M > 0 && s_log == 0) {
      pos = lower_bound_smem(sk, M, id);
      return pos < M && sk[pos] == id;
    }
    int lo = 0, n = K;
    if (M > 0) {
      // sample i is key (i+1)*2^s - 1: c samples below id means blocks 0..c-1 are entirely below it
      const int c = lower_bound_smem(sk, M, id);
      lo = c << s_log;
      n = min(1 << s_log, K - lo);
    }
    pos = lo + lower_bound_global(gk + lo, n, id);
    return pos < K && gload(gk + pos) == id;
  }

  // U independent lookups with their memory accesses interleaved: one round of table reads (two buckets per id),
  // then one round of verifying key reads (only ids with a matching fingerprint).  Lists without a table, and the
  // ids the table cannot answer, take find().  id < 0 is "nothing to look up".
  // The warp-cooperative form of the search in global memory (all 32 lanes must call, converged): the warp serves
  // one id at a time — 32 pivots spread over the remaining range are read by the 32 lanes, a ballot counts the
  // pivots below the id and picks the sub-range, so a list of 20,000 keys takes 3 rounds (+ 1 read for the
  // equality test) instead of 15 dependent probes, and the last round's 32 keys are one coalesced 256-byte read.
  // Four ids are in flight at once.  The price is that the 32 x U ids of a batch are served one after the other
  // rather than side by side.
  template <int U>
  __device__ __forceinline__ void find_batch_warp(const int64_t (&id)[U], bool (&found)[U], int (&pos)[U]) const {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      found[u] = false;
      pos[u] = 0;
    }
    if (K == 0) return;
#pragma unroll 1
    for (int u = 0; u < U; ++u) {
#pragma unroll 1
      for (int src = 0; src < 32; src += 4) {
        long long q[4];
        int lo[4], n[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          q[t] = __shfl_sync(kFull, id[u], src + t);
          lo[t] = 0;
          n[t] = q[t] >= 0 ? K : 0;
        }
        while (n[0] > 0 || n[1] > 0 || n[2] > 0 || n[3] > 0) {  // warp-uniform: q, lo and n are the same in every lane
          long long kv[4];
          int step[4];
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            step[t] = (n[t] + 31) >> 5;
            const long long p = static_cast<long long>(lo[t]) + static_cast<long long>(lane + 1) * step[t] - 1;
            kv[t] = (n[t] > 0 && p < lo[t] + n[t]) ? gload(gk + p) : 0x7fffffffffffffffLL;
          }
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            if (n[t] > 0) {
              const int c = __popc(__ballot_sync(kFull, kv[t] < q[t]));
              const int nlo = min(lo[t] + c * step[t], lo[t] + n[t]);
              n[t] = min(step[t] - 1, lo[t] + n[t] - nlo);
              lo[t] = nlo;
            }
          }
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const bool f = q[t] >= 0 && lo[t] < K && gload(gk + lo[t]) == q[t];
          if (lane == src + t) {
            found[u] = f;
            pos[u] = f ? lo[t] : 0;
          }
        }
      }
    }
  }

  template <int U>
  __device__ __forceinline__ void find_batch(const int64_t (&id)[U], bool (&found)[U], int (&pos)[U]) const {
    if (nbk == 0 && warp_search && M == 0) {
      find_batch_warp<U>(id, found, pos);
      return;
    }
    if (nbk == 0) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        pos[u] = 0;
        found[u] = id[u] >= 0 && find(id[u], pos[u]);
      }
      return;
    }
    unsigned hit[U];   // index + 1 of the matching slot with the smallest index (>= 2^18: no fingerprint matched)
    bool full[U];      // both buckets full: the key may have been left out of the table
#pragma unroll
    for (int u = 0; u < U; ++u) {
      unsigned b1, b2, tag;
      key_hash(id[u], nbk, b1, b2, tag);
      const uint4 x = tab[b1], y = tab[b2];
      hit[u] = min(min(min(x.x ^ tag, x.y ^ tag), min(x.z ^ tag, x.w ^ tag)),
                   min(min(y.x ^ tag, y.y ^ tag), min(y.z ^ tag, y.w ^ tag)));
      full[u] = x.w != 0u && y.w != 0u;  // the slots of a bucket fill in order
    }
    int64_t kv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      pos[u] = static_cast<int>(hit[u]) - 1;  // < K for a match: slots only ever hold indices of this list
      kv[u] = 0;
      if (hit[u] <= kSlotPosMask && id[u] >= 0) kv[u] = (M > 0) ? sk[pos[u]] : gload(gk + pos[u]);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const bool has = hit[u] <= kSlotPosMask && id[u] >= 0;
      found[u] = has && kv[u] == id[u];
      // a matching fingerprint of another key, or no match with nowhere left to look: the exact search decides
      if (id[u] >= 0 && !found[u] && (has || full[u])) found[u] = find(id[u], pos[u]);
      if (!found[u]) pos[u] = 0;
    }
  }
};

// Thread groups that can stage keys together: the whole block, or a subset of warps on a named barrier.
struct BlockGroup {
  int tid, size;
  __device__ __forceinline__ BlockGroup() : tid(threadIdx.x), size(blockDim.x) {}
  __device__ __forceinline__ void sync() const { __syncthreads(); }
  __device__ __forceinline__ bool sync_or(bool p) const { return __syncthreads_or(p ? 1 : 0) != 0; }
};
struct NamedGroup {
  int tid, size, bar_id;
  __device__ __forceinline__ NamedGroup(int t, int s, int b) : tid(t), size(s), bar_id(b) {}
  __device__ __forceinline__ void sync() const {
    __syncwarp();
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(size) : "memory");
  }
  __device__ __forceinline__ bool sync_or(bool p) const {
    unsigned out;
    __syncwarp();
    asm volatile(
        "{\n"
        " .reg .pred p, q;\n"
        " setp.ne.u32 q, %3, 0;\n"
        " bar.red.or.pred p, %1, %2, q;\n"
        " selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(out)
        : "r"(bar_id), "r"(size), "r"(static_cast<unsigned>(p))
        : "memory");
    return out != 0;
  }
};

// One key into the table: the emptier of its two buckets first, the first free slot of it (claimed with a
// compare-and-swap, so concurrent inserts never share a slot; a slot is only tried after the one before it was
// seen occupied, so the occupied slots of a bucket are always its first ones); a key that finds both buckets full
// is left out.
__device__ __forceinline__ void table_place(unsigned* slots, unsigned b1, unsigned b2, unsigned tag, const uint4& x,
                                            const uint4& y, int index) {
  const int c1 = (x.x != 0u) + (x.y != 0u) + (x.z != 0u) + (x.w != 0u);
  const int c2 = (y.x != 0u) + (y.y != 0u) + (y.z != 0u) + (y.w != 0u);
  const unsigned val = tag | static_cast<unsigned>(index + 1);
  const unsigned first = (c1 <= c2) ? b1 : b2, second = (c1 <= c2) ? b2 : b1;
  bool done = false;
  for (int j = min(c1, c2); j < 4 && !done; ++j) done = atomicCAS(slots + first * 4 + j, 0u, val) == 0u;
  for (int j = max(c1, c2); j < 4 && !done; ++j) done = atomicCAS(slots + second * 4 + j, 0u, val) == 0u;
}
__device__ __forceinline__ void table_insert(unsigned* slots, unsigned nbk, long long key, int index) {
  unsigned b1, b2, tag;
  key_hash(key, nbk, b1, b2, tag);
  const uint4 x = reinterpret_cast<const uint4*>(slots)[b1], y = reinterpret_cast<const uint4*>(slots)[b2];
  table_place(slots, b1, b2, tag, x, y, index);
}

// Stage keys [kb, kb+K) of the key array for the group.  Starts with a group barrier (everyone is done
// with the previously staged keys) and ends with one.  Returns false, group-uniformly, if the bounded
// wait for the bulk copy expired.  `index` asks for the hash table; `n_lookups` is how many lookups the
// caller is about to make against these keys (the table is built only when they pay for it).
template <typename G>
__device__ __forceinline__ bool stage_keys(const JoinArgs& a, const SearchSmem& sm, uint32_t bar, uint32_t& phase,
                                           long long kb, int K, bool index, long long n_lookups, StagedKeys& st,
                                           const G& g) {
  // The area may hold ordinary (generic-proxy) stores of an earlier staging — a table, sampled keys, the
  // unaligned head / tail key — at addresses the bulk copy below writes through the async proxy: every thread
  // orders its own earlier stores against the async proxy before the barrier that precedes the copy.
  fence_proxy_async_smem();
  g.sync();
  st.gk = a.edge_keys + kb;
  st.K = K;
  st.M = 0;
  st.s_log = 0;
  st.nbk = 0;
  st.declined = false;
  st.warp_search = a.warp_search != 0;
  st.tab = reinterpret_cast<const uint4*>(sm.base);
  st.sk = reinterpret_cast<const int64_t*>(sm.base);
  if (a.key_cap <= 0 || K <= 0 || sm.bytes < 16) {
    g.sync();
    return true;
  }

  const bool sampled_forced = a.min_stride_log2 != 0;
  const bool table_ok = index && sm.index && !sampled_forced && K > 1 && K <= kTableMaxKeys;
  const bool want_table = table_ok && n_lookups * kTableAmort >= K;
  st.declined = table_ok && !want_table;
  const int tab_bytes = table_buckets(K) * 16, key_bytes = search_keys_bytes(K);
  const bool may_stage = K <= a.key_cap && !sampled_forced;
  // [table | keys] when both fit; the table alone for a longer list; else the keys alone or a sampled top of the tree
  const bool both = want_table && may_stage && tab_bytes + key_bytes <= sm.bytes;
  const bool table = both || (want_table && tab_bytes <= sm.bytes);
  const bool staged = both || (!table && may_stage && key_bytes <= sm.bytes);
  int64_t* skeys = reinterpret_cast<int64_t*>(sm.base + (both ? tab_bytes : 0));
  unsigned* slots = reinterpret_cast<unsigned*>(sm.base);
  bool expired = false;

  if (table) {  // cleared while the copy below is in flight
    uint4* t4 = reinterpret_cast<uint4*>(slots);
    for (int b = g.tid; b < table_buckets(K); b += g.size) t4[b] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (staged) {
    // slot of key i is i + shift, so that 16-byte aligned global addresses land on 16-byte aligned slots
    const int shift = static_cast<int>(kb & 1);
    const int i0 = shift;                       // first key whose address is 16-byte aligned
    int nbulk = (K - i0) & ~1;                  // keys moved by the bulk copy (even count)
    if (nbulk > 0 && !CCR_CHK(a.edge_keys + kb + i0, nbulk * 8)) nbulk = 0;  // (checked build: the copy is left out)
    st.sk = skeys + shift;
    st.M = K;
    if (g.tid == 0 && nbulk > 0) {
      mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nbulk) * 8u);
      bulk_copy_g2s(smem_u32(skeys + i0 + shift), a.edge_keys + kb + i0, static_cast<uint32_t>(nbulk) * 8u, bar);
    }
    // the (at most one) key before and after the 16-byte aligned middle, by two other threads
    if (g.tid == 1 && shift) skeys[shift] = gload(a.edge_keys + kb);
    if (g.tid == 2 && ((K - i0) & 1)) skeys[K - 1 + shift] = gload(a.edge_keys + kb + K - 1);
    if (nbulk > 0) {
      expired = !mbar_wait_bounded(bar, phase);
      phase ^= 1u;
    }
  } else if (!table) {
    int s_log = a.min_stride_log2;
    const int cap = min(a.key_cap, sm.bytes / 8);
    while ((K >> s_log) > cap) ++s_log;
    st.s_log = s_log;
    st.M = K >> s_log;
    for (int i = g.tid; i < st.M; i += g.size)
      skeys[i] = gload(a.edge_keys + kb + ((static_cast<long long>(i) + 1) << s_log) - 1);
  }
  if (g.sync_or(expired)) return false;

  if (table) {
    const unsigned nbk = static_cast<unsigned>(table_buckets(K));
    const int64_t* S = st.sk;
    // several keys of a thread in flight: the bucket reads and compare-and-swaps of one overlap the others'
    constexpr int kIlp = CCR_BUILD_ILP;
    int i = g.tid;
    for (; i + (kIlp - 1) * g.size < K; i += kIlp * g.size) {
      long long kk[kIlp];
#pragma unroll
      for (int q = 0; q < kIlp; ++q) kk[q] = staged ? S[i + q * g.size] : gload(st.gk + i + q * g.size);
      unsigned b1[kIlp], b2[kIlp], tag[kIlp];
      uint4 x[kIlp], y[kIlp];
#pragma unroll
      for (int q = 0; q < kIlp; ++q) {
        key_hash(kk[q], nbk, b1[q], b2[q], tag[q]);
        x[q] = reinterpret_cast<const uint4*>(slots)[b1[q]];
        y[q] = reinterpret_cast<const uint4*>(slots)[b2[q]];
      }
#pragma unroll
      for (int q = 0; q < kIlp; ++q) table_place(slots, b1[q], b2[q], tag[q], x[q], y[q], i + q * g.size);
    }
    for (; i < K; i += g.size) table_insert(slots, nbk, staged ? S[i] : gload(st.gk + i), i);
    st.nbk = nbk;
    g.sync();
  }
  return true;
}

}  // namespace ccr
