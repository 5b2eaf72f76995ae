// Key staging and the per-candidate sorted search (Algorithm 1 steps 2-3 of the paper).
//
// A request's sorted author ids are staged in shared memory by one 1-D TMA bulk copy (K <= key_cap), or as
// a sampled top of the search tree (K > key_cap: every 2^s-th key; the last <= 2^s keys of a search are
// read from global memory / L2), or not at all (key_cap == 0).
//
// Fully staged lists also get a bucket index over the key range: bucket b = (key - kmin) >> shift, with
// (first, end) positions of the keys that fall in it.  A lookup is then one index load plus a branch-free
// lower bound over the few keys of one bucket (about one key per bucket for evenly spread ids, never more
// than log2 K steps) instead of log2 K dependent shared-memory probes over the whole list.  The bucket
// function is monotone in the key, so a bucket's keys are contiguous and the result is exactly the lower
// bound / equality test of Algorithm 1; an id in an empty bucket is simply not found.
#pragma once

#include "ccr_device.cuh"

namespace ccr {

// Shared memory a search needs: the key area and the bucket index.
struct SearchSmem {
  int64_t* keys;   // key_cap + 2 slots
  int2* tab;       // tab_cap entries (0 = no index)
  int tab_cap;     // power of two
};

__host__ __device__ inline int pow2_ceil(int x) {
  int p = 1;
  while (p < x) p <<= 1;
  return p;
}
// bytes of the search area for a given key capacity (keys, then the bucket index), 16-byte aligned pieces
__host__ __device__ inline int search_keys_bytes(int key_cap) { return (key_cap + 2) * 8; }
constexpr int kMaxBuckets = 4096;  // 32 KB of index at most; longer lists simply get more keys per bucket
__host__ __device__ inline int search_tab_cap(int key_cap, bool want_index) {
  if (!want_index || key_cap <= 0) return 0;
  const int p = pow2_ceil(key_cap);
  return p < kMaxBuckets ? p : kMaxBuckets;
}
__host__ __device__ inline int search_bytes(int key_cap, bool want_index) {
  return search_keys_bytes(key_cap) + search_tab_cap(key_cap, want_index) * 8;
}
__device__ __forceinline__ SearchSmem carve_search(unsigned char* base, int key_cap, bool want_index) {
  SearchSmem s;
  s.keys = reinterpret_cast<int64_t*>(base);
  s.tab = reinterpret_cast<int2*>(base + search_keys_bytes(key_cap));
  s.tab_cap = search_tab_cap(key_cap, want_index);
  return s;
}

// Keys of the request a block is currently serving.
struct StagedKeys {
  const int64_t* sk;  // shared-memory copy (index i = key i when s_log == 0, sample i otherwise)
  const int64_t* gk;  // the request's keys in global memory
  const int2* tab;    // bucket index over sk (only when nb > 0)
  long long kmin, kmax;
  int K;              // keys in the request
  int M;              // staged entries (0 = nothing staged)
  int s_log;          // log2 of the sampling stride
  int nb;             // buckets in the index (0 = none)
  int shift;          // bucket = (key - kmin) >> shift

  // Algorithm 1 steps 2-3 for one id: found = some key equals id; pos = its index (meaningful when found).
  __device__ __forceinline__ bool find(int64_t id, int& pos) const {
    pos = 0;
    if (K == 0) return false;
    if (M > 0 && s_log == 0) {
      int lo = 0, n = M;
      if (nb > 0) {
        if (id < kmin || id > kmax) return false;
        const int2 e = tab[static_cast<unsigned long long>(id - kmin) >> shift];
        lo = min(max(e.x, 0), M);             // clamps only matter for unsorted (contract-breaking) keys
        n = min(max(e.y, lo), M) - lo;
      }
      pos = lo + lower_bound_smem(sk + lo, n, id);
      return pos < lo + n && sk[pos] == id;
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

  // U independent lookups with their shared-memory accesses interleaved: one round of bucket-index loads,
  // then one round of up to P key loads per id (a bucket of evenly spread ids holds about one key).
  // Ids whose bucket is longer, and lists without an index, take find().  id < 0 is "nothing to look up".
  template <int U, int P = 4>
  __device__ __forceinline__ void find_batch(const int64_t (&id)[U], bool (&found)[U], int (&pos)[U]) const {
    if (!(K > 0 && M > 0 && s_log == 0 && nb > 0)) {
#pragma unroll
      for (int u = 0; u < U; ++u) found[u] = id[u] >= 0 && find(id[u], pos[u]);
      return;
    }
    int lo[U], n[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const bool in = id[u] >= kmin && id[u] <= kmax;
      const int2 e = in ? tab[static_cast<unsigned long long>(id[u] - kmin) >> shift] : make_int2(0, 0);
      lo[u] = min(max(e.x, 0), M);
      n[u] = min(max(e.y, lo[u]), M) - lo[u];
    }
    int64_t k[U][P];
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
      for (int j = 0; j < P; ++j) k[u][j] = (j < n[u]) ? sk[lo[u] + j] : 0;  // lo + j < lo + n <= M
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      found[u] = false;
      pos[u] = 0;
#pragma unroll
      for (int j = 0; j < P; ++j) {
        if (j < n[u] && k[u][j] == id[u]) {
          found[u] = true;
          pos[u] = lo[u] + j;
        }
      }
      if (n[u] > P && !found[u]) found[u] = find(id[u], pos[u]);  // long bucket: bounded binary search
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

// Stage keys [kb, kb+K) of the key array for the group.  Starts with a group barrier (everyone is done
// with the previously staged keys) and ends with one.  Returns false, group-uniformly, if the bounded
// wait for the bulk copy expired.  `index` asks for the bucket index (built only for fully staged lists).
template <typename G>
__device__ __forceinline__ bool stage_keys(const JoinArgs& a, const SearchSmem& sm, uint32_t bar, uint32_t& phase,
                                           long long kb, int K, bool index, StagedKeys& st, const G& g) {
  // The key area may hold ordinary (generic-proxy) stores of an earlier staging — sampled keys, the unaligned
  // head / tail key — at addresses the bulk copy below writes through the async proxy: every thread orders its
  // own earlier stores against the async proxy before the barrier that precedes the copy.
  fence_proxy_async_smem();
  g.sync();
  int64_t* skeys = sm.keys;
  st.gk = a.edge_keys + kb;
  st.K = K;
  st.M = 0;
  st.s_log = 0;
  st.sk = skeys;
  st.tab = sm.tab;
  st.nb = 0;
  st.shift = 0;
  st.kmin = st.kmax = 0;
  bool expired = false;
  if (a.key_cap > 0 && K > 0) {
    if (K <= a.key_cap && a.min_stride_log2 == 0) {
      // slot of key i is i + shift, so that 16-byte aligned global addresses land on 16-byte aligned slots
      const int shift = static_cast<int>(kb & 1);
      const int i0 = shift;                       // first key whose address is 16-byte aligned
      const int nbulk = (K - i0) & ~1;            // keys moved by the bulk copy (even count)
      st.sk = skeys + shift;
      st.M = K;
      if (g.tid == 0 && nbulk > 0) {
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nbulk) * 8u);
        bulk_copy_g2s(smem_u32(skeys + i0 + shift), a.edge_keys + kb + i0, static_cast<uint32_t>(nbulk) * 8u, bar);
      }
      // the (at most one) key before and after the 16-byte aligned middle, by two other threads
      if (g.tid == 1 && shift) skeys[shift] = __ldg(a.edge_keys + kb);
      if (g.tid == 2 && ((K - i0) & 1)) skeys[K - 1 + shift] = __ldg(a.edge_keys + kb + K - 1);
      if (nbulk > 0) {
        expired = !mbar_wait_bounded(bar, phase);
        phase ^= 1u;
      }
    } else {
      int s_log = a.min_stride_log2;
      while ((K >> s_log) > a.key_cap) ++s_log;
      st.s_log = s_log;
      st.M = K >> s_log;
      for (int i = g.tid; i < st.M; i += g.size)
        skeys[i] = __ldg(a.edge_keys + kb + ((static_cast<long long>(i) + 1) << s_log) - 1);
    }
  }
  if (g.sync_or(expired)) return false;

  if (index && sm.tab_cap > 0 && st.M > 1 && st.s_log == 0) {
    const int M = st.M;
    const int64_t* S = st.sk;
    st.kmin = S[0];
    st.kmax = S[M - 1];
    const unsigned long long range = static_cast<unsigned long long>(st.kmax - st.kmin);
    const int nb = min(sm.tab_cap, pow2_ceil(M));
    int shift = 0;
    while ((range >> shift) >= static_cast<unsigned long long>(nb)) ++shift;  // group-uniform, <= 63 steps
    st.nb = nb;
    st.shift = shift;
    int2* tab = sm.tab;
    for (int b = g.tid; b < nb; b += g.size) tab[b] = make_int2(0, 0);
    g.sync();
    for (int i = g.tid; i < M; i += g.size) {
      const unsigned long long b = static_cast<unsigned long long>(S[i] - st.kmin) >> shift;
      if (b >= static_cast<unsigned long long>(nb)) continue;  // only possible with unsorted (contract-breaking) keys
      const bool first = (i == 0) || ((static_cast<unsigned long long>(S[i - 1] - st.kmin) >> shift) != b);
      const bool last = (i == M - 1) || ((static_cast<unsigned long long>(S[i + 1] - st.kmin) >> shift) != b);
      if (first) tab[b].x = i;
      if (last) tab[b].y = i + 1;
    }
    g.sync();
  }
  return true;
}

}  // namespace ccr
