// TEST INFRASTRUCTURE — CPU oracle for the edge-feature join.  Not part of the product path:
// only the tests, the smoke check and the benchmark's cpu_baseline / reference legs may call it.
// It shares no code with the CUDA library (no common headers, helpers, tables or constants).
//
// What it computes, and where the paper defines it:
//   * Eq. 1 (Section 3.1): O_j = F_i if some affinity record i has a_i = d_j, else the zero vector.
//     The binary search of Algorithm 1 reaches exactly this result, so the oracle is the definition,
//     evaluated with std::lower_bound per candidate.
//   * Algorithm 1, steps 2-4: pos = searchsorted(a_sorted, d) (lower bound: only then can the
//     equality test of step 3 hit), valid = (pos < K) and (a_sorted[min(pos, K-1)] == d),
//     O = zeros; O[valid] = F_sorted[pos].  K == 0 means nothing is found and no key is read.
//   * Section 6.3 / Section 6.3.1 ("Batching and Padding"): document features are gathered from the
//     GPU-resident index by position, for the flattened positions of all requests in request order;
//     a position of -1 is an unresolved id (Eq. 6) and yields a zero row here.
//   * Section 3: request features are given per request and shared by all its candidates.
//   * Second-degree lookups (engagers of a post looked up in the same viewer keys) are only named by
//     the paper (abstract, Section 1); the reduction below is this build's reading and is
//     PARITY UNPINNED by the paper: for each edge dim, over the found engager slots in ascending slot
//     order, either max (strict > in fp32, the earlier slot wins ties, the winner's 16 bits are kept)
//     or sum (fp32 accumulator starting at +0.0f, one round-to-nearest add per slot, one
//     round-to-nearest-even conversion to fp16 at the end; a NaN sum is stored as 0x7fff).
//
// Output row j (byte-packed, values copied bit for bit in their own dtype):
//   [ doc section | edge section | edge2 section (second-degree stores only) | request section ]
// out_mask[j]: bit0 author found; bits 1..4 engager slot 0..3 found; bits 5..7 OR of (1 << type) over
// the found slots (type 0 reacted, 1 commented, 2 reshared).
//
//   * Algorithm 1 step 1 (ccr_oracle_sort_edges): a_sorted, idx = sort(a); F_sorted = gather(F, idx), per
//     request, as std::stable_sort of the record indices by key followed by a row-by-row copy.
//
//   * Eq. 6 (Section 6.3.1, ccr_oracle_resolve_ids): pos(q) = H[q] if q is indexed, else -1, evaluated with
//     std::lower_bound on the ascending id array (the paper's own first design).
//
//   * Section 4.1.2 "Derived Features" (ccr_oracle_cosine): the member representation is n_chunks medoid
//     embeddings of `dim` values each, the item embedding has `dim` values; per chunk k the cosine similarity
//     cos_k = <m_k, x> / (|m_k| |x|) is computed in float32 and stored as float16.  The paper fixes the
//     precision, not the order or the guard; this build's reading: the three sums (dot, |m|^2, |x|^2) are
//     float32 fused-multiply-add chains from +0 over the elements in ascending order, the denominator is
//     sqrtf(|x|^2) * sqrtf(|m|^2) (one rounded product), a denominator below 1e-8 (or NaN) is replaced by 1e-8
//     (so a zero vector gives 0), the quotient is rounded once to float16 (ties to even), NaN is stored as 0x7fff.
//
// Plain, slow and unblocked on purpose; single-threaded unless n_threads > 1, in which case the flat
// candidate range is cut into contiguous chunks, one std::thread each.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

float half_bits_to_float(uint16_t h) {
  const uint32_t sign = static_cast<uint32_t>(h & 0x8000u) << 16;
  const uint32_t exp = (h >> 10) & 0x1fu;
  uint32_t man = h & 0x3ffu;
  uint32_t bits;
  if (exp == 0) {
    if (man == 0) {
      bits = sign;
    } else {  // subnormal half: man * 2^-24, renormalised
      int shifts = 0;
      while ((man & 0x400u) == 0) {
        man <<= 1;
        ++shifts;
      }
      man &= 0x3ffu;
      bits = sign | (static_cast<uint32_t>(113 - shifts) << 23) | (man << 13);
    }
  } else if (exp == 31) {
    bits = sign | 0x7f800000u | (man << 13);
  } else {
    bits = sign | ((exp + 112u) << 23) | (man << 13);
  }
  float f;
  std::memcpy(&f, &bits, 4);
  return f;
}

// fp32 -> fp16, round to nearest, ties to even; overflow goes to infinity; NaN becomes 0x7fff.
uint16_t float_to_half_bits(float f) {
  uint32_t x;
  std::memcpy(&x, &f, 4);
  const uint16_t sign = static_cast<uint16_t>((x >> 16) & 0x8000u);
  const uint32_t ax = x & 0x7fffffffu;
  if (ax > 0x7f800000u) return 0x7fffu;
  if (ax == 0x7f800000u) return sign | 0x7c00u;
  const int e = static_cast<int>(ax >> 23) - 127;
  if (e >= 16) return sign | 0x7c00u;
  if (e >= -14) {
    const uint32_t man = ax & 0x7fffffu;
    uint32_t h = (static_cast<uint32_t>(e + 15) << 10) | (man >> 13);
    const uint32_t rem = man & 0x1fffu;
    if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) ++h;  // a carry into the exponent is correct
    return sign | static_cast<uint16_t>(h);
  }
  if (e < -25) return sign;
  const uint32_t man = (ax & 0x7fffffu) | 0x800000u;
  const int shift = -e - 1;  // 14..24
  uint32_t h = man >> shift;
  const uint32_t rem = man & ((1u << shift) - 1u);
  const uint32_t halfway = 1u << (shift - 1);
  if (rem > halfway || (rem == halfway && (h & 1u))) ++h;
  return sign | static_cast<uint16_t>(h);
}

struct Problem {
  int64_t n_docs;
  const uint8_t* doc_feats;
  int64_t doc_b;
  const int64_t* author_ids;
  int32_t max_actors;
  const int64_t* actor_ids;
  const uint8_t* actor_types;
  int32_t edge_dim;
  int64_t edge_b;
  uint64_t reduce_sum_mask;
  int32_t n_req;
  const int64_t* edge_keys;
  const uint8_t* edge_feats;
  const int64_t* edge_offsets;
  const int32_t* cand_idx;
  const int64_t* cand_offsets;
  const uint8_t* req_feats;
  int64_t req_b;
  bool second;  // an edge2 section exists
  int64_t out_b;
  uint8_t* out_rows;
  uint8_t* out_mask;
};

// Membership of `id` among request r's keys (Algorithm 1 steps 2-3).
bool lookup(const Problem& p, int32_t r, int64_t id, int64_t* pos_out) {
  const int64_t* keys = p.edge_keys + p.edge_offsets[r];
  const int64_t K = p.edge_offsets[r + 1] - p.edge_offsets[r];
  if (K <= 0) return false;
  const int64_t pos = std::lower_bound(keys, keys + K, id) - keys;
  if (pos < K && keys[pos] == id) {
    *pos_out = pos;
    return true;
  }
  return false;
}

void join_one(const Problem& p, int32_t r, int64_t j) {
  uint8_t* row = p.out_rows + j * p.out_b;
  uint8_t* sec_doc = row;
  uint8_t* sec_edge = sec_doc + p.doc_b;
  uint8_t* sec_edge2 = sec_edge + p.edge_b;
  uint8_t* sec_req = p.second ? sec_edge2 + p.edge_b : sec_edge2;
  const int64_t idx = p.cand_idx[j];
  uint8_t m = 0;
  if (idx < 0 || idx >= p.n_docs) {
    std::memset(row, 0, static_cast<size_t>(p.out_b - p.req_b));
  } else {
    std::memcpy(sec_doc, p.doc_feats + idx * p.doc_b, static_cast<size_t>(p.doc_b));
    int64_t pos = 0;
    if (lookup(p, r, p.author_ids[idx], &pos)) {
      std::memcpy(sec_edge, p.edge_feats + (p.edge_offsets[r] + pos) * p.edge_b, static_cast<size_t>(p.edge_b));
      m |= 1u;
    } else {
      std::memset(sec_edge, 0, static_cast<size_t>(p.edge_b));
    }
    if (p.second) {
      int64_t slot_pos[4];
      bool slot_found[4] = {false, false, false, false};
      for (int s = 0; s < p.max_actors; ++s) {
        const int64_t act = p.actor_ids[idx * p.max_actors + s];
        if (act < 0) continue;  // empty slot
        if (lookup(p, r, act, &slot_pos[s])) {
          slot_found[s] = true;
          m |= static_cast<uint8_t>(1u << (1 + s));
          m |= static_cast<uint8_t>(1u << (5 + (p.actor_types[idx * p.max_actors + s] % 3)));
        }
      }
      uint16_t* out2 = reinterpret_cast<uint16_t*>(sec_edge2);
      for (int d = 0; d < p.edge_dim; ++d) {
        const bool is_sum = (p.reduce_sum_mask >> (d & 63)) & 1u;
        bool any = false;
        uint16_t best = 0;
        float acc = 0.0f;
        for (int s = 0; s < p.max_actors; ++s) {
          if (!slot_found[s]) continue;
          uint16_t v;
          std::memcpy(&v, p.edge_feats + (p.edge_offsets[r] + slot_pos[s]) * p.edge_b + 2 * d, 2);
          if (is_sum) {
            volatile float t = acc + half_bits_to_float(v);  // one rounded fp32 add, never fused
            acc = t;
          } else if (!any || half_bits_to_float(v) > half_bits_to_float(best)) {
            best = v;
          }
          any = true;
        }
        uint16_t res = 0;
        if (any) res = is_sum ? float_to_half_bits(acc) : best;
        std::memcpy(&out2[d], &res, 2);
      }
    }
  }
  if (p.req_b > 0) std::memcpy(sec_req, p.req_feats + static_cast<int64_t>(r) * p.req_b, static_cast<size_t>(p.req_b));
  p.out_mask[j] = m;
}

void join_range(const Problem& p, int64_t j_begin, int64_t j_end) {
  for (int32_t r = 0; r < p.n_req; ++r) {
    const int64_t lo = std::max(j_begin, p.cand_offsets[r]);
    const int64_t hi = std::min(j_end, p.cand_offsets[r + 1]);
    for (int64_t j = lo; j < hi; ++j) join_one(p, r, j);
  }
}

}  // namespace

extern "C" {

uint32_t ccr_oracle_half_to_float_bits(uint16_t h) {
  const float f = half_bits_to_float(h);
  uint32_t b;
  std::memcpy(&b, &f, 4);
  return b;
}

uint16_t ccr_oracle_float_bits_to_half(uint32_t b) {
  float f;
  std::memcpy(&f, &b, 4);
  return float_to_half_bits(f);
}

// All pointers are host memory owned by the caller.  Returns 0, or a negative code for arguments the
// oracle does not define (second-degree with a non-fp16 edge table, more than 4 engager slots).
int ccr_oracle_join(int64_t n_docs, const void* doc_feats, int64_t doc_row_bytes, const int64_t* author_ids,
                    int32_t max_actors, const int64_t* actor_ids, const uint8_t* actor_types,
                    int32_t edge_dim, int32_t edge_elem_bytes, uint64_t reduce_sum_mask,
                    int32_t n_req, const int64_t* edge_keys, const void* edge_feats, const int64_t* edge_offsets,
                    const int32_t* cand_idx, const int64_t* cand_offsets,
                    const void* req_feats, int64_t req_row_bytes, int32_t first_degree_only,
                    void* out_rows, uint8_t* out_mask, int32_t n_threads) {
  Problem p;
  p.n_docs = n_docs;
  p.doc_feats = static_cast<const uint8_t*>(doc_feats);
  p.doc_b = doc_row_bytes;
  p.author_ids = author_ids;
  p.max_actors = max_actors;
  p.actor_ids = actor_ids;
  p.actor_types = actor_types;
  p.edge_dim = edge_dim;
  p.edge_b = static_cast<int64_t>(edge_dim) * edge_elem_bytes;
  p.reduce_sum_mask = reduce_sum_mask;
  p.n_req = n_req;
  p.edge_keys = edge_keys;
  p.edge_feats = static_cast<const uint8_t*>(edge_feats);
  p.edge_offsets = edge_offsets;
  p.cand_idx = cand_idx;
  p.cand_offsets = cand_offsets;
  p.req_feats = static_cast<const uint8_t*>(req_feats);
  p.req_b = req_row_bytes;
  p.second = (max_actors > 0) && !first_degree_only;
  if (p.second && (edge_elem_bytes != 2 || max_actors > 4 || edge_dim > 64)) return -1;
  p.out_b = p.doc_b + p.edge_b + (p.second ? p.edge_b : 0) + p.req_b;
  p.out_rows = static_cast<uint8_t*>(out_rows);
  p.out_mask = out_mask;
  const int64_t total = n_req > 0 ? cand_offsets[n_req] : 0;
  if (n_threads <= 1 || total < 2) {
    join_range(p, 0, total);
    return 0;
  }
  std::vector<std::thread> pool;
  const int64_t chunk = (total + n_threads - 1) / n_threads;
  for (int t = 0; t < n_threads; ++t) {
    const int64_t a = std::min<int64_t>(total, t * chunk), b = std::min<int64_t>(total, a + chunk);
    if (a < b) pool.emplace_back([&p, a, b] { join_range(p, a, b); });
  }
  for (auto& th : pool) th.join();
  return 0;
}

// Algorithm 1 step 1 for a ragged batch: records [edge_offsets[r], edge_offsets[r+1]) of every request are
// put in ascending key order (equal keys keep their input order).  perm_out (optional) receives, per output
// record, the index of its source record inside the request.
int ccr_oracle_sort_edges(int32_t n_req, const int64_t* keys_in, const void* feats_in, const int64_t* edge_offsets,
                          int64_t row_bytes, int64_t* keys_out, void* feats_out, int32_t* perm_out) {
  const uint8_t* fin = static_cast<const uint8_t*>(feats_in);
  uint8_t* fout = static_cast<uint8_t*>(feats_out);
  for (int32_t r = 0; r < n_req; ++r) {
    const int64_t e0 = edge_offsets[r], K = edge_offsets[r + 1] - e0;
    if (K < 0) return -1;
    std::vector<int32_t> idx(static_cast<size_t>(K));
    for (int64_t i = 0; i < K; ++i) idx[static_cast<size_t>(i)] = static_cast<int32_t>(i);
    std::stable_sort(idx.begin(), idx.end(),
                     [&](int32_t x, int32_t y) { return keys_in[e0 + x] < keys_in[e0 + y]; });
    for (int64_t i = 0; i < K; ++i) {
      const int32_t src = idx[static_cast<size_t>(i)];
      keys_out[e0 + i] = keys_in[e0 + src];
      std::memcpy(fout + (e0 + i) * row_bytes, fin + (e0 + src) * row_bytes, static_cast<size_t>(row_bytes));
      if (perm_out) perm_out[e0 + i] = src;
    }
  }
  return 0;
}

// Eq. 6: out_pos[i] = position of query i in the index (positions[rank] when given, else the rank), or -1.
int ccr_oracle_resolve_ids(int64_t n_ids, const int64_t* sorted_ids, const int32_t* positions, int64_t n_queries,
                           const int64_t* queries, int32_t* out_pos) {
  for (int64_t i = 0; i < n_queries; ++i) {
    const int64_t* it = std::lower_bound(sorted_ids, sorted_ids + n_ids, queries[i]);
    const int64_t rank = it - sorted_ids;
    out_pos[i] = (rank < n_ids && *it == queries[i]) ? (positions ? positions[rank] : static_cast<int32_t>(rank)) : -1;
  }
  return 0;
}

// Section 4.1.2, derived features: for candidate j of request r with position p = cand_idx[j], x = elements
// [item_first, item_first + dim) of document row p (float16; a position outside [0, n_docs) gives x = 0) and
// m_k = member_emb[r][k * dim .. (k + 1) * dim) (float16): out[j * 16 + k] = float16(cos_k), k < n_chunks <= 8;
// the other entries of the 16-value (32-byte) block are +0.
int ccr_oracle_cosine(int64_t n_docs, const void* doc_feats, int64_t doc_row_bytes, int32_t item_first, int32_t dim,
                      int32_t n_chunks, int32_t n_req, const uint16_t* member_emb, const int32_t* cand_idx,
                      const int64_t* cand_offsets, uint16_t* out) {
  if (dim <= 0 || n_chunks <= 0 || n_chunks > 8 || item_first < 0) return -1;
  if (static_cast<int64_t>(item_first + dim) * 2 > doc_row_bytes) return -2;
  std::vector<float> x(dim);
  for (int32_t r = 0; r < n_req; ++r) {
    for (int64_t j = cand_offsets[r]; j < cand_offsets[r + 1]; ++j) {
      const int64_t p = cand_idx[j];
      const bool in_range = p >= 0 && p < n_docs;
      const uint16_t* row = reinterpret_cast<const uint16_t*>(static_cast<const uint8_t*>(doc_feats) + (in_range ? p : 0) * doc_row_bytes);
      float nx = 0.0f;
      for (int32_t e = 0; e < dim; ++e) {
        x[e] = in_range ? half_bits_to_float(row[item_first + e]) : 0.0f;
        nx = std::fmaf(x[e], x[e], nx);
      }
      for (int32_t k = 0; k < 16; ++k) out[j * 16 + k] = 0;
      for (int32_t k = 0; k < n_chunks; ++k) {
        const uint16_t* m = member_emb + (static_cast<int64_t>(r) * n_chunks + k) * dim;
        float dot = 0.0f, nm = 0.0f;
        for (int32_t e = 0; e < dim; ++e) {
          const float me = half_bits_to_float(m[e]);
          dot = std::fmaf(x[e], me, dot);
          nm = std::fmaf(me, me, nm);
        }
        float den = std::sqrt(nx) * std::sqrt(nm);
        if (!(den > 1e-8f)) den = 1e-8f;
        out[j * 16 + k] = float_to_half_bits(dot / den);
      }
    }
  }
  return 0;
}

}  // extern "C"
