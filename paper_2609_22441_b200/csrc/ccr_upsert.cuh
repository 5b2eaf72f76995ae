// Store write path by position (Section 6.2, "Scaling ingestion": bootstrap step 3, "GPU scatter features to
// assigned positions"; the same scatter serves steady-state updates).  The host side of the paper's protocol —
// telling new from existing ids, the prefix sum that assigns positions, the hash-map update after the write —
// stays with the caller; this is the device step: row i of the batch goes to row positions[i] of the index.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "ccr_device.cuh"

namespace ccr {

constexpr int kUpsertThreads = 256;
constexpr int kUpsertUnroll = 4;  // 16-byte chunks a thread has in flight

struct UpsertArgs {
  long long n;               // rows in the batch
  long long n_docs;          // capacity of the store
  const int32_t* positions;  // [n] target rows; outside [0, n_docs) = skip the row
  const uint8_t* src_rows;   // [n, doc_b] or null
  uint8_t* dst_rows;         // the store's feature matrix
  int row_ch;                // doc_b / 16
  const int64_t* src_author;        // [n] or null
  const int64_t* src_actor;         // [n, max_actors] or null (second-degree stores)
  const uint8_t* src_type;          // [n, max_actors] or null
  int64_t* dst_author;       // first-degree stores
  IdRec* dst_recs;           // second-degree stores
  int max_actors;
};

// One thread per 16-byte chunk of the batch, kUpsertUnroll chunks in flight: the source is read front to back,
// every target row is written as row_ch contiguous chunks by neighbouring lanes.  Streaming loads (the batch is
// read once); default stores (the row is about to be read by joins).  The ids follow, one thread per row.
__global__ void __launch_bounds__(kUpsertThreads) upsert_kernel(const UpsertArgs a) {
  const long long tid = blockIdx.x * static_cast<long long>(kUpsertThreads) + threadIdx.x;
  const long long stride = static_cast<long long>(gridDim.x) * kUpsertThreads;
  if (a.src_rows != nullptr) {
    const long long chunks = a.n * a.row_ch;
    const uint4* src = reinterpret_cast<const uint4*>(a.src_rows);
    uint4* dst = reinterpret_cast<uint4*>(a.dst_rows);
    for (long long c0 = tid; c0 < chunks; c0 += stride * kUpsertUnroll) {
      uint4 v[kUpsertUnroll];
      long long target[kUpsertUnroll];
#pragma unroll
      for (int u = 0; u < kUpsertUnroll; ++u) {
        const long long c = c0 + u * stride;
        target[u] = -1;
        if (c < chunks) {
          const long long i = c / a.row_ch;
          const int p = gload(a.positions + i);
          if (p >= 0 && p < a.n_docs) target[u] = static_cast<long long>(p) * a.row_ch + (c - i * a.row_ch);
          v[u] = CCR_CHK(src + c, 16) ? __ldcs(src + c) : make_uint4(0u, 0u, 0u, 0u);
        }
      }
#pragma unroll
      for (int u = 0; u < kUpsertUnroll; ++u)
        if (target[u] >= 0 && CCR_CHK(dst + target[u], 16)) dst[target[u]] = v[u];
    }
  }
  if (a.src_author == nullptr && a.src_actor == nullptr && a.src_type == nullptr) return;
  for (long long i = tid; i < a.n; i += stride) {
    const int p = gload(a.positions + i);
    if (p < 0 || p >= a.n_docs) continue;
    if (a.dst_recs == nullptr) {
      if (a.src_author) gstore(a.dst_author + p, gload(a.src_author + i));
      continue;
    }
    if (!CCR_CHK(a.dst_recs + p, static_cast<int>(sizeof(IdRec)))) continue;
    IdRec& r = a.dst_recs[p];
    if (a.src_author) r.author = gload(a.src_author + i);
    if (a.src_actor) {
#pragma unroll
      for (int s = 0; s < 4; ++s) r.actor[s] = s < a.max_actors ? gload(a.src_actor + i * a.max_actors + s) : -1;
    }
    if (a.src_type) {
#pragma unroll
      for (int s = 0; s < 4; ++s) r.type[s] = s < a.max_actors ? gload(a.src_type + i * a.max_actors + s) : 0;
    }
  }
}

}  // namespace ccr
