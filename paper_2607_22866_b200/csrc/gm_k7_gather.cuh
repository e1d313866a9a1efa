// K7 — moves the compacted chunks from the staging buffer into C (the write of Numeric() in
// Algorithm 3 once C.rowPtr is known).  Chunk k holds chunk_nnz[k] finished entries at staging
// position chunk_off[k]; they go to C position chunk_base[k].  The flattened output space of the
// batch (prefix sums of chunk_nnz) is cut into equal tiles, one per block; a thread finds the chunk
// of its output position in a shared-memory copy of the tile's chunk table, so both the reads and
// the writes are contiguous runs.  Pure streaming: 2 * (4 + value bytes) per entry.
#pragma once
#include "gm_common.cuh"

namespace gm {

constexpr int kGatherThreads = 256;
constexpr int kGatherTile = 4096;
#ifndef GM_GATHER_BATCH
#define GM_GATHER_BATCH 4
#endif
constexpr int kGatherBatch = GM_GATHER_BATCH;  // positions a thread has in flight
constexpr int kGatherChunkCap = 1024;  // chunks staged in shared memory per tile; more -> per-element search

template <typename V>
__global__ void __launch_bounds__(kGatherThreads) k7_gather(
    const int32_t* __restrict__ s_col_in, const V* __restrict__ s_val_in,  // staging buffer (compacted chunks)
    const i64* __restrict__ chunk_off, const i64* __restrict__ chunk_nnz_off, const i64* __restrict__ chunk_base,
    i64 n_chunks, const TileMeta* __restrict__ tile_meta, int32_t* __restrict__ c_col, V* __restrict__ c_val,
    i64 c_capacity, int* __restrict__ err) {
  __shared__ int s_rel[kGatherChunkCap + 1];
  __shared__ i64 s_src[kGatherChunkCap];
  __shared__ i64 s_dst[kGatherChunkCap];
  const i64 n_out = chunk_nnz_off[n_chunks];
  const i64 t0 = static_cast<i64>(blockIdx.x) * kGatherTile;
  if (t0 >= n_out) return;
  const int tn = static_cast<int>(min(static_cast<i64>(kGatherTile), n_out - t0));
  const TileMeta tm = tile_meta[blockIdx.x];
  const i64 k_lo = tm.first;
  const int n_k = tm.n;
  if (n_k <= kGatherChunkCap) {
    for (int i = threadIdx.x; i <= n_k; i += kGatherThreads) {
      s_rel[i] = (i == n_k) ? tn + 1 : clamp_rel(chunk_nnz_off[k_lo + i] - t0, -(1 << 30), tn + 1);
      if (i < n_k) {
        s_src[i] = chunk_off[k_lo + i];
        s_dst[i] = chunk_base[k_lo + i];
      }
    }
    __syncthreads();
    // each thread walks kGatherTile / kGatherThreads positions strided by the block; its chunk index only grows.
    // Positions are taken kGatherBatch at a time, all loads before the first store, so that a thread has that
    // many independent loads in flight (one at a time left the kernel waiting on memory at full occupancy).
    int cur = 0;
    for (int q0 = threadIdx.x; q0 < tn; q0 += kGatherBatch * kGatherThreads) {
      i64 dst[kGatherBatch];
      int32_t col[kGatherBatch];
      V val[kGatherBatch];
#pragma unroll
      for (int u = 0; u < kGatherBatch; ++u) {
        const int q = q0 + u * kGatherThreads;
        dst[u] = -1;
        if (q < tn) {
          // last chunk whose start is <= q (empty chunks share a start with their successor and are skipped)
          int lo = cur, hi = n_k - 1;
          while (lo < hi) {
            const int mid = lo + ((hi - lo + 1) >> 1);
            if (s_rel[mid] <= q) lo = mid; else hi = mid - 1;
          }
          cur = lo;
          const i64 r = static_cast<i64>(q) - s_rel[cur];
          dst[u] = s_dst[cur] + r;
          const i64 src = s_src[cur] + r;
          col[u] = s_col_in[src];
          val[u] = s_val_in[src];
        }
      }
#pragma unroll
      for (int u = 0; u < kGatherBatch; ++u) {
        if (dst[u] >= 0) {
          if (dst[u] < c_capacity) {
            c_col[dst[u]] = col[u];
            c_val[dst[u]] = val[u];
          } else {
            dev_set_error(err, kDevCapacity);
          }
        }
      }
    }
  } else {
    for (int q = threadIdx.x; q < tn; q += kGatherThreads) {
      const i64 p = t0 + q;
      const i64 k = last_le(chunk_nnz_off, k_lo, k_lo + n_k - 1, p);
      const i64 r = p - chunk_nnz_off[k];
      const i64 dst = chunk_base[k] + r;
      if (dst < c_capacity) {
        c_col[dst] = s_col_in[chunk_off[k] + r];
        c_val[dst] = s_val_in[chunk_off[k] + r];
      } else {
        dev_set_error(err, kDevCapacity);
      }
    }
  }
}

}  // namespace gm
