// K7 — moves the compacted chunks from the staging buffer into C (the write of Numeric() in
// Algorithm 3 once C.rowPtr is known).  Chunk k holds chunk_nnz[k] finished entries at staging
// position chunk_off[k]; they go to C position chunk_base[k].  The flattened output space of the
// batch (prefix sums of chunk_nnz) is cut into equal tiles, one per block; a thread finds the chunk
// of its output position in a shared-memory copy of the tile's chunk table, so both the reads and
// the writes are contiguous runs.  Pure streaming: 2 * (4 + value bytes) per entry.
// ALT: chunks that left the multisplit hierarchy early may lie in the other staging buffer (see ExitTags); their
// table entry carries a flag bit and the copy reads from there.
#pragma once
#include "gm_common.cuh"

namespace gm {

constexpr int kGatherThreads = 256;
constexpr int kGatherTile = 4096;
#ifndef GM_GATHER_BATCH
#define GM_GATHER_BATCH 6
#endif
// rows a warp has in flight.  The kernel is bound by bytes in flight (fp32 moved 4.3 TB/s where fp64, with twice the
// bytes per load, moved 6.1): measured 36.0 / 32.3 / 34.9 ms per step on R-MAT scale 20 with 4 / 6 / 8.
constexpr int kGatherBatch = GM_GATHER_BATCH;
constexpr int kGatherChunkCap = 1024;  // chunks staged in shared memory per tile; more -> per-element search

constexpr i64 kGatherAltBit = i64{1} << 62;

template <typename V, bool ALT = false>
__global__ void __launch_bounds__(kGatherThreads) k7_gather(
    const int32_t* __restrict__ s_col_in, const V* __restrict__ s_val_in,  // staging buffer (compacted chunks)
    const i64* __restrict__ chunk_off, const i64* __restrict__ chunk_nnz_off, const i64* __restrict__ chunk_base,
    i64 n_chunks, const TileMeta* __restrict__ tile_meta, int32_t* __restrict__ c_col, V* __restrict__ c_val,
    i64 c_capacity, int* __restrict__ err,
    const int32_t* __restrict__ s_col_alt = nullptr, const V* __restrict__ s_val_alt = nullptr,  // ALT: the other buffer,
    const unsigned char* __restrict__ tags = nullptr, u32 alt_bits = 0) {  // the chunks' tags, and which tags live there
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
        if constexpr (ALT) {
          if ((alt_bits >> tags[k_lo + i]) & 1u) s_src[i] |= kGatherAltBit;  // (tag 0 never has its bit set)
        }
        s_dst[i] = chunk_base[k_lo + i];
      }
    }
    __syncthreads();
    // A warp takes rows of 32 consecutive positions (row w, w + 8, ...), kGatherBatch rows at a time with all loads
    // before the first store.  Chunks hold hundreds of entries on average, so a row usually lies inside one chunk:
    // the warp keeps a uniform chunk cursor, and only a row that crosses a chunk boundary lets its lanes step on
    // from there (the per-position binary search this replaces cost more instructions than the copy itself).
    constexpr int kWarps = kGatherThreads / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int cur = 0;  // warp-uniform: last chunk whose start is <= the row's first position
    for (int r0 = warp * 32; r0 < tn; r0 += kGatherBatch * kWarps * 32) {
      i64 dst[kGatherBatch];
      int32_t col[kGatherBatch];
      V val[kGatherBatch];
#pragma unroll
      for (int u = 0; u < kGatherBatch; ++u) {
        const int q0 = r0 + u * kWarps * 32;
        const int q = q0 + lane;
        dst[u] = -1;
        if (q0 < tn) {  // (uniform)
          while (s_rel[cur + 1] <= q0) ++cur;  // empty chunks share a start with their successor and are skipped
          int k = cur;
          if (s_rel[cur + 1] < q0 + 32) {      // the row crosses into later chunks
            if (q < tn)
              while (s_rel[k + 1] <= q) ++k;
          }
          if (q < tn) {
            const i64 r = static_cast<i64>(q) - s_rel[k];
            dst[u] = s_dst[k] + r;
            i64 src = s_src[k];
            bool alt = false;
            if constexpr (ALT) { alt = (src & kGatherAltBit) != 0; src &= ~kGatherAltBit; }
            src += r;
            col[u] = (alt ? s_col_alt : s_col_in)[src];
            val[u] = (alt ? s_val_alt : s_val_in)[src];
          }
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
        bool alt = false;
        if constexpr (ALT) alt = (alt_bits >> tags[k]) & 1u;
        c_col[dst] = (alt ? s_col_alt : s_col_in)[chunk_off[k] + r];
        c_val[dst] = (alt ? s_val_alt : s_val_in)[chunk_off[k] + r];
      } else {
        dev_set_error(err, kDevCapacity);
      }
    }
  }
}

}  // namespace gm
