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
// Output positions per block.  Measured on R-MAT scale 20 fp32 (ms per step of this kernel) with 2048 / 4096 / 8192 /
// 16384: 33.6 / 30.2 / 28.9 / 28.6; the clipped-Zipf pair, whose chunks hold a few entries each, prefers 8192 to 16384
// (0.95 against 1.18 ms: fewer tiles with more chunks than the shared table holds).
constexpr int kGatherTile = 8192;
// Rows of 64 positions a warp has in flight.  With 4-byte accesses and rows of 32 the kernel wanted six in flight
// (36.0 / 32.3 / 34.9 ms with 4 / 6 / 8); with paired accesses one row of 64 is best (30.2 / 30.5 / 35.3 / 38.7 ms with
// 1 / 2 / 3 / 4 at 4096 positions per block: registers cost occupancy).
constexpr int kGatherBatch = 1;
constexpr int kGatherChunkCap = 1024;  // chunks staged in shared memory per tile; more -> per-element search

constexpr i64 kGatherAltBit = i64{1} << 62;
template <typename V> struct Pair;
template <> struct Pair<float> { using type = float2; };
template <> struct Pair<double> { using type = double2; };

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
    // A warp takes rows of 64 consecutive positions, kGatherBatch rows at a time with all loads before the first
    // store.  Chunks hold hundreds of entries on average, so a row usually lies inside one chunk (the warp keeps a
    // uniform chunk cursor); then every lane copies two neighbouring entries with one 8-byte load per array (16-byte
    // for fp64 values): the kernel is bound by the bytes it has in flight, and a load instruction then carries twice
    // as many.  If the row's source starts at an odd index the pairs start one entry early, and lane 0, whose first
    // entry is not the row's, fetches the row's last one instead.  A row that crosses a chunk boundary lets every lane
    // find the chunks of its two positions from the cursor on.
    constexpr int kWarps = kGatherThreads / 32;
    constexpr int kRow = 64;
    using V2 = typename Pair<V>::type;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int cur = 0;  // warp-uniform: last chunk whose start is <= the row's first position
    for (int r0 = warp * kRow; r0 < tn; r0 += kGatherBatch * kWarps * kRow) {
      i64 d0[kGatherBatch], d1[kGatherBatch];  // where the lane's two entries go (-1: nothing)
      int32_t c0[kGatherBatch], c1[kGatherBatch];
      V v0[kGatherBatch], v1[kGatherBatch];
#pragma unroll
      for (int u = 0; u < kGatherBatch; ++u) {
        const int q0 = r0 + u * kWarps * kRow;
        d0[u] = -1;
        d1[u] = -1;
        if (q0 < tn) {  // (uniform)
          while (s_rel[cur + 1] <= q0) ++cur;  // empty chunks share a start with their successor and are skipped
          if (q0 + kRow <= min(s_rel[cur + 1], tn)) {
            i64 src = s_src[cur];
            bool alt = false;
            if constexpr (ALT) { alt = (src & kGatherAltBit) != 0; src &= ~kGatherAltBit; }
            const int32_t* const colp = alt ? s_col_alt : s_col_in;
            const V* const valp = alt ? s_val_alt : s_val_in;
            const i64 off = static_cast<i64>(q0) - s_rel[cur];
            const i64 src0 = src + off, dst0 = s_dst[cur] + off;
            const i64 odd = src0 & 1;
            const i64 a = src0 - odd + 2 * lane;  // even: the pair is naturally aligned
            const int2 cc = *reinterpret_cast<const int2*>(colp + a);
            const V2 vv = *reinterpret_cast<const V2*>(valp + a);
            c0[u] = cc.x; c1[u] = cc.y;
            v0[u] = vv.x; v1[u] = vv.y;
            d0[u] = dst0 - odd + 2 * lane;
            d1[u] = d0[u] + 1;
            if (odd && lane == 0) {
              c0[u] = colp[src0 + kRow - 1];
              v0[u] = valp[src0 + kRow - 1];
              d0[u] = dst0 + kRow - 1;
            }
          } else {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int q = q0 + h * 32 + lane;
              if (q < tn) {
                int k = cur;
                while (s_rel[k + 1] <= q) ++k;
                const i64 r = static_cast<i64>(q) - s_rel[k];
                i64 src = s_src[k];
                bool alt = false;
                if constexpr (ALT) { alt = (src & kGatherAltBit) != 0; src &= ~kGatherAltBit; }
                src += r;
                const int32_t c = (alt ? s_col_alt : s_col_in)[src];
                const V v = (alt ? s_val_alt : s_val_in)[src];
                if (h == 0) { c0[u] = c; v0[u] = v; d0[u] = s_dst[k] + r; }
                else { c1[u] = c; v1[u] = v; d1[u] = s_dst[k] + r; }
              }
            }
          }
        }
      }
#pragma unroll
      for (int u = 0; u < kGatherBatch; ++u) {
        if (max(d0[u], d1[u]) >= c_capacity) {
          dev_set_error(err, kDevCapacity);
        } else if (d0[u] >= 0 && d1[u] == d0[u] + 1 && !(d0[u] & 1)) {
          *reinterpret_cast<int2*>(c_col + d0[u]) = make_int2(c0[u], c1[u]);
          V2 vv;
          vv.x = v0[u]; vv.y = v1[u];
          *reinterpret_cast<V2*>(c_val + d0[u]) = vv;
        } else {
          if (d0[u] >= 0) { c_col[d0[u]] = c0[u]; c_val[d0[u]] = v0[u]; }
          if (d1[u] >= 0) { c_col[d1[u]] = c1[u]; c_val[d1[u]] = v1[u]; }
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
