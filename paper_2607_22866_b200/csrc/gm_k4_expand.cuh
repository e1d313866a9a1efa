// K4 — expansion of the heavy rows' intermediate products (OuterProductKernel, Algorithm 4).
//
// The flattened product space of the heavy rows is cut into equal tiles, one per block (static,
// locally computed partition, as in Algorithm 4's GroupRange).  Products are generated in row
// order, so row h of the intermediate matrix owns the contiguous range [heavy_base[h],
// heavy_base[h+1]) and no atomic reservation of output ranges is needed: segment s (one stored
// entry of A scaled row of B) starts at seg_off[s], and product p of the tile is
//     col = B.col[seg_bstart[s] + (p - seg_off[s])],  val = A.val[seg_j[s]] * B.val[...]
// for the segment s that contains p (Eq. 3 with a division-free search).  Each warp walks a
// contiguous part of the tile, so reads of B and writes of the staging buffer are coalesced runs.
//
// The kernel can also count, for the first multisplit level, how many of the products it writes fall
// into each (row, child) bin — the Histogram step of Algorithm 3 — while the columns are still in
// registers, which saves a pass over the staging buffer (4 bytes per product).
#pragma once
#include "gm_common.cuh"

namespace gm {

constexpr int kExpandThreads = 256;
constexpr int kExpandTile = 8192;     // products per block
constexpr int kExpandSegCap = 1024;   // segments staged in shared memory; tiles with more take the slow path
constexpr int kExpandUnroll = 4;
constexpr int kExpandHistCap = 2048;      // (row, child) bins of the fused histogram kept in shared memory
constexpr int kExpandHistParents = 256;

template <typename V>
__global__ void __launch_bounds__(kExpandThreads) k4_expand(
    const i64* __restrict__ seg_off, const i64* __restrict__ seg_bstart, const i64* __restrict__ seg_j,
    const TileMeta* __restrict__ tile_meta,  // per tile: first segment and number of segments
    const V* __restrict__ a_val, const int32_t* __restrict__ b_col, const V* __restrict__ b_val,
    i64 elem0, i64 n_elems,           // first product of the batch (global heavy numbering), batch size
    int32_t* __restrict__ x_col, V* __restrict__ x_val,
    // fused level-0 histogram (hist_F == 0: off): rows of the batch as parents
    const TileMeta* __restrict__ row_meta, const i64* __restrict__ row_off, int hist_F, int hist_shift,
    u32* __restrict__ counts) {
  __shared__ u32 s_hist[kExpandHistCap];
  __shared__ int s_roff[kExpandHistParents + 1];
  __shared__ int s_rel[kExpandSegCap + 1];
  __shared__ i64 s_bstart[kExpandSegCap];
  __shared__ V s_aval[kExpandSegCap];

  const i64 t0 = static_cast<i64>(blockIdx.x) * kExpandTile;
  const int tn = static_cast<int>(min(static_cast<i64>(kExpandTile), n_elems - t0));
  const i64 p0 = elem0 + t0;  // global product index of the tile's first element
  const TileMeta tm = tile_meta[blockIdx.x];
  const i64 s_lo = tm.first;
  const i64 n_seg = tm.n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // fused histogram set-up: hist_mode 0 = off, 1 = bins in shared memory, 2 = too many rows in the tile (global atomics)
  int hist_mode = 0, h_npar = 1;
  TileMeta rm{};
  const u32 h_mask = static_cast<u32>(hist_F - 1);
  if (hist_F > 0) {
    rm = row_meta[blockIdx.x];
    h_npar = rm.n;
    hist_mode = (rm.n > kExpandHistParents || static_cast<i64>(rm.n) * hist_F > kExpandHistCap) ? 2 : 1;
    if (hist_mode == 1) {
      for (int b = threadIdx.x; b < rm.n * hist_F; b += kExpandThreads) s_hist[b] = 0;
      if (rm.n > 2)
        for (int k = threadIdx.x; k <= rm.n; k += kExpandThreads)
          s_roff[k] = (k == rm.n) ? tn + 1 : clamp_rel(row_off[rm.first + k] - t0, -1, tn + 1);
    }
  }
  if (hist_mode == 1) __syncthreads();  // bins zeroed before anybody counts (uniform: same record for all threads)
  // row (parent) of tile position q, as an index into the tile's bins; -1 = global path
  auto find_par = [&](int q) -> i64 {
    if (hist_mode == 1) {
      int par = q >= rm.off1 ? 1 : 0;
      if (h_npar > 2) {
        int lo = 0, hi = h_npar - 1;
        while (lo < hi) {
          const int mid = lo + ((hi - lo + 1) >> 1);
          if (s_roff[mid] <= q) lo = mid; else hi = mid - 1;
        }
        par = lo;
      }
      return par;
    }
    return last_le(row_off, rm.first, rm.first + rm.n - 1, t0 + q);
  };
  auto count_in = [&](i64 par, int32_t c) {
    const u32 child = (static_cast<u32>(c) >> hist_shift) & h_mask;
    if (hist_mode == 1) atomicAdd(&s_hist[static_cast<int>(par) * hist_F + child], 1u);
    else atomicAdd(&counts[par * hist_F + child], 1u);
  };
  auto count_product = [&](int q, int32_t c) {
    if (hist_mode != 0) count_in(find_par(q), c);
  };
  constexpr int kPerWarp = kExpandTile / (kExpandThreads / 32);
  const int w0 = warp * kPerWarp;
  const int w1 = min(tn, w0 + kPerWarp);

  if (n_seg <= kExpandSegCap) {
    for (int k = threadIdx.x; k <= n_seg; k += kExpandThreads) {
      // start of segment k relative to the tile; > -2^31 because a row of B has < 2^31 entries
      s_rel[k] = (k == n_seg) ? tn + 1 : static_cast<int>(max(seg_off[s_lo + k] - p0, static_cast<i64>(INT_MIN)));
      if (k < n_seg) {
        s_bstart[k] = seg_bstart[s_lo + k];
        s_aval[k] = a_val[seg_j[s_lo + k]];
      }
    }
    __syncthreads();
    // warp-uniform start: last segment whose start is <= w0 (zero-length segments are skipped by taking the last)
    int cur = 0;
    {
      int lo = 0, hi = static_cast<int>(n_seg) - 1;
      while (lo < hi) {
        const int mid = lo + ((hi - lo + 1) >> 1);
        if (s_rel[mid] <= w0) lo = mid; else hi = mid - 1;
      }
      cur = lo;
    }
    if (w0 < w1)
    for (int q0 = w0; q0 < w1; q0 += 32 * kExpandUnroll) {
      int32_t col[kExpandUnroll];
      V val[kExpandUnroll], av[kExpandUnroll];
      // heavy rows mostly multiply long rows of B: when the next 32 * kExpandUnroll products all come from the
      // segment the warp is in, nobody searches and the segment's data stays in uniform registers
      while (q0 >= s_rel[cur + 1]) ++cur;  // uniform: cur is the same in every lane here
      if (q0 + 32 * kExpandUnroll <= min(s_rel[cur + 1], w1)) {
        const i64 src0 = s_bstart[cur] + (q0 - s_rel[cur]) + lane;
        const V a = s_aval[cur];
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
          col[u] = b_col[src0 + u * 32];
          val[u] = b_val[src0 + u * 32];
        }
        const i64 par = hist_mode != 0 ? find_par(q0) : 0;  // a segment lies inside one row
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
          const int q = q0 + u * 32 + lane;
          x_col[t0 + q] = col[u];
          x_val[t0 + q] = a * val[u];
          if (hist_mode != 0) count_in(par, col[u]);
        }
        continue;
      }
#pragma unroll
      for (int u = 0; u < kExpandUnroll; ++u) {
        const int q = q0 + u * 32 + lane;
        if (q < w1) {
          int s = cur;
          while (q >= s_rel[s + 1]) ++s;
          const i64 src = s_bstart[s] + (q - s_rel[s]);
          col[u] = b_col[src];
          val[u] = b_val[src];
          av[u] = s_aval[s];
          cur = s;
        }
        cur = __shfl_sync(0xffffffffu, cur, 31);  // monotone: the last lane is furthest
        // lanes past w1 keep their stale cur; lane 31 is only past w1 in the last step
      }
#pragma unroll
      for (int u = 0; u < kExpandUnroll; ++u) {
        const int q = q0 + u * 32 + lane;
        if (q < w1) {
          x_col[t0 + q] = col[u];
          x_val[t0 + q] = av[u] * val[u];
          count_product(q, col[u]);
        }
      }
    }
  } else {
    // slow path: more segments than the shared table holds (very short rows of B): search per element
    for (int q = threadIdx.x; q < tn; q += kExpandThreads) {
      const i64 p = p0 + q;
      const i64 s = last_le(seg_off, s_lo, s_lo + n_seg - 1, p);
      const i64 src = seg_bstart[s] + (p - seg_off[s]);
      const int32_t c = b_col[src];
      x_col[t0 + q] = c;
      x_val[t0 + q] = a_val[seg_j[s]] * b_val[src];
      count_product(q, c);
    }
  }
  if (hist_mode == 1) {
    __syncthreads();
    const i64 g0 = rm.first * hist_F;
    for (int b = threadIdx.x; b < h_npar * hist_F; b += kExpandThreads) {
      const u32 c = s_hist[b];
      if (c) atomicAdd(&counts[g0 + b], c);
    }
  }
}

}  // namespace gm
