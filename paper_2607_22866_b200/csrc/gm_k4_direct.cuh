// K4d — expansion straight into the first multisplit level's children (Algorithm 4 and the first level of
// Algorithm 5 in one pass over the products).
//
// A row of B has ascending columns, so the entries of B[k,:] that belong to level-0 child c of any row of C
// are one contiguous piece of the row, [bound[k][c], bound[k][c+1]).  A segment (one stored entry of a heavy
// row of A times one row of B) therefore contributes one contiguous run to every child, and where that run
// goes follows from counts alone, without looking at a single product:
//     run start = child_off[row][c] + (entries of the row's earlier segments in child c)
// The second term is a prefix sum over segments, column by column, of cnt[s][c] = bound[k_s][c+1] - bound[k_s][c].
// The expansion kernel then writes every product to its final level-0 position, and the separate histogram
// and multisplit passes over the staging buffer (4 + 2 * (4 + s_v) bytes per product) are not needed for the
// first level.  Deeper levels run as in Algorithm 5.
//
//   k_child_bounds   (plan)   bound[k][c], c = 0..F, for every row of B
//   k_g_tile_sums, k_g_scan_tiles, k_g_write   (per batch)   G[s][c] = sum of cnt[s'][c] over the batch's segments s' < s,
//                                                             and H[s][c] = G[s][c] - bound[k_s][c]
//   k_g_row_counts   (per batch)   (row, child) counts, whose exclusive scan is child_off
//   k_g_row_base     (per batch)   R[row][c] = child_off[row][c] - G[first segment of the row][c]
// so that the product at position i of B[k_s,:] (child c) goes to R[row][c] + H[s][c] + i  (32-bit wrap-around
// arithmetic; the result is a position inside the batch).
//   k4_expand_direct (per batch)   the products, in place
#pragma once
#include "gm_common.cuh"
#include "gm_k4_expand.cuh"

namespace gm {

constexpr int kGTile = 128;            // segments per tile of the column-wise prefix sum
constexpr int kDirectTableCap = 4096;  // (segment, child) run starts of one product tile kept in shared memory

// bound[k * (F + 1) + c] = number of entries of B[k,:] with (col >> shift) < c
__global__ void k_child_bounds(const i64* __restrict__ b_row_ptr, const int32_t* __restrict__ b_col, i64 n_rows_b, int F,
                               int shift, u32* __restrict__ bound) {
  const i64 n = n_rows_b * (F + 1);
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 k = i / (F + 1);
    const u32 c = static_cast<u32>(i - k * (F + 1));
    const i64 rs = b_row_ptr[k];
    i64 lo = rs, hi = b_row_ptr[k + 1];
    while (lo < hi) {
      const i64 mid = (lo + hi) >> 1;
      if ((static_cast<u32>(b_col[mid]) >> shift) >= c) hi = mid; else lo = mid + 1;
    }
    bound[i] = static_cast<u32>(lo - rs);
  }
}

// One thread per (tile of kGTile segments, child): a block of 256 threads covers 256 / F tiles (F <= 256).
__global__ void __launch_bounds__(256) k_g_tile_sums(const int32_t* __restrict__ seg_brow, i64 seg0, i64 n_seg_b,
                                                     const u32* __restrict__ bound, int F, u32* __restrict__ tile_sums) {
  const int c = threadIdx.x & (F - 1);
  const i64 tile = static_cast<i64>(blockIdx.x) * (256 / F) + threadIdx.x / F;
  const i64 s_begin = tile * kGTile;
  if (s_begin >= n_seg_b) return;
  const i64 s_end = min(n_seg_b, s_begin + kGTile);
  u32 sum = 0;
  for (i64 s = s_begin; s < s_end; ++s) {
    const u32* bp = bound + static_cast<i64>(seg_brow[seg0 + s]) * (F + 1) + c;
    sum += bp[1] - bp[0];
  }
  tile_sums[tile * F + c] = sum;
}

// Exclusive prefix over the tiles, one block per child: 256 tiles at a time with a carry.
__global__ void __launch_bounds__(256) k_g_scan_tiles(u32* __restrict__ tile_sums, i64 n_tiles, int F) {
  __shared__ u32 s_tmp[33];
  const int c = blockIdx.x;
  u32 carry = 0;
  for (i64 t0 = 0; t0 < n_tiles; t0 += 256) {
    const i64 t = t0 + threadIdx.x;
    const u32 v = t < n_tiles ? tile_sums[t * F + c] : 0u;
    u32 total;
    const u32 ex = block_exclusive_scan(v, s_tmp, &total);
    if (t < n_tiles) tile_sums[t * F + c] = carry + ex;
    carry += total;
    __syncthreads();  // s_tmp is reused by the next round
  }
}

// G[s * F + c] for s = 0..n_seg_b (the last row holds the batch's totals per child).
__global__ void __launch_bounds__(256) k_g_write(const int32_t* __restrict__ seg_brow, i64 seg0, i64 n_seg_b,
                                                 const u32* __restrict__ bound, int F, const u32* __restrict__ tile_sums,
                                                 u32* __restrict__ G, u32* __restrict__ H) {
  const int c = threadIdx.x & (F - 1);
  const i64 tile = static_cast<i64>(blockIdx.x) * (256 / F) + threadIdx.x / F;
  const i64 s_begin = tile * kGTile;
  if (s_begin >= n_seg_b) return;
  const i64 s_end = min(n_seg_b, s_begin + kGTile);
  u32 run = tile_sums[tile * F + c];
  for (i64 s = s_begin; s < s_end; ++s) {
    const u32* bp = bound + static_cast<i64>(seg_brow[seg0 + s]) * (F + 1) + c;
    const u32 b0 = bp[0];
    G[s * F + c] = run;
    H[s * F + c] = run - b0;
    run += bp[1] - b0;
  }
  if (s_end == n_seg_b) G[n_seg_b * F + c] = run;
}

// counts[r * F + c] = products of row r (of the batch) in child c
__global__ void k_g_row_counts(const u32* __restrict__ G, const i64* __restrict__ row_seg, i64 seg0, i64 n_rows_b, int F,
                               u32* __restrict__ counts) {
  const i64 n = n_rows_b * F;
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 r = i / F;
    const int c = static_cast<int>(i - r * F);
    counts[i] = G[(row_seg[r + 1] - seg0) * F + c] - G[(row_seg[r] - seg0) * F + c];
  }
}

// R[r * F + c] = child_off[r * F + c] - G[first segment of row r][c]  (mod 2^32)
__global__ void k_g_row_base(const u32* __restrict__ G, const i64* __restrict__ row_seg, i64 seg0, i64 n_rows_b, int F,
                             const i64* __restrict__ child_off, u32* __restrict__ R) {
  const i64 n = n_rows_b * F;
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 r = i / F;
    const int c = static_cast<int>(i - r * F);
    R[i] = static_cast<u32>(child_off[i]) - G[(row_seg[r] - seg0) * F + c];
  }
}

// Products per block: the row-order expansion's 8192 for a first level of few children, half of that from 32
// children on.  Measured, ms per step of this kernel with 2048 / 4096 / 8192 / 16384: R-MAT scale 20 fp32 (32 children)
// 71.9 / 60.3 / 61.7 / 67.4, R-MAT scale 21 fp64 (128 children) 80.5 / 72.5 / 77.9 / -; with 8 children (R-MAT scale 18
// fp32) 4096 took 2.03 ms under the profiler where 8192 takes 1.89, with 16 (scale 19) 21.8 against 21.4 ms per step.
constexpr int kDirectTileSmall = 4096;
constexpr int kDirectTileFanout = 32;  // from this fan-out on
inline int direct_tile(int F) { return F >= kDirectTileFanout ? kDirectTileSmall : kExpandTile; }
template <typename V, int kDirectTile>
__global__ void __launch_bounds__(kExpandThreads) k4_expand_direct(
    const i64* __restrict__ seg_off, const i64* __restrict__ seg_bstart, const i64* __restrict__ seg_j,
    const TileMeta* __restrict__ tile_meta,  // per tile: first segment and number of segments
    const V* __restrict__ a_val, const int32_t* __restrict__ b_col, const V* __restrict__ b_val,
    i64 elem0, i64 n_elems,  // first product of the batch (global heavy numbering), batch size
    const TileMeta* __restrict__ row_meta, const i64* __restrict__ row_off,  // the batch's rows: tile records, product offsets
    i64 seg0,                          // first segment of the batch
    int F, int shift,
    const u32* __restrict__ R,  // (row of the batch, child): child_off - G at the row's first segment
    const u32* __restrict__ H,  // (segment of the batch, child): G - bound
    int32_t* __restrict__ y_col, V* __restrict__ y_val) {
  __shared__ int s_tq[kDirectTableCap];  // (segment in tile, child) -> destination minus tile position
  __shared__ int s_roff[kExpandHistParents + 1];
  __shared__ int s_rel[kExpandSegCap + 1];
  __shared__ i64 s_bstart[kExpandSegCap];
  __shared__ V s_aval[kExpandSegCap];

  const i64 t0 = static_cast<i64>(blockIdx.x) * kDirectTile;
  const int tn = static_cast<int>(min(static_cast<i64>(kDirectTile), n_elems - t0));
  const i64 p0 = elem0 + t0;  // global product index of the tile's first element
  const TileMeta tm = tile_meta[blockIdx.x];
  const TileMeta rm = row_meta[blockIdx.x];
  const i64 s_lo = tm.first;
  const i64 n_seg = tm.n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const u32 fmask = static_cast<u32>(F - 1);
  const int log2F = 31 - __clz(F);
  const bool rows_staged = rm.n > 2 && rm.n <= kExpandHistParents;
  const bool table = n_seg <= kExpandSegCap && static_cast<i64>(n_seg) * F <= kDirectTableCap;

  // row of the batch (relative to the tile's first row) that owns tile position q
  auto row_of = [&](int q) -> i64 {
    if (rm.n <= 2) return q >= rm.off1 ? 1 : 0;
    if (rows_staged) {
      int lo = 0, hi = rm.n - 1;
      while (lo < hi) {
        const int mid = lo + ((hi - lo + 1) >> 1);
        if (s_roff[mid] <= q) lo = mid; else hi = mid - 1;
      }
      return lo;
    }
    return last_le(row_off, rm.first, rm.first + rm.n - 1, t0 + q) - rm.first;
  };
  // final position of the product at tile position q, of segment s (global numbering), row `par`, child c:
  // a segment starts at the beginning of its row of B, so the product's index in that row is p0 + q - seg_off[s]
  auto dst_global = [&](i64 s, i64 par, u32 c, int q) -> i64 {
    const u32 d = R[(rm.first + par) * F + c] + H[(s - seg0) * F + c] + static_cast<u32>(p0 + q - seg_off[s]);
    return static_cast<i64>(d);
  };

  if (rows_staged)
    for (int k = threadIdx.x; k <= rm.n; k += kExpandThreads)
      s_roff[k] = (k == rm.n) ? tn + 1 : clamp_rel(row_off[rm.first + k] - t0, -1, tn + 1);

  constexpr int kPerWarp = kDirectTile / (kExpandThreads / 32);
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
    if (table) {
      for (int idx = threadIdx.x; idx < static_cast<int>(n_seg) * F; idx += kExpandThreads) {
        const int k = idx >> log2F;
        const u32 c = static_cast<u32>(idx) & fmask;
        const i64 par = row_of(max(s_rel[k], 0));
        s_tq[idx] = static_cast<int>(R[(rm.first + par) * F + c] + H[(s_lo + k - seg0) * F + c] - static_cast<u32>(s_rel[k]));
      }
      __syncthreads();
    }
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
      int seg[kExpandUnroll];
      while (q0 >= s_rel[cur + 1]) ++cur;  // uniform: cur is the same in every lane here
      if (q0 + 32 * kExpandUnroll <= min(s_rel[cur + 1], w1)) {
        // the next 32 * kExpandUnroll products all come from the segment the warp is in
        const i64 src0 = s_bstart[cur] + (q0 - s_rel[cur]) + lane;
        const V a = s_aval[cur];
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
          col[u] = b_col[src0 + u * 32];
          val[u] = b_val[src0 + u * 32];
        }
        const i64 par = table ? 0 : row_of(q0);  // a segment lies inside one row
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
          const int q = q0 + u * 32 + lane;
          const u32 c = (static_cast<u32>(col[u]) >> shift) & fmask;
          const i64 dst = table ? static_cast<i64>(s_tq[(cur << log2F) + c]) + q : dst_global(s_lo + cur, par, c, q);
          y_col[dst] = col[u];
          y_val[dst] = a * val[u];
        }
        continue;
      }
#pragma unroll
      for (int u = 0; u < kExpandUnroll; ++u) {
        const int q = q0 + u * 32 + lane;
        seg[u] = 0;
        if (q < w1) {
          int s = cur;
          while (q >= s_rel[s + 1]) ++s;
          const i64 src = s_bstart[s] + (q - s_rel[s]);
          col[u] = b_col[src];
          val[u] = b_val[src];
          av[u] = s_aval[s];
          seg[u] = s;
          cur = s;
        }
        cur = __shfl_sync(0xffffffffu, cur, 31);  // monotone: the last lane is furthest
        // lanes past w1 keep their stale cur; lane 31 is only past w1 in the last step
      }
#pragma unroll
      for (int u = 0; u < kExpandUnroll; ++u) {
        const int q = q0 + u * 32 + lane;
        if (q < w1) {
          const u32 c = (static_cast<u32>(col[u]) >> shift) & fmask;
          const i64 dst = table ? static_cast<i64>(s_tq[(seg[u] << log2F) + c]) + q
                                : dst_global(s_lo + seg[u], row_of(q), c, q);
          y_col[dst] = col[u];
          y_val[dst] = av[u] * val[u];
        }
      }
    }
  } else {
    // more segments than the shared table holds (very short rows of B): search per element
    __syncthreads();  // s_roff
    for (int q = threadIdx.x; q < tn; q += kExpandThreads) {
      const i64 p = p0 + q;
      const i64 s = last_le(seg_off, s_lo, s_lo + n_seg - 1, p);
      const i64 src = seg_bstart[s] + (p - seg_off[s]);
      const int32_t cc = b_col[src];
      const u32 c = (static_cast<u32>(cc) >> shift) & fmask;
      const i64 dst = dst_global(s, row_of(q), c, q);
      y_col[dst] = cc;
      y_val[dst] = a_val[seg_j[s]] * b_val[src];
    }
  }
}

}  // namespace gm
