// K4c — expansion in outer-product order (Eq. 2, Algorithm 2 and Algorithm 4 as printed): C^ = sum over i of
// A[x_heavy, i] (x) B[i, :], so that a row of B is read once and reused by every heavy row that holds column i.
//
// MaskedCsr2Csc of Algorithm 3 becomes a counting sort of the batch's segments by their row of B (the entries of
// the batch's heavy rows grouped by column: the masked CSC of A[x_heavy, :]); the rows of B that no heavy row touches
// simply own no segment.  Where the paper reserves each slice's output range with an atomic on C^.rowPtr, the
// segment table already knows it (row-order offsets), so a segment's products go to  seg_off[s] - elem0 + index in
// the row of B  whatever the order in which segments are processed: the staging buffer ends up identical to the
// row-order expansion's.  The tile walk is the row-order kernel's, over the flattened product space in CSC order.
// Option expand_order = 1; the first multisplit level then runs as separate passes (the per-tile row bins of the
// fused histogram and the direct placement both lean on row order).
#pragma once
#include "gm_common.cuh"
#include "gm_k4_expand.cuh"

namespace gm {

// cnt[k] += segments of the batch that copy row k of B
__global__ void k_csc_count(const int32_t* __restrict__ seg_brow, i64 seg0, i64 n_seg_b, int32_t* __restrict__ cnt) {
  for (i64 s = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; s < n_seg_b; s += static_cast<i64>(gridDim.x) * blockDim.x)
    atomicAdd(&cnt[seg_brow[seg0 + s]], 1);
}

// perm[position in CSC order] = segment (relative to the batch), len = its products; the order inside a column is
// whatever the atomics give (it does not matter: every segment has its own destination)
__global__ void k_csc_scatter(const int32_t* __restrict__ seg_brow, const i64* __restrict__ seg_off, i64 seg0, i64 n_seg_b,
                              u64* __restrict__ cursor, int32_t* __restrict__ perm, int32_t* __restrict__ len) {
  for (i64 s = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; s < n_seg_b; s += static_cast<i64>(gridDim.x) * blockDim.x) {
    const u64 pos = atomicAdd(&cursor[seg_brow[seg0 + s]], 1ull);
    perm[pos] = static_cast<int32_t>(s);
    len[pos] = static_cast<int32_t>(seg_off[seg0 + s + 1] - seg_off[seg0 + s]);
  }
}

template <typename V>
__global__ void __launch_bounds__(kExpandThreads) k4_expand_csc(
    const i64* __restrict__ cs_off,   // n_seg_b + 1: flattened product space of the batch in CSC order (starts at 0)
    const int32_t* __restrict__ perm,  // CSC position -> segment relative to seg0
    const i64* __restrict__ seg_off, const i64* __restrict__ seg_bstart, const i64* __restrict__ seg_j, i64 seg0,
    const TileMeta* __restrict__ tile_meta,  // per tile: first CSC position and number of positions
    const V* __restrict__ a_val, const int32_t* __restrict__ b_col, const V* __restrict__ b_val,
    i64 elem0, i64 n_elems, int32_t* __restrict__ x_col, V* __restrict__ x_val) {
  __shared__ int s_rel[kExpandSegCap + 1];
  __shared__ u32 s_dst[kExpandSegCap];  // staging position of tile position q = s_dst[segment] + q (mod 2^32)
  __shared__ i64 s_bstart[kExpandSegCap];
  __shared__ V s_aval[kExpandSegCap];

  const i64 t0 = static_cast<i64>(blockIdx.x) * kExpandTile;
  const int tn = static_cast<int>(min(static_cast<i64>(kExpandTile), n_elems - t0));
  const TileMeta tm = tile_meta[blockIdx.x];
  const i64 w_lo = tm.first;
  const i64 n_seg = tm.n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kPerWarp = kExpandTile / (kExpandThreads / 32);
  const int w0 = warp * kPerWarp;
  const int w1 = min(tn, w0 + kPerWarp);

  if (n_seg <= kExpandSegCap) {
    for (int k = threadIdx.x; k <= n_seg; k += kExpandThreads) {
      if (k == n_seg) { s_rel[k] = tn + 1; continue; }
      const i64 rel = max(cs_off[w_lo + k] - t0, static_cast<i64>(INT_MIN));
      const i64 s = seg0 + perm[w_lo + k];
      s_rel[k] = static_cast<int>(rel);
      s_dst[k] = static_cast<u32>(seg_off[s] - elem0 - rel);
      s_bstart[k] = seg_bstart[s];
      s_aval[k] = a_val[seg_j[s]];
    }
    __syncthreads();
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
      u32 dst[kExpandUnroll];
      while (q0 >= s_rel[cur + 1]) ++cur;  // uniform
      if (q0 + 32 * kExpandUnroll <= min(s_rel[cur + 1], w1)) {
        const i64 src0 = s_bstart[cur] + (q0 - s_rel[cur]) + lane;
        const V a = s_aval[cur];
        const u32 d0 = s_dst[cur] + static_cast<u32>(q0 + lane);
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
          col[u] = b_col[src0 + u * 32];
          val[u] = b_val[src0 + u * 32];
        }
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
          x_col[d0 + u * 32] = col[u];
          x_val[d0 + u * 32] = a * val[u];
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
          dst[u] = s_dst[s] + static_cast<u32>(q);
          cur = s;
        }
        cur = __shfl_sync(0xffffffffu, cur, 31);
      }
#pragma unroll
      for (int u = 0; u < kExpandUnroll; ++u) {
        const int q = q0 + u * 32 + lane;
        if (q < w1) {
          x_col[dst[u]] = col[u];
          x_val[dst[u]] = av[u] * val[u];
        }
      }
    }
  } else {
    // more segments than the shared window holds (very short rows of B): search per element
    for (int q = threadIdx.x; q < tn; q += kExpandThreads) {
      const i64 p = t0 + q;
      const i64 w = last_le(cs_off, w_lo, w_lo + n_seg - 1, p);
      const i64 s = seg0 + perm[w];
      const i64 i = p - cs_off[w];
      const i64 src = seg_bstart[s] + i;
      const i64 d = seg_off[s] - elem0 + i;
      x_col[d] = b_col[src];
      x_val[d] = a_val[seg_j[s]] * b_val[src];
    }
  }
}

}  // namespace gm
