// K1 — row analysis (InterOffsets and ThreshPartition of Algorithm 3, Section III-A).
//   nz_len[j]  = nnz(B[A.col[j], :])                       (gather of B.rowPtr over A's entries)
//   nz_off     = exclusive scan of nz_len                   (the flattened product space, row order)
//   IP_i       = nz_off[A.rowPtr[i+1]] - nz_off[A.rowPtr[i]]
//   heavy iff IP_i > tau; light rows are binned by IP_i for the symbolic pass.
// For the heavy rows it also lays out the expansion kernel's segment table: one segment per stored
// entry of a heavy row (a whole row of B scaled by one value of A), in row order, so that heavy row
// h owns the contiguous product range [heavy_base[h], heavy_base[h+1]).
#pragma once
#include "gm_common.cuh"

namespace gm {

constexpr int kMaxLightBins = 8;

struct LightBins {
  int n_bins;
  int cap[kMaxLightBins];  // bin b holds rows with cap[b-1] < size <= cap[b]
};

__device__ __forceinline__ int light_bin_of(const LightBins& lb, i64 size) {
  int b = 0;
  while (b < lb.n_bins - 1 && size > lb.cap[b]) ++b;
  return b;
}

__global__ void k1_nz_len(const int32_t* __restrict__ a_col, i64 nnz_a, const i64* __restrict__ b_row_ptr,
                          int32_t* __restrict__ nz_len) {
  for (i64 j = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; j < nnz_a;
       j += static_cast<i64>(gridDim.x) * blockDim.x) {
    const int32_t c = a_col[j];
    nz_len[j] = static_cast<int32_t>(b_row_ptr[c + 1] - b_row_ptr[c]);
  }
}

struct K1Totals {
  u64 products_total;
  u64 products_heavy;
  u64 products_max_row;
  u64 c_nnz_upper;
  u64 rows_heavy;
  u64 rows_empty;
  u64 nnz_a_heavy;
  u64 pad;
};

__global__ void k1_row_products(const i64* __restrict__ a_row_ptr, i64 n_rows, const i64* __restrict__ nz_off,
                                i64 tau, i64 c_cols, i64* __restrict__ ip, int32_t* __restrict__ heavy_flag,
                                K1Totals* __restrict__ totals) {
  u64 tot = 0, hev = 0, mx = 0, up = 0, nh = 0, ne = 0, nzh = 0;
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_rows;
       i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 s = a_row_ptr[i], e = a_row_ptr[i + 1];
    const i64 p = nz_off[e] - nz_off[s];
    ip[i] = p;
    const bool heavy = p > tau;
    heavy_flag[i] = heavy ? 1 : 0;
    tot += p;
    if (heavy) { hev += p; ++nh; nzh += (e - s); }
    if (p == 0) ++ne;
    mx = p > static_cast<i64>(mx) ? p : mx;
    up += p < c_cols ? p : c_cols;
  }
  tot = warp_sum(tot); hev = warp_sum(hev); up = warp_sum(up); nh = warp_sum(nh); ne = warp_sum(ne);
  nzh = warp_sum(nzh);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const u64 m2 = __shfl_xor_sync(0xffffffffu, mx, o); mx = m2 > mx ? m2 : mx; }
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&totals->products_total, tot);
    atomicAdd(&totals->products_heavy, hev);
    atomicMax(&totals->products_max_row, mx);
    atomicAdd(&totals->c_nnz_upper, up);
    atomicAdd(&totals->rows_heavy, nh);
    atomicAdd(&totals->rows_empty, ne);
    atomicAdd(&totals->nnz_a_heavy, nzh);
  }
}

// x_heavy[h] = original row of heavy row h; heavy_ip[h], heavy_nnz[h] feed the two heavy prefix sums.
__global__ void k1_heavy_scatter(const int32_t* __restrict__ heavy_flag, const i64* __restrict__ heavy_pos,
                                 const i64* __restrict__ ip, const i64* __restrict__ a_row_ptr, i64 n_rows,
                                 int32_t* __restrict__ x_heavy, i64* __restrict__ heavy_ip, i64* __restrict__ heavy_nnz) {
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_rows;
       i += static_cast<i64>(gridDim.x) * blockDim.x) {
    if (heavy_flag[i]) {
      const i64 h = heavy_pos[i];
      x_heavy[h] = static_cast<int32_t>(i);
      heavy_ip[h] = ip[i];
      heavy_nnz[h] = a_row_ptr[i + 1] - a_row_ptr[i];
    }
  }
}

// Segment s (the s-th stored entry of the heavy rows, in row order) starts at product seg_off[s],
// copies B's entries from position seg_bstart[s], and is scaled by A.val[seg_j[s]].
__global__ void k1_heavy_segments(const int32_t* __restrict__ x_heavy, i64 n_heavy, const i64* __restrict__ heavy_nz_off,
                                  const i64* __restrict__ heavy_base, const i64* __restrict__ a_row_ptr,
                                  const int32_t* __restrict__ a_col, const i64* __restrict__ nz_off,
                                  const i64* __restrict__ b_row_ptr, i64 n_seg, i64* __restrict__ seg_off,
                                  i64* __restrict__ seg_bstart, i64* __restrict__ seg_j,
                                  int32_t* __restrict__ seg_brow, int32_t* __restrict__ seg_hrow) {
  for (i64 s = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; s <= n_seg;
       s += static_cast<i64>(gridDim.x) * blockDim.x) {
    if (s == n_seg) { seg_off[s] = heavy_base[n_heavy]; continue; }
    const i64 h = last_le(heavy_nz_off, 0, n_heavy - 1, s);  // rows with no entries are never heavy
    const i64 r = x_heavy[h];
    const i64 rs = a_row_ptr[r];
    const i64 j = rs + (s - heavy_nz_off[h]);
    seg_off[s] = heavy_base[h] + (nz_off[j] - nz_off[rs]);
    seg_bstart[s] = b_row_ptr[a_col[j]];
    seg_j[s] = j;
    seg_brow[s] = a_col[j];
    seg_hrow[s] = static_cast<int32_t>(h);
  }
}

// Bins rows by a per-row size (IP_i for the symbolic pass, nnz(C[i,:]) for the numeric pass).  Rows
// with size 0, rows flagged in `skip` (heavy rows) and rows above the last cap are left out.  Bin b's list
// starts at rows_out + b * bin_stride; bin_fill[b] counts it.  Each block reserves one contiguous range
// per bin, so row order is preserved inside a block.
template <typename SizeT>
__global__ void __launch_bounds__(256) k1_bin_rows(const SizeT* __restrict__ size, const int32_t* __restrict__ skip,
                                                   i64 n_rows, LightBins lb, i64 bin_stride,
                                                   int* __restrict__ bin_fill, int32_t* __restrict__ rows_out,
                                                   i64 row0 = 0) {  // size/skip start at row row0; rows_out gets global ids
  __shared__ int s_cnt[kMaxLightBins];
  __shared__ int s_base[kMaxLightBins];
  const i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (threadIdx.x < kMaxLightBins) s_cnt[threadIdx.x] = 0;
  __syncthreads();
  int bin = -1, rank = 0;
  if (i < n_rows && !(skip && skip[i])) {
    const i64 sz = static_cast<i64>(size[i]);
    if (sz > 0 && sz <= lb.cap[lb.n_bins - 1]) bin = light_bin_of(lb, sz);
  }
  // rank inside the block in row order: warp ballot per bin, then per-warp bases
  __shared__ int s_warp[8][kMaxLightBins];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b = 0; b < lb.n_bins; ++b) {
    const u32 m = __ballot_sync(0xffffffffu, bin == b);
    if (bin == b) rank = __popc(m & lanemask_lt());
    if (lane == 0) s_warp[warp][b] = __popc(m);
  }
  __syncthreads();
  if (threadIdx.x < lb.n_bins) {
    int run = 0;
    for (int w = 0; w < 8; ++w) { const int c = s_warp[w][threadIdx.x]; s_warp[w][threadIdx.x] = run; run += c; }
    s_cnt[threadIdx.x] = run;
    s_base[threadIdx.x] = run ? atomicAdd(&bin_fill[threadIdx.x], run) : 0;
  }
  __syncthreads();
  if (bin >= 0)
    rows_out[bin * bin_stride + s_base[bin] + s_warp[warp][bin] + rank] = static_cast<int32_t>(row0 + i);
}

}  // namespace gm
