// Device-wide exclusive prefix sum in three launches (tile sums, spine, tile scans): no block ever
// waits on another, so there is no spin loop to bound.  Used for every row_ptr-like array on the
// path (InterOffsets, C^.rowPtr, C^_reord.rowPtr, C.rowPtr of Algorithm 3).
#pragma once
#include "gm_common.cuh"

namespace gm {

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;

inline i64 scan_tmp_elems(i64 n) { return (n + kScanTile - 1) / kScanTile + 1; }

template <typename In>
__global__ void __launch_bounds__(kScanThreads) scan_tile_sums(const In* __restrict__ in, i64 n, i64* __restrict__ tile_sum) {
  __shared__ i64 tmp[33];
  const i64 t0 = static_cast<i64>(blockIdx.x) * kScanTile;
  i64 s = 0;
#pragma unroll
  for (int k = 0; k < kScanItems; ++k) {
    const i64 i = t0 + k * kScanThreads + threadIdx.x;
    if (i < n) s += static_cast<i64>(in[i]);
  }
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) tmp[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    i64 w = threadIdx.x < kScanThreads / 32 ? tmp[threadIdx.x] : 0;
    w = warp_sum(w);
    if (threadIdx.x == 0) tile_sum[blockIdx.x] = w;
  }
}

// One block: tile_sum -> exclusive prefixes (+ carry_in).  Writes the grand total (+ carry) to
// out_total (may be null) and to carry_out (may be null, may alias carry_in).
__global__ void __launch_bounds__(1024) scan_spine(i64* __restrict__ tile_sum, i64 n_tiles, const i64* carry_in,
                                                  i64* carry_out, i64* out_total) {
  __shared__ i64 tmp[33];
  __shared__ i64 running;
  if (threadIdx.x == 0) running = carry_in ? *carry_in : 0;
  __syncthreads();
  for (i64 b = 0; b < n_tiles; b += blockDim.x) {
    const i64 i = b + threadIdx.x;
    const i64 v = i < n_tiles ? tile_sum[i] : 0;
    i64 total;
    const i64 ex = block_exclusive_scan(v, tmp, &total);
    const i64 base = running;
    if (i < n_tiles) tile_sum[i] = base + ex;
    __syncthreads();
    if (threadIdx.x == 0) running = base + total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    if (out_total) *out_total = running;
    if (carry_out) *carry_out = running;
  }
}

template <typename In, typename Out>
__global__ void __launch_bounds__(kScanThreads) scan_tiles(const In* __restrict__ in, i64 n, const i64* __restrict__ tile_base,
                                                          Out* __restrict__ out, Out* __restrict__ out2) {
  __shared__ i64 tmp[33];
  const i64 t0 = static_cast<i64>(blockIdx.x) * kScanTile + static_cast<i64>(threadIdx.x) * kScanItems;
  i64 v[kScanItems];
  i64 s = 0;
#pragma unroll
  for (int k = 0; k < kScanItems; ++k) {
    v[k] = (t0 + k < n) ? static_cast<i64>(in[t0 + k]) : 0;
    s += v[k];
  }
  i64 total;
  i64 ex = block_exclusive_scan(s, tmp, &total) + tile_base[blockIdx.x];
#pragma unroll
  for (int k = 0; k < kScanItems; ++k) {
    if (t0 + k < n) {
      out[t0 + k] = static_cast<Out>(ex);
      if (out2) out2[t0 + k] = static_cast<Out>(ex);
    }
    ex += v[k];
  }
}

// out[0..n) = carry + exclusive prefix sums of in, out[n] = carry + total (out has n + 1 entries).
// out2 (optional, n entries) receives a second copy of out[0..n).  tmp has scan_tmp_elems(n) entries.
// `in` and `out` may alias when In and Out have the same size.
template <typename In, typename Out>
void exclusive_scan(const In* in, Out* out, i64 n, i64* tmp, const i64* carry_in, i64* carry_out, Out* out2,
                    cudaStream_t st) {
  static_assert(sizeof(Out) == 8, "offsets are 64-bit");
  const i64 tiles = (n + kScanTile - 1) / kScanTile;
  if (tiles > 0) scan_tile_sums<In><<<static_cast<unsigned>(tiles), kScanThreads, 0, st>>>(in, n, tmp);
  scan_spine<<<1, 1024, 0, st>>>(tmp, tiles, carry_in, carry_out, reinterpret_cast<i64*>(out + n));
  if (tiles > 0)
    scan_tiles<In, Out><<<static_cast<unsigned>(tiles), kScanThreads, 0, st>>>(in, n, tmp, out, out2);
}

}  // namespace gm
