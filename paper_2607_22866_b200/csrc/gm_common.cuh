// Shared device helpers: warp/block reductions and scans, search, error flag.
#pragma once
#include <cuda_runtime.h>

#include <climits>
#include <cstdint>

namespace gm {

using u32 = uint32_t;
using u64 = unsigned long long;
using i64 = int64_t;

// Device-side status word: kernels never trap; they record the first problem here and skip the access.
enum DevError : int {
  kDevOk = 0,
  kDevCapacity = 1,      // a write would have gone past the room reserved for C
  kDevTableFull = 2,     // a light-row hash table overflowed (planner bug)
  kDevBadChunk = 3,      // an element landed in a chunk that does not own its column
  kDevTimeout = 4,       // a bounded wait on an asynchronous copy gave up
};

__device__ __forceinline__ void dev_set_error(int* flag, int code) { atomicCAS(flag, 0, code); }

__device__ __forceinline__ u32 lanemask_lt() {
  u32 m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

template <typename T>
__device__ __forceinline__ T warp_sum(T v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename T>
__device__ __forceinline__ T warp_inclusive_scan(T v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    T n = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += n;
  }
  return v;
}

// Exclusive scan of one value per thread over the whole block (blockDim.x a multiple of 32, at most 1024).
// `warp_tmp` points to 33 T's of shared memory.  Returns the exclusive prefix; *total gets the block sum.
// Contains two __syncthreads(); callers may reuse warp_tmp right after it returns only after another barrier.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T v, T* warp_tmp, T* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  const T inc = warp_inclusive_scan(v);
  if (lane == 31) warp_tmp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    T w = lane < nwarps ? warp_tmp[lane] : T(0);
    const T winc = warp_inclusive_scan(w);
    warp_tmp[lane] = winc - w;
    if (lane == 31) warp_tmp[32] = winc;
  }
  __syncthreads();
  *total = warp_tmp[32];
  return warp_tmp[warp] + inc - v;
}

// Largest index s in [lo, hi] with a[s] <= x, assuming a[lo] <= x and a non-decreasing.
template <typename T, typename X>
__device__ __forceinline__ i64 last_le(const T* __restrict__ a, i64 lo, i64 hi, X x) {
  while (lo < hi) {
    const i64 mid = lo + ((hi - lo + 1) >> 1);
    if (static_cast<X>(a[mid]) <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ int clamp_rel(i64 v, int lo, int hi) {
  return v < lo ? lo : (v > hi ? hi : static_cast<int>(v));
}

// ---- asynchronous bulk copies into shared memory (cp.async.bulk + mbarrier), this block's own memory only
__device__ __forceinline__ u32 smem_u32(const void* p) { return static_cast<u32>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(u64* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
// one arrival that also announces `bytes` of copies (0: a plain arrival)
__device__ __forceinline__ void mbar_arrive_expect_tx(u64* bar, u32 bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u64* bar, u32 parity) {
  u32 ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// 1-D bulk copy global -> this block's shared memory; both addresses 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, u32 bytes, u64* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// Bounded wait: polls with back-off at most `limit` times; false = gave up (the caller records kDevTimeout).
__device__ __forceinline__ bool mbar_wait_bounded(u64* bar, u32 parity, int limit) {
  for (int spins = 0; spins < limit; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(64);
  }
  return mbar_try_wait(bar, parity);
}
constexpr int kCopySpinLimit = 1 << 22;  // default number of polls before a wait on bulk copies gives up

// What a tile-per-block kernel needs to know about the groups (rows, parents, segments) its tile touches.
struct __align__(16) TileMeta {
  i64 first;  // group that contains the tile's first element
  int n;      // groups touched, first .. first + n - 1 (empty ones in between included)
  int off1;   // start of group first + 1 relative to the tile (tile + 1 if n == 1)
};

// For every tile of `tile` consecutive elements (positions bias + t*tile ... of a flattened space whose
// groups start at off[0..n_off)): the TileMeta above.  Run as its own small launch so that the searches of
// all tiles overlap; a block that searched for its own tile would keep all its threads waiting through ~20
// dependent global loads, and with this record the common tile (one or two groups) needs a single load.
__global__ void k_tile_bounds(const i64* __restrict__ off, i64 n_off, i64 bias, i64 n_elems, int tile,
                              TileMeta* __restrict__ meta, const i64* __restrict__ n_elems_dev = nullptr) {
  if (n_elems_dev) n_elems = *n_elems_dev;  // size only known on the device (then the grid covers an upper bound)
  const i64 n_tiles = (n_elems + tile - 1) / tile;
  for (i64 t = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; t < n_tiles;
       t += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 p0 = bias + t * tile;
    const i64 p1 = bias + min(n_elems, (t + 1) * tile) - 1;
    const i64 f = last_le(off, 0, n_off - 1, p0);
    const i64 l = last_le(off, f, n_off - 1, p1);
    TileMeta m;
    m.first = f;
    m.n = static_cast<int>(min(l - f + 1, static_cast<i64>(INT_MAX)));
    m.off1 = m.n >= 2 ? clamp_rel(off[f + 1] - p0, -1, tile + 1) : tile + 1;
    meta[t] = m;
  }
}


}  // namespace gm
