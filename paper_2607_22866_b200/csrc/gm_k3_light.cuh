// K3 — light rows: Gustavson's method (Algorithm 1) with a shared-memory hash accumulator
// (Section III-E: hashing with linear probing, then a bitonic sort of the row).
//
// One *group* of G threads owns one row at a time: G = 8 or 32 threads of a warp for short rows,
// the whole block for long ones.  Inside a group, sub-groups of LPN lanes take one stored entry of
// A[i,:] each and stride over the matching row of B.
//   symbolic pass: insert columns only, count successful first insertions -> nnz(C[i,:])
//   numeric pass : insert columns and add values, compact the occupied slots into a sort buffer as
//                  (column << 32 | slot), bitonic-sort it, write columns and values in order.
#pragma once
#include "gm_common.cuh"

namespace gm {

constexpr int32_t kEmptyKey = -1;

template <int G>
__device__ __forceinline__ u32 group_mask() {
  if constexpr (G >= 32) {
    return 0xffffffffu;
  } else {
    const u32 lane = threadIdx.x & 31;
    return ((1u << G) - 1u) << (lane & ~(G - 1));
  }
}

template <int G>
__device__ __forceinline__ void group_sync() {
  if constexpr (G >= 64) {
    __syncthreads();
  } else {
    __syncwarp(group_mask<G>());
  }
}

__device__ __forceinline__ u32 hash_slot(int32_t col, u32 slots) {
  const u32 h = static_cast<u32>(col) * 0x9E3779B1u;
  return static_cast<u32>((static_cast<u64>(h) * slots) >> 32);
}

// Shared-memory layout of one group: [sort buffer: cap x u64][values: slots x V][keys: slots x i32]
// Groups narrower than a warp share one: their regions are staggered by `group` words, because power-of-two
// region sizes would put the same array index of every group of a warp into the same bank (measured on the
// 8-lane groups: half of all shared-memory wavefronts were conflict replays).
template <typename V, bool NUMERIC>
__host__ __device__ inline size_t light_group_bytes(int slots, int cap, int group) {
  size_t b = static_cast<size_t>(slots) * 4;
  if (NUMERIC) b += static_cast<size_t>(slots) * sizeof(V) + static_cast<size_t>(cap) * 8;
  b = (b + 15) & ~size_t{15};
  if (group < 32) b += static_cast<size_t>(group) * 4;  // 8 lanes: 32 bytes, keeps 16-byte alignment
  return b;
}

template <typename V, int G, int LPN, int BT, bool NUMERIC>
__global__ void __launch_bounds__(BT) k3_light_rows(
    const i64* __restrict__ a_row_ptr, const int32_t* __restrict__ a_col, const V* __restrict__ a_val,
    const i64* __restrict__ b_row_ptr, const int32_t* __restrict__ b_col, const V* __restrict__ b_val,
    const int32_t* __restrict__ rows, const int* __restrict__ n_rows_ptr, int slots, int cap,
    int32_t* __restrict__ row_nnz,                         // symbolic: out
    const i64* __restrict__ c_row_ptr, int32_t* __restrict__ c_col, V* __restrict__ c_val, i64 c_capacity,  // numeric
    int* __restrict__ err) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int kGroups = BT / G;
  const int gid = threadIdx.x / G;   // group inside the block
  const int t = threadIdx.x % G;     // thread inside the group
  unsigned char* base = smem_raw + static_cast<size_t>(gid) * light_group_bytes<V, NUMERIC>(slots, cap, G);
  u64* sortbuf = reinterpret_cast<u64*>(base);
  V* vals = reinterpret_cast<V*>(base + (NUMERIC ? static_cast<size_t>(cap) * 8 : 0));
  int32_t* keys = reinterpret_cast<int32_t*>(base + (NUMERIC ? static_cast<size_t>(cap) * 8 + static_cast<size_t>(slots) * sizeof(V) : 0));
  __shared__ int s_count[kGroups];

  const int n_rows = *n_rows_ptr;
  for (int ri = blockIdx.x * kGroups + gid; ri < n_rows; ri += gridDim.x * kGroups) {
    const int row = rows[ri];
    for (int s = t; s < slots; s += G) {
      keys[s] = kEmptyKey;
      if (NUMERIC) vals[s] = V(0);
    }
    if (t == 0) s_count[gid] = 0;
    group_sync<G>();

    // ---- accumulate (Algorithm 1, inner two loops)
    int inserted = 0;
    const i64 rs = a_row_ptr[row], re = a_row_ptr[row + 1];
    constexpr int kSub = G / LPN;
    const int sub = t / LPN, sl = t % LPN;
    for (i64 j = rs + sub; j < re; j += kSub) {
      const int32_t brow = a_col[j];
      V av = V(0);
      if (NUMERIC) av = a_val[j];
      const i64 be = b_row_ptr[brow + 1];
      for (i64 k = b_row_ptr[brow] + sl; k < be; k += LPN) {
        const int32_t c = b_col[k];
        u32 h = hash_slot(c, static_cast<u32>(slots));
        int probes = 0;
        for (;;) {
          int32_t cur = keys[h];
          if (cur == kEmptyKey) {
            cur = atomicCAS(&keys[h], kEmptyKey, c);
            if (cur == kEmptyKey) { ++inserted; cur = c; }
          }
          if (cur == c) {
            if (NUMERIC) atomicAdd(&vals[h], av * b_val[k]);
            break;
          }
          h = (h + 1 == static_cast<u32>(slots)) ? 0u : h + 1;
          if (++probes > slots) { dev_set_error(err, kDevTableFull); break; }
        }
      }
    }

    if (!NUMERIC) {
      // ---- symbolic: nnz(C[row,:]) = number of first insertions
      if constexpr (G <= 32) {
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) inserted += __shfl_xor_sync(group_mask<G>(), inserted, o, G);
        if (t == 0) row_nnz[row] = inserted;
        group_sync<G>();
      } else {
        if (inserted) atomicAdd(&s_count[gid], inserted);
        group_sync<G>();
        if (t == 0) row_nnz[row] = s_count[gid];
        group_sync<G>();
      }
      continue;
    }

    // ---- numeric: compact -> sort -> write
    group_sync<G>();
    const i64 out0 = c_row_ptr[row];
    const int n = static_cast<int>(c_row_ptr[row + 1] - out0);
    if constexpr (G >= 32) {
      // one counter update per warp and step: the occupied lanes take consecutive places
      const u32 lane = threadIdx.x & 31;
      for (int s0 = 0; s0 < slots; s0 += G) {
        const int s = s0 + t;
        const int32_t c = s < slots ? keys[s] : kEmptyKey;
        const u32 occ = __ballot_sync(0xffffffffu, c != kEmptyKey);
        int idx = 0;
        if (lane == 0 && occ) idx = atomicAdd(&s_count[gid], __popc(occ));
        idx = __shfl_sync(0xffffffffu, idx, 0) + __popc(occ & lanemask_lt());
        if (c != kEmptyKey && idx < cap) sortbuf[idx] = (static_cast<u64>(static_cast<u32>(c)) << 32) | static_cast<u32>(s);
      }
    } else {
      for (int s = t; s < slots; s += G) {
        const int32_t c = keys[s];
        if (c != kEmptyKey) {
          const int idx = atomicAdd(&s_count[gid], 1);
          if (idx < cap) sortbuf[idx] = (static_cast<u64>(static_cast<u32>(c)) << 32) | static_cast<u32>(s);
        }
      }
    }
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    group_sync<G>();
    if (s_count[gid] != n || n > cap) { dev_set_error(err, kDevTableFull); group_sync<G>(); continue; }
    for (int s = n + t; s < n2; s += G) sortbuf[s] = ~u64{0};
    group_sync<G>();
    for (int k = 2; k <= n2; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int p = t; p < (n2 >> 1); p += G) {
          const int i = 2 * p - (p & (j - 1));
          const int q = i + j;
          const u64 x = sortbuf[i], y = sortbuf[q];
          const bool up = (i & k) == 0;
          if ((x > y) == up) { sortbuf[i] = y; sortbuf[q] = x; }
        }
        group_sync<G>();
      }
    }
    if (out0 + n > c_capacity) {
      dev_set_error(err, kDevCapacity);
    } else {
      for (int s = t; s < n; s += G) {
        const u64 kv = sortbuf[s];
        c_col[out0 + s] = static_cast<int32_t>(kv >> 32);
        c_val[out0 + s] = vals[static_cast<u32>(kv)];
      }
    }
    group_sync<G>();
  }
}

}  // namespace gm
