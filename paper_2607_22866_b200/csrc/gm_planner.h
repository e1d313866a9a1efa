// Host-side planner (Section III-D, GetMagnusParams) and the batch cutter.  Pure C++: no CUDA.
#pragma once
#include <cstdint>
#include <vector>

#include "gmagnus.h"

namespace gm {

constexpr int kMultisplitBinCap = 2048;  // (parent, child) bins one multisplit tile keeps in smem
constexpr int kMinSmemBytes = 16384;
// threads of one dense-accumulator block when `ctas_per_sm` of them share an SM (1024 threads per SM in total)
int acc_block_threads(int ctas_per_sm);

inline int ilog2_floor(uint64_t x) {
  int l = 0;
  while (x >>= 1) ++l;
  return l;
}
inline uint64_t pow2_floor(uint64_t x) { return x ? (uint64_t{1} << ilog2_floor(x)) : 0; }
inline uint64_t pow2_ceil(uint64_t x) {
  if (x <= 1) return 1;
  return uint64_t{1} << (ilog2_floor(x - 1) + 1);
}

int value_bytes(int dtype);

// Fills `out` from (C.m, dtype, smem_bytes) and the overrides in `opts` (may be null).
int planner_params(int64_t c_cols, int dtype, size_t smem_bytes, const gm_plan_opts* opts,
                   gm_params* out);

// Shared memory the light-row kernel needs for a table of `slots` entries plus a sort buffer for
// `cap` (power of two) output entries.
size_t light_smem_bytes(int64_t slots, int64_t cap, int val_bytes, bool numeric);
// Shared memory one chunk accumulator of width W needs.
size_t acc_smem_bytes(int64_t W, int val_bytes, bool numeric);

struct Batch {
  int64_t h0, h1;      // heavy rows [h0, h1) (positions in the heavy-row list)
  int64_t elem0, elems;  // first product (global heavy numbering) and count
};

// Cuts the heavy rows into consecutive batches of at most `stage_elems` products.  heavy_prefix has
// n_heavy + 1 entries (exclusive prefix sums of IP over the heavy rows).  A row is never split; returns
// false if some row alone exceeds stage_elems.
bool cut_batches(const int64_t* heavy_prefix, int64_t n_heavy, int64_t stage_elems,
                 std::vector<Batch>* out);

}  // namespace gm
