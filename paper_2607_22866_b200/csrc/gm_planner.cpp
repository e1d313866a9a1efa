// Host-side planner: parameter selection of Section III-D re-derived for one B200 SM's shared
// memory, and the cutter that splits the heavy rows into staging-buffer batches.
#include "gm_planner.h"

#include <algorithm>

namespace gm {

int value_bytes(int dtype) { return dtype == GM_F32 ? 4 : dtype == GM_F64 ? 8 : 0; }

size_t light_smem_bytes(int64_t slots, int64_t cap, int val_bytes, bool numeric) {
  // keys + (numeric: values + 64-bit sort buffer of `cap` entries)
  size_t b = static_cast<size_t>(slots) * 4;
  if (numeric) b += static_cast<size_t>(slots) * val_bytes + static_cast<size_t>(cap) * 8;
  return b;
}

int acc_block_threads(int ctas_per_sm) { return 1024 / ctas_per_sm; }

size_t acc_smem_bytes(int64_t W, int val_bytes, bool numeric) {
  // bitmap (1 bit per column) + an 8-byte list entry per bitmap word (flush) + (numeric: one value per column);
  // a fifth of the column bytes is kept back for the kernels' other tables
  size_t b = static_cast<size_t>(W / 32) * 12 + 256;
  if (numeric) b += static_cast<size_t>(W) * val_bytes + static_cast<size_t>(W) * val_bytes / 5;
  return b;
}

int planner_params(int64_t c_cols, int dtype, size_t smem_bytes, const gm_plan_opts* opts,
                   gm_params* out) {
  if (!out || c_cols < 0) return GM_ERR_INVALID_ARG;
  const int sv = value_bytes(dtype);
  if (!sv) return GM_ERR_DTYPE;
  if (smem_bytes < static_cast<size_t>(kMinSmemBytes) || smem_bytes > (size_t{1} << 20))
    return GM_ERR_UNSUPPORTED_SMEM;
  gm_plan_opts o{};
  if (opts) o = *opts;
  *out = gm_params{};
  const int64_t S = static_cast<int64_t>(smem_bytes);
  const int64_t reserve = 1024;  // static shared memory of the kernels
  const int64_t se = 4 + sv;     // bytes of one (column, value) pair

  // --- tau (Eq. 4).  The paper's capacity is s_LM / (alpha * bytes per entry) with alpha = 2 table
  // slots per stored entry.  Here the numeric pass also keeps a 64-bit sort buffer of `cap` entries
  // next to the table and cap is a power of two (bitonic sort), so: the largest power of two cap
  // with cap * 8 + 1.5 * cap * se <= S, and as many slots as fit, at most alpha * cap.
  int64_t cap = 16;
  while ((cap * 2) * 8 + 3 * (cap * 2) * se / 2 <= S - reserve) cap *= 2;
  if (o.tau < 0) return GM_ERR_INVALID_ARG;
  if (o.tau > cap) return GM_ERR_INVALID_ARG;  // would not fit the light-row accumulator

  // --- W = n_denseNumeric: columns one dense accumulator (values + bitmap) covers, power of two.
  int ctas = o.acc_ctas_per_sm ? o.acc_ctas_per_sm : 1;
  if (ctas != 1 && ctas != 2 && ctas != 4 && ctas != 8) return GM_ERR_INVALID_ARG;
  out->acc_ctas_per_sm = ctas;
  const int64_t acc_budget = S / ctas - reserve;
  out->acc_block_threads = acc_block_threads(ctas);
  int64_t W = 32;
  while (static_cast<int64_t>(acc_smem_bytes(W * 2, sv, true)) <= acc_budget && W < (int64_t{1} << 30)) W *= 2;
  if (static_cast<int64_t>(acc_smem_bytes(W, sv, true)) > acc_budget) return GM_ERR_UNSUPPORTED_SMEM;
  if (o.chunk_width) {
    const int64_t w = o.chunk_width;
    if (w < 32 || (w & (w - 1)) || w > W) return GM_ERR_INVALID_ARG;
    W = w;
  } else {
    // no point in an accumulator wider than the column space
    W = std::min<int64_t>(W, std::max<int64_t>(32, static_cast<int64_t>(pow2_ceil(static_cast<uint64_t>(std::max<int64_t>(c_cols, 1))))));
  }
  out->chunk_width = static_cast<int32_t>(W);
  const int log2W = ilog2_floor(static_cast<uint64_t>(W));

  // --- n_chunksRequired = C.m / n_denseNumeric, rounded UP to a power of two so that every chunk
  // fits its accumulator and chunk = col >> log2(W).
  const int64_t need = std::max<int64_t>(1, (c_cols + W - 1) / W);
  const int64_t required = static_cast<int64_t>(pow2_ceil(static_cast<uint64_t>(need)));
  if (required > (int64_t{1} << 30)) return GM_ERR_CAPACITY;
  out->chunks_required = static_cast<int32_t>(required);

  // --- default tau.  The capacity is an upper limit.  A light row pays for a hash table and an n log^2 n sort
  // in one block; a heavy row pays per chunk (a one-warp register sort for the small ones).  Measured on
  // B200: with up to 32 chunks per row the heavy path is cheaper from about 512 products on, with more
  // chunks per row from about 1024 (R-MAT 20: 445 ms at 4096, 414 ms at 512; R-MAT 21 in fp64, 128 chunks:
  // 610 ms at 4096, 530 ms at 1024).
  int64_t tau = o.tau > 0 ? o.tau : std::min<int64_t>(cap, required <= 32 ? 512 : 1024);
  const int64_t top_cap = static_cast<int64_t>(pow2_ceil(static_cast<uint64_t>(std::max<int64_t>(tau, 16))));
  out->tau = tau;
  out->light_slots = static_cast<int32_t>(std::min<int64_t>(2 * top_cap, (S - reserve - 8 * top_cap) / se));

  // --- n_chunksMax (Eq. 6) with n_groupRows = 2, 32 subgroups per work group, 4-byte histogram
  // counters and 8-byte offsets, half of s_LM given to the permuted elements; floored to a power
  // of two and capped by what one multisplit tile of this build can bin.
  int64_t fmax;
  if (o.max_fanout) {
    fmax = o.max_fanout;
    if (fmax < 2 || (fmax & (fmax - 1)) || fmax > kMultisplitBinCap) return GM_ERR_INVALID_ARG;
  } else {
    const int64_t n_min_group_elems = S / (2 * se);
    const int64_t raw = (S - n_min_group_elems * se - 4) / (2 * (32 * 4 + 8));
    fmax = static_cast<int64_t>(pow2_floor(static_cast<uint64_t>(std::max<int64_t>(raw, 2))));
    fmax = std::min<int64_t>(std::max<int64_t>(fmax, 2), 256);
  }
  out->max_fanout = static_cast<int32_t>(fmax);

  // --- n_levels (Eq. 7) and v_chunks: max fan-out on every level but the last.
  int L = 0;
  if (required > 1) {
    const int lr = ilog2_floor(static_cast<uint64_t>(required));
    const int lf = ilog2_floor(static_cast<uint64_t>(fmax));
    L = (lr + lf - 1) / lf;
    if (L > GM_MAX_LEVELS) return GM_ERR_CAPACITY;
    int64_t rest = required;
    for (int l = 0; l < L - 1; ++l) {
      out->fanout[l] = static_cast<int32_t>(fmax);
      rest /= fmax;
    }
    out->fanout[L - 1] = static_cast<int32_t>(rest);
    int sh = log2W;
    for (int l = L - 1; l >= 0; --l) {
      out->shift[l] = sh;
      sh += ilog2_floor(static_cast<uint64_t>(out->fanout[l]));
    }
  }
  out->n_levels = L;
  return GM_OK;
}

bool cut_batches(const int64_t* heavy_prefix, int64_t n_heavy, int64_t stage_elems,
                 std::vector<Batch>* out) {
  out->clear();
  int64_t h = 0;
  while (h < n_heavy) {
    const int64_t base = heavy_prefix[h];
    // last h1 with prefix[h1] - base <= stage_elems
    const int64_t* end = std::upper_bound(heavy_prefix + h, heavy_prefix + n_heavy + 1, base + stage_elems);
    int64_t h1 = (end - heavy_prefix) - 1;
    if (h1 <= h) return false;  // row h alone does not fit
    out->push_back(Batch{h, h1, base, heavy_prefix[h1] - base});
    h = h1;
  }
  return true;
}

}  // namespace gm

extern "C" int gm_planner_params(int64_t c_cols, int32_t dtype, size_t smem_bytes,
                                 const gm_plan_opts* opts, gm_params* out) {
  return gm::planner_params(c_cols, dtype, smem_bytes, opts, out);
}

extern "C" int64_t gm_planner_batches(const int64_t* heavy_prefix, int64_t n_heavy, int64_t stage_elems,
                                      int64_t* bounds_out, int64_t max_bounds) {
  if (!heavy_prefix || !bounds_out || n_heavy < 0 || stage_elems <= 0) return GM_ERR_INVALID_ARG;
  std::vector<gm::Batch> b;
  if (!gm::cut_batches(heavy_prefix, n_heavy, stage_elems, &b)) return GM_ERR_CAPACITY;
  if (static_cast<int64_t>(b.size()) + 1 > max_bounds) return GM_ERR_CAPACITY;
  bounds_out[0] = 0;
  for (size_t i = 0; i < b.size(); ++i) bounds_out[i + 1] = b[i].h1;
  return static_cast<int64_t>(b.size());
}
