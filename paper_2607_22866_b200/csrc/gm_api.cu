// C ABI of the library (see include/gmagnus.h): plan = setup phase of Algorithm 3, execute = the
// light and heavy paths, batching of the heavy rows and assembly of C.
#include <algorithm>
#include <climits>
#include <cstddef>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <vector>

#include "gm_common.cuh"
#include "gm_k1_analysis.cuh"
#include "gm_k3_light.cuh"
#include "gm_k4_expand.cuh"
#include "gm_k4_direct.cuh"
#include "gm_k4_stream.cuh"
#include "gm_k4_csc.cuh"
#include "gm_k5_multisplit.cuh"
#include "gm_k6_accumulate.cuh"
#include "gm_k7_gather.cuh"
#include "gm_planner.h"
#include "gm_scan.cuh"
#include "gmagnus.h"

namespace gm {

// ------------------------------------------------------------------------------------------------
// errors, allocator
// ------------------------------------------------------------------------------------------------
static thread_local std::string g_last_error;

static int fail(int code, const std::string& msg) {
  g_last_error = msg;
  return code;
}

#define GM_CUDA(expr)                                                                              \
  do {                                                                                             \
    cudaError_t e_ = (expr);                                                                       \
    if (e_ != cudaSuccess)                                                                         \
      return fail(GM_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e_));               \
  } while (0)

#define GM_TRY(expr)                \
  do {                              \
    int rc_ = (expr);               \
    if (rc_ != GM_OK) return rc_;   \
  } while (0)

struct Allocator {
  gm_alloc_fn alloc = nullptr;
  gm_free_fn free = nullptr;
  void* user = nullptr;
};
static Allocator g_alloc;

static void* default_alloc(size_t bytes, cudaStream_t st) {
  static bool pool_ready = false;
  if (!pool_ready) {
    int dev = 0;
    cudaMemPool_t pool;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetDefaultMemPool(&pool, dev) == cudaSuccess) {
      unsigned long long thr = ~0ull;  // keep freed blocks cached: repeated plans reuse them
      cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &thr);
    }
    pool_ready = true;
  }
  void* p = nullptr;
  if (cudaMallocAsync(&p, bytes, st) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return p;
}

static void* dev_alloc(size_t bytes, cudaStream_t st) {
  if (bytes == 0) bytes = 16;
  if (g_alloc.alloc) {
    void* p = g_alloc.alloc(bytes, st, g_alloc.user);
    // the kernels use 16-byte accesses into what they are given: a hook that hands out less aligned memory is
    // treated like one that has none
    if (p && reinterpret_cast<uintptr_t>(p) % 256 != 0) {
      if (g_alloc.free) g_alloc.free(p, st, g_alloc.user);
      fail(GM_ERR_OOM, "the allocator hook returned a pointer that is not 256-byte aligned");
      return nullptr;
    }
    return p;
  }
  return default_alloc(bytes, st);
}
static void dev_free(void* p, cudaStream_t st) {
  if (!p) return;
  if (g_alloc.free) g_alloc.free(p, st, g_alloc.user);
  else cudaFreeAsync(p, st);
}

struct Buf {
  void* p = nullptr;
  size_t bytes = 0;
  template <typename T> T* as() const { return static_cast<T*>(p); }
};

// ------------------------------------------------------------------------------------------------
// plan
// ------------------------------------------------------------------------------------------------
struct PhaseTimes {
  enum Phase { kLightSym, kLightNum, kExpand, kHist, kSplit, kAccSym, kAccNum, kAccSmall, kAccMid, kScan, kCount };
  struct Rec { int phase; cudaEvent_t a, b; };
  std::vector<Rec> recs;
  std::vector<cudaEvent_t> pool;
  size_t used = 0;
  bool enabled = false;
  cudaEvent_t get() {
    if (used == pool.size()) { cudaEvent_t e; cudaEventCreate(&e); pool.push_back(e); }
    return pool[used++];
  }
  void begin(int phase, cudaStream_t st) {
    if (!enabled) return;
    Rec r{phase, get(), get()};
    cudaEventRecord(r.a, st);
    recs.push_back(r);
  }
  void end(cudaStream_t st) {
    if (!enabled) return;
    cudaEventRecord(recs.back().b, st);
  }
  void reset() { recs.clear(); used = 0; }
  void collect(float* out) {
    for (int i = 0; i < kCount; ++i) out[i] = 0.f;
    for (auto& r : recs) { float ms = 0.f; cudaEventElapsedTime(&ms, r.a, r.b); out[r.phase] += ms; }
  }
  ~PhaseTimes() { for (auto e : pool) cudaEventDestroy(e); }
};

}  // namespace gm

// Where gm_spgemm_host wants C: entries are copied to the host batch by batch, while later batches compute.
struct HostSink {
  int32_t* h_col = nullptr;
  void* h_val = nullptr;
  int64_t capacity = 0;          // entries the host buffers hold
  cudaStream_t copy_stream = nullptr;
  int64_t* h_totals = nullptr;   // pinned: entries of C up to the end of each batch
  std::vector<cudaEvent_t> events;
  int64_t copied = 0;            // entries already on their way to the host
};

struct gm_plan {
  gm_csr A{}, B{};
  int sv = 4;
  size_t smem_bytes = 0;
  gm_plan_opts opts{};
  gm_plan_info info{};
  gm_exec_stats stats{};
  int num_sms = 148;
  cudaStream_t plan_stream = nullptr;
  gm::LightBins bins{};
  int bin_slots[gm::kMaxLightBins]{};
  std::vector<gm::Batch> batches;
  std::vector<int32_t> x_heavy_host;
  int64_t max_batch_rows = 0;
  int64_t n_seg = 0;
  std::vector<gm::Buf> owned;
  // device arrays
  int64_t* nz_off = nullptr;       // nnzA + 1
  int64_t* ip = nullptr;           // nA
  int32_t* heavy_flag = nullptr;   // nA
  int32_t* x_heavy = nullptr;      // nH
  int64_t* heavy_base = nullptr;   // nH + 1
  int64_t* seg_off = nullptr;      // n_seg + 1
  int64_t* seg_bstart = nullptr;   // n_seg
  int64_t* seg_j = nullptr;        // n_seg
  int32_t* seg_brow = nullptr;     // n_seg: row of B the segment copies
  uint32_t* child_bound = nullptr; // n_rows(B) x (F0 + 1): where each level-0 child starts inside a row of B
  uint32_t* seg_prefix = nullptr;  // G: (segments of a batch + 1) x F0
  uint32_t* seg_h = nullptr;       // H: segments of a batch x F0 (G minus the child boundary of the segment's row of B)
  uint32_t* seg_tile_sums = nullptr;
  bool direct = false;             // the expansion writes the level-0 children itself
  bool stream = false;             // ... with the rows of B brought in by bulk copies (needs 16-byte aligned B arrays)
  int32_t* seg_hrow = nullptr;     // n_seg: heavy row (position in the heavy-row list) of every segment
  uint32_t* seg_rec = nullptr;     // segment records of a batch for the bulk-copy expansion (run starts + entry of A)
  // outer-product (CSC) order of the expansion, option expand_order = 1: per batch, the segments sorted by row of B
  bool csc = false;
  int32_t* csc_cnt = nullptr;      // n_rows(B) + 1: segments per row of B
  int64_t* csc_ptr = nullptr;      // n_rows(B) + 1: their exclusive scan (the masked CSC's column pointer)
  gm::u64* csc_cursor = nullptr;   // n_rows(B) + 1: scatter cursors
  int32_t* csc_perm = nullptr;     // segments of a batch in CSC order
  int32_t* csc_len = nullptr;      // their product counts
  int64_t* csc_off = nullptr;      // ... and the exclusive scan: the flattened product space in CSC order
  int small_max = 0, mid_max = 0;  // size classes of the final chunks: <= small_max one warp, <= mid_max one small block
  int exit_max = -1;               // chunks of at most this many products leave the multisplit hierarchy early (-1: none)
  unsigned char* exit_tag[2]{};    // per (parent, child) of a level: where the chunk left the hierarchy (ping-pong)
  unsigned char* parent_tag = nullptr;  // per parent of the level that runs: != 0, not split
  std::vector<int64_t> heavy_nz_off_host;
  int64_t* heavy_nz_off = nullptr; // nH + 1
  int32_t* sym_rows = nullptr;     // bins x nA
  int* sym_fill = nullptr;         // 8
  int32_t* num_rows = nullptr;     // bins x nA
  int* num_fill = nullptr;         // 8
  int32_t* row_nnz = nullptr;      // nA
  int64_t* scan_tmp = nullptr;
  int64_t* c_total = nullptr;      // [0] running nnz(C) (device carry), [1] heavy entries, [2] products and [3] entries of
                                   // small chunks, [4] products and [5] entries of mid-size chunks, [6] products and
                                   // [7] chunks that left the hierarchy early, [8] products the levels did not move
  int* err = nullptr;
  // heavy workspace
  int32_t* stage_col[2]{};
  void* stage_val[2]{};
  gm::u32* counts = nullptr;       // max_batch_rows * chunks_required
  gm::u64* cursor = nullptr;       // same
  int64_t* level_off[2]{};         // max_batch_rows * chunks_required + 1 each (ping-pong)
  gm::u32* chunk_nnz = nullptr;
  int64_t* chunk_nnz_off = nullptr;
  int64_t* chunk_base = nullptr;   // numeric pass: position in C of every chunk's first entry
  int32_t* mid_list = nullptr;     // accumulate kernels: chunks of the mid-size class
  int32_t* big_list = nullptr;     // ... and of the big class (the longest from the front, the others from the back)
  int* acc_counters = nullptr;     // list lengths and tickets (see k6_classify)
  gm::TileMeta* row_meta = nullptr;   // per tile of the expansion kernel: heavy rows it touches (fused histogram)
  gm::TileMeta* tile_meta = nullptr;  // per tile of the expansion / multisplit kernels: groups it touches
  gm::PhaseTimes times;
  HostSink* sink = nullptr;        // set by gm_spgemm_host for the duration of one execute
  // light rows run next to the heavy path on a stream of the plan's own (Algorithm 3 keeps separate queues for them)
  cudaStream_t light_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_light = nullptr;
};

#ifndef GM_MID_MIN_BLOCKS
#define GM_MID_MIN_BLOCKS 7
#endif
namespace gm {

template <typename T>
static int plan_alloc(gm_plan* p, T** out, size_t n, cudaStream_t st) {
  Buf b;
  b.bytes = n * sizeof(T);
  b.p = dev_alloc(b.bytes, st);
  if (!b.p) return fail(GM_ERR_OOM, "device allocation of " + std::to_string(b.bytes) + " bytes failed");
  p->owned.push_back(b);
  p->info.workspace_bytes += static_cast<int64_t>(b.bytes);
  *out = static_cast<T*>(b.p);
  return GM_OK;
}

static unsigned grid_for(i64 n, int threads, int num_sms, int per_sm = 16) {
  i64 g = (n + threads - 1) / threads;
  const i64 cap = static_cast<i64>(num_sms) * per_sm;
  if (g > cap) g = cap;
  if (g < 1) g = 1;
  return static_cast<unsigned>(g);
}

// structure_only: the caller reads row_ptr and col_idx alone (values and dtype are not looked at)
static int check_csr_arg(const gm_csr* M, const char* name, bool structure_only = false) {
  if (!M) return fail(GM_ERR_INVALID_ARG, std::string(name) + " is null");
  if (M->n_rows < 0 || M->n_cols < 0 || M->nnz < 0 || M->n_cols > INT32_MAX || M->n_rows > INT32_MAX)
    return fail(GM_ERR_INVALID_ARG, std::string(name) + ": sizes out of range");
  if (!M->row_ptr || (M->nnz > 0 && (!M->col_idx || (!structure_only && !M->vals))))
    return fail(GM_ERR_INVALID_ARG, std::string(name) + ": null array");
  if (!structure_only && M->dtype != GM_F32 && M->dtype != GM_F64)
    return fail(GM_ERR_DTYPE, std::string(name) + ": unknown dtype");
  return GM_OK;
}

__global__ void k_validate_csr(const i64* __restrict__ row_ptr, const int32_t* __restrict__ col, i64 n_rows, i64 n_cols,
                               i64 nnz, int* __restrict__ bad) {
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_rows;
       i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 s = row_ptr[i], e = row_ptr[i + 1];
    if ((i == 0 && s != 0) || e < s || e > nnz || (i == n_rows - 1 && e != nnz)) { *bad = 1; continue; }
    for (i64 k = s; k < e; ++k) {
      const int32_t c = col[k];
      if (c < 0 || c >= n_cols || (k > s && col[k - 1] >= c)) { *bad = 1; break; }
    }
  }
}

static int build_plan(gm_plan* p, cudaStream_t st) {
  const gm_csr& A = p->A;
  const gm_csr& B = p->B;
  const i64 nA = A.n_rows, nnzA = A.nnz;
  gm_plan_info& info = p->info;
  info.n_rows = nA;
  info.n_cols_c = B.n_cols;

  int dev = 0;
  GM_CUDA(cudaGetDevice(&dev));
  // (two attribute queries: cudaGetDeviceProperties fills in the whole structure and takes milliseconds)
  int num_sms = 0, smem_optin = 0;
  GM_CUDA(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
  GM_CUDA(cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  p->num_sms = num_sms;
  if (p->smem_bytes > static_cast<size_t>(smem_optin))
    return fail(GM_ERR_UNSUPPORTED_SMEM, "smem_bytes exceeds the device's opt-in shared memory per block");
  {
    const int rc = planner_params(B.n_cols, A.dtype, p->smem_bytes, &p->opts, &info.params);
    if (rc != GM_OK) return fail(rc, "planner rejected the parameters");
  }
  const gm_params& prm = info.params;
  {
    // size classes of the final chunks (Section III-E bins chunks by size)
    const gm_plan_opts& o = p->opts;
    if (o.small_chunk_max < -1 || o.small_chunk_max > kAccSmallChunk || o.mid_chunk_max < -1 || o.mid_chunk_max > (1 << 15))
      return fail(GM_ERR_INVALID_ARG, "small_chunk_max / mid_chunk_max out of range");
    p->small_max = o.small_chunk_max < 0 ? 0 : (o.small_chunk_max ? o.small_chunk_max : kAccSmallDefault);
    int mid = o.mid_chunk_max < 0 ? 0 : (o.mid_chunk_max ? o.mid_chunk_max : (p->sv == 4 ? 4096 : 2048));
    // several mid-chunk blocks must fit an SM next to each other for the class to pay
    while (mid > p->small_max && mid_smem_bytes(prm.chunk_width, p->sv, mid) + 1024 > p->smem_bytes / GM_MID_MIN_BLOCKS) mid /= 2;
    if (prm.chunk_width > 65536) mid = 0;  // the kernel keeps a chunk's columns as 16-bit offsets
    p->mid_max = std::max(mid, p->small_max);
    if (o.early_exit < -1 || o.early_exit > kAccSmallChunk) return fail(GM_ERR_INVALID_ARG, "early_exit out of range");
    // early exit needs the one-warp sort (the only accumulate kernel that takes a chunk wider than W) and a level
    // after the first
    p->exit_max = (o.early_exit < 0 || p->small_max <= 0 || prm.n_levels < 2) ? -1
                  : std::min(o.early_exit ? o.early_exit : p->small_max, p->small_max);
  }

  GM_TRY(plan_alloc(p, &p->err, 4, st));
  GM_CUDA(cudaMemsetAsync(p->err, 0, 4 * sizeof(int), st));
  if (p->opts.validate_inputs) {
    for (const gm_csr* M : {&A, &B}) {
      if (M->n_rows == 0) continue;
      k_validate_csr<<<grid_for(M->n_rows, 256, p->num_sms), 256, 0, st>>>(M->row_ptr, M->col_idx, M->n_rows,
                                                                          M->n_cols, M->nnz, p->err + 1);
    }
    info.launches += 2;
    int bad = 0;
    GM_CUDA(cudaMemcpyAsync(&bad, p->err + 1, sizeof(int), cudaMemcpyDeviceToHost, st));
    GM_CUDA(cudaStreamSynchronize(st));
    if (bad) return fail(GM_ERR_BAD_CSR, "row_ptr not monotone / columns out of range or not strictly ascending");
  }

  // ---- K1: products per stored entry, flattened product space, products per row
  int32_t* nz_len = nullptr;
  K1Totals* totals = nullptr;
  int64_t* heavy_pos = nullptr;
  GM_TRY(plan_alloc(p, &nz_len, static_cast<size_t>(nnzA) + 1, st));
  GM_TRY(plan_alloc(p, &p->nz_off, static_cast<size_t>(nnzA) + 1, st));
  GM_TRY(plan_alloc(p, &p->ip, static_cast<size_t>(nA) + 1, st));
  GM_TRY(plan_alloc(p, &p->heavy_flag, static_cast<size_t>(nA) + 1, st));
  GM_TRY(plan_alloc(p, &heavy_pos, static_cast<size_t>(nA) + 1, st));
  GM_TRY(plan_alloc(p, &totals, 1, st));
  GM_TRY(plan_alloc(p, &p->row_nnz, static_cast<size_t>(nA) + 1, st));
  GM_TRY(plan_alloc(p, &p->c_total, 16, st));
  GM_TRY(plan_alloc(p, &p->scan_tmp, static_cast<size_t>(scan_tmp_elems(std::max<i64>(std::max(nnzA, nA), 1))), st));
  GM_CUDA(cudaMemsetAsync(totals, 0, sizeof(K1Totals), st));
  if (nnzA > 0) k1_nz_len<<<grid_for(nnzA, 256, p->num_sms, 32), 256, 0, st>>>(A.col_idx, nnzA, B.row_ptr, nz_len);
  exclusive_scan<int32_t, i64>(nz_len, p->nz_off, nnzA, p->scan_tmp, nullptr, nullptr, nullptr, st);
  if (nA > 0) {
    k1_row_products<<<grid_for(nA, 256, p->num_sms), 256, 0, st>>>(A.row_ptr, nA, p->nz_off, prm.tau, B.n_cols, p->ip,
                                                                  p->heavy_flag, totals);
  }
  exclusive_scan<int32_t, i64>(p->heavy_flag, heavy_pos, nA, p->scan_tmp, nullptr, nullptr, nullptr, st);
  info.launches += (nnzA > 0 ? 3 : 1) + (nA > 0 ? 3 : 1) + (nA > 0 ? 2 : 0) + 1;

  // ---- light rows: bins by IP_i for the symbolic pass
  {
    const int top_cap = static_cast<int>(pow2_ceil(static_cast<uint64_t>(std::max<i64>(prm.tau, 16))));
    const int std_caps[] = {16, 64, 256, 1024, 4096, 16384, 65536};
    int nb = 0;
    for (int c : std_caps)
      if (c < top_cap && nb < kMaxLightBins - 1) { p->bins.cap[nb] = c; p->bin_slots[nb] = 2 * c; ++nb; }
    p->bins.cap[nb] = top_cap;
    p->bin_slots[nb] = prm.light_slots;
    p->bins.n_bins = nb + 1;
  }
  GM_TRY(plan_alloc(p, &p->sym_rows, static_cast<size_t>(p->bins.n_bins) * static_cast<size_t>(std::max<i64>(nA, 1)), st));
  GM_TRY(plan_alloc(p, &p->num_rows, static_cast<size_t>(p->bins.n_bins) * static_cast<size_t>(std::max<i64>(nA, 1)), st));
  GM_TRY(plan_alloc(p, &p->sym_fill, 8, st));
  GM_TRY(plan_alloc(p, &p->num_fill, 8, st));
  GM_CUDA(cudaMemsetAsync(p->sym_fill, 0, 8 * sizeof(int), st));
  if (nA > 0) {
    // tau may be below the top bin's capacity (forced tau): rows with tau < IP <= cap are heavy and skipped
    k1_bin_rows<i64><<<static_cast<unsigned>((nA + 255) / 256), 256, 0, st>>>(p->ip, p->heavy_flag, nA, p->bins, nA,
                                                                             p->sym_fill, p->sym_rows);
  }

  // ---- first host sync: totals
  K1Totals ht{};
  int fill[8] = {0};
  GM_CUDA(cudaMemcpyAsync(&ht, totals, sizeof(ht), cudaMemcpyDeviceToHost, st));
  GM_CUDA(cudaMemcpyAsync(fill, p->sym_fill, sizeof(fill), cudaMemcpyDeviceToHost, st));
  GM_CUDA(cudaStreamSynchronize(st));
  info.products_total = static_cast<int64_t>(ht.products_total);
  info.products_heavy = static_cast<int64_t>(ht.products_heavy);
  info.products_max_row = static_cast<int64_t>(ht.products_max_row);
  info.c_nnz_upper = static_cast<int64_t>(ht.c_nnz_upper);
  info.rows_heavy = static_cast<int64_t>(ht.rows_heavy);
  info.rows_empty = static_cast<int64_t>(ht.rows_empty);
  info.rows_light = nA - info.rows_heavy - info.rows_empty;
  info.nnz_a_heavy = static_cast<int64_t>(ht.nnz_a_heavy);
  for (int b = 0; b < 8; ++b) info.light_bin_rows[b] = fill[b];
  const i64 nH = info.rows_heavy;
  p->n_seg = info.nnz_a_heavy;

  // ---- heavy rows: lists, prefix sums, segment table
  if (nH > 0) {
    int64_t *heavy_ip = nullptr, *heavy_nnz = nullptr;
    GM_TRY(plan_alloc(p, &p->x_heavy, static_cast<size_t>(nH), st));
    GM_TRY(plan_alloc(p, &heavy_ip, static_cast<size_t>(nH) + 1, st));
    GM_TRY(plan_alloc(p, &heavy_nnz, static_cast<size_t>(nH) + 1, st));
    GM_TRY(plan_alloc(p, &p->heavy_base, static_cast<size_t>(nH) + 1, st));
    GM_TRY(plan_alloc(p, &p->heavy_nz_off, static_cast<size_t>(nH) + 1, st));
    GM_TRY(plan_alloc(p, &p->seg_off, static_cast<size_t>(p->n_seg) + 1, st));
    GM_TRY(plan_alloc(p, &p->seg_bstart, static_cast<size_t>(p->n_seg) + 1, st));
    GM_TRY(plan_alloc(p, &p->seg_j, static_cast<size_t>(p->n_seg) + 1, st));
    GM_TRY(plan_alloc(p, &p->seg_brow, static_cast<size_t>(p->n_seg) + 1, st));
    GM_TRY(plan_alloc(p, &p->seg_hrow, static_cast<size_t>(p->n_seg) + 1, st));
    k1_heavy_scatter<<<grid_for(nA, 256, p->num_sms), 256, 0, st>>>(p->heavy_flag, heavy_pos, p->ip, A.row_ptr, nA,
                                                                   p->x_heavy, heavy_ip, heavy_nnz);
    exclusive_scan<i64, i64>(heavy_ip, p->heavy_base, nH, p->scan_tmp, nullptr, nullptr, nullptr, st);
    exclusive_scan<i64, i64>(heavy_nnz, p->heavy_nz_off, nH, p->scan_tmp, nullptr, nullptr, nullptr, st);
    k1_heavy_segments<<<grid_for(p->n_seg + 1, 256, p->num_sms, 32), 256, 0, st>>>(
        p->x_heavy, nH, p->heavy_nz_off, p->heavy_base, A.row_ptr, A.col_idx, p->nz_off, B.row_ptr, p->n_seg, p->seg_off,
        p->seg_bstart, p->seg_j, p->seg_brow, p->seg_hrow);
    info.launches += 8;
    std::vector<int64_t> hb(static_cast<size_t>(nH) + 1);
    p->x_heavy_host.resize(static_cast<size_t>(nH));
    GM_CUDA(cudaMemcpyAsync(hb.data(), p->heavy_base, hb.size() * sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    GM_CUDA(cudaMemcpyAsync(p->x_heavy_host.data(), p->x_heavy, static_cast<size_t>(nH) * sizeof(int32_t),
                            cudaMemcpyDeviceToHost, st));
    p->heavy_nz_off_host.resize(static_cast<size_t>(nH) + 1);
    GM_CUDA(cudaMemcpyAsync(p->heavy_nz_off_host.data(), p->heavy_nz_off, (static_cast<size_t>(nH) + 1) * sizeof(int64_t),
                            cudaMemcpyDeviceToHost, st));
    GM_CUDA(cudaStreamSynchronize(st));

    // The expansion writes the first level's children itself (see gm_k4_direct.cuh) unless asked to run that
    // level as separate histogram and multisplit passes.
    // That takes a row of F0 run starts per segment, which pays when segments are long compared with the
    // fan-out (R-MAT products: ~1000 products per segment) and not when they are short (a clipped-Zipf pair
    // with F0 = 256 and ~60 products per segment measured 3x slower that way).
    const bool long_segments = prm.n_levels > 0 &&
                               info.products_heavy >= 2 * static_cast<i64>(prm.fanout[0]) * std::max<i64>(info.nnz_a_heavy, 1);
    // ... and a table of F0 + 1 boundaries per row of B, which must stay small (at most 1 GB, or what a staging
    // buffer of the default size takes)
    const i64 bound_bytes = prm.n_levels > 0 ? B.n_rows * static_cast<i64>(prm.fanout[0] + 1) * 4 : 0;
    const bool bounds_fit = bound_bytes <= std::max<i64>(i64{1} << 30, std::min<i64>(info.products_heavy, i64{1} << 29) * (4 + p->sv));
    p->csc = p->opts.expand_order == 1;
    p->direct = prm.n_levels > 0 && prm.fanout[0] <= 256 && !p->csc &&
                (p->opts.level0_multisplit == 2 || (p->opts.level0_multisplit == 0 && long_segments && bounds_fit));
    info.level0_direct = p->direct ? 1 : 0;
    {
      const size_t warp_smem = stream_warp_smem_bytes(prm.n_levels > 0 ? prm.fanout[0] : 2, p->sv);
      p->stream = p->direct && p->opts.expand_staging == 1 && reinterpret_cast<uintptr_t>(B.col_idx) % 16 == 0 &&
                  reinterpret_cast<uintptr_t>(B.vals) % 16 == 0 && p->smem_bytes >= kStreamWarps * warp_smem + 1024;
    }
    // one staging buffer is enough when no multisplit pass runs (no levels, or one level done by the expansion)
    const int n_buf = prm.n_levels > (p->direct ? 1 : 0) ? 2 : 1;

    // ---- batches: consecutive heavy rows whose products fit one staging buffer.  Default size: a fifth of the
    // device's memory for staging (fewer, longer launches: on R-MAT scale 20, 2^31 products per batch instead of
    // 2^29 took 7 % off the step), at least 2^29 products, at most what 32-bit tile positions allow.
    i64 stage = p->opts.stage_elems;
    if (stage <= 0) {
      size_t free_b = 0, total_b = 0;
      GM_CUDA(cudaMemGetInfo(&free_b, &total_b));
      stage = std::max<i64>(i64{1} << 29, static_cast<i64>(total_b / 5) / (static_cast<i64>(n_buf) * (4 + p->sv)));
      stage = std::max(stage, info.products_max_row);  // a row is never split
    }
    stage = std::min(stage, info.products_heavy);
    const i64 kMaxStage = (i64{1} << 31) - kSplitTile;  // batch-relative positions are 32-bit in the multisplit tiles
    if (stage > kMaxStage) stage = kMaxStage;
    if (info.products_max_row > stage)
      return fail(GM_ERR_CAPACITY, "a heavy row has " + std::to_string(info.products_max_row) +
                                       " products, more than one staging half-buffer holds (" + std::to_string(stage) + ")");
    if (!cut_batches(hb.data(), nH, stage, &p->batches)) return fail(GM_ERR_CAPACITY, "batch cutting failed");
    info.n_batches = static_cast<int64_t>(p->batches.size());
    info.stage_elems = 0;
    for (const Batch& b : p->batches) {
      info.stage_elems = std::max(info.stage_elems, b.elems);
      p->max_batch_rows = std::max(p->max_batch_rows, b.h1 - b.h0);
    }
    // the accumulate kernel streams whole tiles: it may read (and ignore) up to one tile past the last product
    const size_t se = static_cast<size_t>(info.stage_elems) + 4096 + 8;
    for (int i = 0; i < n_buf; ++i) {
      GM_TRY(plan_alloc(p, &p->stage_col[i], se, st));
      unsigned char* v = nullptr;
      GM_TRY(plan_alloc(p, &v, se * static_cast<size_t>(p->sv), st));
      p->stage_val[i] = v;
    }
    const size_t n_chunks_max = static_cast<size_t>(p->max_batch_rows) * static_cast<size_t>(prm.chunks_required);
    GM_TRY(plan_alloc(p, &p->level_off[0], n_chunks_max + 1, st));
    if (prm.n_levels > 0) {
      GM_TRY(plan_alloc(p, &p->counts, n_chunks_max + 1, st));
      GM_TRY(plan_alloc(p, &p->cursor, n_chunks_max + 1, st));
      GM_TRY(plan_alloc(p, &p->level_off[1], n_chunks_max + 1, st));
    }
    GM_TRY(plan_alloc(p, &p->chunk_nnz, n_chunks_max + 1, st));
    GM_TRY(plan_alloc(p, &p->chunk_nnz_off, n_chunks_max + 1, st));
    GM_TRY(plan_alloc(p, &p->chunk_base, n_chunks_max + 1, st));
    GM_TRY(plan_alloc(p, &p->mid_list, n_chunks_max + 1, st));
    GM_TRY(plan_alloc(p, &p->big_list, n_chunks_max + 1, st));
    GM_TRY(plan_alloc(p, &p->acc_counters, 8, st));
    if (p->exit_max >= 0) {
      GM_TRY(plan_alloc(p, &p->exit_tag[0], n_chunks_max + 1, st));
      GM_TRY(plan_alloc(p, &p->exit_tag[1], n_chunks_max + 1, st));
      GM_TRY(plan_alloc(p, &p->parent_tag, n_chunks_max + 1, st));
    }
    const size_t n_tiles_max = static_cast<size_t>(info.stage_elems) / std::min({kExpandTile, kSplitTile, kGatherTile, kDirectTileSmall}) + 2;
    GM_TRY(plan_alloc(p, &p->tile_meta, n_tiles_max, st));
    GM_TRY(plan_alloc(p, &p->row_meta, n_tiles_max, st));
    if (p->direct) {
      const int F0 = prm.fanout[0];
      i64 max_seg_b = 0;
      for (const Batch& b : p->batches)
        max_seg_b = std::max(max_seg_b, p->heavy_nz_off_host[static_cast<size_t>(b.h1)] - p->heavy_nz_off_host[static_cast<size_t>(b.h0)]);
      GM_TRY(plan_alloc(p, &p->child_bound, static_cast<size_t>(B.n_rows) * static_cast<size_t>(F0 + 1) + 1, st));
      GM_TRY(plan_alloc(p, &p->seg_prefix, (static_cast<size_t>(max_seg_b) + 1) * static_cast<size_t>(F0), st));
      GM_TRY(plan_alloc(p, &p->seg_h, (static_cast<size_t>(max_seg_b) + 1) * static_cast<size_t>(F0), st));
      GM_TRY(plan_alloc(p, &p->seg_tile_sums, (static_cast<size_t>(max_seg_b) / kGTile + 2) * static_cast<size_t>(F0), st));
      if (p->stream)
        GM_TRY(plan_alloc(p, &p->seg_rec, (static_cast<size_t>(max_seg_b) + 1) * static_cast<size_t>(stream_rec_words(F0)), st));
      if (B.n_rows > 0) {
        k_child_bounds<<<grid_for(B.n_rows * (F0 + 1), 256, p->num_sms, 32), 256, 0, st>>>(B.row_ptr, B.col_idx, B.n_rows, F0,
                                                                                        prm.shift[0], p->child_bound);
        ++info.launches;
      }
    }
    i64 csc_scan_len = 0;
    if (p->csc) {
      i64 max_seg_b = 0;
      for (const Batch& b : p->batches)
        max_seg_b = std::max(max_seg_b, p->heavy_nz_off_host[static_cast<size_t>(b.h1)] - p->heavy_nz_off_host[static_cast<size_t>(b.h0)]);
      GM_TRY(plan_alloc(p, &p->csc_cnt, static_cast<size_t>(B.n_rows) + 1, st));
      GM_TRY(plan_alloc(p, &p->csc_ptr, static_cast<size_t>(B.n_rows) + 2, st));
      GM_TRY(plan_alloc(p, &p->csc_cursor, static_cast<size_t>(B.n_rows) + 2, st));
      GM_TRY(plan_alloc(p, &p->csc_perm, static_cast<size_t>(max_seg_b) + 1, st));
      GM_TRY(plan_alloc(p, &p->csc_len, static_cast<size_t>(max_seg_b) + 1, st));
      GM_TRY(plan_alloc(p, &p->csc_off, static_cast<size_t>(max_seg_b) + 2, st));
      csc_scan_len = std::max<i64>(B.n_rows, max_seg_b);
    }
    int64_t* tmp2 = nullptr;  // the per-batch scans can be longer than the ones above
    GM_TRY(plan_alloc(p, &tmp2, static_cast<size_t>(scan_tmp_elems(std::max<i64>({static_cast<i64>(n_chunks_max), nnzA, nA, csc_scan_len, 1}))), st));
    p->scan_tmp = tmp2;
  }
  GM_CUDA(cudaStreamSynchronize(st));
  return GM_OK;
}

// ------------------------------------------------------------------------------------------------
// execute
// ------------------------------------------------------------------------------------------------
template <typename V, bool NUMERIC, int G, int LPN, int BT>
static int launch_light_one(gm_plan* p, const int32_t* rows, const int* n_rows_dev, i64 n_rows_upper, int slots, int cap,
                            const i64* c_row_ptr, int32_t* c_col, V* c_val, i64 c_capacity, cudaStream_t st) {
  constexpr int kGroups = BT / G;
  const size_t smem = kGroups * light_group_bytes<V, NUMERIC>(slots, cap, G);
  auto kern = k3_light_rows<V, G, LPN, BT, NUMERIC>;
  // (static shared memory counts towards the 48 KB that need no opt-in)
  if (smem > 32 * 1024) GM_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  const unsigned grid = grid_for(n_rows_upper, kGroups, p->num_sms, 2048 / BT * 4);
  kern<<<grid, BT, smem, st>>>(p->A.row_ptr, p->A.col_idx, static_cast<const V*>(p->A.vals), p->B.row_ptr, p->B.col_idx,
                               static_cast<const V*>(p->B.vals), rows, n_rows_dev, slots, cap, p->row_nnz, c_row_ptr, c_col,
                               c_val, c_capacity, p->err);
  ++p->stats.launches;
  GM_CUDA(cudaGetLastError());
  return GM_OK;
}

template <typename V, bool NUMERIC>
static int launch_light(gm_plan* p, const int32_t* rows_all, const int* fill_dev, const i64* rows_upper,
                        const i64* c_row_ptr, int32_t* c_col, V* c_val, i64 c_capacity, cudaStream_t st) {
  const i64 stride = std::max<i64>(p->A.n_rows, 1);
  for (int b = 0; b < p->bins.n_bins; ++b) {
    if (rows_upper[b] <= 0) continue;
    const int cap = p->bins.cap[b], slots = p->bin_slots[b];
    const int32_t* rows = rows_all + static_cast<size_t>(b) * stride;
    const int* nd = fill_dev + b;
    const i64 up = rows_upper[b];
#define GM_LIGHT(G, LPN, BT) launch_light_one<V, NUMERIC, G, LPN, BT>(p, rows, nd, up, slots, cap, c_row_ptr, c_col, c_val, c_capacity, st)
    int rc;
    if (cap <= 16) rc = GM_LIGHT(8, 1, 256);
    else if (cap <= 64) rc = GM_LIGHT(32, 4, 256);
    else if (cap <= 256) rc = GM_LIGHT(128, 8, 128);
    else if (cap <= 1024) rc = GM_LIGHT(256, 16, 256);
    else if (cap <= 4096) rc = GM_LIGHT(512, 32, 512);
    else rc = GM_LIGHT(1024, 32, 1024);
#undef GM_LIGHT
    GM_TRY(rc);
  }
  return GM_OK;
}

__global__ void k_heavy_row_counts(const i64* __restrict__ chunk_nnz_off, int log2_chunks_per_row, i64 n_rows_b,
                                   const int32_t* __restrict__ x_heavy, i64 h0, int32_t* __restrict__ row_nnz,
                                   i64* __restrict__ heavy_total) {
  if (blockIdx.x == 0 && threadIdx.x == 0)
    atomicAdd(reinterpret_cast<u64*>(heavy_total), static_cast<u64>(chunk_nnz_off[n_rows_b << log2_chunks_per_row]));
  for (i64 r = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; r < n_rows_b;
       r += static_cast<i64>(gridDim.x) * blockDim.x) {
    row_nnz[x_heavy[h0 + r]] =
        static_cast<int32_t>(chunk_nnz_off[(r + 1) << log2_chunks_per_row] - chunk_nnz_off[r << log2_chunks_per_row]);
  }
}

__global__ void k_rebase(const i64* __restrict__ in, i64 n, i64 bias, i64* __restrict__ out) {
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
       i += static_cast<i64>(gridDim.x) * blockDim.x)
    out[i] = in[i] - bias;
}

template <typename V>
struct HeavyBatchState {
  int32_t* fin_col = nullptr;  // staging buffer that holds the final chunks
  V* fin_val = nullptr;
  const i64* chunk_off = nullptr;    // n_chunks + 1 batch-relative offsets
  i64 n_chunks = 0;
  int log2_cpr = 0;
  // chunks that left the multisplit hierarchy early (tags == nullptr: none can have)
  const unsigned char* tags = nullptr;
  int32_t* alt_col = nullptr;  // the staging buffer that is not fin_col
  V* alt_val = nullptr;
  ExitTags xt;
};

// K6: accumulate every chunk of the batch and compact it in place; chunk_nnz receives the entry counts.
// Three kernels, one per size class of the chunks (see gm_k6_accumulate.cuh).
template <typename V>
static int launch_accumulate(gm_plan* p, const Batch& b, const HeavyBatchState<V>& hs, cudaStream_t st) {
  const gm_params& prm = p->info.params;
  const int W = prm.chunk_width;
  const int bt = prm.acc_block_threads;
  const int small_max = p->small_max, mid_max = p->mid_max;
  GM_CUDA(cudaMemsetAsync(p->acc_counters, 0, 8 * sizeof(int), st));
  GM_CUDA(cudaMemsetAsync(p->chunk_nnz, 0, static_cast<size_t>(hs.n_chunks) * sizeof(u32), st));
  if (p->opts.validate_inputs) {
    k6_validate_chunks<<<grid_for(hs.n_chunks * 32, 256, p->num_sms, 8), 256, 0, st>>>(
        hs.fin_col, hs.chunk_off, hs.n_chunks, hs.log2_cpr, W, p->B.n_cols, p->err, hs.tags, hs.alt_col, hs.xt);
    ++p->stats.launches;
  }
  k6_classify<<<grid_for(hs.n_chunks, 256, p->num_sms), 256, 0, st>>>(hs.chunk_off, hs.n_chunks, small_max, mid_max, p->mid_list,
                                                                     p->big_list, p->acc_counters);
  ++p->stats.launches;
  if (small_max > 0) {
    p->times.begin(PhaseTimes::kAccSmall, st);
    // as many blocks as are resident at once: the warps share out the chunks statically, so a block that had to wait
    // for a free slot would start its share when the others are done
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k6_small_chunks<V>, kSmallWarps * 32, 0) != cudaSuccess || per_sm < 1)
      per_sm = 4;
    k6_small_chunks<V><<<static_cast<unsigned>(p->num_sms * per_sm), kSmallWarps * 32, 0, st>>>(
        hs.fin_col, hs.fin_val, hs.chunk_off, hs.n_chunks, W, small_max, p->chunk_nnz,
        reinterpret_cast<u64*>(p->c_total + 2), hs.tags, hs.alt_col, hs.alt_val, hs.xt);
    ++p->stats.launches;
    p->times.end(st);
  }
  if (mid_max > small_max) {
    p->times.begin(PhaseTimes::kAccMid, st);
    const size_t smem = mid_smem_bytes(W, sizeof(V), mid_max);
    auto kern = k6_mid_chunks<V>;
    if (smem > 32 * 1024) GM_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    const int per_sm = std::max<int>(1, std::min<int>(2048 / kMidThreads, static_cast<int>((p->smem_bytes - 1024) / (smem + 1024))));
    const unsigned grid = static_cast<unsigned>(std::min<i64>(hs.n_chunks, static_cast<i64>(p->num_sms) * per_sm));
    kern<<<grid, kMidThreads, smem, st>>>(hs.fin_col, hs.fin_val, hs.chunk_off, p->mid_list, p->acc_counters, hs.log2_cpr, W,
                                          mid_max, p->chunk_nnz, reinterpret_cast<u64*>(p->c_total + 4));
    ++p->stats.launches;
    p->times.end(st);
  }
  p->times.begin(PhaseTimes::kAccNum, st);
  {
    const size_t smem = acc_smem_bytes_big(W, sizeof(V));
    const int per_sm = 1024 / bt;
    const unsigned grid = static_cast<unsigned>(std::min<i64>(hs.n_chunks, static_cast<i64>(p->num_sms) * per_sm));
#define GM_ACC(BT)                                                                                                   \
  do {                                                                                                               \
    auto kern = k6_accumulate<V, BT>;                                                                                \
    if (smem > 32 * 1024)                                                                                            \
      GM_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));     \
    kern<<<grid, BT, smem, st>>>(hs.fin_col, hs.fin_val, hs.chunk_off, hs.n_chunks, p->big_list, p->acc_counters,    \
                                 hs.log2_cpr, W, p->chunk_nnz);                                                      \
  } while (0)
    if (bt == 1024) GM_ACC(1024);
    else if (bt == 512) GM_ACC(512);
    else if (bt == 256) GM_ACC(256);
    else GM_ACC(128);
#undef GM_ACC
  }
  p->times.end(st);
  ++p->stats.launches;
  GM_CUDA(cudaGetLastError());
  return GM_OK;
}

// K7: once C.rowPtr covers the batch's rows, move the compacted chunks into C.
template <typename V>
static int launch_gather(gm_plan* p, const Batch& b, const HeavyBatchState<V>& hs, const i64* c_row_ptr,
                         int32_t* c_col, V* c_val, i64 c_capacity, cudaStream_t st) {
  k6_chunk_bases<<<grid_for(hs.n_chunks, 256, p->num_sms), 256, 0, st>>>(p->chunk_nnz_off, hs.n_chunks, hs.log2_cpr,
                                                                         p->x_heavy, b.h0, c_row_ptr, p->chunk_base);
  // the batch's heavy entry count is only known on the device: it is at most the batch's product count
  const unsigned grid = static_cast<unsigned>((b.elems + kGatherTile - 1) / kGatherTile);
  k_tile_bounds<<<grid_for(grid, 256, p->num_sms), 256, 0, st>>>(p->chunk_nnz_off, hs.n_chunks, 0, 0, kGatherTile,
                                                               p->tile_meta, p->chunk_nnz_off + hs.n_chunks);
  if (hs.tags && hs.xt.alt_bits)
    k7_gather<V, true><<<grid, kGatherThreads, 0, st>>>(hs.fin_col, hs.fin_val, hs.chunk_off, p->chunk_nnz_off, p->chunk_base,
                                                        hs.n_chunks, p->tile_meta, c_col, c_val, c_capacity, p->err,
                                                        hs.alt_col, hs.alt_val, hs.tags, hs.xt.alt_bits);
  else
    k7_gather<V><<<grid, kGatherThreads, 0, st>>>(hs.fin_col, hs.fin_val, hs.chunk_off, p->chunk_nnz_off, p->chunk_base,
                                                  hs.n_chunks, p->tile_meta, c_col, c_val, c_capacity, p->err);
  p->stats.launches += 3;
  GM_CUDA(cudaGetLastError());
  return GM_OK;
}

// Expansion, every multisplit level and the accumulate of one batch.  Leaves the compacted chunks in
// the staging buffer and the per-chunk entry counts (and their scan) in chunk_nnz / chunk_nnz_off,
// and writes the heavy rows' entry counts into row_nnz.
template <typename V>
static int heavy_batch_front(gm_plan* p, const Batch& b, HeavyBatchState<V>* hs, cudaStream_t st) {
  const gm_params& prm = p->info.params;
  const i64 rows_b = b.h1 - b.h0;
  PhaseTimes& tm = p->times;
  // level-0 parents are the batch's rows: offsets relative to the batch
  i64* off_cur = p->level_off[0];
  i64* off_nxt = p->level_off[1];
  k_rebase<<<grid_for(rows_b + 1, 256, p->num_sms), 256, 0, st>>>(p->heavy_base + b.h0, rows_b + 1, b.elem0, off_cur);
  ++p->stats.launches;
  int cur = 0;
  i64 n_par = rows_b;
  int first_level = 0;
  if (p->direct) {
    // ---- run starts of every (segment, child) from counts alone, then the products straight into the children
    const int F = prm.fanout[0];
    const i64 seg0 = p->heavy_nz_off_host[static_cast<size_t>(b.h0)];
    const i64 n_seg_b = p->heavy_nz_off_host[static_cast<size_t>(b.h1)] - seg0;
    const i64 n_gt = (n_seg_b + kGTile - 1) / kGTile;
    const i64 n_child = rows_b * F;
    const unsigned ggrid = static_cast<unsigned>((n_gt + (256 / F) - 1) / (256 / F));
    tm.begin(PhaseTimes::kHist, st);
    k_g_tile_sums<<<ggrid, 256, 0, st>>>(p->seg_brow, seg0, n_seg_b, p->child_bound, F, p->seg_tile_sums);
    k_g_scan_tiles<<<static_cast<unsigned>(F), 256, 0, st>>>(p->seg_tile_sums, n_gt, F);
    k_g_write<<<ggrid, 256, 0, st>>>(p->seg_brow, seg0, n_seg_b, p->child_bound, F, p->seg_tile_sums, p->seg_prefix, p->seg_h);
    k_g_row_counts<<<grid_for(n_child, 256, p->num_sms, 32), 256, 0, st>>>(p->seg_prefix, p->heavy_nz_off + b.h0, seg0, rows_b, F,
                                                                          p->counts);
    p->stats.launches += 4;
    tm.end(st);
    tm.begin(PhaseTimes::kScan, st);
    exclusive_scan<u32, i64>(p->counts, off_nxt, n_child, p->scan_tmp, nullptr, nullptr, nullptr, st);
    // (the cursor array of the multisplit is free in this mode: it holds R)
    u32* const row_base = reinterpret_cast<u32*>(p->cursor);
    k_g_row_base<<<grid_for(n_child, 256, p->num_sms, 32), 256, 0, st>>>(p->seg_prefix, p->heavy_nz_off + b.h0, seg0, rows_b, F,
                                                                        off_nxt, row_base);
    p->stats.launches += 4;
    tm.end(st);
    tm.begin(PhaseTimes::kExpand, st);
    if (p->stream) {
      // one contiguous range of the batch's products per warp; the grid fills the SMs' shared memory
      const size_t smem = kStreamWarps * stream_warp_smem_bytes(F, sizeof(V));
      const int per_sm = std::max<int>(1, std::min<int>(16, static_cast<int>((p->smem_bytes - 1024) / (smem + 1024))));
      const i64 n_warps = static_cast<i64>(p->num_sms) * per_sm * kStreamWarps;
      const i64 per_warp = std::max<i64>(4096, ((b.elems + n_warps - 1) / n_warps + 127) & ~i64{127});
      const i64 n_ranges = (b.elems + per_warp - 1) / per_warp;
      const unsigned grid = static_cast<unsigned>((n_ranges + kStreamWarps - 1) / kStreamWarps);
      k_seg_records<V><<<grid_for(n_seg_b * stream_rec_words(F), 256, p->num_sms, 32), 256, 0, st>>>(
          p->seg_h, row_base, p->seg_hrow, p->seg_j, static_cast<const V*>(p->A.vals), seg0, n_seg_b, b.h0, F, p->seg_rec);
      k_tile_bounds<<<grid_for(n_ranges, 256, p->num_sms), 256, 0, st>>>(p->seg_off, p->n_seg, b.elem0, b.elems,
                                                                       static_cast<int>(per_warp), p->tile_meta);
      auto kern = k4_expand_stream<V>;
      GM_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
      const int spin = p->opts.debug_spin_limit != 0 ? p->opts.debug_spin_limit : kCopySpinLimit;
      kern<<<grid, kStreamWarps * 32, smem, st>>>(p->seg_off, p->seg_bstart, p->n_seg, p->tile_meta, p->B.col_idx,
                                                  static_cast<const V*>(p->B.vals), p->B.nnz, b.elem0, b.elems, per_warp, seg0,
                                                  p->seg_rec, F, prm.shift[0], p->stage_col[0], static_cast<V*>(p->stage_val[0]),
                                                  spin, p->err);
      k4_expand_short<V><<<grid_for(n_seg_b * 32, 256, p->num_sms, 8), 256, 0, st>>>(
          p->seg_off, p->seg_bstart, p->B.col_idx, static_cast<const V*>(p->B.vals), seg0, n_seg_b, p->seg_rec, F, prm.shift[0],
          p->stage_col[0], static_cast<V*>(p->stage_val[0]));
    } else {
      const int tile = direct_tile(F);
      const unsigned grid = static_cast<unsigned>((b.elems + tile - 1) / tile);
      k_tile_bounds<<<grid_for(grid, 256, p->num_sms), 256, 0, st>>>(p->seg_off, p->n_seg, b.elem0, b.elems, tile, p->tile_meta);
      k_tile_bounds<<<grid_for(grid, 256, p->num_sms), 256, 0, st>>>(off_cur, rows_b, 0, b.elems, tile, p->row_meta);
      auto kern = tile == kDirectTileSmall ? k4_expand_direct<V, kDirectTileSmall> : k4_expand_direct<V, kExpandTile>;
      kern<<<grid, kExpandThreads, 0, st>>>(
          p->seg_off, p->seg_bstart, p->seg_j, p->tile_meta, static_cast<const V*>(p->A.vals), p->B.col_idx,
          static_cast<const V*>(p->B.vals), b.elem0, b.elems, p->row_meta, off_cur, seg0, F, prm.shift[0], row_base, p->seg_h,
          p->stage_col[0], static_cast<V*>(p->stage_val[0]));
    }
    p->stats.launches += 3;
    GM_CUDA(cudaGetLastError());
    tm.end(st);
    std::swap(off_cur, off_nxt);
    n_par = n_child;
    first_level = 1;
  }
  // the expansion kernel counts the first level's (row, child) bins while it writes, unless asked not to
  const bool fuse_hist = !p->direct && prm.n_levels > 0 && !p->opts.separate_histogram && !p->csc;
  if (p->csc) {
    // ---- outer-product order: masked CSR -> CSC of the batch's segments (counting sort by row of B), then the
    // expansion walks the product space in that order
    tm.begin(PhaseTimes::kExpand, st);
    const i64 seg0 = p->heavy_nz_off_host[static_cast<size_t>(b.h0)];
    const i64 n_seg_b = p->heavy_nz_off_host[static_cast<size_t>(b.h1)] - seg0;
    const i64 nB = p->B.n_rows;
    GM_CUDA(cudaMemsetAsync(p->csc_cnt, 0, static_cast<size_t>(nB + 1) * sizeof(int32_t), st));
    k_csc_count<<<grid_for(n_seg_b, 256, p->num_sms, 16), 256, 0, st>>>(p->seg_brow, seg0, n_seg_b, p->csc_cnt);
    exclusive_scan<int32_t, i64>(p->csc_cnt, p->csc_ptr, nB, p->scan_tmp, nullptr, nullptr, reinterpret_cast<i64*>(p->csc_cursor), st);
    k_csc_scatter<<<grid_for(n_seg_b, 256, p->num_sms, 16), 256, 0, st>>>(p->seg_brow, p->seg_off, seg0, n_seg_b, p->csc_cursor,
                                                                          p->csc_perm, p->csc_len);
    exclusive_scan<int32_t, i64>(p->csc_len, p->csc_off, n_seg_b, p->scan_tmp, nullptr, nullptr, nullptr, st);
    const unsigned grid = static_cast<unsigned>((b.elems + kExpandTile - 1) / kExpandTile);
    k_tile_bounds<<<grid_for(grid, 256, p->num_sms), 256, 0, st>>>(p->csc_off, n_seg_b, 0, b.elems, kExpandTile, p->tile_meta);
    k4_expand_csc<V><<<grid, kExpandThreads, 0, st>>>(p->csc_off, p->csc_perm, p->seg_off, p->seg_bstart, p->seg_j, seg0,
                                                      p->tile_meta, static_cast<const V*>(p->A.vals), p->B.col_idx,
                                                      static_cast<const V*>(p->B.vals), b.elem0, b.elems, p->stage_col[0],
                                                      static_cast<V*>(p->stage_val[0]));
    p->stats.launches += 10;
    GM_CUDA(cudaGetLastError());
    tm.end(st);
  } else if (!p->direct) {
  tm.begin(PhaseTimes::kExpand, st);
  {
    static_assert(kExpandTile == kSplitTile, "the fused histogram shares the multisplit's tiles");
    const unsigned grid = static_cast<unsigned>((b.elems + kExpandTile - 1) / kExpandTile);
    k_tile_bounds<<<grid_for(grid, 256, p->num_sms), 256, 0, st>>>(p->seg_off, p->n_seg, b.elem0, b.elems, kExpandTile,
                                                                 p->tile_meta);
    ++p->stats.launches;
    if (fuse_hist) {
      GM_CUDA(cudaMemsetAsync(p->counts, 0, static_cast<size_t>(rows_b) * prm.fanout[0] * sizeof(u32), st));
      k_tile_bounds<<<grid_for(grid, 256, p->num_sms), 256, 0, st>>>(off_cur, rows_b, 0, b.elems, kExpandTile, p->row_meta);
      ++p->stats.launches;
    }
    k4_expand<V><<<grid, kExpandThreads, 0, st>>>(p->seg_off, p->seg_bstart, p->seg_j, p->tile_meta,
                                                  static_cast<const V*>(p->A.vals), p->B.col_idx,
                                                  static_cast<const V*>(p->B.vals), b.elem0, b.elems, p->stage_col[0],
                                                  static_cast<V*>(p->stage_val[0]), p->row_meta, off_cur,
                                                  fuse_hist ? prm.fanout[0] : 0, fuse_hist ? prm.shift[0] : 0, p->counts);
    ++p->stats.launches;
    GM_CUDA(cudaGetLastError());
  }
  tm.end(st);
  }
  if (prm.n_levels > first_level) {
    GM_CUDA(cudaFuncSetAttribute(k5_level<V, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(split_smem_bytes<V>(true))));
    GM_CUDA(cudaFuncSetAttribute(k5_level<V, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(split_smem_bytes<V>(true))));
    GM_CUDA(cudaFuncSetAttribute(k5_level<V, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(split_smem_bytes<V>(true))));
    GM_CUDA(cudaFuncSetAttribute(k5_level<V, true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(split_smem_bytes<V>(true))));
  }
  bool hist_ready = false;  // the previous level's multisplit counted this level's bins while it wrote
  // early exit: tags of the current parents (none before the first level that can leave chunks behind)
  const unsigned char* tag_cur = nullptr;
  int tag_buf = 0;
  int level_buf[GM_MAX_LEVELS + 1] = {0};  // staging buffer a level read from
  for (int l = first_level; l < prm.n_levels; ++l) {
    const int F = prm.fanout[l];
    const i64 n_child = n_par * F;
    const unsigned grid = static_cast<unsigned>((b.elems + kSplitTile - 1) / kSplitTile);
    const int32_t* xc = p->stage_col[cur];
    const V* xv = static_cast<const V*>(p->stage_val[cur]);
    tm.begin(PhaseTimes::kHist, st);
    k_tile_bounds<<<grid_for(grid, 256, p->num_sms), 256, 0, st>>>(off_cur, n_par, 0, b.elems, kSplitTile, p->tile_meta);
    ++p->stats.launches;
    if (!(l == 0 && fuse_hist) && !hist_ready) {
      GM_CUDA(cudaMemsetAsync(p->counts, 0, static_cast<size_t>(n_child) * sizeof(u32), st));
      k5_level<V, false><<<grid, kSplitThreads, split_smem_bytes<V>(false), st>>>(
          xc, xv, b.elems, off_cur, n_par, p->tile_meta, F, prm.shift[l], p->counts, nullptr, nullptr, nullptr, 0, 0, nullptr);
      ++p->stats.launches;
      GM_CUDA(cudaGetLastError());
    }
    // Early exit: a parent of a level after the first that holds few products stays where it is; its span of columns
    // must still fit the sort's packed key
    level_buf[l] = cur;
    const int span_bits = prm.shift[l] + ilog2_floor(static_cast<uint64_t>(F));
    const bool can_exit = p->exit_max >= 0 && l >= 1 && span_bits + kSmallIdxBits <= 32;
    const bool exiting = can_exit || tag_cur != nullptr;
    if (exiting) {
      unsigned char* tag_nxt = p->exit_tag[tag_buf];
      k5_exit_flags<<<grid_for(n_child, 256, p->num_sms, 32), 256, 0, st>>>(
          off_cur, n_par, ilog2_floor(static_cast<uint64_t>(F)), tag_cur, can_exit ? p->exit_max : -1, l + 1, p->counts,
          p->parent_tag, tag_nxt, reinterpret_cast<u64*>(p->c_total + 6));
      ++p->stats.launches;
      tag_cur = tag_nxt;
      tag_buf ^= 1;
      hs->xt.set(l + 1, false, span_bits);  // (which buffer: known once the last level has run)
    }
    tm.end(st);
    tm.begin(PhaseTimes::kScan, st);
    exclusive_scan<u32, i64>(p->counts, off_nxt, n_child, p->scan_tmp, nullptr, nullptr, reinterpret_cast<i64*>(p->cursor), st);
    p->stats.launches += 3;
    tm.end(st);
    tm.begin(PhaseTimes::kSplit, st);
    // the counts of this level have been scanned: the array is free to receive the next level's
    const bool next = l + 1 < prm.n_levels && !p->opts.separate_histogram;
    if (next) GM_CUDA(cudaMemsetAsync(p->counts, 0, static_cast<size_t>(n_child) * prm.fanout[l + 1] * sizeof(u32), st));
    if (exiting && next) {
      k5_level<V, true, true, true><<<grid, kSplitThreads, split_smem_bytes<V>(true), st>>>(
          xc, xv, b.elems, off_cur, n_par, p->tile_meta, F, prm.shift[l], nullptr, p->cursor, p->stage_col[cur ^ 1],
          static_cast<V*>(p->stage_val[cur ^ 1]), prm.fanout[l + 1], prm.shift[l + 1], p->counts, p->parent_tag);
    } else if (exiting) {
      k5_level<V, true, false, true><<<grid, kSplitThreads, split_smem_bytes<V>(true), st>>>(
          xc, xv, b.elems, off_cur, n_par, p->tile_meta, F, prm.shift[l], nullptr, p->cursor, p->stage_col[cur ^ 1],
          static_cast<V*>(p->stage_val[cur ^ 1]), 0, 0, nullptr, p->parent_tag);
    } else if (next) {
      k5_level<V, true, true><<<grid, kSplitThreads, split_smem_bytes<V>(true), st>>>(
          xc, xv, b.elems, off_cur, n_par, p->tile_meta, F, prm.shift[l], nullptr, p->cursor, p->stage_col[cur ^ 1],
          static_cast<V*>(p->stage_val[cur ^ 1]), prm.fanout[l + 1], prm.shift[l + 1], p->counts);
    } else {
      k5_level<V, true, false><<<grid, kSplitThreads, split_smem_bytes<V>(true), st>>>(
          xc, xv, b.elems, off_cur, n_par, p->tile_meta, F, prm.shift[l], nullptr, p->cursor, p->stage_col[cur ^ 1],
          static_cast<V*>(p->stage_val[cur ^ 1]), 0, 0, nullptr);
    }
    p->stats.split_products += b.elems;
    hist_ready = next;
    ++p->stats.launches;
    GM_CUDA(cudaGetLastError());
    tm.end(st);
    std::swap(off_cur, off_nxt);
    cur ^= 1;
    n_par = n_child;
  }
  hs->fin_col = p->stage_col[cur];
  hs->fin_val = static_cast<V*>(p->stage_val[cur]);
  hs->chunk_off = off_cur;
  hs->n_chunks = n_par;
  hs->log2_cpr = ilog2_floor(static_cast<uint64_t>(prm.chunks_required));
  hs->tags = tag_cur;
  if (tag_cur) {
    hs->alt_col = p->stage_col[cur ^ 1];
    hs->alt_val = static_cast<V*>(p->stage_val[cur ^ 1]);
    for (int l = 1; l < prm.n_levels; ++l)
      if (level_buf[l] != cur) hs->xt.alt_bits |= 1u << (l + 1);
  }
  p->stats.final_chunks += n_par;
  p->stats.staged_products += b.elems;

  GM_TRY((launch_accumulate<V>(p, b, *hs, st)));  // (records its own two phases)
  tm.begin(PhaseTimes::kScan, st);
  exclusive_scan<u32, i64>(p->chunk_nnz, p->chunk_nnz_off, hs->n_chunks, p->scan_tmp, nullptr, nullptr, nullptr, st);
  k_heavy_row_counts<<<grid_for(rows_b, 256, p->num_sms), 256, 0, st>>>(p->chunk_nnz_off, hs->log2_cpr, rows_b, p->x_heavy,
                                                                        b.h0, p->row_nnz, p->c_total + 1);
  p->stats.launches += 4;
  tm.end(st);
  return GM_OK;
}

static int dev_error_to_status(int code) {
  switch (code) {
    case kDevOk: return GM_OK;
    case kDevCapacity: return fail(GM_ERR_CAPACITY, "C did not fit the room reserved for it (raise c_capacity or stage fewer products)");
    case kDevTableFull: return fail(GM_ERR_INTERNAL, "a light-row hash table overflowed");
    case kDevBadChunk: return fail(GM_ERR_INTERNAL, "an intermediate product reached a chunk that does not own its column");
    case kDevTimeout: return fail(GM_ERR_TIMEOUT, "a bounded wait on an asynchronous copy gave up");
    default: return fail(GM_ERR_INTERNAL, "unknown device error code");
  }
}

template <typename V>
static int execute_t(gm_plan* p, cudaStream_t st, gm_csr* C) {
  const gm_csr& A = p->A;
  const gm_csr& B = p->B;
  const i64 nA = A.n_rows;
  gm_plan_info& info = p->info;
  PhaseTimes& tm = p->times;
  p->stats = gm_exec_stats{};
  tm.reset();
  cudaEvent_t ev_total0 = nullptr, ev_total1 = nullptr;
  if (tm.enabled) { ev_total0 = tm.get(); ev_total1 = tm.get(); cudaEventRecord(ev_total0, st); }

  GM_CUDA(cudaMemsetAsync(p->err, 0, sizeof(int), st));
  GM_CUDA(cudaMemsetAsync(p->row_nnz, 0, static_cast<size_t>(nA + 1) * sizeof(int32_t), st));
  GM_CUDA(cudaMemsetAsync(p->c_total, 0, 16 * sizeof(int64_t), st));

  // ---- result row_ptr
  i64* c_row_ptr = static_cast<i64*>(dev_alloc(static_cast<size_t>(nA + 1) * sizeof(i64), st));
  if (!c_row_ptr) return fail(GM_ERR_OOM, "allocation of C.row_ptr failed");
  int32_t* c_col = nullptr;
  V* c_val = nullptr;
  // ---- light and heavy rows are independent until C.row_ptr is formed: the light rows' kernels go to a second
  // stream, forked from and joined back into the caller's with events (never when single_stream is set)
  bool fork = !p->opts.single_stream && info.rows_light > 0 && info.rows_heavy > 0;
  if (fork && !p->light_stream) {
    // one second stream per device for the life of the process (creating and destroying a stream per plan cost more
    // than the overlap gained on millisecond products); executes that share it are ordered by their own events
    static cudaStream_t side_streams[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
      fork = false;
    } else {
      if (!side_streams[dev] && cudaStreamCreateWithFlags(&side_streams[dev], cudaStreamNonBlocking) != cudaSuccess) {
        cudaGetLastError();
        side_streams[dev] = nullptr;
      }
      p->light_stream = side_streams[dev];
      if (!p->light_stream || cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&p->ev_light, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        p->light_stream = nullptr;
        fork = false;
      }
    }
  }
  cudaStream_t lst = fork ? p->light_stream : st;
  auto fork_light = [&]() { if (fork) { cudaEventRecord(p->ev_fork, st); cudaStreamWaitEvent(lst, p->ev_fork, 0); } };
  auto join_light = [&]() { if (fork) { cudaEventRecord(p->ev_light, lst); cudaStreamWaitEvent(st, p->ev_light, 0); } };
  auto cleanup = [&]() {
    if (fork) cudaStreamSynchronize(lst);
    if (p->sink && p->sink->copy_stream) cudaStreamSynchronize(p->sink->copy_stream);  // copies out of C in flight
    dev_free(c_row_ptr, st);
    dev_free(c_col, st);
    dev_free(c_val, st);
  };
#define GM_TRY_C(expr) do { int rc2_ = (expr); if (rc2_ != GM_OK) { cudaStreamSynchronize(st); cleanup(); return rc2_; } } while (0)

  // ---- light rows, symbolic (Algorithm 3: Symbolic(A[x_light,:], B))
  fork_light();
  tm.begin(PhaseTimes::kLightSym, lst);
  GM_TRY_C((launch_light<V, false>(p, p->sym_rows, p->sym_fill, info.light_bin_rows, nullptr, nullptr, nullptr, 0, lst)));
  tm.end(lst);
  bool light_counted = !fork;  // the heavy path joins before the first prefix sum over the per-row counts

  // a row's numeric bin is never above its symbolic bin
  i64 num_upper[kMaxLightBins] = {0};
  {
    i64 run = 0;
    for (int b = p->bins.n_bins - 1; b >= 0; --b) { run += info.light_bin_rows[b]; num_upper[b] = run; }
  }
  // numeric pass of the light rows in [r0, r1) (all of them by default)
  auto light_numeric_range = [&](i64 capacity, i64 r0, i64 r1, cudaStream_t s2) -> int {
    tm.begin(PhaseTimes::kLightNum, s2);
    if (info.rows_light > 0 && r1 > r0) {
      GM_CUDA(cudaMemsetAsync(p->num_fill, 0, 8 * sizeof(int), s2));
      k1_bin_rows<int32_t><<<static_cast<unsigned>((r1 - r0 + 255) / 256), 256, 0, s2>>>(
          p->row_nnz + r0, p->heavy_flag + r0, r1 - r0, p->bins, std::max<i64>(nA, 1), p->num_fill, p->num_rows, r0);
      ++p->stats.launches;
      GM_TRY((launch_light<V, true>(p, p->num_rows, p->num_fill, num_upper, c_row_ptr, c_col, c_val, capacity, s2)));
    }
    tm.end(s2);
    return GM_OK;
  };
  auto light_numeric = [&](i64 capacity, cudaStream_t s2) -> int { return light_numeric_range(capacity, 0, nA, s2); };

  const size_t n_batches = p->batches.size();
  i64 capacity = 0;
  i64 total = 0;
  i64 heavy_total = 0;
  int dev_err = 0;
  if (n_batches <= 1) {
    // ---- everything is resident at once: count, allocate C exactly, then fill
    HeavyBatchState<V> hs;
    if (n_batches == 1) GM_TRY_C(heavy_batch_front<V>(p, p->batches[0], &hs, st));
    join_light();
    light_counted = true;
    tm.begin(PhaseTimes::kScan, st);
    exclusive_scan<int32_t, i64>(p->row_nnz, c_row_ptr, nA, p->scan_tmp, nullptr, p->c_total, nullptr, st);
    p->stats.launches += 3;
    tm.end(st);
    if (cudaMemcpyAsync(&total, p->c_total, sizeof(i64), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
      cleanup();
      return fail(GM_ERR_CUDA, std::string("symbolic phase failed: ") + cudaGetErrorString(cudaGetLastError()));
    }
    capacity = total;
    c_col = static_cast<int32_t*>(dev_alloc(static_cast<size_t>(std::max<i64>(total, 1)) * sizeof(int32_t), st));
    c_val = static_cast<V*>(dev_alloc(static_cast<size_t>(std::max<i64>(total, 1)) * sizeof(V), st));
    if (!c_col || !c_val) { cleanup(); return fail(GM_ERR_OOM, "allocation of C (" + std::to_string(total) + " entries) failed"); }
    // the gather of the heavy rows and the numeric pass of the light rows write different rows of C
    fork_light();
    if (n_batches == 1) {
      tm.begin(PhaseTimes::kAccSym, st);
      GM_TRY_C((launch_gather<V>(p, p->batches[0], hs, c_row_ptr, c_col, c_val, capacity, st)));
      tm.end(st);
    }
    GM_TRY_C(light_numeric(capacity, lst));
    join_light();
  } else {
    // ---- heavy rows in several staging-buffer fills: C is appended in row order into reserved room
    // Room for C.  Given: use it.  Derived: the structural upper bound sum_i min(IP_i, C.m), cut
    // down to what the device can hold; if the allocator refuses (its own cache can hide free
    // memory from cudaMemGetInfo, or the estimate was too bold) retry with less.
    std::vector<i64> tries;
    if (p->opts.c_capacity > 0) {
      tries.push_back(p->opts.c_capacity);
    } else {
      size_t free_b = 0, total_b = 0;
      GM_CUDA(cudaMemGetInfo(&free_b, &total_b));
      const i64 entry = static_cast<i64>(4 + sizeof(V));
      const i64 inputs = (A.nnz + (&A == &B ? 0 : B.nnz)) * entry + (A.n_rows + B.n_rows + 2) * 8;
      const i64 by_total = (static_cast<i64>(total_b) - info.workspace_bytes - inputs - (nA + 1) * 8 - (i64{3} << 30)) / entry;
      const i64 by_free = (static_cast<i64>(free_b) - (nA + 1) * 8 - (i64{1} << 30)) / entry;
      const i64 hi = std::max<i64>(1, std::min<i64>(info.c_nnz_upper, std::max(by_total, by_free)));
      const i64 lo = std::max<i64>(1, std::min<i64>(info.c_nnz_upper, by_free));
      tries.push_back(hi);
      for (int k = 1; k <= 8 && hi > lo; ++k) tries.push_back(hi - (hi - lo) * k / 8);
    }
    for (i64 cand : tries) {
      capacity = cand;
      c_col = static_cast<int32_t*>(dev_alloc(static_cast<size_t>(capacity) * sizeof(int32_t), st));
      c_val = c_col ? static_cast<V*>(dev_alloc(static_cast<size_t>(capacity) * sizeof(V), st)) : nullptr;
      if (c_col && c_val) break;
      dev_free(c_col, st);
      c_col = nullptr;
      c_val = nullptr;
    }
    if (!c_col || !c_val) { cleanup(); return fail(GM_ERR_OOM, "allocation of C (room for " + std::to_string(capacity) + " entries) failed"); }
    for (size_t bi = 0; bi < n_batches; ++bi) {
      const Batch& b = p->batches[bi];
      HeavyBatchState<V> hs;
      GM_TRY_C(heavy_batch_front<V>(p, b, &hs, st));
      if (!light_counted) { join_light(); light_counted = true; }
      // rows [r0, r1) of C get their offsets now: every light row in the range was counted up front
      const i64 r0 = bi == 0 ? 0 : p->x_heavy_host[static_cast<size_t>(b.h0)];
      const i64 r1 = bi + 1 == n_batches ? nA : p->x_heavy_host[static_cast<size_t>(p->batches[bi + 1].h0)];
      tm.begin(PhaseTimes::kScan, st);
      exclusive_scan<int32_t, i64>(p->row_nnz + r0, c_row_ptr + r0, r1 - r0, p->scan_tmp, p->c_total, p->c_total, nullptr, st);
      p->stats.launches += 3;
      tm.end(st);
      tm.begin(PhaseTimes::kAccSym, st);
      GM_TRY_C((launch_gather<V>(p, b, hs, c_row_ptr, c_col, c_val, capacity, st)));
      tm.end(st);
      if (HostSink* sk = p->sink) {
        // The caller wants C on the host: finish rows [r0, r1) now (their light rows too), note how many entries
        // of C that makes, and send the previous batch's entries on their way while this batch computes.
        GM_TRY_C(light_numeric_range(capacity, r0, r1, st));
        if (sk->events.size() <= bi) {
          cudaEvent_t ev = nullptr;
          if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) { cleanup(); return fail(GM_ERR_CUDA, "event creation failed"); }
          sk->events.push_back(ev);
        }
        cudaMemcpyAsync(&sk->h_totals[bi], p->c_total, sizeof(i64), cudaMemcpyDeviceToHost, st);
        cudaEventRecord(sk->events[bi], st);
        auto send = [&](size_t done) {
          if (cudaEventSynchronize(sk->events[done]) != cudaSuccess) return;
          const i64 end = std::min<i64>(sk->h_totals[done], sk->capacity);
          if (end > sk->copied) {
            cudaStreamWaitEvent(sk->copy_stream, sk->events[done], 0);
            cudaMemcpyAsync(sk->h_col + sk->copied, c_col + sk->copied, static_cast<size_t>(end - sk->copied) * sizeof(int32_t),
                            cudaMemcpyDeviceToHost, sk->copy_stream);
            cudaMemcpyAsync(static_cast<V*>(sk->h_val) + sk->copied, c_val + sk->copied,
                            static_cast<size_t>(end - sk->copied) * sizeof(V), cudaMemcpyDeviceToHost, sk->copy_stream);
            sk->copied = end;
          }
        };
        if (bi > 0) send(bi - 1);
        if (bi + 1 == n_batches) send(bi);
      }
    }
    if (!p->sink) GM_TRY_C(light_numeric(capacity, st));
    if (cudaMemcpyAsync(&total, p->c_total, sizeof(i64), cudaMemcpyDeviceToHost, st) != cudaSuccess) {
      cleanup();
      return fail(GM_ERR_CUDA, "copy of nnz(C) failed");
    }
  }
  if (tm.enabled) cudaEventRecord(ev_total1, st);
  // heavy entries; products and entries of small chunks; of mid-size chunks; products and chunks that left the
  // hierarchy early; products the multisplit levels left in place
  i64 tail_totals[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  cudaMemcpyAsync(tail_totals, p->c_total + 1, 8 * sizeof(i64), cudaMemcpyDeviceToHost, st);
  cudaError_t e1 = cudaMemcpyAsync(&dev_err, p->err, sizeof(int), cudaMemcpyDeviceToHost, st);
  cudaError_t e2 = cudaStreamSynchronize(st);
  if (e1 != cudaSuccess || e2 != cudaSuccess) {
    cleanup();
    return fail(GM_ERR_CUDA, std::string("execute failed: ") + cudaGetErrorString(e2 != cudaSuccess ? e2 : e1));
  }
  if (dev_err != kDevOk || total > capacity) {
    cleanup();
    if (dev_err == kDevOk) dev_err = kDevCapacity;
    return dev_error_to_status(dev_err);
  }
#undef GM_TRY_C
  p->stats.c_nnz = total;
  heavy_total = tail_totals[0];
  p->stats.c_nnz_heavy = heavy_total;
  p->stats.small_chunk_products = tail_totals[1];
  p->stats.small_chunk_entries = tail_totals[2];
  p->stats.mid_chunk_products = tail_totals[3];
  p->stats.mid_chunk_entries = tail_totals[4];
  p->stats.early_exit_products = tail_totals[5];
  p->stats.early_exit_chunks = tail_totals[6];
  p->stats.split_products -= tail_totals[7];
  p->stats.c_capacity = capacity;
  if (tm.enabled) {
    float ph[PhaseTimes::kCount];
    tm.collect(ph);
    p->stats.ms_light_symbolic = ph[PhaseTimes::kLightSym];
    p->stats.ms_light_numeric = ph[PhaseTimes::kLightNum];
    p->stats.ms_expand = ph[PhaseTimes::kExpand];
    p->stats.ms_histogram = ph[PhaseTimes::kHist];
    p->stats.ms_multisplit = ph[PhaseTimes::kSplit];
    p->stats.ms_gather = ph[PhaseTimes::kAccSym];
    p->stats.ms_accumulate = ph[PhaseTimes::kAccNum];
    p->stats.ms_small_chunks = ph[PhaseTimes::kAccSmall];
    p->stats.ms_mid_chunks = ph[PhaseTimes::kAccMid];
    p->stats.ms_scan = ph[PhaseTimes::kScan];
    cudaEventElapsedTime(&p->stats.ms_total, ev_total0, ev_total1);
  }
  C->n_rows = nA;
  C->n_cols = B.n_cols;
  C->nnz = total;
  C->row_ptr = c_row_ptr;
  C->col_idx = c_col;
  C->vals = c_val;
  C->dtype = A.dtype;
  C->reserved = 0;
  return GM_OK;
}

}  // namespace gm

// ------------------------------------------------------------------------------------------------
// extern "C"
// ------------------------------------------------------------------------------------------------
using namespace gm;

extern "C" {

int gm_set_allocator(gm_alloc_fn alloc_fn, gm_free_fn free_fn, void* user) {
  if ((alloc_fn == nullptr) != (free_fn == nullptr)) return fail(GM_ERR_INVALID_ARG, "alloc and free must be given together");
  g_alloc.alloc = alloc_fn;
  g_alloc.free = free_fn;
  g_alloc.user = user;
  return GM_OK;
}

int gm_spgemm_plan_ex(const gm_csr* A, const gm_csr* B, size_t smem_bytes, const gm_plan_opts* opts, void* cuda_stream,
                      gm_plan** plan_out) {
  if (!plan_out) return fail(GM_ERR_INVALID_ARG, "plan_out is null");
  *plan_out = nullptr;
  GM_TRY(check_csr_arg(A, "A"));
  GM_TRY(check_csr_arg(B, "B"));
  if (A->dtype != B->dtype) return fail(GM_ERR_DTYPE, "A and B have different value types");
  if (A->n_cols != B->n_rows) return fail(GM_ERR_DIM_MISMATCH, "A.n_cols != B.n_rows");
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) {
    cudaGetLastError();
    return fail(GM_ERR_CUDA, "no CUDA device: this library has no CPU path");
  }
  gm_plan* p = new gm_plan();
  p->A = *A;
  p->B = *B;
  p->sv = value_bytes(A->dtype);
  p->smem_bytes = smem_bytes;
  if (opts) p->opts = *opts;
  p->plan_stream = static_cast<cudaStream_t>(cuda_stream);
  const char* env = std::getenv("GM_TIMING");
  p->times.enabled = env && env[0] == '1';
  const int rc = build_plan(p, p->plan_stream);
  if (rc != GM_OK) {
    cudaStreamSynchronize(p->plan_stream);
    gm_plan_destroy(p);
    return rc;
  }
  *plan_out = p;
  return GM_OK;
}

int gm_spgemm_plan(const gm_csr* A, const gm_csr* B, size_t smem_bytes, gm_plan** plan_out) {
  return gm_spgemm_plan_ex(A, B, smem_bytes, nullptr, nullptr, plan_out);
}

int gm_spgemm_execute(gm_plan* plan, void* cuda_stream, gm_csr* C_out) {
  if (!plan || !C_out) return fail(GM_ERR_INVALID_ARG, "plan or C_out is null");
  std::memset(C_out, 0, sizeof(*C_out));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  return plan->A.dtype == GM_F32 ? execute_t<float>(plan, st, C_out) : execute_t<double>(plan, st, C_out);
}

int gm_plan_get_info(const gm_plan* plan, gm_plan_info* out) {
  if (!plan || !out) return fail(GM_ERR_INVALID_ARG, "null argument");
  *out = plan->info;
  return GM_OK;
}

int gm_exec_get_stats(const gm_plan* plan, gm_exec_stats* out) {
  if (!plan || !out) return fail(GM_ERR_INVALID_ARG, "null argument");
  *out = plan->stats;
  return GM_OK;
}

int gm_plan_set_timing(gm_plan* plan, int enable) {
  if (!plan) return fail(GM_ERR_INVALID_ARG, "null plan");
  plan->times.enabled = enable != 0;
  return GM_OK;
}

int gm_plan_get_row_products(const gm_plan* plan, int64_t* ip_out_device, void* cuda_stream) {
  if (!plan || !ip_out_device) return fail(GM_ERR_INVALID_ARG, "null argument");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (plan->A.n_rows > 0)
    GM_CUDA(cudaMemcpyAsync(ip_out_device, plan->ip, static_cast<size_t>(plan->A.n_rows) * sizeof(int64_t),
                            cudaMemcpyDeviceToDevice, st));
  return GM_OK;
}

void gm_csr_free(gm_csr* C) {
  if (!C) return;
  dev_free(const_cast<int64_t*>(C->row_ptr), nullptr);
  dev_free(const_cast<int32_t*>(C->col_idx), nullptr);
  dev_free(const_cast<void*>(C->vals), nullptr);
  std::memset(C, 0, sizeof(*C));
}

void gm_plan_destroy(gm_plan* plan) {
  if (!plan) return;
  if (plan->ev_fork) cudaEventDestroy(plan->ev_fork);
  if (plan->ev_light) cudaEventDestroy(plan->ev_light);
  for (auto& b : plan->owned) dev_free(b.p, plan->plan_stream);
  delete plan;
}

int gm_spgemm_host(const gm_csr* A_host, const gm_csr* B_host, size_t smem_bytes, const gm_plan_opts* opts, gm_csr* C_host,
                   int64_t c_capacity) {
  GM_TRY(check_csr_arg(A_host, "A_host"));
  GM_TRY(check_csr_arg(B_host, "B_host"));
  if (!C_host || !C_host->row_ptr || c_capacity < 0) return fail(GM_ERR_INVALID_ARG, "C_host needs caller-owned buffers");
  if (A_host->dtype != B_host->dtype) return fail(GM_ERR_DTYPE, "A and B have different value types");
  const size_t sv = static_cast<size_t>(value_bytes(A_host->dtype));
  cudaStream_t st = nullptr;
  GM_CUDA(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
  gm_csr dev[2];
  std::vector<void*> tmp;
  int rc = GM_OK;
  auto upload = [&](const gm_csr* H, gm_csr* D) -> int {
    *D = *H;
    void* rp = dev_alloc(static_cast<size_t>(H->n_rows + 1) * 8, st);
    void* ci = dev_alloc(static_cast<size_t>(H->nnz) * 4, st);
    void* va = dev_alloc(static_cast<size_t>(H->nnz) * sv, st);
    tmp.push_back(rp); tmp.push_back(ci); tmp.push_back(va);
    if (!rp || !ci || !va) return fail(GM_ERR_OOM, "device allocation for an input failed");
    GM_CUDA(cudaMemcpyAsync(rp, H->row_ptr, static_cast<size_t>(H->n_rows + 1) * 8, cudaMemcpyHostToDevice, st));
    if (H->nnz > 0) {
      GM_CUDA(cudaMemcpyAsync(ci, H->col_idx, static_cast<size_t>(H->nnz) * 4, cudaMemcpyHostToDevice, st));
      GM_CUDA(cudaMemcpyAsync(va, H->vals, static_cast<size_t>(H->nnz) * sv, cudaMemcpyHostToDevice, st));
    }
    D->row_ptr = static_cast<const int64_t*>(rp);
    D->col_idx = static_cast<const int32_t*>(ci);
    D->vals = va;
    return GM_OK;
  };
  gm_plan* plan = nullptr;
  gm_csr C{};
  rc = upload(A_host, &dev[0]);
  if (rc == GM_OK) rc = upload(B_host, &dev[1]);
  if (rc == GM_OK) rc = gm_spgemm_plan_ex(&dev[0], &dev[1], smem_bytes, opts, st, &plan);
  // With several batches, C's entries travel to the host batch by batch while later batches compute.
  HostSink sink;
  bool use_sink = false;
  if (rc == GM_OK && plan->batches.size() > 1 && C_host->col_idx && C_host->vals && c_capacity > 0) {
    sink.h_col = const_cast<int32_t*>(C_host->col_idx);
    sink.h_val = const_cast<void*>(C_host->vals);
    sink.capacity = c_capacity;
    use_sink = cudaStreamCreateWithFlags(&sink.copy_stream, cudaStreamNonBlocking) == cudaSuccess &&
               cudaMallocHost(reinterpret_cast<void**>(&sink.h_totals), plan->batches.size() * sizeof(int64_t)) == cudaSuccess;
    if (use_sink) plan->sink = &sink;
  }
  if (rc == GM_OK) rc = gm_spgemm_execute(plan, st, &C);
  if (plan) plan->sink = nullptr;
  if (rc == GM_OK) {
    C_host->n_rows = C.n_rows;
    C_host->n_cols = C.n_cols;
    C_host->nnz = C.nnz;
    C_host->dtype = C.dtype;
    cudaError_t e = cudaMemcpyAsync(const_cast<int64_t*>(C_host->row_ptr), C.row_ptr, static_cast<size_t>(C.n_rows + 1) * 8,
                                    cudaMemcpyDeviceToHost, st);
    if (C.nnz > c_capacity) {
      rc = fail(GM_ERR_CAPACITY, "C has " + std::to_string(C.nnz) + " entries, more than c_capacity");
    } else if (C.nnz > 0 && e == cudaSuccess) {
      if (!C_host->col_idx || !C_host->vals) {
        rc = fail(GM_ERR_INVALID_ARG, "C_host->col_idx / vals are null");
      } else {
        const int64_t done = use_sink ? sink.copied : 0;  // entries the batches have already sent
        if (C.nnz > done) {
          e = cudaMemcpyAsync(const_cast<int32_t*>(C_host->col_idx) + done, C.col_idx + done,
                              static_cast<size_t>(C.nnz - done) * 4, cudaMemcpyDeviceToHost, st);
          if (e == cudaSuccess)
            e = cudaMemcpyAsync(static_cast<char*>(const_cast<void*>(C_host->vals)) + static_cast<size_t>(done) * sv,
                                static_cast<const char*>(C.vals) + static_cast<size_t>(done) * sv,
                                static_cast<size_t>(C.nnz - done) * sv, cudaMemcpyDeviceToHost, st);
        }
      }
    }
    if (use_sink && cudaStreamSynchronize(sink.copy_stream) != cudaSuccess && e == cudaSuccess) e = cudaErrorUnknown;
    cudaError_t e2 = cudaStreamSynchronize(st);
    if (rc == GM_OK && (e != cudaSuccess || e2 != cudaSuccess)) rc = fail(GM_ERR_CUDA, "copy of C to the host failed");
    dev_free(const_cast<int64_t*>(C.row_ptr), st);
    dev_free(const_cast<int32_t*>(C.col_idx), st);
    dev_free(const_cast<void*>(C.vals), st);
  }
  if (plan) {
    plan->plan_stream = st;
    gm_plan_destroy(plan);
  }
  for (void* q : tmp) dev_free(q, st);
  cudaStreamSynchronize(st);
  if (sink.copy_stream) {
    cudaStreamSynchronize(sink.copy_stream);
    cudaStreamDestroy(sink.copy_stream);
  }
  for (cudaEvent_t ev : sink.events) cudaEventDestroy(ev);
  if (sink.h_totals) cudaFreeHost(sink.h_totals);
  cudaStreamDestroy(st);
  return rc;
}

const char* gm_status_string(int status) {
  switch (status) {
    case GM_OK: return "GM_OK";
    case GM_ERR_INVALID_ARG: return "GM_ERR_INVALID_ARG";
    case GM_ERR_DIM_MISMATCH: return "GM_ERR_DIM_MISMATCH";
    case GM_ERR_DTYPE: return "GM_ERR_DTYPE";
    case GM_ERR_BAD_CSR: return "GM_ERR_BAD_CSR";
    case GM_ERR_OOM: return "GM_ERR_OOM";
    case GM_ERR_CAPACITY: return "GM_ERR_CAPACITY";
    case GM_ERR_CUDA: return "GM_ERR_CUDA";
    case GM_ERR_TIMEOUT: return "GM_ERR_TIMEOUT";
    case GM_ERR_UNSUPPORTED_SMEM: return "GM_ERR_UNSUPPORTED_SMEM";
    case GM_ERR_INTERNAL: return "GM_ERR_INTERNAL";
    default: return "GM_ERR_UNKNOWN";
  }
}

const char* gm_last_error(void) { return g_last_error.c_str(); }

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Row analysis without any allocation (see gm_row_products_noalloc in gmagnus.h)
// ------------------------------------------------------------------------------------------------
namespace gm {

constexpr i64 kNoAllocMaxNnz = GM_NOALLOC_MAX_NNZ_A;

// Scratch of the no-allocation entry point, part of the library image on every device that loads it.
// In host code this name is only a handle for cudaGetSymbolAddress, not a device address.
struct NoAllocScratch {
  i64 nz_off[kNoAllocMaxNnz + 8];                    // prefix sums of the products per stored entry of A
  i64 scan_tmp[kNoAllocMaxNnz / kScanTile + 8];      // tile sums of the prefix sum
  int32_t nz_len[kNoAllocMaxNnz + 8];                // products per stored entry of A
};
static __device__ __align__(256) NoAllocScratch g_noalloc_scratch;

__global__ void k1_row_products_only(const i64* __restrict__ a_row_ptr, i64 n_rows, const i64* __restrict__ nz_off,
                                     i64* __restrict__ ip) {
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_rows;
       i += static_cast<i64>(gridDim.x) * blockDim.x)
    ip[i] = nz_off[a_row_ptr[i + 1]] - nz_off[a_row_ptr[i]];
}

constexpr int kNoAllocMaxDevices = 64;
static NoAllocScratch* g_noalloc_ptr[kNoAllocMaxDevices] = {nullptr};
static int g_noalloc_sms[kNoAllocMaxDevices] = {0};

}  // namespace gm

extern "C" int gm_row_products_noalloc(const gm_csr* A, const gm_csr* B, int64_t* ip_out_device, void* cuda_stream) {
  GM_TRY(check_csr_arg(A, "A", true));
  GM_TRY(check_csr_arg(B, "B", true));
  if (!ip_out_device && A->n_rows > 0) return fail(GM_ERR_INVALID_ARG, "ip_out_device is null");
  if (A->n_cols != B->n_rows) return fail(GM_ERR_DIM_MISMATCH, "A.n_cols != B.n_rows");
  if (A->nnz > kNoAllocMaxNnz)
    return fail(GM_ERR_CAPACITY, "gm_row_products_noalloc handles at most " + std::to_string(kNoAllocMaxNnz) +
                                     " stored entries of A (got " + std::to_string(A->nnz) + "): its scratch is a fixed array");
  int dev = 0;
  GM_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kNoAllocMaxDevices) return fail(GM_ERR_INVALID_ARG, "device index out of range");
  if (!g_noalloc_ptr[dev]) {
    // set-up, once per device, with that device current: the device address behind the symbol
    void* ptr = nullptr;
    GM_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    int sms = 0;
    GM_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    g_noalloc_sms[dev] = sms;
    g_noalloc_ptr[dev] = static_cast<NoAllocScratch*>(ptr);
  }
  NoAllocScratch* sc = g_noalloc_ptr[dev];
  const int sms = g_noalloc_sms[dev];
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // scratch members are addressed through the device pointer, never through the host-side symbol
  int32_t* nz_len = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(sc) + offsetof(NoAllocScratch, nz_len));
  i64* nz_off = reinterpret_cast<i64*>(reinterpret_cast<char*>(sc) + offsetof(NoAllocScratch, nz_off));
  i64* scan_tmp = reinterpret_cast<i64*>(reinterpret_cast<char*>(sc) + offsetof(NoAllocScratch, scan_tmp));
  if (A->nnz > 0) k1_nz_len<<<grid_for(A->nnz, 256, sms, 32), 256, 0, st>>>(A->col_idx, A->nnz, B->row_ptr, nz_len);
  exclusive_scan<int32_t, i64>(nz_len, nz_off, A->nnz, scan_tmp, nullptr, nullptr, nullptr, st);
  if (A->n_rows > 0)
    k1_row_products_only<<<grid_for(A->n_rows, 256, sms), 256, 0, st>>>(A->row_ptr, A->n_rows, nz_off, ip_out_device);
  GM_CUDA(cudaGetLastError());
  return GM_OK;
}
