/*
 * gmagnus.h — C ABI of the B200 (sm_100a) SpGEMM library:  C = A * B  for CSR matrices with
 * irregular, power-law structure, following the gMAGNUS method (light rows: Gustavson with a
 * shared-memory hash accumulator; heavy rows: expansion of the intermediate products into a
 * staging buffer, hierarchical multisplit by column chunk, dense shared-memory accumulation).
 *
 * Conventions
 *   - Every function returns an int status: GM_OK (0) or a negative GM_ERR_* code.  No exception
 *     crosses this boundary, nothing aborts, and no kernel traps.  gm_last_error() gives a text
 *     for the last failure on the calling thread.
 *   - Unless a function says "host", every pointer inside a gm_csr is a DEVICE pointer on the
 *     current CUDA device.  Inputs stay owned by the caller and must stay valid and unchanged
 *     until the plan that borrowed them is destroyed.
 *   - CSR layout (Section II-A of the paper): row_ptr has n_rows + 1 int64 entries with
 *     row_ptr[0] = 0 and row_ptr[n_rows] = nnz; row i owns entries [row_ptr[i], row_ptr[i+1]) of
 *     col_idx (int32) and vals (float or double).  Columns inside a row must be strictly
 *     ascending.  Explicitly stored zeros are ordinary entries.
 *   - The result follows Eq. 1 / Algorithm 1: C[i,:] = sum_j A[i,j] * B[j,:], rows sorted by
 *     column, one entry per column that receives at least one product (structural zeros are
 *     kept).  The order in which the products of one entry are summed is unspecified, so values
 *     can differ in the last bits from run to run; the structure never does.
 *   - There is no CPU fallback: every function that computes needs a CUDA device and fails with
 *     GM_ERR_CUDA without one.
 */
#ifndef GMAGNUS_H_
#define GMAGNUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { GM_F32 = 0, GM_F64 = 1 } gm_dtype;

enum {
  GM_OK = 0,
  GM_ERR_INVALID_ARG = -1,      /* null pointer, negative size, bad option value              */
  GM_ERR_DIM_MISMATCH = -2,     /* A.n_cols != B.n_rows                                        */
  GM_ERR_DTYPE = -3,            /* A and B value types differ or are unknown                   */
  GM_ERR_BAD_CSR = -4,          /* validation (option validate_inputs) found a malformed input */
  GM_ERR_OOM = -5,              /* a device allocation failed                                  */
  GM_ERR_CAPACITY = -6,         /* a fixed capacity (staging, C, 32-bit batch offsets) is too small */
  GM_ERR_CUDA = -7,             /* a CUDA runtime call failed / no device                      */
  GM_ERR_TIMEOUT = -8,          /* a bounded device-side wait gave up                          */
  GM_ERR_UNSUPPORTED_SMEM = -9, /* smem_bytes above the device's opt-in maximum or below 16 KB */
  GM_ERR_INTERNAL = -10         /* a device-side consistency check failed                      */
};

/* A CSR matrix.  For inputs all arrays are caller-owned device memory.  For the result of
 * gm_spgemm_execute the arrays are allocated by the library (through the allocator hook) and
 * released with gm_csr_free; col_idx / vals may have room for more than nnz entries. */
typedef struct gm_csr {
  int64_t n_rows, n_cols, nnz;
  const int64_t* row_ptr; /* n_rows + 1 */
  const int32_t* col_idx; /* nnz        */
  const void* vals;       /* nnz values of `dtype` */
  int32_t dtype;          /* gm_dtype   */
  int32_t reserved;
} gm_csr;

#define GM_MAX_LEVELS 8

/* Planner overrides.  Zero-initialise, then set only what you need: 0 always means "derive it".
 * None of these can change C; they change how the work is split (Section III-D). */
typedef struct gm_plan_opts {
  int64_t tau;             /* heavy-row threshold: row i is heavy iff IP_i > tau               */
  int32_t chunk_width;     /* W: columns per final chunk (power of two)                        */
  int32_t max_fanout;      /* n_chunksMax: most children one multisplit level may produce (pow2) */
  int32_t acc_ctas_per_sm; /* 1, 2, 4 or 8: how many chunk accumulators share one SM (sets W)  */
  int64_t stage_elems;     /* capacity, in intermediate products, of each staging half-buffer  */
  int64_t c_capacity;      /* room, in entries, reserved for C when heavy rows need > 1 batch  */
  int32_t separate_histogram; /* 1: always run the stand-alone histogram kernel per level (otherwise a
                              first level that runs as separate passes is counted by the expansion) */
  int32_t validate_inputs; /* 1: debug mode.  row_ptr / col_idx of A and B are checked on the device first
                              (GM_ERR_BAD_CSR), and before every chunk accumulation a pass over the staging buffer
                              checks that each product lies in the columns its chunk owns (GM_ERR_INTERNAL)     */
  int32_t single_stream;   /* 1: every kernel of a call runs on the caller's stream.  0 (default): the light rows'
                              kernels run on a second stream of the plan's, forked from and joined back into the
                              caller's stream with events, next to the heavy rows' kernels (Algorithm 3)      */
  int32_t level0_multisplit; /* first multisplit level: 1 = separate histogram and multisplit passes over
                              the staging buffer (Algorithm 5 as printed); 2 = the expansion kernel writes
                              the first level's children itself; 0 (default) = the latter when the heavy
                              rows' segments are long compared with the fan-out, else the former        */
  int32_t small_chunk_max; /* final chunks of at most this many products are sorted by one warp each (Section
                              III-A's branch for light chunks); 0 = default (128), -1 = none, at most 512        */
  int32_t mid_chunk_max;   /* final chunks of at most this many products (and more than small_chunk_max) get one
                              128-thread block each, symbolic then numeric pass over a compact array; larger
                              ones go to the dense W-column accumulator.  0 = default (4096 for fp32, 2048 for
                              fp64, less when shared memory is short), -1 = none                                 */
  int32_t expand_staging;  /* 1: the expansion that writes the first level's children brings the rows of B into
                              shared memory with bulk asynchronous copies (one pipeline per warp; needs B's arrays
                              16-byte aligned, otherwise ignored).  0 (default) / -1: ordinary loads, one tile of
                              products per block — measured faster on B200 at every size tried               */
  int32_t debug_spin_limit; /* testing aid: polls a kernel spends on a wait for bulk copies before it gives up and
                              the call returns GM_ERR_TIMEOUT (0 = the default, about four million).  Negative:
                              the copies are announced but withheld, so the wait runs out after that many polls
                              with nothing in flight (how the tests reach the time-out path)                     */
  int32_t expand_order;    /* 1: the expansion runs in outer-product order (Eq. 2, Algorithm 4 as printed): the
                              batch's segments are sorted by row of B (masked CSR->CSC), so a row of B is read once
                              for all heavy rows that use it; the first multisplit level then runs as separate
                              passes.  0 (default): row order                                                   */
  int32_t early_exit;      /* Algorithm 3's early exit (only heavy chunks recurse): from the second level on, a chunk
                              with at most this many products is not split further; it stays in the level's input
                              buffer and is accumulated by the one-warp sort over its whole column span.  0 =
                              default (small_chunk_max), -1 = every chunk goes through every level, at most
                              small_chunk_max                                                                  */
} gm_plan_opts;

/* What the host planner derives from (C.m, value size, smem_bytes): Section III-D. */
typedef struct gm_params {
  int64_t tau;               /* light-row capacity: largest IP_i handled in shared memory      */
  int32_t light_slots;       /* hash-table slots behind tau                                    */
  int32_t chunk_width;       /* W                                                              */
  int32_t chunks_required;   /* ceil(C.m / W) rounded up to a power of two                     */
  int32_t max_fanout;        /* n_chunksMax, floored to a power of two                         */
  int32_t n_levels;          /* number of multisplit levels (0 when one chunk covers C.m)      */
  int32_t fanout[GM_MAX_LEVELS]; /* v_chunks: children per parent at each level                */
  int32_t shift[GM_MAX_LEVELS];  /* child at level l = (col >> shift[l]) & (fanout[l] - 1)     */
  int32_t acc_ctas_per_sm;
  int32_t acc_block_threads; /* threads of one accumulate block                                  */
} gm_params;

typedef struct gm_plan_info {
  gm_params params;
  int64_t n_rows, n_cols_c;
  int64_t products_total;  /* IP = sum_i IP_i                                                  */
  int64_t products_heavy;  /* sum of IP_i over heavy rows (= size of the intermediate matrix)  */
  int64_t products_max_row;
  int64_t rows_heavy, rows_light, rows_empty;
  int64_t nnz_a_heavy;     /* stored entries of A inside heavy rows                            */
  int64_t c_nnz_upper;     /* sum_i min(IP_i, C.m): an upper bound on nnz(C)                   */
  int64_t n_batches;       /* heavy rows are processed in this many staging-buffer fills       */
  int64_t stage_elems;     /* capacity of one staging half-buffer, in products                 */
  int64_t workspace_bytes; /* device memory held by the plan                                   */
  int64_t light_bin_rows[8]; /* light rows per size class of the symbolic pass                 */
  int64_t launches;        /* kernels launched while planning                                  */
  int64_t level0_direct;   /* 1: the expansion kernel writes the first level's children itself  */
} gm_plan_info;

/* Filled by the most recent gm_spgemm_execute on the plan.  Times are CUDA-event milliseconds on
 * the execute stream and are only recorded when the plan was made with GM_TIMING=1 in the
 * environment or through gm_plan_set_timing(plan, 1); otherwise they are 0. */
typedef struct gm_exec_stats {
  int64_t c_nnz;
  int64_t c_nnz_heavy;         /* entries of C that belong to heavy rows                       */
  int64_t c_capacity;          /* entries the C arrays have room for                           */
  int64_t staged_products;     /* products written to the staging buffer (all batches)         */
  int64_t final_chunks;        /* (row, chunk) pairs handed to the accumulate kernel           */
  int64_t launches;            /* kernels launched by this execute                             */
  int64_t small_chunk_products; /* products in chunks handled by the one-warp-per-chunk kernel   */
  int64_t small_chunk_entries;  /* entries of C those chunks produced                            */
  float ms_light_symbolic, ms_light_numeric, ms_expand, ms_histogram, ms_multisplit,
      ms_accumulate, ms_gather, ms_scan, ms_total;
  float ms_small_chunks;       /* the one-warp-per-chunk kernel; ms_accumulate is the dense-accumulator kernel alone */
  float ms_mid_chunks;         /* the one-small-block-per-chunk kernel                                          */
  float reserved[3];
  int64_t mid_chunk_products;  /* products in chunks handled by the one-small-block-per-chunk kernel             */
  int64_t mid_chunk_entries;   /* entries of C those chunks produced                                             */
  int64_t early_exit_products; /* products of chunks that left the multisplit hierarchy before its last level    */
  int64_t early_exit_chunks;   /* ... and how many chunks did                                                     */
  int64_t split_products;      /* products moved by multisplit passes, summed over the levels                     */
} gm_exec_stats;

typedef struct gm_plan gm_plan; /* opaque, owned by the library */

/* Device allocator hook.  alloc(bytes, stream, user) returns a device pointer aligned to at least
 * 256 bytes (the kernels use 16-byte accesses into the workspace and into C), or NULL; it is
 * called from host code of plan/execute only, never from a kernel.  Passing NULLs restores the
 * default (stream-ordered cudaMallocAsync on the device's default pool). */
typedef void* (*gm_alloc_fn)(size_t bytes, void* cuda_stream, void* user);
typedef void (*gm_free_fn)(void* ptr, void* cuda_stream, void* user);
int gm_set_allocator(gm_alloc_fn alloc_fn, gm_free_fn free_fn, void* user);

/* Host-only, no CUDA call: the parameter selection of Section III-D (GetMagnusParams) re-derived
 * for the given shared-memory budget.  tau follows Eq. 4 read as capacity = bytes / (slot bytes
 * per stored entry); chunks_required = C.m / W rounded up to a power of two; max_fanout follows
 * Eq. 6; n_levels follows Eq. 7 and the split puts max_fanout on every level but the last.
 * c_cols = C.m, opts may be NULL.  Errors: GM_ERR_INVALID_ARG, GM_ERR_UNSUPPORTED_SMEM. */
int gm_planner_params(int64_t c_cols, int32_t dtype, size_t smem_bytes, const gm_plan_opts* opts,
                      gm_params* out);

/* Host-only, no CUDA call: cuts the heavy rows into consecutive batches whose intermediate products
 * fit one staging half-buffer (the paper keeps the whole intermediate matrix resident, Section
 * III-A; batching is this library's addition for matrices whose intermediate matrix exceeds HBM).
 * heavy_prefix: n_heavy + 1 exclusive prefix sums of IP_i over the heavy rows (host).  Writes the
 * batch boundaries (heavy-row positions, first = 0, last = n_heavy) to bounds_out (room for
 * max_bounds entries) and returns the number of batches, or GM_ERR_CAPACITY if one row alone
 * exceeds stage_elems or bounds_out is too small.  A row is never split across batches. */
int64_t gm_planner_batches(const int64_t* heavy_prefix, int64_t n_heavy, int64_t stage_elems,
                           int64_t* bounds_out, int64_t max_bounds);

/* Setup phase of Algorithm 3 (GetMagnusParams, InterOffsets, ThreshPartition) plus everything
 * else that depends only on the structure of A and B: counts the intermediate products of every
 * row (IP_i = sum over entries j of A[i,:] of nnz(B[A.col[j],:])), splits rows into light and
 * heavy (IP_i > tau), bins the light rows by size, lays out the heavy rows' flattened product
 * space, cuts it into batches that fit the staging buffer, and allocates the workspace.
 *   A, B        host structs holding device pointers (see gm_csr); A.n_cols must equal B.n_rows
 *   smem_bytes  shared memory per block the kernels may use (s_LM); at most the device's opt-in
 *               maximum (232448 on B200), at least 16384
 *   plan_out    receives the plan; release it with gm_plan_destroy
 * Runs on `cuda_stream` (gm_spgemm_plan: the legacy default stream) and synchronises it before
 * returning, because the planner needs counts on the host.  The plan borrows A's and B's arrays. */
int gm_spgemm_plan(const gm_csr* A, const gm_csr* B, size_t smem_bytes, gm_plan** plan_out);
int gm_spgemm_plan_ex(const gm_csr* A, const gm_csr* B, size_t smem_bytes,
                      const gm_plan_opts* opts, void* cuda_stream, gm_plan** plan_out);

/* The rest of Algorithm 3: light rows by Gustavson's method with a shared-memory hash accumulator
 * (symbolic, then numeric); heavy rows, batch by batch, through the expansion (outer-product)
 * kernel (Algorithm 4), one histogram + multisplit (Algorithm 5) per level (by default the first
 * level is done by the expansion kernel itself, see gm_plan_opts.level0_multisplit), the
 * chunk-accumulate kernels (the chunks are binned by size as in Section III-E: small ones by a one-warp
 * sort, mid-size ones by a small block in a symbolic and a numeric pass, the others in the dense
 * shared-memory accumulator; every chunk is compacted in place and its entries counted) and, once
 * C.row_ptr is known by prefix sums over the per-row counts, the gather of the chunks into C.
 *   C_out  host struct filled with device pointers allocated through the allocator hook;
 *          C_out->nnz is exact.  Release with gm_csr_free.
 * Work is enqueued on `cuda_stream` (the light rows' kernels on a second stream ordered inside it by events,
 * unless single_stream is set); the call returns after synchronising that stream, because nnz(C) is needed
 * on the host.
 * A plan can be executed any number of times (values of A and B may change in between, their
 * structure may not).  Two executes of the same plan must not overlap.
 * Errors: GM_ERR_CAPACITY (C did not fit the reserved room; only possible when the heavy rows
 * need more than one batch), GM_ERR_OOM, GM_ERR_CUDA, GM_ERR_INTERNAL. */
int gm_spgemm_execute(gm_plan* plan, void* cuda_stream, gm_csr* C_out);

/* Convenience for callers whose matrices live in HOST memory (all pointers in A_host / B_host and
 * in C_host are host pointers; pinned memory makes the copies faster).  Copies A and B to the
 * device, plans, executes, and copies C back.  C_host->row_ptr / col_idx / vals must point to
 * caller-owned buffers with room for n_rows + 1 / c_capacity / c_capacity entries; on return
 * C_host->nnz is set.  If nnz(C) > c_capacity only row_ptr is copied and GM_ERR_CAPACITY is
 * returned (C_host->nnz then tells the room needed).  Synchronous.  When the heavy rows take several
 * batches, the rows of every batch (its light rows included) are finished and copied out while the next
 * batch computes, so the copy of C overlaps the computation; the buffers hold valid entries only after
 * the call has returned GM_OK. */
int gm_spgemm_host(const gm_csr* A_host, const gm_csr* B_host, size_t smem_bytes,
                   const gm_plan_opts* opts, gm_csr* C_host, int64_t c_capacity);

/* Plan queries (host structs out). */
int gm_plan_get_info(const gm_plan* plan, gm_plan_info* out);
int gm_exec_get_stats(const gm_plan* plan, gm_exec_stats* out);
int gm_plan_set_timing(gm_plan* plan, int enable);
/* Copies IP_i (row-analysis result, InterOffsets of Section III-A) for all rows of A into the
 * DEVICE array ip_out (n_rows int64), on `cuda_stream`. */
int gm_plan_get_row_products(const gm_plan* plan, int64_t* ip_out_device, void* cuda_stream);

/* Row analysis for callers that must not allocate.  The paper has no counterpart: this is a packaging
 * variant of the row-analysis kernels behind gm_spgemm_plan.
 *
 * Some callers cannot let a library allocate device memory on their behalf: a service that hands a
 * fixed memory budget to each component at start-up, code that runs between the begin and end of a
 * latency-critical section where an allocation (which may synchronise the whole device) is not
 * acceptable, or a host whose allocator is owned by another runtime.  For them this entry point
 * computes IP_i = sum over stored entries j of A[i,:] of nnz(B[A.col[j],:]) for every row of A and
 * allocates nothing: no cudaMalloc / cudaFree, no stream-ordered allocation, no allocator hook.
 * Its scratch (products per stored entry, their prefix sums, tile sums of the scan) lives in a
 * fixed array inside the library image: about 12.6 MB of device memory on every GPU that loads the
 * library, held until the process exits.
 *   A, B           host structs with DEVICE pointers, as for gm_spgemm_plan; only row_ptr and col_idx are
 *                  read, so vals may be NULL and dtype is ignored.  Columns of A are not range-checked:
 *                  an entry of A.col_idx outside [0, B.n_rows) reads past B.row_ptr
 *   ip_out_device  DEVICE array of A->n_rows int64, written by the call
 *   cuda_stream    the work is enqueued there; the call does not synchronise
 * Limit: A->nnz <= GM_NOALLOC_MAX_NNZ_A (1,048,576); larger inputs are rejected with GM_ERR_CAPACITY
 * and nothing is launched.  Any number of rows.
 * The first call on each device looks up the address of the scratch array (one
 * cudaGetSymbolAddress with that device current); make that first call before starting any stream
 * capture.  Every call uses the same scratch array: everything in it is rewritten before it is
 * read, so nothing needs clearing, but two calls whose kernels can overlap on the GPU (different
 * streams, or concurrent host threads) race on it — serialise them. */
#define GM_NOALLOC_MAX_NNZ_A 1048576
int gm_row_products_noalloc(const gm_csr* A, const gm_csr* B, int64_t* ip_out_device, void* cuda_stream);

/* Releases the arrays of a result produced by gm_spgemm_execute and zeroes the struct. */
void gm_csr_free(gm_csr* C);
void gm_plan_destroy(gm_plan* plan);

const char* gm_status_string(int status);
const char* gm_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* GMAGNUS_H_ */
