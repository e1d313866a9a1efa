// CPU oracle for CSR SpGEMM  C = A * B.   TEST INFRASTRUCTURE ONLY.
//
// This file is the correctness reference the CUDA path is compared with.  It is deliberately
// plain and slow, shares no code with the CUDA library, and must only be used by the tests, by the
// smoke check and by the benchmark's CPU-baseline / reference legs.  The product never calls it.
//
// What it computes is the definition of the result, Gustavson's row-wise formulation (Eq. 1,
// Algorithm 1 of the paper):  for each row i, for each stored entry j of A[i,:] in stored order,
// for each stored entry k of B[A.col[j],:] in stored order,
//        accumBuff[B.col[k]] += A.val[j] * B.val[k]
// followed by "SortAndWrite": the touched columns are emitted in ascending order.  An output entry
// exists iff at least one product lands on it (structural zeros are kept, whatever the sum).
//
// Besides the sum it returns, per output entry, abs = sum |A.val[j] * B.val[k]|, the scale the
// value tolerance is stated against.  Arithmetic: fp32 inputs are widened to double (every
// fp32 x fp32 product is exact in double) and summed in double; fp64 inputs are multiplied and
// summed in long double (x87 80-bit) and rounded to double once at the end, so the reference's own
// rounding error stays far below the 1e-12 relative tolerance used for fp64.
//
// The number of intermediate products of row i is, by definition (Section III-A, InterOffsets),
//        IP_i = sum over stored entries j of A[i,:] of nnz(B[A.col[j],:]).
//
// Parity pins (tests/test_oracle_pins.py): brute-force dense products on tiny inputs, A*I = A,
// I*B = B, permutation products, the product-count identity, closed forms for the 5-point
// Laplacian squared and the fixed-degree random matrix, symmetry, and a cross-check against an
// independent library routine.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <thread>
#include <vector>

namespace {

struct CsrView {
  int64_t n_rows, n_cols;
  const int64_t* row_ptr;
  const int32_t* col;
  const void* val;
};

template <typename In, typename Acc>
struct RowWorker {
  // Dense accumulator over the column space of C, as in Algorithm 1, with a stamp array instead
  // of re-zeroing and a list of touched columns for SortAndWrite.
  std::vector<Acc> accum, accum_abs;
  std::vector<int64_t> stamp;
  std::vector<int32_t> touched;
  explicit RowWorker(int64_t c_cols) : accum(c_cols), accum_abs(c_cols), stamp(c_cols, -1) {}

  // Returns the number of output entries of row i; when out_col != nullptr also writes them.
  int64_t row(const CsrView& A, const CsrView& B, int64_t i, int32_t* out_col, double* out_val,
              double* out_abs) {
    const In* a_val = static_cast<const In*>(A.val);
    const In* b_val = static_cast<const In*>(B.val);
    touched.clear();
    for (int64_t j = A.row_ptr[i]; j < A.row_ptr[i + 1]; ++j) {
      const int64_t brow = A.col[j];
      const Acc a = static_cast<Acc>(a_val[j]);
      for (int64_t k = B.row_ptr[brow]; k < B.row_ptr[brow + 1]; ++k) {
        const int32_t c = B.col[k];
        const Acc p = a * static_cast<Acc>(b_val[k]);
        if (stamp[c] != i) {
          stamp[c] = i;
          accum[c] = 0;
          accum_abs[c] = 0;
          touched.push_back(c);
        }
        accum[c] += p;
        accum_abs[c] += (p < 0 ? -p : p);
      }
    }
    std::sort(touched.begin(), touched.end());
    if (out_col) {
      for (size_t t = 0; t < touched.size(); ++t) {
        const int32_t c = touched[t];
        out_col[t] = c;
        out_val[t] = static_cast<double>(accum[c]);
        out_abs[t] = static_cast<double>(accum_abs[c]);
      }
    }
    return static_cast<int64_t>(touched.size());
  }
};

int resolve_threads(int requested, int64_t c_cols) {
  int t = requested > 0 ? requested : static_cast<int>(std::thread::hardware_concurrency());
  if (t < 1) t = 1;
  // keep the per-thread dense accumulators within ~24 GB in total
  const double per_thread = static_cast<double>(c_cols) * (2 * sizeof(long double) + 8);
  const int cap = static_cast<int>(std::max(1.0, 24e9 / std::max(per_thread, 1.0)));
  return std::min(t, cap);
}

// mode 0: count only (row_nnz_out[i - r0]);  mode 1: fill, positions from local_row_ptr.
template <typename In, typename Acc>
int run_rows(const CsrView& A, const CsrView& B, int64_t r0, int64_t r1, int threads, int mode,
             int64_t* row_nnz_out, const int64_t* local_row_ptr, int32_t* out_col, double* out_val,
             double* out_abs) {
  const int T = resolve_threads(threads, B.n_cols);
  std::atomic<int64_t> next(r0);
  const int64_t block = 16;
  auto body = [&]() {
    RowWorker<In, Acc> w(B.n_cols);
    for (;;) {
      const int64_t b0 = next.fetch_add(block);
      if (b0 >= r1) break;
      const int64_t b1 = std::min(r1, b0 + block);
      for (int64_t i = b0; i < b1; ++i) {
        if (mode == 0) {
          row_nnz_out[i - r0] = w.row(A, B, i, nullptr, nullptr, nullptr);
        } else {
          const int64_t p = local_row_ptr[i - r0];
          w.row(A, B, i, out_col + p, out_val + p, out_abs + p);
        }
      }
    }
  };
  std::vector<std::thread> pool;
  for (int t = 1; t < T; ++t) pool.emplace_back(body);
  body();
  for (auto& th : pool) th.join();
  return T;
}

}  // namespace

extern "C" {

// IP_i for every row of A (definition of InterOffsets, Section III-A).  Returns the total.
int64_t oracle_row_products(int64_t a_rows, const int64_t* a_row_ptr, const int32_t* a_col,
                            const int64_t* b_row_ptr, int64_t* ip_out) {
  int64_t total = 0;
  for (int64_t i = 0; i < a_rows; ++i) {
    int64_t s = 0;
    for (int64_t j = a_row_ptr[i]; j < a_row_ptr[i + 1]; ++j)
      s += b_row_ptr[a_col[j] + 1] - b_row_ptr[a_col[j]];
    ip_out[i] = s;
    total += s;
  }
  return total;
}

// Symbolic pass over rows [r0, r1): row_nnz_out[i - r0] = number of entries of C[i,:].
// dtype: 0 = fp32 inputs, 1 = fp64 inputs.  Returns the number of threads used, < 0 on bad input.
int oracle_spgemm_count(int64_t a_rows, int64_t a_cols, const int64_t* a_row_ptr,
                        const int32_t* a_col, const void* a_val, int64_t b_rows, int64_t b_cols,
                        const int64_t* b_row_ptr, const int32_t* b_col, const void* b_val,
                        int dtype, int64_t r0, int64_t r1, int threads, int64_t* row_nnz_out) {
  if (a_cols != b_rows || r0 < 0 || r1 > a_rows || r0 > r1) return -1;
  CsrView A{a_rows, a_cols, a_row_ptr, a_col, a_val}, B{b_rows, b_cols, b_row_ptr, b_col, b_val};
  if (dtype == 0)
    return run_rows<float, double>(A, B, r0, r1, threads, 0, row_nnz_out, nullptr, nullptr,
                                   nullptr, nullptr);
  if (dtype == 1)
    return run_rows<double, long double>(A, B, r0, r1, threads, 0, row_nnz_out, nullptr, nullptr,
                                         nullptr, nullptr);
  return -2;
}

// Numeric pass over rows [r0, r1).  local_row_ptr (r1 - r0 + 1 entries, starting at 0) is the
// exclusive scan of the counts from oracle_spgemm_count; outputs hold local_row_ptr[r1 - r0]
// entries: ascending columns per row, the sum, and the sum of absolute products.
int oracle_spgemm_fill(int64_t a_rows, int64_t a_cols, const int64_t* a_row_ptr,
                       const int32_t* a_col, const void* a_val, int64_t b_rows, int64_t b_cols,
                       const int64_t* b_row_ptr, const int32_t* b_col, const void* b_val,
                       int dtype, int64_t r0, int64_t r1, int threads,
                       const int64_t* local_row_ptr, int32_t* out_col, double* out_val,
                       double* out_abs) {
  if (a_cols != b_rows || r0 < 0 || r1 > a_rows || r0 > r1) return -1;
  CsrView A{a_rows, a_cols, a_row_ptr, a_col, a_val}, B{b_rows, b_cols, b_row_ptr, b_col, b_val};
  if (dtype == 0)
    return run_rows<float, double>(A, B, r0, r1, threads, 1, nullptr, local_row_ptr, out_col,
                                   out_val, out_abs);
  if (dtype == 1)
    return run_rows<double, long double>(A, B, r0, r1, threads, 1, nullptr, local_row_ptr,
                                         out_col, out_val, out_abs);
  return -2;
}

}  // extern "C"
