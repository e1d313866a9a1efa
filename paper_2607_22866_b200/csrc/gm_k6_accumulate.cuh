// K6 — chunk accumulation (the dense accumulator of Section III-E applied to the rows of
// C^_reord): every final chunk (heavy row h, chunk c) owns the W consecutive columns
// [c*W, (c+1)*W), so its products are summed into a W-entry dense accumulator in shared memory; a
// bitmap records which columns received a product (structural zeros are kept), a block-wide prefix
// sum over the bitmap words gives every occupied column its rank, and the chunk is written to C in
// ascending column order at   C.rowPtr[row] + (entries of the row's earlier chunks) + rank.
//   symbolic launch: bitmap only -> entries per chunk (feeds C.rowPtr)
//   numeric launch : values + bitmap -> C.col / C.val
// Blocks are persistent and take chunks in a strided order; the accumulator is cleaned while it is
// written out, so a chunk costs time proportional to its products and its output, not to W.
#pragma once
#include "gm_common.cuh"

namespace gm {

template <typename V, bool NUMERIC, int BT>
__global__ void __launch_bounds__(BT) k6_accumulate(
    const int32_t* __restrict__ x_col, const V* __restrict__ x_val,
    const i64* __restrict__ chunk_off,   // n_chunks + 1, batch-relative element offsets
    i64 n_chunks, int log2_chunks_per_row, int W, i64 c_cols,
    u32* __restrict__ chunk_nnz,                     // symbolic out
    const i64* __restrict__ chunk_nnz_off,           // numeric in: exclusive scan of chunk_nnz (n_chunks + 1)
    const int32_t* __restrict__ x_heavy, i64 h0,     // heavy rows of the batch: original row = x_heavy[h0 + r]
    const i64* __restrict__ c_row_ptr, int32_t* __restrict__ c_col, V* __restrict__ c_val, i64 c_capacity,
    int* __restrict__ err) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_words = W >> 5;
  V* acc = reinterpret_cast<V*>(smem_raw);
  u32* bitmap = reinterpret_cast<u32*>(smem_raw + (NUMERIC ? static_cast<size_t>(W) * sizeof(V) : 0));
  u32* word_prefix = bitmap + n_words;
  __shared__ u32 s_scan[33];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kWarps = BT / 32;
  const u32 wmask = static_cast<u32>(W - 1);

  if (NUMERIC)
    for (int s = tid; s < W; s += BT) acc[s] = V(0);
  for (int w = tid; w < n_words; w += BT) bitmap[w] = 0u;
  __syncthreads();

  const int words_per_thread = (n_words + BT - 1) / BT;
  for (i64 k = blockIdx.x; k < n_chunks; k += gridDim.x) {
    const i64 e0 = chunk_off[k], e1 = chunk_off[k + 1];
    if (e0 == e1) {
      if (!NUMERIC && tid == 0) chunk_nnz[k] = 0u;
      continue;
    }
    const i64 chunk = k & ((i64{1} << log2_chunks_per_row) - 1);
    const i64 col_base = chunk * W;
    // ---- accumulate
    for (i64 e = e0 + tid; e < e1; e += BT) {
      const u32 c = static_cast<u32>(x_col[e]);
      const u32 cl = c & wmask;
      if (static_cast<i64>(c) - cl != col_base) { dev_set_error(err, kDevBadChunk); continue; }
      if (NUMERIC) atomicAdd(&acc[cl], x_val[e]);
      const u32 bit = 1u << (cl & 31);
      if (!(bitmap[cl >> 5] & bit)) atomicOr(&bitmap[cl >> 5], bit);
    }
    __syncthreads();
    // ---- rank the occupied columns: popcount per bitmap word, block-wide exclusive scan
    u32 local = 0;
    const int wb = tid * words_per_thread;
    for (int i = 0; i < words_per_thread; ++i)
      if (wb + i < n_words) local += __popc(bitmap[wb + i]);
    u32 total;
    u32 ex = block_exclusive_scan(local, s_scan, &total);
    if constexpr (!NUMERIC) {
      for (int i = 0; i < words_per_thread; ++i)
        if (wb + i < n_words) bitmap[wb + i] = 0u;
      if (tid == 0) chunk_nnz[k] = total;
      __syncthreads();
      continue;
    }
    if constexpr (NUMERIC) {
    for (int i = 0; i < words_per_thread; ++i) {
      if (wb + i < n_words) {
        word_prefix[wb + i] = ex;
        ex += __popc(bitmap[wb + i]);
      }
    }
    __syncthreads();
    // ---- write out in column order and clean the accumulator
    const i64 row_in_batch = k >> log2_chunks_per_row;
    const i64 row = x_heavy[h0 + row_in_batch];
    const i64 out0 = c_row_ptr[row] + (chunk_nnz_off[k] - chunk_nnz_off[row_in_batch << log2_chunks_per_row]);
    const bool fits = out0 + total <= c_capacity;
    if (!fits) dev_set_error(err, kDevCapacity);
    for (int w = warp; w < n_words; w += kWarps) {
      const u32 word = bitmap[w];
      if (word == 0u) continue;
      if ((word >> lane) & 1u) {
        const int slot = (w << 5) + lane;
        if (fits) {
          const i64 pos = out0 + word_prefix[w] + __popc(word & lanemask_lt());
          c_col[pos] = static_cast<int32_t>(col_base + slot);
          c_val[pos] = acc[slot];
        }
        acc[slot] = V(0);
      }
      __syncwarp();
      if (lane == 0) bitmap[w] = 0u;
    }
    __syncthreads();
    }
  }
}

}  // namespace gm
