// K6 — chunk accumulation (the dense accumulator of Section III-E applied to the rows of
// C^_reord): every final chunk (heavy row h, chunk c) owns the W consecutive columns
// [c*W, (c+1)*W), so its products are summed into a W-entry dense accumulator in shared memory; a
// bitmap records which columns received a product (structural zeros are kept), a block-wide prefix
// sum over the bitmap words gives every occupied column its rank, and the chunk is written to C in
// ascending column order.
//
// One pass, no symbolic twin: the position of a chunk in C is only known once every earlier chunk has been
// counted, so the kernel writes the compacted chunk *in place*, over the start of the chunk's own (already
// consumed) products in the staging buffer — the output of a chunk never has more entries than its input —
// and reports the entry count.  A prefix sum over those counts gives C.rowPtr, and the gather kernel below
// moves the compacted chunks to   C.rowPtr[row] + (entries of the row's earlier chunks).
//
// B200 design.  The chunks of a batch lie back to back in the staging buffer, so the kernel does
// not fetch chunk by chunk: the element space is cut into equal segments (static flattened
// partition, as in Algorithms 4 and 5), persistent blocks claim segments with a ticket, and each
// block *streams* its segment through a ring of shared-memory tiles filled by bulk asynchronous
// copies (cp.async.bulk + mbarrier), independent of chunk boundaries.  A chunk boundary only
// triggers a flush of the accumulator.  The flush cleans what it writes, so a chunk costs time
// proportional to its products and its output, not to W.  All waits are bounded.
#pragma once
#include "gm_common.cuh"

namespace gm {

// A block of BT threads streams tiles of PT * BT products (PT = 2 or 4 per thread) and keeps the offsets of BT
// chunks at a time in shared memory.  Few threads with several products each: the per-tile and per-chunk
// control code is executed by every warp, so a wide block multiplies it.
constexpr i64 kAccSegment = i64{1} << 18;  // elements per ticket
constexpr int kAccSpinLimit = 1 << 24;  // polls of an mbarrier before the kernel gives up

__device__ __forceinline__ u32 smem_u32(const void* p) { return static_cast<u32>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(u64* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(u64* bar, u32 bytes) {
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

// Number of ring stages that fit next to the accumulator of a block of `bt` threads.
__host__ __device__ inline int acc_ring_stages(size_t smem_budget, int W, int val_bytes, bool numeric, int bt, int pt) {
  const size_t fixed = static_cast<size_t>(W / 32) * 12 + (numeric ? static_cast<size_t>(W) * val_bytes : 0) +
                       static_cast<size_t>(bt) * 4 + 256;
  const size_t stage = static_cast<size_t>(pt * bt) * (4 + (numeric ? val_bytes : 0));
  if (smem_budget <= fixed) return 0;
  size_t s = (smem_budget - fixed) / stage;
  return static_cast<int>(s > 8 ? 8 : s);
}
__host__ __device__ inline size_t acc_stream_smem_bytes(int W, int val_bytes, bool numeric, int stages, int bt, int pt) {
  return static_cast<size_t>(W / 32) * 12 + (numeric ? static_cast<size_t>(W) * val_bytes : 0) +
         static_cast<size_t>(bt) * 4 +
         static_cast<size_t>(stages) * pt * bt * (4 + (numeric ? val_bytes : 0)) + 256;
}

// seg_first[s] = first chunk whose start offset is >= s * kAccSegment (s = 0..n_segs).
__global__ void k6_prepare(const i64* __restrict__ chunk_off, i64 n_chunks, i64 n_segs, i64* __restrict__ seg_first) {
  const i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i <= n_segs) {
    const i64 target = i * kAccSegment;
    i64 lo = 0, hi = n_chunks;  // first k in [0, n_chunks] with chunk_off[k] >= target
    while (lo < hi) {
      const i64 mid = (lo + hi) >> 1;
      if (chunk_off[mid] >= target) hi = mid; else lo = mid + 1;
    }
    seg_first[i] = lo;
  }
}

// Position in C of every chunk's first entry, once C.rowPtr of the batch's rows is known.
__global__ void k6_chunk_bases(const i64* __restrict__ chunk_nnz_off, i64 n_chunks, int log2_chunks_per_row,
                               const int32_t* __restrict__ x_heavy, i64 h0, const i64* __restrict__ c_row_ptr,
                               i64* __restrict__ chunk_base) {
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_chunks;
       i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 r = i >> log2_chunks_per_row;
    chunk_base[i] = c_row_ptr[x_heavy[h0 + r]] + (chunk_nnz_off[i] - chunk_nnz_off[r << log2_chunks_per_row]);
  }
}

// One product into the accumulator.  Measured on B200 (shared memory, 1024 threads per SM, products per clock
// per SM): native integer atomics 12; floating-point atomicAdd 3.7 on uniform columns and 2.0 when a quarter of
// the products hit 64 hot columns (a hand-written compare-and-swap loop was a third slower than the built-in); ranking equal columns first with a warp
// match (match.any) only 0.5 — so there is no warp-level deduplication here, and the bitmap is tested before
// it is set so that repeated columns cost a load instead of an atomic.
template <typename V, bool NUMERIC>
__device__ __forceinline__ void acc_add(bool valid, u32 cl, V v, V* acc, u32* bitmap) {
  if (valid) {
    if constexpr (NUMERIC) atomicAdd(&acc[cl], v);
    const u32 bit = 1u << (cl & 31);
    if (!(bitmap[cl >> 5] & bit)) atomicOr(&bitmap[cl >> 5], bit);
  }
}

// Small chunks.  Going through the block-wide accumulator costs every chunk a few thousand cycles of barriers,
// prefix sums and dependent shared-memory round trips whatever it holds, and most chunks of a power-law product
// hold few products.  Chunks of at most kAccSmallChunk products are therefore handled before the streaming
// kernel runs, by ONE warp each and with no block-wide step, so that every SM works on dozens of them at a
// time: the warp loads the chunk, sorts (column, position) keys packed into one word in registers (bitonic
// network of ascending-only comparators: one shuffle and one min/max per key and step), adds up runs of equal
// columns in the original order and writes the result over the chunk's start in the staging buffer.  This
// is the paper's separate branch for light chunks (Section III-A), with a sort where the paper uses a hash
// table.  The streaming kernel skips these chunks.
#ifndef GM_SMALL_PER_LANE
#define GM_SMALL_PER_LANE 16
#endif
constexpr int kSmallMaxPerLane = GM_SMALL_PER_LANE;
constexpr int kAccSmallChunk = 32 * kSmallMaxPerLane;
constexpr int kSmallIdxBits = kSmallMaxPerLane == 32 ? 10 : (kSmallMaxPerLane == 16 ? 9 : 8);  // position of a product inside its chunk
constexpr int kSmallWarps = 4;            // warps per block of the small-chunk kernel
#ifndef GM_ACC_LIST_MIN
#define GM_ACC_LIST_MIN 512
#endif
constexpr u32 kAccListMin = GM_ACC_LIST_MIN;  // chunks with more entries than this balance their dense words over the block

// Sorts 32 * K packed keys, K per lane, element e = r * 32 + lane in key[r]; ascending in e afterwards.
// Steps whose partner sits in another lane are the same instruction sequence for every step width, so they run
// as loops over the width; only the steps that pair registers are unrolled.  (Fully unrolled, the networks of
// all K together did not fit the instruction cache, and the warps of a block run different K.)
template <int K>
__device__ __forceinline__ void warp_sort_keys(u32 (&key)[K], int lane) {
  auto lane_step = [&](int mask, bool lower) {  // partner: same register, lane ^ mask; the lower lane keeps the smaller key
#pragma unroll
    for (int r = 0; r < K; ++r) {
      const u32 o = __shfl_xor_sync(0xffffffffu, key[r], mask);
      key[r] = lower ? min(key[r], o) : max(key[r], o);
    }
  };
  // merges inside one register row (k = 2 .. 32): first step partner e ^ (k - 1), then e ^ j for j = k/4 .. 1
#pragma unroll 1
  for (int k = 2; k <= 32; k <<= 1) {
    lane_step(k - 1, (lane & (k >> 1)) == 0);
#pragma unroll 1
    for (int j = k >> 2; j > 0; j >>= 1) lane_step(j, (lane & j) == 0);
  }
  // merges across register rows (k = 64 .. 32 K)
#pragma unroll
  for (int k = 64; k <= 32 * K; k <<= 1) {
    const int rm = k / 32 - 1;  // first step: partner register r ^ rm, partner lane lane ^ 31
#pragma unroll
    for (int r = 0; r < K; ++r) {
      if ((r ^ rm) > r) {
        const u32 a = key[r], b = key[r ^ rm];
        const u32 oa = __shfl_xor_sync(0xffffffffu, b, 31);
        const u32 ob = __shfl_xor_sync(0xffffffffu, a, 31);
        key[r] = min(a, oa);
        key[r ^ rm] = max(b, ob);
      }
    }
#pragma unroll
    for (int j = k >> 2; j >= 32; j >>= 1) {  // partner in the same lane
      const int rj = j / 32;
#pragma unroll
      for (int r = 0; r < K; ++r) {
        if ((r & rj) == 0) {
          const u32 a = key[r], b = key[r | rj];
          key[r] = min(a, b);
          key[r | rj] = max(a, b);
        }
      }
    }
#pragma unroll 1
    for (int j = 16; j > 0; j >>= 1) lane_step(j, (lane & j) == 0);
  }
}

// One small chunk by one warp.  s_key / s_val: 32 * K entries of this warp's shared memory.
template <typename V, int K>
__device__ __forceinline__ int small_chunk(int32_t* col, V* val, int n, u32 wmask, u32* s_key, V* s_val,
                                           u32* nnz_out) {
  const int lane = threadIdx.x & 31;
  u32 key[K];
  int32_t c_first = 0;
#pragma unroll
  for (int r = 0; r < K; ++r) {
    const int e = r * 32 + lane;
    key[r] = 0xffffffffu;  // padding sorts to the end
    if (e < n) {
      const int32_t c = col[e];
      if (e == 0) c_first = c;
      key[r] = ((static_cast<u32>(c) & wmask) << kSmallIdxBits) | static_cast<u32>(e);
      s_val[e] = val[e];
    }
  }
  const u32 col_base = static_cast<u32>(__shfl_sync(0xffffffffu, c_first, 0)) & ~wmask;
  warp_sort_keys<K>(key, lane);
#pragma unroll
  for (int r = 0; r < K; ++r) s_key[r * 32 + lane] = key[r];
  __syncwarp();
  // runs of equal columns: the lane that owns a run's first element adds the run up and writes it
  int base = 0;
#pragma unroll
  for (int r = 0; r < K; ++r) {
    if (r * 32 < n) {  // warp-uniform
      const int e = r * 32 + lane;
      const u32 c = key[r] >> kSmallIdxBits;
      const bool head = e < n && (e == 0 || (s_key[e - 1] >> kSmallIdxBits) != c);
      const u32 heads = __ballot_sync(0xffffffffu, head);
      if (head) {
        V sum = s_val[key[r] & ((1u << kSmallIdxBits) - 1u)];
        for (int q = e + 1; q < n; ++q) {
          const u32 kq = s_key[q];
          if ((kq >> kSmallIdxBits) != c) break;
          sum += s_val[kq & ((1u << kSmallIdxBits) - 1u)];
        }
        const int p = base + __popc(heads & lanemask_lt());
        col[p] = static_cast<int32_t>(col_base | c);
        val[p] = sum;
      }
      base += __popc(heads);
    }
  }
  if (lane == 0) *nnz_out = static_cast<u32>(base);
  __syncwarp();  // the warp's shared memory is reused by its next chunk
  return base;
}

template <typename V>
__global__ void __launch_bounds__(kSmallWarps * 32) k6_small_chunks(
    int32_t* x_col, V* x_val, const i64* __restrict__ chunk_off, i64 n_chunks, int W, int small_max,
    u32* __restrict__ chunk_nnz,
    u64* __restrict__ totals) {  // [0] += products, [1] += entries of the chunks handled here (statistics)
  __shared__ u32 s_key[kSmallWarps][32 * kSmallMaxPerLane];
  __shared__ V s_val[kSmallWarps][32 * kSmallMaxPerLane];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const u32 wmask = static_cast<u32>(W - 1);
  const i64 n_groups = (n_chunks + 31) >> 5;
  __shared__ u64 s_sum[kSmallWarps][2];  // statistics, kept out of the registers of the sort
  if (lane == 0) { s_sum[w][0] = 0; s_sum[w][1] = 0; }
  // a warp looks at 32 consecutive chunks at a time and works through the small ones among them
  for (i64 g = static_cast<i64>(blockIdx.x) * kSmallWarps + w; g < n_groups; g += static_cast<i64>(gridDim.x) * kSmallWarps) {
    const i64 k = (g << 5) + lane;
    i64 cs = 0;
    int cn = 0;
    if (k < n_chunks) {
      cs = chunk_off[k];
      cn = static_cast<int>(min(chunk_off[k + 1] - cs, static_cast<i64>(INT_MAX)));
    }
    u32 todo = __ballot_sync(0xffffffffu, cn > 0 && cn <= small_max);
    while (todo) {
      const int src = __ffs(todo) - 1;
      todo &= todo - 1;
      const i64 s0 = __shfl_sync(0xffffffffu, cs, src);
      const int n = __shfl_sync(0xffffffffu, cn, src);
      int32_t* col = x_col + s0;
      V* val = x_val + s0;
      u32* out = &chunk_nnz[(g << 5) + src];
      int m;
      if (n <= 32) m = small_chunk<V, 1>(col, val, n, wmask, s_key[w], s_val[w], out);
      else if (n <= 64) m = small_chunk<V, 2>(col, val, n, wmask, s_key[w], s_val[w], out);
      else if (n <= 128) m = small_chunk<V, 4>(col, val, n, wmask, s_key[w], s_val[w], out);
      else if (kSmallMaxPerLane == 8 || n <= 256) m = small_chunk<V, 8>(col, val, n, wmask, s_key[w], s_val[w], out);
      else if (kSmallMaxPerLane == 16 || n <= 512) m = small_chunk<V, (kSmallMaxPerLane >= 16 ? 16 : 8)>(col, val, n, wmask, s_key[w], s_val[w], out);
      else m = small_chunk<V, kSmallMaxPerLane>(col, val, n, wmask, s_key[w], s_val[w], out);
      if (lane == 0) { s_sum[w][0] += static_cast<u64>(n); s_sum[w][1] += static_cast<u64>(m); }
    }
  }
  if (lane == 0 && s_sum[w][0]) {
    atomicAdd(&totals[0], s_sum[w][0]);
    atomicAdd(&totals[1], s_sum[w][1]);
  }
}

template <typename V, bool NUMERIC, int BT, int PT>
__global__ void __launch_bounds__(BT, 1) k6_accumulate(
    int32_t* x_col, V* x_val,            // staging buffer: products in, compacted chunks out (in place)
    const i64* __restrict__ chunk_off,   // n_chunks + 1 batch-relative element offsets
    i64 n_chunks, const i64* __restrict__ seg_first, i64 n_segs, int* __restrict__ ticket,
    int log2_chunks_per_row, int W, int stages, int small_max,
    u32* __restrict__ chunk_nnz,         // out, pre-zeroed: entries per chunk (empty chunks are never visited)
    int* __restrict__ err) {
  extern __shared__ __align__(128) unsigned char smem_acc_raw[];
  constexpr int kAccTile = PT * BT;
  constexpr int kAccMetaCap = BT;
  const int n_words = W >> 5;
  // layout: [ring cols][ring vals][acc][dense-word list][bitmap][chunk offsets of the metadata window]
  int32_t* r_col = reinterpret_cast<int32_t*>(smem_acc_raw);
  V* r_val = reinterpret_cast<V*>(smem_acc_raw + static_cast<size_t>(stages) * kAccTile * 4);
  unsigned char* after_ring = smem_acc_raw + static_cast<size_t>(stages) * kAccTile * (4 + (NUMERIC ? sizeof(V) : 0));
  V* acc = reinterpret_cast<V*>(after_ring);
  // n_words entries {bits | word index, prefix}; W * sizeof(V) is a multiple of 128, so the list is 8-byte aligned
  u64* dense_list = reinterpret_cast<u64*>(after_ring + (NUMERIC ? static_cast<size_t>(W) * sizeof(V) : 0));
  u32* bitmap = reinterpret_cast<u32*>(dense_list + n_words);
  int* m_off = reinterpret_cast<int*>(bitmap + n_words);
  __shared__ u64 full_bar[8];
  __shared__ u32 s_scan[33];
  __shared__ i64 s_seg[2];
  __shared__ int s_abort;
  __shared__ int s_dense_n[2];  // used by alternate chunks, so that resetting one needs no barrier of its own

  const int tid = threadIdx.x, lane = tid & 31;
  const u32 wmask = static_cast<u32>(W - 1);
  constexpr u32 kStageBytesCol = kAccTile * 4;
  constexpr u32 kStageBytesVal = NUMERIC ? kAccTile * sizeof(V) : 0;
  constexpr int kPerThread = kAccTile / BT;  // elements of a full tile per thread
  constexpr int kWarps = BT / 32;
  static_assert(kAccTile % BT == 0, "tile must be a multiple of the block");
  // the flush gives every thread wpt consecutive bitmap words (wpt is a power of two, at most 32)
  const int wpt = n_words > BT ? n_words / BT : 1;

  if (NUMERIC)
    for (int s = tid; s < W; s += BT) acc[s] = V(0);
  for (int w = tid; w < n_words; w += BT) bitmap[w] = 0u;
  if (tid == 0) {
    for (int s = 0; s < stages; ++s) mbar_init(&full_bar[s], 1);
    s_abort = 0;
    s_dense_n[0] = 0;
    s_dense_n[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  u32 phase_bits = 0;  // bit s = parity to wait for on stage s
  int dpar = 0;        // which dense-word counter the current chunk uses

  for (;;) {
    if (tid == 0) {
      const int s = atomicAdd(ticket, 1);
      s_seg[0] = s < n_segs ? seg_first[s] : -1;
      s_seg[1] = s < n_segs ? seg_first[s + 1] : -1;
    }
    __syncthreads();
    const i64 k_first = s_seg[0], k_end = s_seg[1];
    __syncthreads();
    if (k_first < 0) break;
    if (k_first >= k_end) continue;
    const i64 lo = chunk_off[k_first], hi = chunk_off[k_end];
    if (lo >= hi) continue;
    const i64 lo_al = lo & ~i64{3};  // 16-byte aligned start of the stream
    const int n_tiles = static_cast<int>((hi - lo_al + kAccTile - 1) / kAccTile);
    const int32_t* g_col = x_col + lo_al;
    const V* g_val = x_val + lo_al;

    auto issue = [&](int j, int st) {  // thread 0 only
      const size_t g = static_cast<size_t>(j) * kAccTile;
      mbar_expect_tx(&full_bar[st], kStageBytesCol + kStageBytesVal);
      bulk_g2s(r_col + st * kAccTile, g_col + g, kStageBytesCol, &full_bar[st]);
      if (NUMERIC) bulk_g2s(r_val + st * kAccTile, g_val + g, kStageBytesVal, &full_bar[st]);
    };
    if (tid == 0)
      for (int j = 0; j < n_tiles && j < stages; ++j) issue(j, j);

    // chunk metadata of the segment, refilled every kAccMetaCap chunks
    i64 m0 = k_first;          // first chunk held in the metadata window
    int kw = 0;                // current chunk = m0 + kw
    const u32 crow_mask = (1u << log2_chunks_per_row) - 1u;
    u32 crow = static_cast<u32>(k_first) & crow_mask;  // index of the current chunk inside its row (kept in step with kw)
    const int log2W = 31 - __clz(W);
    auto load_meta = [&]() {
      for (int i = tid; i < kAccMetaCap; i += BT) {
        const i64 kk = m0 + i;
        if (kk <= k_end) m_off[i] = static_cast<int>(chunk_off[kk] - lo_al);
      }
    };
    load_meta();
    __syncthreads();

    int pos = static_cast<int>(lo - lo_al);      // stream-relative position of the next element
    const int end = static_cast<int>(hi - lo_al);
    bool aborted = false;
    int st = 0;

    for (int j = 0; j < n_tiles; ++j) {
      // ---- wait for the tile (bounded, with back-off so that the poll does not eat issue slots)
      {
        const u32 par = (phase_bits >> st) & 1u;
        int spins = 0;
        while (!mbar_try_wait(&full_bar[st], par)) {
          __nanosleep(40);
          if (*static_cast<volatile int*>(&s_abort)) break;  // somebody gave up: no tile will be issued any more
          if (++spins > kAccSpinLimit) { s_abort = 1; break; }
        }
        phase_bits ^= (1u << st);
      }
      const int tile_lo = j * kAccTile;
      const int tile_hi = min(end, tile_lo + kAccTile);
      int32_t* tc = r_col + st * kAccTile - tile_lo;
      V* tv = r_val + st * kAccTile - tile_lo;
      while (pos < tile_hi) {
        // make sure the current chunk and its end are inside the metadata window
        if (kw + 33 >= kAccMetaCap) {  // the look-ahead below reads 32 chunks
          __syncthreads();
          m0 += kw;
          kw = 0;
          load_meta();
          __syncthreads();
        }
        const int ce = m_off[kw + 1];
        if (ce - m_off[kw] <= small_max) {
          // an empty chunk, or a small one that the small-chunk kernel has dealt with: how many of the next 32
          // chunks are like that?  Every warp evaluates the same shared-memory metadata, so the answer is
          // uniform without a barrier.
          const i64 kc = m0 + kw + lane;
          const bool skip = kc < k_end && m_off[kw + lane + 1] - m_off[kw + lane] <= small_max;
          const u32 not_skip = ~__ballot_sync(0xffffffffu, skip);
          const int run = not_skip ? __ffs(not_skip) - 1 : 32;  // >= 1
          kw += run;
          crow = (crow + static_cast<u32>(run)) & crow_mask;
          pos = m_off[kw];
          continue;
        }
        const int sub_hi = min(tile_hi, ce);
        const u32 col_base = crow << log2W;
        if (!s_abort) {
          for (int base = pos; base < sub_hi; base += BT * kPerThread) {
            // slots of this warp that still hold products of the sub-range (warp-uniform): a short sub-range
            // must not pay for the whole unrolled body
            const int wq = base + (tid & ~31);
            const int nu = wq >= sub_hi ? 0 : min(kPerThread, (sub_hi - wq + BT - 1) / BT);
            if (nu == kPerThread && wq + (kPerThread - 1) * BT + 32 <= sub_hi) {
              u32 cl[kPerThread];
              V v[kPerThread];
#pragma unroll
              for (int u = 0; u < kPerThread; ++u) {
                const int q = base + u * BT + tid;
                cl[u] = static_cast<u32>(tc[q]) & wmask;
                if (NUMERIC) v[u] = tv[q];
              }
#pragma unroll
              for (int u = 0; u < kPerThread; ++u) acc_add<V, NUMERIC>(true, cl[u], v[u], acc, bitmap);
            } else {
              for (int u = 0; u < nu; ++u) {
                const int q = base + u * BT + tid;
                if (q < sub_hi) acc_add<V, NUMERIC>(true, static_cast<u32>(tc[q]) & wmask, NUMERIC ? tv[q] : V(0), acc, bitmap);
              }
            }
          }
        }
        pos = sub_hi;
        if (pos < ce) break;  // chunk continues in the next tile
        // ---- chunk complete: flush
        __syncthreads();
        const int wb = tid * wpt;
        const bool warp_has_words = (tid & ~31) * wpt < n_words;  // warp-uniform
        u32 pc = 0;
        u32 word0 = 0;  // the thread's first (for wpt == 1: only) word stays in a register
        if (wb < n_words) {
          word0 = bitmap[wb];
          pc = __popc(word0);
          for (int i = 1; i < wpt; ++i) pc += __popc(bitmap[wb + i]);
        }
        // Block-wide exclusive prefix with one barrier: every warp publishes its sum, then adds up the sums of
        // the warps before it (and all of them, for the chunk's entry count) on its own.
        const u32 inc = warp_inclusive_scan(pc);
        if (lane == 31) s_scan[tid >> 5] = inc;
        __syncthreads();
        const u32 wsum = lane < kWarps ? s_scan[lane] : 0u;
        const u32 total = __reduce_add_sync(0xffffffffu, wsum);
        u32 ex = __reduce_add_sync(0xffffffffu, lane < (tid >> 5) ? wsum : 0u) + inc - pc;
        if (tid == 0) chunk_nnz[m0 + kw] = total;
        {
          // in place: the chunk's products [m_off[kw], ce) are all in shared memory or consumed by now
          int32_t* const c_col = x_col + lo_al + m_off[kw];
          V* const c_val = x_val + lo_al + m_off[kw];
          // Words with few bits are written by their owner.  In a chunk with many entries the dense words
          // cluster at the low end (hub columns), i.e. in the first warps, so they go to a list that all warps
          // then share out evenly; there the 32 lanes of a warp write one word at a time.  A chunk with few
          // entries cannot be far out of balance and skips the list and its barrier.
          const bool use_list = total > kAccListMin;  // block-uniform
          if (warp_has_words) {
            for (int i = 0; i < wpt; ++i) {
              const u32 word = i == 0 ? word0 : (wb + i < n_words ? bitmap[wb + i] : 0u);
              const u32 wpc = __popc(word);
              const bool dense = use_list && wpc > 4;
              if (use_list) {
                const u32 dmask = __ballot_sync(0xffffffffu, dense);
                if (dmask) {
                  int lbase = 0;
                  if (lane == 0) lbase = atomicAdd(&s_dense_n[dpar], __popc(dmask));
                  lbase = __shfl_sync(0xffffffffu, lbase, 0);
                  if (dense)  // {bits, word index, prefix} in one entry: the write-out needs a single load
                    dense_list[lbase + __popc(dmask & lanemask_lt())] =
                        (static_cast<u64>((static_cast<u32>(wb + i) << 16) | ex) << 32) | word;
                }
              }
              if (!dense && wpc) {
                u32 wbits = word;
                u32 p = ex;
                while (wbits) {
                  const int b = __ffs(wbits) - 1;
                  wbits &= wbits - 1;
                  const int slot = ((wb + i) << 5) + b;
                  c_col[p] = static_cast<int32_t>(col_base + slot);
                  c_val[p] = acc[slot];
                  acc[slot] = V(0);
                  ++p;
                }
              }
              if (wpc) bitmap[wb + i] = 0u;  // a listed word's bits travel in its list entry
              ex += wpc;
            }
          }
          if (use_list) {
            __syncthreads();
            const int n_dense = s_dense_n[dpar];
            auto emit = [&](u64 e) {
              const u32 word = static_cast<u32>(e);
              if ((word >> lane) & 1u) {
                const u32 hi32 = static_cast<u32>(e >> 32);
                const int slot = static_cast<int>((hi32 >> 16) << 5) + lane;
                const u32 p = (hi32 & 0xffffu) + __popc(word & lanemask_lt());
                c_col[p] = static_cast<int32_t>(col_base + slot);
                c_val[p] = acc[slot];
                acc[slot] = V(0);
              }
            };
            for (int i = tid >> 5; i < n_dense; i += 2 * kWarps) {  // two words in flight per warp
              const u64 e0 = dense_list[i];
              const bool two = i + kWarps < n_dense;
              const u64 e1 = two ? dense_list[i + kWarps] : 0ull;
              emit(e0);
              emit(e1);
            }
            if (tid == 0) s_dense_n[dpar ^ 1] = 0;  // next list's counter: last read two barriers ago
            dpar ^= 1;
          }
        }
        __syncthreads();
        ++kw;
        crow = (crow + 1u) & crow_mask;
      }
      // ---- the stage is free again once every warp has finished the tile.  Only the warp that refills it has to
      // wait for that: the others announce that they are done (named barrier 1 + stage) and go on to the next
      // tile, whose data is in another stage.  A warp cannot arrive twice on a barrier before it has completed:
      // its next use of this stage waits for the refill, which is issued after the barrier.
      // (Only for the block that has an SM to itself: the named barriers of narrower blocks, several per SM, would
      // not fit the SM's sixteen.)
      if constexpr (BT == 1024) {
        if (j + stages < n_tiles) {  // (uniform)
          if (tid < 32) {
            asm volatile("bar.sync %0, %1;" ::"r"(1 + st), "r"(BT) : "memory");
            if (tid == 0 && !*static_cast<volatile int*>(&s_abort)) issue(j + stages, st);
          } else {
            asm volatile("bar.arrive %0, %1;" ::"r"(1 + st), "r"(BT) : "memory");
          }
        }
      } else {
        __syncthreads();
        if (tid == 0 && j + stages < n_tiles && !*static_cast<volatile int*>(&s_abort)) issue(j + stages, st);
      }
      st = (st + 1 == stages) ? 0 : st + 1;
    }
    __syncthreads();  // every warp is through the segment
    aborted = s_abort != 0;
    if (aborted) {
      // Tiles that were issued but not consumed still target this block's shared memory: give each a
      // bounded chance to land before the block exits (its barrier answers at once if it already did).
      if (tid == 0) {
        dev_set_error(err, kDevTimeout);
        for (int s2 = 0; s2 < stages; ++s2) {
          int spins = 0;
          while (!mbar_try_wait(&full_bar[s2], (phase_bits >> s2) & 1u) && ++spins < (1 << 20)) {
          }
        }
      }
      __syncthreads();
      return;
    }
  }
}

}  // namespace gm
