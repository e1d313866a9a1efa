// K6 — chunk accumulation (the dense accumulator of Section III-E applied to the rows of
// C^_reord): every final chunk (heavy row h, chunk c) owns the W consecutive columns
// [c*W, (c+1)*W), so its products can be summed in shared memory; a bitmap records which columns
// received a product (structural zeros are kept), a prefix sum over the bitmap words gives every
// occupied column its rank, and the chunk comes out in ascending column order.
//
// One pass over the staging buffer, no symbolic twin: the position of a chunk in C is only known once
// every earlier chunk has been counted, so each kernel writes the compacted chunk *in place*, over the
// start of the chunk's own (already consumed) products — the output of a chunk never has more entries
// than its input — and reports the entry count.  A prefix sum over those counts gives C.rowPtr, and the
// gather kernel moves the compacted chunks to  C.rowPtr[row] + (entries of the row's earlier chunks).
//
// B200 design.  The chunks of a power-law product span five orders of magnitude (most hold a few dozen
// products, a few hold millions), and what a chunk costs beyond its products is the width of the team
// that has to synchronise for it.  So the chunks are binned by size (the binning of Section III-E) and
// every bin gets a team of its own width:
//   k6_classify      one thread per chunk: lists of the mid-size and of the big chunks
//   k6_small_chunks  n <= 128 products (an option, at most 512): one warp per chunk, register sort, no barrier at all
//   k6_mid_chunks    n <= a few thousand: one 128-thread block per chunk, several blocks per SM.  Symbolic
//                    then numeric as in Algorithm 3: pass 1 sets the column bitmap, a prefix sum over the
//                    bitmap words ranks the columns, pass 2 adds every product to a *compact* array of the
//                    chunk's entries and notes its column in a second one (their size is bounded by the chunk's
//                    products, not by W, which is what lets many chunks share an SM), the write-out is a plain
//                    copy of the two; the second pass re-reads the chunk from L2
//   k6_accumulate    the rest: one 1024-thread block per SM with the dense W-column accumulator, products
//                    streamed from HBM with 16-byte loads one tile ahead in registers, one flush per chunk
// The mid-size and the big kernel are persistent grids that take chunks from a list with an atomic ticket, the
// small one shares the chunk table out statically; nothing waits on anything but block-wide barriers.
#pragma once
#include "gm_common.cuh"

namespace gm {

// Where the chunks that left the multisplit hierarchy early live.  A final chunk's tag (0: it went through every
// level) is 1 + the level whose pass left it behind; per tag, one bit says whether that level's input was the
// other staging buffer than the one the last level wrote, and five bits give log2 of the columns the chunk spans.
struct ExitTags {
  u32 alt_bits = 0;
  u64 span_pack = 0;
  __host__ __device__ bool alt(int tag) const { return (alt_bits >> tag) & 1u; }
  __host__ __device__ int span_bits(int tag) const { return static_cast<int>((span_pack >> (5 * tag)) & 31u); }
  void set(int tag, bool other_buffer, int bits) {
    if (other_buffer) alt_bits |= 1u << tag;
    span_pack |= static_cast<u64>(bits) << (5 * tag);
  }
};

constexpr int kMidThreads = 128;        // threads of one mid-chunk team
constexpr int kHugeChunk = 1 << 16;     // big chunks with more products than this are handed out first

// Lists for the mid and big kernels.  Chunk ids are batch-relative and fit 32 bits.  Big chunks above kHugeChunk
// are appended from the front of big_list, the others from its back, so that a ticket order front-to-back gives
// the long ones out first (fewer blocks idle at the end of the launch).
// counters: [0] mid chunks, [1] huge chunks, [2] other big chunks, [3] ticket of the mid kernel, [4] ticket of
// the big kernel (all zeroed by the host before the launch).
__global__ void k6_classify(const i64* __restrict__ chunk_off, i64 n_chunks, int small_max, int mid_max,
                            int32_t* __restrict__ mid_list, int32_t* __restrict__ big_list, int* __restrict__ counters) {
  const int lane = threadIdx.x & 31;
  for (i64 k0 = (static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x) & ~i64{31}; k0 < n_chunks;
       k0 += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 k = k0 + lane;
    i64 n = 0;
    if (k < n_chunks) n = chunk_off[k + 1] - chunk_off[k];
    const bool mid = n > small_max && n <= mid_max;
    const bool huge = n > small_max && !mid && n > kHugeChunk;
    const bool big = n > small_max && !mid && !huge;
    const u32 m_mid = __ballot_sync(0xffffffffu, mid);
    const u32 m_huge = __ballot_sync(0xffffffffu, huge);
    const u32 m_big = __ballot_sync(0xffffffffu, big);
    int b_mid = 0, b_huge = 0, b_big = 0;
    if (lane == 0) {
      if (m_mid) b_mid = atomicAdd(&counters[0], __popc(m_mid));
      if (m_huge) b_huge = atomicAdd(&counters[1], __popc(m_huge));
      if (m_big) b_big = atomicAdd(&counters[2], __popc(m_big));
    }
    b_mid = __shfl_sync(0xffffffffu, b_mid, 0);
    b_huge = __shfl_sync(0xffffffffu, b_huge, 0);
    b_big = __shfl_sync(0xffffffffu, b_big, 0);
    if (mid) mid_list[b_mid + __popc(m_mid & lanemask_lt())] = static_cast<int32_t>(k);
    if (huge) big_list[b_huge + __popc(m_huge & lanemask_lt())] = static_cast<int32_t>(k);
    if (big) big_list[n_chunks - 1 - (b_big + __popc(m_big & lanemask_lt()))] = static_cast<int32_t>(k);
  }
}

// Debug net (plan option validate_inputs): every product that reaches the accumulate kernels must lie in the W
// columns its chunk owns.  One warp per chunk; a violation sets kDevBadChunk (the kernels themselves mask the
// column and would fold a misplaced product into the wrong entry silently).
// Chunks that left the hierarchy early (tag != 0, see ExitTags) own the columns of all the final chunks they stand for.
__global__ void k6_validate_chunks(const int32_t* __restrict__ x_col, const i64* __restrict__ chunk_off, i64 n_chunks,
                                   int log2_chunks_per_row, int W, i64 n_cols, int* __restrict__ err,
                                   const unsigned char* __restrict__ tags, const int32_t* __restrict__ x_col_alt,
                                   ExitTags xt) {
  const int lane = threadIdx.x & 31;
  const int log2W = 31 - __clz(W);
  const u32 crow_mask = (1u << log2_chunks_per_row) - 1u;
  const i64 n_warps = static_cast<i64>(gridDim.x) * (blockDim.x >> 5);
  for (i64 k = static_cast<i64>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); k < n_chunks; k += n_warps) {
    const int tag = tags ? tags[k] : 0;
    const int32_t* col = tag && xt.alt(tag) ? x_col_alt : x_col;
    const int bits = tag ? xt.span_bits(tag) : log2W;  // columns the chunk owns: 2^bits
    const u32 want = (static_cast<u32>(k) & crow_mask) >> (bits - log2W);
    bool bad = false;
    for (i64 q = chunk_off[k] + lane; q < chunk_off[k + 1]; q += 32) {
      const int32_t c = col[q];
      bad |= c < 0 || c >= n_cols || (static_cast<u32>(c) >> bits) != want ||
             (static_cast<u32>(k) & ((1u << (bits - log2W)) - 1u)) != 0;  // an early chunk's products sit in its first slot
    }
    if (bad) dev_set_error(err, kDevBadChunk);
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

// Small chunks.  Going through the block-wide accumulator costs every chunk a few thousand cycles of barriers,
// prefix sums and dependent shared-memory round trips whatever it holds, and most chunks of a power-law product
// hold few products.  Chunks of at most small_max (<= kAccSmallChunk) products are therefore handled before the streaming
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
constexpr int kAccSmallChunk = 32 * kSmallMaxPerLane;  // largest chunk the one-warp sort can take
// Default hand-over to the mid-size kernel.  The sort costs n log^2 n; measured on B200 (R-MAT scale 20 fp32 / scale 21
// fp64, small + mid kernels together, ms per step) with chunks up to 64 / 96 / 128 / 192 / 256 products sorted:
// 42.4 / 41.4 / 41.0 / 41.1 / 42.8 and 81.7 / 77.4 / 75.2 / 75.5 / 76.5.
constexpr int kAccSmallDefault = 128;
constexpr int kSmallIdxBits = kSmallMaxPerLane == 32 ? 10 : (kSmallMaxPerLane == 16 ? 9 : 8);  // position of a product inside its chunk
constexpr int kSmallWarps = 4;            // warps per block of the small-chunk kernel
// Eight blocks per SM: without the bound the compiler takes 105-120 registers and four blocks fit; measured on R-MAT
// scale 20 fp32 / scale 21 fp64, ms of this kernel with room for 6 / 7 / 8 blocks: 10.0 / 9.9 / 10.1 and
// 44.0 / 43.6 / 41.6.
constexpr int kSmallBlocksPerSm = 8;

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
__global__ void __launch_bounds__(kSmallWarps * 32, kSmallBlocksPerSm) k6_small_chunks(
    int32_t* x_col, V* x_val, const i64* __restrict__ chunk_off, i64 n_chunks, int W, int small_max,
    u32* __restrict__ chunk_nnz,
    u64* __restrict__ totals,  // [0] += products, [1] += entries of the chunks handled here (statistics)
    const unsigned char* __restrict__ tags,  // per chunk, or NULL: != 0 for chunks that left the hierarchy early
    int32_t* x_col_alt, V* x_val_alt, ExitTags xt) {
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
    int cn = 0, ctag = 0;
    if (k < n_chunks) {
      cs = chunk_off[k];
      cn = static_cast<int>(min(chunk_off[k + 1] - cs, static_cast<i64>(INT_MAX)));
      if (tags) ctag = tags[k];
    }
    u32 todo = __ballot_sync(0xffffffffu, cn > 0 && cn <= small_max);
    // (Requesting the next chunk's first products before the current chunk is sorted was tried: no gain at 64
    // registers, and the extra live state spilled in the fp64 kernel, 42 -> 60 ms on R-MAT scale 21.)
    while (todo) {
      const int src = __ffs(todo) - 1;
      todo &= todo - 1;
      const i64 s0 = __shfl_sync(0xffffffffu, cs, src);
      const int n = __shfl_sync(0xffffffffu, cn, src);
      const int tag = __shfl_sync(0xffffffffu, ctag, src);
      // an early chunk lies in the buffer it was left in and is sorted over all the columns it spans
      const bool alt = tag && xt.alt(tag);
      int32_t* col = (alt ? x_col_alt : x_col) + s0;
      V* val = (alt ? x_val_alt : x_val) + s0;
      const u32 wm = tag ? (1u << xt.span_bits(tag)) - 1u : wmask;
      u32* out = &chunk_nnz[(g << 5) + src];
      int m;
      if (n <= 32) m = small_chunk<V, 1>(col, val, n, wm, s_key[w], s_val[w], out);
      else if (n <= 64) m = small_chunk<V, 2>(col, val, n, wm, s_key[w], s_val[w], out);
      else if (n <= 128) m = small_chunk<V, 4>(col, val, n, wm, s_key[w], s_val[w], out);
      else if (kSmallMaxPerLane == 8 || n <= 256) m = small_chunk<V, 8>(col, val, n, wm, s_key[w], s_val[w], out);
      else if (kSmallMaxPerLane == 16 || n <= 512) m = small_chunk<V, (kSmallMaxPerLane >= 16 ? 16 : 8)>(col, val, n, wm, s_key[w], s_val[w], out);
      else m = small_chunk<V, kSmallMaxPerLane>(col, val, n, wm, s_key[w], s_val[w], out);
      if (lane == 0) { s_sum[w][0] += static_cast<u64>(n); s_sum[w][1] += static_cast<u64>(m); }
    }
  }
  if (lane == 0 && s_sum[w][0]) {
    atomicAdd(&totals[0], s_sum[w][0]);
    atomicAdd(&totals[1], s_sum[w][1]);
  }
}


// ---------------------------------------------------------------------------------------------------------
// Mid-size chunks: one block of kMidThreads threads per chunk, symbolic pass then numeric pass.
// Shared memory: bitmap (W/32 words) | rank of every word's first entry (16 bits each) | the chunk's values,
// compact (mid_max entries) | the chunk's columns, compact (16 bits each: W <= 65536).  In the scan a thread owns
// consecutive bitmap words and moves them with 16-byte accesses.
// ---------------------------------------------------------------------------------------------------------
// Products a thread holds per tile.  The unrolled slots are executed whether a chunk fills them or not, and most
// chunks of this class are small: measured on R-MAT scale 20 fp32 / scale 21 fp64, ms per step of this kernel with
// 8 / 4 / 2 slots: 39.9 / 37.6 / 44.7 and 48.1 / 41.6 / 47.3.
constexpr int kMidPer = 4;
constexpr int kMidTile = kMidThreads * kMidPer;     // 512: chunks up to this size are read from HBM once

inline size_t mid_smem_bytes(int W, int val_bytes, int mid_max) {
  const size_t n_words = static_cast<size_t>(W) / 32;
  return ((n_words * 6 + 15) & ~size_t{15}) + static_cast<size_t>(mid_max) * (val_bytes + 2) + 64;
}

struct ChunkTask {
  i64 k;       // chunk (batch-relative), -1: no more work
  i64 lo, hi;  // its products in the staging buffer
};

// Work distribution: chunks are handed out by an atomic ticket over a list.  Getting from a ticket to the chunk's
// products is a chain of three dependent global accesses (ticket, list entry, chunk bounds: two microseconds
// end to end), and a block's barriers wait for the one thread that walks it.  So thread 0 keeps three tasks in
// flight, one step of the chain each: at the start of a chunk it *issues* the ticket of the task three ahead, the
// list read of the task two ahead and the bounds read of the next task, and it only touches the results when the
// chunk's own work is done, by which time they have arrived.
struct TaskPipe {
  int* ticket;
  int n_list, n_front;
  const int32_t* list;
  i64 list_flip;  // >= 0: list positions past n_front are read from the back (see k6_classify)
  const i64* chunk_off;
  int tk2 = 0;    // ticket of the task two ahead (arrived)
  i64 k1 = -1;    // chunk of the next task (arrived)
  int tk3 = 0;    // in flight during a chunk
  i64 k2 = -1, lo1 = 0, hi1 = 0;

  __device__ __forceinline__ i64 list_at(int t) const {
    if (t >= n_list) return -1;
    return (list_flip < 0 || t < n_front) ? list[t] : list[list_flip - (t - n_front)];
  }
  // fills `first` with the first task (blocking, once per block) and primes the pipe
  __device__ __forceinline__ void start(ChunkTask* first) {
    const int t0 = atomicAdd(ticket, 1);
    const int t1 = atomicAdd(ticket, 1);
    tk2 = atomicAdd(ticket, 1);
    const i64 k0 = list_at(t0);
    k1 = list_at(t1);
    ChunkTask task{k0, 0, 0};
    if (k0 >= 0) { task.lo = chunk_off[k0]; task.hi = chunk_off[k0 + 1]; }
    *first = task;
  }
  __device__ __forceinline__ void issue() {  // start of a chunk
    tk3 = atomicAdd(ticket, 1);
    k2 = list_at(tk2);
    if (k1 >= 0) { lo1 = chunk_off[k1]; hi1 = chunk_off[k1 + 1]; }
  }
  __device__ __forceinline__ void publish(ChunkTask* next) {  // when the chunk's products are done
    *next = ChunkTask{k1, lo1, hi1};
    k1 = k2;
    tk2 = tk3;
  }
};

template <typename V>
__global__ void __launch_bounds__(kMidThreads) k6_mid_chunks(
    int32_t* x_col, V* x_val,            // staging buffer: products in, compacted chunks out (in place)
    const i64* __restrict__ chunk_off, const int32_t* __restrict__ mid_list, int* __restrict__ counters,
    int log2_chunks_per_row, int W, int mid_max,
    u32* __restrict__ chunk_nnz,         // out: entries per chunk
    u64* __restrict__ totals) {          // [0] += products, [1] += entries of the chunks handled here (statistics)
  extern __shared__ __align__(16) unsigned char smem_mid_raw[];
  constexpr int T = kMidThreads;
  const int n_words = W >> 5;
  u32* bitmap = reinterpret_cast<u32*>(smem_mid_raw);                 // n_words
  unsigned short* wpre = reinterpret_cast<unsigned short*>(bitmap + n_words);  // n_words: rank of the word's first entry
  V* oval = reinterpret_cast<V*>(smem_mid_raw + ((static_cast<size_t>(n_words) * 6 + 15) & ~size_t{15}));
  unsigned short* ocol = reinterpret_cast<unsigned short*>(oval + mid_max);  // the entries' columns inside the chunk
  __shared__ u32 s_wsum[T / 32];
  __shared__ ChunkTask s_task[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const u32 wmask = static_cast<u32>(W - 1);
  const u32 crow_mask = (1u << log2_chunks_per_row) - 1u;
  const int log2W = 31 - __clz(W);
  // every thread owns wpt consecutive bitmap words in the scan (eight for W = 32768: two 16-byte accesses)
  const int wpt = n_words > T ? n_words / T : 1;
  const int wb = tid * wpt;
  const bool own = wb < n_words;

  for (int w = tid; w < n_words; w += T) bitmap[w] = 0u;
  for (int i = tid; i < mid_max; i += T) oval[i] = V(0);
  TaskPipe pipe{&counters[3], counters[0], 0, mid_list, -1, chunk_off};
  if (tid == 0) pipe.start(&s_task[0]);
  __syncthreads();
  u64 sum_n = 0, sum_m = 0;
  int par = 0;
  ChunkTask task = s_task[0];
  // first tile of the first chunk
  u32 c_reg[kMidPer];
  auto load_cols = [&](const ChunkTask& tk, int tile) {
#pragma unroll
    for (int u = 0; u < kMidPer; ++u) {
      const i64 q = tk.lo + static_cast<i64>(tile) * kMidTile + u * T + tid;
      c_reg[u] = q < tk.hi ? static_cast<u32>(x_col[q]) & wmask : 0xffffffffu;
    }
  };
  if (task.k >= 0) load_cols(task, 0);

  while (task.k >= 0) {
    const int n = static_cast<int>(task.hi - task.lo);
    int32_t* const col = x_col + task.lo;
    V* const val = x_val + task.lo;
    const u32 col_base = (static_cast<u32>(task.k) & crow_mask) << log2W;
    const int n_tiles = (n + kMidTile - 1) / kMidTile;
    if (tid == 0) pipe.issue();

    // ---- pass 1 (symbolic): mark the columns.  The values of the first tile are requested now, for pass 2.
    V v_reg[kMidPer];
#pragma unroll
    for (int u = 0; u < kMidPer; ++u) {
      const int q = u * T + tid;
      if (q < n) v_reg[u] = val[q];
    }
    for (int tile = 0;;) {
#pragma unroll
      for (int u = 0; u < kMidPer; ++u)
        if (c_reg[u] != 0xffffffffu) atomicOr(&bitmap[c_reg[u] >> 5], 1u << (c_reg[u] & 31));
      if (++tile >= n_tiles) break;
      load_cols(task, tile);
    }
    __syncthreads();
    // ---- ranks: exclusive prefix over the words' populations
    u32 pc = 0;
    uint4 b0 = make_uint4(0, 0, 0, 0), b1 = b0;  // the usual case: eight words per thread
    if (own) {
      if (wpt == 8) {
        b0 = *reinterpret_cast<const uint4*>(bitmap + wb);
        b1 = *reinterpret_cast<const uint4*>(bitmap + wb + 4);
        pc = __popc(b0.x) + __popc(b0.y) + __popc(b0.z) + __popc(b0.w) + __popc(b1.x) + __popc(b1.y) + __popc(b1.z) + __popc(b1.w);
      } else {
        for (int i = 0; i < wpt; ++i) pc += __popc(bitmap[wb + i]);
      }
    }
    const u32 inc = warp_inclusive_scan(pc);
    if (lane == 31) s_wsum[warp] = inc;
    __syncthreads();
    u32 ex = inc - pc, total = 0;
#pragma unroll
    for (int w = 0; w < T / 32; ++w) {
      const u32 ws = s_wsum[w];
      if (w < warp) ex += ws;
      total += ws;
    }
    if (own) {
      if (wpt == 8) {
        u32 r0 = ex, r1 = r0 + __popc(b0.x), r2 = r1 + __popc(b0.y), r3 = r2 + __popc(b0.z), r4 = r3 + __popc(b0.w);
        u32 r5 = r4 + __popc(b1.x), r6 = r5 + __popc(b1.y), r7 = r6 + __popc(b1.z);
        *reinterpret_cast<uint4*>(wpre + wb) = make_uint4(r0 | (r1 << 16), r2 | (r3 << 16), r4 | (r5 << 16), r6 | (r7 << 16));
      } else {
        u32 run = ex;
        for (int i = 0; i < wpt; ++i) {
          wpre[wb + i] = static_cast<unsigned short>(run);
          run += __popc(bitmap[wb + i]);
        }
      }
    }
    if (n_tiles > 1) load_cols(task, 0);  // (a single tile is still in registers)
    __syncthreads();
    // ---- pass 2 (numeric): every product to the slot of its column's rank
    for (int tile = 0;;) {
#pragma unroll
      for (int u = 0; u < kMidPer; ++u) {
        const u32 c = c_reg[u];
        if (c != 0xffffffffu) {
          const u32 r = static_cast<u32>(wpre[c >> 5]) + __popc(bitmap[c >> 5] & ((1u << (c & 31)) - 1u));
          atomicAdd(&oval[r], v_reg[u]);
          ocol[r] = static_cast<unsigned short>(c);  // (every product of the column writes the same value)
        }
      }
      if (++tile >= n_tiles) break;
      load_cols(task, tile);
#pragma unroll
      for (int u = 0; u < kMidPer; ++u) {
        const int q = tile * kMidTile + u * T + tid;
        if (q < n) v_reg[u] = val[q];
      }
    }
    if (tid == 0) pipe.publish(&s_task[par ^ 1]);
    __syncthreads();
    // the next chunk's first columns are requested before this chunk is written out
    const ChunkTask next = s_task[par ^ 1];
    if (next.k >= 0) load_cols(next, 0);
    // ---- write-out in place: columns from the bitmap, values from the compact array.  The words are dealt out
    // round-robin here, not in the runs of the scan: the dense words of a power-law chunk are its first ones (hub
    // columns), and one thread writing all their columns held the block up (cycle counters on R-MAT scale 20: 10.5 k
    // of thread 0's 21 k cycles per chunk were this loop, 6 k of the last thread's).
    // ---- write-out in place, from the compact arrays: position i of the chunk's result takes column ocol[i] and
    // value oval[i], so the copy is coalesced and the same for every thread.  (Walking the bitmap instead, each
    // thread the columns of its own words, took 37.4 ms on R-MAT scale 20 where this takes 32.7: the dense words
    // of a power-law chunk are its first ones, and their owners' serial loops were most of the kernel's instructions.)
    if ((n_words & 3) == 0) {
      for (int w = tid * 4; w < n_words; w += T * 4) *reinterpret_cast<uint4*>(bitmap + w) = make_uint4(0, 0, 0, 0);
    } else {
      for (int w = tid; w < n_words; w += T) bitmap[w] = 0u;
    }
    for (int i = tid; i < static_cast<int>(total); i += T) {
      col[i] = static_cast<int32_t>(col_base + ocol[i]);
      val[i] = oval[i];
      oval[i] = V(0);
    }
    if (tid == 0) {
      chunk_nnz[task.k] = total;
      sum_n += static_cast<u64>(n);
      sum_m += total;
    }
    __syncthreads();
    task = next;
    par ^= 1;
  }
  if (tid == 0 && sum_n) {
    atomicAdd(&totals[0], sum_n);
    atomicAdd(&totals[1], sum_m);
  }
}

// ---------------------------------------------------------------------------------------------------------
// Big chunks: the dense accumulator.
//
// What binds this kernel is the shared-memory pipe (measured on B200 with a stream of products from HBM, products
// per clock per SM: integer atomics >= 3, limited by the stream; floating-point add 2.1 on uniform columns, 1.7
// with a bitmap test-and-set next to it), so a product costs one shared-memory operation, the floating-point atomic
// add, and only the first product of a column pays a second one:
//  * First-touch bitmap.  An idle slot holds -0.0, which is the identity of the addition, and a product that is a
//    zero of either sign is added as +0.0; a slot that received anything is then never -0.0 again (x + (-x) rounds
//    to +0.0).  The add returns the slot's old value, so the thread that sees -0.0 knows it was first and sets the
//    column's bit with an integer atomic: one per entry of C instead of a load per product, structural zeros kept.
//  * Bank spreading.  Columns of power-law matrices made by recursive quadrant picks have biased low bits
//    (bit = 0 three times out of four), so a quarter of all products would land in bank 0: measured 1.1
//    products per clock per SM, against 1.9 with the slot of a column rotated inside its group of 32 by a
//    hash of the group index (bitmap words likewise).  The rotation is undone when the flush walks a group.
// ---------------------------------------------------------------------------------------------------------
#ifndef GM_ACC_LIST_MIN
#define GM_ACC_LIST_MIN 512
#endif
constexpr u32 kAccListMin = GM_ACC_LIST_MIN;  // chunks with more entries than this balance their dense words over the block
#ifndef GM_ACC_DENSE_MIN
#define GM_ACC_DENSE_MIN 4
#endif
constexpr u32 kAccDenseMin = GM_ACC_DENSE_MIN;  // a group with more entries than this is written by a whole warp

inline size_t acc_smem_bytes_big(int W, int val_bytes) {
  const size_t n_words = static_cast<size_t>(W / 32);
  return static_cast<size_t>(W) * val_bytes + n_words * 8 + ((n_words + 31) & ~size_t{31}) * 4 + 64;
}

template <typename V> struct Vec4;
template <> struct Vec4<float> {
  float4 d;
  __device__ __forceinline__ void load(const float* p) { d = *reinterpret_cast<const float4*>(p); }
  __device__ __forceinline__ float get(int u) const { return u == 0 ? d.x : u == 1 ? d.y : u == 2 ? d.z : d.w; }
};
template <> struct Vec4<double> {
  double2 a, b;
  __device__ __forceinline__ void load(const double* p) {
    a = *reinterpret_cast<const double2*>(p);
    b = *reinterpret_cast<const double2*>(p + 2);
  }
  __device__ __forceinline__ double get(int u) const { return u == 0 ? a.x : u == 1 ? a.y : u == 2 ? b.x : b.y; }
};

__device__ __forceinline__ float acc_idle(float) { return __uint_as_float(0x80000000u); }
__device__ __forceinline__ double acc_idle(double) { return __longlong_as_double(static_cast<long long>(0x8000000000000000ull)); }
__device__ __forceinline__ bool acc_touched(float x) { return __float_as_uint(x) != 0x80000000u; }
__device__ __forceinline__ bool acc_touched(double x) { return static_cast<u64>(__double_as_longlong(x)) != 0x8000000000000000ull; }
__device__ __forceinline__ float plus_zero(float v) { return __fadd_rn(v, 0.0f); }   // -0.0 -> +0.0, everything else unchanged
__device__ __forceinline__ double plus_zero(double v) { return __dadd_rn(v, 0.0); }

// rotation of a group of 32 columns inside the accumulator
__device__ __forceinline__ u32 group_rot(u32 group) { return (group * 0x9E3779B1u) >> 27; }
__device__ __forceinline__ u32 acc_slot(u32 cl) { return (cl & ~31u) | ((cl + group_rot(cl >> 5)) & 31u); }

template <typename V, int BT>
__global__ void __launch_bounds__(BT, 1024 / BT) k6_accumulate(
    int32_t* x_col, V* x_val,            // staging buffer: products in, compacted chunks out (in place)
    const i64* __restrict__ chunk_off, i64 n_chunks, const int32_t* __restrict__ big_list, int* __restrict__ counters,
    int log2_chunks_per_row, int W,
    u32* __restrict__ chunk_nnz) {       // out: entries per chunk
  extern __shared__ __align__(128) unsigned char smem_acc_raw[];
  const int n_words = W >> 5;
  // layout: [acc][dense-word list][bitmap, whole groups of 32 words]
  V* acc = reinterpret_cast<V*>(smem_acc_raw);
  // n_words entries {bits | word index, prefix}; W * sizeof(V) is a multiple of 128, so the list is 8-byte aligned
  u64* dense_list = reinterpret_cast<u64*>(smem_acc_raw + static_cast<size_t>(W) * sizeof(V));
  u32* bitmap = reinterpret_cast<u32*>(dense_list + n_words);
  __shared__ u32 s_scan[33];
  __shared__ ChunkTask s_task[2];
  __shared__ int s_dense_n[2];  // used by alternate chunks, so that resetting one needs no barrier of its own

  constexpr int kWarps = BT / 32;
  constexpr int kTile = 4 * BT;  // products per step: four consecutive ones per thread, two 16-byte loads
  const int tid = threadIdx.x, lane = tid & 31;
  const u32 wmask = static_cast<u32>(W - 1);
  const u32 crow_mask = (1u << log2_chunks_per_row) - 1u;
  const int log2W = 31 - __clz(W);
  // the flush gives every thread wpt consecutive groups of 32 columns (wpt is a power of two, at most 32)
  const int wpt = n_words > BT ? n_words / BT : 1;
  const V idle = acc_idle(V(0));

  for (int s = tid; s < W; s += BT) acc[s] = idle;
  for (int w = tid; w < ((n_words + 31) & ~31); w += BT) bitmap[w] = 0u;
  TaskPipe pipe{&counters[4], counters[1] + counters[2], counters[1], big_list, n_chunks - 1, chunk_off};
  if (tid == 0) {
    s_dense_n[0] = 0;
    s_dense_n[1] = 0;
    pipe.start(&s_task[0]);
  }
  __syncthreads();
  int dpar = 0;  // which dense-word counter the current chunk uses
  int par = 0;
  ChunkTask task = s_task[0];
  // first tile of the first chunk: the stream starts at the 16-byte boundary below the chunk
  int4 c4 = make_int4(0, 0, 0, 0);
  Vec4<V> v4;
  auto load_tile = [&](i64 p, i64 hi) {
    if (p < hi) {
      c4 = *reinterpret_cast<const int4*>(x_col + p);
      v4.load(x_val + p);
    }
  };
  if (task.k >= 0) load_tile((task.lo & ~i64{3}) + static_cast<i64>(tid) * 4, task.hi);
  auto add = [&](u32 cl, V v) {
    const V old = atomicAdd(&acc[acc_slot(cl)], plus_zero(v));
    if (!acc_touched(old)) atomicOr(&bitmap[acc_slot(cl >> 5)], 1u << (cl & 31));  // first product of this column
  };

  while (task.k >= 0) {
    const i64 lo = task.lo, hi = task.hi;
    const u32 col_base = (static_cast<u32>(task.k) & crow_mask) << log2W;
    if (tid == 0) pipe.issue();

    // ---- accumulate: the tile after the current one is already on its way while this one is added
    for (i64 p = (lo & ~i64{3}) + static_cast<i64>(tid) * 4; p - static_cast<i64>(tid) * 4 < hi; p += kTile) {
      const int4 c = c4;
      const Vec4<V> v = v4;
      load_tile(p + kTile, hi);
      if (p >= lo && p + 3 < hi) {
        add(static_cast<u32>(c.x) & wmask, v.get(0));
        add(static_cast<u32>(c.y) & wmask, v.get(1));
        add(static_cast<u32>(c.z) & wmask, v.get(2));
        add(static_cast<u32>(c.w) & wmask, v.get(3));
      } else if (p < hi) {
        if (p >= lo) add(static_cast<u32>(c.x) & wmask, v.get(0));
        if (p + 1 >= lo && p + 1 < hi) add(static_cast<u32>(c.y) & wmask, v.get(1));
        if (p + 2 >= lo && p + 2 < hi) add(static_cast<u32>(c.z) & wmask, v.get(2));
        if (p + 3 >= lo && p + 3 < hi) add(static_cast<u32>(c.w) & wmask, v.get(3));
      }
    }
    // ---- chunk complete: flush
    __syncthreads();
    if (tid == 0) pipe.publish(&s_task[par ^ 1]);  // read after the next barrier
    const int wb = tid * wpt;
    const bool warp_has_words = (tid & ~31) * wpt < n_words;  // warp-uniform
    u32 pc = 0;
    u32 word0 = 0;  // the thread's first (for wpt == 1: only) word stays in a register
    if (wb < n_words) {
      word0 = bitmap[acc_slot(static_cast<u32>(wb))];
      pc = __popc(word0);
      for (int i = 1; i < wpt; ++i) pc += __popc(bitmap[acc_slot(static_cast<u32>(wb + i))]);
    }
    // Block-wide exclusive prefix with one barrier: every warp publishes its sum, then adds up the sums of
    // the warps before it (and all of them, for the chunk's entry count) on its own.
    const u32 inc = warp_inclusive_scan(pc);
    if (lane == 31) s_scan[tid >> 5] = inc;
    __syncthreads();
    const u32 wsum = lane < kWarps ? s_scan[lane] : 0u;
    const u32 total = __reduce_add_sync(0xffffffffu, wsum);
    u32 ex = __reduce_add_sync(0xffffffffu, lane < (tid >> 5) ? wsum : 0u) + inc - pc;
    if (tid == 0) chunk_nnz[task.k] = total;
    // the next chunk's first tile is requested before this chunk is written out
    const ChunkTask next = s_task[par ^ 1];
    if (next.k >= 0) load_tile((next.lo & ~i64{3}) + static_cast<i64>(tid) * 4, next.hi);
    {
      // in place: the chunk's products have all been consumed by now
      int32_t* const c_col = x_col + lo;
      V* const c_val = x_val + lo;
      // Groups with few entries are written by their owner.  In a chunk with many entries the dense groups
      // cluster at the low end (hub columns), i.e. in the first warps, so they go to a list that all warps
      // then share out evenly; there the 32 lanes of a warp write one group at a time.  A chunk with few
      // entries cannot be far out of balance and skips the list and its barrier.
      const bool use_list = total > kAccListMin;  // block-uniform
      if (warp_has_words) {
        for (int i = 0; i < wpt; ++i) {
          const u32 word = i == 0 ? word0 : (wb + i < n_words ? bitmap[acc_slot(static_cast<u32>(wb + i))] : 0u);
          const u32 wpc = __popc(word);
          const bool dense = use_list && wpc > kAccDenseMin;
          if (use_list) {
            const u32 dmask = __ballot_sync(0xffffffffu, dense);
            if (dmask) {
              int lbase = 0;
              if (lane == 0) lbase = atomicAdd(&s_dense_n[dpar], __popc(dmask));
              lbase = __shfl_sync(0xffffffffu, lbase, 0);
              if (dense)  // {bits, group index, prefix} in one entry: the write-out needs a single load
                dense_list[lbase + __popc(dmask & lanemask_lt())] =
                    (static_cast<u64>((static_cast<u32>(wb + i) << 16) | ex) << 32) | word;
            }
          }
          if (!dense && wpc) {
            u32 wbits = word;
            u32 p = ex;
            const u32 rot = group_rot(static_cast<u32>(wb + i));
            while (wbits) {
              const int b = __ffs(wbits) - 1;
              wbits &= wbits - 1;
              const int slot = ((wb + i) << 5) + static_cast<int>((static_cast<u32>(b) + rot) & 31u);
              c_col[p] = static_cast<int32_t>(col_base + ((wb + i) << 5) + b);
              c_val[p] = acc[slot];
              acc[slot] = idle;
              ++p;
            }
          }
          if (wpc) bitmap[acc_slot(static_cast<u32>(wb + i))] = 0u;  // a listed word's bits travel in its list entry
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
            const u32 grp = hi32 >> 16;
            const int slot = static_cast<int>((grp << 5) + ((static_cast<u32>(lane) + group_rot(grp)) & 31u));
            const u32 p = (hi32 & 0xffffu) + __popc(word & lanemask_lt());
            c_col[p] = static_cast<int32_t>(col_base + (grp << 5) + lane);
            c_val[p] = acc[slot];
            acc[slot] = idle;
          }
        };
        for (int i = tid >> 5; i < n_dense; i += 2 * kWarps) {  // two groups in flight per warp
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
    task = next;
    par ^= 1;
  }
}

}  // namespace gm
