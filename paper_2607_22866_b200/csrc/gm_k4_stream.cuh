// K4 — expansion straight into the first level's children (see gm_k4_direct.cuh for where a product goes), built
// around the copy engine: the B200 form of Algorithm 4's "contiguous B-row copies scaled by a".
//
// A heavy row's products are long contiguous pieces of rows of B.  The tile-per-block kernels read them with
// ordinary loads, a handful in flight per thread, spent about fifty warp instructions per 32 products on finding
// segments and destinations, and took 18 us per tile: bound by latency and issue slots, at 40 % of the write
// bandwidth.  Here every warp is a pipeline of its own:
//   * the flattened product space of the batch is cut into one contiguous range per warp (static partition, as
//     GroupRange in Algorithm 4); the warp walks the segments of its range, 32 segments' metadata at a time in
//     registers (one coalesced load per array, the next window requested a window ahead);
//   * every piece of a row of B is cut into slices of at most kStreamSlice elements; for each slice lane 0 asks
//     the copy engine (cp.async.bulk, completion counted by an mbarrier) for the slice's columns, its values and
//     the segment's record — the run start of every level-0 child plus the entry of A — into one of kStreamStages
//     ring stages of the warp's shared memory, several slices ahead of the one being consumed;
//   * consuming a slice is then all there is per product: two shared-memory loads, the child from the column, the
//     run start from the record, one multiply, two stores.
// Nothing waits on a global load in the steady state, and no block-wide barrier exists.
//
// Bulk copies need 16-byte aligned addresses and sizes, and a piece starts anywhere: the copy takes the enclosing
// aligned span (up to three elements of the neighbouring rows of B on either side, never past the last aligned
// element of B's arrays) and the consumer skips what is not the piece's; the last one to three elements of B's
// arrays, when a piece needs them, are fetched with plain loads.
// Every wait is bounded (mbar_wait_bounded): when one gives up the warp records kDevTimeout, gives the copies it
// still has in flight a second, long, bounded chance to land and returns.  A negative spin_limit is the test hook
// for that path: copies are announced to the barrier but withheld.
#pragma once
#include "gm_common.cuh"

namespace gm {

// Sizing.  A warp on its own issues an instruction every four to five cycles (measured: four warps per SM ran at
// 20 % issue utilisation with no stall to speak of), so the SM needs a dozen or more of these pipelines, which
// bounds a warp's ring to about 16 KB; and what a slice costs beyond its products (walking to it, three copy
// requests, a barrier) is about a hundred instructions, so segments shorter than kShortSegment products — nearly
// half of the segments of a power-law product, with 3 % of its products — are left to a kernel of their own
// (k4_expand_short, one warp per segment, plain loads) and the walker steps over them.
#ifndef GM_STREAM_SLICE_F32
#define GM_STREAM_SLICE_F32 512
#endif
#ifndef GM_STREAM_SLICE_F64
#define GM_STREAM_SLICE_F64 256
#endif
#ifndef GM_STREAM_STAGES
#define GM_STREAM_STAGES 4
#endif
constexpr int kShortSegment = 128;
template <typename V> struct StreamSlice { static constexpr int value = sizeof(V) == 4 ? GM_STREAM_SLICE_F32 : GM_STREAM_SLICE_F64; };
constexpr int kStreamStages = GM_STREAM_STAGES;  // slices (and segment records) a warp has in flight
constexpr int kStreamWarps = 4;      // warps per block
constexpr int kRecExtra = 4;         // 32-bit words after the F run starts of a segment record (the entry of A)

// 32-bit words of a segment record: the F run starts (padded to whole 16-byte units) and the entry of A
__host__ __device__ inline int stream_rec_words(int F) { return ((F + 3) & ~3) + kRecExtra; }
__host__ __device__ inline size_t stream_warp_smem_bytes(int F, int val_bytes) {
  const int slice = val_bytes == 4 ? GM_STREAM_SLICE_F32 : GM_STREAM_SLICE_F64;
  // (a multiple of 128 bytes, so that every warp's stages start on the 16-byte boundaries bulk copies need)
  const size_t b = static_cast<size_t>(kStreamStages) *
                   (static_cast<size_t>(slice) * (4 + val_bytes) + static_cast<size_t>(stream_rec_words(F)) * 4 + 32 + 8);
  return (b + 127) & ~static_cast<size_t>(127);
}

// rec[s * stream_rec_words(F) + c] = H[s * F + c] + R[row(s) * F + c]  (run start of child c for the segment's products,
// minus the index in the row of B), and the segment's entry of A behind the (padded) run starts
template <typename V>
__global__ void k_seg_records(const u32* __restrict__ H, const u32* __restrict__ R, const int32_t* __restrict__ seg_hrow,
                              const i64* __restrict__ seg_j, const V* __restrict__ a_val, i64 seg0, i64 n_seg_b, i64 h0, int F,
                              u32* __restrict__ rec) {
  const int stride = stream_rec_words(F);
  const int fpad = stride - kRecExtra;
  const i64 n = n_seg_b * stride;
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 s = i / stride;
    const int c = static_cast<int>(i - s * stride);
    u32 out = 0;
    if (c < F) {
      out = H[s * F + c] + R[(static_cast<i64>(seg_hrow[seg0 + s]) - h0) * F + c];
    } else if (c >= fpad) {
      const V a = a_val[seg_j[seg0 + s]];
      if (sizeof(V) == 4) {
        if (c == fpad) out = __float_as_uint(static_cast<float>(a));
      } else {
        const u64 bits = static_cast<u64>(__double_as_longlong(static_cast<double>(a)));
        if (c == fpad) out = static_cast<u32>(bits);
        if (c == fpad + 1) out = static_cast<u32>(bits >> 32);
      }
    }
    rec[i] = out;
  }
}

struct __align__(16) SliceDesc {
  i64 ca;       // position in B's arrays of stage position 0 (a multiple of four)
  int v0, v1;   // the piece's elements inside the slice: stage positions [v0, v1)
  int i_base;   // index in the row of B of stage position 0 (can be -3 .. -1 at the start of a row)
  int n_plain;  // how many of the piece's last elements lie past the last aligned element of B's arrays (0 .. 3)
  int rec_slot; // which of the warp's record slots holds the segment's record
  int pad;
};

template <typename V>
__global__ void __launch_bounds__(kStreamWarps * 32) k4_expand_stream(
    const i64* __restrict__ seg_off, const i64* __restrict__ seg_bstart, i64 n_seg_all,  // segment table of all heavy rows
    const TileMeta* __restrict__ warp_meta,  // per warp range: the segment that holds its first product
    const int32_t* __restrict__ b_col, const V* __restrict__ b_val, i64 nnz_b,
    i64 elem0, i64 n_elems, i64 per_warp,   // first product of the batch (global heavy numbering), batch size, range per warp
    i64 seg0, const u32* __restrict__ rec, int F, int shift,
    int32_t* __restrict__ y_col, V* __restrict__ y_val, int spin_limit, int* __restrict__ err) {
  extern __shared__ __align__(128) unsigned char smem_stream_raw[];
  constexpr int NS = kStreamStages;
  constexpr int SL = StreamSlice<V>::value;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int rec_words = stream_rec_words(F);
  const int fpad = rec_words - kRecExtra;
  // this warp's shared memory: [values NS x SL][columns NS x SL][records NS x rec_words][descriptors NS][barriers NS]
  unsigned char* base = smem_stream_raw + static_cast<size_t>(warp) * stream_warp_smem_bytes(F, sizeof(V));
  V* st_val = reinterpret_cast<V*>(base);
  int32_t* st_col = reinterpret_cast<int32_t*>(st_val + NS * SL);
  u32* st_rec = reinterpret_cast<u32*>(st_col + NS * SL);
  SliceDesc* st_desc = reinterpret_cast<SliceDesc*>(st_rec + NS * rec_words);
  u64* st_bar = reinterpret_cast<u64*>(st_desc + NS);

  const i64 wid = static_cast<i64>(blockIdx.x) * kStreamWarps + warp;
  const i64 p_lo = wid * per_warp;
  if (p_lo >= n_elems) return;
  const i64 g_lo = elem0 + p_lo;
  const i64 g_hi = elem0 + min(n_elems, p_lo + per_warp);
  const bool withhold = spin_limit < 0;
  const int wait_limit = withhold ? -spin_limit : spin_limit;
  const u32 fmask = static_cast<u32>(F - 1);
  const i64 nnz_b_al = nnz_b & ~i64{3};  // bulk copies stay below this element

  if (lane == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(&st_bar[s], 1);
    mbar_fence_init();
  }
  __syncwarp();

  // ---- segment window: lane l holds segment w_base + l
  i64 w_base = warp_meta[wid].first;
  auto load_window = [&](i64 b, i64& so, i64& so1, i64& bs) {
    const i64 idx = min(b + lane, n_seg_all - 1);
    so = seg_off[idx];
    so1 = seg_off[idx + 1];
    bs = seg_bstart[idx];
  };
  i64 w_so, w_so1, w_bs, n_so, n_so1, n_bs;
  load_window(w_base, w_so, w_so1, w_bs);
  load_window(w_base + 32, n_so, n_so1, n_bs);

  // ---- walker over the pieces and slices of the range (uniform across the warp)
  i64 sg = w_base;     // current segment
  i64 pos = g_lo;      // first product not yet cut into slices
  i64 cur = 0, a_end = 0, src_lo = 0, src_hi = 0, bstart_seg = 0, seg_cur = 0;  // current piece (cur >= a_end: none)
  auto next_slice = [&](SliceDesc& d, i64& ca, int& n_copy, i64& seg_of) -> bool {
    while (cur >= a_end) {
      if (pos >= g_hi) return false;
      if (sg >= w_base + 32) {  // next window (requested a window ago), and request the one after it
        w_base += 32;
        w_so = n_so; w_so1 = n_so1; w_bs = n_bs;
        load_window(w_base + 32, n_so, n_so1, n_bs);
      }
      const int j = static_cast<int>(sg - w_base);
      const i64 so = __shfl_sync(0xffffffffu, static_cast<long long>(w_so), j);
      const i64 so1 = __shfl_sync(0xffffffffu, static_cast<long long>(w_so1), j);
      const i64 bs = __shfl_sync(0xffffffffu, static_cast<long long>(w_bs), j);
      const i64 pe = min(g_hi, so1);
      if (pe <= pos) { ++sg; continue; }  // a segment without products (empty row of B)
      if (so1 - so < kShortSegment) {     // short segments belong to k4_expand_short, whole
        pos = pe;
        if (pe == so1) ++sg;
        continue;
      }
      src_lo = bs + (pos - so);
      src_hi = bs + (pe - so);
      cur = src_lo & ~i64{3};
      a_end = (src_hi + 3) & ~i64{3};
      bstart_seg = bs;
      seg_cur = sg;
      pos = pe;
      if (pe == so1) ++sg;
    }
    ca = cur;
    const i64 cb = min(a_end, cur + SL);
    cur = cb;
    const i64 lo = max(src_lo, ca), hi = min(src_hi, cb);
    d.ca = ca;
    d.v0 = static_cast<int>(lo - ca);
    d.v1 = static_cast<int>(hi - ca);
    d.i_base = static_cast<int>(ca - bstart_seg);
    const i64 copy_end = min(cb, nnz_b_al);
    n_copy = copy_end > ca ? static_cast<int>(copy_end - ca) : 0;
    d.n_plain = hi > max(copy_end, ca) ? static_cast<int>(hi - max(copy_end, ca)) : 0;
    seg_of = seg_cur;
    return true;
  };

  int n_fly = 0;                 // slices issued and not yet consumed
  int st_i = 0, st_c = 0;        // ring stage of the next slice to issue / to consume
  u32 par_c = 0;                 // barrier parity of the next use of every stage, bit per stage (consumer's view)
  i64 rec_seg = -1;              // segment whose record was copied last, and the slot it went to
  int rec_slot = NS - 1;
  bool more = true;
  for (;;) {
    // ---- issue: keep the ring full
    while (more && n_fly < NS) {
      SliceDesc d;
      i64 ca, seg_of;
      int n_copy;
      more = next_slice(d, ca, n_copy, seg_of);
      if (!more) break;
      // A record is copied when the segment changes, into the next record slot: the slices that used that slot's
      // previous record were issued at least NS slices ago and have been consumed.
      const bool new_rec = seg_of != rec_seg;
      if (new_rec) {
        rec_seg = seg_of;
        rec_slot = rec_slot + 1 == NS ? 0 : rec_slot + 1;
      }
      d.rec_slot = rec_slot;
      if (lane == 0) {
        st_desc[st_i] = d;
        const u32 bytes = static_cast<u32>(n_copy) * static_cast<u32>(4 + sizeof(V)) + (new_rec ? static_cast<u32>(rec_words) * 4u : 0u);
        mbar_arrive_expect_tx(&st_bar[st_i], bytes);
        if (!withhold) {
          if (n_copy > 0) {
            bulk_g2s(st_col + st_i * SL, b_col + ca, static_cast<u32>(n_copy) * 4u, &st_bar[st_i]);
            bulk_g2s(st_val + st_i * SL, b_val + ca, static_cast<u32>(n_copy) * static_cast<u32>(sizeof(V)), &st_bar[st_i]);
          }
          if (new_rec)
            bulk_g2s(st_rec + rec_slot * rec_words, rec + (seg_of - seg0) * rec_words, static_cast<u32>(rec_words) * 4u, &st_bar[st_i]);
        }
      }
      st_i = st_i + 1 == NS ? 0 : st_i + 1;
      ++n_fly;
    }
    if (n_fly == 0) break;
    __syncwarp();  // descriptors written by lane 0
    // ---- consume the oldest slice
    const int st = st_c;
    if (!mbar_wait_bounded(&st_bar[st], (par_c >> st) & 1u, wait_limit)) {
      dev_set_error(err, kDevTimeout);
      if (!withhold) {  // the other copies in flight still target this warp's shared memory
        int s2 = st;
        for (int k = 0; k < n_fly; ++k) {
          mbar_wait_bounded(&st_bar[s2], (par_c >> s2) & 1u, kCopySpinLimit);
          s2 = s2 + 1 == NS ? 0 : s2 + 1;
        }
      }
      return;
    }
    par_c ^= 1u << st;
    const SliceDesc d = st_desc[st];
    const int32_t* sc = st_col + st * SL;
    const V* sv = st_val + st * SL;
    if (d.n_plain > 0) {  // the last elements of B's arrays, which no aligned copy may cover: plain loads (rare)
      if (lane < d.n_plain) {
        const int e = d.v1 - d.n_plain + lane;
        st_col[st * SL + e] = b_col[d.ca + e];
        st_val[st * SL + e] = b_val[d.ca + e];
      }
      __syncwarp();
    }
    const u32* rc = st_rec + d.rec_slot * rec_words;
    V a;
    if (sizeof(V) == 4) a = static_cast<V>(__uint_as_float(rc[fpad]));
    else a = static_cast<V>(__longlong_as_double(static_cast<long long>(static_cast<u64>(rc[fpad]) | (static_cast<u64>(rc[fpad + 1]) << 32))));
    const u32 ib = static_cast<u32>(d.i_base);
    int e0 = d.v0 + lane;
    for (; e0 + 96 < d.v1; e0 += 128) {  // four full rows of 32 products: no bounds checks
      int32_t col[4];
      V val[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { col[u] = sc[e0 + u * 32]; val[u] = sv[e0 + u * 32]; }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const u32 dst = rc[(static_cast<u32>(col[u]) >> shift) & fmask] + ib + static_cast<u32>(e0 + u * 32);
        y_col[dst] = col[u];
        y_val[dst] = a * val[u];
      }
    }
    for (; e0 < d.v1; e0 += 32) {
      const int32_t c1 = sc[e0];
      const u32 dst = rc[(static_cast<u32>(c1) >> shift) & fmask] + ib + static_cast<u32>(e0);
      y_col[dst] = c1;
      y_val[dst] = a * sv[e0];
    }
    __syncwarp();  // the stage is free for the next copy only when every lane has read it
    st_c = st_c + 1 == NS ? 0 : st_c + 1;
    --n_fly;
  }
}

// Segments of fewer than kShortSegment products: one warp per segment, plain loads (a row of B of a few dozen
// entries is one or two coalesced requests), the run starts of the segment's record in a register per lane.
template <typename V>
__global__ void __launch_bounds__(256) k4_expand_short(
    const i64* __restrict__ seg_off, const i64* __restrict__ seg_bstart, const int32_t* __restrict__ b_col,
    const V* __restrict__ b_val, i64 seg0, i64 n_seg_b, const u32* __restrict__ rec, int F, int shift,
    int32_t* __restrict__ y_col, V* __restrict__ y_val) {
  const int lane = threadIdx.x & 31;
  const int rec_words = stream_rec_words(F);
  const int fpad = rec_words - kRecExtra;
  const u32 fmask = static_cast<u32>(F - 1);
  const i64 n_warps = static_cast<i64>(gridDim.x) * (blockDim.x >> 5);
  for (i64 s = static_cast<i64>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); s < n_seg_b; s += n_warps) {
    const i64 so = seg_off[seg0 + s];
    const int len = static_cast<int>(min(seg_off[seg0 + s + 1] - so, static_cast<i64>(kShortSegment)));
    if (len <= 0 || seg_off[seg0 + s + 1] - so >= kShortSegment) continue;
    const i64 bs = seg_bstart[seg0 + s];
    const u32* rc = rec + s * rec_words;
    V a;
    if (sizeof(V) == 4) a = static_cast<V>(__uint_as_float(rc[fpad]));
    else a = static_cast<V>(__longlong_as_double(static_cast<long long>(static_cast<u64>(rc[fpad]) | (static_cast<u64>(rc[fpad + 1]) << 32))));
    for (int e = lane; e < len; e += 32) {
      const int32_t c1 = b_col[bs + e];
      const u32 dst = rc[(static_cast<u32>(c1) >> shift) & fmask] + static_cast<u32>(e);
      y_col[dst] = c1;
      y_val[dst] = a * b_val[bs + e];
    }
  }
}

}  // namespace gm
