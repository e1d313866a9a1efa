// K5 — one level of the hierarchical multisplit (Histogram + MultisplitKernel, Algorithm 5).
//
// Input: the staging buffer X, whose elements are grouped by *parent* (a heavy row at level 0, a
// chunk of the previous level afterwards); parent P owns [parent_off[P], parent_off[P+1]).
// Output: Y, where the elements of every parent are regrouped into F children by
//     child = (col >> shift) & (F - 1)
// and child (P, c) owns [child_off[P*F+c], child_off[P*F+c+1]) — the children tile their parent's
// range in order, so child_off is the plain exclusive scan of the (parent, child) count matrix.
//
// Both kernels use the same static partition of the flattened element space into tiles (GroupRange
// of Algorithm 5) and the same per-tile binning: bin = parent_in_tile * F + child, counted with a
// shared-memory integer atomic per element, whose return value is the element's rank inside its bin.
//   k5_histogram : adds the tile's bin counts to the global count matrix.
//   k5_multisplit: reserves the tile's share of every child's output range with one global atomic
//                  per non-empty bin (the cursor array starts as a copy of child_off), permutes
//                  the tile by bin in shared memory, and writes it out bin after bin, so each
//                  child receives a contiguous, coalesced run.
// A tile whose bins do not fit the shared table (very many tiny parents) falls back to one global
// atomic per element.
// When another level follows, the multisplit kernel also counts that level's (parent, child) bins while it writes
// its tile out — the column is in a register and the element's child, which is the next level's parent, is known
// — so deeper levels need no histogram pass over the staging buffer (4 bytes per product and a launch saved).
//
// Early exit (Algorithm 3: only heavy chunks recurse; Section III-A: light chunks take their own accumulation
// branch).  From the second level on, a parent that holds few products is not split any further: its products stay
// where they are, in the level's *input* buffer, and the parent's whole range is booked to its child 0 all the way
// down, so the chunk table keeps its regular (row, chunk) shape and the parent's range in either staging buffer
// stays its own.  k5_exit_flags marks such parents and rewrites their row of the count matrix; the multisplit
// kernel (EXIT) drops their products before ranking, loads no values for them and returns at once from a tile
// that holds nothing else.  The final chunks carry the tag of the level they left at, from which the accumulate and
// gather kernels know the buffer and the column span.
#pragma once
#include "gm_common.cuh"

namespace gm {

#ifndef GM_SPLIT_THREADS
#define GM_SPLIT_THREADS 512
#endif
constexpr int kSplitThreads = GM_SPLIT_THREADS;
constexpr int kSplitItems = 16;
constexpr int kSplitTile = kSplitThreads * kSplitItems;  // 8192 elements per block
constexpr int kSplitBinCap = 4 * kSplitThreads;           // bins (parent, child) per tile in shared memory
constexpr int kSplitParentCap = kSplitThreads / 2;        // parents per tile on the fast path

template <typename V>
constexpr size_t split_smem_bytes(bool multisplit) {
  // bins + parent offsets + parent starts (+ permuted columns and values + the next level's bins)
  size_t b = kSplitBinCap * 4 + (kSplitParentCap + 1) * 4 + kSplitParentCap * 4 + 64;
  if (multisplit) b += static_cast<size_t>(kSplitTile) * (4 + sizeof(V)) + kSplitBinCap * 4 + kSplitParentCap;
  return b;
}

struct SplitTileInfo {
  i64 p_lo;   // first parent touching the tile
  int n_par;  // parents touching the tile (including empty ones in between)
};

// Marks the parents of a level that leave the hierarchy here (tag != 0) and books their products to child 0.
// One thread per (parent, child).  tag_in: the parents' tags from the level before (NULL at the first level that
// can exit); a parent that left earlier keeps its tag.  counts: the level's count matrix, already filled.
__global__ void k5_exit_flags(const i64* __restrict__ parent_off, i64 n_parents, int log2F,
                              const unsigned char* __restrict__ tag_in, int exit_max, int level_tag,
                              u32* __restrict__ counts, unsigned char* __restrict__ parent_tag,
                              unsigned char* __restrict__ child_tag,
                              u64* __restrict__ totals) {  // [0] += products, [1] += parents that leave at this level,
                                                           // [2] += products that this level does not move
  const i64 n_child = n_parents << log2F;
  u64 prod = 0, par = 0, stay = 0;
  for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_child;
       i += static_cast<i64>(gridDim.x) * blockDim.x) {
    const i64 P = i >> log2F;
    const int c = static_cast<int>(i & ((i64{1} << log2F) - 1));
    const i64 n = parent_off[P + 1] - parent_off[P];
    int tag = tag_in ? tag_in[P] : 0;
    if (!tag && n <= exit_max) {
      tag = level_tag;
      if (c == 0 && n > 0) { prod += static_cast<u64>(n); ++par; }
    }
    if (tag && c == 0) stay += static_cast<u64>(n);
    child_tag[i] = static_cast<unsigned char>(tag);
    if (c == 0) parent_tag[P] = static_cast<unsigned char>(tag);
    if (tag) counts[i] = c == 0 ? static_cast<u32>(n) : 0u;
  }
  for (int o = 16; o > 0; o >>= 1) {
    prod += __shfl_xor_sync(0xffffffffu, prod, o);
    par += __shfl_xor_sync(0xffffffffu, par, o);
    stay += __shfl_xor_sync(0xffffffffu, stay, o);
  }
  if ((threadIdx.x & 31) == 0 && stay) {
    if (prod) atomicAdd(&totals[0], prod);
    if (par) atomicAdd(&totals[1], par);
    atomicAdd(&totals[2], stay);
  }
}

// NEXT: the multisplit also counts the next level's bins.  EXIT: parents with parent_tag != 0 are left where they are.
template <typename V, bool MULTISPLIT, bool NEXT = false, bool EXIT = false>
__global__ void __launch_bounds__(kSplitThreads, 1024 / kSplitThreads) k5_level(
    const int32_t* __restrict__ x_col, const V* __restrict__ x_val, i64 n_elems,
    const i64* __restrict__ parent_off, i64 n_parents, const TileMeta* __restrict__ tile_meta, int F, int shift,
    u32* __restrict__ counts,     // histogram: (n_parents * F) counters, zero-initialised
    u64* __restrict__ cursor,     // multisplit: (n_parents * F) write cursors, start = child_off
    int32_t* __restrict__ y_col, V* __restrict__ y_val,
    int next_F, int next_shift,   // multisplit: fan-out and shift of the level after this one (next_F == 0: none)
    u32* __restrict__ next_counts,    // ... and its (n_parents * F * next_F) counters, zero-initialised
    const unsigned char* __restrict__ parent_tag = nullptr) {  // EXIT: per parent, != 0: not split at this level
  extern __shared__ __align__(16) unsigned char smem_raw[];
  u32* s_bin = reinterpret_cast<u32*>(smem_raw);                     // kSplitBinCap: counts -> starts -> deltas
  int* s_poff = reinterpret_cast<int*>(s_bin + kSplitBinCap);        // kSplitParentCap + 1: parent starts rel. to tile
  int* s_pstart = s_poff + kSplitParentCap + 1;                      // kSplitParentCap: first permuted slot of a parent
  V* s_val = reinterpret_cast<V*>(s_pstart + kSplitParentCap + 15);  // aligned below
  s_val = reinterpret_cast<V*>((reinterpret_cast<uintptr_t>(s_val)) & ~uintptr_t{15});
  int32_t* s_col = reinterpret_cast<int32_t*>(s_val + kSplitTile);
  u32* s_next = reinterpret_cast<u32*>(s_col + kSplitTile);  // kSplitBinCap: (bin, next child) counts of the tile
  unsigned char* s_ptag = reinterpret_cast<unsigned char*>(s_next + kSplitBinCap);  // kSplitParentCap: tags of the tile's parents
  __shared__ u32 s_scan[33];

  const i64 t0 = static_cast<i64>(blockIdx.x) * kSplitTile;
  const int tn = static_cast<int>(min(static_cast<i64>(kSplitTile), n_elems - t0));
  const int tid = threadIdx.x;
  const u32 lane = tid & 31;
  // The tile's columns do not depend on any metadata: issue their loads first so that the metadata round
  // trips below (tile bounds, then parent offsets) overlap with them instead of preceding them.
  int32_t col[kSplitItems];
#pragma unroll
  for (int k = 0; k < kSplitItems; ++k) {
    const int q = k * kSplitThreads + tid;
    col[k] = q < tn ? x_col[t0 + q] : 0;
  }
  const TileMeta tm = tile_meta[blockIdx.x];  // same address for every thread: one broadcast load
#pragma unroll
  for (int k = 0; k < kSplitBinCap / kSplitThreads; ++k) s_bin[k * kSplitThreads + tid] = 0;
  const i64 p_lo = tm.first;
  const u32 fmask = static_cast<u32>(F - 1);

  if constexpr (EXIT && MULTISPLIT) {
    // a tile of many small parents that all stay behind (the usual tile once a level's chunks are light) moves nothing
    if (tm.n > 2) {
      int moves = 0;
      for (int k = tid; k < tm.n; k += kSplitThreads) moves |= parent_tag[p_lo + k] == 0;
      if (!__syncthreads_or(moves)) return;
    }
  }
  if (tm.n > kSplitParentCap || static_cast<i64>(tm.n) * F > kSplitBinCap) {
    // ---- slow path: one global atomic per element
    for (int q = tid; q < tn; q += kSplitThreads) {
      const i64 p = t0 + q;
      const i64 par = last_le(parent_off, p_lo, p_lo + tm.n - 1, p);
      if (EXIT && MULTISPLIT && parent_tag[par]) continue;
      const int32_t c = x_col[p];  // (the hoisted registers are striped differently; this path is rare)
      const i64 gbin = par * F + ((static_cast<u32>(c) >> shift) & fmask);
      if (MULTISPLIT) {
        const u64 dst = atomicAdd(&cursor[gbin], 1ull);
        y_col[dst] = c;
        y_val[dst] = x_val[p];
        if (NEXT)
          atomicAdd(&next_counts[gbin * next_F + ((static_cast<u32>(c) >> next_shift) & static_cast<u32>(next_F - 1))], 1u);
      } else {
        atomicAdd(&counts[gbin], 1u);
      }
    }
    return;
  }
  const int n_par = tm.n;
  const int n_bins = n_par * F;
  int bin_bits = 0;
  while ((1 << bin_bits) < n_bins) ++bin_bits;
  // one or two parents (the usual tile): the boundary came with the tile record; more: stage their offsets
  if (n_par > 2)
    for (int k = tid; k <= n_par; k += kSplitThreads)
      s_poff[k] = (k == n_par) ? tn + 1 : clamp_rel(parent_off[p_lo + k] - t0, -1, tn + 1);
  bool ex0 = false, ex1 = false;  // EXIT: the tile's first two parents stay behind
  if constexpr (EXIT && MULTISPLIT) {
    ex0 = parent_tag[p_lo] != 0;
    ex1 = n_par > 1 ? parent_tag[p_lo + 1] != 0 : true;
    if (n_par <= 2 && ex0 && ex1) return;  // (uniform) nothing of this tile moves
    if (n_par > 2)
      for (int k = tid; k < n_par; k += kSplitThreads) s_ptag[k] = parent_tag[p_lo + k];
  }
  __syncthreads();

  // ---- local histogram; every element learns its rank inside its bin
  u32 rank_bin[kSplitItems];  // (rank << 11) | bin
  static_assert(kSplitBinCap <= 2048 && kSplitTile <= (1 << 21), "rank/bin packing");
#pragma unroll
  for (int k = 0; k < kSplitItems; ++k) {
    const int q = k * kSplitThreads + tid;
    u32 bin = 0xffffffffu;
    if (q < tn) {
      int par = q >= tm.off1 ? 1 : 0;
      if (n_par > 2) {
        int lo = 0, hi = n_par - 1;
        while (lo < hi) {
          const int mid = lo + ((hi - lo + 1) >> 1);
          if (s_poff[mid] <= q) lo = mid; else hi = mid - 1;
        }
        par = lo;
      }
      bin = static_cast<u32>(par * F) + ((static_cast<u32>(col[k]) >> shift) & fmask);
      if constexpr (EXIT && MULTISPLIT) {
        const bool stay = n_par > 2 ? s_ptag[par] != 0 : (par ? ex1 : ex0);
        if (stay) bin = 0xffffffffu;
      }
    }
    // Rank inside the bin.  A shared-memory atomic that returns its old value costs one wavefront per lane
    // that hits the same address, and with few bins (or one hot child) that is every lane.  So the lanes of a
    // warp first find their peers in the same bin with one ballot per bin bit (the hardware match.any
    // instruction measured 25x slower than this on B200), the lowest peer adds the group's size once, and
    // every member takes base + its position among the peers.
    u32 rank = 0;
    if (MULTISPLIT) {
      // Products reach a parent in runs that come from one row of B, i.e. with ascending columns, so
      // neighbouring lanes usually fall into the same bin.  A run of equal bins is found with one shuffle and
      // one ballot; its first lane adds the run's length to the bin with one atomic and the members take
      // base + their offset in the run.  Only when a warp has many short runs (columns in random order) are the
      // peers of a bin matched across the whole warp, one ballot per bin bit, so that a hot bin still costs one
      // atomic per warp and not one per lane.
      const u32 prev = __shfl_up_sync(0xffffffffu, bin, 1);
      const bool head = lane == 0 || bin != prev;
      const u32 heads = __ballot_sync(0xffffffffu, head);
      if (__popc(heads) <= 12) {
        const u32 below = heads & (lanemask_lt() | (1u << lane));      // heads at or before this lane
        const int start = 31 - __clz(below);                            // first lane of my run
        const u32 above = heads & ~((2u << lane) - 1u);                 // heads after this lane
        const int endl = above ? __ffs(above) - 1 : 32;                 // one past the last lane of my run
        u32 base = 0;
        if (head && bin != 0xffffffffu) base = atomicAdd(&s_bin[bin], static_cast<u32>(endl - start));
        base = __shfl_sync(0xffffffffu, base, start);
        rank = base + static_cast<u32>(lane - start);
      } else {
        u32 peers = 0xffffffffu;
#pragma unroll 1
        for (int b = 0; b < bin_bits; ++b) {
          const bool bit = (bin >> b) & 1u;
          const u32 bal = __ballot_sync(0xffffffffu, bit);
          peers &= bit ? bal : ~bal;
        }
        peers &= __ballot_sync(0xffffffffu, bin != 0xffffffffu);
        const int leader = __ffs(peers) - 1;
        u32 base = 0;
        if (bin != 0xffffffffu && static_cast<int>(lane) == leader) base = atomicAdd(&s_bin[bin], static_cast<u32>(__popc(peers)));
        base = __shfl_sync(0xffffffffu, base, leader < 0 ? 0 : leader);
        rank = base + __popc(peers & lanemask_lt());
      }
    } else {
      if (bin != 0xffffffffu) atomicAdd(&s_bin[bin], 1u);
    }
    rank_bin[k] = (rank << 11) | (bin & 2047u);
    if (EXIT && bin == 0xffffffffu) rank_bin[k] = 0xffffffffu;  // (a rank never reaches 2^21 - 1: not a valid pair)
  }
  __syncthreads();

  // ---- scan of the bin counts; global update (histogram) or range reservation (multisplit)
  constexpr int kBinsPerThread = kSplitBinCap / kSplitThreads;
  u32 cnt[kBinsPerThread];
  u32 sum = 0;
#pragma unroll
  for (int k = 0; k < kBinsPerThread; ++k) {
    const int b = tid * kBinsPerThread + k;
    cnt[k] = b < n_bins ? s_bin[b] : 0u;
    sum += cnt[k];
  }
  const i64 gbin0 = p_lo * F;
  if (!MULTISPLIT) {
#pragma unroll
    for (int k = 0; k < kBinsPerThread; ++k) {
      const int b = tid * kBinsPerThread + k;
      if (cnt[k]) atomicAdd(&counts[gbin0 + b], cnt[k]);
    }
    return;
  }
  u32 total;
  u32 start = block_exclusive_scan(sum, s_scan, &total);
  const int tv = EXIT ? static_cast<int>(total) : tn;  // elements of the tile that move
  u32 delta[kBinsPerThread];
#pragma unroll
  for (int k = 0; k < kBinsPerThread; ++k) {
    const int b = tid * kBinsPerThread + k;
    if (b < n_bins) {
      s_bin[b] = start;  // own slots only: nobody else reads them before the barrier
      if ((b % F) == 0) s_pstart[b / F] = static_cast<int>(start);
      delta[k] = cnt[k] ? static_cast<u32>(atomicAdd(&cursor[gbin0 + b], static_cast<u64>(cnt[k]))) - start : 0u;
    }
    start += cnt[k];
  }
  __syncthreads();

  // ---- permute into shared memory (the irregular part stays on chip)
#pragma unroll
  for (int h = 0; h < kSplitItems; h += 8) {
    V v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int q = (h + k) * kSplitThreads + tid;
      if (q < tn && !(EXIT && rank_bin[h + k] == 0xffffffffu)) v[k] = x_val[t0 + q];
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int q = (h + k) * kSplitThreads + tid;
      if (q < tn && !(EXIT && rank_bin[h + k] == 0xffffffffu)) {
        const u32 rb = rank_bin[h + k];
        const u32 dst = s_bin[rb & 2047u] + (rb >> 11);
        s_col[dst] = col[h + k];
        s_val[dst] = v[k];
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < kBinsPerThread; ++k) {
    const int b = tid * kBinsPerThread + k;
    if (b < n_bins) s_bin[b] = delta[k];  // global position of slot s in bin b is s + delta[b] (mod 2^32 within the batch)
  }
  __syncthreads();

  // ---- coalesced write: slot s belongs to the bin recomputed from its column and its parent.  The next level's
  // bins are counted on the way: in shared memory when the tile's (bin, next child) pairs fit, else one global
  // atomic per element.  Equal pairs sit next to each other (a bin's slots are contiguous and columns come in
  // ascending runs), so the first lane of a run of equal pairs adds the run's length.
  constexpr bool count_next = MULTISPLIT && NEXT;
  const bool next_in_smem = count_next && n_bins * next_F <= kSplitBinCap;
  const u32 nmask = static_cast<u32>(next_F - 1);
  if (next_in_smem) {
    for (int b = tid; b < n_bins * next_F; b += kSplitThreads) s_next[b] = 0;
    __syncthreads();
  }
  auto count_pair = [&](bool valid, u32 bin, int32_t c) {
    if constexpr (!count_next) return;
    const u32 pair = valid ? bin * static_cast<u32>(next_F) + ((static_cast<u32>(c) >> next_shift) & nmask) : 0xffffffffu;
    const u32 prev = __shfl_up_sync(0xffffffffu, pair, 1);
    const bool head = lane == 0 || pair != prev;
    const u32 heads = __ballot_sync(0xffffffffu, head);
    if (head && valid) {
      const u32 above = heads & ~((2u << lane) - 1u);
      const u32 len = static_cast<u32>((above ? __ffs(above) - 1 : 32) - static_cast<int>(lane));
      if (next_in_smem) atomicAdd(&s_next[pair], len);
      else atomicAdd(&next_counts[gbin0 * next_F + pair], len);
    }
  };
  if constexpr (!count_next) {
    if (n_par == 1) {
      // the usual tile (one parent): the bin is the child, nothing to search
#pragma unroll 4
      for (int s = tid; s < tv; s += kSplitThreads) {
        const int32_t c = s_col[s];
        const u32 dst = static_cast<u32>(s) + s_bin[(static_cast<u32>(c) >> shift) & fmask];
        y_col[dst] = c;
        y_val[dst] = s_val[s];
      }
      return;
    }
    for (int s = tid; s < tv; s += kSplitThreads) {
      const int32_t c = s_col[s];
      int par = 0;
      {
        int lo = 0, hi = n_par - 1;
        while (lo < hi) {
          const int mid = lo + ((hi - lo + 1) >> 1);
          if (s_pstart[mid] <= s) lo = mid; else hi = mid - 1;
        }
        par = lo;
      }
      const u32 bin = static_cast<u32>(par * F) + ((static_cast<u32>(c) >> shift) & fmask);
      const u32 dst = static_cast<u32>(s) + s_bin[bin];
      y_col[dst] = c;
      y_val[dst] = s_val[s];
    }
    return;
  }
  if (n_par == 1) {
    // the usual tile (one parent): the bin is the child, nothing to search
    for (int s0 = 0; s0 < tv; s0 += kSplitThreads) {  // (whole warps stay in the loop: count_pair shuffles)
      const int s = s0 + tid;
      const bool valid = s < tv;
      int32_t c = 0;
      u32 bin = 0;
      if (valid) {
        c = s_col[s];
        bin = (static_cast<u32>(c) >> shift) & fmask;
        const u32 dst = static_cast<u32>(s) + s_bin[bin];
        y_col[dst] = c;
        y_val[dst] = s_val[s];
      }
      count_pair(valid, bin, c);
    }
  } else {
    for (int s0 = 0; s0 < tv; s0 += kSplitThreads) {
      const int s = s0 + tid;
      const bool valid = s < tv;
      int32_t c = 0;
      u32 bin = 0;
      if (valid) {
        c = s_col[s];
        int par = 0;
        {
          int lo = 0, hi = n_par - 1;
          while (lo < hi) {
            const int mid = lo + ((hi - lo + 1) >> 1);
            if (s_pstart[mid] <= s) lo = mid; else hi = mid - 1;
          }
          par = lo;
        }
        bin = static_cast<u32>(par * F) + ((static_cast<u32>(c) >> shift) & fmask);
        const u32 dst = static_cast<u32>(s) + s_bin[bin];
        y_col[dst] = c;
        y_val[dst] = s_val[s];
      }
      count_pair(valid, bin, c);
    }
  }
  if (next_in_smem) {
    __syncthreads();
    for (int b = tid; b < n_bins * next_F; b += kSplitThreads) {
      const u32 cnt2 = s_next[b];
      if (cnt2) atomicAdd(&next_counts[gbin0 * next_F + b], cnt2);
    }
  }
}

}  // namespace gm
