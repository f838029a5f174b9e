// Relation-store kernels: validation + key packing (paper kernel table: `pack`), unpacking,
// leading-column offsets (the join index), semiring segmented reduce-by-key (`groupby`:
// boundary detection then per-group reduction) and the merge-path set difference / union
// with tag improvement (`dedup`, `set_ops`; Algorithm 1 lines 8-9).
#pragma once
#include "common.cuh"

namespace xlog {

// ---------------------------------------------------------------------------------
// load-time validation: per-column maximum, negative keys, NaN / semiring-zero tags
// ---------------------------------------------------------------------------------
struct ColPtrs { const int32_t* c[kMaxArity]; };
struct ColPtrsMut { int32_t* c[kMaxArity]; };

// Validation, column maxima and an order test in one read of the input: *unordered is raised when some row is not
// lexicographically greater than the row before it (rows that arrive strictly increasing need no sort and hold no duplicates).
static __global__ void __launch_bounds__(256) k_col_stats(ColPtrs cols, const float* __restrict__ tags, int64_t n, int arity, int sr,
                                                   int32_t* __restrict__ col_max /*[arity]*/, uint32_t* __restrict__ err,
                                                   uint32_t* __restrict__ unordered) {
  int32_t mx[kMaxArity] = {0, 0, 0, 0};
  uint32_t e = 0;
  bool out_of_order = false;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    int cmp = 0;                                        // sign of (row i - row i-1), decided by the first differing column
#pragma unroll
    for (int c = 0; c < kMaxArity; ++c)
      if (c < arity) {
        const int32_t v = cols.c[c][i];
        if (v < 0) e |= kErrNegativeKey;
        mx[c] = max(mx[c], v);
        if (i > 0 && cmp == 0) { const int32_t p = cols.c[c][i - 1]; cmp = v > p ? 1 : v < p ? -1 : 0; }
      }
    if (i > 0 && cmp <= 0) out_of_order = true;
    if (tags) {
      const float t = tags[i];
      const bool zero = sr == 0 || sr == 2 ? t == -INFINITY : sr == 1 ? t == INFINITY : false;
      if (isnan(t) || zero) e |= kErrBadTag;
    }
  }
#pragma unroll
  for (int c = 0; c < kMaxArity; ++c) {
#pragma unroll
    for (int d = 16; d; d >>= 1) mx[c] = max(mx[c], __shfl_xor_sync(0xffffffffu, mx[c], d));
  }
#pragma unroll
  for (int d = 16; d; d >>= 1) e |= __shfl_xor_sync(0xffffffffu, e, d);
  if (lane_id() == 0) {
    for (int c = 0; c < arity; ++c) atomicMax(&col_max[c], mx[c]);
    if (e) atomicOr(err, e);
  }
  if (__any_sync(0xffffffffu, out_of_order) && lane_id() == 0) atomicOr(unordered, 1u);
}

template <typename K>
__global__ void __launch_bounds__(256) k_pack(ColPtrs cols, const float* __restrict__ tags, int64_t n, KeyLayout L, DictSet D, float one,
                                              K* __restrict__ keys, float* __restrict__ tag_out) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    int32_t v[kMaxArity];
#pragma unroll
    for (int c = 0; c < kMaxArity; ++c) {
      v[c] = c < L.arity ? cols.c[c][i] : 0;
      if (c < L.arity && D.n[c]) v[c] = (int32_t)dict_rank(D.v[c], D.n[c], v[c]);
    }
    keys[i] = pack_key<K>(L, v);
    float t = tags ? tags[i] : one;
    if (t == 0.f) t = 0.f;                         // -0.0 -> +0.0
    tag_out[i] = t;
  }
}

template <typename K>
__global__ void __launch_bounds__(256) k_unpack(const K* __restrict__ keys, int64_t n, KeyLayout L, DictSet D, ColPtrsMut cols) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const K k = keys[i];
#pragma unroll
    for (int c = 0; c < kMaxArity; ++c)
      if (c < L.arity) {
        const int32_t code = key_col<K>(L, k, c);
        cols.c[c][i] = D.n[c] ? D.v[c][min((uint32_t)code, D.n[c] - 1)] : code;
      }
  }
}

// off[v] = first row whose leading column is >= v, for v in [0, domain]  (off[domain] = n).
static __global__ void __launch_bounds__(256) k_build_offsets(const int32_t* __restrict__ lead, uint32_t n, int64_t domain,
                                                       uint32_t* __restrict__ off) {
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v <= domain; v += (int64_t)gridDim.x * blockDim.x) {
    uint32_t lo = 0, hi = n;
    while (lo < hi) {
      const uint32_t mid = lo + ((hi - lo) >> 1);
      if ((int64_t)lead[mid] < v) lo = mid + 1; else hi = mid;
    }
    off[v] = lo;
  }
}

template <typename K>
__global__ void __launch_bounds__(256) k_check_sorted(const K* __restrict__ keys, int64_t n, uint32_t* __restrict__ err) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x + 1; i < n; i += (int64_t)gridDim.x * blockDim.x)
    if (!(keys[i - 1] < keys[i])) atomicOr(err, kErrNotSorted);
}

// ---------------------------------------------------------------------------------
// count aggregate: group sizes from group-head positions, and the trailing count column
// (paper Listing 7: count is a head column)
// ---------------------------------------------------------------------------------
static __global__ void __launch_bounds__(256) k_group_sizes(const uint32_t* __restrict__ head_pos, uint32_t u, uint32_t* __restrict__ counts,
                                                     uint32_t* __restrict__ max_count) {
  uint32_t m = 0;
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < u; i += gridDim.x * blockDim.x) {
    const uint32_t cnt = head_pos[i + 1] - head_pos[i];
    counts[i] = cnt;
    m = max(m, cnt);
  }
#pragma unroll
  for (int d = 16; d; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
  if (lane_id() == 0 && m) atomicMax(max_count, m);
}

template <typename Kin, typename Kout>
__global__ void __launch_bounds__(256) k_append_count(const Kin* __restrict__ keys, const uint32_t* __restrict__ counts, uint32_t u,
                                                      int count_bits, Kout* __restrict__ out) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < u; i += gridDim.x * blockDim.x)
    out[i] = ((Kout)keys[i] << count_bits) | (Kout)counts[i];
}

// ---------------------------------------------------------------------------------
// segmented scan machinery for reduce-by-key
// ---------------------------------------------------------------------------------
// (flag, value) pairs; flag = "a segment starts somewhere in the covered range".
// Inclusive warp scan:  value = combination of everything since the last segment start.
template <typename Op>
__device__ __forceinline__ void warp_seg_scan_incl(bool& f, typename Op::A& v) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const typename Op::A vn = shfl_up(v, d);
    const int fn = __shfl_up_sync(0xffffffffu, (int)f, d);
    if ((int)lane_id() >= d) {
      if (!f) v = Op::combine(vn, v);
      f = f || fn;
    }
  }
}

// Block-wide: given each thread's summary (f, v), return the carry entering the thread:
// combination of all items of earlier threads since the last segment start, and whether
// such a start exists in earlier threads (carry_f).  Also returns the block summary.
template <int BLOCK, typename Op>
__device__ __forceinline__ void block_seg_scan_excl(bool f, typename Op::A v, bool* shf, typename Op::A* shv,
                                                    bool& carry_f, typename Op::A& carry_v, bool& block_f,
                                                    typename Op::A& block_v) {
  constexpr int W = BLOCK / 32;
  bool fi = f;
  typename Op::A vi = v;
  warp_seg_scan_incl<Op>(fi, vi);
  if (lane_id() == 31) { shf[warp_id()] = fi; shv[warp_id()] = vi; }
  __syncthreads();
  // carry from earlier warps (sequential over at most W-1 warp summaries)
  bool wf = false;
  typename Op::A wv = Op::identity();
  for (int w = 0; w < (int)warp_id(); ++w) {
    if (shf[w]) { wf = true; wv = shv[w]; } else wv = Op::combine(wv, shv[w]);
  }
  // exclusive within the warp = inclusive of the previous lane
  typename Op::A pv = shfl_up(vi, 1);
  int pf = __shfl_up_sync(0xffffffffu, (int)fi, 1);
  if (lane_id() == 0) { carry_f = wf; carry_v = wv; }
  else if (pf) { carry_f = true; carry_v = pv; }
  else { carry_f = wf; carry_v = Op::combine(wv, pv); }
  // block summary
  bool bf = false;
  typename Op::A bv = Op::identity();
  for (int w = 0; w < W; ++w) {
    if (shf[w]) { bf = true; bv = shv[w]; } else bv = Op::combine(bv, shv[w]);
  }
  block_f = bf; block_v = bv;
  __syncthreads();
}

constexpr int kRbkBlock = 256;
constexpr int kRbkItems = 8;
constexpr int kRbkTile = kRbkBlock * kRbkItems;

// Pass 1: per tile, the number of segment heads and the combination of the tile's open tail
// (everything from its last head to its end; the whole tile if it has no head).
template <typename K, typename Op>
__global__ void __launch_bounds__(kRbkBlock) k_rbk_tiles(const K* __restrict__ keys, const float* __restrict__ tags, uint32_t n,
                                                         uint32_t* __restrict__ tile_heads, typename Op::A* __restrict__ tile_tail) {
  __shared__ bool shf[kRbkBlock / 32];
  __shared__ typename Op::A shv[kRbkBlock / 32];
  __shared__ uint32_t shc[kRbkBlock / 32 + 1];
  const uint64_t base = (uint64_t)blockIdx.x * kRbkTile + (uint64_t)threadIdx.x * kRbkItems;
  K prev = 0;
  if (base > 0 && base - 1 < n) prev = keys[base - 1];
  bool f = false;
  typename Op::A v = Op::identity();
  uint32_t heads = 0;
#pragma unroll
  for (int i = 0; i < kRbkItems; ++i) {
    const uint64_t p = base + i;
    if (p < n) {
      const K k = keys[p];
      const bool head = p == 0 || k != prev;
      prev = k;
      const typename Op::A x = Op::lift(tags[p]);
      if (head) { f = true; v = x; ++heads; } else v = Op::combine(v, x);
    }
  }
  bool cf, bf; typename Op::A cv, bv;
  block_seg_scan_excl<kRbkBlock, Op>(f, v, shf, shv, cf, cv, bf, bv);
  uint32_t total;
  block_scan_excl<kRbkBlock, uint32_t>(heads, shc, total);
  if (threadIdx.x == 0) { tile_heads[blockIdx.x] = total; tile_tail[blockIdx.x] = bv; }
}

// Pass 2 (one block): head_base = exclusive sum of tile_heads; carry_in[t] = combination of the
// open tails of the tiles before t back to (and including) the last tile that has a head.
template <typename Op>
__global__ void __launch_bounds__(1024) k_rbk_spine(uint32_t* __restrict__ tile_heads /*in: counts, out: exclusive base*/,
                                                    const typename Op::A* __restrict__ tile_tail,
                                                    typename Op::A* __restrict__ carry_in, uint32_t ntiles,
                                                    uint32_t* __restrict__ total_heads) {
  __shared__ bool shf[32];
  __shared__ typename Op::A shv[32];
  __shared__ uint32_t shc[33];
  uint32_t run_heads = 0;
  bool run_f = false;                         // unused except for symmetry
  typename Op::A run_v = Op::identity();      // carry entering the current chunk
  for (uint32_t base = 0; base < ntiles; base += 1024) {
    const uint32_t t = base + threadIdx.x;
    const uint32_t h = t < ntiles ? tile_heads[t] : 0u;
    const bool f = h > 0;
    const typename Op::A v = t < ntiles ? tile_tail[t] : Op::identity();
    bool cf, bf; typename Op::A cv, bv;
    block_seg_scan_excl<1024, Op>(f, v, shf, shv, cf, cv, bf, bv);
    uint32_t total;
    const uint32_t e = block_scan_excl<1024, uint32_t>(h, shc, total);
    if (t < ntiles) {
      tile_heads[t] = run_heads + e;
      carry_in[t] = cf ? cv : Op::combine(run_v, cv);
    }
    run_v = bf ? bv : Op::combine(run_v, bv);
    run_f = run_f || bf;
    run_heads += total;
  }
  if (threadIdx.x == 0) *total_heads = run_heads;
}

// Pass 3: emit one (key, combined tag) per segment, at the tile holding the segment's last row.
// head_pos (optional) receives the row index of each segment head, so segment length (the
// count aggregate) is head_pos[u+1] - head_pos[u].
template <typename K, typename Op>
__global__ void __launch_bounds__(kRbkBlock) k_rbk_emit(const K* __restrict__ keys, const float* __restrict__ tags, uint32_t n,
                                                        const uint32_t* __restrict__ head_base,
                                                        const typename Op::A* __restrict__ carry_in, K* __restrict__ out_keys,
                                                        float* __restrict__ out_tags, uint32_t* __restrict__ head_pos) {
  __shared__ bool shf[kRbkBlock / 32];
  __shared__ typename Op::A shv[kRbkBlock / 32];
  __shared__ uint32_t shc[kRbkBlock / 32 + 1];
  const uint64_t base = (uint64_t)blockIdx.x * kRbkTile + (uint64_t)threadIdx.x * kRbkItems;
  K key[kRbkItems + 1];
  float tg[kRbkItems];
  K prev = 0;
  if (base > 0 && base - 1 < n) prev = keys[base - 1];
#pragma unroll
  for (int i = 0; i < kRbkItems; ++i) {
    const uint64_t p = base + i;
    key[i] = p < n ? keys[p] : K(0);
    tg[i] = p < n ? tags[p] : 0.f;
  }
  key[kRbkItems] = base + kRbkItems < n ? keys[base + kRbkItems] : K(0);

  bool f = false;
  typename Op::A v = Op::identity();
  uint32_t heads = 0;
  {
    K pk = prev;
#pragma unroll
    for (int i = 0; i < kRbkItems; ++i) {
      const uint64_t p = base + i;
      if (p < n) {
        const bool head = p == 0 || key[i] != pk;
        pk = key[i];
        const typename Op::A x = Op::lift(tg[i]);
        if (head) { f = true; v = x; ++heads; } else v = Op::combine(v, x);
      }
    }
  }
  bool cf, bf; typename Op::A cv, bv;
  block_seg_scan_excl<kRbkBlock, Op>(f, v, shf, shv, cf, cv, bf, bv);
  uint32_t total;
  uint32_t hidx = block_scan_excl<kRbkBlock, uint32_t>(heads, shc, total) + head_base[blockIdx.x];   // heads before this thread
  typename Op::A acc = cf ? cv : Op::combine(carry_in[blockIdx.x], cv);
  K pk = prev;
#pragma unroll
  for (int i = 0; i < kRbkItems; ++i) {
    const uint64_t p = base + i;
    if (p < n) {
      const bool head = p == 0 || key[i] != pk;
      pk = key[i];
      const typename Op::A x = Op::lift(tg[i]);
      if (head) {
        acc = x;
        if (head_pos) head_pos[hidx] = (uint32_t)p;
        ++hidx;
      } else acc = Op::combine(acc, x);
      const bool last = p + 1 == n || key[i + 1] != key[i];
      if (last) { out_keys[hidx - 1] = key[i]; out_tags[hidx - 1] = Op::lower(acc); }
    }
  }
}

// ---------------------------------------------------------------------------------
// merge-path difference / union with tag improvement
// ---------------------------------------------------------------------------------
// A = reduced candidates (strictly increasing keys), B = full relation (strictly increasing).
// Merge order puts A before B on equal keys, so a matching pair is adjacent.
//   A row without a match          -> new tuple:      goes to full' and to delta'
//   A row whose tag strictly beats -> improved tuple: goes to delta'; the B row carries the new tag
//   B row                          -> goes to full' with tag = B oplus matching A
constexpr int kMrgBlock = 256;
constexpr int kMrgItems = 8;
constexpr int kMrgTile = kMrgBlock * kMrgItems;

template <typename K>
__global__ void __launch_bounds__(256) k_merge_partition(const K* __restrict__ A, uint32_t na, const uint32_t* __restrict__ na_ptr,
                                                         const K* __restrict__ B, uint32_t nb, uint32_t ntiles,
                                                         uint32_t* __restrict__ a_start /*[ntiles+1]*/) {
  const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t > ntiles) return;
  if (na_ptr) na = min(na, *na_ptr);                   // the exact row count may still live on the device only
  const uint64_t diag = min((uint64_t)t * kMrgTile, (uint64_t)na + nb);
  uint32_t lo = diag > nb ? (uint32_t)(diag - nb) : 0u;
  uint32_t hi = (uint32_t)min((uint64_t)na, diag);
  while (lo < hi) {
    const uint32_t mid = lo + ((hi - lo) >> 1);
    if (A[mid] <= B[diag - 1 - mid]) lo = mid + 1; else hi = mid;
  }
  a_start[t] = lo;
}

struct MergeCounts { uint32_t* tile_nf; uint32_t* tile_nd; };

template <typename K, typename Op, bool EMIT>
__global__ void __launch_bounds__(kMrgBlock) k_merge(const K* __restrict__ A, const float* __restrict__ TA, uint32_t na,
                                                     const uint32_t* __restrict__ na_ptr, const K* __restrict__ B,
                                                     float* __restrict__ TB, uint32_t nb, const uint32_t* __restrict__ a_start,
                                                     uint32_t* __restrict__ tile_nf, uint32_t* __restrict__ tile_nd,
                                                     K* __restrict__ FK, float* __restrict__ FT, K* __restrict__ DK,
                                                     float* __restrict__ DT, int inplace, const uint32_t* __restrict__ total_f) {
  if (na_ptr) na = min(na, *na_ptr);
  // inplace < 0: decide here from the merged row count (no new key <=> full' would have exactly nb rows)
  if (EMIT && inplace < 0) inplace = *total_f == nb ? 1 : 0;
  __shared__ K sk[kMrgTile + 2];
  __shared__ float st[kMrgTile];
  __shared__ uint32_t shc[kMrgBlock / 32 + 1];
  __shared__ K peek[2];
  __shared__ float peek_t;
  const uint32_t t = blockIdx.x;
  const uint64_t d0 = (uint64_t)t * kMrgTile;
  if (d0 >= (uint64_t)na + nb) {                        // tile beyond the data (grid sized from an upper bound)
    if (!EMIT && threadIdx.x == 0) { tile_nf[t] = 0; tile_nd[t] = 0; }
    return;
  }
  const uint64_t d1 = min(d0 + kMrgTile, (uint64_t)na + nb);
  const uint32_t a0 = a_start[t], a1 = a_start[t + 1];
  const uint32_t b0 = (uint32_t)(d0 - a0), b1 = (uint32_t)(d1 - a1);
  const uint32_t la = a1 - a0, lb = b1 - b0;
  for (uint32_t i = threadIdx.x; i < la; i += kMrgBlock) { sk[i] = A[a0 + i]; st[i] = TA[a0 + i]; }
  for (uint32_t i = threadIdx.x; i < lb; i += kMrgBlock) { sk[la + i] = B[b0 + i]; st[la + i] = TB[b0 + i]; }
  if (threadIdx.x == 0) {
    // the A row just before this tile (a match for the tile's first B row) and the B row just after it
    peek[0] = a0 > 0 ? A[a0 - 1] : K(0);
    peek_t = a0 > 0 ? TA[a0 - 1] : 0.f;
    peek[1] = b1 < nb ? B[b1] : K(0);
  }
  __syncthreads();
  const K* sa = sk;
  const K* sb = sk + la;
  const float* ta = st;
  const float* tb = st + la;
  const bool have_prev_a = a0 > 0, have_next_b = b1 < nb;

  // this thread's diagonal inside the tile
  const uint32_t diag = min((uint32_t)threadIdx.x * kMrgItems, la + lb);
  uint32_t lo = diag > lb ? diag - lb : 0u, hi = min(la, diag);
  while (lo < hi) {
    const uint32_t mid = (lo + hi) >> 1;
    if (sa[mid] <= sb[diag - 1 - mid]) lo = mid + 1; else hi = mid;
  }
  uint32_t ai = lo, bi = diag - lo;
  const uint32_t steps = min((uint32_t)kMrgItems, la + lb - diag);

  // walk 1: count outputs
  uint32_t nf = 0, nd = 0;
  {
    uint32_t x = ai, y = bi;
    for (uint32_t s = 0; s < steps; ++s) {
      const bool takeA = x < la && (y >= lb || sa[x] <= sb[y]);
      if (takeA) {
        const K k = sa[x];
        const bool has = y < lb ? sb[y] == k : (have_next_b && peek[1] == k);
        if (!has) { ++nf; ++nd; }
        else {
          const float bt = y < lb ? tb[y] : TB[b1];
          if (Op::better(ta[x], bt)) ++nd;
        }
        ++x;
      } else { ++nf; ++y; }
    }
  }
  uint32_t tot_f, tot_d;
  const uint32_t of = block_scan_excl<kMrgBlock, uint32_t>(nf, shc, tot_f);
  const uint32_t od = block_scan_excl<kMrgBlock, uint32_t>(nd, shc, tot_d);
  if (!EMIT) {
    if (threadIdx.x == 0) { tile_nf[t] = tot_f; tile_nd[t] = tot_d; }
    return;
  }
  // walk 2: write.  tile_nf / tile_nd now hold exclusive bases.
  uint32_t pf = tile_nf[t] + of, pd = tile_nd[t] + od;
  uint32_t x = ai, y = bi;
  for (uint32_t s = 0; s < steps; ++s) {
    const bool takeA = x < la && (y >= lb || sa[x] <= sb[y]);
    if (takeA) {
      const K k = sa[x];
      const bool has = y < lb ? sb[y] == k : (have_next_b && peek[1] == k);
      if (!has) {
        if (!inplace) { FK[pf] = k; FT[pf] = ta[x]; }
        ++pf;
        DK[pd] = k; DT[pd] = ta[x]; ++pd;
      } else {
        const float bt = y < lb ? tb[y] : TB[b1];
        if (Op::better(ta[x], bt)) {
          DK[pd] = k; DT[pd] = ta[x]; ++pd;
          if (inplace) TB[y < lb ? b0 + y : b1] = ta[x];
        }
      }
      ++x;
    } else {
      if (!inplace) {
        const K k = sb[y];
        float v = tb[y];
        // matching A row, if any, is the one merged just before this B row
        if (x > 0) { if (sa[x - 1] == k) v = Op::lower(Op::combine(Op::lift(v), Op::lift(ta[x - 1]))); }
        else if (have_prev_a && peek[0] == k) v = Op::lower(Op::combine(Op::lift(v), Op::lift(peek_t)));
        FK[pf] = k; FT[pf] = v;
      }
      ++pf; ++y;
    }
  }
}

}  // namespace xlog
