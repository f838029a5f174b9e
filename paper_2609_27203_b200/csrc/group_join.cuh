// Grouped join into a tag mirror, for the rule shape  h(a, c) :- h(a, b), r(b, c)  (transitive closure,
// multi-source reachability): many delta rows share the probed value b and differ only in the carried column a.
//
// The mirror of such a relation is addressed with the probed column as the major part of the index and the
// carried column as the minor part, so (1) the delta, which is the changed bitmap read in index order, comes out
// grouped by b, and (2) the slots of (a_1, c), (a_2, c), ... lie next to each other.  A segment = the delta rows of one
// b (k rows) joined with r's run of b (d rows) = k * d candidates, enumerated with the carried row as the fast index:
// candidate p of the segment is (row p % k, neighbour p / k).  Consecutive lanes therefore read one neighbour (a
// broadcast) and consecutive slots (a few sectors instead of one per candidate).
//
//   k_seg_flags     where a delta row starts a new segment, and whether that segment has matches
//   k_seg_first     first row of every segment;  k_seg_build  the segments with matches: first row, rows, k * d candidates
//   k_group_expand  tiles of 1024 candidates over the segments' candidate ranges; sink = the tag mirror
#pragma once
#include "common.cuh"
#include "join.cuh"

namespace xlog {

// flags[i]: low word = 1 where row i starts a new segment (the index bits above the carried bits change); high word = 1
// where that segment also has something to join (its rows found matches).  One scan of the pairs numbers both kinds.
static __global__ void __launch_bounds__(256) k_seg_flags(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ deg, uint32_t n,
                                                         int carried_bits, uint64_t* __restrict__ flags) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const bool head = i == 0 || (keys[i] >> carried_bits) != (keys[i - 1] >> carried_bits);
    flags[i] = head ? (1ull | ((deg[i] ? 1ull : 0ull) << 32)) : 0ull;
  }
}

// first_all[a] = first row of segment a (all segments, n_all + 1 entries, the last one = n)
static __global__ void __launch_bounds__(256) k_seg_first(const uint64_t* __restrict__ flags, const uint64_t* __restrict__ idx, uint32_t n,
                                                         uint32_t n_all, uint32_t* __restrict__ first_all) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i <= n; i += gridDim.x * blockDim.x) {
    if (i == n) first_all[n_all] = n;
    else if (flags[i] & 1ull) first_all[(uint32_t)idx[i]] = i;
  }
}

// the segments with matches, densely numbered: first row, number of rows, candidates = rows * degree
static __global__ void __launch_bounds__(256) k_seg_build(const uint64_t* __restrict__ flags, const uint64_t* __restrict__ idx, uint32_t n,
                                                         const uint32_t* __restrict__ first_all, const uint32_t* __restrict__ deg,
                                                         uint32_t* __restrict__ seg_first, uint32_t* __restrict__ seg_rows,
                                                         uint64_t* __restrict__ seg_cand) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    if (!(flags[i] >> 32)) continue;
    const uint32_t a = (uint32_t)idx[i], b = (uint32_t)(idx[i] >> 32);
    const uint32_t rows = first_all[a + 1] - i;
    seg_first[b] = i;
    seg_rows[b] = rows;
    seg_cand[b] = (uint64_t)rows * deg[i];
  }
}

constexpr int kGrpItems = 4;
constexpr int kGrpTile = kExpBlock * kGrpItems;        // candidates per block = segments staged per block at most

// Block b produces candidates [b * kGrpTile, ...) of the segment candidate space (seg_start = exclusive scan of seg_cand).
// tile_rows[b] = first and last segment touching the tile.
template <int SINK>
__global__ void __launch_bounds__(kExpBlock, 8) k_group_expand(JoinSpec S, const uint64_t* __restrict__ seg_start, const uint32_t* __restrict__ seg_first,
                                                               const uint32_t* __restrict__ seg_rows, const uint4* __restrict__ rowinfo,
                                                               const uint2* __restrict__ tile_rows, uint64_t total, MirrorArgs mr) {
  // per staged segment: {bias, first delta row, rows k, first row of the looked-up run}.  A candidate at tile position q
  // has in-segment index t = q + bias (for the tile's first segment, which may have begun in an earlier tile, the bias
  // and the run's first row already account for the whole neighbours consumed before the tile, so t stays small);
  // neighbour j = t / k, row = t % k, with the division done as a multiplication by sinv = ceil(2^32 / k).
  __shared__ uint4 sseg[kGrpTile];
  __shared__ uint32_t sinv[kGrpTile];
  __shared__ uint16_t ssegidx[kGrpTile];
  __shared__ uint32_t swarp[kExpBlock / 32];
  const uint64_t t_lo = (uint64_t)blockIdx.x * kGrpTile;
  const uint64_t t_hi = min(t_lo + kGrpTile, total);
  if (t_lo >= t_hi) return;
  const uint2 tr = tile_rows[blockIdx.x];
  const uint32_t g_lo = tr.x, nseg = tr.y - tr.x + 1;  // at most kGrpTile: every listed segment holds a candidate of the tile
  const uint32_t ntile = (uint32_t)(t_hi - t_lo);
#pragma unroll
  for (int i = 0; i < kGrpItems; ++i) ssegidx[i * kExpBlock + threadIdx.x] = 0;
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < nseg && i < (uint32_t)kGrpTile; i += kExpBlock) {
    const uint64_t st = seg_start[g_lo + i];
    const uint32_t f = seg_first[g_lo + i];
    const uint32_t rows = seg_rows[g_lo + i];
    uint32_t inner = rowinfo[f].x;
    uint32_t bias;
    if (st <= t_lo) {                                    // the tile's first segment
      const uint64_t before = t_lo - st;                 // its candidates that belong to earlier tiles
      const uint64_t j0 = before / rows;
      inner += (uint32_t)j0;
      bias = (uint32_t)(before - j0 * rows);
    } else {
      const uint32_t rel = (uint32_t)(st - t_lo);
      bias = 0u - rel;
      if (i > 0) ssegidx[rel] = (uint16_t)i;             // rel < ntile: the segment has a candidate in the tile
    }
    sseg[i] = make_uint4(bias, f, rows, inner);
    sinv[i] = rows > 1 ? 0xffffffffu / rows + 1u : 0u;
  }
  __syncthreads();
  // segment of every candidate position: running maximum over the marks (as in the row-wise kernel)
  uint32_t loc[kGrpItems];
  uint32_t run = 0;
#pragma unroll
  for (int i = 0; i < kGrpItems; ++i) { run = max(run, (uint32_t)ssegidx[threadIdx.x * kGrpItems + i]); loc[i] = run; }
  uint32_t incl = run;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) { const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d); if ((int)lane_id() >= d) incl = max(incl, o); }
  if (lane_id() == 31) swarp[warp_id()] = incl;
  __syncthreads();
  uint32_t carry = 0;
  for (int w = 0; w < (int)warp_id(); ++w) carry = max(carry, swarp[w]);
  const uint32_t prev = __shfl_up_sync(0xffffffffu, incl, 1);
  if (lane_id() > 0) carry = max(carry, prev);
#pragma unroll
  for (int i = 0; i < kGrpItems; ++i) ssegidx[threadIdx.x * kGrpItems + i] = (uint16_t)max(loc[i], carry);
  __syncthreads();

  const float* __restrict__ itg = S.inner_tag;
  const int32_t* __restrict__ ic0 = S.inner_col[0];
  const uint32_t m0 = (uint32_t)S.inner_mult[0];
  uint32_t key[kGrpItems];
  float tag[kGrpItems];
#pragma unroll
  for (int k = 0; k < kGrpItems; ++k) {
    const uint32_t q = threadIdx.x + k * kExpBlock;
    key[k] = 0xffffffffu; tag[k] = 0.f;                  // 0xffffffff marks a position past the tile's end
    if (q < ntile) {
      const uint32_t li = ssegidx[q];
      const uint4 sr = sseg[li];
      const uint32_t t = q + sr.x;
      uint32_t j = t;                                    // k == 1
      if (sr.z > 1) {
        j = sr.z < (1u << 15) ? __umulhi(t, sinv[li]) : t / sr.z;        // the product form is exact while t * k < 2^32
      }
      const uint32_t row = t - j * sr.z;
      const uint32_t ir = sr.w + j;
      const uint4 info = rowinfo[sr.y + row];            // count record of the delta row: tag and the carried part of the head key
      key[k] = info.z + (uint32_t)__ldcs(ic0 + ir) * m0;
      tag[k] = __uint_as_float(info.y) + __ldcs(itg + ir);
    }
  }
  int32_t cur[kGrpItems];
#pragma unroll
  for (int k = 0; k < kGrpItems; ++k) {
    cur[k] = SINK == kSinkMin ? (int32_t)0x80000000 : 0x7fffffff;          // nothing improves on this
    if (key[k] <= mr.key_max) cur[k] = XLOG_TABLE_LOAD(mr.table + key[k]);
    else if (threadIdx.x + k * kExpBlock < ntile) atomicOr(mr.err, kErrHeadRange);
  }
#pragma unroll
  for (int k = 0; k < kGrpItems; ++k) {
    const int32_t v = f2ord(tag[k]);
    if (SINK == kSinkMin ? v < cur[k] : v > cur[k]) mirror_commit<SINK>(mr, key[k], v);
  }
}

// ---- segment-stationary variant: a warp takes a slice of one segment's neighbours and keeps the delta rows in its lanes -
// For segments with many candidates (k rows x d neighbours) the per-candidate work shrinks to two shuffles, a
// multiply-add, the slot read and a compare: lanes hold the rows (k' = k rounded up to a power of two, 32 / k' neighbours
// per step), 32 neighbours at a time are read coalesced into registers and handed round with shuffles.
// An item = (segment, slice of seg_slice(k) neighbours); seg_slice keeps k * slice near 4096 candidates.
__host__ __device__ __forceinline__ uint32_t seg_slice(uint32_t rows) {
  const uint32_t s = 4096u / (rows < 1u ? 1u : rows);
  return s < 32u ? 32u : (s & ~31u);
}

static __global__ void __launch_bounds__(256) k_seg_items(const uint32_t* __restrict__ seg_first, const uint32_t* __restrict__ seg_rows, uint32_t n_seg,
                                                         const uint32_t* __restrict__ deg, uint32_t* __restrict__ items) {
  for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g <= n_seg; g += gridDim.x * blockDim.x) {
    uint32_t n = 0;
    if (g < n_seg) { const uint32_t sl = seg_slice(seg_rows[g]); n = (deg[seg_first[g]] + sl - 1) / sl; }
    items[g] = n;                                        // items[n_seg] = 0: the scan then has n_seg + 1 entries
  }
}
static __global__ void __launch_bounds__(256) k_seg_item_fill(uint32_t n_seg, const uint32_t* __restrict__ item_off, uint32_t* __restrict__ item_seg) {
  for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g < n_seg; g += gridDim.x * blockDim.x)
    for (uint32_t it = item_off[g]; it < item_off[g + 1]; ++it) item_seg[it] = g;
}

template <int SINK>
__global__ void __launch_bounds__(256, 8) k_seg_expand(JoinSpec S, uint32_t n_items, const uint32_t* __restrict__ item_off, const uint32_t* __restrict__ item_seg,
                                                    const uint32_t* __restrict__ seg_first, const uint32_t* __restrict__ seg_rows,
                                                    const uint32_t* __restrict__ deg, const uint4* __restrict__ rowinfo, MirrorArgs mr) {
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  const float* __restrict__ itg = S.inner_tag;
  const int32_t* __restrict__ ic0 = S.inner_col[0];
  const uint32_t m0 = (uint32_t)S.inner_mult[0];
  uint32_t e = 0;
  for (uint32_t it = warp; it < n_items; it += nwarps) {
    const uint32_t g = item_seg[it];
    const uint32_t f = seg_first[g], rows = seg_rows[g];
    const uint32_t d = deg[f], lo = rowinfo[f].x;
    const uint32_t sl = seg_slice(rows);
    const uint32_t j_begin = (it - item_off[g]) * sl, j_end = min(d, j_begin + sl);
    for (uint32_t row0 = 0; row0 < rows; row0 += 32) {
      const uint32_t kp = min(rows - row0, 32u);
      uint32_t kq = 1;                                   // kp rounded up to a power of two
      while (kq < kp) kq <<= 1;
      const uint32_t per = 32u / kq;                     // neighbours per step
      const uint32_t my_row = lane & (kq - 1), jsub = lane / kq;
      const bool has_row = my_row < kp;
      uint32_t ckey = 0;
      float otag = 0.f;
      if (has_row) { const uint4 info = rowinfo[f + row0 + my_row]; ckey = info.z; otag = __uint_as_float(info.y); }
      for (uint32_t jb = j_begin; jb < j_end; jb += 32) {
        const uint32_t nj = min(32u, j_end - jb);
        uint32_t zr = 0;
        float wr = 0.f;
        if (lane < nj) { zr = (uint32_t)__ldcs(ic0 + lo + jb + lane); wr = __ldcs(itg + lo + jb + lane); }
        // four steps at a time: keys first, then the four slot reads together, then the reductions of those that improve
        for (uint32_t s0 = 0; s0 < nj; s0 += 4 * per) {
          uint32_t key[4];
          int32_t v[4], cur[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t jj = s0 + u * per + jsub;
            const uint32_t z = __shfl_sync(0xffffffffu, zr, jj & 31);
            const float w = __shfl_sync(0xffffffffu, wr, jj & 31);
            key[u] = 0xffffffffu;                        // nothing to do
            v[u] = 0;
            if (has_row && jj < nj) {
              key[u] = ckey + z * m0;
              v[u] = f2ord(otag + w);
              if (key[u] > mr.key_max) { e |= kErrHeadRange; key[u] = 0xffffffffu; }
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            cur[u] = SINK == kSinkMin ? (int32_t)0x80000000 : 0x7fffffff;
            if (key[u] != 0xffffffffu) cur[u] = XLOG_TABLE_LOAD(mr.table + key[u]);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (SINK == kSinkMin ? v[u] < cur[u] : v[u] > cur[u]) mirror_commit<SINK>(mr, key[u], v[u]);
        }
      }
    }
  }
  if (e) atomicOr(mr.err, e);
}

}  // namespace xlog
