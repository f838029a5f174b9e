// Fused directed-triangle aggregate  h(x, count) :- e(x,y), e(y,z), e(z,x)  (paper: "Worst-case-
// optimal joins" and the fused triangle counting of "Head-to-head comparisons": triangles are
// counted and their tags combined without ever materialising the tri relation).
//
// For every edge (x,y) the sorted out-list of y is intersected with the sorted in-list of x; each
// common z contributes (w_xy otimes w_yz) otimes w_zx to x's group.  One warp per edge walks the
// shorter list and binary-searches the longer one; per-edge partial aggregates are then combined
// per x in a fixed order (edges of x are contiguous in the store), so results are reproducible.
#pragma once
#include "common.cuh"

namespace xlog {

struct TriGraph {
  uint32_t n_edges;
  const int32_t* src;            // column 0 of the store (ascending)
  const int32_t* dst;            // column 1
  const float* w;                // tags in stored order
  // second atom's relation (the same store when all three atoms name one relation): column 1 and tags, with
  int64_t out_domain, in_domain;
  const uint32_t* out_off;       // offsets over its column 0: out-list of v is s_dst[out_off[v] .. out_off[v+1])
  const int32_t* s_dst;
  const float* s_w;
  // third atom's relation, transposed:
  const uint32_t* in_off;        // offsets over dst of the transposed copy
  const int32_t* in_src;         // transposed copy: sources of the edges into v, ascending
  const float* in_w;             // and their tags
};

constexpr uint32_t kTriChunk = 1024;     // walked entries per work item (32 sweeps of a warp)

// Two ways to intersect out(y) with in(x).  Search: walk the shorter list, binary-search the longer one (about log2 of its
// length dependent reads per walked entry).  Bitmap: a block marks in(x) in a shared-memory bitmap (one bit per node, plus
// a running popcount per word, so that a hit's place in in(x) - needed for its tag - is one popcount away) and its warps
// walk the out-lists of ALL of x's neighbours y against it: one load and one bit test per walked entry.  The bitmap way
// walks out(y) even where in(x) is the shorter list, and it pays for building the bitmap, so it is taken per x, from two
// sums over x's edges that depend on the graph alone: the entries either way would walk.
constexpr int64_t kTriBitmapMaxDomain = (int64_t)1 << 19;      // nodes (sources and targets alike): 64 KB of bits and 64 KB of running counts
#ifndef XLOG_TRI_UNROLL
#define XLOG_TRI_UNROLL 8
#endif
constexpr int kTriBitmapUnroll = XLOG_TRI_UNROLL;                            // sweeps of 32 list entries a warp reads before it tests them
#ifndef XLOG_TRI_UNIT_ITEMS
#define XLOG_TRI_UNIT_ITEMS 512
#endif
constexpr uint32_t kTriUnitItems = XLOG_TRI_UNIT_ITEMS;        // work items per (x, slice) unit of the bitmap kernel

struct TriRoute {
  const unsigned long long* sum_out;   // per x: sum over its edges (x,y) of |out(y)|            (entries the bitmap way walks)
  const unsigned long long* sum_min;   // per x: sum over its edges of min(|out(y)|, |in(x)|)    (entries the search way walks)
  int enabled;
};

// Measured on R-MAT 18: a searched entry costs 10.2 ps of kernel time, an entry tested against the bitmap 3.9 ps; building
// costs about the in-list's length plus a scan of the bitmap's words.  The bitmap way is taken where it walks at most
// kTriBitmapRatioX2 / 2 times the entries of the search way.
#ifndef XLOG_TRI_BITMAP_RATIO_X2
#define XLOG_TRI_BITMAP_RATIO_X2 5
#endif
constexpr unsigned long long kTriBitmapRatioX2 = XLOG_TRI_BITMAP_RATIO_X2;
__device__ __forceinline__ bool tri_bitmap_route(const TriGraph& G, const TriRoute& R, int32_t x, uint32_t lb) {
  if (!R.enabled || lb < 32u) return false;
  const unsigned long long so = R.sum_out[x], sm = R.sum_min[x];
  return so >= 8192ull && 2ull * (so + 16ull * lb + 32768ull) < kTriBitmapRatioX2 * sm;
}

// Per-x sums for the choice above; sums must be zero on entry.  Edges are sorted by x, so a warp's 32 edges mostly share
// one x: then one lane adds for all.
static __global__ void __launch_bounds__(256) k_tri_route_sums(TriGraph G, unsigned long long* __restrict__ sum_out, unsigned long long* __restrict__ sum_min) {
  const uint32_t n32 = (G.n_edges + 31u) & ~31u;
  for (uint32_t e = blockIdx.x * blockDim.x + threadIdx.x; e < n32; e += gridDim.x * blockDim.x) {
    int32_t x = -1;
    uint32_t la = 0, lb = 0;
    if (e < G.n_edges) {
      x = G.src[e];
      const int32_t y = G.dst[e];
      if (y < G.out_domain) la = G.out_off[y + 1] - G.out_off[y];
      if (x < G.in_domain) lb = G.in_off[x + 1] - G.in_off[x];
      if (x >= G.in_domain) x = -1;
    }
    const int32_t x0 = __shfl_sync(0xffffffffu, x, 0);
    if (__all_sync(0xffffffffu, x == x0)) {
      const unsigned long long a = __reduce_add_sync(0xffffffffu, la), m = __reduce_add_sync(0xffffffffu, min(la, lb));
      if (lane_id() == 0 && x0 >= 0 && a) { atomicAdd(sum_out + x0, a); atomicAdd(sum_min + x0, m); }
    } else if (x >= 0 && la) {
      atomicAdd(sum_out + x, (unsigned long long)la);
      atomicAdd(sum_min + x, (unsigned long long)min(la, lb));
    }
  }
}

// Work items of the aggregate: an edge whose shorter list has n entries is cut into ceil(n / kTriChunk) items, so that a
// hub edge (tens of thousands of entries to walk) is shared by many warps instead of serialising one; an edge with an
// empty list gets none.  items[e] for e < n_edges, items[n_edges] = 0 (so that the exclusive scan has n_edges + 1 entries).
// *walked accumulates the total number of entries to walk (one probe each), *walked_bitmap those of them the bitmap kernel walks.
static __global__ void __launch_bounds__(256) k_tri_plan(TriGraph G, TriRoute R, uint32_t* __restrict__ items, unsigned long long* __restrict__ walked,
                                                         unsigned long long* __restrict__ walked_bitmap) {
  unsigned long long mine = 0, mine_bm = 0;
  for (uint32_t e = blockIdx.x * blockDim.x + threadIdx.x; e <= G.n_edges; e += gridDim.x * blockDim.x) {
    uint32_t n = 0;
    if (e < G.n_edges) {
      const int32_t x = G.src[e], y = G.dst[e];
      uint32_t la = 0, lb = 0;
      if (y < G.out_domain) la = G.out_off[y + 1] - G.out_off[y];
      if (x < G.in_domain) lb = G.in_off[x + 1] - G.in_off[x];
      // the bitmap way walks out(y) whichever list is shorter
      const bool bm = lb && tri_bitmap_route(G, R, x, lb);
      const uint32_t w = bm ? la : min(la, lb);
      n = (w + kTriChunk - 1) / kTriChunk;
      mine += w;
      if (bm) mine_bm += w;
    }
    items[e] = n;
  }
#pragma unroll
  for (int d = 16; d; d >>= 1) { mine += __shfl_down_sync(0xffffffffu, mine, d); mine_bm += __shfl_down_sync(0xffffffffu, mine_bm, d); }
  if (lane_id() == 0 && mine) atomicAdd(walked, mine);
  if (lane_id() == 0 && mine_bm) atomicAdd(walked_bitmap, mine_bm);
}

// item -> edge, written by the edge (item_off = exclusive scan of items)
static __global__ void __launch_bounds__(256) k_tri_item_edges(uint32_t n_edges, const uint32_t* __restrict__ item_off, uint32_t* __restrict__ item_edge) {
  for (uint32_t e = blockIdx.x * blockDim.x + threadIdx.x; e < n_edges; e += gridDim.x * blockDim.x)
    for (uint32_t it = item_off[e]; it < item_off[e + 1]; ++it) item_edge[it] = e;
}

// One warp per work item: partial count and aggregate of its slice of the walked list.
template <typename Op>
__global__ void __launch_bounds__(256) k_tri_edges(TriGraph G, TriRoute R, int times, uint32_t n_items, const uint32_t* __restrict__ item_off,
                                                   const uint32_t* __restrict__ item_edge, uint32_t* __restrict__ item_cnt,
                                                   typename Op::A* __restrict__ item_acc) {
  typedef typename Op::A A;
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  for (uint32_t it = warp; it < n_items; it += nwarps) {
    const uint32_t e = item_edge[it];
    const uint32_t first = (it - item_off[e]) * kTriChunk;                     // this item's slice of the walked list
    const int32_t x = G.src[e], y = G.dst[e];
    const float wxy = G.w[e];
    const uint32_t a0 = G.out_off[y], a1 = G.out_off[y + 1];                   // out(y): candidates z with s(y,z)
    const uint32_t b0 = G.in_off[x], b1 = G.in_off[x + 1];                     // in(x):  candidates z with t(z,x)
    const uint32_t la = a1 - a0, lb = b1 - b0;
    if (tri_bitmap_route(G, R, x, lb)) continue;                               // k_tri_bitmap's item
    uint32_t cnt = 0;
    A acc = Op::identity();
    const bool walk_a = la <= lb;
    const int32_t* wl = walk_a ? G.s_dst + a0 : G.in_src + b0;                  // walked list
    const int32_t* sl = walk_a ? G.in_src + b0 : G.s_dst + a0;                  // searched list
    const uint32_t nw = walk_a ? la : lb, ns = walk_a ? lb : la;
    const uint32_t last = min(first + kTriChunk, nw);
    // the walked list ascends, so whatever the last lane found in one sweep bounds every search of the next sweep
    uint32_t floor = 0;
    for (uint32_t i0 = first; i0 < last; i0 += 32) {
      const uint32_t i = i0 + lane;
      uint32_t lo = floor, hi = ns;
      int32_t z = 0;
      if (i < last) {
        z = wl[i];
        while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (sl[mid] < z) lo = mid + 1; else hi = mid; }
      }
      floor = __shfl_sync(0xffffffffu, lo, 31);
      if (i < last && lo < ns && sl[lo] == z) {
        const float wyz = walk_a ? G.s_w[a0 + i] : G.s_w[a0 + lo];
        const float wzx = walk_a ? G.in_w[b0 + lo] : G.in_w[b0 + i];
        const float t = times ? (wxy * wyz) * wzx : (wxy + wyz) + wzx;
        acc = Op::combine(acc, Op::lift(t));
        ++cnt;
      }
    }
    // most work items of a sparse graph end with no hit or with hits in one lane only: skip the combining tree for those
    const unsigned with_hits = __ballot_sync(0xffffffffu, cnt != 0u);
    if (with_hits == 0u) {
      if (lane == 0) { item_cnt[it] = 0u; item_acc[it] = Op::identity(); }
      continue;
    }
    if ((with_hits & (with_hits - 1u)) == 0u) {
      if (cnt) { item_cnt[it] = cnt; item_acc[it] = acc; }
      continue;
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
      cnt += __shfl_down_sync(0xffffffffu, cnt, d);
      const A o = shfl_down(acc, d);
      acc = Op::combine(acc, o);
    }
    if (lane == 0) { item_cnt[it] = cnt; item_acc[it] = acc; }
  }
}

// Units of the bitmap kernel: the work items of one x in slices of kTriUnitItems.  units[x] for x < domain, units[domain] = 0.
static __global__ void __launch_bounds__(256) k_tri_unit_count(TriGraph G, TriRoute R, const uint32_t* __restrict__ edge_off, int64_t domain,
                                                               const uint32_t* __restrict__ item_off, uint32_t* __restrict__ units) {
  for (int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; x <= domain; x += (int64_t)gridDim.x * blockDim.x) {
    uint32_t n = 0;
    if (x < domain && x < G.in_domain) {
      const uint32_t lb = G.in_off[x + 1] - G.in_off[x];
      if (lb && tri_bitmap_route(G, R, (int32_t)x, lb)) n = (item_off[edge_off[x + 1]] - item_off[edge_off[x]] + kTriUnitItems - 1) / kTriUnitItems;
    }
    units[x] = n;
  }
}

// unit -> (x, first item), written by the x (unit_off = exclusive scan of units)
static __global__ void __launch_bounds__(256) k_tri_unit_fill(const uint32_t* __restrict__ edge_off, int64_t domain, const uint32_t* __restrict__ item_off,
                                                              const uint32_t* __restrict__ unit_off, uint2* __restrict__ unit) {
  for (int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; x < domain; x += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t u0 = unit_off[x], u1 = unit_off[x + 1];
    const uint32_t first = item_off[edge_off[x]];
    for (uint32_t u = u0; u < u1; ++u) unit[u] = make_uint2((uint32_t)x, first + (u - u0) * kTriUnitItems);
  }
}

// One block per unit: mark in(x), then the block's warps walk the unit's work items (slices of the out-lists of x's
// neighbours) against the bitmap, warp w taking items w, w + 8, ...  Hits are rare among the walked entries (one in ten),
// so a warp does not combine them where they fall: it queues them in shared memory, in entry order, and reads their tags
// and folds them 32 at a time, a lane each.  A warp's partial result covers all its items of the unit; it is written to the first of them, the
// others get the identity (the per-x combination that follows reads every item of x anyway).  The assignment of entries to
// lanes depends on the graph alone, so results repeat from run to run.  Dynamic shared memory: 2 * words * 4 bytes (bits,
// then, per word, the place in in(x) of the first entry marked in it).
template <typename Op>
__global__ void __launch_bounds__(256) k_tri_bitmap(TriGraph G, int times, uint32_t n_units, const uint2* __restrict__ unit, const uint32_t* __restrict__ edge_off,
                                                    const uint32_t* __restrict__ item_off, const uint32_t* __restrict__ item_edge, uint32_t words,
                                                    uint32_t* __restrict__ item_cnt, typename Op::A* __restrict__ item_acc) {
  typedef typename Op::A A;
  extern __shared__ uint32_t tri_smem[];
  __shared__ uint32_t s_queue[8][32 * kTriBitmapUnroll + 32];      // a group's hits plus what an earlier group left
  uint32_t* bits = tri_smem;
  uint32_t* before = tri_smem + words;
  const unsigned lane = lane_id(), wid = warp_id();
  uint32_t* queue = s_queue[wid];
  int32_t have = -1;                                                         // the x whose in-list the bitmap holds
  for (uint32_t i = threadIdx.x; i < words; i += 256) bits[i] = 0u;
  for (uint32_t u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int32_t x = (int32_t)unit[u].x;
    const uint32_t b0 = G.in_off[x], b1 = G.in_off[x + 1];
    if (x != have) {
      __syncthreads();
      if (have >= 0) {                                                         // unmark the previous in-list: only the words it touched
        const uint32_t p0 = G.in_off[have], p1 = G.in_off[have + 1];
        for (uint32_t i = p0 + threadIdx.x; i < p1; i += 256) bits[(uint32_t)G.in_src[i] >> 5] = 0u;
        __syncthreads();
      }
      // in(x) ascends, so the entries that fall into one bitmap word are neighbours in the list: the entry that opens a word
      // notes its place there, and the place of any marked z is that plus the marked bits below z in its word
      for (uint32_t i = b0 + threadIdx.x; i < b1; i += 256) {
        const uint32_t z = (uint32_t)G.in_src[i];
        atomicOr(bits + (z >> 5), 1u << (z & 31));
        if (i == b0 || ((uint32_t)G.in_src[i - 1] >> 5) != (z >> 5)) before[z >> 5] = i - b0;
      }
      __syncthreads();
      have = x;
    }
    const uint32_t it_lo = unit[u].y, it_end = min(it_lo + kTriUnitItems, item_off[edge_off[x + 1]]);
    uint32_t cnt = 0;                                                          // hits so far (uniform across the warp)
    A acc = Op::identity();
    for (uint32_t it = it_lo + wid; it < it_end; it += 8) {
      const uint32_t e = item_edge[it];
      const uint32_t first = (it - item_off[e]) * kTriChunk;
      const int32_t y = G.dst[e];
      const float wxy = G.w[e];
      const uint32_t a0 = G.out_off[y], a1 = G.out_off[y + 1];
      const uint32_t last = min(first + kTriChunk, a1 - a0);
      if (it != it_lo + wid && lane == 0) { item_cnt[it] = 0u; item_acc[it] = Op::identity(); }
      uint32_t qn = 0;                                                         // queued hits of this item (uniform across the warp)
      // kTriBitmapUnroll sweeps at a time: their list reads are in flight together
      for (uint32_t i0 = first; i0 < last; i0 += 32 * kTriBitmapUnroll) {
        uint32_t z[kTriBitmapUnroll];
#pragma unroll
        for (int k = 0; k < kTriBitmapUnroll; ++k) {
          const uint32_t i = i0 + k * 32 + lane;
          z[k] = i < last ? (uint32_t)__ldcs(G.s_dst + a0 + i) : 0xffffffffu;
        }
        // bit tests of the eight sweeps without a branch; a lane's hits as a bit per sweep
        uint32_t wd[kTriBitmapUnroll];
        uint32_t hb = 0;
#pragma unroll
        for (int k = 0; k < kTriBitmapUnroll; ++k) {
          wd[k] = z[k] < words * 32u ? bits[z[k] >> 5] : 0u;
          hb |= ((wd[k] >> (z[k] & 31)) & 1u) << k;
        }
        if (__ballot_sync(0xffffffffu, hb != 0u) == 0u) continue;              // uniform: no hit in these sweeps
        // queue places: a warp-wide prefix over the lanes' hit counts; a hit is queued as (place of z in in(x), place of the
        // entry in this item's slice of out(y)) in one word: its two tags are read when the queue is folded
        const uint32_t mine = __popc(hb);
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d); if ((int)lane >= d) incl += o; }
        uint32_t at = qn + incl - mine;
        qn += __shfl_sync(0xffffffffu, incl, 31);
#pragma unroll
        for (int k = 0; k < kTriBitmapUnroll; ++k)
          if ((hb >> k) & 1u)
            queue[at++] = ((before[z[k] >> 5] + __popc(wd[k] & ((1u << (z[k] & 31)) - 1u))) << 10) | (i0 - first + k * 32 + lane);
        __syncwarp();
        while (qn >= 32) {                                                     // fold 32 queued hits, a lane each, from the queue's end
          const uint32_t h = queue[qn - 32 + lane];
          const float wyz = G.s_w[a0 + first + (h & 1023u)], wzx = G.in_w[b0 + (h >> 10)];
          acc = Op::combine(acc, Op::lift(times ? (wxy * wyz) * wzx : (wxy + wyz) + wzx));
          qn -= 32;
          cnt += 32;
        }
        __syncwarp();
      }
      if (lane < qn) {                                                         // what is left of this item's hits (the tag of (x,y) changes with the item)
        const uint32_t h = queue[lane];
        const float wyz = G.s_w[a0 + first + (h & 1023u)], wzx = G.in_w[b0 + (h >> 10)];
        acc = Op::combine(acc, Op::lift(times ? (wxy * wyz) * wzx : (wxy + wyz) + wzx));
      }
      cnt += qn;
      __syncwarp();
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
      const A o = shfl_down(acc, d);
      acc = Op::combine(acc, o);
    }
    if (lane == 0 && it_lo + wid < it_end) { item_cnt[it_lo + wid] = cnt; item_acc[it_lo + wid] = acc; }
  }
}

// Matches per edge (the count step of the materialising variant): one warp per edge.
static __global__ void __launch_bounds__(256) k_tri_count_edges(TriGraph G, uint32_t* __restrict__ edge_cnt) {
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  for (uint32_t e = warp; e < G.n_edges; e += nwarps) {
    const int32_t x = G.src[e], y = G.dst[e];
    uint32_t a0 = 0, a1 = 0, b0 = 0, b1 = 0;
    if (y < G.out_domain) { a0 = G.out_off[y]; a1 = G.out_off[y + 1]; }
    if (x < G.in_domain) { b0 = G.in_off[x]; b1 = G.in_off[x + 1]; }
    const uint32_t la = a1 - a0, lb = b1 - b0;
    uint32_t cnt = 0;
    if (la && lb) {
      const bool walk_a = la <= lb;
      const int32_t* wl = walk_a ? G.s_dst + a0 : G.in_src + b0;
      const int32_t* sl = walk_a ? G.in_src + b0 : G.s_dst + a0;
      const uint32_t nw = walk_a ? la : lb, ns = walk_a ? lb : la;
      uint32_t floor = 0;
      for (uint32_t i0 = 0; i0 < nw; i0 += 32) {
        const uint32_t i = i0 + lane;
        uint32_t lo = floor, hi = ns;
        int32_t z = 0;
        if (i < nw) {
          z = wl[i];
          while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (sl[mid] < z) lo = mid + 1; else hi = mid; }
        }
        floor = __shfl_sync(0xffffffffu, lo, 31);
        if (i < nw && lo < ns && sl[lo] == z) ++cnt;
      }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) cnt += __shfl_down_sync(0xffffffffu, cnt, d);
    if (lane == 0) edge_cnt[e] = cnt;
  }
}

// One warp per x: combine the partials of the work items of its edges (contiguous, in edge and slice order), write count,
// tag and a presence flag.
template <typename Op>
__global__ void __launch_bounds__(256) k_tri_groups(const uint32_t* __restrict__ out_off, int64_t domain, const uint32_t* __restrict__ item_off,
                                                    const uint32_t* __restrict__ edge_cnt, const typename Op::A* __restrict__ edge_acc,
                                                    uint32_t* __restrict__ grp_cnt, float* __restrict__ grp_tag,
                                                    uint32_t* __restrict__ flag, uint32_t* __restrict__ max_cnt,
                                                    uint32_t* __restrict__ err) {
  typedef typename Op::A A;
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  for (int64_t x = warp; x < domain; x += nwarps) {
    const uint32_t e0 = item_off[out_off[x]], e1 = item_off[out_off[x + 1]];
    uint64_t cnt = 0;
    A acc = Op::identity();
    for (uint32_t e = e0 + lane; e < e1; e += 32) {
      cnt += edge_cnt[e];
      acc = Op::combine(acc, edge_acc[e]);
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
      cnt += __shfl_down_sync(0xffffffffu, cnt, d);
      const A o = shfl_down(acc, d);
      acc = Op::combine(acc, o);
    }
    if (lane == 0) {
      if (cnt > 0x7fffffffull) { atomicOr(err, kErrCountOverflow); cnt = 0x7fffffffull; }
      grp_cnt[x] = (uint32_t)cnt;
      grp_tag[x] = cnt ? Op::lower(acc) : 0.f;
      flag[x] = cnt ? 1u : 0u;
      if (cnt) atomicMax(max_cnt, (uint32_t)cnt);
    }
  }
}

// Materialising variant  tri(x,y,z) :- e(x,y), e(y,z), e(z,x)  (paper: "Worst-case-optimal joins": count ->
// device prefix scan -> materialise over flat sorted-column storage).  edge_off = exclusive scan of the
// per-edge match counts.  One warp per edge walks the shorter list in order, 32 entries at a time; a
// ballot ranks the hits, so an edge's rows come out in increasing z and the whole output is already
// sorted by (x,y,z) and duplicate-free: no sort, no reduce.
template <typename K>
__global__ void __launch_bounds__(256) k_tri_materialise(TriGraph G, int times, const uint64_t* __restrict__ edge_off, KeyLayout L,
                                                         K* __restrict__ out_keys, float* __restrict__ out_tags) {
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  for (uint32_t e = warp; e < G.n_edges; e += nwarps) {
    const int32_t x = G.src[e], y = G.dst[e];
    const float wxy = G.w[e];
    uint32_t a0 = 0, a1 = 0, b0 = 0, b1 = 0;
    if (y < G.out_domain) { a0 = G.out_off[y]; a1 = G.out_off[y + 1]; }
    if (x < G.in_domain) { b0 = G.in_off[x]; b1 = G.in_off[x + 1]; }
    const uint32_t la = a1 - a0, lb = b1 - b0;
    if (!la || !lb) continue;
    const bool walk_a = la <= lb;
    const int32_t* wl = walk_a ? G.s_dst + a0 : G.in_src + b0;
    const int32_t* sl = walk_a ? G.in_src + b0 : G.s_dst + a0;
    const uint32_t nw = walk_a ? la : lb, ns = walk_a ? lb : la;
    uint64_t pos = edge_off[e];
    const K xy = ((K)(uint32_t)x << L.shift[0]) | ((K)(uint32_t)y << L.shift[1]);
    uint32_t floor = 0;                                   // see k_tri_edges
    for (uint32_t i0 = 0; i0 < nw; i0 += 32) {
      const uint32_t i = i0 + lane;
      bool hit = false;
      int32_t z = 0;
      uint32_t lo = floor;
      if (i < nw) {
        z = wl[i];
        uint32_t hi = ns;
        while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (sl[mid] < z) lo = mid + 1; else hi = mid; }
        hit = lo < ns && sl[lo] == z;
      }
      floor = __shfl_sync(0xffffffffu, lo, 31);
      const unsigned m = __ballot_sync(0xffffffffu, hit);
      if (hit) {
        const float wyz = walk_a ? G.s_w[a0 + i] : G.s_w[a0 + lo];
        const float wzx = walk_a ? G.in_w[b0 + lo] : G.in_w[b0 + i];
        const uint64_t o = pos + __popc(m & lanemask_lt());
        out_keys[o] = xy | ((K)(uint32_t)z << L.shift[2]);
        out_tags[o] = times ? (wxy * wyz) * wzx : (wxy + wyz) + wzx;
      }
      pos += __popc(m);
    }
  }
}

// Keep the x that have at least one triangle: pos = exclusive scan of flag.
template <typename K>
__global__ void __launch_bounds__(256) k_tri_compact(const uint32_t* __restrict__ flag, const uint32_t* __restrict__ pos, int64_t domain,
                                                     const uint32_t* __restrict__ grp_cnt, const float* __restrict__ grp_tag,
                                                     K* __restrict__ keys, uint32_t* __restrict__ counts, float* __restrict__ tags) {
  for (int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; x < domain; x += (int64_t)gridDim.x * blockDim.x)
    if (flag[x]) { const uint32_t p = pos[x]; keys[p] = (K)x; counts[p] = grp_cnt[x]; tags[p] = grp_tag[x]; }
}

// ---- the binary-join plan of the same query (paper: "WCOJ vs. the binary-join plan") -------------------------------
// Step one materialises every two-path (x,y,z) of the first two atoms with the ordinary join kernels; step two, here,
// keeps the paths that the closing atom closes: one thread per path looks (last column, x) up in the closing relation's
// store (offsets over its column 0, then a binary search in the run's sorted column 1).  count -> scan -> emit, in
// input order, so the output is sorted by (x,y,z) like the worst-case-optimal path's.
struct ChainProbe {
  int last;                      // index of the path's last column: 2 for the two-paths (x,y,z) of the triangle, 3 for the three-paths of the four-cycle
  KeyLayout L;                   // layout of the path keys (x,y,z[,w]): wide enough for everything the joined atoms hold
  KeyLayout out;                 // layout of the head relation (its bounds take t into account as well)
  int64_t t_domain;
  const uint32_t* t_off;         // offsets over the third relation's column 0
  const int32_t* t_col1;         // its column 1, ascending inside each run
  const float* t_w;
  int times;
};

template <typename K>
__device__ __forceinline__ bool chain_lookup(const ChainProbe& P, K key, uint32_t& pos) {
  const int32_t x = key_col<K>(P.L, key, 0), z = key_col<K>(P.L, key, P.last);
  if (z >= P.t_domain) return false;
  uint32_t lo = P.t_off[z];
  const uint32_t end = P.t_off[z + 1];
  uint32_t hi = end;
  while (lo < hi) { const uint32_t mid = lo + ((hi - lo) >> 1); if (P.t_col1[mid] < x) lo = mid + 1; else hi = mid; }
  pos = lo;
  return lo < end && P.t_col1[lo] == x;
}

template <typename K>
__global__ void __launch_bounds__(256) k_chain_probe_count(ChainProbe P, const K* __restrict__ keys, uint64_t n, uint32_t* __restrict__ hit) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    uint32_t pos;
    hit[i] = chain_lookup<K>(P, keys[i], pos) ? 1u : 0u;
  }
}

template <typename K, typename KH>
__global__ void __launch_bounds__(256) k_chain_probe_emit(ChainProbe P, const K* __restrict__ keys, const float* __restrict__ tags, uint64_t n,
                                                          const uint32_t* __restrict__ hit, const uint64_t* __restrict__ off,
                                                          KH* __restrict__ out_keys, float* __restrict__ out_tags) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    if (!hit[i]) continue;
    uint32_t pos = 0;
    chain_lookup<K>(P, keys[i], pos);
    const float w = P.t_w[pos];
    KH hk = 0;
#pragma unroll
    for (int col = 0; col < kMaxArity; ++col)
      if (col <= P.last) hk |= (KH)(uint32_t)key_col<K>(P.L, keys[i], col) << P.out.shift[col];
    out_keys[off[i]] = hk;
    out_tags[off[i]] = P.times ? tags[i] * w : tags[i] + w;
  }
}

}  // namespace xlog
