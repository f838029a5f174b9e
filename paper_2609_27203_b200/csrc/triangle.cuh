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

// Work items of the aggregate: an edge whose shorter list has n entries is cut into ceil(n / kTriChunk) items, so that a
// hub edge (tens of thousands of entries to walk) is shared by many warps instead of serialising one; an edge with an
// empty list gets none.  items[e] for e < n_edges, items[n_edges] = 0 (so that the exclusive scan has n_edges + 1 entries).
// *walked accumulates the total number of entries to walk (one sorted-list probe each).
static __global__ void __launch_bounds__(256) k_tri_plan(TriGraph G, uint32_t* __restrict__ items, unsigned long long* __restrict__ walked) {
  unsigned long long mine = 0;
  for (uint32_t e = blockIdx.x * blockDim.x + threadIdx.x; e <= G.n_edges; e += gridDim.x * blockDim.x) {
    uint32_t n = 0;
    if (e < G.n_edges) {
      const int32_t x = G.src[e], y = G.dst[e];
      uint32_t la = 0, lb = 0;
      if (y < G.out_domain) la = G.out_off[y + 1] - G.out_off[y];
      if (x < G.in_domain) lb = G.in_off[x + 1] - G.in_off[x];
      n = (min(la, lb) + kTriChunk - 1) / kTriChunk;
      mine += min(la, lb);
    }
    items[e] = n;
  }
#pragma unroll
  for (int d = 16; d; d >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, d);
  if (lane_id() == 0 && mine) atomicAdd(walked, mine);
}

// item -> edge, written by the edge (item_off = exclusive scan of items)
static __global__ void __launch_bounds__(256) k_tri_item_edges(uint32_t n_edges, const uint32_t* __restrict__ item_off, uint32_t* __restrict__ item_edge) {
  for (uint32_t e = blockIdx.x * blockDim.x + threadIdx.x; e < n_edges; e += gridDim.x * blockDim.x)
    for (uint32_t it = item_off[e]; it < item_off[e + 1]; ++it) item_edge[it] = e;
}

// One warp per work item: partial count and aggregate of its slice of the walked list.
template <typename Op>
__global__ void __launch_bounds__(256) k_tri_edges(TriGraph G, int times, uint32_t n_items, const uint32_t* __restrict__ item_off,
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
#pragma unroll
    for (int d = 16; d; d >>= 1) {
      cnt += __shfl_down_sync(0xffffffffu, cnt, d);
      const A o = shfl_down(acc, d);
      acc = Op::combine(acc, o);
    }
    if (lane == 0) { item_cnt[it] = cnt; item_acc[it] = acc; }
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
