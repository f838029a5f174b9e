// Grouped join into a tag mirror, for the rule shape  h(a, c) :- h(a, b), r(b, c)  (transitive closure,
// multi-source reachability): many delta rows share the probed value b and differ only in the carried column a.
//
// The mirror of such a relation is addressed with the probed column as the major part of the index and the
// carried column as the minor part, so (1) the delta, which is the changed bitmap read in index order, comes out
// grouped by b, and (2) the slots of (a_1, c), (a_2, c), ... lie next to each other.  A segment = the delta rows of one
// b (k rows) joined with r's run of b (d rows) = k * d candidates.  A warp keeps the k rows in its lanes and walks the
// d neighbours: one read of r's run serves all k rows, and the lanes of a step touch consecutive slots (a few sectors
// instead of one per candidate).
//
//   k_join_count_flags  the join's count step, plus where a delta row starts a new segment and the candidate total
//   k_seg_first         first row of every segment
//   k_seg_items / k_seg_item_fill / k_seg_expand   work items (slices of a segment's neighbours) and the join itself
#pragma once
#include "common.cuh"
#include "join.cuh"

namespace xlog {

// Count step of the grouped join: the row's degree and count record as in k_join_count, plus flags[i] = 1 where row i
// starts a new segment (the index bits above the carried bits change) and the sum of all degrees (= candidates).
template <typename KO>
__global__ void __launch_bounds__(256) k_join_count_flags(JoinSpec S, const KO* __restrict__ okeys, const float* __restrict__ otags, uint32_t n_outer,
                                                          int carried_bits, uint32_t* __restrict__ deg, uint4* __restrict__ rowinfo,
                                                          uint32_t* __restrict__ flags, unsigned long long* __restrict__ total, uint32_t* __restrict__ err) {
  unsigned long long d = 0;                              // a grid-stride loop, so that the total costs one atomic per warp
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_outer; i += gridDim.x * blockDim.x) {
    const uint32_t di = join_count_row<KO>(S, okeys, otags, i, rowinfo, err);
    deg[i] = di;
    d += di;
    flags[i] = (i == 0 || (okeys[i] >> carried_bits) != (okeys[i - 1] >> carried_bits)) ? 1u : 0u;
  }
#pragma unroll
  for (int s = 16; s; s >>= 1) d += __shfl_down_sync(0xffffffffu, d, s);
  if (lane_id() == 0 && d) atomicAdd(total, d);
}

// seg_first[a] = first row of segment a (n_seg + 1 entries, the last one = n); idx = exclusive scan of flags
static __global__ void __launch_bounds__(256) k_seg_first(const uint32_t* __restrict__ flags, const uint32_t* __restrict__ idx, uint32_t n,
                                                         uint32_t n_seg, uint32_t* __restrict__ seg_first) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i <= n; i += gridDim.x * blockDim.x) {
    if (i == n) seg_first[n_seg] = n;
    else if (flags[i]) seg_first[idx[i]] = i;
  }
}

// ---- a warp takes a slice of one segment's neighbours and keeps the delta rows in its lanes ------------------------------
// For segments with many candidates (k rows x d neighbours) the per-candidate work shrinks to two shuffles, a
// multiply-add, the slot read and a compare: lanes hold the rows (k' = k rounded up to a power of two, 32 / k' neighbours
// per step), 32 neighbours at a time are read coalesced into registers and handed round with shuffles.
// An item = (segment, slice of seg_slice(k) neighbours); seg_slice keeps k * slice near 4096 candidates.
__host__ __device__ __forceinline__ uint32_t seg_slice(uint32_t rows) {
  const uint32_t s = 4096u / (rows < 1u ? 1u : rows);
  return s < 32u ? 32u : (s & ~31u);
}

// *neighbours accumulates the looked-up rows read by the join (one run per segment, whatever its number of delta rows)
static __global__ void __launch_bounds__(256) k_seg_items(const uint32_t* __restrict__ seg_first, uint32_t n_seg, const uint32_t* __restrict__ deg,
                                                         uint32_t* __restrict__ items, unsigned long long* __restrict__ neighbours) {
  unsigned long long mine = 0;
  for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g <= n_seg; g += gridDim.x * blockDim.x) {
    uint32_t n = 0;
    if (g < n_seg) {
      const uint32_t f = seg_first[g];
      const uint32_t sl = seg_slice(seg_first[g + 1] - f), dg = deg[f];      // a segment without matches gets no item
      n = (dg + sl - 1) / sl;
      mine += dg;
    }
    items[g] = n;                                        // items[n_seg] = 0: the scan then has n_seg + 1 entries
  }
#pragma unroll
  for (int s = 16; s; s >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, s);
  if (lane_id() == 0 && mine) atomicAdd(neighbours, mine);
}
static __global__ void __launch_bounds__(256) k_seg_item_fill(uint32_t n_seg, const uint32_t* __restrict__ item_off, uint32_t* __restrict__ item_seg) {
  for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g < n_seg; g += gridDim.x * blockDim.x)
    for (uint32_t it = item_off[g]; it < item_off[g + 1]; ++it) item_seg[it] = g;
}

template <int SINK>
__global__ void __launch_bounds__(256, 8) k_seg_expand(JoinSpec S, uint32_t n_items, const uint32_t* __restrict__ item_off, const uint32_t* __restrict__ item_seg,
                                                    const uint32_t* __restrict__ seg_first, const uint32_t* __restrict__ deg,
                                                    const uint4* __restrict__ rowinfo, MirrorArgs mr) {
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  const float* __restrict__ itg = S.inner_tag;
  const int32_t* __restrict__ ic0 = S.inner_col[0];
  const uint32_t m0 = (uint32_t)S.inner_mult[0];
  uint32_t e = 0;
  for (uint32_t it = warp; it < n_items; it += nwarps) {
    const uint32_t g = item_seg[it];
    const uint32_t f = seg_first[g], rows = seg_first[g + 1] - f;
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
