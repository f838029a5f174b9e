// Grouped join driven by the changed bitmap, for the rule shape  h(a, c) :- h(a, b), r(b, c)  over a tag mirror whose
// index is (probed column b, carried column a) with at least 32 slots per value of b (group_join.cuh explains the
// layout).  A word of the changed bitmap then covers 32 consecutive carried values of ONE b: a "unit".  The delta of a
// round (Algorithm 1 line 5) is never written out as a row list:
//
//   k_bm_plan    reads the bitmap once.  For every non-zero word: clears it, settles which of its keys are new (against
//                the bitmap of keys the relation holds), copies the unit's 32 tags into a snapshot table (the tags as
//                they stood when the round began: the join below runs while other warps lower the live table), and
//                cuts r's run of b into slices of kBmSlice neighbours, one work item {word, mask, first row, rows} each.
//                Blocks reserve item room with one atomic add, so the item order varies from run to run; nothing
//                that is derived depends on it.  Totals (changed keys, new keys, candidates, items, neighbour rows
//                read) are accumulated in five counters.
//   k_bm_expand  a warp per item: lane l owns carried value 32 * chunk + l.  32 neighbours at a time are read coalesced
//                and handed round with shuffles; per neighbour c the warp reads the 32 slots (c, .) of the unit's chunk in
//                one 128-byte access, lanes whose bit is set in the mask compare their candidate with the slot, and
//                the improving ones issue the atomic min / max; one lane ORs the ballot of improving lanes into the
//                changed bitmap (lane number = bit number).
//
// Against the row-list form (k_join_count_flags ... k_seg_expand) this drops the delta list, its count / scan / segment
// passes and the per-candidate row arithmetic; what is left per neighbour is two shuffles, a shift-add, the slot read,
// an add, the order map, a compare and a vote.
#pragma once
#include "common.cuh"
#include "join.cuh"

namespace xlog {

constexpr int kBmSlice = 256;                     // neighbours per work item
constexpr int kBmPlanBlock = 256;
constexpr int kBmPlanSweeps = 4;                  // bitmap words per thread
constexpr int kBmPlanTile = kBmPlanBlock * kBmPlanSweeps;
constexpr int kBmSmallItems = 2;                  // a word with more items than this is expanded by the whole block

enum { kBmChanged = 0, kBmNew = 1, kBmCandidates = 2, kBmItems = 3, kBmNeighbours = 4, kBmTotals = 5 };

struct BmPlan {
  uint32_t* words;                 // changed bitmap, nwords words; cleared as it is read
  uint32_t* present;               // bitmap of the keys the relation holds
  uint32_t nwords;
  const int32_t* table;            // live tag mirror
  int32_t* snap;                   // same size: the tags of the units that changed, as of the start of the round
  int unit_shift;                  // word index >> unit_shift = value of the probed column (log2 of words per value)
  const uint32_t* off;             // offsets of the looked-up relation over its probed column
  uint32_t domain;                 // off has domain + 1 entries
  uint4* items;                    // out: {word, mask, first row of the slice, rows in the slice}
  unsigned long long* totals;      // kBmTotals counters, zeroed by the caller
};

static __global__ void __launch_bounds__(kBmPlanBlock) k_bm_plan(BmPlan P) {
  __shared__ uint32_t sh[kBmPlanBlock / 32 + 1];
  __shared__ uint32_t s_base;
  __shared__ uint32_t s_nact, s_nbig;
  __shared__ uint32_t s_act[kBmPlanTile];          // active words of the tile
  __shared__ uint4 s_big[kBmPlanTile];             // {word, mask, first row, degree} of words with many items; .x reused
  __shared__ uint32_t s_big_base[kBmPlanTile];
  if (threadIdx.x == 0) { s_nact = 0; s_nbig = 0; }
  __syncthreads();
  uint32_t m[kBmPlanSweeps], lo[kBmPlanSweeps], dg[kBmPlanSweeps], nit[kBmPlanSweeps];
  uint32_t my_items = 0, changed = 0, fresh = 0;
  unsigned long long cand = 0, nbrs = 0;
#pragma unroll
  for (int j = 0; j < kBmPlanSweeps; ++j) {
    const uint32_t wi = (blockIdx.x * kBmPlanSweeps + j) * kBmPlanBlock + threadIdx.x;
    m[j] = wi < P.nwords ? P.words[wi] : 0u;
    lo[j] = dg[j] = nit[j] = 0;
    if (m[j]) {
      P.words[wi] = 0u;
      const uint32_t had = P.present[wi];
      const uint32_t nw = m[j] & ~had;
      if (nw) P.present[wi] = had | m[j];
      fresh += __popc(nw);
      changed += __popc(m[j]);
      const uint32_t b = wi >> P.unit_shift;
      if (b < P.domain) { lo[j] = P.off[b]; dg[j] = P.off[b + 1] - lo[j]; }
      nit[j] = (dg[j] + kBmSlice - 1) / kBmSlice;
      my_items += nit[j];
      cand += (unsigned long long)__popc(m[j]) * dg[j];
      nbrs += dg[j];
      s_act[atomicAdd(&s_nact, 1u)] = wi;
    }
  }
  uint32_t tile_items;
  uint32_t pos = block_scan_excl<kBmPlanBlock, uint32_t>(my_items, sh, tile_items);
  if (threadIdx.x == 0 && tile_items) s_base = (uint32_t)atomicAdd(P.totals + kBmItems, (unsigned long long)tile_items);
  __syncthreads();
  // items: a word with few items is written by its own thread, one with many by the whole block
#pragma unroll
  for (int j = 0; j < kBmPlanSweeps; ++j) {
    if (!nit[j]) continue;
    const uint32_t wi = (blockIdx.x * kBmPlanSweeps + j) * kBmPlanBlock + threadIdx.x;
    if (nit[j] <= kBmSmallItems) {
      for (uint32_t s = 0; s < nit[j]; ++s)
        P.items[s_base + pos + s] = make_uint4(wi, m[j], lo[j] + s * kBmSlice, min((uint32_t)kBmSlice, dg[j] - s * kBmSlice));
    } else {
      const uint32_t k = atomicAdd(&s_nbig, 1u);
      s_big[k] = make_uint4(wi, m[j], lo[j], dg[j]);
      s_big_base[k] = s_base + pos;
    }
    pos += nit[j];
  }
  __syncthreads();
  for (uint32_t k = 0; k < s_nbig; ++k) {
    const uint4 g = s_big[k];
    const uint32_t n = (g.w + kBmSlice - 1) / kBmSlice, base = s_big_base[k];
    for (uint32_t s = threadIdx.x; s < n; s += kBmPlanBlock)
      P.items[base + s] = make_uint4(g.x, g.y, g.z + s * kBmSlice, min((uint32_t)kBmSlice, g.w - s * kBmSlice));
  }
  // snapshot: the 32 tags of every active word, one 128-byte line per warp step
  const uint32_t nact = s_nact;
  for (uint32_t k = warp_id(); k < nact; k += kBmPlanBlock / 32) {
    const size_t at = (size_t)s_act[k] * 32 + lane_id();
    P.snap[at] = __ldcg(P.table + at);
  }
  // totals: one atomic per warp and counter
  changed = __reduce_add_sync(0xffffffffu, changed);
  fresh = __reduce_add_sync(0xffffffffu, fresh);
#pragma unroll
  for (int s = 16; s; s >>= 1) { cand += __shfl_down_sync(0xffffffffu, cand, s); nbrs += __shfl_down_sync(0xffffffffu, nbrs, s); }
  if (lane_id() == 0 && changed) {
    atomicAdd(P.totals + kBmChanged, (unsigned long long)changed);
    if (fresh) atomicAdd(P.totals + kBmNew, (unsigned long long)fresh);
    if (cand) atomicAdd(P.totals + kBmCandidates, cand);
    if (nbrs) atomicAdd(P.totals + kBmNeighbours, nbrs);
  }
}

struct BmExpand {
  const uint4* items;
  uint32_t n_items;
  const int32_t* z;                // looked-up relation's other column, in index order
  const float* w;                  // its tags
  uint32_t z_max;                  // largest value the head's second column may take
  int carried_bits;                // slot = (z << carried_bits) + 32 * chunk + lane
  const int32_t* snap;
  int32_t* table;
  uint32_t* changed;
  uint32_t* err;
};

template <int SINK>
__global__ void __launch_bounds__(256, 8) k_bm_expand(BmExpand E) {
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  const uint32_t chunk_mask = (1u << (E.carried_bits - 5)) - 1u;
  const int32_t never = SINK == kSinkMin ? (int32_t)0x80000000 : 0x7fffffff;       // no candidate improves on this
  uint32_t e = 0;
  for (uint32_t it = warp; it < E.n_items; it += nwarps) {
    const uint4 item = E.items[it];                      // word, mask, first row, rows
    const bool mine = (item.y >> lane) & 1u;
    const uint32_t sub = ((item.x & chunk_mask) << 5) + lane;
    const float t = mine ? ord2f(__ldcg(E.snap + (size_t)item.x * 32 + lane)) : 0.f;
    for (uint32_t jb = 0; jb < item.w; jb += 32) {
      const uint32_t nj = min(32u, item.w - jb);
      uint32_t zr = 0;
      float wr = 0.f;
      if (lane < nj) {
        zr = (uint32_t)__ldcs(E.z + item.z + jb + lane);
        wr = __ldcs(E.w + item.z + jb + lane);
        if (zr > E.z_max) { e |= kErrHeadRange; zr = E.z_max; }      // the fixpoint fails; keep the access in range
      }
      for (uint32_t s0 = 0; s0 < nj; s0 += 4) {
        uint32_t key[4];
        int32_t v[4], cur[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t z = __shfl_sync(0xffffffffu, zr, (s0 + u) & 31);
          const float w = __shfl_sync(0xffffffffu, wr, (s0 + u) & 31);
          key[u] = (z << E.carried_bits) + sub;
          v[u] = f2ord(t + w);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          cur[u] = never;
          if (mine && s0 + u < nj) cur[u] = XLOG_TABLE_LOAD(E.table + key[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const bool better = SINK == kSinkMin ? v[u] < cur[u] : v[u] > cur[u];
          if (better) { if (SINK == kSinkMin) atomicMin(E.table + key[u], v[u]); else atomicMax(E.table + key[u], v[u]); }
          const unsigned bal = __ballot_sync(0xffffffffu, better);
          if (bal && lane == 0) atomicOr(E.changed + (key[u] >> 5), bal);
        }
      }
    }
  }
  if (e) atomicOr(E.err, e);
}

}  // namespace xlog
