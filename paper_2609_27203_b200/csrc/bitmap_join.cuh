// Grouped join driven by the changed bitmap, for the rule shape  h(a, c) :- h(a, b), r(b, c)  over a tag mirror whose
// index is (probed column b, carried column a) with 32 to 1024 slots per value of b (group_join.cuh explains the
// layout).  The changed bitmap then holds W = slots / 32 whole words per value of b, and a round (Algorithm 1 lines
// 5-9) is two kernels:
//
//   k_bm_plan    reads the bitmap once.  For every b with a changed key: clears its words, settles which keys are new
//                (against the bitmap of keys the relation holds), writes the changed keys of b as (tag, a) pairs, in
//                key order, to a dense list (the tags as they stood when the round began: the join runs while other
//                warps lower the live table), and cuts the work into items {first neighbour row, neighbours | keys of
//                the pass, first pair of the pass}: r's run of b in slices of kBmSlice neighbours, times ceil(k / 32)
//                passes over the k changed keys of b.  A block reserves its list room with one atomic add, so the
//                order of items and of pair runs varies from run to run; nothing derived depends on it.
//                Totals (changed keys, new keys, candidates, items, neighbour rows read) go to counters.
//   k_bm_expand  a warp per item.  The lanes take the pass's k keys (k rounded up to a power of two k'), so one step of
//                the warp covers 32 / k' neighbours.  32 neighbours at a time are read coalesced and staged in shared
//                memory; per candidate: one broadcast read of (neighbour's slot base, weight), the slot read, an add,
//                the order map, a compare, and for the few that improve the atomic min / max and the bit in the changed
//                bitmap.
//
// Against the row-list form (k_join_count_flags ... k_seg_expand) this drops the delta row list with its count / scan /
// segment passes (about a hundred launches per fixpoint on the 64-source reachability workload) and most of the per-item
// and per-candidate index arithmetic.
#pragma once
#ifndef XLOG_BM_BLOCKS
#define XLOG_BM_BLOCKS 8         // resident blocks per SM of the join kernel (32 registers per thread)
#endif
#include "common.cuh"
#include "join.cuh"

namespace xlog {

constexpr int kBmSlice = 256;                     // neighbours per work item
constexpr int kBmPlanBlock = 256;
constexpr int kBmPlanSweeps = 4;                  // bitmap words per thread
constexpr int kBmPlanTile = kBmPlanBlock * kBmPlanSweeps;
constexpr int kBmMaxWordsLog2 = 5;                // at most 32 bitmap words (1024 slots) per value of the probed column
#ifndef XLOG_BM_UNROLL
#define XLOG_BM_UNROLL 4
#endif
constexpr int kBmUnroll = XLOG_BM_UNROLL;         // steps per group: slot reads a lane keeps in flight
constexpr uint32_t kBmSmallItems = 8;             // a b with more items than this has them written by its whole warp

// kBmReserve: room handed out so far, pairs in the low 32 bits and items in the high 32 bits (one atomic add per block)
enum { kBmChanged = 0, kBmNew = 1, kBmCandidates = 2, kBmReserve = 3, kBmNeighbours = 4, kBmTotals = 5 };

struct BmPlan {
  uint32_t* words;                 // changed bitmap, nwords words; cleared as it is read
  uint32_t* present;               // bitmap of the keys the relation holds
  uint32_t nwords;
  const int32_t* table;            // live tag mirror
  uint2* pairs;                    // out: (tag bits, carried value) of the changed keys, the keys of one b contiguous and ascending
  int words_log2;                  // log2 W
  const uint32_t* off;             // offsets of the looked-up relation over its probed column
  uint32_t domain;                 // off has domain + 1 entries
  uint4* items;                    // out: {first neighbour row, neighbours | keys of the pass << 16, first pair of the pass, b}
  unsigned long long* totals;      // kBmTotals counters, zeroed by the caller
};

__device__ __forceinline__ uint4 bm_item(uint32_t lo, uint32_t dg, uint32_t k, uint32_t first_pair, uint32_t slice, uint32_t pass, uint32_t b) {
  return make_uint4(lo + slice * kBmSlice, min((uint32_t)kBmSlice, dg - slice * kBmSlice) | (min(32u, k - pass * 32) << 16), first_pair + pass * 32, b);
}

// A block takes kBmPlanTile words (thread t: words t, t + 256, ... of the tile).  One block-wide prefix over (changed
// keys, items) in word order (two barriers) and one 64-bit atomic add reserve its room in the pair list and the item
// list; the changed keys are then staged in shared memory, half a tile at a time, so that the tag reads and the pair
// writes of the whole block are independent of one another and coalesced.
#ifndef XLOG_BM_PLAN_BLOCKS
#define XLOG_BM_PLAN_BLOCKS 6
#endif
static __global__ void __launch_bounds__(kBmPlanBlock, XLOG_BM_PLAN_BLOCKS) k_bm_plan(BmPlan P) {
  constexpr int NW = kBmPlanBlock / 32;
  constexpr int kHalf = kBmPlanSweeps / 2;
  __shared__ unsigned long long s_warp[kBmPlanSweeps * NW];      // (sweep, warp) totals, then their exclusive prefixes; pairs low, items high
  __shared__ unsigned long long s_base, s_tot;
  __shared__ uint16_t s_list[kHalf * kBmPlanBlock * 32];         // changed keys of half a tile: (sweep in half, thread, bit)
  const unsigned lane = lane_id(), wid = warp_id();
  const uint32_t W = 1u << P.words_log2, slot_mask = (32u << P.words_log2) - 1u;
  const uint32_t tile0 = blockIdx.x * kBmPlanTile;
  uint32_t m[kBmPlanSweeps], k[kBmPlanSweeps], lo[kBmPlanSweeps], dg[kBmPlanSweeps];
  unsigned long long incl[kBmPlanSweeps];
  uint32_t changed = 0, fresh = 0;
  unsigned long long cand = 0, nbrs = 0;
#pragma unroll
  for (int j = 0; j < kBmPlanSweeps; ++j) {
    const uint32_t wi = tile0 + j * kBmPlanBlock + threadIdx.x;
    m[j] = wi < P.nwords ? P.words[wi] : 0u;
  }
#pragma unroll
  for (int j = 0; j < kBmPlanSweeps; ++j) {
    const uint32_t wi = tile0 + j * kBmPlanBlock + threadIdx.x;
    if (m[j]) {
      P.words[wi] = 0u;
      const uint32_t had = P.present[wi];
      const uint32_t nw = m[j] & ~had;
      if (nw) P.present[wi] = had | m[j];
      fresh += __popc(nw);
      changed += __popc(m[j]);
    }
    // the W words of one b sit in W adjacent lanes: the b's changed keys
    uint32_t kk = __popc(m[j]);
    for (uint32_t d = 1; d < W; d <<= 1) kk += __shfl_xor_sync(0xffffffffu, kk, d);
    k[j] = kk;
    lo[j] = dg[j] = 0;
    if (kk && (lane & (W - 1)) == 0) {                   // the b's first word speaks for it
      const uint32_t b = wi >> P.words_log2;
      if (b < P.domain) { lo[j] = P.off[b]; dg[j] = P.off[b + 1]; }
    }
  }
#pragma unroll
  for (int j = 0; j < kBmPlanSweeps; ++j) {
    dg[j] -= lo[j];
    uint32_t nit = 0;
    if (dg[j]) {
      nit = ((dg[j] + kBmSlice - 1) / kBmSlice) * ((k[j] + 31) / 32);
      cand += (unsigned long long)k[j] * dg[j];
      nbrs += dg[j];
    }
    unsigned long long v = (unsigned long long)__popc(m[j]) | ((unsigned long long)nit << 32);
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const unsigned long long o = __shfl_up_sync(0xffffffffu, v, d); if ((int)lane >= d) v += o; }
    incl[j] = v;
    if (lane == 31) s_warp[j * NW + wid] = v;
  }
  __syncthreads();
  if (wid == 0) {
    // exclusive prefix over the (sweep, warp) totals in sweep-major order; their sum reserves the block's list room
    static_assert(kBmPlanSweeps * NW == 32, "one lane per (sweep, warp) total");
    const unsigned long long t = s_warp[lane];
    unsigned long long v = t;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const unsigned long long o = __shfl_up_sync(0xffffffffu, v, d); if ((int)lane >= d) v += o; }
    s_warp[lane] = v - t;
    // pairs (low half) never carry into the items (high half): a launch has fewer than 2^32 pairs
    if (lane == 31) { s_tot = v; s_base = v ? atomicAdd(P.totals + kBmReserve, v) : 0ull; }
  }
  __syncthreads();
  const uint32_t pair_base = (uint32_t)s_base, item_base = (uint32_t)(s_base >> 32);
  if ((uint32_t)s_tot == 0) return;                       // no changed key in this tile (uniform)
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    // the changed keys of sweeps [h * kHalf, (h + 1) * kHalf), staged at their position relative to the half's first pair
    const uint32_t half_first = (uint32_t)s_warp[h * kHalf * NW];
    const uint32_t n_half = (h == 0 ? (uint32_t)s_warp[kHalf * NW] : (uint32_t)s_tot) - half_first;
    if (n_half == 0) continue;                           // uniform
#pragma unroll
    for (int jj = 0; jj < kHalf; ++jj) {
      const int j = h * kHalf + jj;
      uint32_t bits = m[j];
      uint32_t p = (uint32_t)s_warp[j * NW + wid] + (uint32_t)incl[j] - __popc(bits) - half_first;
      while (bits) {
        const int bit = __ffs(bits) - 1;
        bits &= bits - 1;
        s_list[p++] = (uint16_t)((jj << 13) | (threadIdx.x << 5) | bit);
      }
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n_half; i += kBmPlanBlock) {
      const uint32_t id = s_list[i];
      const uint32_t key = ((tile0 + (h * kHalf + (id >> 13)) * kBmPlanBlock + ((id >> 5) & 255u)) << 5) + (id & 31u);
      P.pairs[pair_base + half_first + i] = make_uint2(__float_as_uint(ord2f(__ldcg(P.table + key))), key & slot_mask);
    }
    __syncthreads();
  }
#pragma unroll
  for (int j = 0; j < kBmPlanSweeps; ++j) {
    if (__ballot_sync(0xffffffffu, dg[j] != 0) == 0) continue;
    const uint32_t wi = tile0 + j * kBmPlanBlock + threadIdx.x;
    const unsigned long long ex = s_warp[j * NW + wid] + incl[j];       // inclusive position of this thread
    const uint32_t pair_pos = pair_base + (uint32_t)ex - __popc(m[j]);  // where this word's pairs begin: for a b's first word, the b's
    const uint32_t slices = (dg[j] + kBmSlice - 1) / kBmSlice, passes = (k[j] + 31) / 32;
    const uint32_t nit = dg[j] ? slices * passes : 0u;
    const uint32_t item_pos = item_base + (uint32_t)(ex >> 32) - nit;
    const uint32_t b = wi >> P.words_log2;
    if (nit && nit <= kBmSmallItems) {
      uint32_t at = item_pos;
      for (uint32_t pass = 0; pass < passes; ++pass)
        for (uint32_t s = 0; s < slices; ++s) P.items[at++] = bm_item(lo[j], dg[j], k[j], pair_pos, s, pass, b);
    }
    unsigned big = __ballot_sync(0xffffffffu, nit > kBmSmallItems);
    while (big) {
      const int src = __ffs(big) - 1;
      big &= big - 1;
      const uint32_t LO = __shfl_sync(0xffffffffu, lo[j], src), DG = __shfl_sync(0xffffffffu, dg[j], src), K = __shfl_sync(0xffffffffu, k[j], src);
      const uint32_t AT = __shfl_sync(0xffffffffu, item_pos, src), PP = __shfl_sync(0xffffffffu, pair_pos, src), B = __shfl_sync(0xffffffffu, b, src);
      const uint32_t SL = (DG + kBmSlice - 1) / kBmSlice, total = SL * ((K + 31) / 32);
      for (uint32_t i = lane; i < total; i += 32) P.items[AT + i] = bm_item(LO, DG, K, PP, i % SL, i / SL, B);
    }
  }
  // totals: one atomic per warp and counter
  changed = __reduce_add_sync(0xffffffffu, changed);
  fresh = __reduce_add_sync(0xffffffffu, fresh);
#pragma unroll
  for (int s = 16; s; s >>= 1) { cand += __shfl_down_sync(0xffffffffu, cand, s); nbrs += __shfl_down_sync(0xffffffffu, nbrs, s); }
  if (lane == 0 && changed) {
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
  int carried_bits;                // slot = (z << carried_bits) + carried value
  const uint2* pairs;
  int32_t* table;
  uint32_t* changed;
  uint32_t* err;
};

// One candidate: `slot` is the address of its slot in the table (zq = z << carried_bits is the slot's b part, the lane's
// carried value sits in the address already), v its order-mapped tag, cur what the slot held when read.  The few that
// improve issue the atomic and set the key's bit: word = (zq >> 5) + the lane's word offset, bit = the lane's own.
template <int SINK>
__device__ __forceinline__ void bm_apply(int32_t* slot, int32_t v, int32_t cur, uint32_t* changed, uint32_t zq, uint32_t word_off, uint32_t bit) {
  if (SINK == kSinkMin ? v < cur : v > cur) {
    if (SINK == kSinkMin) atomicMin(slot, v); else atomicMax(slot, v);
    atomicOr(changed + (zq >> 5) + word_off, bit);
  }
}

// The lanes take the pass's k keys; with k' <= 16 of them (k rounded up to a power of two) a step covers 32 / k'
// neighbours.  A batch of 32 neighbours is staged in shared memory as (z << carried_bits, w) and read back with one
// broadcast load per step; a group of kBmUnroll steps keeps that many slot reads per lane in flight.
template <int SINK>
__global__ void __launch_bounds__(256, XLOG_BM_BLOCKS) k_bm_expand(BmExpand E) {
  __shared__ uint2 s_nb[256 / 32][32];
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  uint2* nb = s_nb[warp_id()];
  const int32_t never = SINK == kSinkMin ? (int32_t)0x80000000 : 0x7fffffff;       // no candidate improves on this
  for (uint32_t it = warp; it < E.n_items; it += nwarps) {
    const uint4 item = E.items[it];                      // first neighbour row, neighbours | keys << 16, first pair, b
    const uint32_t n = item.y & 0xffffu, kp = item.y >> 16;
    const uint32_t kq = kp <= 1 ? 1u : 1u << (32 - __clz(kp - 1));       // kp rounded up to a power of two
    const uint32_t per = 32u / kq, row = lane & (kq - 1), jsub = lane / kq;
    const bool active = row < kp;
    uint32_t src = 0;
    float t = 0.f;
    if (active) { const uint2 p = E.pairs[item.z + row]; t = __uint_as_float(p.x); src = p.y; }
    int32_t* const tbase = E.table + src;
    const uint32_t bit = 1u << (src & 31), word_off = src >> 5;
    for (uint32_t jb = 0; jb < n; jb += 32) {
      const uint32_t nj = min(32u, n - jb);
      __syncwarp();
      if (lane < nj) {
        uint32_t zr = (uint32_t)__ldcs(E.z + item.x + jb + lane);
        const float wr = __ldcs(E.w + item.x + jb + lane);
        if (zr > E.z_max) { atomicOr(E.err, kErrHeadRange); zr = E.z_max; }      // the fixpoint fails; keep the access in range
        nb[lane] = make_uint2(zr << E.carried_bits, __float_as_uint(wr));
      }
      __syncwarp();
      uint32_t sb = jsub;
      // whole groups: every lane's neighbour exists
      for (; sb - jsub + kBmUnroll * per <= nj; sb += kBmUnroll * per) {
        uint2 q[kBmUnroll];
        int32_t cur[kBmUnroll];
#pragma unroll
        for (int u = 0; u < kBmUnroll; ++u) {
          q[u] = nb[sb + u * per];
          cur[u] = never;
          if (active) cur[u] = XLOG_TABLE_LOAD(tbase + q[u].x);
        }
#pragma unroll
        for (int u = 0; u < kBmUnroll; ++u)
          bm_apply<SINK>(tbase + q[u].x, f2ord(t + __uint_as_float(q[u].y)), cur[u], E.changed, q[u].x, word_off, bit);
      }
      for (; sb - jsub < nj; sb += per) {
        const uint2 q = nb[sb & 31];
        int32_t cur = never;
        if (active && sb < nj) cur = XLOG_TABLE_LOAD(tbase + q.x);
        bm_apply<SINK>(tbase + q.x, f2ord(t + __uint_as_float(q.y)), cur, E.changed, q.x, word_off, bit);
      }
    }
  }
}

}  // namespace xlog
