// Resident fixpoint rounds (Section "GPU-Native Symbolic Substrate": the iteration body of the
// semi-naive loop runs as a device-resident graph with fixed capacities, an overflow flag and no
// host reads inside the loop).  One round over a tag mirror (mirror.cuh) is a fixed sequence of
// launches whose sizes are read from a small state block in device memory:
//
//   per rule with a recursive atom:  k_res_count -> k_res_tile_sums -> k_res_spine -> k_res_apply
//                                    -> k_res_partition -> k_res_expand
//   then:                            k_mirror_changed_count -> k_res_round_end -> k_mirror_changed_emit
//
// Every kernel has a fixed grid and strides over however much work the state block announces, so the
// sequence can be captured once as the body of a CUDA-graph WHILE node; k_res_round_end decides whether
// the body runs again.  The host reads the state block once, after the loop.
#pragma once
#include <cuda_runtime.h>

#include "common.cuh"
#include "join.cuh"
#include "scan.cuh"

namespace xlog {

enum { kResOk = 0, kResCap = 1, kResOverflow = 2 };

struct ResState {
  uint32_t n_delta;                  // rows of the current delta
  uint32_t rounds;                   // rounds completed by the resident loop
  uint32_t max_rounds;               // rounds it may still complete before giving up
  uint32_t status;                   // kResOk / kResCap (round budget used up) / kResOverflow (a round needs more tiles than planned)
  uint32_t ntiles;                   // expand tiles of the rule being evaluated
  uint32_t max_tiles;                // capacity of the tile-row array
  unsigned long long total;          // candidates of the rule being evaluated
  unsigned long long round_cand;     // candidates of the running round so far
  unsigned long long candidates;     // candidates of all completed rounds
  unsigned long long new_seen;       // value of the mirror's new-tuple counter at the end of the last completed round
  unsigned long long n_new;          // new tuples / improved tags of all completed rounds
  unsigned long long n_improved;
};

static __global__ void k_res_init(ResState* st, uint32_t n_delta, uint32_t max_rounds, uint32_t max_tiles, unsigned long long new_seen) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    ResState s{};
    s.n_delta = n_delta; s.max_rounds = max_rounds; s.max_tiles = max_tiles; s.new_seen = new_seen;
    *st = s;
  }
}

template <typename KO>
__global__ void __launch_bounds__(256) k_res_count(JoinSpec S, const KO* __restrict__ okeys, const float* __restrict__ otags,
                                                   const ResState* __restrict__ st, uint32_t* __restrict__ deg, uint4* __restrict__ rowinfo,
                                                   uint32_t* __restrict__ err) {
  const uint32_t n = st->status == kResOk ? st->n_delta : 0;
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
    join_count_row<KO>(S, okeys, otags, i, deg, rowinfo, err);
}

static __global__ void __launch_bounds__(kScanBlock) k_res_tile_sums(const uint32_t* __restrict__ deg, const ResState* __restrict__ st,
                                                                     uint64_t* __restrict__ tile_sums) {
  __shared__ uint64_t sh[kScanBlock / 32 + 1];
  const uint32_t n = st->status == kResOk ? st->n_delta : 0;
  const uint32_t tiles = (n + kScanTile - 1) / kScanTile;
  for (uint32_t t = blockIdx.x; t < tiles; t += gridDim.x) {
    const uint32_t base = t * kScanTile;
    uint64_t s = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) {
      const uint32_t p = base + i * kScanBlock + threadIdx.x;
      if (p < n) s += deg[p];
    }
    uint64_t total;
    block_scan_excl<kScanBlock, uint64_t>(s, sh, total);
    if (threadIdx.x == 0) tile_sums[t] = total;
  }
}

// One block: exclusive scan of the tile sums in place; publishes the rule's candidate total and tile count.
static __global__ void __launch_bounds__(1024) k_res_spine(uint64_t* __restrict__ tile_sums, ResState* __restrict__ st) {
  __shared__ uint64_t sh[1024 / 32 + 1];
  const uint32_t n = st->status == kResOk ? st->n_delta : 0;
  const uint32_t tiles = (n + kScanTile - 1) / kScanTile;
  uint64_t carry = 0;
  for (uint32_t base = 0; base < tiles; base += 1024) {
    const uint32_t p = base + threadIdx.x;
    const uint64_t x = p < tiles ? tile_sums[p] : 0;
    uint64_t total;
    const uint64_t e = block_scan_excl<1024, uint64_t>(x, sh, total);
    if (p < tiles) tile_sums[p] = carry + e;
    carry += total;
  }
  if (threadIdx.x == 0) {
    const uint64_t nt = (carry + kExpTile - 1) / kExpTile;
    st->total = carry;
    if (nt > st->max_tiles) { st->status = kResOverflow; st->ntiles = 0; }
    else { st->ntiles = (uint32_t)nt; st->round_cand += carry; }
  }
}

static __global__ void __launch_bounds__(kScanBlock) k_res_apply(const uint32_t* __restrict__ deg, const ResState* __restrict__ st,
                                                                 const uint64_t* __restrict__ tile_base, uint64_t* __restrict__ start) {
  __shared__ uint64_t sh[kScanBlock / 32 + 1];
  const uint32_t n = st->status == kResOk ? st->n_delta : 0;
  const uint32_t tiles = (n + kScanTile - 1) / kScanTile;
  for (uint32_t t = blockIdx.x; t < tiles; t += gridDim.x) {
    const uint32_t base = t * kScanTile + threadIdx.x * kScanItems;
    uint64_t x[kScanItems];
    uint64_t s = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) { x[i] = base + i < n ? deg[base + i] : 0; s += x[i]; }
    uint64_t total;
    uint64_t run = block_scan_excl<kScanBlock, uint64_t>(s, sh, total) + tile_base[t];
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) { if (base + i < n) start[base + i] = run; run += x[i]; }
  }
}

// first and last outer row of every expand tile (see k_expand_partition)
static __global__ void __launch_bounds__(256) k_res_partition(const uint64_t* __restrict__ start, const ResState* __restrict__ st,
                                                              uint2* __restrict__ tile_rows) {
  if (st->status != kResOk) return;
  const uint32_t n = st->n_delta, ntiles = st->ntiles;
  const uint64_t total = st->total;
  for (uint32_t t = blockIdx.x * blockDim.x + threadIdx.x; t < ntiles; t += gridDim.x * blockDim.x) {
    const uint64_t t_lo = (uint64_t)t * kExpTile;
    const uint64_t t_hi = min(t_lo + kExpTile, total);
    uint32_t r[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const uint64_t target = k == 0 ? t_lo : t_hi - 1;
      uint32_t lo = 0, hi = n;
      while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if (start[mid] <= target) lo = mid + 1; else hi = mid;
      }
      r[k] = lo - 1;
    }
    tile_rows[t] = make_uint2(r[0], r[1]);
  }
}

// persistent blocks: block b takes tiles b, b + gridDim.x, ...
template <typename KO, int MODE, int SINK>
__global__ void __launch_bounds__(kExpBlock) k_res_expand(JoinSpec S, const KO* __restrict__ okeys, const ResState* __restrict__ st,
                                                          const uint64_t* __restrict__ start, const uint4* __restrict__ rowinfo,
                                                          const uint2* __restrict__ tile_rows, uint32_t* __restrict__ err, MirrorArgs mr) {
  __shared__ ExpSmem sm;
  if (st->status != kResOk) return;
  const uint32_t ntiles = st->ntiles, n = st->n_delta;
  const uint64_t total = st->total;
  const BwdArgs bw{};
  uint32_t e = 0, n_new = 0;
  for (uint32_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
    const uint64_t t_lo = (uint64_t)t * kExpTile;
    const uint64_t t_hi = min(t_lo + kExpTile, total);
    expand_tile<KO, uint32_t, MODE, SINK>(sm, S, okeys, n, start, rowinfo, tile_rows[t], t_lo, t_hi, 0, (uint32_t*)nullptr, (float*)nullptr, bw, mr, e,
                                          n_new);
    __syncthreads();
  }
  if (e) atomicOr(err, e);
  n_new = __reduce_add_sync(0xffffffffu, n_new);
  if (lane_id() == 0 && n_new) atomicAdd(mr.n_new, (unsigned long long)n_new);
}

// One block, after k_mirror_changed_count: scan the per-tile counts of changed keys, close the round's books and decide
// whether another round runs.  `handle` is the WHILE node's condition (ignored when use_handle == 0: the host drives).
static __global__ void __launch_bounds__(1024) k_res_round_end(uint32_t* __restrict__ ch_sums, uint32_t ch_tiles, ResState* __restrict__ st,
                                                               const unsigned long long* __restrict__ new_counter,
                                                               cudaGraphConditionalHandle handle, int use_handle) {
  __shared__ uint32_t sh[1024 / 32 + 1];
  const bool live = st->status == kResOk;
  uint32_t carry = 0;
  for (uint32_t base = 0; base < ch_tiles; base += 1024) {
    const uint32_t p = base + threadIdx.x;
    const uint32_t x = p < ch_tiles ? ch_sums[p] : 0;
    uint32_t total;
    const uint32_t e = block_scan_excl<1024, uint32_t>(x, sh, total);
    if (p < ch_tiles) ch_sums[p] = carry + e;
    carry += total;
  }
  if (threadIdx.x == 0) {
    unsigned again = 0;
    if (live) {
      const unsigned long long seen = *new_counter;
      const unsigned long long fresh = seen - st->new_seen;
      st->new_seen = seen;
      st->n_new += fresh;
      st->n_improved += (unsigned long long)carry - fresh;
      st->candidates += st->round_cand;
      st->round_cand = 0;
      st->n_delta = carry;
      st->rounds += 1;
      if (carry > 0) {
        if (st->rounds >= st->max_rounds) st->status = kResCap; else again = 1;
      }
    }
    if (use_handle) cudaGraphSetConditional(handle, again);
  }
}

}  // namespace xlog
