// Resident fixpoint rounds (Section "GPU-Native Symbolic Substrate": the iteration body of the
// semi-naive loop runs as a device-resident graph with fixed capacities, an overflow flag and no
// host reads inside the loop).  One round over a tag mirror (mirror.cuh) is a fixed sequence of
// launches whose sizes are read from a small state block in device memory:
//
//   per rule with a recursive atom:  k_res_count_scan -> k_res_expand
//   then:                            k_res_emit (next delta, round bookkeeping, loop condition)
//
// With a single such rule (the usual case) the count and scan of the NEXT round ride on the emit kernel
// (k_res_emit_count), so a round is two launches: k_res_expand -> k_res_emit_count; only the first round's
// count is a launch of its own, before the loop.
//
// Every kernel has a fixed grid and strides over however much work the state block announces, so the
// sequence can be captured once as the body of a CUDA-graph WHILE node; k_res_round_end decides whether
// the body runs again.  The host reads the state block once, after the loop.
#pragma once
#include <cuda_runtime.h>

#include "common.cuh"
#include "join.cuh"
#include "mirror.cuh"
#include "scan.cuh"

namespace xlog {

enum { kResOk = 0, kResCap = 1, kResOverflow = 2, kResError = 3 };

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

constexpr int kResMaxVariants = 16;
// the small counters of a head's resident rounds, one uint32 array: per rule the count kernel's tile ticket, the emit
// kernel's two counters (rows reserved, blocks done), and k_res_emit_count's 64-bit reservation word
enum { kResTkEmit = kResMaxVariants, kResTkReserve = kResMaxVariants + 2, kResTickets = kResMaxVariants + 4 };
static_assert((kResTkReserve * 4) % 8 == 0, "the reservation counter is a 64-bit word");
#ifndef XLOG_RES_EC_SPLIT
#define XLOG_RES_EC_SPLIT 4
#endif
constexpr int kResEcSplit = XLOG_RES_EC_SPLIT;         // threads to a bitmap word in k_res_emit_count
constexpr int kResEcWords = kMirBlock / kResEcSplit;             // bitmap words per sweep of k_res_emit_count: 2048 keys, so that mid-sized key spaces still give hundreds of blocks
constexpr int kResRowBits = 25;                        // k_res_emit_count reserves (candidates << kResRowBits | rows) with one atomic add
constexpr int kResScanItems = 4;                       // rows per thread in the fused count + scan: short dependent chains
constexpr int kResScanTile = kScanBlock * kResScanItems;
constexpr uint64_t kScanFlagAgg = 1ull << 62, kScanFlagIncl = 2ull << 62, kScanValMask = (1ull << 62) - 1;

__device__ __forceinline__ unsigned long long ld_volatile_u64(const unsigned long long* p) { return *reinterpret_cast<const volatile unsigned long long*>(p); }
__device__ __forceinline__ void st_volatile_u64(unsigned long long* p, unsigned long long v) { *reinterpret_cast<volatile unsigned long long*>(p) = v; }

// Scratch that must be zero when a round starts: scan status words and tile tickets of every rule.
struct ResScratch {
  unsigned long long* scan_status;   // [kResMaxVariants][scan_tiles_cap]
  uint32_t scan_tiles_cap;
  uint32_t* tickets;                 // [kResMaxVariants], then the emit kernel's two counters
};

static __global__ void __launch_bounds__(1024) k_res_init(ResState* st, ResScratch sc, uint32_t n_variants, uint32_t n_delta, uint32_t max_rounds,
                                                          uint32_t max_tiles, unsigned long long new_seen) {
  if (threadIdx.x == 0) {
    ResState s{};
    s.n_delta = n_delta; s.max_rounds = max_rounds; s.max_tiles = max_tiles; s.new_seen = new_seen;
    *st = s;
  }
  // everything, not just what the first round will touch: an abandoned loop leaves its last round's words behind
  for (size_t i = threadIdx.x; i < (size_t)n_variants * sc.scan_tiles_cap; i += blockDim.x) sc.scan_status[i] = 0;
  for (uint32_t i = threadIdx.x; i < kResTickets; i += blockDim.x) sc.tickets[i] = 0;
}

// Count, scan and partition of one rule in a single launch.  Blocks draw 1024-row tiles from a ticket counter (so a tile
// only ever waits for tiles that running blocks already own).  For its tile a block computes every row's degree and
// row record, reduces the degrees, resolves its exclusive prefix by looking back through the status words of the tiles
// before it (aggregate first, inclusive prefix once known: a chained scan), writes the rows' start offsets, and - since
// a row knows which candidate positions it covers - the first / last row of every expand tile whose boundary it covers.
// The last tile publishes the candidate total and the expand tile count.  Waits are bounded: a status word that stays
// empty for spin_limit polls (a value of the context) raises the internal-error flag and stops the resident loop.
template <typename KO>
__global__ void __launch_bounds__(kScanBlock) k_res_count_scan(JoinSpec S, const KO* __restrict__ okeys, const float* __restrict__ otags,
                                                               ResState* __restrict__ st, uint4* __restrict__ rowinfo, uint64_t* __restrict__ start,
                                                               uint2* __restrict__ tile_rows, unsigned long long* __restrict__ status,
                                                               uint32_t* __restrict__ ticket, uint32_t* __restrict__ err, uint32_t spin_limit) {
  __shared__ uint64_t sh[kScanBlock / 32 + 1];
  __shared__ uint32_t sdeg[kResScanTile];
  __shared__ uint32_t s_tile;
  __shared__ uint64_t s_excl;
  if (st->status != kResOk) return;
  const uint32_t n = st->n_delta, max_tiles = st->max_tiles;
  const uint32_t tiles = (n + kResScanTile - 1) / kResScanTile;
  if (tiles == 0) {
    if (blockIdx.x == 0 && threadIdx.x == 0) { st->total = 0; st->ntiles = 0; }
    return;
  }
  for (;;) {
    if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
    __syncthreads();
    const uint32_t t = s_tile;
    if (t >= tiles) break;
#pragma unroll
    for (int i = 0; i < kResScanItems; ++i) {
      const uint32_t row = t * kResScanTile + i * kScanBlock + threadIdx.x;
      sdeg[i * kScanBlock + threadIdx.x] = row < n ? join_count_row<KO>(S, okeys, otags, row, rowinfo, err) : 0u;
    }
    __syncthreads();
    uint32_t x[kResScanItems];
    uint64_t s = 0;
#pragma unroll
    for (int i = 0; i < kResScanItems; ++i) { x[i] = sdeg[threadIdx.x * kResScanItems + i]; s += x[i]; }
    uint64_t total;
    const uint64_t in_tile = block_scan_excl<kScanBlock, uint64_t>(s, sh, total);
    if (warp_id() == 0) {
      // look back 32 tiles at a time: lane l polls tile (base - l) until it holds at least an aggregate; the nearest
      // inclusive prefix among them ends the walk
      uint64_t excl = 0;
      bool timeout = false;
      if (t > 0) {
        if (lane_id() == 0) st_volatile_u64(status + t, kScanFlagAgg | total);
        int64_t base = (int64_t)t - 1;
        for (;;) {
          const int64_t idx = base - (int64_t)lane_id();
          unsigned long long v = kScanFlagIncl;                         // before tile 0: an inclusive prefix of zero
          if (idx >= 0) {
            uint32_t spins = 0;
            for (;;) {
              v = ld_volatile_u64(status + idx);
              if (v & ~kScanValMask) break;
              if (++spins > spin_limit) { timeout = true; v = kScanFlagIncl; break; }
              if (spins > 64) __nanosleep(32);
            }
          }
          const unsigned incl = __ballot_sync(0xffffffffu, (v & ~kScanValMask) == kScanFlagIncl);
          const int first = incl ? __ffs(incl) - 1 : 31;                // lanes 0 .. first contribute
          unsigned long long part = (int)lane_id() <= first ? (v & kScanValMask) : 0ull;
#pragma unroll
          for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
          excl += part;
          if (incl) break;
          base -= 32;
        }
        timeout = __any_sync(0xffffffffu, timeout);
      }
      if (lane_id() == 0) {
        st_volatile_u64(status + t, kScanFlagIncl | (excl + total));
        if (timeout) { atomicOr(err, kErrInternal); st->status = kResError; }
        s_excl = excl;
        if (t == tiles - 1 && !timeout) {
          const uint64_t all = excl + total;
          const uint64_t nt = (all + kExpTileMirror - 1) / kExpTileMirror;
          st->total = all;
          if (nt > max_tiles) { st->status = kResOverflow; st->ntiles = 0; }
          else {
            st->ntiles = (uint32_t)nt; st->round_cand += all;
            if (nt) tile_rows[nt - 1].y = n - 1;           // rows after the last candidate have no matches: harmless to include
          }
        }
      }
    }
    __syncthreads();
    uint64_t run = s_excl + in_tile;
#pragma unroll
    for (int i = 0; i < kResScanItems; ++i) {
      const uint32_t row = t * kResScanTile + threadIdx.x * kResScanItems + i;
      if (row < n) {
        start[row] = run;
        if (x[i]) {
          // expand tile u begins at position u * kExpTileMirror and ends at (u + 1) * kExpTileMirror - 1
          const uint64_t end = run + x[i];                                       // one past the row's last position
          for (uint64_t u = (run + kExpTileMirror - 1) / kExpTileMirror; u * kExpTileMirror < end && u < max_tiles; ++u) tile_rows[u].x = row;
          for (uint64_t u = (run + kExpTileMirror) / kExpTileMirror; u * kExpTileMirror <= end && u <= max_tiles; ++u) tile_rows[u - 1].y = row;
        }
        run += x[i];
      }
    }
    if (tiles <= gridDim.x) break;            // every block draws one ticket first, so all tiles are already taken
    __syncthreads();
  }
}

// persistent blocks: block b takes tiles b, b + gridDim.x, ...
template <typename KO, int MODE, int SINK>
__global__ void __launch_bounds__(kExpBlock, kExpMirrorBlocksPerSM) k_res_expand(JoinSpec S, const KO* __restrict__ okeys, const ResState* __restrict__ st,
                                                          const uint64_t* __restrict__ start, const uint4* __restrict__ rowinfo,
                                                          const uint2* __restrict__ tile_rows, uint32_t* __restrict__ err, MirrorArgs mr) {
  __shared__ ExpSmem<ExpShapeT<true>> sm;
  if (st->status != kResOk) return;
  const uint32_t ntiles = st->ntiles, n = st->n_delta;
  const uint64_t total = st->total;
  const BwdArgs bw{};
  uint32_t e = 0;
  for (uint32_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
    const uint64_t t_lo = (uint64_t)t * kExpTileMirror;
    const uint64_t t_hi = min(t_lo + kExpTileMirror, total);
    expand_tile<KO, uint32_t, MODE, SINK>(sm, S, okeys, n, start, rowinfo, tile_rows[t], t_lo, t_hi, 0, (uint32_t*)nullptr, (float*)nullptr, bw, mr, e);
    __syncthreads();
  }
  if (e) atomicOr(err, e);
}

// Tail of a round's last kernel, called by every thread of every block: the block that finishes last closes the
// round's books, clears the scratch of the next round and decides whether it runs.  `handle` is the WHILE node's
// condition (ignored when use_handle == 0: the host drives).  ctr[0] = rows reserved so far, ctr[1] = blocks done;
// both are left at zero.  reserve != nullptr: the kernel has also counted the next round's join (see
// k_res_emit_count); the word holds (candidates << kResRowBits | rows) and is left at zero.
__device__ __forceinline__ void res_close_round(const bool live, ResState* __restrict__ st, const ResScratch& sc, uint32_t n_variants,
                                                const unsigned long long* __restrict__ new_counter, uint32_t* __restrict__ ctr,
                                                cudaGraphConditionalHandle handle, int use_handle, uint32_t& s_last,
                                                unsigned long long* __restrict__ reserve, uint2* __restrict__ tile_rows) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = atomicAdd(&ctr[1], 1u) == gridDim.x - 1 ? 1u : 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  unsigned long long next_total = 0;
  uint32_t changed = 0;
  if (live) {
    if (reserve) {
      const unsigned long long r = ld_volatile_u64(reserve);
      changed = (uint32_t)(r & ((1ull << kResRowBits) - 1));
      next_total = r >> kResRowBits;
    } else changed = *reinterpret_cast<volatile uint32_t*>(&ctr[0]);
  }
  if (live && !reserve) {
    const uint32_t tiles = (st->n_delta + kResScanTile - 1) / kResScanTile + 1;
    for (uint32_t v = 0; v < n_variants; ++v)
      for (uint32_t i = threadIdx.x; i < tiles && i < sc.scan_tiles_cap; i += blockDim.x) sc.scan_status[(size_t)v * sc.scan_tiles_cap + i] = 0;
    for (uint32_t i = threadIdx.x; i < kResMaxVariants; i += blockDim.x) sc.tickets[i] = 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned again = 0;
    if (live) {
      const unsigned long long seen = *new_counter;
      const unsigned long long fresh = seen - st->new_seen;
      st->new_seen = seen;
      st->n_new += fresh;
      st->n_improved += (unsigned long long)changed - fresh;
      st->candidates += st->round_cand;
      st->round_cand = 0;
      st->n_delta = changed;
      st->rounds += 1;
      if (changed > 0) {
        if (st->rounds >= st->max_rounds) st->status = kResCap; else again = 1;
      }
      if (reserve) {                                     // the next round's join, as k_res_count_scan's last tile would announce it
        const unsigned long long nt = (next_total + kExpTileMirror - 1) / kExpTileMirror;
        st->total = next_total;
        st->ntiles = 0;
        if (again) {
          if (nt > st->max_tiles) { st->status = kResOverflow; again = 0; }
          else {
            st->ntiles = (uint32_t)nt; st->round_cand = next_total;
            if (nt) tile_rows[nt - 1].y = changed - 1;
          }
        }
      }
    }
    ctr[0] = 0; ctr[1] = 0;
    if (reserve) *reserve = 0ull;
    if (use_handle) cudaGraphSetConditional(handle, again);
  }
}

// Last kernel of a round: compact the changed bitmap into the next delta and close the round.  Inside the resident
// loop the delta need not be in key order (the join reads it row by row and max / min do not care about order), so a
// block reserves room for its tile's keys with one atomic add instead of waiting for a prefix sum; row order in the
// delta therefore varies from run to run, the relation derived does not.  res_close_round ends the kernel.
template <int SW>
__global__ void __launch_bounds__(kMirBlock) k_res_emit(uint32_t* __restrict__ words, uint32_t* __restrict__ present, uint32_t nwords,
                                                        unsigned long long* __restrict__ new_total, const int32_t* __restrict__ table,
                                                        uint32_t* __restrict__ keys, float* __restrict__ tags, ResState* __restrict__ st,
                                                        ResScratch sc, uint32_t n_variants, const unsigned long long* __restrict__ new_counter,
                                                        uint32_t* __restrict__ ctr, cudaGraphConditionalHandle handle, int use_handle) {
  __shared__ uint32_t sh[kMirBlock / 32 + 1];
  __shared__ uint32_t list[kMirBlock * 32];
  __shared__ uint32_t s_base, s_last;
  const bool live = st->status == kResOk;                // an abandoned round keeps its bitmap and its delta
  if (live) {
    uint32_t w[SW];
    uint32_t cnt = 0, fresh = 0;
#pragma unroll
    for (int j = 0; j < SW; ++j) {
      const uint32_t wi = (blockIdx.x * SW + j) * kMirBlock + threadIdx.x;
      w[j] = wi < nwords ? words[wi] : 0u;
      cnt += __popc(w[j]);
      if (w[j]) {                                        // changed keys the relation did not hold yet are new tuples
        const uint32_t had = present[wi];
        fresh += __popc(w[j] & ~had);
        if (w[j] & ~had) present[wi] = had | w[j];
      }
    }
    uint32_t tile_total;
    block_scan_excl<kMirBlock, uint32_t>(cnt, sh, tile_total);
    if (tile_total) {                                    // uniform across the block
      fresh = __reduce_add_sync(0xffffffffu, fresh);
      if (lane_id() == 0 && fresh) atomicAdd(new_total, (unsigned long long)fresh);
      if (threadIdx.x == 0) s_base = atomicAdd(&ctr[0], tile_total);
      __syncthreads();
      uint32_t out = s_base;
#pragma unroll
      for (int j = 0; j < SW; ++j) {
        const uint32_t wi = (blockIdx.x * SW + j) * kMirBlock + threadIdx.x;
        uint32_t bits = w[j];
        uint32_t total;
        uint32_t pos = block_scan_excl<kMirBlock, uint32_t>((uint32_t)__popc(bits), sh, total);
        if (total == 0) continue;
        if (bits) words[wi] = 0u;
        while (bits) {
          const int b = __ffs(bits) - 1;
          bits &= bits - 1;
          list[pos++] = (wi << 5) + b;
        }
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < total; i += kMirBlock) {
          const uint32_t key = list[i];
          keys[out + i] = key;
          tags[out + i] = ord2f(__ldcg(table + key));
        }
        out += total;
        __syncthreads();
      }
    }
  }
  res_close_round(live, st, sc, n_variants, new_counter, ctr, handle, use_handle, s_last, nullptr, nullptr);
}

// k_res_emit with the next round's count and scan folded in, for a head with one rule over it.  A block handles its
// bitmap tile sweep by sweep (kResEcWords words, at most 2048 changed keys): compact the sweep's keys into shared memory, sum
// their degrees (the rule's matches per key: two offset reads), reserve rows AND candidate positions with ONE 64-bit
// atomic add - so that row order and candidate order agree across blocks and the start offsets increase with the row
// index, which is all the join's partition needs - then write, per key, the delta row, its 16-byte row record and its
// start offset, 1024 keys per step (four to a thread) with a block-wide prefix sum over their degrees, and mark the first / last row of
// every join tile whose boundary the row covers.  No look-back and no wait: the only cross-block word is the reservation.
template <int SW>
__global__ void __launch_bounds__(kMirBlock) k_res_emit_count(uint32_t* __restrict__ words, uint32_t* __restrict__ present, uint32_t nwords,
                                                              unsigned long long* __restrict__ new_total, const int32_t* __restrict__ table,
                                                              uint32_t* __restrict__ keys, float* __restrict__ tags, ResState* __restrict__ st,
                                                              ResScratch sc, const unsigned long long* __restrict__ new_counter,
                                                              uint32_t* __restrict__ ctr, cudaGraphConditionalHandle handle, int use_handle,
                                                              JoinSpec S, uint4* __restrict__ rowinfo, uint64_t* __restrict__ start,
                                                              uint2* __restrict__ tile_rows, uint32_t* __restrict__ err) {
  __shared__ uint32_t sh[kMirBlock / 32 + 1];
  __shared__ uint64_t sh64[kMirBlock / 32 + 1];
  __shared__ uint32_t list[kResEcWords * 32];
  __shared__ unsigned long long s_res;
  __shared__ uint32_t s_last;
  unsigned long long* reserve = reinterpret_cast<unsigned long long*>(sc.tickets + kResTkReserve);
  const bool live = st->status == kResOk;                // an abandoned round keeps its bitmap and its delta
  if (live) {
    const uint32_t max_tiles = st->max_tiles;
    constexpr int kSubBits = 32 / kResEcSplit;           // kResEcSplit threads to a word, kSubBits bits each
    const uint32_t sub = threadIdx.x % kResEcSplit;
#pragma unroll 1
    for (int j = 0; j < SW; ++j) {
      const uint32_t wi = (blockIdx.x * SW + j) * kResEcWords + threadIdx.x / kResEcSplit;
      const uint32_t full = wi < nwords ? words[wi] : 0u;
      uint32_t bits = (full >> (kSubBits * sub)) & ((1u << kSubBits) - 1u);
      uint32_t fresh = 0;
      __syncwarp();
      if (full && sub == 0) {                            // changed keys the relation did not hold yet are new tuples
        const uint32_t had = present[wi];
        fresh = __popc(full & ~had);
        if (fresh) present[wi] = had | full;
        words[wi] = 0u;
      }
      uint32_t total;
      uint32_t pos = block_scan_excl<kMirBlock, uint32_t>((uint32_t)__popc(bits), sh, total);
      if (total == 0) continue;                          // uniform across the block
      fresh = __reduce_add_sync(0xffffffffu, fresh);
      if (lane_id() == 0 && fresh) atomicAdd(new_total, (unsigned long long)fresh);
      while (bits) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1;
        list[pos++] = (wi << 5) + kSubBits * sub + b;
      }
      __syncthreads();
      // the sweep's candidate total
      uint64_t dsum = 0;
#pragma unroll 4
      for (uint32_t i = threadIdx.x; i < total; i += kMirBlock) dsum += join_count_kv<uint32_t>(S, list[i], 0.f, 0, nullptr, err);
      uint64_t cand_total;
      block_scan_excl<kMirBlock, uint64_t>(dsum, sh64, cand_total);
      if (threadIdx.x == 0) s_res = atomicAdd(reserve, (unsigned long long)(cand_total << kResRowBits) | total);
      __syncthreads();
      const uint32_t row0 = (uint32_t)(s_res & ((1ull << kResRowBits) - 1));
      uint64_t run0 = s_res >> kResRowBits;
      // kItems consecutive keys per thread and step: their slot reads and offset reads are in flight together
      constexpr int kItems = 4;
      for (uint32_t i0 = 0; i0 < total; i0 += kMirBlock * kItems) {
        const uint32_t ib = i0 + threadIdx.x * kItems;
        uint32_t key[kItems], d[kItems];
        float tag[kItems];
#pragma unroll
        for (int k = 0; k < kItems; ++k) {
          key[k] = ib + k < total ? list[ib + k] : 0u;
          tag[k] = ib + k < total ? ord2f(__ldcg(table + key[k])) : 0.f;
        }
        uint32_t mine = 0;
#pragma unroll
        for (int k = 0; k < kItems; ++k) {
          d[k] = 0;
          if (ib + k < total) {
            const uint32_t row = row0 + ib + k;
            keys[row] = key[k];
            tags[row] = tag[k];
            d[k] = join_count_kv<uint32_t>(S, key[k], tag[k], row, rowinfo, err);
          }
          mine += d[k];
        }
        uint64_t step_total;
        uint64_t run = run0 + block_scan_excl<kMirBlock, uint64_t>((uint64_t)mine, sh64, step_total);
#pragma unroll
        for (int k = 0; k < kItems; ++k)
          if (ib + k < total) {
            const uint32_t row = row0 + ib + k;
            start[row] = run;
            if (d[k]) {
              // join tile u begins at position u * kExpTileMirror and ends at (u + 1) * kExpTileMirror - 1
              const uint64_t end = run + d[k];                                     // one past the row's last position
              for (uint64_t u = (run + kExpTileMirror - 1) / kExpTileMirror; u * kExpTileMirror < end && u < max_tiles; ++u) tile_rows[u].x = row;
              for (uint64_t u = (run + kExpTileMirror) / kExpTileMirror; u * kExpTileMirror <= end && u <= max_tiles; ++u) tile_rows[u - 1].y = row;
            }
            run += d[k];
          }
        run0 += step_total;
      }
      __syncthreads();
    }
  }
  res_close_round(live, st, sc, 1, new_counter, ctr, handle, use_handle, s_last, reserve, tile_rows);
}

}  // namespace xlog
