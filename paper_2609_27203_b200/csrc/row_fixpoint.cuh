// Row-local fixpoint for the rule shape  h(a, c) :- h(a, b), r(b, c)  (transitive closure, multi-source reachability)
// over a max / min semiring, when one value of a owns few enough keys to live in shared memory.
//
// The rule never changes a: the tuples of one a are derived from the tuples of that a and from r alone.  The rounds of
// Algorithm 1 therefore fall apart into one independent sequence of rounds per value of a, and the whole fixpoint of the
// stratum is ONE launch without any grid-wide step: a block takes a value of a, loads its row of the tag mirror (one slot
// per value of c, in the relation's own key order) into shared memory and runs that row's rounds there - delta list from
// the changed bits, tags of the delta set aside before the join (the join lowers the row while other warps still read
// the delta), candidates applied with shared-memory atomics, new keys settled against the row's bitmap of present keys -
// until the row's delta is empty, then writes the row back.  Round r of a row is exactly round r of the global
// semi-naive loop restricted to that a, so the counters add up to the global ones: candidates, new and improved keys are
// sums over rows and rounds, and the number of global rounds is the largest number of rounds any row needed.
//
// The same holds for several mutually recursive heads whose rules all have this shape with one shared first column,
//   h_i(a, c) :- h_j(a, b), r(b, c)      (odd / even walks),
// as long as the heads share one key layout: a block then holds one row per head, a round closes every head's changed
// bits into its delta first and then applies every rule from its source head's delta to its target head's row.
#pragma once
#include "common.cuh"
#include "join.cuh"

namespace xlog {

constexpr int kRowMaxBits = 13;                  // keys per value of a: at most 8192 (row, tags set aside and delta list: 80 KB)
constexpr int kRowBlock = 256;
constexpr int kRowChunk = 1024;                  // delta rows whose candidates are laid out together

// Totals of the launch, in the control words.
enum { kRowCandidates = 0, kRowChanged = 1, kRowNew = 2, kRowRounds = 3, kRowCapped = 4, kRowTotals = 5 };

constexpr int kRowMaxHeads = 4, kRowMaxRules = 8;

struct RowHead {
  int32_t* table;                  // tag mirror in the relation's key order: slot = a << c_bits | c
  uint32_t* changed;               // changed bitmap: what the seed round derived; left all zero
  uint32_t* present;               // keys the relation holds
  int is_max;                      // oplus: max (1) or min (0)
};

struct RowRule {                   // heads[dst](a, c) :- heads[src](a, b), r(b, c)
  int src, dst;
  const uint32_t* off;             // r's offsets over its probed column
  uint32_t domain;                 // off has domain + 1 entries
  const int32_t* z;                // r's other column, in index order
  const float* w;                  // its tags
};

struct RowFix {
  RowHead heads[kRowMaxHeads];
  RowRule rules[kRowMaxRules];
  int n_heads, n_rules;
  uint32_t n_rows;                 // values of a
  int c_bits;                      // log2 of the slots per row (at least 5: a row owns whole bitmap words), the same for every head
  uint32_t z_max;                  // largest value a head's second column may take
  uint32_t max_rounds;             // rounds a row may run before the iteration cap is reached
  unsigned long long* totals;      // kRowTotals counters, zeroed by the caller
  uint32_t* err;
};

// per head: row tags (4 B per slot), delta tags (4 B), delta slots (2 B), changed and present bits
inline size_t row_fix_smem(int c_bits, int n_heads) { return (size_t)n_heads * (((size_t)10 << c_bits) + ((size_t)2 << c_bits) / 8); }

template <int NH>
__global__ void __launch_bounds__(kRowBlock) k_row_fixpoint(const __grid_constant__ RowFix P) {
  extern __shared__ uint32_t row_smem[];
  __shared__ uint32_t s_scan[kRowBlock / 32 + 1];
  __shared__ uint32_t s_lo[kRowChunk], s_start[kRowChunk + 1];      // per delta row of a chunk: first row of r's run, first candidate position
  __shared__ uint32_t s_nd[NH];                                      // delta rows of every head in the running round
  const uint32_t S = 1u << P.c_bits, W = S >> 5;
  const uint32_t per_head = 2 * S + 2 * W + S / 2;                   // words of shared memory per head
  const unsigned lane = lane_id();
  unsigned long long cand = 0;                    // thread 0's
  uint32_t n_changed = 0, n_new = 0, max_rounds_seen = 0, capped = 0;
  for (uint32_t a = blockIdx.x; a < P.n_rows; a += gridDim.x) {
    const size_t base = (size_t)a << P.c_bits;
    uint32_t any = 0;
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      uint32_t* chg = row_smem + h * per_head + 2 * S;
      uint32_t* pres = chg + W;
      for (uint32_t i = threadIdx.x; i < W; i += kRowBlock) {
        const uint32_t m = P.heads[h].changed[(base >> 5) + i];
        chg[i] = m;
        pres[i] = P.heads[h].present[(base >> 5) + i];
        any |= m;
      }
    }
    if (__syncthreads_or(any != 0u) == 0) continue;                            // nothing of this a changed in the seed round
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      int32_t* row = reinterpret_cast<int32_t*>(row_smem + h * per_head);
      for (uint32_t i = threadIdx.x; i < S; i += kRowBlock) row[i] = P.heads[h].table[base + i];
      for (uint32_t i = threadIdx.x; i < W; i += kRowBlock) P.heads[h].changed[(base >> 5) + i] = 0u;
    }
    __syncthreads();
    uint32_t rounds = 0;
    for (;;) {
      // close the round before, head by head: its changed keys are the delta now (ascending), the new ones among them enter the relation
      uint32_t nd_all = 0;
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        int32_t* row = reinterpret_cast<int32_t*>(row_smem + h * per_head);
        float* dtag = reinterpret_cast<float*>(row_smem + h * per_head + S);
        uint32_t* chg = row_smem + h * per_head + 2 * S;
        uint32_t* pres = chg + W;
        uint16_t* didx = reinterpret_cast<uint16_t*>(pres + W);
        uint32_t carry = 0;
        for (uint32_t i0 = 0; i0 < W; i0 += kRowBlock) {
          const uint32_t i = i0 + threadIdx.x;
          uint32_t m = i < W ? chg[i] : 0u;
          if (m) {
            n_new += __popc(m & ~pres[i]);
            pres[i] |= m;
            chg[i] = 0u;
          }
          uint32_t total;
          uint32_t at = carry + block_scan_excl<kRowBlock, uint32_t>((uint32_t)__popc(m), s_scan, total);
          while (m) {
            const uint32_t slot = (i << 5) + (__ffs(m) - 1);
            m &= m - 1;
            didx[at] = (uint16_t)slot;
            dtag[at] = ord2f(row[slot]);
            ++at;
          }
          carry += total;
        }
        if (threadIdx.x == 0) s_nd[h] = carry;
        nd_all += carry;
      }
      __syncthreads();
      if (nd_all == 0) break;
      if (threadIdx.x == 0) n_changed += nd_all;
      if (rounds >= P.max_rounds) { capped = 1; break; }
      ++rounds;
      // the joins, rule by rule and kRowChunk delta rows at a time: every row's run of r is looked up at once (one round trip
      // to memory for the whole chunk), a prefix over the run lengths lays the chunk's candidates out in a line, and the
      // threads stride over that line (the row of a position by binary search in the shared-memory prefix): a second
      // round trip for the candidates' columns and tags, whatever the mix of short and long runs
      for (int q = 0; q < P.n_rules; ++q) {
        const RowRule& R = P.rules[q];
        const uint32_t nd = s_nd[R.src];
        const float* dtag = reinterpret_cast<const float*>(row_smem + R.src * per_head + S);
        const uint16_t* didx = reinterpret_cast<const uint16_t*>(row_smem + R.src * per_head + 2 * S + 2 * W);
        int32_t* row = reinterpret_cast<int32_t*>(row_smem + R.dst * per_head);
        uint32_t* chg = row_smem + R.dst * per_head + 2 * S;
        const bool is_max = P.heads[R.dst].is_max != 0;
        for (uint32_t r0 = 0; r0 < nd; r0 += kRowChunk) {
          const uint32_t nr = min((uint32_t)kRowChunk, nd - r0);
          uint32_t carry_c = 0;
          for (uint32_t i0 = 0; i0 < nr; i0 += kRowBlock) {
            const uint32_t i = i0 + threadIdx.x;
            uint32_t lo = 0, dg = 0;
            if (i < nr) {
              const uint32_t b = didx[r0 + i];
              if (b < R.domain) { lo = R.off[b]; dg = R.off[b + 1] - lo; }
              s_lo[i] = lo;
            }
            uint32_t total;
            const uint32_t ex = block_scan_excl<kRowBlock, uint32_t>(dg, s_scan, total);
            if (i < nr) s_start[i] = carry_c + ex;
            carry_c += total;
          }
          if (threadIdx.x == 0) s_start[nr] = carry_c;
          __syncthreads();
          const uint32_t ncand = carry_c;
          if (threadIdx.x == 0) cand += ncand;
          for (uint32_t p = threadIdx.x; p < ncand; p += kRowBlock) {
            uint32_t lo = 0, hi = nr;                                           // last row whose start is <= p
            while (hi - lo > 1) { const uint32_t mid = (lo + hi) >> 1; if (s_start[mid] <= p) lo = mid; else hi = mid; }
            const uint32_t e = s_lo[lo] + (p - s_start[lo]);
            const uint32_t c = (uint32_t)R.z[e];
            if (c > P.z_max || c >= S) { atomicOr(P.err, kErrHeadRange); continue; }
            const int32_t v = f2ord(dtag[r0 + lo] + R.w[e]);
            const int32_t cur = row[c];
            if (is_max ? v > cur : v < cur) {
              if (is_max) atomicMax(row + c, v); else atomicMin(row + c, v);
              atomicOr(chg + (c >> 5), 1u << (c & 31));
            }
          }
          __syncthreads();
        }
      }
    }
    max_rounds_seen = max(max_rounds_seen, rounds);
    __syncthreads();
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      const int32_t* row = reinterpret_cast<const int32_t*>(row_smem + h * per_head);
      const uint32_t* pres = row_smem + h * per_head + 2 * S + W;
      for (uint32_t i = threadIdx.x; i < S; i += kRowBlock) P.heads[h].table[base + i] = row[i];
      for (uint32_t i = threadIdx.x; i < W; i += kRowBlock) P.heads[h].present[(base >> 5) + i] = pres[i];
    }
    __syncthreads();
  }
  // totals: per warp, then one atomic per counter
  n_new = __reduce_add_sync(0xffffffffu, n_new);
  if (lane == 0 && n_new) atomicAdd(P.totals + kRowNew, (unsigned long long)n_new);
  if (threadIdx.x == 0) {
    if (cand) atomicAdd(P.totals + kRowCandidates, cand);
    if (n_changed) atomicAdd(P.totals + kRowChanged, (unsigned long long)n_changed);
    if (max_rounds_seen) atomicMax(P.totals + kRowRounds, (unsigned long long)max_rounds_seen);
    if (capped) atomicMax(P.totals + kRowCapped, 1ull);
  }
}

}  // namespace xlog
