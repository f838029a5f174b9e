// Path doubling over a tag mirror:  p(x,z) :- p(x,y), p(y,z)  for one binary max/min relation p over a small dense domain
// (Section "Semi-naive evaluation on GPU": a rule with two recursive atoms takes one delta variant per occurrence).
//
// The mirror of p is a matrix, row x holding the tags of p(x, .).  Both delta variants of a round read the matrix as it
// stood when the round began (a snapshot copy) and never need a sorted index of p:
//   delta at the first atom:   for every delta row (x,y):   row_x  <-  row_x oplus (d_xy otimes snapshot row_y)
//   delta at the second atom:  for every y with p(x,y) in the snapshot:  row_x[z]  <-  row_x[z] oplus (p_xy otimes d_yz) over delta rows (y,z)
// A block owns one row x: it keeps the row in shared memory, applies every candidate of both variants there (the first
// variant's candidates arrive as whole coalesced rows, a thread owning its columns; the second's as scattered columns,
// with shared-memory atomics), and writes back only the entries that improved, setting their bits in the changed bitmap
// (a block owns its row's bitmap words, so plain stores do).  No candidate is written to memory, nothing is sorted, and
// the only global atomic is the candidate counter.
//
//   k_dense_rowstart  first delta row of every x (the delta list is in key order)
//   k_dense_round     the round itself
#pragma once
#include "common.cuh"
#include "join.cuh"

namespace xlog {

constexpr int kDenseRoundBlock = 256;

// rowstart[x] = index of the first delta key with column 0 >= x, for x in 0 .. rows (rowstart[rows] = n)
static __global__ void __launch_bounds__(256) k_dense_rowstart(const uint32_t* __restrict__ dkeys, uint32_t n, int bits1, uint32_t rows,
                                                              uint32_t* __restrict__ rowstart) {
  const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x > rows) return;
  const uint64_t want = (uint64_t)x << bits1;
  uint32_t lo = 0, hi = n;
  while (lo < hi) { const uint32_t mid = lo + ((hi - lo) >> 1); if ((uint64_t)dkeys[mid] < want) lo = mid + 1; else hi = mid; }
  rowstart[x] = lo;
}

struct DenseRound {
  const int32_t* snap;             // the matrix as of the start of the round: rows x L order-mapped tags
  int32_t* table;                  // the live matrix
  uint32_t* changed;               // one bit per slot
  const uint32_t* dkeys;           // delta keys (x << bits1 | y), ascending
  const float* dtags;
  const uint32_t* rowstart;        // rows + 1 entries
  uint32_t rows;                   // 2^bits of column 0
  int bits1;                       // L = 2^bits1 columns
  unsigned long long* candidates;  // += bindings of both variants
};

// COLS = columns per thread (row length / 256, at least 1): a thread keeps its columns of row x in registers while the
// first variant streams snapshot rows past them, four delta rows (4 * COLS loads per thread) in flight at a time.
template <int SINK, int COLS>
__global__ void __launch_bounds__(kDenseRoundBlock) k_dense_round(DenseRound D) {
  extern __shared__ int32_t dsm[];
  const uint32_t L = 1u << D.bits1;
  int32_t* acc = dsm;              // row x with this round's candidates applied
  int32_t* old = dsm + L;          // row x of the snapshot
  uint32_t* ylist = reinterpret_cast<uint32_t*>(dsm + 2 * L);      // the y of the second variant
  __shared__ uint32_t s_ny;
  __shared__ unsigned long long s_cnt;
  const int32_t empty = SINK == kSinkMin ? kMirrorEmptyMin : kMirrorEmptyMax;
  const uint32_t x = blockIdx.x;
  const size_t row0 = (size_t)x << D.bits1;
  if (threadIdx.x == 0) { s_ny = 0; s_cnt = 0; }
  int32_t a[COLS];
#pragma unroll
  for (int k = 0; k < COLS; ++k) {
    const uint32_t z = threadIdx.x + k * kDenseRoundBlock;
    a[k] = z < L ? D.snap[row0 + z] : empty;
    if (z < L) old[z] = a[k];
  }
  uint32_t cnt = 0;
  // delta at the first atom: whole rows of the snapshot stream past the thread's columns
  const uint32_t e0 = D.rowstart[x], e1 = D.rowstart[x + 1];
  for (uint32_t e = e0; e < e1; e += 4) {
    const int32_t* ry[4];
    float d[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      ry[u] = nullptr; d[u] = 0.f;
      if (e + u < e1) {
        const uint32_t y = D.dkeys[e + u] & (L - 1);
        if (y < D.rows) { ry[u] = D.snap + ((size_t)y << D.bits1); d[u] = D.dtags[e + u]; }     // else: no such row, p(y, .) is empty
      }
    }
    int32_t s[4][COLS];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int k = 0; k < COLS; ++k) {
        const uint32_t z = threadIdx.x + k * kDenseRoundBlock;
        s[u][k] = (ry[u] && z < L) ? ry[u][z] : empty;
      }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int k = 0; k < COLS; ++k)
        if (s[u][k] != empty) {
          const int32_t v = f2ord(d[u] + ord2f(s[u][k]));
          a[k] = SINK == kSinkMin ? min(a[k], v) : max(a[k], v);
          ++cnt;
        }
  }
#pragma unroll
  for (int k = 0; k < COLS; ++k) {
    const uint32_t z = threadIdx.x + k * kDenseRoundBlock;
    if (z < L) acc[z] = a[k];
  }
  __syncthreads();
  // delta at the second atom: the y that row x holds in the snapshot and that have delta rows
  for (uint32_t y = threadIdx.x; y < L && y < D.rows; y += kDenseRoundBlock)
    if (old[y] != empty && D.rowstart[y + 1] > D.rowstart[y]) ylist[atomicAdd(&s_ny, 1u)] = y;
  __syncthreads();
  const uint32_t ny = s_ny;
  // a warp per y: its delta row in steps of 32 entries, shared-memory atomics into the row
  for (uint32_t i = warp_id(); i < ny; i += kDenseRoundBlock / 32) {
    const uint32_t y = ylist[i];
    const float pxy = ord2f(old[y]);
    const uint32_t r0 = D.rowstart[y], r1 = D.rowstart[y + 1];
    for (uint32_t e = r0 + lane_id(); e < r1; e += 32) {
      const uint32_t z = D.dkeys[e] & (L - 1);
      const int32_t v = f2ord(pxy + D.dtags[e]);
      if (SINK == kSinkMin) atomicMin(&acc[z], v); else atomicMax(&acc[z], v);
      ++cnt;
    }
  }
  __syncthreads();
  // write back what improved; 32 consecutive columns share one bitmap word, which this block owns
  for (uint32_t z0 = 0; z0 < L; z0 += kDenseRoundBlock) {
    const uint32_t z = z0 + threadIdx.x;
    bool better = false;
    if (z < L) {
      better = SINK == kSinkMin ? acc[z] < old[z] : acc[z] > old[z];
      if (better) D.table[row0 + z] = acc[z];
    }
    const unsigned bal = __ballot_sync(0xffffffffu, better);
    if (bal && lane_id() == 0) {
      if (L >= 32) D.changed[(row0 + z) >> 5] = bal;
      else atomicOr(D.changed + ((row0 + z) >> 5), bal << ((row0 + z) & 31));      // short rows share words
    }
  }
  unsigned long long c64 = cnt;
#pragma unroll
  for (int s2 = 16; s2; s2 >>= 1) c64 += __shfl_down_sync(0xffffffffu, c64, s2);
  if (lane_id() == 0 && c64) atomicAdd(&s_cnt, c64);
  __syncthreads();
  if (threadIdx.x == 0 && s_cnt) atomicAdd(D.candidates, s_cnt);
}

inline size_t dense_round_smem(int bits1) { return (size_t)3 * 4 * ((size_t)1 << bits1); }

}  // namespace xlog
