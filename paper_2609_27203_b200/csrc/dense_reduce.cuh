// Segmented reduce-by-key for idempotent semirings (max / min) that sorts only the HIGH key bits:
// after a radix sort on bits [L, nbits) every run of equal high bits ("group") spans at most 2^L
// distinct keys, so the group is reduced in a direct-addressed shared-memory table instead of being
// sorted further (paper kernel table: `groupby` = boundary detection + per-group reduction; here the
// boundary is the high-bit group and the reduction is an atomic max/min per table slot).
// Against the full sort + segmented scan this saves the low-bit sort passes and the reduce reads.
// max/min are exact and order-independent, so the result is bit-identical to the sorted path.
//
//   k_group_bounds   first row of every group (binary search; rows are sorted by key >> L)
//   k_group_plan     one block: parts per group (big groups are split), work-item prefix, spill slots
//   k_dense_reduce   one block per work item: table in shared memory; a group in one piece is emitted
//                    at once, pieces of a split group merge through a spill table in global memory and
//                    the last piece to finish emits
//   k_dense_compact  move each group's reduced rows to their final, dense position
#pragma once
#include "common.cuh"

namespace xlog {

constexpr int kDenseBits = 12;                         // table slots per group = 2^12 (16 KB of shared memory)
constexpr int kDenseSlots = 1 << kDenseBits;
constexpr int kDenseBlock = 256;
constexpr int kDensePer = kDenseSlots / kDenseBlock;   // table slots owned by one thread at emit time
constexpr int kDenseMaxGroupBits = 16;

template <typename Op> struct DenseOp;
template <> struct DenseOp<OpMin> {
  static constexpr int32_t empty = 0x7fffffff;
  __device__ __forceinline__ static void upd(int32_t* p, int32_t v) { atomicMin(p, v); }
};
template <> struct DenseOp<OpMax> {
  static constexpr int32_t empty = (int32_t)0x80000000;
  __device__ __forceinline__ static void upd(int32_t* p, int32_t v) { atomicMax(p, v); }
};

// How the rows are grouped.  A key is (top | mid | low): `low` = L table bits, `mid` = M bits that were radix
// sorted, `top` = T bits by which the candidate stream was already ordered when it was produced (leading head
// columns carried over from the leading columns of the sorted outer relation).  A stable sort on the mid bits
// alone leaves the rows ordered by (mid, top), so the group number is  g = mid << T | top  and increases along
// the array; with T = 0 this is simply key >> L.
struct GroupShape { int L, M, T; };
template <typename K>
__device__ __forceinline__ uint32_t group_of(const GroupShape& S, K key) {
  const uint32_t mid = (uint32_t)(key >> S.L) & ((1u << S.M) - 1u);
  const uint32_t top = S.T ? (uint32_t)(key >> (S.L + S.M)) : 0u;
  return (mid << S.T) | top;
}
template <typename K>
__device__ __forceinline__ K group_key(const GroupShape& S, uint32_t g, uint32_t slot) {
  const uint32_t top = g & ((1u << S.T) - 1u), mid = g >> S.T;
  return ((K)top << (S.L + S.M)) | ((K)mid << S.L) | (K)slot;
}

// gstart[g] = first row whose group number is >= g, for g in [0, G]
template <typename K>
__global__ void __launch_bounds__(256) k_group_bounds(const K* __restrict__ keys, uint32_t n, GroupShape S, uint32_t G,
                                                      uint32_t* __restrict__ gstart) {
  for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g <= G; g += gridDim.x * blockDim.x) {
    uint32_t lo = 0, hi = n;
    while (lo < hi) {
      const uint32_t mid = lo + ((hi - lo) >> 1);
      if (group_of<K>(S, keys[mid]) < g) lo = mid + 1; else hi = mid;
    }
    gstart[g] = lo;
  }
}

// One block.  parts[g] = ceil(size/part) ; part_base = exclusive scan of parts ; spill[g] = index of the
// group's spill table if it is split (exclusive scan of "parts > 1").  totals[0] = work items, totals[1] = spill tables.
static __global__ void __launch_bounds__(1024) k_group_plan(const uint32_t* __restrict__ gstart, uint32_t G, uint32_t part,
                                                            uint32_t* __restrict__ part_base, uint32_t* __restrict__ spill,
                                                            uint32_t* __restrict__ done, uint32_t* __restrict__ totals) {
  __shared__ uint32_t sh[33];
  uint32_t run_p = 0, run_s = 0;
  for (uint32_t base = 0; base < G; base += 1024) {
    const uint32_t g = base + threadIdx.x;
    uint32_t p = 0;
    if (g < G) { const uint32_t sz = gstart[g + 1] - gstart[g]; p = (sz + part - 1) / part; done[g] = 0; }
    uint32_t tp, ts;
    const uint32_t ep = block_scan_excl<1024, uint32_t>(p, sh, tp);
    const uint32_t es = block_scan_excl<1024, uint32_t>(p > 1 ? 1u : 0u, sh, ts);
    if (g < G) { part_base[g] = run_p + ep; spill[g] = run_s + es; }
    run_p += tp; run_s += ts;
  }
  if (threadIdx.x == 0) { part_base[G] = run_p; totals[0] = run_p; totals[1] = run_s; }
}

static __global__ void __launch_bounds__(256) k_fill_i32(int32_t* __restrict__ p, uint64_t n, int32_t v) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) p[i] = v;
}

template <typename K, typename Op>
__global__ void __launch_bounds__(kDenseBlock) k_dense_reduce(const K* __restrict__ keys, const float* __restrict__ tags, GroupShape S,
                                                               uint32_t G, uint32_t part, const uint32_t* __restrict__ gstart,
                                                               const uint32_t* __restrict__ part_base, const uint32_t* __restrict__ spill,
                                                               uint32_t n_spill_tables, int32_t* __restrict__ spill_tab,
                                                               uint32_t* __restrict__ done, K* __restrict__ out_keys,
                                                               float* __restrict__ out_tags, uint32_t* __restrict__ ucount) {
  __shared__ int32_t tbl[kDenseSlots];
  __shared__ uint32_t sh[kDenseBlock / 32 + 1];
  __shared__ uint32_t s_g, s_last;
  const uint32_t item = blockIdx.x;
  if (item >= part_base[G]) return;
  if (threadIdx.x == 0) {                              // group of this work item: last g with part_base[g] <= item
    uint32_t lo = 0, hi = G;
    while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (part_base[mid] <= item) lo = mid + 1; else hi = mid; }
    s_g = lo - 1;
  }
#pragma unroll
  for (int i = 0; i < kDensePer; ++i) tbl[i * kDenseBlock + threadIdx.x] = DenseOp<Op>::empty;
  __syncthreads();
  const uint32_t g = s_g;
  const uint32_t g0 = gstart[g], g1 = gstart[g + 1];
  const uint32_t nparts = part_base[g + 1] - part_base[g];
  const uint32_t r0 = g0 + (item - part_base[g]) * part;
  const uint32_t r1 = min(r0 + part, g1);
  const uint32_t mask = (1u << S.L) - 1u;
  // reduce this piece into the table; 4 independent loads per thread in flight
  for (uint32_t i = r0 + threadIdx.x; i < r1; i += 4 * kDenseBlock) {
    K k[4]; float t[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t j = i + u * kDenseBlock;
      if (j < r1) { k[u] = keys[j]; t[u] = tags[j]; }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (i + u * kDenseBlock < r1) DenseOp<Op>::upd(&tbl[(uint32_t)k[u] & mask], f2ord(t[u]));
  }
  __syncthreads();
  if (nparts > 1) {
    // merge into the group's spill table; the piece that arrives last reads the merged table back
    if (spill[g] >= n_spill_tables) return;            // cannot happen: capacity is n/part + 1 tables
    int32_t* gt = spill_tab + (uint64_t)spill[g] * kDenseSlots;
#pragma unroll
    for (int i = 0; i < kDensePer; ++i) {
      const int s = i * kDenseBlock + threadIdx.x;
      const int32_t v = tbl[s];
      if (v != DenseOp<Op>::empty) DenseOp<Op>::upd(&gt[s], v);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&done[g], 1u) == nparts - 1 ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
#pragma unroll
    for (int i = 0; i < kDensePer; ++i) {
      const int s = i * kDenseBlock + threadIdx.x;
      tbl[s] = __ldcg(&gt[s]);
    }
    __syncthreads();
  }
  // emit the occupied slots in key order at the group's own offset of the output buffer
  const int s0 = threadIdx.x * kDensePer;              // this thread's consecutive slots
  uint32_t cnt = 0;
#pragma unroll
  for (int i = 0; i < kDensePer; ++i) cnt += tbl[s0 + i] != DenseOp<Op>::empty ? 1u : 0u;
  uint32_t total;
  uint32_t pos = g0 + block_scan_excl<kDenseBlock, uint32_t>(cnt, sh, total);
#pragma unroll
  for (int i = 0; i < kDensePer; ++i) {
    const int32_t v = tbl[s0 + i];
    if (v != DenseOp<Op>::empty) {
      out_keys[pos] = group_key<K>(S, g, (uint32_t)(s0 + i));
      out_tags[pos] = ord2f(v);
      ++pos;
    }
  }
  if (threadIdx.x == 0) ucount[g] = total;
}

// One thread per output row: find its group in upos (exclusive scan of the per-group row counts) and
// copy the row from the group's offset to its final, dense position.
template <typename K>
__global__ void __launch_bounds__(256) k_dense_compact(const K* __restrict__ in_keys, const float* __restrict__ in_tags,
                                                       const uint32_t* __restrict__ gstart, const uint32_t* __restrict__ upos,
                                                       uint32_t G, const uint32_t* __restrict__ u_ptr, K* __restrict__ out_keys,
                                                       float* __restrict__ out_tags) {
  const uint32_t u = *u_ptr;
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < u; i += gridDim.x * blockDim.x) {
    uint32_t lo = 0, hi = G;                           // last group with upos[g] <= i
    while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (upos[mid] <= i) lo = mid + 1; else hi = mid; }
    const uint32_t g = lo - 1;
    const uint32_t src = gstart[g] + (i - upos[g]);
    out_keys[i] = in_keys[src];
    out_tags[i] = in_tags[src];
  }
}

}  // namespace xlog
