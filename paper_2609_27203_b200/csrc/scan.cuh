// Exclusive prefix sum over a device array (paper kernel table: `scan`, the building
// block of compaction, dedup and group-by).  Three launches, no inter-block waiting:
// per-tile sums, a single-block spine scan, per-tile scan with the spine offset.
#pragma once
#include "common.cuh"

namespace xlog {

constexpr int kScanBlock = 256;
constexpr int kScanItems = 16;
constexpr int kScanTile = kScanBlock * kScanItems;

template <typename Tin, typename Tout>
__global__ void __launch_bounds__(kScanBlock) k_scan_tile_sums(const Tin* __restrict__ in, int64_t n, Tout* __restrict__ tile_sums) {
  __shared__ Tout sh[kScanBlock / 32 + 1];
  const int64_t base = (int64_t)blockIdx.x * kScanTile;
  Tout s = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    const int64_t p = base + i * kScanBlock + threadIdx.x;
    if (p < n) s += (Tout)in[p];
  }
  Tout total;
  block_scan_excl<kScanBlock, Tout>(s, sh, total);
  if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}

// One block: exclusive scan of `m` values in place; the grand total goes to *total_out.
template <typename T>
__global__ void __launch_bounds__(1024) k_scan_spine(T* __restrict__ v, int64_t m, T* __restrict__ total_out) {
  __shared__ T sh[1024 / 32 + 1];
  T carry = 0;
  for (int64_t base = 0; base < m; base += 1024) {
    const int64_t p = base + threadIdx.x;
    const T x = p < m ? v[p] : T(0);
    T total;
    const T e = block_scan_excl<1024, T>(x, sh, total);
    if (p < m) v[p] = carry + e;
    carry += total;
  }
  if (threadIdx.x == 0 && total_out) *total_out = carry;
}

// One block: exclusive scans of two arrays of the same length in one launch.
template <typename T>
__global__ void __launch_bounds__(1024) k_scan_spine2(T* __restrict__ a, T* __restrict__ b, int64_t m, T* __restrict__ total_a,
                                                      T* __restrict__ total_b) {
  __shared__ T sh[1024 / 32 + 1];
  T ca = 0, cb = 0;
  for (int64_t base = 0; base < m; base += 1024) {
    const int64_t p = base + threadIdx.x;
    const T xa = p < m ? a[p] : T(0), xb = p < m ? b[p] : T(0);
    T ta, tb;
    const T ea = block_scan_excl<1024, T>(xa, sh, ta);
    const T eb = block_scan_excl<1024, T>(xb, sh, tb);
    if (p < m) { a[p] = ca + ea; b[p] = cb + eb; }
    ca += ta; cb += tb;
  }
  if (threadIdx.x == 0) { *total_a = ca; *total_b = cb; }
}

// One block: out = exclusive scan of in (n elements), grand total to *total_out.  For short arrays,
// where the three-launch scan would be all launch latency.
template <typename Tin, typename Tout>
__global__ void __launch_bounds__(1024) k_scan_block(const Tin* __restrict__ in, int64_t n, Tout* __restrict__ out,
                                                     Tout* __restrict__ total_out) {
  __shared__ Tout sh[1024 / 32 + 1];
  constexpr int PER = 16;
  Tout carry = 0;
  for (int64_t base = 0; base < n; base += 1024 * PER) {
    Tout x[PER];
    Tout s = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int64_t p = base + (int64_t)threadIdx.x * PER + i;
      x[i] = p < n ? (Tout)in[p] : Tout(0);
      s += x[i];
    }
    Tout total;
    Tout run = carry + block_scan_excl<1024, Tout>(s, sh, total);
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int64_t p = base + (int64_t)threadIdx.x * PER + i;
      if (p < n) out[p] = run;
      run += x[i];
    }
    carry += total;
  }
  if (threadIdx.x == 0) *total_out = carry;
}

template <typename Tin, typename Tout>
__global__ void __launch_bounds__(kScanBlock) k_scan_apply(const Tin* __restrict__ in, int64_t n, const Tout* __restrict__ tile_base,
                                                           Tout* __restrict__ out) {
  __shared__ Tout sh[kScanBlock / 32 + 1];
  // blocked arrangement: thread t owns items [t*kScanItems, (t+1)*kScanItems) of the tile
  const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
  Tout x[kScanItems];
  Tout s = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    x[i] = base + i < n ? (Tout)in[base + i] : Tout(0);
    s += x[i];
  }
  Tout total;
  Tout run = block_scan_excl<kScanBlock, Tout>(s, sh, total) + tile_base[blockIdx.x];
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    if (base + i < n) out[base + i] = run;
    run += x[i];
  }
}

}  // namespace xlog
