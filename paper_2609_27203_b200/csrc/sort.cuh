// Stable LSD radix sort of (key, 32-bit payload) pairs over the significant key bits only
// (paper kernel table: `sort`, per-pass histogram, prefix sum, scatter -- there with 4-bit
// digits and 8 passes per 32-bit key; here digits are up to 8 bits and only the bits the
// key layout actually uses are sorted, e.g. 28 bits -> 4 passes of 7 bits).
//
// Per pass:  k_sort_hist   per-tile digit counts            (reads keys)
//            scan          exclusive scan, digit-major      (tiny)
//            k_sort_scatter rank inside the tile with warp match, order the tile in shared
//                          memory, write each digit's run contiguously (reads+writes pairs)
// No block waits on another block, so there is no spin loop anywhere in the sort.
#pragma once
#include "common.cuh"
#include "scan.cuh"

namespace xlog {

constexpr int kSortBlock = 512;
constexpr int kSortWarps = kSortBlock / 32;
constexpr int kSortMaxBins = 256;
constexpr int kHistGroup = 8;            // tiles per histogram block: 8 counters = one 32-byte sector per digit

template <typename K> struct SortCfg { static constexpr int items = sizeof(K) == 4 ? 16 : 12; };
template <typename K> constexpr int sort_tile() { return kSortBlock * SortCfg<K>::items; }

// hist[d * ntiles + tile] = number of keys of `tile` whose digit is d
template <typename K>
__global__ void __launch_bounds__(kSortBlock) k_sort_hist(const K* __restrict__ keys, uint32_t n, int shift, int nbins,
                                                          uint32_t ntiles, uint32_t* __restrict__ hist) {
  constexpr int TILE = kSortBlock * SortCfg<K>::items;
  __shared__ uint32_t cnt[kHistGroup][kSortMaxBins];
  for (int i = threadIdx.x; i < kHistGroup * kSortMaxBins; i += kSortBlock) (&cnt[0][0])[i] = 0;
  __syncthreads();
  const uint32_t mask = (uint32_t)nbins - 1u;
  const uint32_t tile0 = blockIdx.x * kHistGroup;
  for (int g = 0; g < kHistGroup; ++g) {
    const uint32_t tile = tile0 + g;
    if (tile >= ntiles) break;
    const uint64_t base = (uint64_t)tile * TILE;
#pragma unroll 4
    for (int i = 0; i < SortCfg<K>::items; ++i) {
      const uint64_t p = base + (uint64_t)i * kSortBlock + threadIdx.x;
      const bool ok = p < n;
      const uint32_t d = ok ? (uint32_t)(keys[p] >> shift) & mask : 0xffffffffu;
      const unsigned peers = __match_any_sync(0xffffffffu, d);
      if (ok && (peers & lanemask_lt()) == 0) atomicAdd(&cnt[g][d], (uint32_t)__popc(peers));
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < nbins * kHistGroup; i += kSortBlock) {
    const int d = i / kHistGroup, g = i % kHistGroup;
    if (tile0 + g < ntiles) hist[(uint64_t)d * ntiles + tile0 + g] = cnt[g][d];
  }
}

// offs = exclusive scan of hist (digit-major), i.e. offs[d*ntiles+tile] is where this tile's
// run of digit d starts in the output.
template <typename K>
__global__ void __launch_bounds__(kSortBlock) k_sort_scatter(const K* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                                                             K* __restrict__ keys_out, uint32_t* __restrict__ vals_out, uint32_t n,
                                                             int shift, int nbins, uint32_t ntiles,
                                                             const uint32_t* __restrict__ offs) {
  constexpr int ITEMS = SortCfg<K>::items;
  constexpr int TILE = kSortBlock * ITEMS;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  K* skeys = reinterpret_cast<K*>(smem_raw);                                   // TILE keys
  uint32_t* svals = reinterpret_cast<uint32_t*>(smem_raw + sizeof(K) * TILE);  // TILE payloads
  uint32_t* whist = svals + TILE;                                              // [kSortWarps][256]
  uint32_t* lbase = whist + kSortWarps * kSortMaxBins;                         // [256] tile-local start of each digit
  uint32_t* goff = lbase + kSortMaxBins;                                       // [256] global start minus local start
  uint32_t* scan_sh = goff + kSortMaxBins;                                     // block scan scratch

  const uint32_t tile = blockIdx.x;
  const uint64_t base = (uint64_t)tile * TILE;
  const uint32_t valid = (uint32_t)min((uint64_t)TILE, (uint64_t)n - base);
  const uint32_t mask = (uint32_t)nbins - 1u;
  const unsigned w = warp_id(), l = lane_id();

  for (int i = threadIdx.x; i < kSortWarps * kSortMaxBins; i += kSortBlock) whist[i] = 0;
  __syncthreads();

  // warp-striped load: item r of lane l sits at tile position w*32*ITEMS + r*32 + l
  K key[ITEMS];
  uint32_t val[ITEMS];
  uint32_t rank[ITEMS];
  const uint32_t wbase = w * 32 * ITEMS;
#pragma unroll
  for (int r = 0; r < ITEMS; ++r) {
    const uint32_t p = wbase + r * 32 + l;
    if (p < valid) { key[r] = keys_in[base + p]; val[r] = vals_in[base + p]; }
    else { key[r] = ~K(0); val[r] = 0; }
  }
  uint32_t* myhist = whist + w * kSortMaxBins;
#pragma unroll
  for (int r = 0; r < ITEMS; ++r) {
    const uint32_t p = wbase + r * 32 + l;
    const uint32_t d = p < valid ? (uint32_t)(key[r] >> shift) & mask : mask;   // padding ranks last in the last bin
    const unsigned peers = __match_any_sync(0xffffffffu, d);
    const int leader = __ffs(peers) - 1;
    uint32_t before = 0;
    if ((int)l == leader) { before = myhist[d]; myhist[d] = before + __popc(peers); }
    before = __shfl_sync(0xffffffffu, before, leader);
    rank[r] = before + __popc(peers & lanemask_lt());
    __syncwarp();
  }
  __syncthreads();

  // per digit: exclusive prefix over warps (in place) and the tile total
  uint32_t total_d = 0;
  if ((int)threadIdx.x < nbins) {
    const int d = threadIdx.x;
    uint32_t run = 0;
#pragma unroll
    for (int ww = 0; ww < kSortWarps; ++ww) {
      const uint32_t c = whist[ww * kSortMaxBins + d];
      whist[ww * kSortMaxBins + d] = run;
      run += c;
    }
    total_d = run;
  }
  uint32_t tile_total;
  const uint32_t lb = block_scan_excl<kSortBlock, uint32_t>(total_d, scan_sh, tile_total);
  if ((int)threadIdx.x < nbins) {
    lbase[threadIdx.x] = lb;
    goff[threadIdx.x] = offs[(uint64_t)threadIdx.x * ntiles + tile] - lb;
  }
  __syncthreads();

  // order the tile in shared memory
#pragma unroll
  for (int r = 0; r < ITEMS; ++r) {
    const uint32_t p = wbase + r * 32 + l;
    const uint32_t d = p < valid ? (uint32_t)(key[r] >> shift) & mask : mask;
    const uint32_t pos = lbase[d] + myhist[d] + rank[r];
    skeys[pos] = key[r];
    svals[pos] = val[r];
  }
  __syncthreads();

  // each digit's run is contiguous in shared memory and in the output
  for (uint32_t i = threadIdx.x; i < valid; i += kSortBlock) {
    const K k = skeys[i];
    const uint32_t d = (uint32_t)(k >> shift) & mask;
    const uint32_t g = goff[d] + i;
    keys_out[g] = k;
    vals_out[g] = svals[i];
  }
}

template <typename K>
constexpr size_t sort_scatter_smem() {
  return (sizeof(K) + 4) * (size_t)sort_tile<K>() + 4 * (size_t)(kSortWarps * kSortMaxBins + 2 * kSortMaxBins + kSortBlock / 32 + 1);
}

struct SortPlan {
  int passes;
  int bits_per_pass;
  uint32_t ntiles;
  size_t hist_entries;       // uint32 entries of scratch for the histogram matrix (reused every pass)
  size_t scan_tiles;         // uint32 entries of scratch for the scan spine
};

template <typename K>
inline SortPlan make_sort_plan(uint64_t n, int nbits) {
  SortPlan p;
  p.passes = (nbits + 7) / 8;
  p.bits_per_pass = p.passes ? (nbits + p.passes - 1) / p.passes : 0;
  p.ntiles = (uint32_t)((n + sort_tile<K>() - 1) / sort_tile<K>());
  p.hist_entries = (size_t)kSortMaxBins * p.ntiles;
  p.scan_tiles = (p.hist_entries + kScanTile - 1) / kScanTile;
  return p;
}

}  // namespace xlog
