// Stable LSD radix sort of (key, 32-bit payload) pairs over the significant key bits only
// (paper kernel table: `sort`, per-pass histogram, prefix sum, scatter -- there with 4-bit
// digits and 8 passes per 32-bit key; here digits are up to 8 bits and only the bits the
// key layout actually uses are sorted, e.g. 28 bits -> 4 passes of 7 bits).
//
// One read of the keys builds the digit histograms of every pass (k_sort_digit_hist); each pass
// is then a single kernel (k_sort_pass) that ranks a tile with warp match, orders it in shared
// memory, and learns where its digit runs start from the tiles before it by decoupled look-back
// over a per-tile status word (count + 2 flag bits).  Tiles take their index from an atomic
// ticket, so a tile only ever waits for tiles that are already running; every wait is bounded
// and a timeout raises the error flag and skips the tile's writes instead of hanging.
#pragma once
#include <string.h>

#include "common.cuh"
#include "scan.cuh"

namespace xlog {

#ifndef XLOG_SORT_BLOCK
#define XLOG_SORT_BLOCK 256
#endif
#ifndef XLOG_SORT_ITEMS
#define XLOG_SORT_ITEMS 16
#endif
#ifndef XLOG_SORT_MINB
#define XLOG_SORT_MINB 4
#endif
constexpr int kSortBlock = XLOG_SORT_BLOCK;
constexpr int kSortWarps = kSortBlock / 32;
constexpr int kSortMaxBins = 256;
constexpr int kSortMaxPasses = 8;
constexpr uint32_t kSortMaxN = (1u << 30) - 1;       // status words keep 30 bits of count
constexpr uint32_t kFlagLocal = 1u << 30, kFlagGlobal = 2u << 30, kCountMask = (1u << 30) - 1;
constexpr uint32_t kSpinLimit = 1u << 22;            // default number of polls of one status word before giving up (a context may lower it)

template <typename K> struct SortCfg { static constexpr int items = XLOG_SORT_ITEMS; };
template <typename K> constexpr int sort_tile() { return kSortBlock * SortCfg<K>::items; }

struct SortPasses {
  int passes;
  int shift[kSortMaxPasses];
  int bits[kSortMaxPasses];
};

// passes covering key bits [lo, hi), least significant first
inline SortPasses make_sort_passes(int lo, int hi) {
  SortPasses p{};
  const int nbits = hi > lo ? hi - lo : 0;
  p.passes = (nbits + 7) / 8;
  int done = 0;
  for (int i = 0; i < p.passes; ++i) {
    const int b = (nbits - done + (p.passes - i) - 1) / (p.passes - i);     // spread the bits evenly
    p.shift[i] = lo + done; p.bits[i] = b; done += b;
  }
  return p;
}

__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_volatile_u32(uint32_t* p, uint32_t v) {
  asm volatile("st.volatile.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// hist[pass * 256 + d] += number of keys whose digit of `pass` is d.  Persistent grid.
// The block that finishes last turns every pass's counts into exclusive bases in place
// (hist[pass*256 + d] = number of keys with a smaller digit in that pass).  `done` starts at 0.
template <typename K>
__global__ void __launch_bounds__(256) k_sort_digit_hist(const K* __restrict__ keys, uint32_t n, SortPasses P,
                                                         uint32_t* __restrict__ hist, uint32_t* __restrict__ done) {
  __shared__ uint32_t sh[kSortMaxPasses * kSortMaxBins];
  __shared__ uint32_t s_last;
  __shared__ uint32_t scan_sh[256 / 32 + 1];
  for (int i = threadIdx.x; i < P.passes * kSortMaxBins; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  // Each thread takes 8 CONSECUTIVE keys (vector loads when the array is 16-byte aligned) and, per pass,
  // adds one count per run of equal digits among them: keys usually arrive in runs (sorted adjacency lists,
  // a constant high digit), and for spread-out digits this is still only one shared-memory add per key.
  constexpr int U = 8;
  const uint64_t chunk = (uint64_t)blockDim.x * U;
  const bool vec = (reinterpret_cast<uintptr_t>(keys) & 15u) == 0;
  for (uint64_t c0 = (uint64_t)blockIdx.x * chunk; c0 < n; c0 += (uint64_t)gridDim.x * chunk) {
    const uint64_t i0 = c0 + (uint64_t)threadIdx.x * U;
    K k[U];
    int cnt = 0;
    if (i0 + U <= n && vec) {
      const uint4* src = reinterpret_cast<const uint4*>(keys + i0);
      uint4 v[U * sizeof(K) / 16];
#pragma unroll
      for (int j = 0; j < (int)(U * sizeof(K) / 16); ++j) v[j] = src[j];
      memcpy(k, v, sizeof(k));
      cnt = U;
    } else {
#pragma unroll
      for (int u = 0; u < U; ++u) if (i0 + u < n) { k[u] = keys[i0 + u]; cnt = u + 1; }
    }
    if (cnt == 0) continue;
#pragma unroll
    for (int p = 0; p < kSortMaxPasses; ++p) {
      if (p < P.passes) {
        const uint32_t m = (1u << P.bits[p]) - 1u;
        uint32_t run_d = (uint32_t)(k[0] >> P.shift[p]) & m, run_n = 1;
#pragma unroll
        for (int u = 1; u < U; ++u) {
          if (u < cnt) {
            const uint32_t d = (uint32_t)(k[u] >> P.shift[p]) & m;
            if (d != run_d) { atomicAdd(&sh[p * kSortMaxBins + run_d], run_n); run_d = d; run_n = 0; }
            ++run_n;
          }
        }
        atomicAdd(&sh[p * kSortMaxBins + run_d], run_n);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < P.passes * kSortMaxBins; i += blockDim.x)
    if (sh[i]) atomicAdd(&hist[i], sh[i]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(done, 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int p = 0; p < P.passes; ++p) {
    const uint32_t v = __ldcg(&hist[p * kSortMaxBins + threadIdx.x]);
    uint32_t total;
    const uint32_t e = block_scan_excl<256, uint32_t>(v, scan_sh, total);
    hist[p * kSortMaxBins + threadIdx.x] = e;
  }
}

// One pass.  status[tile*256 + d]: 0 = not ready, kFlagLocal|count = this tile's count of digit d,
// kFlagGlobal|count = count summed over tiles 0..tile.  ticket: one counter per pass, starts at 0.
// Lanes of the warp whose digit equals this lane's: one ballot per digit bit (the hardware
// match instruction is an order of magnitude slower than BITS ballots on this part).
template <int BITS>
__device__ __forceinline__ unsigned match_digit(uint32_t d) {
  unsigned peers = 0xffffffffu;
#pragma unroll
  for (int b = 0; b < BITS; ++b) {
    const bool bit = (d >> b) & 1u;
    const unsigned m = __ballot_sync(0xffffffffu, bit);
    peers &= bit ? m : ~m;
  }
  return peers;
}

// Body of one tile; FULL = the tile has no padding (all bounds tests fold away).
template <typename K, int BITS, bool FULL>
__device__ __forceinline__ void sort_tile_body(const K* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                                               K* __restrict__ keys_out, uint32_t* __restrict__ vals_out, const uint64_t base,
                                               const uint32_t valid, const uint32_t tile, const int shift,
                                               const uint32_t* __restrict__ digit_base, uint32_t* __restrict__ status,
                                               uint32_t* __restrict__ err, const uint32_t spin_limit, K* skeys, uint32_t* svals, uint32_t* whist,
                                               uint32_t* lbase, uint32_t* goff, uint32_t* scan_sh) {
  constexpr int ITEMS = SortCfg<K>::items;
  constexpr int TILE = kSortBlock * ITEMS;
  constexpr int nbins = 1 << BITS;
  constexpr uint32_t mask = (uint32_t)nbins - 1u;
  const unsigned w = warp_id(), l = lane_id();

  // warp-striped load: item r of lane l sits at tile position w*32*ITEMS + r*32 + l
  K key[ITEMS];
  uint32_t rank[ITEMS];
  const uint32_t wbase = w * 32 * ITEMS + l;
  const K* kin = keys_in + base + wbase;
#pragma unroll
  for (int r = 0; r < ITEMS; ++r) key[r] = (FULL || wbase + r * 32 < valid) ? kin[r * 32] : ~K(0);
  uint32_t* myhist = whist + w * kSortMaxBins;
#pragma unroll
  for (int r = 0; r < ITEMS; ++r) {
    // padding carries all-ones keys: it ranks last in the last bin
    const uint32_t d = (uint32_t)(key[r] >> shift) & mask;
    const unsigned peers = match_digit<BITS>(d);
    const int leader = __ffs(peers) - 1;
    uint32_t before = 0;
    if ((int)l == leader) { before = myhist[d]; myhist[d] = before + __popc(peers); }
    before = __shfl_sync(0xffffffffu, before, leader);
    rank[r] = before + __popc(peers & lanemask_lt());
    __syncwarp();
  }
  __syncthreads();

  // per digit: exclusive prefix over warps (in place) and the tile total; publish the tile's counts
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
    if (!FULL && d == nbins - 1) total_d -= (uint32_t)TILE - valid;             // padding is not data
    st_volatile_u32(&status[(uint64_t)tile * kSortMaxBins + d], (tile == 0 ? kFlagGlobal : kFlagLocal) | total_d);
  }
  uint32_t tile_total;
  const uint32_t lb = block_scan_excl<kSortBlock, uint32_t>(total_d, scan_sh, tile_total);
  if ((int)threadIdx.x < nbins) lbase[threadIdx.x] = lb;
  __syncthreads();

  // order the tile's keys in shared memory; remember each item's slot for its payload
#pragma unroll
  for (int r = 0; r < ITEMS; ++r) {
    const uint32_t d = (uint32_t)(key[r] >> shift) & mask;
    rank[r] += lbase[d] + myhist[d];
    if (FULL || rank[r] < valid) skeys[rank[r]] = key[r];
  }
  // payloads: same slots
  const uint32_t* vin = vals_in + base + wbase;
#pragma unroll
  for (int r = 0; r < ITEMS; ++r)
    if (FULL || wbase + r * 32 < valid) svals[rank[r]] = vin[r * 32];

  // decoupled look-back: keys with digit d in all earlier tiles
  if ((int)threadIdx.x < nbins) {
    const int d = threadIdx.x;
    uint32_t excl = 0;
    bool timeout = false;
    if (tile > 0) {
      int64_t look = (int64_t)tile - 1;
      uint32_t spins = 0;
      while (true) {
        const uint32_t s = ld_volatile_u32(&status[(uint64_t)look * kSortMaxBins + d]);
        const uint32_t flag = s & ~kCountMask;
        if (flag == 0) {
          if (++spins > spin_limit) { timeout = true; break; }
          __nanosleep(64);
          continue;
        }
        excl += s & kCountMask;
        if (flag == kFlagGlobal || look == 0) break;
        --look;
        spins = 0;
      }
      // a wait that gave up publishes nothing: the tiles behind this one must run into the same gap, not past it
      if (!timeout) st_volatile_u32(&status[(uint64_t)tile * kSortMaxBins + d], kFlagGlobal | ((excl + total_d) & kCountMask));
    }
    if (timeout) { atomicOr(err, kErrInternal); scan_sh[kSortBlock / 32 + 2] = 1u; }
    goff[d] = digit_base[d] + excl - lb;
  }
  __syncthreads();
  if (scan_sh[kSortBlock / 32 + 2]) return;             // a wait ran out: the error flag is set, write nothing

  // each digit's run is contiguous in shared memory and in the output
#pragma unroll 4
  for (uint32_t i = threadIdx.x; i < (FULL ? (uint32_t)TILE : valid); i += kSortBlock) {
    const K k = skeys[i];
    const uint32_t d = (uint32_t)(k >> shift) & mask;
    const uint32_t g = goff[d] + i;
    keys_out[g] = k;
    vals_out[g] = svals[i];
  }
}

// One pass.  status[tile*256 + d]: 0 = not ready, kFlagLocal|count = this tile's count of digit d,
// kFlagGlobal|count = count summed over tiles 0..tile.  ticket: one counter per pass, starts at 0.
template <typename K, int BITS>
__global__ void __launch_bounds__(kSortBlock, sizeof(K) == 4 ? XLOG_SORT_MINB : XLOG_SORT_MINB / 2) k_sort_pass(const K* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                                                          K* __restrict__ keys_out, uint32_t* __restrict__ vals_out, uint32_t n,
                                                          int shift, const uint32_t* __restrict__ digit_base,
                                                          uint32_t* __restrict__ status, uint32_t* __restrict__ ticket,
                                                          uint32_t* __restrict__ err, uint32_t spin_limit) {
  constexpr int ITEMS = SortCfg<K>::items;
  constexpr int TILE = kSortBlock * ITEMS;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  K* skeys = reinterpret_cast<K*>(smem_raw);                                   // TILE keys
  uint32_t* svals = reinterpret_cast<uint32_t*>(smem_raw + sizeof(K) * TILE);  // TILE payloads
  uint32_t* whist = svals + TILE;                                              // [kSortWarps][256]
  uint32_t* lbase = whist + kSortWarps * kSortMaxBins;                         // [256] tile-local start of each digit
  uint32_t* goff = lbase + kSortMaxBins;                                       // [256] global start minus local start
  uint32_t* scan_sh = goff + kSortMaxBins;                                     // block scan scratch + ticket + abort flag

  if (threadIdx.x == 0) { scan_sh[kSortBlock / 32 + 1] = atomicAdd(ticket, 1u); scan_sh[kSortBlock / 32 + 2] = 0u; }
  for (int i = threadIdx.x; i < kSortWarps * (1 << BITS); i += kSortBlock) whist[(i >> BITS) * kSortMaxBins + (i & ((1 << BITS) - 1))] = 0;
  __syncthreads();
  const uint32_t tile = scan_sh[kSortBlock / 32 + 1];
  const uint64_t base = (uint64_t)tile * TILE;
  const uint32_t valid = (uint32_t)min((uint64_t)TILE, (uint64_t)n - base);
  if (valid == (uint32_t)TILE)
    sort_tile_body<K, BITS, true>(keys_in, vals_in, keys_out, vals_out, base, valid, tile, shift, digit_base, status, err, spin_limit, skeys, svals,
                                  whist, lbase, goff, scan_sh);
  else
    sort_tile_body<K, BITS, false>(keys_in, vals_in, keys_out, vals_out, base, valid, tile, shift, digit_base, status, err, spin_limit, skeys, svals,
                                   whist, lbase, goff, scan_sh);
}

template <typename K>
constexpr size_t sort_pass_smem() {
  return (sizeof(K) + 4) * (size_t)sort_tile<K>() + 4 * (size_t)(kSortWarps * kSortMaxBins + 2 * kSortMaxBins + kSortBlock / 32 + 4);
}

}  // namespace xlog
