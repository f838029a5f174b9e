// Tag mirror of a max/min head relation: a direct-addressed table with one order-mapped tag per
// possible packed key, used by the fixpoint of a linear recursive rule set in place of
// sort -> reduce-by-key -> diff/merge (Algorithm 1 lines 6-9).  The join kernel applies every
// candidate to its slot with one atomic max/min; the keys whose slot improved in a round are
// flagged in a bitmap, and compacting that bitmap in key order yields the next delta, already
// sorted and free of duplicates.  After the last round the table itself is compacted into the
// relation's sorted (key, tag) arrays.  max and min are exact and order-independent, so the
// relation is bit-identical to the one the sorting path derives.
//
//   k_mirror_scatter        loaded facts -> table
//   k_mirror_changed_count  set bits per tile of the changed bitmap
//   k_mirror_changed_emit   bitmap -> delta (keys ascending, tags read from the table); clears the bitmap
//   k_mirror_full_count     occupied slots per 4096-slot tile
//   k_mirror_full_emit      table -> relation
#pragma once
#include "common.cuh"

namespace xlog {

constexpr int kMirBlock = 256;
constexpr int kMirSlotsPerTile = kMirBlock * 16;       // table slots per tile (four int4 per thread)

// `from` / `to`: the relation's own key layout and the mirror's (the same columns, possibly with the order of
// significance changed: see group_join.cuh)
__device__ __forceinline__ uint32_t relayout_key(const KeyLayout& from, const KeyLayout& to, uint32_t key) {
  uint32_t out = 0;
#pragma unroll
  for (int c = 0; c < kMaxArity; ++c)
    if (c < from.arity) out |= (uint32_t)key_col<uint32_t>(from, key, c) << to.shift[c];
  return out;
}

template <typename K>
__global__ void __launch_bounds__(256) k_mirror_scatter(const K* __restrict__ keys, const float* __restrict__ tags, uint32_t n,
                                                        KeyLayout from, KeyLayout to, int32_t* __restrict__ table, uint32_t* __restrict__ present) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    const uint32_t key = relayout_key(from, to, (uint32_t)keys[i]);
    table[key] = f2ord(tags[i]);
    atomicOr(present + (key >> 5), 1u << (key & 31));
  }
}

// The changed bitmap is handled in tiles of SW * 256 words (SW "sweeps" of one word per thread).  Small domains take
// SW = 1 so that there are enough tiles to occupy the GPU; large ones SW = 4 to keep the list of tile counts short.
// nwords is the bitmap's (padded) length.
// Also settles which changed keys are new: those whose bit in `present` (the keys the relation holds) was clear; the
// bits are set here and the count of new keys is added to *new_total.
template <int SW>
__global__ void __launch_bounds__(kMirBlock) k_mirror_changed_count(const uint32_t* __restrict__ words, uint32_t* __restrict__ present,
                                                                    uint32_t nwords, uint32_t* __restrict__ tile_sums,
                                                                    unsigned long long* __restrict__ new_total) {
  __shared__ uint32_t sh[kMirBlock / 32 + 1];
  uint32_t s = 0, fresh = 0;
#pragma unroll
  for (int j = 0; j < SW; ++j) {
    const uint32_t wi = (blockIdx.x * SW + j) * kMirBlock + threadIdx.x;
    const uint32_t w = wi < nwords ? words[wi] : 0u;
    s += __popc(w);
    if (w) {
      const uint32_t had = present[wi];
      fresh += __popc(w & ~had);
      if (w & ~had) present[wi] = had | w;
    }
  }
  uint32_t total;
  block_scan_excl<kMirBlock, uint32_t>(s, sh, total);
  if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
  fresh = __reduce_add_sync(0xffffffffu, fresh);
  if (lane_id() == 0 && fresh) atomicAdd(new_total, (unsigned long long)fresh);
}

// One block per tile.  In a sweep every thread expands the set bits of one word into a key list in shared memory
// (at most 8192 keys); then the whole block turns the list into output rows, so the table reads are independent of
// one another and the writes are coalesced however unevenly the bits are spread.
template <typename K, int SW>
__global__ void __launch_bounds__(kMirBlock) k_mirror_changed_emit(uint32_t* __restrict__ words, uint32_t nwords,
                                                                   const uint32_t* __restrict__ tile_base, const int32_t* __restrict__ table,
                                                                   K* __restrict__ keys, float* __restrict__ tags,
                                                                   const uint32_t* __restrict__ skip_if_nonzero) {
  __shared__ uint32_t sh[kMirBlock / 32 + 1];
  __shared__ uint32_t list[kMirBlock * 32];
  if (skip_if_nonzero && *skip_if_nonzero) return;       // the round was abandoned: keep the bitmap and the old delta
  uint32_t out = tile_base[blockIdx.x];
#pragma unroll 1
  for (int j = 0; j < SW; ++j) {
    const uint32_t wi = (blockIdx.x * SW + j) * kMirBlock + threadIdx.x;
    uint32_t bits = wi < nwords ? words[wi] : 0u;
    uint32_t total;
    uint32_t pos = block_scan_excl<kMirBlock, uint32_t>((uint32_t)__popc(bits), sh, total);
    if (total == 0) continue;                            // uniform across the block
    if (bits) words[wi] = 0u;
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      list[pos++] = (wi << 5) + b;
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < total; i += kMirBlock) {
      const uint32_t key = list[i];
      keys[out + i] = (K)key;
      tags[out + i] = ord2f(__ldcg(table + key));
    }
    out += total;
    __syncthreads();
  }
}

// Slots are read in a striped arrangement (coalesced int4 loads); the output order is the slot order, so the four
// stripes of a tile are scanned one after the other.
static __global__ void __launch_bounds__(kMirBlock) k_mirror_full_count(const int4* __restrict__ table4, uint64_t nquads, int32_t empty,
                                                                        uint32_t* __restrict__ tile_sums) {
  __shared__ uint32_t sh[kMirBlock / 32 + 1];
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint64_t q = ((uint64_t)blockIdx.x * 4 + i) * kMirBlock + threadIdx.x;
    if (q < nquads) {
      const int4 v = table4[q];
      s += (v.x != empty) + (v.y != empty) + (v.z != empty) + (v.w != empty);
    }
  }
  uint32_t total;
  block_scan_excl<kMirBlock, uint32_t>(s, sh, total);
  if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}

template <typename K>
__global__ void __launch_bounds__(kMirBlock) k_mirror_full_emit(const int4* __restrict__ table4, uint64_t nquads, int32_t empty,
                                                                const uint32_t* __restrict__ tile_base, KeyLayout from, KeyLayout to,
                                                                K* __restrict__ keys, float* __restrict__ tags) {
  __shared__ uint32_t sh[kMirBlock / 32 + 1];
  uint32_t run = tile_base[blockIdx.x];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint64_t q = ((uint64_t)blockIdx.x * 4 + i) * kMirBlock + threadIdx.x;
    int4 v = make_int4(empty, empty, empty, empty);
    if (q < nquads) v = table4[q];
    const uint32_t s = (v.x != empty) + (v.y != empty) + (v.z != empty) + (v.w != empty);
    uint32_t total;
    uint32_t pos = run + block_scan_excl<kMirBlock, uint32_t>(s, sh, total);
    run += total;
    const int32_t e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (e[j] != empty) {
        keys[pos] = (K)relayout_key(from, to, (uint32_t)(q * 4 + j));      // slot index (mirror layout) -> the relation's key
        tags[pos] = ord2f(e[j]);
        ++pos;
      }
  }
}

// ---- table -> relation when the mirror's minor column is the relation's major one ----------------------------------
// A grouped mirror (group_join.cuh) is indexed (column 1, column 0), the relation is ordered (column 0, column 1).  With at
// most 64 values of column 0 the rows can be written straight to their final places, no sort: a block takes kMtNodes
// values c of column 1 (one per thread); k_mirror_t_count counts, per value a of column 0, the tile's present keys
// (c, a); an exclusive scan over (a, tile) gives every (a, tile) run its place; k_mirror_t_emit stages the tile's tags in
// shared memory with coalesced reads and writes each column's rows in order of c: a warp's rows of one a are contiguous.
constexpr int kMtNodes = 128;

__device__ __forceinline__ unsigned long long mt_mask(const uint32_t* __restrict__ present, uint32_t c, uint32_t n_nodes, int slots) {
  if (c >= n_nodes) return 0ull;
  if (slots == 64) return *reinterpret_cast<const unsigned long long*>(present + 2 * (size_t)c);
  const uint32_t w = present[((size_t)c * slots) >> 5];          // slots is 1, 2, 4, 8, 16 or 32: a word holds 32 / slots values of c
  return (unsigned long long)((w >> ((c * slots) & 31)) & (slots == 32 ? 0xffffffffu : ((1u << slots) - 1u)));
}

static __global__ void __launch_bounds__(kMtNodes) k_mirror_t_count(const uint32_t* __restrict__ present, uint32_t n_nodes, uint32_t ntiles, int slots,
                                                                   uint32_t* __restrict__ cnt) {
  __shared__ uint32_t s_cnt[64];
  if (threadIdx.x < 64) s_cnt[threadIdx.x] = 0;
  __syncthreads();
  const unsigned long long mask = mt_mask(present, blockIdx.x * kMtNodes + threadIdx.x, n_nodes, slots);
  // only the columns some lane of the warp has; the two 32-bit halves of the mask one after the other
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const uint32_t m32 = (uint32_t)(mask >> (32 * half));
    for (uint32_t cols = __reduce_or_sync(0xffffffffu, m32); cols; cols &= cols - 1) {
      const int a = __ffs(cols) - 1;
      const unsigned bal = __ballot_sync(0xffffffffu, (m32 >> a) & 1u);
      if (lane_id() == 0) atomicAdd(&s_cnt[32 * half + a], (uint32_t)__popc(bal));
    }
  }
  __syncthreads();
  if ((int)threadIdx.x < slots) cnt[(size_t)threadIdx.x * ntiles + blockIdx.x] = s_cnt[threadIdx.x];
}

template <typename K>
__global__ void __launch_bounds__(kMtNodes) k_mirror_t_emit(const uint32_t* __restrict__ present, const int32_t* __restrict__ table, uint32_t n_nodes,
                                                           uint32_t ntiles, int slots, const uint32_t* __restrict__ base, int shift0, int shift1,
                                                           K* __restrict__ keys, float* __restrict__ tags) {
  constexpr int NW = kMtNodes / 32;
  __shared__ int32_t s_tag[kMtNodes * 65];
  __shared__ uint32_t s_wcnt[NW][64];
  __shared__ uint32_t s_base[64];
  const uint32_t c = blockIdx.x * kMtNodes + threadIdx.x;
  const int slots_log2 = 31 - __clz(slots);
  if ((int)threadIdx.x < slots) s_base[threadIdx.x] = base[(size_t)threadIdx.x * ntiles + blockIdx.x];
  const unsigned long long mask = mt_mask(present, c, n_nodes, slots);
  const uint32_t m32[2] = {(uint32_t)mask, (uint32_t)(mask >> 32)};
  const uint32_t warp_cols[2] = {__reduce_or_sync(0xffffffffu, m32[0]), __reduce_or_sync(0xffffffffu, m32[1])};
  for (int a = lane_id(); a < 64; a += 32) s_wcnt[warp_id()][a] = 0;
  __syncwarp();
#pragma unroll
  for (int half = 0; half < 2; ++half)
    for (uint32_t cols = warp_cols[half]; cols; cols &= cols - 1) {
      const int a = __ffs(cols) - 1;
      const unsigned bal = __ballot_sync(0xffffffffu, (m32[half] >> a) & 1u);
      if (lane_id() == 0) s_wcnt[warp_id()][32 * half + a] = __popc(bal);
    }
  __syncthreads();
  if (__syncthreads_or(mask != 0ull) == 0) return;       // nothing present in this tile
  // the tile's slots are contiguous in the table: a straight 16-byte-vector copy into the padded shared array, all of a
  // thread's reads in flight together (empty slots come along; their values are never used)
  const size_t tile_slot0 = (size_t)blockIdx.x * kMtNodes * slots;
  const int4* __restrict__ src = reinterpret_cast<const int4*>(table + tile_slot0);
  const uint32_t nvec = (uint32_t)min((size_t)(kMtNodes * slots / 4), ((size_t)n_nodes * slots - tile_slot0 + 3) / 4);
#pragma unroll 8
  for (uint32_t v = threadIdx.x; v < nvec; v += kMtNodes) {
    const int4 x = __ldcs(src + v);
    const int32_t e[4] = {x.x, x.y, x.z, x.w};
    const uint32_t i = v * 4;
    if (slots >= 4) {
      // the four slots of a vector belong to one c
      int32_t* dst = s_tag + (i >> slots_log2) * 65 + (i & (slots - 1));
      dst[0] = e[0]; dst[1] = e[1]; dst[2] = e[2]; dst[3] = e[3];
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) s_tag[((i + j) >> slots_log2) * 65 + ((i + j) & (slots - 1))] = e[j];
    }
  }
  // where each warp's rows of column a begin: the (a, tile) base plus the earlier warps' counts
  if (threadIdx.x < 64) {
    uint32_t run = s_base[threadIdx.x];
#pragma unroll
    for (int w = 0; w < NW; ++w) { const uint32_t n = s_wcnt[w][threadIdx.x]; s_wcnt[w][threadIdx.x] = run; run += n; }
  }
  __syncthreads();
  const int32_t* my_tags = s_tag + threadIdx.x * 65;
  const K ckey = (K)c << shift1;
  const uint32_t* my_base = s_wcnt[warp_id()];
#pragma unroll
  for (int half = 0; half < 2; ++half)
    for (uint32_t cols = warp_cols[half]; cols; cols &= cols - 1) {
      const int a = __ffs(cols) - 1;
      const bool mine = (m32[half] >> a) & 1u;
      const unsigned bal = __ballot_sync(0xffffffffu, mine);
      if (mine) {
        const uint32_t pos = my_base[32 * half + a] + __popc(bal & lanemask_lt());
        keys[pos] = ((K)(uint32_t)(32 * half + a) << shift0) | ckey;
        tags[pos] = ord2f(my_tags[32 * half + a]);
      }
    }
}

}  // namespace xlog
