// Four-cycle join  c4(x,y,z,w) :- r(x,y), s(y,z), t(z,w), u(w,x)  (paper: "Worst-case-optimal joins": coverage spans
// the triangle and 4-cycles; count -> device prefix scan -> materialise over flat sorted-column storage).
//
// The first two atoms are joined by the ordinary join kernels into the two-paths (x,y,z), sorted by (x,y,z).  The last
// variable is then bound by both remaining atoms at once: for every two-path the sorted out-list of z in t is intersected
// with the sorted in-list of x in u, so no three-path that u does not close is ever written.  A two-path's rows come out
// in increasing w, hence the output is already sorted by (x,y,z,w) and duplicate-free: no sort, no reduce.
//
// Work distribution: a thread per two-path while the shorter of its two lists has at most kC4Serial entries (the usual
// case: walk it, binary-search the other list from the last position reached); the two-paths of a warp with longer lists
// are then taken one after the other by the whole warp (32 walked entries per sweep, hits ranked by a ballot).
#pragma once
#include "common.cuh"

namespace xlog {

struct Cycle4 {
  KeyLayout L2;                  // layout of the two-path keys (x,y,z)
  KeyLayout L;                   // layout of the head relation (x,y,z,w)
  int64_t t_domain, u_domain;
  const uint32_t* t_off;         // t indexed on column 0: out-list of z = t_w[t_off[z] .. t_off[z+1]), ascending
  const int32_t* t_w;
  const float* t_tag;
  const uint32_t* u_off;         // u indexed on column 1: in-list of x = u_w[u_off[x] .. u_off[x+1]), ascending
  const int32_t* u_w;
  const float* u_tag;
  int times;                     // otimes is * (sum-product) instead of +
};

constexpr uint32_t kC4Serial = 16;

// EMIT = false: cnt[i] = number of w closing two-path i.  EMIT = true: writes them at off[i]...
template <typename K2, typename K, bool EMIT>
__global__ void __launch_bounds__(256) k_cycle4(Cycle4 P, const K2* __restrict__ keys2, const float* __restrict__ tags2, uint64_t n,
                                                uint32_t* __restrict__ cnt, const uint64_t* __restrict__ off,
                                                K* __restrict__ out_keys, float* __restrict__ out_tags) {
  const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  for (uint64_t base = warp * 32; base < n; base += nwarps * 32) {
    const uint64_t i = base + lane;
    const bool valid = i < n;
    uint32_t a0 = 0, a1 = 0, b0 = 0, b1 = 0;
    K prefix = 0;
    float tag = 0.f;
    uint64_t pos = 0;
    if (valid) {
      const K2 k2 = keys2[i];
      const int32_t x = key_col<K2>(P.L2, k2, 0), y = key_col<K2>(P.L2, k2, 1), z = key_col<K2>(P.L2, k2, 2);
      if (z < P.t_domain) { a0 = P.t_off[z]; a1 = P.t_off[z + 1]; }
      if (x < P.u_domain) { b0 = P.u_off[x]; b1 = P.u_off[x + 1]; }
      if (EMIT) {
        prefix = ((K)(uint32_t)x << P.L.shift[0]) | ((K)(uint32_t)y << P.L.shift[1]) | ((K)(uint32_t)z << P.L.shift[2]);
        tag = tags2[i];
        pos = off[i];
      }
    }
    const uint32_t la = a1 - a0, lb = b1 - b0;
    const bool any = valid && la && lb;
    const bool serial = any && min(la, lb) <= kC4Serial;
    uint32_t mine = 0;
    if (serial) {
      const bool walk_a = la <= lb;
      const int32_t* wl = walk_a ? P.t_w + a0 : P.u_w + b0;
      const int32_t* sl = walk_a ? P.u_w + b0 : P.t_w + a0;
      const uint32_t nw = walk_a ? la : lb, ns = walk_a ? lb : la;
      uint32_t lo = 0;
      for (uint32_t j = 0; j < nw && lo < ns; ++j) {
        const int32_t w = wl[j];
        uint32_t hi = ns;
        while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (sl[mid] < w) lo = mid + 1; else hi = mid; }
        if (lo < ns && sl[lo] == w) {
          if (EMIT) {
            const float wt = walk_a ? P.t_tag[a0 + j] : P.t_tag[a0 + lo];
            const float wu = walk_a ? P.u_tag[b0 + lo] : P.u_tag[b0 + j];
            out_keys[pos + mine] = prefix | ((K)(uint32_t)w << P.L.shift[3]);
            out_tags[pos + mine] = P.times ? (tag * wt) * wu : (tag + wt) + wu;
          }
          ++mine;
        }
      }
    }
    // the warp's two-paths with two long lists, one after the other
    unsigned big = __ballot_sync(0xffffffffu, any && !serial);
    while (big) {
      const int src = __ffs(big) - 1;
      big &= big - 1;
      const uint32_t A0 = __shfl_sync(0xffffffffu, a0, src), A1 = __shfl_sync(0xffffffffu, a1, src);
      const uint32_t B0 = __shfl_sync(0xffffffffu, b0, src), B1 = __shfl_sync(0xffffffffu, b1, src);
      const K pre = (K)__shfl_sync(0xffffffffu, (unsigned long long)prefix, src);
      const float tg = __shfl_sync(0xffffffffu, tag, src);
      uint64_t o = __shfl_sync(0xffffffffu, (unsigned long long)pos, src);
      const uint32_t LA = A1 - A0, LB = B1 - B0;
      const bool walk_a = LA <= LB;
      const int32_t* wl = walk_a ? P.t_w + A0 : P.u_w + B0;
      const int32_t* sl = walk_a ? P.u_w + B0 : P.t_w + A0;
      const uint32_t nw = walk_a ? LA : LB, ns = walk_a ? LB : LA;
      uint32_t floor = 0, total = 0;
      for (uint32_t j0 = 0; j0 < nw; j0 += 32) {
        const uint32_t j = j0 + lane;
        bool hit = false;
        int32_t w = 0;
        uint32_t lo = floor;
        if (j < nw) {
          w = wl[j];
          uint32_t hi = ns;
          while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (sl[mid] < w) lo = mid + 1; else hi = mid; }
          hit = lo < ns && sl[lo] == w;
        }
        floor = __shfl_sync(0xffffffffu, lo, 31);        // lanes past the end keep the previous floor: only read after the loop ends
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (EMIT && hit) {
          const float wt = walk_a ? P.t_tag[A0 + j] : P.t_tag[A0 + lo];
          const float wu = walk_a ? P.u_tag[B0 + lo] : P.u_tag[B0 + j];
          const uint64_t at = o + __popc(m & lanemask_lt());
          out_keys[at] = pre | ((K)(uint32_t)w << P.L.shift[3]);
          out_tags[at] = P.times ? (tg * wt) * wu : (tg + wt) + wu;
        }
        o += __popc(m);
        total += __popc(m);
      }
      if ((int)lane == src) mine = total;
    }
    if (!EMIT && valid) cnt[i] = mine;
  }
}

// The same join with u's in-list of x marked in a shared-memory bitmap.  The two-paths are sorted by x, so a block takes a
// chunk of them and works through its runs of equal x: mark the in-list (w values below kC4BmWords * 32), then a warp per
// two-path tests the entries of t's out-list of z against the bitmap (one load and a bit test per probe); only a hit, in
// the writing launch, needs its place in the in-list (for its tag): the in-list ascends, so the entries that fall into one
// bitmap word are neighbours, the entry that opens a word notes its place in a second shared-memory table, and a hit's
// place is that plus the marked bits below it in its word (in-lists of 65,536 entries and more are searched instead).
// Then the marked words are cleared again.  Dynamic shared memory: kC4BmSmem bytes.
constexpr uint32_t kC4BmWords = 8192;    // 32 KB of shared memory: w < 2^18
constexpr uint32_t kC4Chunk = 1024;      // two-paths per block step
constexpr size_t kC4BmSmem = (size_t)kC4BmWords * 4 + (size_t)kC4BmWords * 2;

template <typename K2, typename K, bool EMIT>
__global__ void __launch_bounds__(256) k_cycle4_bitmap(Cycle4 P, const K2* __restrict__ keys2, const float* __restrict__ tags2, uint64_t n,
                                                       uint32_t* __restrict__ cnt, const uint64_t* __restrict__ off,
                                                       K* __restrict__ out_keys, float* __restrict__ out_tags) {
  extern __shared__ uint32_t c4_smem[];
  uint32_t* bm = c4_smem;
  uint16_t* first = reinterpret_cast<uint16_t*>(c4_smem + kC4BmWords);      // per word: place in the in-list of the first entry marked in it
  __shared__ unsigned long long run_end_s;
  const unsigned lane = lane_id(), wid = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  for (uint32_t i = threadIdx.x; i < kC4BmWords; i += blockDim.x) bm[i] = 0u;
  __syncthreads();
  const uint64_t nchunks = (n + kC4Chunk - 1) / kC4Chunk;
  for (uint64_t ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
    uint64_t cur = ch * kC4Chunk;
    const uint64_t cend = min(n, cur + (uint64_t)kC4Chunk);
    while (cur < cend) {
      const int32_t x = key_col<K2>(P.L2, keys2[cur], 0);
      if (threadIdx.x == 0) {                              // end of the run of x inside the chunk
        uint64_t lo = cur + 1, hi = cend;
        while (lo < hi) { const uint64_t mid = (lo + hi) >> 1; if (key_col<K2>(P.L2, keys2[mid], 0) <= x) lo = mid + 1; else hi = mid; }
        run_end_s = lo;
      }
      uint32_t b0 = 0, b1 = 0;
      if (x < P.u_domain) { b0 = P.u_off[x]; b1 = P.u_off[x + 1]; }
      const bool ranked = EMIT && b1 - b0 < 65536u;
      for (uint32_t j = b0 + threadIdx.x; j < b1; j += blockDim.x) {
        const uint32_t w = (uint32_t)P.u_w[j];
        atomicOr(&bm[w >> 5], 1u << (w & 31));
        if (ranked && (j == b0 || ((uint32_t)P.u_w[j - 1] >> 5) != (w >> 5))) first[w >> 5] = (uint16_t)(j - b0);
      }
      __syncthreads();
      const uint64_t rend = run_end_s;
      if (b1 > b0) {
        // 32 two-paths at a time: their keys and list bounds are read by one lane each, then the warp takes them in turn,
        // two sweeps of t's out-list per step
        for (uint64_t base = cur + (uint64_t)wid * 32; base < rend; base += (uint64_t)nwarp * 32) {
          const uint64_t i = base + lane;
          const bool valid = i < rend;
          uint32_t a0 = 0, a1 = 0;
          K prefix = 0;
          float tag = 0.f;
          uint64_t pos = 0;
          if (valid) {
            const K2 k2 = keys2[i];
            const int32_t y = key_col<K2>(P.L2, k2, 1), z = key_col<K2>(P.L2, k2, 2);
            if (z < P.t_domain) { a0 = P.t_off[z]; a1 = P.t_off[z + 1]; }
            if (EMIT) {
              prefix = ((K)(uint32_t)x << P.L.shift[0]) | ((K)(uint32_t)y << P.L.shift[1]) | ((K)(uint32_t)z << P.L.shift[2]);
              tag = tags2[i];
              pos = off[i];
            }
          }
          uint32_t mine = 0;
          unsigned todo = __ballot_sync(0xffffffffu, valid && a1 > a0);
          while (todo) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            const uint32_t A0 = __shfl_sync(0xffffffffu, a0, src), A1 = __shfl_sync(0xffffffffu, a1, src);
            K pre = 0;
            float tg = 0.f;
            uint64_t o = 0;
            if (EMIT) {
              pre = (K)__shfl_sync(0xffffffffu, (unsigned long long)prefix, src);
              tg = __shfl_sync(0xffffffffu, tag, src);
              o = __shfl_sync(0xffffffffu, (unsigned long long)pos, src);
            }
            uint32_t total = 0;
            for (uint32_t j0 = A0; j0 < A1; j0 += 64) {
              const uint32_t j[2] = {j0 + lane, j0 + 32 + lane};
              uint32_t w[2];
              bool hit[2];
#pragma unroll
              for (int u = 0; u < 2; ++u) w[u] = j[u] < A1 ? (uint32_t)P.t_w[j[u]] : 0xffffffffu;
#pragma unroll
              for (int u = 0; u < 2; ++u) hit[u] = (w[u] >> 5) < kC4BmWords && ((bm[w[u] >> 5] >> (w[u] & 31)) & 1u);
              const unsigned m0 = __ballot_sync(0xffffffffu, hit[0]), m1 = __ballot_sync(0xffffffffu, hit[1]);
              if (EMIT) {
#pragma unroll
                for (int u = 0; u < 2; ++u)
                  if (hit[u]) {
                    uint32_t lo = b0, hi = b1;             // where w sits in the in-list: its tag
                    if (ranked) lo = b0 + first[w[u] >> 5] + __popc(bm[w[u] >> 5] & ((1u << (w[u] & 31)) - 1u));
                    else while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if ((uint32_t)P.u_w[mid] < w[u]) lo = mid + 1; else hi = mid; }
                    const uint64_t at = o + total + (u ? __popc(m0) : 0) + __popc((u ? m1 : m0) & lanemask_lt());
                    out_keys[at] = pre | ((K)w[u] << P.L.shift[3]);
                    out_tags[at] = P.times ? (tg * P.t_tag[j[u]]) * P.u_tag[lo] : (tg + P.t_tag[j[u]]) + P.u_tag[lo];
                  }
              }
              total += __popc(m0) + __popc(m1);
            }
            if ((int)lane == src) mine = total;
          }
          if (!EMIT && valid) cnt[i] = mine;
        }
      } else if (!EMIT) {
        for (uint64_t i = cur + threadIdx.x; i < rend; i += blockDim.x) cnt[i] = 0u;
      }
      __syncthreads();
      for (uint32_t j = b0 + threadIdx.x; j < b1; j += blockDim.x) bm[(uint32_t)P.u_w[j] >> 5] = 0u;
      __syncthreads();
      cur = rend;
    }
  }
}

// ---- the binary-join chain of the four-cycle ---------------------------------------------------------------------------
// The plan a binary-join engine takes: every three-path (x,y,z,w) of r, s and t is written out (two-paths joined with t on
// z), and u is then probed with (w, x) (k_chain_probe_* in triangle.cuh).  Chosen by the skew test when the three-paths
// stay within a small multiple of the inputs; the multiway plan above never writes a three-path that u does not close.
template <typename K2>
__global__ void __launch_bounds__(256) k_c4_chain_count(Cycle4 P, const K2* __restrict__ keys2, uint64_t n, uint32_t* __restrict__ cnt) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const int32_t z = key_col<K2>(P.L2, keys2[i], 2);
    cnt[i] = z < P.t_domain ? P.t_off[z + 1] - P.t_off[z] : 0u;
  }
}

// A warp takes 32 two-paths; each one's run of t is written by the whole warp (coalesced however long the run).
template <typename K2, typename K>
__global__ void __launch_bounds__(256) k_c4_chain_expand(Cycle4 P, const K2* __restrict__ keys2, const float* __restrict__ tags2, uint64_t n,
                                                         const uint64_t* __restrict__ off, K* __restrict__ out_keys, float* __restrict__ out_tags) {
  const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  const unsigned lane = lane_id();
  for (uint64_t base = warp * 32; base < n; base += nwarps * 32) {
    const uint64_t i = base + lane;
    uint32_t a0 = 0, a1 = 0;
    K prefix = 0;
    float tag = 0.f;
    uint64_t pos = 0;
    if (i < n) {
      const K2 k2 = keys2[i];
      const int32_t x = key_col<K2>(P.L2, k2, 0), y = key_col<K2>(P.L2, k2, 1), z = key_col<K2>(P.L2, k2, 2);
      if (z < P.t_domain) { a0 = P.t_off[z]; a1 = P.t_off[z + 1]; }
      prefix = ((K)(uint32_t)x << P.L.shift[0]) | ((K)(uint32_t)y << P.L.shift[1]) | ((K)(uint32_t)z << P.L.shift[2]);
      tag = tags2[i];
      pos = off[i];
    }
    unsigned todo = __ballot_sync(0xffffffffu, a1 > a0);
    while (todo) {
      const int src = __ffs(todo) - 1;
      todo &= todo - 1;
      const uint32_t A0 = __shfl_sync(0xffffffffu, a0, src), A1 = __shfl_sync(0xffffffffu, a1, src);
      const K pre = (K)__shfl_sync(0xffffffffu, (unsigned long long)prefix, src);
      const float tg = __shfl_sync(0xffffffffu, tag, src);
      const uint64_t o = __shfl_sync(0xffffffffu, (unsigned long long)pos, src);
      for (uint32_t j = lane; j < A1 - A0; j += 32) {
        out_keys[o + j] = pre | ((K)(uint32_t)P.t_w[A0 + j] << P.L.shift[3]);
        const float wt = P.t_tag[A0 + j];
        out_tags[o + j] = P.times ? tg * wt : tg + wt;
      }
    }
  }
}

}  // namespace xlog
