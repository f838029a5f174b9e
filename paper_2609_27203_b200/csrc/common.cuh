// Shared device-side definitions: key layouts, semiring operators, warp/block primitives.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <math.h>

namespace xlog {

constexpr int kMaxArity = 4;
constexpr int kMaxVars = 8;
constexpr int kSMs = 148;                 // B200: 2 dies x 74 SMs; grids are sized in multiples of this

// Device error word bits (set by kernels, read by the host after each round).
enum : uint32_t {
  kErrHeadRange = 1u,        // head column value left [0, 2^bits)
  kErrNegativeKey = 2u,
  kErrBadTag = 4u,           // NaN or semiring zero
  kErrCountOverflow = 8u,
  kErrNotSorted = 16u,       // invariant check failed
  kErrInternal = 32u,
};

// Bit layout of a packed row key: column c occupies `bits[c]` bits at `shift[c]`;
// column 0 is most significant, so unsigned key order == lexicographic row order.
struct KeyLayout {
  int arity;
  int shift[kMaxArity];
  uint32_t mask[kMaxArity];               // (1 << bits) - 1, bits <= 31
  int total_bits;
};

// Optional order-preserving dictionaries: a column whose values come from a small set stores the
// rank of the value in the sorted set instead of the value (dense ids, as the paper's symbol table
// makes strings dense: Section "Reversible symbols").  n[c] == 0: column c holds plain values.
struct DictSet {
  const int32_t* v[kMaxArity];
  uint32_t n[kMaxArity];
};
__device__ __forceinline__ uint32_t dict_rank(const int32_t* v, uint32_t n, int64_t value) {   // lower bound
  uint32_t lo = 0, hi = n;
  while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if ((int64_t)v[mid] < value) lo = mid + 1; else hi = mid; }
  return lo;
}

template <typename K>
__host__ __device__ __forceinline__ K pack_key(const KeyLayout& L, const int32_t* cols) {
  K k = 0;
#pragma unroll
  for (int c = 0; c < kMaxArity; ++c)
    if (c < L.arity) k |= (K)((uint32_t)cols[c]) << L.shift[c];
  return k;
}
template <typename K>
__host__ __device__ __forceinline__ int32_t key_col(const KeyLayout& L, K k, int c) {
  return (int32_t)((uint32_t)(k >> L.shift[c]) & L.mask[c]);
}

// ---- semiring operators -------------------------------------------------------
// Each operator has an accumulator type A, lift (tag -> A), combine (associative),
// lower (A -> tag).  MAX/MIN are exact and order-independent; LSE carries
// (max, sum of exp(v - max)) so that a fixed combination tree gives a result that is
// reproducible run to run and accurate to a few ulp; SUM accumulates in double.
struct OpMax {
  typedef float A;
  static constexpr int id = 0;
  __device__ __forceinline__ static A lift(float v) { return v; }
  __device__ __forceinline__ static A combine(A a, A b) { return fmaxf(a, b); }
  __device__ __forceinline__ static float lower(A a) { return a; }
  __device__ __forceinline__ static A identity() { return -INFINITY; }
  __device__ __forceinline__ static bool better(float a, float b) { return a > b; }
};
struct OpMin {
  typedef float A;
  static constexpr int id = 1;
  __device__ __forceinline__ static A lift(float v) { return v; }
  __device__ __forceinline__ static A combine(A a, A b) { return fminf(a, b); }
  __device__ __forceinline__ static float lower(A a) { return a; }
  __device__ __forceinline__ static A identity() { return INFINITY; }
  __device__ __forceinline__ static bool better(float a, float b) { return a < b; }
};
struct OpLse {
  typedef float2 A;                        // x = running max, y = sum exp(v - max)
  static constexpr int id = 2;
  __device__ __forceinline__ static A lift(float v) { return make_float2(v, 1.f); }
  __device__ __forceinline__ static A combine(A a, A b) {
    if (a.y == 0.f) return b;
    if (b.y == 0.f) return a;
    const float m = fmaxf(a.x, b.x);
    return make_float2(m, a.y * expf(a.x - m) + b.y * expf(b.x - m));
  }
  __device__ __forceinline__ static float lower(A a) { return a.x + logf(a.y); }
  __device__ __forceinline__ static A identity() { return make_float2(-INFINITY, 0.f); }
  __device__ __forceinline__ static bool better(float, float) { return false; }
};
struct OpSum {
  typedef double A;
  static constexpr int id = 3;
  __device__ __forceinline__ static A lift(float v) { return (double)v; }
  __device__ __forceinline__ static A combine(A a, A b) { return a + b; }
  __device__ __forceinline__ static float lower(A a) { return (float)a; }
  __device__ __forceinline__ static A identity() { return 0.0; }
  __device__ __forceinline__ static bool better(float, float) { return false; }
};

// ---- shuffles for the accumulator types ---------------------------------------
__device__ __forceinline__ float shfl_up(float v, int d) { return __shfl_up_sync(0xffffffffu, v, d); }
__device__ __forceinline__ double shfl_up(double v, int d) { return __shfl_up_sync(0xffffffffu, v, d); }
__device__ __forceinline__ float2 shfl_up(float2 v, int d) {
  return make_float2(__shfl_up_sync(0xffffffffu, v.x, d), __shfl_up_sync(0xffffffffu, v.y, d));
}
__device__ __forceinline__ float shfl_down(float v, int d) { return __shfl_down_sync(0xffffffffu, v, d); }
__device__ __forceinline__ double shfl_down(double v, int d) { return __shfl_down_sync(0xffffffffu, v, d); }
__device__ __forceinline__ float2 shfl_down(float2 v, int d) {
  return make_float2(__shfl_down_sync(0xffffffffu, v.x, d), __shfl_down_sync(0xffffffffu, v.y, d));
}
__device__ __forceinline__ float shfl_idx(float v, int l) { return __shfl_sync(0xffffffffu, v, l); }
__device__ __forceinline__ double shfl_idx(double v, int l) { return __shfl_sync(0xffffffffu, v, l); }
__device__ __forceinline__ float2 shfl_idx(float2 v, int l) {
  return make_float2(__shfl_sync(0xffffffffu, v.x, l), __shfl_sync(0xffffffffu, v.y, l));
}

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ unsigned warp_id() { return threadIdx.x >> 5; }
__device__ __forceinline__ unsigned lanemask_lt() { return (1u << lane_id()) - 1u; }

// Inclusive warp scan (sum).
template <typename T>
__device__ __forceinline__ T warp_scan_incl(T v) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    T n = __shfl_up_sync(0xffffffffu, v, d);
    if ((int)lane_id() >= d) v += n;
  }
  return v;
}

// Exclusive block scan (sum) of one value per thread; `total` is returned to every
// thread.  `sh` must hold BLOCK/32 + 1 elements; the caller may reuse it after the call.
template <int BLOCK, typename T>
__device__ __forceinline__ T block_scan_excl(T v, T* sh, T& total) {
  constexpr int W = BLOCK / 32;
  const T incl = warp_scan_incl(v);
  if (lane_id() == 31) sh[warp_id()] = incl;
  __syncthreads();
  if (warp_id() == 0) {
    T w = lane_id() < (unsigned)W ? sh[lane_id()] : T(0);
    const T wi = warp_scan_incl(w);
    if (lane_id() < (unsigned)W) sh[lane_id()] = wi - w;
    if (lane_id() == (unsigned)(W - 1)) sh[W] = wi;
  }
  __syncthreads();
  const T r = sh[warp_id()] + incl - v;
  total = sh[W];
  __syncthreads();
  return r;
}

// order-preserving map float -> int32 (so integer atomicMin/atomicMax implement the float ones)
__device__ __forceinline__ int32_t f2ord(float f) { const int32_t i = __float_as_int(f); return i ^ ((i >> 31) & 0x7fffffff); }
__device__ __forceinline__ float ord2f(int32_t i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

}  // namespace xlog
