// xlog_reduce_by_key_static: the segmented semiring reduce-by-key with its scratch memory in a
// fixed device array that is part of the library image, so the call allocates nothing.
//
// Who needs this: code that runs where device allocation is forbidden or not possible -- inside
// a latency-critical serving loop whose memory was handed out once at start-up, in a process
// whose memory pool is owned by another component (so a cudaMalloc here would bypass its
// accounting or fail), or on a stream where an implicit device synchronisation caused by an
// allocation is unacceptable.  Such callers pass inputs and outputs they already own and the
// library brings its own, bounded, scratch.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "../../include/xlog.h"
#include "common.cuh"
#include "relops.cuh"

namespace {

using namespace xlog;

constexpr int64_t kMaxRows = XLOG_STATIC_REDUCE_MAX_ROWS;
constexpr int64_t kMaxTiles = (kMaxRows + kRbkTile - 1) / kRbkTile;
// per tile: head count (4 B) + open-tail accumulator (8 B) + carry-in accumulator (8 B); one 256 B slot for the group total
constexpr size_t kHeadsOff = 0;
constexpr size_t kTailOff = (kMaxTiles * 4 + 255) / 256 * 256;
constexpr size_t kCarryOff = kTailOff + (kMaxTiles * 8 + 255) / 256 * 256;
constexpr size_t kTotalOff = kCarryOff + (kMaxTiles * 8 + 255) / 256 * 256;
constexpr size_t kScratchBytes = kTotalOff + 256;

// Every GPU that loads the library holds this array until the process exits.  In host code the
// name is only a handle; the device address comes from cudaGetSymbolAddress (below).
static __device__ __align__(256) unsigned char g_reduce_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};

// Once per device, with that device current: resolve the array's device address.
xlog_status scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return XLOG_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_reduce_scratch) != cudaSuccess || !p) return XLOG_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return XLOG_OK;
}

// The first CUDA error of the call, or cudaSuccess (the caller formats it: asking the runtime again would find it cleared).
template <typename Op>
cudaError_t run(cudaStream_t s, unsigned char* scratch, const uint32_t* keys, const float* tags, uint32_t n, uint32_t* out_keys,
                float* out_tags, int64_t* n_out) {
  typedef typename Op::A A;
  static_assert(sizeof(A) <= 8, "accumulator must fit the 8-byte scratch slots");
  uint32_t* heads = reinterpret_cast<uint32_t*>(scratch + kHeadsOff);
  A* tails = reinterpret_cast<A*>(scratch + kTailOff);
  A* carry = reinterpret_cast<A*>(scratch + kCarryOff);
  uint32_t* total = reinterpret_cast<uint32_t*>(scratch + kTotalOff);
  const unsigned tiles = (n + kRbkTile - 1) / kRbkTile;
  // every slot the later kernels read is written first by an earlier kernel of this call, so
  // nothing left behind by the previous call is ever observed
  k_rbk_tiles<uint32_t, Op><<<tiles, kRbkBlock, 0, s>>>(keys, tags, n, heads, tails);
  k_rbk_spine<Op><<<1, 1024, 0, s>>>(heads, tails, carry, tiles, total);
  k_rbk_emit<uint32_t, Op><<<tiles, kRbkBlock, 0, s>>>(keys, tags, n, heads, carry, out_keys, out_tags, (uint32_t*)nullptr);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  uint32_t u = 0;
  if ((e = cudaMemcpyAsync(&u, total, sizeof(u), cudaMemcpyDeviceToHost, s)) != cudaSuccess) return e;
  if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return e;
  *n_out = u;
  return cudaSuccess;
}

// [a, a + na) and [b, b + nb) share a byte
bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
  return a0 < b0 + nb && b0 < a0 + na;
}

}  // namespace

extern "C" xlog_status xlog_reduce_by_key_static(void* stream, xlog_semiring sr, const int32_t* keys, const float* tags, int64_t n,
                                                 int32_t* out_keys, float* out_tags, int64_t* n_out, char* errbuf, size_t errbuf_len) {
  const bool can_say = errbuf && errbuf_len;
  if (can_say) errbuf[0] = 0;
  if (!n_out || n < 0 || (int)sr < 0 || (int)sr > 3 || (n > 0 && (!keys || !tags || !out_keys || !out_tags))) {
    if (can_say) snprintf(errbuf, errbuf_len, "xlog_reduce_by_key_static: bad argument (n=%lld, semiring=%d)", (long long)n, (int)sr);
    return XLOG_ERR_INVALID_ARGUMENT;
  }
  if (n > kMaxRows) {
    if (can_say) snprintf(errbuf, errbuf_len, "xlog_reduce_by_key_static: n=%lld exceeds the static scratch limit of %lld rows",
                          (long long)n, (long long)kMaxRows);
    return XLOG_ERR_CAPACITY_EXCEEDED;
  }
  if (n == 0) { *n_out = 0; return XLOG_OK; }
  {
    // the emit kernel writes group u while other blocks still read rows >= u: an output on top of an input is a race
    const size_t bytes = (size_t)n * 4;
    if (overlaps(out_keys, bytes, keys, bytes) || overlaps(out_keys, bytes, tags, bytes) || overlaps(out_tags, bytes, keys, bytes) ||
        overlaps(out_tags, bytes, tags, bytes) || overlaps(out_keys, bytes, out_tags, bytes)) {
      if (can_say) snprintf(errbuf, errbuf_len, "xlog_reduce_by_key_static: the outputs may overlap neither the inputs nor each other");
      return XLOG_ERR_INVALID_ARGUMENT;
    }
  }
  unsigned char* scratch = nullptr;
  xlog_status st = scratch_for_current_device(&scratch);
  if (st != XLOG_OK) {
    if (can_say) snprintf(errbuf, errbuf_len, "xlog_reduce_by_key_static: cannot resolve the scratch array on the current device");
    return st;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint32_t* k = reinterpret_cast<const uint32_t*>(keys);       // keys are >= 0: same order as unsigned
  uint32_t* ok = reinterpret_cast<uint32_t*>(out_keys);
  cudaError_t e;
  switch (sr) {
    case XLOG_SR_MAXPLUS: e = run<OpMax>(s, scratch, k, tags, (uint32_t)n, ok, out_tags, n_out); break;
    case XLOG_SR_MINPLUS: e = run<OpMin>(s, scratch, k, tags, (uint32_t)n, ok, out_tags, n_out); break;
    case XLOG_SR_LOGSUMEXP: e = run<OpLse>(s, scratch, k, tags, (uint32_t)n, ok, out_tags, n_out); break;
    default: e = run<OpSum>(s, scratch, k, tags, (uint32_t)n, ok, out_tags, n_out); break;
  }
  if (e == cudaSuccess) return XLOG_OK;
  if (can_say) snprintf(errbuf, errbuf_len, "xlog_reduce_by_key_static: CUDA error: %s", cudaGetErrorString(e));
  return XLOG_ERR_CUDA;
}
