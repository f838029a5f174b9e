// xlog_device_copy / xlog_device_read: a plain device-to-device copy kernel and a read-only kernel of the library's own,
// used by the benchmark to measure the bandwidth of the memory level a working set lives in (buffers smaller than L2 give
// the L2 rate that the cache-resident join kernels are held against; larger buffers give the HBM rate).
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/xlog.h"
#include "common.cuh"

namespace {

constexpr int kReadPasses = 16;

__global__ void __launch_bounds__(256) k_copy16(const int4* __restrict__ src, int4* __restrict__ dst, uint64_t n16) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x * 4;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x * 4 + threadIdx.x; i < n16; i += stride) {
    int4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) if (i + u * 256 < n16) v[u] = src[i + u * 256];
#pragma unroll
    for (int u = 0; u < 4; ++u) if (i + u * 256 < n16) dst[i + u * 256] = v[u];
  }
}

// Read-only counterpart: eight 16-byte loads per thread in flight, folded into one word that is stored only if it takes a
// value no input produces in practice (so the loads cannot be dropped and nothing is written).
__global__ void __launch_bounds__(256) k_read16(const int4* __restrict__ src, uint64_t n16, int passes, uint32_t* __restrict__ sink) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x * 8;
  uint32_t acc = 0;
  for (int p = 0; p < passes; ++p)
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x * 8 + threadIdx.x; i < n16; i += stride) {
      int4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = i + u * 256 < n16 ? __ldcg(src + i + u * 256) : make_int4(0, 0, 0, 0);
#pragma unroll
      for (int u = 0; u < 8; ++u) acc ^= (uint32_t)(v[u].x ^ v[u].y ^ v[u].z ^ v[u].w) + (uint32_t)p;
    }
  if (acc == 0x9e3779b9u) sink[0] = acc;
}

// Random 4-byte reads (one 32-byte sector each) from a table of n4 words: eight independent loads per thread in flight,
// addresses from a multiplicative hash of a running counter.
__global__ void __launch_bounds__(256) k_gather4(const uint32_t* __restrict__ src, uint32_t n4, uint32_t per_thread, uint32_t* __restrict__ sink) {
  uint32_t x = (blockIdx.x * blockDim.x + threadIdx.x) * 2654435761u + 12345u;
  uint32_t acc = 0;
  for (uint32_t i = 0; i < per_thread; i += 8) {
    uint32_t v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      x = x * 1664525u + 1013904223u;
      v[u] = __ldcg(src + (uint32_t)(((uint64_t)(x ^ (x >> 15)) * n4) >> 32));
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) acc ^= v[u] + i;
  }
  if (acc == 0x9e3779b9u) sink[0] = acc;
}

}  // namespace

extern "C" xlog_status xlog_device_gather(void* stream, const void* src, uint64_t bytes, uint64_t reads, void* sink) {
  if (!src || !sink || bytes < 4 || bytes > ((uint64_t)1 << 34) || (bytes & 3u) || ((uintptr_t)src & 3u) || ((uintptr_t)sink & 3u)) return XLOG_ERR_INVALID_ARGUMENT;
  const unsigned grid = xlog::kSMs * 8;
  const uint64_t threads = (uint64_t)grid * 256;
  const uint64_t per_thread = ((reads + threads - 1) / threads + 7) / 8 * 8;
  if (per_thread > 0xffffffffull) return XLOG_ERR_INVALID_ARGUMENT;
  k_gather4<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint32_t*>(src), (uint32_t)(bytes / 4), (uint32_t)per_thread, static_cast<uint32_t*>(sink));
  return cudaGetLastError() == cudaSuccess ? XLOG_OK : XLOG_ERR_CUDA;
}

extern "C" xlog_status xlog_device_read(void* stream, const void* src, uint64_t bytes, int32_t repeats, void* sink) {
  if (!src || !sink || (bytes & 15u) || repeats < 1 || ((uintptr_t)src & 15u) || ((uintptr_t)sink & 3u)) return XLOG_ERR_INVALID_ARGUMENT;
  if (bytes == 0) return XLOG_OK;
  const uint64_t n16 = bytes / 16;
  const unsigned grid = (unsigned)((n16 + 2047) / 2048 < (uint64_t)xlog::kSMs * 8 ? (n16 + 2047) / 2048 : (uint64_t)xlog::kSMs * 8);
  // sixteen passes over the buffer per launch, so that a buffer of a few MB is not timed by its launch
  for (int r = 0; r < repeats; r += kReadPasses) {
    const int passes = repeats - r < kReadPasses ? repeats - r : kReadPasses;
    k_read16<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const int4*>(src), n16, passes, static_cast<uint32_t*>(sink));
  }
  return cudaGetLastError() == cudaSuccess ? XLOG_OK : XLOG_ERR_CUDA;
}

extern "C" xlog_status xlog_device_copy(void* stream, void* dst, const void* src, uint64_t bytes, int32_t repeats) {
  if (!dst || !src || (bytes & 15u) || repeats < 1 || ((uintptr_t)dst & 15u) || ((uintptr_t)src & 15u)) return XLOG_ERR_INVALID_ARGUMENT;
  if (bytes == 0) return XLOG_OK;
  const uint64_t n16 = bytes / 16;
  const unsigned grid = (unsigned)((n16 + 1023) / 1024 < (uint64_t)xlog::kSMs * 8 ? (n16 + 1023) / 1024 : (uint64_t)xlog::kSMs * 8);
  for (int r = 0; r < repeats; ++r) k_copy16<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const int4*>(src), static_cast<int4*>(dst), n16);
  return cudaGetLastError() == cudaSuccess ? XLOG_OK : XLOG_ERR_CUDA;
}
