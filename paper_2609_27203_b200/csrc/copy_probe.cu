// xlog_device_copy: a plain device-to-device copy kernel of the library's own, used by the benchmark to measure the
// bandwidth of the memory level a working set lives in (a pair of buffers smaller than L2 copied back and forth gives the
// L2 rate that the cache-resident join kernels are held against; larger buffers give the HBM rate).
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/xlog.h"
#include "common.cuh"

namespace {

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

}  // namespace

extern "C" xlog_status xlog_device_copy(void* stream, void* dst, const void* src, uint64_t bytes, int32_t repeats) {
  if (!dst || !src || (bytes & 15u) || repeats < 1 || ((uintptr_t)dst & 15u) || ((uintptr_t)src & 15u)) return XLOG_ERR_INVALID_ARGUMENT;
  if (bytes == 0) return XLOG_OK;
  const uint64_t n16 = bytes / 16;
  const unsigned grid = (unsigned)((n16 + 1023) / 1024 < (uint64_t)xlog::kSMs * 8 ? (n16 + 1023) / 1024 : (uint64_t)xlog::kSMs * 8);
  for (int r = 0; r < repeats; ++r) k_copy16<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const int4*>(src), static_cast<int4*>(dst), n16);
  return cudaGetLastError() == cudaSuccess ? XLOG_OK : XLOG_ERR_CUDA;
}
