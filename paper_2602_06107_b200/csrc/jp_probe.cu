// Measurement aid: how fast this GPU streams a buffer through plain kernels, so that
// the row stream's achieved bandwidth can be read against a read-only rate as well as
// against a copy.  Not part of the method.
#include <cuda_runtime.h>

#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {
namespace {

constexpr int PNT = 512;
constexpr int PUNROLL = 4;

// Each thread walks the buffer in 16-byte vectors strided by the grid; with dst the
// vectors are written back out (a copy), without it they are folded into one word per
// thread that is stored only if it is a value the data will not produce.
__global__ void __launch_bounds__(PNT) probe_kernel(const uint4* src, uint4* dst, int64_t nvec, uint32_t* sink) {
  const int64_t stride = (int64_t)gridDim.x * PNT;
  int64_t i = (int64_t)blockIdx.x * PNT + threadIdx.x;
  uint32_t acc = 0u;
  for (; i + (PUNROLL - 1) * stride < nvec; i += PUNROLL * stride) {
    uint4 v[PUNROLL];
#pragma unroll
    for (int j = 0; j < PUNROLL; ++j) v[j] = ldg_stream(src + i + j * stride);
#pragma unroll
    for (int j = 0; j < PUNROLL; ++j) {
      if (dst) stg_stream(dst + i + j * stride, v[j]);
      else acc ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
    }
  }
  for (; i < nvec; i += stride) {
    const uint4 v = ldg_stream(src + i);
    if (dst) stg_stream(dst + i, v);
    else acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  if (!dst && acc == 0x9e3779b9u && sink) *sink = acc;
}

}  // namespace
}  // namespace jp

extern "C" jp_status jp_probe_stream(const void* src, void* dst, int64_t bytes, int reps, void* cuda_stream,
                                     float* out_ms_per_rep) {
  using namespace jp;
  if (!src || bytes < 16 || reps < 1 || !out_ms_per_rep) return JP_ERR_INVALID_ARG;
  if (((uintptr_t)src & 15u) || ((uintptr_t)dst & 15u)) return JP_ERR_ALIGNMENT;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess) return JP_ERR_CUDA;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return JP_ERR_CUDA;
  const int64_t nvec = bytes / 16;
  const int grid = sms * 4;
  probe_kernel<<<grid, PNT, 0, s>>>((const uint4*)src, (uint4*)dst, nvec, nullptr);   // warm-up
  cudaEventRecord(e0, s);
  for (int r = 0; r < reps; ++r) probe_kernel<<<grid, PNT, 0, s>>>((const uint4*)src, (uint4*)dst, nvec, nullptr);
  cudaEventRecord(e1, s);
  cudaError_t e = cudaEventSynchronize(e1);
  float ms = 0.f;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return JP_ERR_CUDA;
  *out_ms_per_rep = ms / (float)reps;
  return JP_OK;
}
