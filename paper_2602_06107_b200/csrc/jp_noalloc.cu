// The batch-level lambda from an acceptance budget, for callers that must not
// allocate: the scratch that the budget solve needs (per-row flag, ratio and
// log-ratio, and one block of scalars) lives in a file-scope device array of a
// fixed size instead of a context's workspace.
//
// The array's name is usable as an address only in device code.  Host code gets
// the device address once per device from cudaGetSymbolAddress, with that device
// current, and hands it to the kernels.
#include <cuda_runtime.h>

#include <mutex>

#include "jp_internal.h"

namespace jp {
namespace {

constexpr int64_t kMaxRows = JP_STATIC_MAX_ROWS;
constexpr size_t kOffScalars = 0;                                        // Scalars
constexpr size_t kOffSolve = 1024;                                       // SolvePartials
constexpr size_t kOffRatio = kOffSolve + sizeof(SolvePartials);          // double[kMaxRows]
constexpr size_t kOffDval = kOffRatio + sizeof(double) * kMaxRows;       // float[kMaxRows]
constexpr size_t kOffFlag = kOffDval + sizeof(float) * kMaxRows;         // uint8_t[kMaxRows]
constexpr size_t kScratchBytes = kOffFlag + kMaxRows;
static_assert(sizeof(Scalars) <= kOffSolve, "the scalar block must fit before the arrays");

// 1.7 MB held by every device that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {};

// flag[i] = row i takes part (mask == NULL: every row does)
__global__ void static_flags_kernel(int64_t T, const uint8_t* mask, uint8_t* flag) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < T) flag[i] = (mask == nullptr || mask[i] != 0) ? 1 : 0;
}

}  // namespace
}  // namespace jp

extern "C" jp_status jp_budget_lambda_static(const float* logp_actor, const float* logp_policy,
                                             const uint8_t* mask, int64_t T, float budget, float* out_lambda,
                                             void* cuda_stream) {
  using namespace jp;
  if (T < 0 || !out_lambda || (T > 0 && (!logp_actor || !logp_policy))) return JP_ERR_INVALID_ARG;
  if (!(budget > 0.f) || budget > 1.f) return JP_ERR_INVALID_ARG;
  if (T > kMaxRows) return JP_ERR_TOO_LARGE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return JP_ERR_CUDA;
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
      // first call on this device: resolve the array's device address (no allocation)
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return JP_ERR_CUDA;
      g_scratch_addr[dev] = (unsigned char*)p;
    }
    base = g_scratch_addr[dev];
  }
  cudaStream_t s = (cudaStream_t)cuda_stream;
  Scalars* sc = (Scalars*)(base + kOffScalars);
  EpilogueArgs a{};
  a.T = T;
  a.sc = sc;
  a.solve = (SolvePartials*)(base + kOffSolve);
  a.rec.ratio = (double*)(base + kOffRatio);
  a.rec.dval = (float*)(base + kOffDval);
  a.rec.flag = (uint8_t*)(base + kOffFlag);
  a.rec.lq = const_cast<float*>(logp_actor);      // read only by the kernels below
  a.rec.lp = const_cast<float*>(logp_policy);
  // the array keeps the last call's contents: the scalar block starts from a known state,
  // and flag / ratio / dval are rewritten for every row in [0, T) before they are read
  cudaError_t e = launch_reset(sc, 1.0f, s);
  if (e != cudaSuccess) return JP_ERR_CUDA;
  if (T > 0) {
    static_flags_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(T, mask, a.rec.flag);
    if (cudaGetLastError() != cudaSuccess) return JP_ERR_CUDA;
    int n = 0;
    e = launch_budget_solve(a, (double)budget, s, &n);
    if (e != cudaSuccess) return JP_ERR_CUDA;
  }
  e = cudaMemcpyAsync(out_lambda, &sc->lambda, sizeof(float), cudaMemcpyDeviceToDevice, s);
  return e == cudaSuccess ? JP_OK : JP_ERR_CUDA;
}
