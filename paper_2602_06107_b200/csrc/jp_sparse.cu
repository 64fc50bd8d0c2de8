// Z_approx when the rollout model is known only through what the rollout stored
// (Algorithm 1, Phase 1: per token log p_inf(a_t) and the log-probabilities of the k_inf
// most likely tokens, TopK_inf(s_t); Phase 2, step 2: V_k = TopK_inf U TopK_new and
// Z_approx = sum over V_k of min(p_inf(x), p_new(x) / lambda)).
//
// The row stream has left, per row, the policy's log-sum-exp and TopK_new with the policy
// logit of every entry.  Here, one warp per row:
//   stored entries x in TopK_inf   min(p_inf(x), p_new(x) / lambda) with p_inf(x) from the
//                                  record and p_new(x) = exp(zp[x] - lse_p), zp[x] fetched
//                                  from the policy row (k_inf scattered 2- or 4-byte reads);
//   entries of TopK_new not stored the paper's sum needs p_inf(x), which nobody kept.  Two
//                                  readings: leave the term out (z_lower: still a lower bound
//                                  of Z, which Section 4.4.2's correction assumes), or bound
//                                  it by the smallest stored probability and all such terms
//                                  together by the mass the record leaves (z_upper).
// Both are written if asked for; the one the call selected goes into the records as the
// row's Z_approx, from where acceptance, kappa and the weights proceed unchanged.
#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {
namespace {

constexpr int SZ_NT = 256;
constexpr int SZ_WARPS = SZ_NT / 32;

template <int DT>
__global__ void __launch_bounds__(SZ_NT) sparse_z_kernel(SparseZArgs A) {
  __shared__ int32_t s_idx[SZ_WARPS][JP_MAX_TOPK];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t r = (int64_t)blockIdx.x * SZ_WARPS + warp;
  if (r >= A.T) return;
  const int k = A.k, k_inf = A.k_inf;
  const bool valid = A.rec.flag[r] == kRowValid;
  double z_lo = 0.0, z_hi = 0.0;
  if (valid) {
    const double log_lambda = log((double)A.sc->lambda);
    const double cp = (double)A.rec.lse_p[r] + (double)A.rec.lse_p_lo[r] + log_lambda;   // p_new / lambda = exp(zp - cp)
    const char* rp = (const char*)A.zp + r * A.ld * Vec<DT>::ESIZE;
    double sum = 0.0, mass = 0.0, p_min = 1.0;
    int n_stored = 0;
    for (int j = lane; j < k_inf; j += 32) {
      int32_t x = A.inf_idx[r * k_inf + j];
      if (x < 0 || (int64_t)x >= A.V) x = -1;                 // an empty or impossible place
      s_idx[warp][j] = x;
      if (x >= 0) {
        const double q = exp((double)A.inf_logp[r * k_inf + j]);
        const double p = exp((double)Vec<DT>::load_scalar(rp, x) - cp);
        sum += fmin(q, p);
        mass += q;
        p_min = fmin(p_min, q);
        n_stored += 1;
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      sum += __shfl_xor_sync(0xffffffffu, sum, off);
      mass += __shfl_xor_sync(0xffffffffu, mass, off);
      p_min = fmin(p_min, __shfl_xor_sync(0xffffffffu, p_min, off));
      n_stored += __shfl_xor_sync(0xffffffffu, n_stored, off);
    }
    __syncwarp();
    if (n_stored == 0) p_min = 1.0;
    double unknown = 0.0;
    const int64_t base = r * (2 * k) + k;                     // TopK_new is the second list of the record
    for (int j = lane; j < k; j += 32) {
      const int32_t x = A.rec.idx[base + j];
      bool count = x >= 0;
      if (count)
        for (int i = 0; i < k_inf; ++i) count &= (s_idx[warp][i] != x);
      if (count) unknown += fmin(p_min, exp((double)A.rec.zp[base + j] - cp));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) unknown += __shfl_xor_sync(0xffffffffu, unknown, off);
    z_lo = sum;
    z_hi = sum + fmin(unknown, fmax(0.0, 1.0 - mass));
  }
  if (lane == 0) {
    A.rec.zk[r] = (float)(A.cap ? z_hi : z_lo);
    if (A.out_z_lower) A.out_z_lower[r] = (float)z_lo;
    if (A.out_z_upper) A.out_z_upper[r] = (float)z_hi;
  }
  if (A.out_idx_p || A.out_val_p) {
    const int64_t base = r * (2 * k) + k;
    for (int j = lane; j < k; j += 32) {
      if (A.out_idx_p) A.out_idx_p[r * k + j] = valid ? A.rec.idx[base + j] : -1;
      if (A.out_val_p) A.out_val_p[r * k + j] = valid ? A.rec.zp[base + j] : 0.f;
    }
  }
}

}  // namespace

cudaError_t launch_sparse_z(const SparseZArgs& a, cudaStream_t s) {
  if (a.T <= 0) return cudaSuccess;
  const unsigned blocks = (unsigned)((a.T + SZ_WARPS - 1) / SZ_WARPS);
  if (a.dtype == JP_BF16) sparse_z_kernel<JP_BF16><<<blocks, SZ_NT, 0, s>>>(a);
  else sparse_z_kernel<JP_F32><<<blocks, SZ_NT, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace jp
