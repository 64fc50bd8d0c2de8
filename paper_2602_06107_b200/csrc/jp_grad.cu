// Fused gradient of the joint objective (Eq. sys_joint_obj) with respect to
// both logit tensors.  With the loss to minimise
//   J = -L^{PPO-OBRS}(theta) - L^{PPO}(omega) + lambda_distill L^{distill}(omega)
// taken as a mean over the N valid proposed tokens and evaluated where the PPO
// ratios and F are 1 (Eq. obrs_ppo, Eq. ppo_rollout, Eq. distill_loss):
//   d_policy[t,v] = cp (1[v=x_t] - p_t(v)),              cp = -(g/N) Mask_t w_t A_t
//   d_actor[t,v]  = ca (1[v=x_t] - q_t(v)) + cd (q_t(v) - p_t(v)),
//                                       ca = -(g/N) A_t,  cd = g lambda_distill / N
// One pass: both rows are read once (the policy row only if cp or cd is
// non-zero), both bf16 gradient rows are written once with 16-byte stores.
// Masked rows are zero-filled without being read.
#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {

constexpr int GNT = 256;
constexpr int GUNROLL = 2;
constexpr int GCTAS_PER_SM = 3;

__device__ __forceinline__ uint4 ld_plain(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p)
               : "memory");
  return v;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&h;
}

// 8 columns starting at c0: bf16 in, bf16 out.
__device__ __forceinline__ void grad8(const uint4& va, const uint4& vp, float lsa, float lsp,
                                      float kq, float kp_actor, float ca, float cp, int64_t c0,
                                      int64_t x, uint4& oa, uint4& op) {
  float ga[8], gp[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    float q = ex2_approx(fmaf(Vec<JP_BF16>::get(va, e), kLog2e, -lsa));
    float p = ex2_approx(fmaf(Vec<JP_BF16>::get(vp, e), kLog2e, -lsp));
    float hot = (c0 + e == x) ? 1.f : 0.f;
    ga[e] = fmaf(kq, q, fmaf(kp_actor, p, ca * hot));   // (cd - ca) q - cd p + ca 1[v=x]
    gp[e] = cp * (hot - p);
  }
  oa = make_uint4(pack_bf16x2(ga[0], ga[1]), pack_bf16x2(ga[2], ga[3]), pack_bf16x2(ga[4], ga[5]),
                  pack_bf16x2(ga[6], ga[7]));
  op = make_uint4(pack_bf16x2(gp[0], gp[1]), pack_bf16x2(gp[2], gp[3]), pack_bf16x2(gp[4], gp[5]),
                  pack_bf16x2(gp[6], gp[7]));
}

template <int DT>
__global__ void __launch_bounds__(GNT, GCTAS_PER_SM) grad_kernel(GradArgs A) {
  __shared__ int s_row;
  const int tid = threadIdx.x;
  const double Nd = (double)(A.n_valid > 0 ? A.n_valid : A.sc->stats.n_valid);
  const float g_over_n = Nd > 0.0 ? (float)((double)A.grad_out / Nd) : 0.f;
  const float cd = g_over_n * A.lambda_distill;
  const int64_t nvec8 = A.V / 8;            // groups of 8 columns (16 B of bf16 output)
  const int tail = (int)(A.V - nvec8 * 8);
  for (;;) {
    if (tid == 0) s_row = atomicAdd(&A.sc->row_counter2, 1);
    __syncthreads();
    const int64_t row = s_row;
    __syncthreads();
    if (row >= A.T) break;
    const int64_t rrow = A.record_offset + row;
    uint4* oa = (uint4*)((char*)A.d_actor + row * A.ld * 2);
    uint4* op = (uint4*)((char*)A.d_policy + row * A.ld * 2);
    bool valid = (A.mask == nullptr || A.mask[row] != 0) && A.rec.flag[rrow] != 0 && g_over_n != 0.f;
    const int64_t x = A.tokens[row];
    if (!valid) {
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      for (int64_t i = tid; i < nvec8; i += GNT) { stg_stream(oa + i, z); stg_stream(op + i, z); }
      if (tid < tail) {
        ((uint16_t*)(oa + nvec8))[tid] = 0;
        ((uint16_t*)(op + nvec8))[tid] = 0;
      }
      continue;
    }
    const float adv = A.adv ? A.adv[row] : 1.f;
    const float ca = -g_over_n * adv;
    const float cp = (A.accept[row] != 0) ? -g_over_n * A.weight[row] * adv : 0.f;
    const float kq = cd - ca;
    const float kp_actor = -cd;
    const float lsa = A.rec.lse_a[rrow] * kLog2e;
    const float lsp = A.rec.lse_p[rrow] * kLog2e;
    const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
    const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;

    for (int64_t i0 = 0; i0 < nvec8; i0 += (int64_t)GNT * GUNROLL) {
      uint4 va[GUNROLL], vp[GUNROLL];
#pragma unroll
      for (int j = 0; j < GUNROLL; ++j) {
        int64_t i = i0 + (int64_t)j * GNT + tid;
        if (i < nvec8) {
          if (DT == JP_BF16) {
            va[j] = ld_plain((const uint4*)ra + i);
            vp[j] = ld_plain((const uint4*)rp + i);
          } else {
            // 8 fp32 logits -> packed as exact-widened halves is not possible; convert per element
            const float4 a0 = ((const float4*)ra)[2 * i], a1 = ((const float4*)ra)[2 * i + 1];
            const float4 p0 = ((const float4*)rp)[2 * i], p1 = ((const float4*)rp)[2 * i + 1];
            float qa[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            float qp[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
            float ga[8], gp[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float q = ex2_approx(fmaf(qa[e], kLog2e, -lsa));
              float p = ex2_approx(fmaf(qp[e], kLog2e, -lsp));
              float hot = (i * 8 + e == x) ? 1.f : 0.f;
              ga[e] = fmaf(kq, q, fmaf(kp_actor, p, ca * hot));
              gp[e] = cp * (hot - p);
            }
            stg_stream(oa + i, make_uint4(pack_bf16x2(ga[0], ga[1]), pack_bf16x2(ga[2], ga[3]),
                                          pack_bf16x2(ga[4], ga[5]), pack_bf16x2(ga[6], ga[7])));
            stg_stream(op + i, make_uint4(pack_bf16x2(gp[0], gp[1]), pack_bf16x2(gp[2], gp[3]),
                                          pack_bf16x2(gp[4], gp[5]), pack_bf16x2(gp[6], gp[7])));
          }
        }
      }
      if (DT == JP_BF16) {
#pragma unroll
        for (int j = 0; j < GUNROLL; ++j) {
          int64_t i = i0 + (int64_t)j * GNT + tid;
          if (i < nvec8) {
            uint4 ga, gp;
            grad8(va[j], vp[j], lsa, lsp, kq, kp_actor, ca, cp, i * 8, x, ga, gp);
            stg_stream(oa + i, ga);
            stg_stream(op + i, gp);
          }
        }
      }
    }
    if (tid < tail) {                        // ragged end of the row
      const int64_t c = nvec8 * 8 + tid;
      float q = ex2_approx(fmaf(Vec<DT>::load_scalar(ra, c), kLog2e, -lsa));
      float p = ex2_approx(fmaf(Vec<DT>::load_scalar(rp, c), kLog2e, -lsp));
      float hot = (c == x) ? 1.f : 0.f;
      float ga = fmaf(kq, q, fmaf(kp_actor, p, ca * hot));
      float gp = cp * (hot - p);
      ((__nv_bfloat16*)A.d_actor)[row * A.ld + c] = __float2bfloat16_rn(ga);
      ((__nv_bfloat16*)A.d_policy)[row * A.ld + c] = __float2bfloat16_rn(gp);
    }
  }
}

cudaError_t launch_grad(const GradArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0) return cudaSuccess;
  int g = sms * GCTAS_PER_SM;
  if (a.T < g) g = (int)a.T;
  if (a.dtype == JP_BF16) grad_kernel<JP_BF16><<<g, GNT, 0, s>>>(a);
  else grad_kernel<JP_F32><<<g, GNT, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace jp
