// Fused gradient of the joint objective (Eq. sys_joint_obj) with respect to
// both logit tensors.  With the loss to minimise
//   J = -L^{PPO-OBRS}(theta) - L^{PPO}(omega) + lambda_distill L^{distill}(omega)
// taken as a mean over the N valid proposed tokens and evaluated where the PPO
// ratios and F are 1 (Eq. obrs_ppo, Eq. ppo_rollout, Eq. distill_loss):
//   d_policy[t,v] = cp (1[v=x_t] - p_t(v)),              cp = -(g/N) Mask_t w_t A_t
//   d_actor[t,v]  = ca (1[v=x_t] - q_t(v)) + cd (q_t(v) - p_t(v)),
//                                       ca = -(g/N) A_t,  cd = g lambda_distill / N
// Away from the first update (Algorithm 1 steps 1, 3, 4; Eq. ppo_rollout) the two
// PPO coefficients take their general form, from per-token scalars only:
//   cp = -(g/N) Mask_t rho_t s_theta r_theta,   ca = -(g/N) F_t s_omega r_omega,
// where s is A_t on the live branch of min(r A, clip(r) A) and 0 on the clipped one.
// One pass: both rows are read once, both bf16 gradient rows are written once with
// 16-byte stores.  Masked rows are zero-filled without being read.  On request the
// same pass leaves the per-token objective terms and KL(p || q) of every row.
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
template <bool KL>
__device__ __forceinline__ void grad8(const uint4& va, const uint4& vp, float lsa, float lsp,
                                      float kq, float kp_actor, float ca, float cp, int64_t c0,
                                      int64_t x, uint4& oa, uint4& op, float& kl) {
  float ga[8], gp[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float za = Vec<JP_BF16>::get(va, e), zp = Vec<JP_BF16>::get(vp, e);
    float q = ex2_approx(fmaf(za, kLog2e, -lsa));
    float p = ex2_approx(fmaf(zp, kLog2e, -lsp));
    if (KL && p > 0.f) kl = fmaf(p, zp - za, kl);       // sum_v p (zp - za); the lse terms are added per row
    float hot = (c0 + e == x) ? 1.f : 0.f;
    ga[e] = fmaf(kq, q, fmaf(kp_actor, p, ca * hot));   // (cd - ca) q - cd p + ca 1[v=x]
    gp[e] = cp * (hot - p);
  }
  oa = make_uint4(pack_bf16x2(ga[0], ga[1]), pack_bf16x2(ga[2], ga[3]), pack_bf16x2(ga[4], ga[5]),
                  pack_bf16x2(ga[6], ga[7]));
  op = make_uint4(pack_bf16x2(gp[0], gp[1]), pack_bf16x2(gp[2], gp[3]), pack_bf16x2(gp[4], gp[5]),
                  pack_bf16x2(gp[6], gp[7]));
}

// min(r A, clip(r, 1 - eps_lo, 1 + eps_hi) A) and its slope in r (A on the live branch, 0 on the clipped one)
__device__ __forceinline__ double ppo_surrogate(double r, double adv, int clip, double eps_lo, double eps_hi,
                                                double* slope) {
  const double unclipped = r * adv;
  if (!clip) { *slope = adv; return unclipped; }
  const double rc = fmin(fmax(r, 1.0 - eps_lo), 1.0 + eps_hi);
  const double clipped = rc * adv;
  if (unclipped <= clipped) { *slope = adv; return unclipped; }
  *slope = 0.0;
  return clipped;
}

template <int DT, bool KL>
__global__ void __launch_bounds__(GNT, GCTAS_PER_SM) grad_kernel(GradArgs A) {
  __shared__ int s_row;
  __shared__ float s_kl[GNT / 32];
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
    bool valid = (A.mask == nullptr || A.mask[row] != 0) && A.rec.flag[rrow] == kRowValid && g_over_n != 0.f;
    const int64_t x = A.tokens[row];
    if (!valid) {
      if (tid == 0) {
        if (A.out_obj_policy) A.out_obj_policy[row] = 0.f;
        if (A.out_obj_actor) A.out_obj_actor[row] = 0.f;
        if (A.out_kl) A.out_kl[row] = 0.f;
      }
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      for (int64_t i = tid; i < nvec8; i += GNT) { stg_stream(oa + i, z); stg_stream(op + i, z); }
      if (tid < tail) {
        ((uint16_t*)(oa + nvec8))[tid] = 0;
        ((uint16_t*)(op + nvec8))[tid] = 0;
      }
      continue;
    }
    const float adv = A.adv ? A.adv[row] : 1.f;
    float ca = -g_over_n * adv;
    float cp = (A.accept[row] != 0) ? -g_over_n * A.weight[row] * adv : 0.f;
    if (A.logp_ref || A.logp_actor_ref || A.logp_inf || A.clip || A.c2 > 0.f || A.out_obj_policy || A.out_obj_actor) {
      // per-token scalars of the general form, in double: the branch of the min is a decision
      const double lq = (double)A.rec.lq[rrow], lp = (double)A.rec.lp[rrow];
      const double r_t = A.logp_ref ? exp(lp - (double)A.logp_ref[row]) : 1.0;
      double inv = 1.0 / r_t;
      if (A.c2 > 0.f) inv = fmin(inv, (double)A.c2);
      const double rho = (double)A.weight[row] * inv;
      double slope_t, slope_o;
      const double s_t = ppo_surrogate(r_t, (double)adv, A.clip, (double)A.eps_lo, (double)A.eps_hi, &slope_t);
      const double m = A.accept[row] != 0 ? 1.0 : 0.0;
      const double lq_ref = A.logp_actor_ref ? (double)A.logp_actor_ref[row] : lq;
      const double r_o = exp(lq - lq_ref);
      double F = 1.0;
      if (A.logp_inf) {
        F = exp(lq_ref - (double)A.logp_inf[row]);
        if (A.tis_cap > 0.f) F = fmin(F, (double)A.tis_cap);
      }
      const double s_o = ppo_surrogate(r_o, (double)adv, A.clip, (double)A.eps_lo, (double)A.eps_hi, &slope_o);
      // (a rejected token contributes nothing, whatever its ratios: p_new(a_t) = 0 makes rho infinite)
      cp = m != 0.0 ? (float)(-(double)g_over_n * rho * slope_t * r_t) : 0.f;
      ca = (float)(-(double)g_over_n * F * slope_o * r_o);
      if (tid == 0) {
        if (A.out_obj_policy) A.out_obj_policy[row] = m != 0.0 ? (float)(rho * s_t) : 0.f;
        if (A.out_obj_actor) A.out_obj_actor[row] = (float)(F * s_o);
      }
    }
    float kl = 0.f;
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
              if (KL && p > 0.f) kl = fmaf(p, qp[e] - qa[e], kl);
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
            grad8<KL>(va[j], vp[j], lsa, lsp, kq, kp_actor, ca, cp, i * 8, x, ga, gp, kl);
            stg_stream(oa + i, ga);
            stg_stream(op + i, gp);
          }
        }
      }
    }
    if (tid < tail) {                        // ragged end of the row
      const int64_t c = nvec8 * 8 + tid;
      const float za_c = Vec<DT>::load_scalar(ra, c), zp_c = Vec<DT>::load_scalar(rp, c);
      float q = ex2_approx(fmaf(za_c, kLog2e, -lsa));
      float p = ex2_approx(fmaf(zp_c, kLog2e, -lsp));
      if (KL && p > 0.f) kl = fmaf(p, zp_c - za_c, kl);
      float hot = (c == x) ? 1.f : 0.f;
      float ga = fmaf(kq, q, fmaf(kp_actor, p, ca * hot));
      float gp = cp * (hot - p);
      ((__nv_bfloat16*)A.d_actor)[row * A.ld + c] = __float2bfloat16_rn(ga);
      ((__nv_bfloat16*)A.d_policy)[row * A.ld + c] = __float2bfloat16_rn(gp);
    }
    if (KL) {
      // KL(p || q) = sum_v p (zp - za) - lse_p + lse_a, summed in a fixed order
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) kl += __shfl_xor_sync(0xffffffffu, kl, off);
      if ((tid & 31) == 0) s_kl[tid >> 5] = kl;
      __syncthreads();
      if (tid == 0) {
        double S = 0.0;
        for (int w = 0; w < GNT / 32; ++w) S += (double)s_kl[w];
        A.out_kl[row] = (float)(S - (double)A.rec.lse_p[rrow] + (double)A.rec.lse_a[rrow]);
      }
    }
  }
}

// J and its three parts over this call's rows: sums in a fixed order (a thread
// walks its rows in turn, then a tree over the block), divided by N.
__global__ void __launch_bounds__(1024) loss_kernel(GradArgs A) {
  __shared__ double sh[3][1024];
  const int tid = threadIdx.x;
  double a = 0.0, b = 0.0, c = 0.0;
  for (int64_t i = tid; i < A.T; i += 1024) {
    a += (double)A.out_obj_policy[i];
    b += (double)A.out_obj_actor[i];
    c += (double)A.out_kl[i];
  }
  sh[0][tid] = a; sh[1][tid] = b; sh[2][tid] = c;
  __syncthreads();
  for (int off = 512; off > 0; off >>= 1) {
    if (tid < off) {
      sh[0][tid] += sh[0][tid + off];
      sh[1][tid] += sh[1][tid + off];
      sh[2][tid] += sh[2][tid + off];
    }
    __syncthreads();
  }
  if (tid == 0) {
    const double Nd = (double)(A.n_valid > 0 ? A.n_valid : A.sc->stats.n_valid);
    const double inv = Nd > 0.0 ? 1.0 / Nd : 0.0;
    const double l1 = sh[0][0] * inv, l2 = sh[1][0] * inv, l3 = sh[2][0] * inv;
    A.out_loss[0] = -l1 - l2 + (double)A.lambda_distill * l3;
    A.out_loss[1] = l1;
    A.out_loss[2] = l2;
    A.out_loss[3] = l3;
  }
}

cudaError_t launch_grad(const GradArgs& a, cudaStream_t s, int sms, int* n_launch) {
  *n_launch = 0;
  if (a.T <= 0) return cudaSuccess;
  int g = sms * GCTAS_PER_SM;
  if (a.T < g) g = (int)a.T;
  const bool kl = a.out_kl != nullptr;
  if (a.dtype == JP_BF16) {
    if (kl) grad_kernel<JP_BF16, true><<<g, GNT, 0, s>>>(a);
    else grad_kernel<JP_BF16, false><<<g, GNT, 0, s>>>(a);
  } else {
    if (kl) grad_kernel<JP_F32, true><<<g, GNT, 0, s>>>(a);
    else grad_kernel<JP_F32, false><<<g, GNT, 0, s>>>(a);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  *n_launch = 1;
  if (a.out_loss) {
    loss_kernel<<<1, 1024, 0, s>>>(a);
    e = cudaGetLastError();
    if (e == cudaSuccess) *n_launch = 2;
  }
  return e;
}

}  // namespace jp
