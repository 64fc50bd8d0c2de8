// Theorem 3.4 per distribution: for every row, the lambda at which the OBRS rule
// a_v = min(1, p_v / (lambda q_v)) accepts exactly a given budget,
//   Z(lambda) = sum_v min(q_v, p_v / lambda) = budget,
// with q, p the softmax of the actor and policy rows, and the divergences
// KL(p || q) and KL(p || q~), q~ = min(q, p / lambda) / Z (Theorem 3.3, Figure 2b).
//
// In u = 1 / lambda, Z(u) = sum_v min(q_v, u p_v) is concave, piecewise linear and
// increasing, with slope S(u) = sum of the p_v still below their cap.  Newton's
// iteration u <- u + (budget - Z(u)) / S(u) started at u = budget (where Z <= budget,
// because Z(u) <= u) climbs monotonically and ends after finitely many steps, when the
// set of capped entries stops changing.  Every step is one pass over the row pair,
// which stays in L2 between passes (one CTA works on one row at a time).  The iteration
// runs in w = u Sa / Sp on the unnormalised terms (see the kernel).
#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {
namespace {

constexpr int RNT = 512;
constexpr int RNW = RNT / 32;
constexpr int kMaxNewton = 48;

struct Red2 { double a, b; };

// Sum of two per-thread values over the CTA in a fixed order; every thread gets the result.
__device__ __forceinline__ Red2 block_sum2(float x, float y, double (*sh)[RNW]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double a = (double)x, b = (double)y;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, off);
    b += __shfl_xor_sync(0xffffffffu, b, off);
  }
  __syncthreads();                       // the previous result has been read by everyone
  if (lane == 0) { sh[0][warp] = a; sh[1][warp] = b; }
  __syncthreads();
  Red2 r{0.0, 0.0};
  for (int w = 0; w < RNW; ++w) { r.a += sh[0][w]; r.b += sh[1][w]; }
  return r;
}
__device__ __forceinline__ Red2 block_max2(float x, float y, double (*sh)[RNW]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, off));
    y = fmaxf(y, __shfl_xor_sync(0xffffffffu, y, off));
  }
  __syncthreads();
  if (lane == 0) { sh[0][warp] = (double)x; sh[1][warp] = (double)y; }
  __syncthreads();
  Red2 r{sh[0][0], sh[1][0]};
  for (int w = 1; w < RNW; ++w) { r.a = fmax(r.a, sh[0][w]); r.b = fmax(r.b, sh[1][w]); }
  return r;
}

// Applies f(za, zp) to every column of the row pair: 16-byte vectors, then the ragged end.
template <int DT, class F>
__device__ __forceinline__ void for_each_pair(const char* ra, const char* rp, int64_t V, F f) {
  constexpr int N = Vec<DT>::N;
  const int64_t nvec = V / N;
  for (int64_t i = threadIdx.x; i < nvec; i += RNT) {
    const uint4 va = ldg_stream((const uint4*)ra + i), vp = ldg_stream((const uint4*)rp + i);
#pragma unroll
    for (int e = 0; e < N; ++e) f(Vec<DT>::get(va, e), Vec<DT>::get(vp, e));
  }
  const int64_t c = nvec * N + threadIdx.x;
  if (c < V) f(Vec<DT>::load_scalar(ra, c), Vec<DT>::load_scalar(rp, c));
}

// Sum of two per-thread doubles over the CTA in a fixed order.
__device__ __forceinline__ Red2 block_sum2d(double a, double b, double (*sh)[RNW]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, off);
    b += __shfl_xor_sync(0xffffffffu, b, off);
  }
  __syncthreads();
  if (lane == 0) { sh[0][warp] = a; sh[1][warp] = b; }
  __syncthreads();
  Red2 r{0.0, 0.0};
  for (int w = 0; w < RNW; ++w) { r.a += sh[0][w]; r.b += sh[1][w]; }
  return r;
}

// Precision.  The root of Z(u) = budget is ill-conditioned when most of the accepted mass
// sits on capped entries: du/u = (dZ/Z) Z / (u P), P the mass still below its cap, and
// Z / (u P) reaches 20 to 50 at budgets near 1.  Three things therefore run at full
// precision: (1) the two normalisers (exp2f, double sums), whose error is common to every
// term; (2) the exponents, taken relative to integers Ma, Mp so that z log2(e) - M is one
// rounding, and the iteration runs on the unnormalised terms with the normalisers folded into
// the budget and into u in double; (3) the last step: once the
// capped set no longer changes, C = sum of capped q and P = sum of uncapped p are summed
// again with exp2f in double and u = (budget - C) / P in closed form.  The Newton passes
// before that only have to find the set; they run on ex2.approx and fp32 sums.
template <int DT>
__global__ void __launch_bounds__(RNT) row_lambda_kernel(RowLambdaArgs A) {
  __shared__ double sh[2][RNW];
  __shared__ int s_row;
  const int tid = threadIdx.x;
  const double b = (double)A.budget;
  for (;;) {
    if (tid == 0) s_row = atomicAdd(&A.sc->row_counter2, 1);
    __syncthreads();
    const int64_t row = s_row;
    __syncthreads();
    if (row >= A.T) break;
    if (A.mask && A.mask[row] == 0) {
      if (tid == 0) {
        A.out_lambda[row] = 0.f;
        if (A.out_kl_before) A.out_kl_before[row] = 0.f;
        if (A.out_kl_after) A.out_kl_after[row] = 0.f;
        if (A.out_iters) A.out_iters[row] = 0;
      }
      continue;
    }
    const char* ra = (const char*)A.za + row * A.ld * Vec<DT>::ESIZE;
    const char* rp = (const char*)A.zp + row * A.ld * Vec<DT>::ESIZE;
    // log-sum-exps: maxima, then sums relative to integer exponents above them (the row is
    // in L2 from here on)
    float ma = JP_NEG_INF, mp = JP_NEG_INF;
    for_each_pair<DT>(ra, rp, A.V, [&](float za, float zp) { ma = fmaxf(ma, za); mp = fmaxf(mp, zp); });
    const Red2 mx = block_max2(ma, mp, sh);
    const float Ma = ceilf((float)mx.a * kLog2e), Mp = ceilf((float)mx.b * kLog2e);
    double sa = 0.0, sp = 0.0;
    for_each_pair<DT>(ra, rp, A.V, [&](float za, float zp) {
      sa += (double)exp2f(fmaf(za, kLog2e, -Ma));
      sp += (double)exp2f(fmaf(zp, kLog2e, -Mp));
    });
    const Red2 ss = block_sum2d(sa, sp, sh);
    // With qh = 2^(za kLog2e - Ma), ph likewise: q = qh / Sa and p = ph / Sp up to the shortfall of
    // the fp32 constant, z (log2 e - kLog2e) in the exponent, which is the same for numerator and
    // sum where it matters (at the entries that carry the mass) and is dropped.  In w = u Sa / Sp:
    //   Z(u) = sum min(q, u p) = (1 / Sa) sum min(qh, w ph) = budget  <=>  sum min(qh, w ph) = budget Sa
    const double Sa = ss.a, Sp = ss.b;
    const double target = b * Sa;

    double w;
    int iters = 0;
    if (b >= 1.0) {
      // everything accepted in full: the largest such lambda is the smallest ratio p/q
      float dmin = __int_as_float(0x7f800000);
      for_each_pair<DT>(ra, rp, A.V, [&](float za, float zp) {
        dmin = fminf(dmin, fmaf(zp, kLog2e, -Mp) - fmaf(za, kLog2e, -Ma));
      });
      const Red2 r = block_max2(-dmin, 0.f, sh);
      w = exp2(r.a);                                   // 1 / min (ph / qh)
    } else {
      w = b * Sa / Sp;                                 // u = budget, where Z(u) <= u
      bool settled = false;
      for (; iters < kMaxNewton && !settled; ++iters) {
        const float wf = (float)w;
        float z = 0.f, s = 0.f;
        for_each_pair<DT>(ra, rp, A.V, [&](float za, float zp) {
          const float q = ex2_approx(fmaf(za, kLog2e, -Ma));
          const float up = wf * ex2_approx(fmaf(zp, kLog2e, -Mp));
          const bool below = up < q;
          z += below ? up : q;
          s += below ? up : 0.f;                       // w * (slope's share): divided by w below
        });
        const Red2 r = block_sum2(z, s, sh);
        const double gap = target - r.a;
        if (!(r.b > 0.0)) break;                       // nothing left below its cap
        const double wn = w + gap / (r.b / w);
        settled = gap <= 1e-5 * target || (float)wn == wf;
        if (wn > w) w = wn;
      }
      // the last step at full precision on the set that w selects; repeated while the set still moves
      for (int rep = 0; rep < 4; ++rep) {
        const float wf = (float)w;
        double C = 0.0, P = 0.0;
        for_each_pair<DT>(ra, rp, A.V, [&](float za, float zp) {
          const float q = exp2f(fmaf(za, kLog2e, -Ma));
          const float ph = exp2f(fmaf(zp, kLog2e, -Mp));
          if (wf * ph < q) P += (double)ph; else C += (double)q;
        });
        const Red2 r = block_sum2d(C, P, sh);
        if (!(r.b > 0.0)) break;
        const double wn = (target - r.a) / r.b;
        const bool same = fabs(wn - w) <= 1e-7 * w;
        if (wn > 0.0) w = wn;
        if (same) break;
      }
    }
    const double u = w * Sp / Sa;
    float kb = 0.f, ka = 0.f, zf = 0.f;
    if (A.out_kl_before || A.out_kl_after) {
      const float la2 = Ma + (float)log2(Sa), lp2 = Mp + (float)log2(Sp);
      const float lnu = (float)log(u);
      const float uf = (float)u;
      for_each_pair<DT>(ra, rp, A.V, [&](float za, float zp) {
        const float lq2 = fmaf(za, kLog2e, -la2), lpp2 = fmaf(zp, kLog2e, -lp2);
        const float p = ex2_approx(lpp2), q = ex2_approx(lq2);
        zf += fminf(q, uf * p);
        if (p > 0.f) {
          const float lq = lq2 * kLn2, lp = lpp2 * kLn2;
          kb = fmaf(p, lp - lq, kb);
          ka = fmaf(p, lp - fminf(lq, lp + lnu), ka);
        }
      });
    }
    const Red2 kk = block_sum2(kb, ka, sh);
    const Red2 zz = block_sum2(zf, 0.f, sh);
    if (tid == 0) {
      A.out_lambda[row] = (float)(1.0 / u);
      if (A.out_kl_before) A.out_kl_before[row] = (float)kk.a;
      if (A.out_kl_after) A.out_kl_after[row] = (float)(kk.b + log(zz.a));
      if (A.out_iters) A.out_iters[row] = iters;
    }
  }
}

}  // namespace

cudaError_t launch_row_lambda(const RowLambdaArgs& a, cudaStream_t s, int sms) {
  if (a.T <= 0) return cudaSuccess;
  int g = sms * 2;
  if (a.T < g) g = (int)a.T;
  if (a.dtype == JP_BF16) row_lambda_kernel<JP_BF16><<<g, RNT, 0, s>>>(a);
  else row_lambda_kernel<JP_F32><<<g, RNT, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace jp
