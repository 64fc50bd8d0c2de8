// O(T) and O(T k) steps that follow the row stream: the batch-level lambda from
// an acceptance budget (Theorem 3.4 applied to the batch's sampled tokens), the
// acceptance probability and decision (Eq. obrs_accept; Algorithm 2's
// "U(0,1) < alpha"), Z_approx over the de-duplicated union of the two top-k
// lists (Section 4.4.1), the batch calibration factor kappa (Section 4.4.2) and
// the OBRS weights (Algorithm 1, step 3).  Every reduction is a fixed tree, so
// results do not change from run to run.
#include "jp_common.cuh"
#include "jp_internal.h"

namespace jp {

__global__ void reset_kernel(Scalars* sc, float lambda_fixed) {
  sc->n_list = 0;
  sc->row_counter2 = 0;
  sc->n_compact = 0;
  sc->status = 0;
  sc->n_bad_token = 0ull;
  sc->lambda = lambda_fixed;
  sc->lambda64 = (double)lambda_fixed;
}

__global__ void clear_flags_kernel(uint8_t* flag, int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) flag[i] = 0;
}

// A streamed row enters the ratios p/q only if its numbers allow it: log q(a_t) finite (a
// sampled token has positive probability under the model that sampled it), the policy's
// log-sum-exp finite, and log p(a_t) a number below +inf (-inf is fine: the target gives the
// token probability 0, the ratio is 0 and the token is rejected).  A NaN or +inf logit, or a
// sampled token of probability 0 under the rollout model, fails this: the row is marked so
// that every later step treats it as masked, and counted once.
__device__ __forceinline__ bool row_finite(const Records& rec, int64_t r) {
  const float lq = rec.lq[r], lp = rec.lp[r];
  // (the allocation-free budget solve has the log-probs only: no log-sum-exp array)
  const float lse_p = rec.lse_p ? rec.lse_p[r] : 0.f;
  return isfinite(lq) && isfinite(lse_p) && lp == lp && lp != __int_as_float(0x7f800000);
}

// d_t = lp - lq in fp32 and r_t = exp(d_t) in double for every valid record row.
__global__ void ratio_kernel(int64_t T, Records rec) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T) return;
  uint8_t f = rec.flag[i];
  if (f == kRowValid && !row_finite(rec, i)) { f = kRowNonFinite; rec.flag[i] = f; }
  if (f == kRowValid) {
    float d = rec.lp[i] - rec.lq[i];
    rec.dval[i] = d;
    rec.ratio[i] = exp((double)d);
  } else {
    rec.dval[i] = 0.f;
    rec.ratio[i] = 0.0;
  }
}

constexpr int SOLVE_NT = 1024;

struct CountSum {
  long long c;
  double s;
};

__device__ __forceinline__ CountSum block_count_sum(long long c, double s, long long* sc, double* ss) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    c += __shfl_xor_sync(0xffffffffu, c, off);
    s += __shfl_xor_sync(0xffffffffu, s, off);
  }
  __syncthreads();
  if (lane == 0) { sc[warp] = c; ss[warp] = s; }
  __syncthreads();
  CountSum r{0, 0.0};
  for (int w = 0; w < SOLVE_NT / 32; ++w) { r.c += sc[w]; r.s += ss[w]; }
  return r;
}

// Solves (1/N) sum_t min(1, r_t / lambda) = budget for lambda.
// g(lambda) = (1/N)[#{r >= lambda} + (1/lambda) sum_{r < lambda} r] is non-increasing.
// The d_t are fp32, so a binary search over the ordered fp32 bit patterns finds
// the two adjacent floats x_lo < x_hi with g(e^{x_lo}) >= budget > g(e^{x_hi});
// no d_t lies strictly between them, so the set {d_t < x_hi} is the partially
// accepted set and lambda = S / (N budget - #{d >= x_hi}) in closed form.
__global__ void __launch_bounds__(SOLVE_NT) budget_solve_kernel(int64_t T, Records rec, Scalars* sc,
                                                                double budget) {
  __shared__ long long s_c[SOLVE_NT / 32];
  __shared__ double s_s[SOLVE_NT / 32];
  const int tid = threadIdx.x;
  long long c = 0;
  double mn = 1e300;
  for (int64_t i = tid; i < T; i += SOLVE_NT)
    if (rec.flag[i] == kRowValid) { c += 1; mn = fmin(mn, rec.ratio[i]); }
  CountSum tot = block_count_sum(c, 0.0, s_c, s_s);
  const long long N = tot.c;
  double lam;
  if (N == 0) {
    lam = 1.0;
  } else if (budget >= 1.0) {
    // largest lambda with full acceptance: min_t r_t
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, off));
    __syncthreads();
    if ((tid & 31) == 0) s_s[tid >> 5] = mn;
    __syncthreads();
    lam = s_s[0];
    for (int w = 1; w < SOLVE_NT / 32; ++w) lam = fmin(lam, s_s[w]);
  } else {
    uint32_t lo = f32_order_bits(JP_NEG_INF);                 // g = 1 >= budget there
    uint32_t hi = f32_order_bits(__int_as_float(0x7f800000));  // g = 0 <  budget there
    long long c_hi = 0;
    double s_hi = 0.0;
    {
      double s = 0.0;
      for (int64_t i = tid; i < T; i += SOLVE_NT)
        if (rec.flag[i] == kRowValid) s += rec.ratio[i];
      s_hi = block_count_sum(0, s, s_c, s_s).s;   // at +inf: nothing >= x, every r below
    }
    while (hi - lo > 1u) {
      uint32_t mid = lo + ((hi - lo) >> 1);
      float x = order_bits_f32(mid);
      long long cg = 0;
      double sl = 0.0;
      for (int64_t i = tid; i < T; i += SOLVE_NT) {
        if (rec.flag[i] == kRowValid) {
          if (rec.dval[i] >= x) cg += 1;
          else sl += rec.ratio[i];
        }
      }
      CountSum r = block_count_sum(cg, sl, s_c, s_s);
      double lx = exp((double)x);
      double g = ((double)r.c + (r.s > 0.0 ? r.s / lx : 0.0)) / (double)N;
      if (g < budget) { hi = mid; c_hi = r.c; s_hi = r.s; }
      else lo = mid;
    }
    lam = s_hi / ((double)N * budget - (double)c_hi);
  }
  if (tid == 0) {
    sc->lambda64 = lam;
    sc->lambda = (float)lam;
  }
}

constexpr int EPI_NT = 256;
constexpr int EPI_WARPS = EPI_NT / 32;

// One warp per record row.  Each block owns a contiguous slice of rows and sums
// its slice in a fixed order.
__global__ void __launch_bounds__(EPI_NT) epilogue_kernel(EpilogueArgs A) {
  __shared__ int32_t s_idx[EPI_WARPS][JP_MAX_TOPK];
  __shared__ long long s_nv[EPI_WARPS], s_na[EPI_WARPS], s_nf[EPI_WARPS];
  __shared__ double s_zk[EPI_WARPS], s_a[EPI_WARPS], s_kl[EPI_WARPS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = A.k;
  const float lambda = A.sc->lambda;
  const float log_lambda = logf(lambda);
  const double log_lambda64 = log((double)lambda);
  const int64_t per = (A.T + A.n_part - 1) / A.n_part;
  const int64_t r0 = (int64_t)blockIdx.x * per;
  const int64_t r1 = min(r0 + per, A.T);
  long long nv = 0, na = 0, nf = 0;
  double szk = 0.0, sa = 0.0, skl = 0.0;
  for (int64_t r = r0 + warp; r < r1; r += EPI_WARPS) {
    uint8_t f = A.rec.flag[r];
    if (f == kRowValid && !row_finite(A.rec, r)) f = kRowNonFinite;
    const bool valid = f == kRowValid;
    const float u = accept_uniform(A.seed, (uint64_t)(A.rng_base + r));
    float a = 0.f, zk = 0.f;
    uint8_t acc = 0;
    if (valid) {
      const float lq = A.rec.lq[r], lp = A.rec.lp[r];
      const float d = lp - lq;
      const float e = d - log_lambda;
      a = fminf(1.0f, expf(e));
      acc = (u < a) ? 1 : 0;
      if (k > 0) {
        // Z_approx = sum over top-k(p_inf) U top-k(p_target) of min(q, p / lambda).  The exponents
        // are formed in double from the two-word log-sum-exps: one fp32 word alone would put a
        // common relative error of ulp(|lse|)/2 on every q and p of the row.
        const double ca = (double)A.rec.lse_a[r] + (double)A.rec.lse_a_lo[r];
        const double cp = (double)A.rec.lse_p[r] + (double)A.rec.lse_p_lo[r] + log_lambda64;
        const int64_t base = r * (2 * k);
        for (int j = lane; j < k; j += 32) s_idx[warp][j] = A.rec.idx[base + j];
        __syncwarp();
        double part = 0.0;
        for (int j = lane; j < 2 * k; j += 32) {
          const int32_t idx = A.rec.idx[base + j];
          bool use = idx >= 0;
          if (use && j >= k) {                 // policy-list entry: skip if the actor list has it
            for (int i = 0; i < k; ++i) use &= (s_idx[warp][i] != idx);
          }
          if (use) {
            const double q = exp((double)A.rec.za[base + j] - ca);
            const double p = exp((double)A.rec.zp[base + j] - cp);
            part += fmin(q, p);
          }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        zk = (float)part;
        __syncwarp();
      } else {
        zk = A.rec.zk[r];
      }
    }
    if (lane == 0) {
      if (f != A.rec.flag[r]) A.rec.flag[r] = f;
      A.rec.a[r] = a;
      A.rec.zk[r] = zk;
      if (A.out_accept) A.out_accept[r] = acc;
      if (A.out_lq) A.out_lq[r] = valid ? A.rec.lq[r] : 0.f;
      if (A.out_lp) A.out_lp[r] = valid ? A.rec.lp[r] : 0.f;
      if (A.aux_a) A.aux_a[r] = a;
      if (A.aux_u) A.aux_u[r] = u;
      if (A.aux_zk) A.aux_zk[r] = zk;
      if (A.aux_zx) A.aux_zx[r] = valid ? A.rec.zx[r] : 0.f;
      if (A.aux_lse_a) A.aux_lse_a[r] = valid ? A.rec.lse_a[r] : 0.f;
      if (A.aux_lse_p) A.aux_lse_p[r] = valid ? A.rec.lse_p[r] : 0.f;
      if (valid) {
        nv += 1; na += acc; szk += (double)zk; sa += (double)a;
        if (A.have_kl) skl += (double)A.rec.kl[r];
      }
      if (f == kRowNonFinite) nf += 1;
    }
    if (k > 0 && (A.aux_idx_a || A.aux_idx_p || A.aux_val_a || A.aux_val_p)) {
      const int64_t base = r * (2 * k);
      for (int j = lane; j < k; j += 32) {
        if (A.aux_idx_a) A.aux_idx_a[r * k + j] = valid ? A.rec.idx[base + j] : -1;
        if (A.aux_idx_p) A.aux_idx_p[r * k + j] = valid ? A.rec.idx[base + k + j] : -1;
        if (A.aux_val_a) A.aux_val_a[r * k + j] = valid ? A.rec.za[base + j] : 0.f;
        if (A.aux_val_p) A.aux_val_p[r * k + j] = valid ? A.rec.zp[base + k + j] : 0.f;
      }
    }
  }
  if (lane == 0) { s_nv[warp] = nv; s_na[warp] = na; s_nf[warp] = nf; s_zk[warp] = szk; s_a[warp] = sa; s_kl[warp] = skl; }
  __syncthreads();
  if (tid == 0) {
    long long tnv = 0, tna = 0, tnf = 0;
    double tzk = 0.0, ta = 0.0, tkl = 0.0;
    for (int w = 0; w < EPI_WARPS; ++w) {
      tnv += s_nv[w]; tna += s_na[w]; tnf += s_nf[w]; tzk += s_zk[w]; ta += s_a[w]; tkl += s_kl[w];
    }
    A.part->n_valid[blockIdx.x] = tnv;
    A.part->n_accept[blockIdx.x] = tna;
    A.part->n_nonfinite[blockIdx.x] = tnf;
    A.part->sum_zk[blockIdx.x] = tzk;
    A.part->sum_a[blockIdx.x] = ta;
    A.part->sum_kl[blockIdx.x] = tkl;
  }
}

// The calibration factor of Section 4.4.2 from the batch's three sums: the realised
// acceptance rate over the mean of Z_approx; 1 when there is no valid token or the mean is 0.
__device__ __forceinline__ double kappa_of(double n, double n_acc, double sum_zk) {
  if (!(n > 0.0) || !(sum_zk > 0.0)) return 1.0;
  return (n_acc / n) / (sum_zk / n);
}

// w_t = min(kappa Z_approx(t) max(lambda, p/q), c1) for a valid record row, 0 otherwise.
__device__ __forceinline__ float obrs_weight(const Records& rec, int64_t r, double kappa, float lambda, float c1) {
  if (rec.flag[r] != kRowValid) return 0.f;
  const float d = rec.lp[r] - rec.lq[r];
  double wt = kappa * (double)rec.zk[r] * fmax((double)lambda, exp((double)d));
  if (c1 > 0.f) wt = fmin(wt, (double)c1);
  return (float)wt;
}

// kappa = alpha_hat / mean Z_approx; w_t = min(kappa Z_approx(t) max(lambda, p/q), c1).
// Every block folds the same partial sums in the same order, then writes its rows.
__global__ void __launch_bounds__(EPI_NT) finalize_kernel(EpilogueArgs A) {
  __shared__ double s_kappa;
  __shared__ long long s_nv[EPI_NT], s_na[EPI_NT], s_nf[EPI_NT];
  __shared__ double s_zk[EPI_NT], s_a[EPI_NT], s_kl[EPI_NT];
  static_assert(kMaxPartials <= EPI_NT, "one thread per partial sum");
  // every block folds the same partial sums in the same fixed tree (so all blocks get
  // the same bits): thread i starts from partial i, halves are added pairwise
  {
    const int i = threadIdx.x;
    const bool have = i < A.n_part;
    s_nv[i] = have ? A.part->n_valid[i] : 0;
    s_na[i] = have ? A.part->n_accept[i] : 0;
    s_nf[i] = have ? A.part->n_nonfinite[i] : 0;
    s_zk[i] = have ? A.part->sum_zk[i] : 0.0;
    s_a[i] = have ? A.part->sum_a[i] : 0.0;
    s_kl[i] = have ? A.part->sum_kl[i] : 0.0;
  }
  __syncthreads();
  for (int half = EPI_NT / 2; half > 0; half >>= 1) {
    if ((int)threadIdx.x < half) {
      s_nv[threadIdx.x] += s_nv[threadIdx.x + half];
      s_na[threadIdx.x] += s_na[threadIdx.x + half];
      s_nf[threadIdx.x] += s_nf[threadIdx.x + half];
      s_zk[threadIdx.x] += s_zk[threadIdx.x + half];
      s_a[threadIdx.x] += s_a[threadIdx.x + half];
      s_kl[threadIdx.x] += s_kl[threadIdx.x + half];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const long long nv = s_nv[0], na = s_na[0];
    const double szk = s_zk[0], sa = s_a[0];
    const double kappa = kappa_of((double)nv, (double)na, szk);
    s_kappa = kappa;
    if (blockIdx.x == 0) {
      jp_stats st;
      st.n_valid = nv; st.n_accept = na;
      st.n_bad_token = (int64_t)A.sc->n_bad_token;
      st.n_nonfinite = s_nf[0];
      st.alpha_hat = nv > 0 ? (double)na / (double)nv : 0.0;
      st.mean_accept_prob = nv > 0 ? sa / (double)nv : 0.0;
      st.z_approx_mean = nv > 0 ? szk / (double)nv : 0.0;
      st.kappa = kappa;
      st.lambda_used = (double)A.sc->lambda;
      st.mean_kl_p_q = (A.have_kl && nv > 0) ? s_kl[0] / (double)nv : __longlong_as_double(0x7ff8000000000000ll);
      st.status = A.sc->status;
      st.pad = 0;
      A.sc->stats = st;
      A.sc->totals[0] = (double)nv; A.sc->totals[1] = (double)na; A.sc->totals[2] = szk; A.sc->totals[3] = sa;
      if (A.out_stats) *A.out_stats = st;
    }
  }
  __syncthreads();
  const int64_t r = (int64_t)blockIdx.x * EPI_NT + threadIdx.x;
  if (r >= A.T) return;
  if (A.out_weight) A.out_weight[r] = obrs_weight(A.rec, r, s_kappa, A.sc->lambda, A.c1);
}

// The log-probs of the sampled tokens as the records hold them so far (0 for rows
// that are masked, bad, non-finite or not streamed yet), plus the validity flags.
__global__ void __launch_bounds__(EPI_NT) logprobs_kernel(int64_t T, Records rec, float* out_lq, float* out_lp,
                                                          uint8_t* out_valid) {
  const int64_t i = (int64_t)blockIdx.x * EPI_NT + threadIdx.x;
  if (i >= T) return;
  const bool v = rec.flag[i] == kRowValid && row_finite(rec, i);
  if (out_lq) out_lq[i] = v ? rec.lq[i] : 0.f;
  if (out_lp) out_lp[i] = v ? rec.lp[i] : 0.f;
  if (out_valid) out_valid[i] = v ? 1 : 0;
}

// The weights again, with a calibration factor the caller supplies (Section 4.4.2: kappa
// is a batch-wide scalar).
__global__ void __launch_bounds__(EPI_NT) reweight_kernel(int64_t T, Records rec, const Scalars* sc, double kappa,
                                                          float c1, float* out_weight) {
  const int64_t r = (int64_t)blockIdx.x * EPI_NT + threadIdx.x;
  if (r >= T) return;
  out_weight[r] = obrs_weight(rec, r, kappa, sc->lambda, c1);
}

// The weights from batch sums the caller supplies in device memory (a batch spread over
// several devices: the shards' sums added up).  totals = (N, accepted, sum of Z_approx[,
// sum of a(x_t)]): kappa is formed here, by the same rule as on one device, and the
// batch-wide statistics are written beside the weights.
__global__ void __launch_bounds__(EPI_NT) reweight_totals_kernel(int64_t T, Records rec, Scalars* sc,
                                                                 const double* totals, float c1, float* out_weight,
                                                                 jp_stats* out_stats) {
  const double n = totals[0], n_acc = totals[1], szk = totals[2], sa = totals[3];
  const double kappa = kappa_of(n, n_acc, szk);
  if (blockIdx.x == 0 && threadIdx.x == 0 && out_stats) {
    jp_stats st = sc->stats;                 // counters of this shard; the batch-wide figures replace the shard's
    st.n_valid = (int64_t)n; st.n_accept = (int64_t)n_acc;
    st.alpha_hat = n > 0.0 ? n_acc / n : 0.0;
    st.mean_accept_prob = n > 0.0 ? sa / n : 0.0;
    st.z_approx_mean = n > 0.0 ? szk / n : 0.0;
    st.kappa = kappa;
    *out_stats = st;
  }
  const int64_t r = (int64_t)blockIdx.x * EPI_NT + threadIdx.x;
  if (r < T && out_weight) out_weight[r] = obrs_weight(rec, r, kappa, sc->lambda, c1);
}

cudaError_t launch_reweight_totals(int64_t T, const Records& rec, Scalars* sc, const double* totals, float c1,
                                   float* out_weight, jp_stats* out_stats, cudaStream_t s) {
  const unsigned blocks = (unsigned)((T + EPI_NT - 1) / EPI_NT);
  reweight_totals_kernel<<<blocks < 1 ? 1 : blocks, EPI_NT, 0, s>>>(T, rec, sc, totals, c1, out_weight, out_stats);
  return cudaGetLastError();
}

cudaError_t launch_reweight(int64_t T, const Records& rec, const Scalars* sc, double kappa, float c1,
                            float* out_weight, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  reweight_kernel<<<(unsigned)((T + EPI_NT - 1) / EPI_NT), EPI_NT, 0, s>>>(T, rec, sc, kappa, c1, out_weight);
  return cudaGetLastError();
}

cudaError_t launch_reset(Scalars* sc, float lambda_fixed, cudaStream_t s) {
  reset_kernel<<<1, 1, 0, s>>>(sc, lambda_fixed);
  return cudaGetLastError();
}

cudaError_t launch_clear_flags(uint8_t* flag, int64_t n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  clear_flags_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(flag, n);
  return cudaGetLastError();
}

cudaError_t launch_budget_solve(const EpilogueArgs& a, double budget, cudaStream_t s, int* n_launch) {
  if (a.T <= 0) return cudaSuccess;
  ratio_kernel<<<(unsigned)((a.T + 255) / 256), 256, 0, s>>>(a.T, a.rec);
  budget_solve_kernel<<<1, SOLVE_NT, 0, s>>>(a.T, a.rec, a.sc, budget);
  *n_launch += 2;
  return cudaGetLastError();
}

cudaError_t launch_epilogue(const EpilogueArgs& a, cudaStream_t s, int* n_launch) {
  epilogue_kernel<<<a.n_part, EPI_NT, 0, s>>>(a);
  unsigned blocks = (unsigned)((a.T + EPI_NT - 1) / EPI_NT);
  finalize_kernel<<<blocks < 1 ? 1 : blocks, EPI_NT, 0, s>>>(a);
  *n_launch += 2;
  return cudaGetLastError();
}

cudaError_t launch_logprobs(int64_t T, const Records& rec, float* out_lq, float* out_lp, uint8_t* out_valid,
                            cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  logprobs_kernel<<<(unsigned)((T + EPI_NT - 1) / EPI_NT), EPI_NT, 0, s>>>(T, rec, out_lq, out_lp, out_valid);
  return cudaGetLastError();
}

}  // namespace jp
