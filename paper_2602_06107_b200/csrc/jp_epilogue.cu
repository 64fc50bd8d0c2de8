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
  sc->n_nonfinite = 0ull;
  sc->lambda = lambda_fixed;
  sc->lambda64 = (double)lambda_fixed;
}

__global__ void clear_flags_kernel(uint8_t* flag, int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) flag[i] = 0;
}

// d_t = lp - lq in fp32 and r_t = exp(d_t) in double for every valid record row.
__global__ void ratio_kernel(int64_t T, Records rec) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T) return;
  if (rec.flag[i]) {
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
    if (rec.flag[i]) { c += 1; mn = fmin(mn, rec.ratio[i]); }
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
        if (rec.flag[i]) s += rec.ratio[i];
      s_hi = block_count_sum(0, s, s_c, s_s).s;   // at +inf: nothing >= x, every r below
    }
    while (hi - lo > 1u) {
      uint32_t mid = lo + ((hi - lo) >> 1);
      float x = order_bits_f32(mid);
      long long cg = 0;
      double sl = 0.0;
      for (int64_t i = tid; i < T; i += SOLVE_NT) {
        if (rec.flag[i]) {
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
  __shared__ long long s_nv[EPI_WARPS], s_na[EPI_WARPS];
  __shared__ double s_zk[EPI_WARPS], s_a[EPI_WARPS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = A.k;
  const float lambda = A.sc->lambda;
  const float log_lambda = logf(lambda);
  const int64_t per = (A.T + A.n_part - 1) / A.n_part;
  const int64_t r0 = (int64_t)blockIdx.x * per;
  const int64_t r1 = min(r0 + per, A.T);
  long long nv = 0, na = 0;
  double szk = 0.0, sa = 0.0;
  for (int64_t r = r0 + warp; r < r1; r += EPI_WARPS) {
    const bool valid = A.rec.flag[r] != 0;
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
        // Z_approx = sum over top-k(p_inf) U top-k(p_target) of min(q, p / lambda)
        const float ca = A.rec.lse_a[r], cp = A.rec.lse_p[r];
        const int64_t base = r * (2 * k);
        for (int j = lane; j < k; j += 32) s_idx[warp][j] = A.rec.idx[base + j];
        __syncwarp();
        float part = 0.f;
        for (int j = lane; j < 2 * k; j += 32) {
          const int32_t idx = A.rec.idx[base + j];
          bool use = idx >= 0;
          if (use && j >= k) {                 // policy-list entry: skip if the actor list has it
            for (int i = 0; i < k; ++i) use &= (s_idx[warp][i] != idx);
          }
          if (use) {
            float q = expf(A.rec.za[base + j] - ca);
            float p = expf(A.rec.zp[base + j] - cp - log_lambda);
            part += fminf(q, p);
          }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        zk = part;
        __syncwarp();
      } else {
        zk = A.rec.zk[r];
      }
    }
    if (lane == 0) {
      A.rec.a[r] = a;
      if (k > 0) A.rec.zk[r] = zk;
      if (A.out_accept) A.out_accept[r] = acc;
      if (A.out_lq) A.out_lq[r] = valid ? A.rec.lq[r] : 0.f;
      if (A.out_lp) A.out_lp[r] = valid ? A.rec.lp[r] : 0.f;
      if (A.aux_a) A.aux_a[r] = a;
      if (A.aux_u) A.aux_u[r] = u;
      if (A.aux_zk) A.aux_zk[r] = zk;
      if (A.aux_zx) A.aux_zx[r] = valid ? A.rec.zx[r] : 0.f;
      if (A.aux_lse_a) A.aux_lse_a[r] = valid ? A.rec.lse_a[r] : 0.f;
      if (A.aux_lse_p) A.aux_lse_p[r] = valid ? A.rec.lse_p[r] : 0.f;
      if (valid) { nv += 1; na += acc; szk += (double)zk; sa += (double)a; }
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
  if (lane == 0) { s_nv[warp] = nv; s_na[warp] = na; s_zk[warp] = szk; s_a[warp] = sa; }
  __syncthreads();
  if (tid == 0) {
    long long tnv = 0, tna = 0;
    double tzk = 0.0, ta = 0.0;
    for (int w = 0; w < EPI_WARPS; ++w) { tnv += s_nv[w]; tna += s_na[w]; tzk += s_zk[w]; ta += s_a[w]; }
    A.part->n_valid[blockIdx.x] = tnv;
    A.part->n_accept[blockIdx.x] = tna;
    A.part->sum_zk[blockIdx.x] = tzk;
    A.part->sum_a[blockIdx.x] = ta;
  }
}

// kappa = alpha_hat / mean Z_approx; w_t = min(kappa Z_approx(t) max(lambda, p/q), c1).
// Every block folds the same partial sums in the same order, then writes its rows.
__global__ void __launch_bounds__(EPI_NT) finalize_kernel(EpilogueArgs A) {
  __shared__ double s_kappa;
  __shared__ long long s_nv[EPI_NT], s_na[EPI_NT];
  __shared__ double s_zk[EPI_NT], s_a[EPI_NT];
  static_assert(kMaxPartials <= EPI_NT, "one thread per partial sum");
  // every block folds the same partial sums in the same fixed tree (so all blocks get
  // the same bits): thread i starts from partial i, halves are added pairwise
  {
    const int i = threadIdx.x;
    const bool have = i < A.n_part;
    s_nv[i] = have ? A.part->n_valid[i] : 0;
    s_na[i] = have ? A.part->n_accept[i] : 0;
    s_zk[i] = have ? A.part->sum_zk[i] : 0.0;
    s_a[i] = have ? A.part->sum_a[i] : 0.0;
  }
  __syncthreads();
  for (int half = EPI_NT / 2; half > 0; half >>= 1) {
    if ((int)threadIdx.x < half) {
      s_nv[threadIdx.x] += s_nv[threadIdx.x + half];
      s_na[threadIdx.x] += s_na[threadIdx.x + half];
      s_zk[threadIdx.x] += s_zk[threadIdx.x + half];
      s_a[threadIdx.x] += s_a[threadIdx.x + half];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const long long nv = s_nv[0], na = s_na[0];
    const double szk = s_zk[0], sa = s_a[0];
    double alpha = nv > 0 ? (double)na / (double)nv : 0.0;
    double mean_zk = nv > 0 ? szk / (double)nv : 0.0;
    double kappa = (nv > 0 && mean_zk > 0.0) ? alpha / mean_zk : 1.0;
    s_kappa = kappa;
    if (blockIdx.x == 0) {
      jp_stats st;
      st.n_valid = nv; st.n_accept = na;
      st.n_bad_token = (int64_t)A.sc->n_bad_token;
      st.n_nonfinite = (int64_t)A.sc->n_nonfinite;
      st.alpha_hat = alpha;
      st.mean_accept_prob = nv > 0 ? sa / (double)nv : 0.0;
      st.z_approx_mean = mean_zk;
      st.kappa = kappa;
      st.lambda_used = (double)A.sc->lambda;
      st.reserved = 0.0;
      st.status = A.sc->status;
      st.pad = 0;
      A.sc->stats = st;
      if (A.out_stats) *A.out_stats = st;
    }
  }
  __syncthreads();
  const double kappa = s_kappa;
  const float lambda = A.sc->lambda;
  int64_t r = (int64_t)blockIdx.x * EPI_NT + threadIdx.x;
  if (r >= A.T) return;
  float w = 0.f;
  if (A.rec.flag[r]) {
    float d = A.rec.lp[r] - A.rec.lq[r];
    double wt = kappa * (double)A.rec.zk[r] * fmax((double)lambda, exp((double)d));
    if (A.c1 > 0.f) wt = fmin(wt, (double)A.c1);
    w = (float)wt;
  }
  if (A.out_weight) A.out_weight[r] = w;
}

// The weights again, with a calibration factor the caller supplies: a batch that
// is spread over several devices sums (N, accepted, sum of Z_approx) over all of
// them (Section 4.4.2: kappa is batch-wide) and hands the resulting kappa back.
// The log-probs of the sampled tokens as the records hold them so far (0 for rows
// that are masked, bad or not streamed yet), plus the validity flags.
__global__ void __launch_bounds__(EPI_NT) logprobs_kernel(int64_t T, Records rec, float* out_lq, float* out_lp,
                                                          uint8_t* out_valid) {
  const int64_t i = (int64_t)blockIdx.x * EPI_NT + threadIdx.x;
  if (i >= T) return;
  const bool v = rec.flag[i] != 0;
  if (out_lq) out_lq[i] = v ? rec.lq[i] : 0.f;
  if (out_lp) out_lp[i] = v ? rec.lp[i] : 0.f;
  if (out_valid) out_valid[i] = v ? 1 : 0;
}

__global__ void __launch_bounds__(EPI_NT) reweight_kernel(int64_t T, Records rec, const Scalars* sc, double kappa,
                                                          float c1, float* out_weight) {
  const int64_t r = (int64_t)blockIdx.x * EPI_NT + threadIdx.x;
  if (r >= T) return;
  const float lambda = sc->lambda;
  float w = 0.f;
  if (rec.flag[r]) {
    float d = rec.lp[r] - rec.lq[r];
    double wt = kappa * (double)rec.zk[r] * fmax((double)lambda, exp((double)d));
    if (c1 > 0.f) wt = fmin(wt, (double)c1);
    w = (float)wt;
  }
  out_weight[r] = w;
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
