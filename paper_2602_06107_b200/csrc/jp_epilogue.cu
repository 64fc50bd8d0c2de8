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
  sc->bs_ticket = 0;
  sc->bs_done = 0;
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

// ---- lambda from an acceptance budget ------------------------------------------------------
// Solves (1/N) sum_t min(1, r_t / lambda) = budget for lambda.
// g(lambda) = (1/N)[#{r >= lambda} + (1/lambda) sum_{r < lambda} r] is non-increasing.
// The d_t = log r_t are fp32, so a search over the ordered fp32 bit patterns finds the two
// adjacent floats x_lo < x_hi with g(e^{x_lo}) >= budget > g(e^{x_hi}); no d_t lies strictly
// between them, so the set {d_t < x_hi} is the partially accepted set and
// lambda = S / (N budget - #{d >= x_hi}) in closed form.
// The search is 16-way: one launch evaluates g at 15 thresholds that split the current
// bracket evenly, so 32 bits take at most 9 launches (plus one that counts N, sums all
// ratios and finds the smallest).  Every launch spreads the rows over many blocks; each
// block leaves its partial counts and sums, and the block that finishes last (a ticket
// counter: no block ever waits) adds them up in block order and narrows the bracket.  The
// sums therefore do not depend on timing.
constexpr int BS_NT = 256;
constexpr int BS_PER_THREAD = 4;
constexpr int BS_ROUNDS = 10;

__device__ __forceinline__ void warp_sum_cs(long long& c, double& s) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    c += __shfl_xor_sync(0xffffffffu, c, off);
    s += __shfl_xor_sync(0xffffffffu, s, off);
  }
}

// True in exactly one block per launch: the one whose ticket is the last.  The partials
// written before the call are visible to that block afterwards.
__device__ __forceinline__ bool last_block_done(Scalars* sc, int* s_flag) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t t = atomicAdd(&sc->bs_ticket, 1u);
    *s_flag = (t == gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (*s_flag) __threadfence();
  return *s_flag != 0;
}

__global__ void __launch_bounds__(BS_NT) budget_init_kernel(int64_t T, Records rec, Scalars* sc, SolvePartials* part,
                                                            double budget) {
  __shared__ long long s_c[BS_NT / 32];
  __shared__ double s_s[BS_NT / 32], s_m[BS_NT / 32];
  __shared__ int s_flag;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  long long c = 0;
  double s = 0.0, mn = 1e300;
  for (int64_t i = (int64_t)blockIdx.x * BS_NT + tid; i < T; i += (int64_t)gridDim.x * BS_NT)
    if (rec.flag[i] == kRowValid) { c += 1; s += rec.ratio[i]; mn = fmin(mn, rec.ratio[i]); }
  warp_sum_cs(c, s);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, off));
  if (lane == 0) { s_c[warp] = c; s_s[warp] = s; s_m[warp] = mn; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < BS_NT / 32; ++w) { c += s_c[w]; s += s_s[w]; mn = fmin(mn, s_m[w]); }
    part->c[blockIdx.x][0] = c; part->s[blockIdx.x][0] = s; part->s[blockIdx.x][1] = mn;
  }
  if (!last_block_done(sc, &s_flag)) return;
  if (tid == 0) {
    long long N = 0;
    double S = 0.0, m = 1e300;
    for (unsigned b = 0; b < gridDim.x; ++b) { N += part->c[b][0]; S += part->s[b][0]; m = fmin(m, part->s[b][1]); }
    sc->bs_N = N;
    sc->bs_lo = f32_order_bits(JP_NEG_INF);                     // g = 1 >= budget there
    sc->bs_hi = f32_order_bits(__int_as_float(0x7f800000));      // g = 0 <  budget there
    sc->bs_c_hi = 0;                                             // at +inf: nothing >= x, every r below
    sc->bs_s_hi = S;
    sc->bs_done = 0;
    if (N == 0) { sc->lambda64 = 1.0; sc->lambda = 1.f; sc->bs_done = 1; }
    else if (budget >= 1.0) { sc->lambda64 = m; sc->lambda = (float)m; sc->bs_done = 1; }   // largest lambda with full acceptance
    sc->bs_ticket = 0;
  }
}

__global__ void __launch_bounds__(BS_NT) budget_round_kernel(int64_t T, Records rec, Scalars* sc, SolvePartials* part,
                                                             double budget) {
  __shared__ long long s_c[BS_NT / 32][kSolveWays];
  __shared__ double s_s[BS_NT / 32][kSolveWays];
  __shared__ int s_flag;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (sc->bs_done) return;                       // every block reads the state the previous launch left
  const uint32_t lo = sc->bs_lo, hi = sc->bs_hi;
  const uint32_t span = hi - lo;                 // >= 2 while not done
  const int nth = span - 1u < (uint32_t)(kSolveWays - 1) ? (int)(span - 1u) : kSolveWays - 1;
  const uint32_t step = span / (uint32_t)(nth + 1);
  // thresholds m_j = lo + j step, j = 1 .. nth, all strictly inside (lo, hi)
  long long cg[kSolveWays];
  double sl[kSolveWays];
#pragma unroll
  for (int j = 0; j < kSolveWays; ++j) { cg[j] = 0; sl[j] = 0.0; }
  for (int64_t i = (int64_t)blockIdx.x * BS_NT + tid; i < T; i += (int64_t)gridDim.x * BS_NT) {
    if (rec.flag[i] != kRowValid) continue;
    const uint32_t ob = f32_order_bits(rec.dval[i]);
    const double r = rec.ratio[i];
#pragma unroll
    for (int j = 1; j < kSolveWays; ++j) {
      if (j <= nth) {
        if (ob >= lo + (uint32_t)j * step) cg[j] += 1;
        else sl[j] += r;
      }
    }
  }
#pragma unroll
  for (int j = 1; j < kSolveWays; ++j) {
    warp_sum_cs(cg[j], sl[j]);
    if (lane == 0) { s_c[warp][j] = cg[j]; s_s[warp][j] = sl[j]; }
  }
  __syncthreads();
  if (tid >= 1 && tid < kSolveWays) {
    long long c = 0;
    double s = 0.0;
    for (int w = 0; w < BS_NT / 32; ++w) { c += s_c[w][tid]; s += s_s[w][tid]; }
    part->c[blockIdx.x][tid] = c;
    part->s[blockIdx.x][tid] = s;
  }
  if (!last_block_done(sc, &s_flag)) return;
  if (tid >= 1 && tid < kSolveWays) {
    long long c = 0;
    double s = 0.0;
    for (unsigned b = 0; b < gridDim.x; ++b) { c += part->c[b][tid]; s += part->s[b][tid]; }
    s_c[0][tid] = c; s_s[0][tid] = s;
  }
  __syncthreads();
  if (tid == 0) {
    const double N = (double)sc->bs_N;
    uint32_t nlo = lo, nhi = hi;
    long long c_hi = sc->bs_c_hi;
    double s_hi = sc->bs_s_hi;
    for (int j = 1; j <= nth; ++j) {              // g falls along the thresholds: the first one below the budget is the new hi
      const uint32_t m = lo + (uint32_t)j * step;
      const double lx = exp((double)order_bits_f32(m));
      const double g = ((double)s_c[0][j] + (s_s[0][j] > 0.0 ? s_s[0][j] / lx : 0.0)) / N;
      if (g < budget) { nhi = m; c_hi = s_c[0][j]; s_hi = s_s[0][j]; break; }
      nlo = m;
    }
    sc->bs_lo = nlo; sc->bs_hi = nhi; sc->bs_c_hi = c_hi; sc->bs_s_hi = s_hi;
    if (nhi - nlo <= 1u) {
      const double lam = s_hi / (N * budget - (double)c_hi);
      sc->lambda64 = lam;
      sc->lambda = (float)lam;
      sc->bs_done = 1;
    }
    sc->bs_ticket = 0;
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
  // launched as a programmatic dependent of the kernel before it (the row stream, or the last
  // step of the budget solve): nothing is read before that kernel has finished
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
  static_assert(kMaxPartials % EPI_NT == 0, "every thread starts from the same number of partial sums");
  asm volatile("griddepcontrol.wait;" ::: "memory");          // a programmatic dependent of epilogue_kernel
  // every block folds the same partial sums in the same fixed order (so all blocks get the
  // same bits): thread i adds up partials i, i + EPI_NT, ... in turn, then halves are added pairwise
  {
    const int i = threadIdx.x;
    long long nv = 0, na = 0, nf = 0;
    double zk = 0.0, a = 0.0, kl = 0.0;
    for (int j = i; j < A.n_part; j += EPI_NT) {
      nv += A.part->n_valid[j]; na += A.part->n_accept[j]; nf += A.part->n_nonfinite[j];
      zk += A.part->sum_zk[j]; a += A.part->sum_a[j]; kl += A.part->sum_kl[j];
    }
    s_nv[i] = nv; s_na[i] = na; s_nf[i] = nf; s_zk[i] = zk; s_a[i] = a; s_kl[i] = kl;
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
  int64_t blocks = (a.T + BS_NT * BS_PER_THREAD - 1) / (BS_NT * BS_PER_THREAD);
  if (blocks > kSolveMaxBlocks) blocks = kSolveMaxBlocks;
  budget_init_kernel<<<(unsigned)blocks, BS_NT, 0, s>>>(a.T, a.rec, a.sc, a.solve, budget);
  for (int r = 0; r < BS_ROUNDS; ++r)
    budget_round_kernel<<<(unsigned)blocks, BS_NT, 0, s>>>(a.T, a.rec, a.sc, a.solve, budget);
  *n_launch += 2 + BS_ROUNDS;
  return cudaGetLastError();
}

cudaError_t launch_epilogue(const EpilogueArgs& a, cudaStream_t s, int* n_launch) {
  // both may be set up while the kernel before them still runs (they wait for its end themselves)
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(EPI_NT);
  cfg.stream = s;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)a.n_part);
  cudaError_t e = cudaLaunchKernelEx(&cfg, epilogue_kernel, a);
  if (e != cudaSuccess) return e;
  const unsigned blocks = (unsigned)((a.T + EPI_NT - 1) / EPI_NT);
  cfg.gridDim = dim3(blocks < 1 ? 1 : blocks);
  e = cudaLaunchKernelEx(&cfg, finalize_kernel, a);
  *n_launch += 2;
  return e;
}

cudaError_t launch_logprobs(int64_t T, const Records& rec, float* out_lq, float* out_lp, uint8_t* out_valid,
                            cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  logprobs_kernel<<<(unsigned)((T + EPI_NT - 1) / EPI_NT), EPI_NT, 0, s>>>(T, rec, out_lq, out_lp, out_valid);
  return cudaGetLastError();
}

}  // namespace jp
