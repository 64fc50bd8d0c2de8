// OBRS token-pass oracle: plain, slow, double-precision CPU code.
//
// TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call, link or
// import this file; it exists so that the CUDA library can be checked against
// an independent statement of what the paper computes.  It shares no code,
// header, table or constant with the CUDA sources.
//
// Every function takes the algorithm's steps in the paper's order, sums in
// ascending index order in double, and uses no blocking or fusion.  OpenMP is
// used over independent rows only.
//
// Notation (paper -> here):  p_inf / q = softmax(actor logits za),
// p_target / p_new / p = softmax(policy logits zp),  lambda = C = c,
// a(x) = acceptance probability,  Z = normaliser = expected acceptance rate,
// Z_approx = top-k estimate,  kappa = batch calibration factor.
//
// Parity pins for every function below live in tests/test_oracle_pins.py.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { JO_BF16 = 0, JO_F32 = 1 };

// Exact widening of one stored logit to double.
inline double logit_at(const void* base, int dtype, int64_t i) {
  if (dtype == JO_BF16) {
    uint32_t bits = (uint32_t)((const uint16_t*)base)[i] << 16;
    float f;
    std::memcpy(&f, &bits, 4);
    return (double)f;
  }
  return (double)((const float*)base)[i];
}

inline bool row_valid(const uint8_t* mask, int64_t t) { return mask == nullptr || mask[t] != 0; }

// log sum_v exp(z_v): the textbook max-shifted form (softmax of the model's
// logits defines p_inf(.|s_t) and p_new(.|s_t); Algorithm 1, Phase 1 / Phase 2 step 1).
double row_lse(const void* z, int dtype, int64_t row0, int64_t V) {
  double m = -std::numeric_limits<double>::infinity();
  for (int64_t v = 0; v < V; ++v) m = std::max(m, logit_at(z, dtype, row0 + v));
  double S = 0.0;
  for (int64_t v = 0; v < V; ++v) S += std::exp(logit_at(z, dtype, row0 + v) - m);
  return m + std::log(S);
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw; SC'11), written from the published
// round function: two 32x32->64 multiplies, xor with the other counter words and
// the round key, key bumped by the Weyl constants each round.
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)M0 * c0;
    uint64_t p1 = (uint64_t)M1 * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

}  // namespace

extern "C" {

int jo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void jo_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

// Raw Philox block, exposed so that the known-answer vectors can pin it.
void jo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

// The uniform the accept test draws for global token index g (Algorithm 2's
// U(0,1)): first output word of Philox keyed on the seed with the counter set
// to g, top 24 bits scaled to [0, 1).
float jo_uniform(uint64_t seed, uint64_t g) {
  uint32_t ctr[4] = {(uint32_t)g, (uint32_t)(g >> 32), 0u, 0u};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  philox4x32_10(ctr, key, out);
  return (float)(out[0] >> 8) * (1.0f / 16777216.0f);
}

// Step 1+2: per valid row the two log-sum-exps and the sampled token's
// log-probabilities  log p_inf(a_t|s_t), log p_new(a_t|s_t)  (Algorithm 1,
// Phase 1 line "store p_inf(a_t|s_t)", Phase 2 step 1).
// Masked rows get 0 in every output.  tokens outside [0,V) mark the row bad:
// outputs 0 and bad[t] = 1.
void jo_lse_gather(int64_t T, int64_t V, int64_t ld, int dtype, const void* za, const void* zp,
                   const int32_t* tokens, const uint8_t* mask, double* lse_a, double* lse_p,
                   double* lq64, double* lp64, float* lq, float* lp, uint8_t* bad) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t t = 0; t < T; ++t) {
    lse_a[t] = lse_p[t] = lq64[t] = lp64[t] = 0.0;
    lq[t] = lp[t] = 0.0f;
    if (bad) bad[t] = 0;
    if (!row_valid(mask, t)) continue;
    int64_t x = tokens[t];
    if (x < 0 || x >= V) {
      if (bad) bad[t] = 1;
      continue;
    }
    lse_a[t] = row_lse(za, dtype, t * ld, V);
    lse_p[t] = row_lse(zp, dtype, t * ld, V);
    lq64[t] = logit_at(za, dtype, t * ld + x) - lse_a[t];
    lp64[t] = logit_at(zp, dtype, t * ld + x) - lse_p[t];
    lq[t] = (float)lq64[t];
    lp[t] = (float)lp64[t];
  }
}

// Step 3: top-k(p) = the k most probable tokens of one distribution (Section
// 4.4.1).  Within a row the logit order is the probability order.  The order
// is total: higher logit first, numerically equal logits (so -0 == +0) by
// lower index.  Output idx[t, 0..k) in that order; rows that are masked get -1.
void jo_topk(int64_t T, int64_t V, int64_t ld, int dtype, const void* z, const uint8_t* mask,
             int k, int32_t* idx) {
  int64_t kk = std::min<int64_t>(k, V);
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t j = 0; j < k; ++j) idx[t * k + j] = -1;
    if (!row_valid(mask, t)) continue;
    std::vector<double> val(V);
    for (int64_t v = 0; v < V; ++v) val[v] = logit_at(z, dtype, t * ld + v);
    std::vector<int32_t> order(V);
    std::iota(order.begin(), order.end(), 0);
    auto before = [&](int32_t i, int32_t j) {
      if (val[i] > val[j]) return true;
      if (val[i] < val[j]) return false;
      return i < j;
    };
    std::partial_sort(order.begin(), order.begin() + kk, order.end(), before);
    for (int64_t j = 0; j < kk; ++j) idx[t * k + j] = order[j];
  }
}

// Step 4 (budget mode): the scalar lambda for which the mean acceptance
// probability over the batch's N valid sampled tokens equals the budget b
// (Theorem 3.4 / Theorem A.1: a unique lambda meets any budget in (0,1]; here
// applied to the empirical token batch, the expectation over x ~ p_inf being
// replaced by the sample mean).  With r_t = p(x_t)/q(x_t) sorted ascending and
// S_j the sum of the j smallest,
//     g(lambda) = (1/N) [ #{r >= lambda} + (1/lambda) sum_{r < lambda} r ]
// is continuous and non-increasing; if exactly the j smallest lie below lambda,
// g = b gives lambda_j = S_j / (N b - (N - j)).  The right j is the smallest one
// with lambda_j <= r_(j+1)  (equivalently g(r_(j+1)) <= b).  b = 1 gives the
// largest lambda with full acceptance, min_t r_t.
// d[t] = lp[t] - lq[t] evaluated in fp32 (the published log-probs), widened.
double jo_lambda_from_budget(int64_t T, const float* lq, const float* lp, const uint8_t* mask,
                             const uint8_t* bad, double budget) {
  std::vector<double> r;
  for (int64_t t = 0; t < T; ++t) {
    if (!row_valid(mask, t) || (bad && bad[t])) continue;
    float d = lp[t] - lq[t];
    r.push_back(std::exp((double)d));
  }
  int64_t N = (int64_t)r.size();
  if (N == 0) return 1.0;
  std::sort(r.begin(), r.end());
  if (budget >= 1.0) return r[0];
  double S = 0.0;
  for (int64_t j = 1; j <= N; ++j) {
    S += r[j - 1];
    double denom = (double)N * budget - (double)(N - j);
    if (denom <= 0.0) continue;
    double lam = S / denom;
    if (j == N || lam <= r[j]) return lam;
  }
  return r[N - 1];  // not reached: j == N always returns
}

// Step 5+6: acceptance probability a(x) = min(1, p_target(x) / (lambda p_inf(x)))
// (Eq. obrs_accept), evaluated in fp32 in a fixed order, and the Bernoulli
// decision  Mask(x) = [U(0,1) < a(x)]  (Algorithm 2; strict "<").
// The uniform for row t is keyed on the global index token_offset + t, padding
// rows included, so the stream does not depend on the mask.
void jo_accept(int64_t T, const float* lq, const float* lp, const uint8_t* mask,
               const uint8_t* bad, float lambda, uint64_t seed, int64_t token_offset,
               float* a_out, float* u_out, uint8_t* accept) {
  float log_lambda = std::log(lambda);
  for (int64_t t = 0; t < T; ++t) {
    float u = jo_uniform(seed, (uint64_t)(token_offset + t));
    u_out[t] = u;
    a_out[t] = 0.0f;
    accept[t] = 0;
    if (!row_valid(mask, t) || (bad && bad[t])) continue;
    float d = lp[t] - lq[t];
    float e = d - log_lambda;
    float a = std::fmin(1.0f, std::exp(e));
    a_out[t] = a;
    accept[t] = (u < a) ? 1 : 0;
  }
}

// Step 7a: Z_approx = sum over V_k = top-k(p_inf) U top-k(p_new) of
// min(p_inf(x), p_new(x)/lambda), every index counted once (Section 4.4.1;
// Algorithm 1 step 2).  idx_a / idx_p are the [T,k] lists from jo_topk.
void jo_z_topk(int64_t T, int64_t V, int64_t ld, int dtype, const void* za, const void* zp,
               const uint8_t* mask, const uint8_t* bad, int k, const int32_t* idx_a,
               const int32_t* idx_p, const double* lse_a, const double* lse_p, double lambda,
               double* zk) {
  (void)V;
#pragma omp parallel for schedule(dynamic, 16)
  for (int64_t t = 0; t < T; ++t) {
    zk[t] = 0.0;
    if (!row_valid(mask, t) || (bad && bad[t])) continue;
    std::vector<int32_t> support;
    for (int j = 0; j < k; ++j)
      if (idx_a[t * k + j] >= 0) support.push_back(idx_a[t * k + j]);
    for (int j = 0; j < k; ++j)
      if (idx_p[t * k + j] >= 0) support.push_back(idx_p[t * k + j]);
    std::sort(support.begin(), support.end());
    support.erase(std::unique(support.begin(), support.end()), support.end());
    double acc = 0.0;
    for (int32_t x : support) {
      double q = std::exp(logit_at(za, dtype, t * ld + x) - lse_a[t]);
      double p = std::exp(logit_at(zp, dtype, t * ld + x) - lse_p[t]);
      acc += std::min(q, p / lambda);
    }
    zk[t] = acc;
  }
}

// Step 7a, with the rollout model known only through what Algorithm 1 Phase 1 stores: per token
// the log-probabilities of its k_inf most likely tokens, inf_idx / inf_logp [T, k_inf] (index
// -1 = empty place).  Phase 2 step 2 sums min(p_inf(x), p_new(x)/lambda) over
// V_k = TopK_inf U TopK_new.  For x in TopK_inf the term is as printed.  For x in TopK_new that
// the rollout did not store, p_inf(x) is not known (the paper does not say what to take); two
// readings, both returned:
//   z_lo  the term is left out: a lower bound of the Z_approx of the dense path, so the
//         inequality Z_approx <= Z on which Section 4.4.2 builds its correction still holds;
//   z_hi  p_inf(x) is replaced by what is known about it, p_inf(x) <= the smallest stored
//         probability, and the unknown terms together by the mass the stored list leaves,
//         1 - sum of the stored probabilities: an upper bound of the dense Z_approx.
// new_idx [T, k] is TopK_new from jo_topk on the policy logits.
void jo_z_sparse(int64_t T, int64_t V, int64_t ld, int dtype, const void* zp, const uint8_t* mask,
                 const uint8_t* bad, int k_inf, const int32_t* inf_idx, const float* inf_logp, int k,
                 const int32_t* new_idx, const double* lse_p, double lambda, double* z_lo, double* z_hi) {
  (void)V;
#pragma omp parallel for schedule(dynamic, 16)
  for (int64_t t = 0; t < T; ++t) {
    z_lo[t] = 0.0;
    z_hi[t] = 0.0;
    if (!row_valid(mask, t) || (bad && bad[t])) continue;
    double stored_sum = 0.0, stored_mass = 0.0, p_min = 1.0;
    int n_stored = 0;
    for (int j = 0; j < k_inf; ++j) {
      const int32_t x = inf_idx[t * k_inf + j];
      if (x < 0) continue;
      const double q = std::exp((double)inf_logp[t * k_inf + j]);
      const double p = std::exp(logit_at(zp, dtype, t * ld + x) - lse_p[t]);
      stored_sum += std::min(q, p / lambda);
      stored_mass += q;
      p_min = std::min(p_min, q);
      ++n_stored;
    }
    double unknown = 0.0;
    for (int j = 0; j < k; ++j) {
      const int32_t x = new_idx[t * k + j];
      if (x < 0) continue;
      bool stored = false;
      for (int i = 0; i < k_inf; ++i) stored = stored || inf_idx[t * k_inf + i] == x;
      if (stored) continue;
      const double p = std::exp(logit_at(zp, dtype, t * ld + x) - lse_p[t]);
      unknown += std::min(n_stored > 0 ? p_min : 1.0, p / lambda);
    }
    z_lo[t] = stored_sum;
    z_hi[t] = stored_sum + std::min(unknown, std::max(0.0, 1.0 - stored_mass));
  }
}

// Logits of an output layer for a set of rows: z[t, v] = sum_h hidden[t, h] * weight[v, h], both
// operands bf16 (every product is exact in double), summed in double in ascending h, rounded once
// to fp32.  (Section 4.4: the logit tensor the method consumes is the output of this product; a
// fused pass forms it tile by tile and never stores it.)
void jo_lmhead_rows(int64_t n_rows, const int64_t* rows, int64_t H, int64_t V, const uint16_t* hidden,
                    int64_t ld_hidden, const uint16_t* weight, int64_t ld_weight, float* out) {
#pragma omp parallel for schedule(dynamic, 64) collapse(2)
  for (int64_t i = 0; i < n_rows; ++i) {
    for (int64_t v = 0; v < V; ++v) {
      const uint16_t* hr = hidden + rows[i] * ld_hidden;
      const uint16_t* wr = weight + v * ld_weight;
      double acc = 0.0;
      for (int64_t h = 0; h < H; ++h) acc += logit_at(hr, 0, h) * logit_at(wr, 0, h);
      out[i * V + v] = (float)acc;
    }
  }
}

// Step 7b: the exact normaliser Z = sum_{x'} min(p_inf(x'), p_target(x')/lambda)
// over the whole vocabulary (Eq. obrs_dist; Appendix A, Z_C).
void jo_z_exact(int64_t T, int64_t V, int64_t ld, int dtype, const void* za, const void* zp,
                const uint8_t* mask, const uint8_t* bad, const double* lse_a,
                const double* lse_p, double lambda, double* z) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t t = 0; t < T; ++t) {
    z[t] = 0.0;
    if (!row_valid(mask, t) || (bad && bad[t])) continue;
    double acc = 0.0;
    for (int64_t v = 0; v < V; ++v) {
      double q = std::exp(logit_at(za, dtype, t * ld + v) - lse_a[t]);
      double p = std::exp(logit_at(zp, dtype, t * ld + v) - lse_p[t]);
      acc += std::min(q, p / lambda);
    }
    z[t] = acc;
  }
}

// Step 8: batch-level bias correction and the OBRS weight (Section 4.4.2;
// Algorithm 1 steps 2-3):
//   alpha_hat = #accepted / #proposed,   kappa = alpha_hat / mean_t Z_approx(t),
//   Z_t = kappa Z_approx(t),   w_OBRS = Z_t max(lambda, p_new(a_t)/p_inf(a_t)),
//   published weight min(w_OBRS, c1)  (c1 <= 0 means no clip).
// "Samples in the batch" = valid proposed tokens.  kappa := 1 if N = 0 or the
// mean is 0.  stats8 = {N, n_accept, alpha_hat, mean a, mean Z_approx, kappa,
// lambda, 0}.
void jo_batch_weights(int64_t T, const float* lq, const float* lp, const uint8_t* mask,
                      const uint8_t* bad, const uint8_t* accept, const float* a,
                      const double* zk, double lambda, double c1, float* w, double* w64,
                      double* stats8) {
  int64_t N = 0, n_acc = 0;
  double sum_zk = 0.0, sum_a = 0.0;
  for (int64_t t = 0; t < T; ++t) {
    if (!row_valid(mask, t) || (bad && bad[t])) continue;
    N += 1;
    n_acc += accept[t] ? 1 : 0;
    sum_zk += zk[t];
    sum_a += (double)a[t];
  }
  double alpha_hat = N > 0 ? (double)n_acc / (double)N : 0.0;
  double mean_zk = N > 0 ? sum_zk / (double)N : 0.0;
  double kappa = (N > 0 && mean_zk > 0.0) ? alpha_hat / mean_zk : 1.0;
  for (int64_t t = 0; t < T; ++t) {
    w[t] = 0.0f;
    if (w64) w64[t] = 0.0;
    if (!row_valid(mask, t) || (bad && bad[t])) continue;
    float d = lp[t] - lq[t];
    double ratio = std::exp((double)d);
    double wt = kappa * zk[t] * std::max(lambda, ratio);
    if (c1 > 0.0) wt = std::min(wt, c1);
    if (w64) w64[t] = wt;
    w[t] = (float)wt;
  }
  stats8[0] = (double)N;
  stats8[1] = (double)n_acc;
  stats8[2] = alpha_hat;
  stats8[3] = N > 0 ? sum_a / (double)N : 0.0;
  stats8[4] = mean_zk;
  stats8[5] = kappa;
  stats8[6] = lambda;
  stats8[7] = 0.0;
}

// Algorithm 1, steps 1, 3 and 4, and Eq. ppo_rollout, per proposed token, away from
// the first update after a rollout (where every ratio is 1):
//   policy:  r_theta = p_new(a)/p_ref(a),
//            rho     = min(w_OBRS, c1) * min(p_ref(a)/p_new(a), c2)     (w already carries c1)
//            obj     = Mask * rho * min(r_theta A, clip(r_theta, 1-eps_lo, 1+eps_hi) A)
//   rollout: r_omega = p_omega(a)/p_omega_ref(a),  F = min(p_omega_ref(a)/p_inf(a), tis_cap)
//            obj     = F * min(r_omega A, clip(r_omega, 1-eps_lo, 1+eps_hi) A)
// `slope` is d obj / d r (rho and F sit under stop-gradient): the coefficient A when the
// unclipped branch of the min is the active one, else 0.  A missing log-prob array
// means that ratio is 1; c2 <= 0 / tis_cap <= 0 mean no cap; clip == 0 means no clipping.
// out8 per token: rho, r_theta, slope_theta, obj_theta, F, r_omega, slope_omega, obj_omega.
void jo_ppo_terms(int64_t T, const float* lq, const float* lp, const uint8_t* mask,
                  const uint8_t* accept, const float* weight, const float* adv,
                  const float* logp_ref, const float* logq_ref, const float* logp_inf, int clip,
                  double eps_lo, double eps_hi, double c2, double tis_cap, double* out8) {
  for (int64_t t = 0; t < T; ++t) {
    double* o = out8 + 8 * t;
    for (int i = 0; i < 8; ++i) o[i] = 0.0;
    if (!row_valid(mask, t)) continue;
    const double A = adv ? (double)adv[t] : 1.0;
    auto surrogate = [&](double r, double* slope) {
      double unclipped = r * A;
      if (!clip) { *slope = A; return unclipped; }
      double rc = std::min(std::max(r, 1.0 - eps_lo), 1.0 + eps_hi);
      double clipped = rc * A;
      if (unclipped <= clipped) { *slope = A; return unclipped; }   // min picks the live branch
      *slope = 0.0;
      return clipped;
    };
    // policy side
    double r_theta = logp_ref ? std::exp((double)lp[t] - (double)logp_ref[t]) : 1.0;
    double inv = 1.0 / r_theta;
    if (c2 > 0.0) inv = std::min(inv, c2);
    double rho = (double)weight[t] * inv;
    double slope_t = 0.0;
    double s_t = surrogate(r_theta, &slope_t);
    double m = accept[t] ? 1.0 : 0.0;
    o[0] = rho; o[1] = r_theta; o[2] = m * rho * slope_t; o[3] = m * rho * s_t;
    // rollout side
    double lq_ref = logq_ref ? (double)logq_ref[t] : (double)lq[t];
    double r_omega = std::exp((double)lq[t] - lq_ref);
    double F = 1.0;
    if (logp_inf) {
      F = std::exp(lq_ref - (double)logp_inf[t]);
      if (tis_cap > 0.0) F = std::min(F, tis_cap);
    }
    double slope_o = 0.0;
    double s_o = surrogate(r_omega, &slope_o);
    o[4] = F; o[5] = r_omega; o[6] = F * slope_o; o[7] = F * s_o;
  }
}

// Step 9: gradient with respect to both logit tensors of the loss to minimise
//   J = -L^{PPO-OBRS}(theta) - L^{PPO}(omega) + lambda_distill L^{distill}(omega)
// (Eq. sys_joint_obj with "update using the gradient of -L"), expectations over
// x ~ p_inf taken as the mean over the N valid proposed tokens, with the
// ratios r_theta = r_omega = 1 and F = 1 at the evaluation point:
//   dJ/dzp[t,v] = -(g/N) Mask_t w_t A_t (1[v=x_t] - p_t(v))
//   dJ/dza[t,v] = -(g/N) A_t (1[v=x_t] - q_t(v)) + (g lambda_distill/N)(q_t(v) - p_t(v))
// Mask_t, w_t and the p inside the KL sit under stop-gradient.  With `ppo8` (the
// output of jo_ppo_terms) the two PPO coefficients take their general form instead.
// rows[0..n_rows) selects which rows are written, each as V doubles.
void jo_grad_rows(int64_t n_rows, const int64_t* rows, int64_t V, int64_t ld, int dtype,
                  const void* za, const void* zp, const int32_t* tokens, const uint8_t* mask,
                  const uint8_t* accept, const float* weight, const float* adv,
                  const double* lse_a, const double* lse_p, double n_valid, double grad_out,
                  double lambda_distill, const double* ppo8, double* d_actor, double* d_policy) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t i = 0; i < n_rows; ++i) {
    int64_t t = rows[i];
    double* da = d_actor + i * V;
    double* dp = d_policy + i * V;
    for (int64_t v = 0; v < V; ++v) da[v] = dp[v] = 0.0;
    if (!row_valid(mask, t) || n_valid <= 0.0) continue;
    int64_t x = tokens[t];
    if (x < 0 || x >= V) continue;
    double A = adv ? (double)adv[t] : 1.0;
    double coef_p = -(grad_out / n_valid) * (accept[t] ? 1.0 : 0.0) * (double)weight[t] * A;
    double coef_a = -(grad_out / n_valid) * A;
    if (ppo8) {
      // general form: d obj / d logit = (d obj / d r) * r * (1[v=x] - prob(v)), both sides
      coef_p = -(grad_out / n_valid) * ppo8[8 * t + 2] * ppo8[8 * t + 1];
      coef_a = -(grad_out / n_valid) * ppo8[8 * t + 6] * ppo8[8 * t + 5];
    }
    double coef_d = grad_out * lambda_distill / n_valid;
    for (int64_t v = 0; v < V; ++v) {
      double q = std::exp(logit_at(za, dtype, t * ld + v) - lse_a[t]);
      double p = std::exp(logit_at(zp, dtype, t * ld + v) - lse_p[t]);
      double onehot = (v == x) ? 1.0 : 0.0;
      dp[v] = coef_p * (onehot - p);
      da[v] = coef_a * (onehot - q) + coef_d * (q - p);
    }
  }
}

// The scalar J itself, as a function of live double logits, with every
// stop-gradient quantity passed in as a constant: used only to differentiate
// numerically against jo_grad_rows.
//   J = -(1/N) sum_t Mask_t w_t S(p_zp(x_t)/p_ref_t) - (1/N) sum_t f_t S(q_za(x_t)/q_ref_t)
//       + lambda_distill (1/N) sum_t KL(pfix_t || q_za(.)),
//   S(r) = min(r A_t, clip(r, 1-eps_lo, 1+eps_hi) A_t)   (S(r) = r A_t when clip == 0);
// w_t stands for the whole stop-gradient weight of the policy term (rho of Algorithm 1),
// f_t for F of Eq. ppo_rollout (NULL: 1).
// za, zp: [T,V] doubles; logp_ref, logq_ref: [T]; pfix: [T,V] probabilities.
double jo_loss(int64_t T, int64_t V, const double* za, const double* zp, const int32_t* tokens,
               const uint8_t* mask, const uint8_t* accept, const double* weight,
               const double* adv, const double* logp_ref, const double* logq_ref,
               const double* pfix, double lambda_distill, const double* f_actor, int clip,
               double eps_lo, double eps_hi) {
  int64_t N = 0;
  for (int64_t t = 0; t < T; ++t) N += row_valid(mask, t) ? 1 : 0;
  if (N == 0) return 0.0;
  double J = 0.0;
  for (int64_t t = 0; t < T; ++t) {
    if (!row_valid(mask, t)) continue;
    const double* ra = za + t * V;
    const double* rp = zp + t * V;
    double ma = ra[0], mp = rp[0];
    for (int64_t v = 1; v < V; ++v) { ma = std::max(ma, ra[v]); mp = std::max(mp, rp[v]); }
    double sa = 0.0, sp = 0.0;
    for (int64_t v = 0; v < V; ++v) { sa += std::exp(ra[v] - ma); sp += std::exp(rp[v] - mp); }
    double lsa = ma + std::log(sa), lsp = mp + std::log(sp);
    int64_t x = tokens[t];
    double A = adv ? adv[t] : 1.0;
    double r_theta = std::exp(rp[x] - lsp - logp_ref[t]);
    double r_omega = std::exp(ra[x] - lsa - logq_ref[t]);
    auto surrogate = [&](double r) {
      if (!clip) return r * A;
      double rc = std::min(std::max(r, 1.0 - eps_lo), 1.0 + eps_hi);
      return std::min(r * A, rc * A);
    };
    J -= (accept[t] ? 1.0 : 0.0) * weight[t] * surrogate(r_theta);
    J -= (f_actor ? f_actor[t] : 1.0) * surrogate(r_omega);
    double kl = 0.0;
    for (int64_t v = 0; v < V; ++v) {
      double pf = pfix[t * V + v];
      if (pf > 0.0) kl += pf * (std::log(pf) - (ra[v] - lsa));
    }
    J += lambda_distill * kl;
  }
  return J / (double)N;
}

// Theorem 3.4, literally: for ONE pair of distributions (a row), the lambda at which the
// OBRS rule a_v = min(1, p_v / (lambda q_v)) accepts exactly the budget,
//   Z(lambda) = sum_v q_v a_v = sum_v min(q_v, p_v / lambda) = budget.
// Z is continuous and non-increasing in lambda.  With the entries ordered by ratio
// r_v = p_v / q_v ascending, on [r_(j), r_(j+1)] the j lowest ratios are accepted in part:
//   Z(lambda) = sum_{i > j} q_(i) + (1 / lambda) sum_{i <= j} p_(i),
// so lambda_j = P_j / (budget - Qtail_j); the j whose lambda_j lies in its own interval
// is the answer.  budget == 1 gives min_v r_v (the largest lambda that accepts everything).
// Also returns KL(p || q) and KL(p || q~), q~ = min(q, p/lambda) / Z (Figure 2b).
void jo_row_lambda(int64_t T, int64_t V, int64_t ld, int dtype, const void* za, const void* zp,
                   const uint8_t* mask, double budget, double* lambda, double* kl_before,
                   double* kl_after) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t t = 0; t < T; ++t) {
    lambda[t] = 0.0;
    if (kl_before) kl_before[t] = 0.0;
    if (kl_after) kl_after[t] = 0.0;
    if (!row_valid(mask, t)) continue;
    const double lsa = row_lse(za, dtype, t * ld, V), lsp = row_lse(zp, dtype, t * ld, V);
    std::vector<double> lq(V), lpv(V);
    std::vector<int64_t> order(V);
    for (int64_t v = 0; v < V; ++v) {
      lq[v] = logit_at(za, dtype, t * ld + v) - lsa;
      lpv[v] = logit_at(zp, dtype, t * ld + v) - lsp;
      order[v] = v;
    }
    std::sort(order.begin(), order.end(), [&](int64_t a, int64_t b) {
      double da = lpv[a] - lq[a], db = lpv[b] - lq[b];
      return da < db || (da == db && a < b);
    });
    // suffix sums of q in ratio order
    std::vector<double> qtail(V + 1, 0.0);
    for (int64_t j = V - 1; j >= 0; --j) qtail[j] = qtail[j + 1] + std::exp(lq[order[j]]);
    double lam = std::exp(lpv[order[0]] - lq[order[0]]);       // budget 1: everything accepted in full
    if (budget < qtail[0]) {
      double phead = 0.0;
      for (int64_t j = 1; j <= V; ++j) {                       // the j lowest ratios are cut
        phead += std::exp(lpv[order[j - 1]]);
        double denom = budget - qtail[j];
        if (denom <= 0.0) continue;
        double cand = phead / denom;
        double lo = std::exp(lpv[order[j - 1]] - lq[order[j - 1]]);
        double hi = j < V ? std::exp(lpv[order[j]] - lq[order[j]]) : HUGE_VAL;
        if (cand >= lo * (1.0 - 1e-15) && cand <= hi * (1.0 + 1e-15)) { lam = cand; break; }
      }
    }
    lambda[t] = lam;
    if (kl_before || kl_after) {
      double kb = 0.0, ka = 0.0, Z = 0.0;
      for (int64_t v = 0; v < V; ++v) {
        double p = std::exp(lpv[v]), q = std::exp(lq[v]);
        double kept = std::min(q, p / lam);
        Z += kept;
        if (p > 0.0) {
          kb += p * (lpv[v] - lq[v]);
          ka += p * (lpv[v] - std::log(kept));
        }
      }
      if (kl_before) kl_before[t] = kb;
      if (kl_after) kl_after[t] = ka + std::log(Z);
    }
  }
}

// Step 10 (diagnostic): KL(p_t || q_t) per row, the actor-policy gap of Figure 2.
void jo_kl_rows(int64_t T, int64_t V, int64_t ld, int dtype, const void* za, const void* zp,
                const uint8_t* mask, const double* lse_a, const double* lse_p, double* kl) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t t = 0; t < T; ++t) {
    kl[t] = 0.0;
    if (!row_valid(mask, t)) continue;
    double acc = 0.0;
    for (int64_t v = 0; v < V; ++v) {
      double lgp = logit_at(zp, dtype, t * ld + v) - lse_p[t];
      double lgq = logit_at(za, dtype, t * ld + v) - lse_a[t];
      double p = std::exp(lgp);
      if (p > 0.0) acc += p * (lgp - lgq);
    }
    kl[t] = acc;
  }
}

}  // extern "C"
