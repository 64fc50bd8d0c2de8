// Internal launch interface between the C-ABI host code and the sm_100a kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "jackpot.h"

namespace jp {

// Per-token records kept in the context's workspace (struct of arrays, indexed
// by record row r = record_offset + t).
struct Records {
  int32_t* idx;     // [cap, 2k]  top-k(p_inf) then top-k(p_target) indices, -1 = empty
  float* za;        // [cap, 2k]  actor logit of every candidate
  float* zp;        // [cap, 2k]  policy logit of every candidate
  float* lse_a;     // [cap]
  float* lse_p;     // [cap]
  float* lse_a_lo;  // [cap] what fp32 rounding took from the log-sum-exp (lse = lse_a + lse_a_lo to ~2^-48)
  float* lse_p_lo;  // [cap]
  float* lq;        // [cap] log p_inf(a_t)
  float* lp;        // [cap] log p_target(a_t)
  float* zk;        // [cap] Z_approx (or exact Z when k >= V)
  float* zx;        // [cap] exact Z when asked for beside Z_approx
  float* a;         // [cap] acceptance probability
  float* kl;        // [cap] KL(p_target || p_inf) of the row, when the caller asked for it
  uint8_t* flag;    // [cap] 1 = valid row with records, 0 = masked / bad token / never streamed,
                    //       2 = streamed, but a log-sum-exp or a log-prob of the sampled token is not finite:
                    //       counted in n_nonfinite and otherwise treated as masked
  double* ratio;    // [cap] p(a_t)/q(a_t) in double, compacted, for the budget solve
  float* dval;      // [cap] lp - lq of the compacted valid rows
};

// Device scalars shared by the kernels of one forward.
struct Scalars {
  int32_t n_list;          // valid rows of the call being streamed (length of the row list)
  int32_t row_counter2;    // persistent-CTA work queue of the exact-Z / gradient kernels
  int32_t n_compact;       // number of valid rows found by the ratio kernel
  int32_t status;
  unsigned long long n_bad_token;
  float lambda;            // lambda in use (fixed, or written by the budget solve)
  float pad;
  double lambda64;
  double totals[4];        // the last forward's batch sums: N, accepted, sum of Z_approx, sum of a(x_t)
  // state of the budget solve between its launches: the bracket [lo, hi] in ordered fp32 bit
  // patterns, count and ratio sum at hi, the number of valid rows, the last-block ticket
  uint32_t bs_lo, bs_hi, bs_ticket, bs_done;
  long long bs_N, bs_c_hi;
  double bs_s_hi;
  jp_stats stats;          // the last forward's batch statistics
};

constexpr uint8_t kRowValid = 1;      // values of Records::flag
constexpr uint8_t kRowNonFinite = 2;

constexpr int kMaxPartials = 1024;
struct Partials {
  long long n_valid[kMaxPartials];
  long long n_accept[kMaxPartials];
  long long n_nonfinite[kMaxPartials];
  double sum_zk[kMaxPartials];
  double sum_a[kMaxPartials];
  double sum_kl[kMaxPartials];
};

// Per-block partial counts and sums of one launch of the budget solve.
constexpr int kSolveMaxBlocks = 256;
constexpr int kSolveWays = 16;
struct SolvePartials {
  long long c[kSolveMaxBlocks][kSolveWays];
  double s[kSolveMaxBlocks][kSolveWays];
};

struct StreamArgs {
  const void* za;          // null: only the policy tensor is streamed (sparse-actor forward)
  const void* zp;
  const float* logp_inf;   // [T] log p_inf(a_t) from the rollout record (only with za == null)
  const int32_t* tokens;
  const uint8_t* mask;
  int64_t T, V, ld;
  int32_t dtype;
  int32_t k;               // 0 = no top-k (exact mode)
  int64_t record_offset;
  Records rec;
  Scalars* sc;
  int32_t* list;           // [T] scratch: the call's valid rows, in no particular order
  uint32_t* spill;         // [kStreamMaxCtas][kStreamSlots][2][kSpillCap] candidate passes that did not fit a CTA's shared memory
};

// Geometry of the stream kernel's spill area (fixed: it depends on neither T nor V).
constexpr int kStreamMaxCtas = 192;   // the grid is one CTA per SM, clamped to this
constexpr int kStreamSlots = 4;       // rows a CTA has in flight
constexpr int kSpillCap = 4096;       // spilled candidates per (CTA, row slot, tensor)
constexpr size_t kSpillBytes = (size_t)kStreamMaxCtas * kStreamSlots * 2 * kSpillCap * sizeof(uint32_t);

struct ExactZArgs {
  const void* za;
  const void* zp;
  int64_t T, V, ld;
  int32_t dtype;
  int64_t record_offset;
  Records rec;
  Scalars* sc;
  float* out;              // rec.zk or rec.zx; null = no exact Z in this pass
  float* out_kl;           // rec.kl; null = no KL(p || q) in this pass
};

struct EpilogueArgs {
  int64_t T;               // record rows to finalise
  int32_t k;               // 0 = zk already holds the exact Z
  uint64_t seed;
  int64_t rng_base;        // accept draw of record row r uses counter rng_base + r
  float c1;
  Records rec;
  Scalars* sc;
  Partials* part;
  SolvePartials* solve;    // scratch of the budget solve
  int32_t n_part;
  int32_t have_kl;         // rec.kl holds KL(p || q) of every valid row: sum it into the statistics
  // outputs, all [T] (any may be null)
  uint8_t* out_accept;
  float* out_weight;
  float* out_lq;
  float* out_lp;
  jp_stats* out_stats;
  int32_t* aux_idx_a; int32_t* aux_idx_p; float* aux_val_a; float* aux_val_p;
  float* aux_a; float* aux_u; float* aux_zk; float* aux_zx; float* aux_lse_a; float* aux_lse_p;
};

struct GradArgs {
  const void* za;
  const void* zp;
  const int32_t* tokens;
  const uint8_t* mask;
  const uint8_t* accept;
  const float* weight;
  const float* adv;
  void* d_actor;
  void* d_policy;
  int64_t T, V, ld;
  int32_t dtype;
  int64_t record_offset;
  float lambda_distill, grad_out;
  int64_t n_valid;         // 0 = read sc->stats.n_valid on the device
  Records rec;
  Scalars* sc;
  // beyond the first update (all optional)
  const float* logp_ref;
  const float* logp_actor_ref;
  const float* logp_inf;
  int32_t clip;            // 1 = PPO clipping on
  float eps_lo, eps_hi, c2, tis_cap;
  float* out_obj_policy;
  float* out_obj_actor;
  float* out_kl;
  double* out_loss;
};

// Z_approx from a stored rollout record (jp_sparse.cu).
struct SparseZArgs {
  const void* zp;
  int64_t T, V, ld;
  int32_t dtype;
  int32_t k, k_inf;
  int32_t cap;             // 0: unknown actor terms left out; 1: capped by what the record implies
  const int32_t* inf_idx;  // [T, k_inf]
  const float* inf_logp;   // [T, k_inf]
  Records rec;
  Scalars* sc;
  float* out_z_lower;      // [T] or null
  float* out_z_upper;      // [T] or null
  int32_t* out_idx_p;      // [T, k] or null
  float* out_val_p;        // [T, k] or null
};

struct RowLambdaArgs {
  const void* za;
  const void* zp;
  const uint8_t* mask;
  int64_t T, V, ld;
  int32_t dtype;
  float budget;
  Scalars* sc;
  float* out_lambda;       // [T]
  float* out_kl_before;    // [T] or null
  float* out_kl_after;     // [T] or null
  int32_t* out_iters;      // [T] or null
};

int stream_grid_size(int device);   // number of SMs
cudaError_t launch_stream(const StreamArgs& a, cudaStream_t s, int sms);
cudaError_t launch_exact_z(const ExactZArgs& a, cudaStream_t s, int sms);
cudaError_t launch_wait_selftest(long long limit_cycles, int32_t* status, cudaStream_t s);
cudaError_t launch_reset(Scalars* sc, float lambda_fixed, cudaStream_t s);
cudaError_t launch_clear_flags(uint8_t* flag, int64_t n, cudaStream_t s);
cudaError_t launch_budget_solve(const EpilogueArgs& a, double budget, cudaStream_t s, int* n_launch);
cudaError_t launch_epilogue(const EpilogueArgs& a, cudaStream_t s, int* n_launch);
cudaError_t launch_reweight(int64_t T, const Records& rec, const Scalars* sc, double kappa, float c1,
                            float* out_weight, cudaStream_t s);
cudaError_t launch_reweight_totals(int64_t T, const Records& rec, Scalars* sc, const double* totals, float c1,
                                   float* out_weight, jp_stats* out_stats, cudaStream_t s);
cudaError_t launch_logprobs(int64_t T, const Records& rec, float* out_lq, float* out_lp, uint8_t* out_valid,
                            cudaStream_t s);
cudaError_t launch_sparse_z(const SparseZArgs& a, cudaStream_t s);
cudaError_t launch_row_lambda(const RowLambdaArgs& a, cudaStream_t s, int sms);

// Vocabulary shards (jp_vshard.cu).  Packed per-row record of one shard, in 4-byte words:
// [0] flag  [1] owner of the sampled token  [2,3] lse actor (hi, lo)  [4,5] lse policy (hi, lo)
// [6,7] the sampled token's two logits (owner only)  [8, 8+2k) global indices of the two lists
// [8+2k, 8+4k) actor logits of the entries  [8+4k, 8+6k) policy logits of the entries.
constexpr int kVshardHeader = 8;
constexpr int kVshardMaxShards = 128;     // shards the merge kernel walks (four per lane of its warp)
constexpr int kVshardMaxEntries = 4096;   // n_shards * k: the keys of one list of every shard, in a warp's shared memory
constexpr int kVshardMaxDests = 16;       // shards a local pass can push its lines to
struct VshardDests {
  float* dst[kVshardMaxDests];
  int n;
};
__host__ __device__ inline int64_t vshard_words(int k) { return kVshardHeader + 6 * (int64_t)k; }
cudaError_t launch_vshard_localize(int64_t T, const int32_t* tokens, const uint8_t* mask, int64_t vocab_offset,
                                   int64_t V_shard, int64_t V_total, int32_t foreign, int32_t* tok_local,
                                   uint8_t* mask_local, Scalars* sc, cudaStream_t s);
cudaError_t launch_vshard_export(int64_t T, int k, const Records& rec, const void* za, const void* zp, int64_t ld,
                                 int32_t dtype, const int32_t* tok_local, const uint8_t* mask_local,
                                 int64_t vocab_offset, const VshardDests& dests, int64_t line0, cudaStream_t s);
cudaError_t launch_vshard_merge(int n_shards, int my_shard, const float* gathered, int64_t T, int k,
                                const Records& rec, Scalars* sc, cudaStream_t s);
cudaError_t launch_grad(const GradArgs& a, cudaStream_t s, int sms, int* n_launch);

// Output layer fused with the row pass (jp_lmhead.cu).
constexpr int kLmheadMaxK = 64;
struct FusedRecordArgs {
  const void* hidden_a; const void* weight_a; const void* hidden_p; const void* weight_p;   // bf16, row-major
  int64_t ld_ha, ld_wa, ld_hp, ld_wp, H_a, H_p;
  const int32_t* tokens; const uint8_t* mask;
  int64_t T, V;
  int32_t k;
  const float* lse_a; const float* lq; const int32_t* idx_a; const float* val_a;   // the actor pass's results
  const float* lse_p; const float* lp; const int32_t* idx_p; const float* val_p;   // the policy pass's
  Records rec;
  Scalars* sc;
};
cudaError_t launch_fused_records(const FusedRecordArgs& a, cudaStream_t s);
size_t lmhead_scratch_bytes(int64_t T, int k, int splits);
int lmhead_splits(int64_t T, int64_t V, int sms);
cudaError_t launch_lmhead(const void* hidden, int64_t ldh, const void* weight, int64_t ldw, const int32_t* tokens,
                          const uint8_t* mask, int64_t T, int64_t H, int64_t V, int k, int splits, void* scratch,
                          int32_t* status, float* out_lse, float* out_logp, int32_t* out_idx, float* out_val,
                          cudaStream_t s);

}  // namespace jp
