// C-ABI host side of libjackpot: argument validation, workspace, launch plans.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <string>

#include "jp_internal.h"

using namespace jp;

struct jp_ctx {
  int device = 0;
  int sms = 148;
  cudaStream_t stream = nullptr;
  char* ws = nullptr;            // workspace: Scalars | Partials | records
  size_t ws_bytes = 0;
  int64_t cap_rows = 0;          // records the workspace is laid out for
  int cap_k = 0;
  Records rec{};
  Scalars* sc = nullptr;
  int32_t* list = nullptr;
  uint32_t* spill = nullptr;
  int32_t* vtok = nullptr;       // a vocabulary shard's view of the call: local token ids ...
  uint8_t* vmask = nullptr;      // ... and row validity (2 = this shard holds the sampled token)
  Partials* part = nullptr;
  SolvePartials* solve = nullptr;
  // state of the records
  bool have_records = false;
  int64_t rec_rows = 0;          // rows covered (T of the forward / T_total of the batch)
  int64_t rec_V = 0;
  int rec_k = 0;                 // 0 = exact mode
  bool rec_kl = false;           // the records hold KL(p || q) of every streamed row
  bool rec_sparse = false;       // the records come from the sparse-actor forward: no actor log-sum-exp in them
  int32_t rec_dtype = 0;
  bool batch_open = false;
  bool batch_exact = false;
  bool vshard_local_done = false;   // jp_vshard_local has run: jp_vshard_merge may follow
  int64_t vshard_T = 0;
  int vshard_k = 0;
  int64_t launches = 0;
  bool timing = false;
  static constexpr int kEvRing = 256;
  cudaEvent_t ev0[kEvRing] = {}, ev1[kEvRing] = {};
  int64_t ev_count = 0;          // stream-kernel launches timed since timing was enabled
  // staging for the host-buffer entry point
  char* lm_scratch = nullptr;    // partial results of the fused output-layer pass
  size_t lm_bytes = 0;
  char* stage = nullptr;
  size_t stage_bytes = 0;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t copy_done[2] = {nullptr, nullptr}, compute_done[2] = {nullptr, nullptr};
  std::string err;
};

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  size_t scalars, partials, solve, idx, za, zp, f[10], flag, ratio, dval, list, spill, vtok, vmask, total;
};

Layout layout_for(int64_t rows, int k) {
  Layout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.scalars = take(sizeof(Scalars));
  L.partials = take(sizeof(Partials));
  L.solve = take(sizeof(SolvePartials));
  size_t cand = (size_t)rows * 2 * (size_t)(k > 0 ? k : 1);
  L.idx = take(cand * 4);
  L.za = take(cand * 4);
  L.zp = take(cand * 4);
  for (int i = 0; i < 10; ++i) L.f[i] = take((size_t)rows * 4);
  L.flag = take((size_t)rows);
  L.ratio = take((size_t)rows * 8);
  L.dval = take((size_t)rows * 4);
  L.list = take((size_t)rows * 4);
  L.spill = take(kSpillBytes);
  L.vtok = take((size_t)rows * 4);
  L.vmask = take((size_t)rows);
  L.total = off;
  return L;
}

jp_status fail(jp_ctx* c, jp_status s, const std::string& msg) {
  if (c) c->err = msg;
  return s;
}

jp_status cuda_fail(jp_ctx* c, cudaError_t e, const char* what) {
  return fail(c, JP_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

jp_status ensure_workspace(jp_ctx* c, int64_t rows, int k) {
  int kk = k > 0 ? k : 1;
  if (c->ws && rows <= c->cap_rows && kk <= c->cap_k) {
    // re-lay out for the current k so that records are dense
  } else {
    int64_t new_rows = rows > c->cap_rows ? rows : c->cap_rows;
    int new_k = kk > c->cap_k ? kk : c->cap_k;
    Layout L = layout_for(new_rows, new_k);
    if (L.total > c->ws_bytes) {
      cudaError_t e = cudaStreamSynchronize(c->stream);
      if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamSynchronize");
      if (c->ws) cudaFree(c->ws);
      c->ws = nullptr;
      c->ws_bytes = 0;
      e = cudaMalloc((void**)&c->ws, L.total);
      if (e != cudaSuccess) return fail(c, JP_ERR_WORKSPACE, std::string("workspace cudaMalloc: ") + cudaGetErrorString(e));
      c->ws_bytes = L.total;
      c->have_records = false;
    }
    c->cap_rows = new_rows;
    c->cap_k = new_k;
  }
  Layout L = layout_for(c->cap_rows, c->cap_k);
  char* b = c->ws;
  c->sc = (Scalars*)(b + L.scalars);
  c->part = (Partials*)(b + L.partials);
  c->solve = (SolvePartials*)(b + L.solve);
  c->rec.idx = (int32_t*)(b + L.idx);
  c->rec.za = (float*)(b + L.za);
  c->rec.zp = (float*)(b + L.zp);
  c->rec.lse_a = (float*)(b + L.f[0]);
  c->rec.lse_p = (float*)(b + L.f[1]);
  c->rec.lq = (float*)(b + L.f[2]);
  c->rec.lp = (float*)(b + L.f[3]);
  c->rec.zk = (float*)(b + L.f[4]);
  c->rec.zx = (float*)(b + L.f[5]);
  c->rec.a = (float*)(b + L.f[6]);
  c->rec.lse_a_lo = (float*)(b + L.f[7]);
  c->rec.lse_p_lo = (float*)(b + L.f[8]);
  c->rec.kl = (float*)(b + L.f[9]);
  c->rec.flag = (uint8_t*)(b + L.flag);
  c->rec.ratio = (double*)(b + L.ratio);
  c->rec.dval = (float*)(b + L.dval);
  c->list = (int32_t*)(b + L.list);
  c->spill = (uint32_t*)(b + L.spill);
  c->vtok = (int32_t*)(b + L.vtok);
  c->vmask = (uint8_t*)(b + L.vmask);
  return JP_OK;
}

jp_status check_shape(jp_ctx* c, const jp_obrs_desc* d, int64_t* ld_out) {
  if (!d) return fail(c, JP_ERR_INVALID_ARG, "desc is NULL");
  if (d->T < 0) return fail(c, JP_ERR_INVALID_ARG, "T < 0");
  if (d->V < 1 || d->V > (int64_t)0x7fffffff) return fail(c, JP_ERR_INVALID_ARG, "V out of range");
  if (d->dtype != JP_BF16 && d->dtype != JP_F32) return fail(c, JP_ERR_INVALID_ARG, "unknown dtype");
  int64_t ld = d->ld ? d->ld : d->V;
  if (ld < d->V) return fail(c, JP_ERR_INVALID_ARG, "ld < V");
  int es = d->dtype == JP_BF16 ? 2 : 4;
  if ((ld * es) % 16 != 0) return fail(c, JP_ERR_ALIGNMENT, "row pitch (ld * element size) must be a multiple of 16 bytes");
  *ld_out = ld;
  return JP_OK;
}

jp_status check_k(jp_ctx* c, int k, int64_t V) {
  if (k < 1) return fail(c, JP_ERR_INVALID_ARG, "k < 1");
  if (k > JP_MAX_TOPK && (int64_t)k < V) return fail(c, JP_ERR_UNSUPPORTED, "JP_MAX_TOPK < k < V is not supported");
  return JP_OK;
}

jp_status check_lambda(jp_ctx* c, float v, int32_t mode) {
  if (mode == JP_LAMBDA_FIXED) {
    if (!(v > 0.f) || !(v < 3.0e38f)) return fail(c, JP_ERR_INVALID_ARG, "lambda must be finite and > 0");
  } else if (mode == JP_LAMBDA_FROM_BUDGET) {
    if (!(v > 0.f) || v > 1.f) return fail(c, JP_ERR_INVALID_ARG, "budget must lie in (0, 1]");
  } else {
    return fail(c, JP_ERR_INVALID_ARG, "unknown lambda_mode");
  }
  return JP_OK;
}

// One more pass over a block of rows: the exact Z (into z_out) and / or KL(p || q).
jp_status extra_pass(jp_ctx* c, const jp_obrs_desc* d, int64_t ld, int64_t record_offset, const void* za,
                     const void* zp, float* z_out, bool want_kl) {
  if (d->T == 0 || (!z_out && !want_kl)) return JP_OK;
  cudaError_t e = cudaMemsetAsync(&c->sc->row_counter2, 0, sizeof(int32_t), c->stream);   // the pass's work queue
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemsetAsync");
  ExactZArgs x{};
  x.za = za; x.zp = zp; x.T = d->T; x.V = d->V; x.ld = ld; x.dtype = d->dtype;
  x.record_offset = record_offset; x.rec = c->rec; x.sc = c->sc;
  x.out = z_out;
  x.out_kl = want_kl ? c->rec.kl : nullptr;
  e = launch_exact_z(x, c->stream, c->sms);
  if (e != cudaSuccess) return cuda_fail(c, e, "exact-Z / KL kernel launch");
  c->launches += 1;
  return JP_OK;
}

// Streams one block of rows into the records at record_offset.
jp_status stream_rows(jp_ctx* c, const jp_obrs_desc* d, int64_t ld, int k_eff, int64_t record_offset,
                      const void* za, const void* zp, const int32_t* tokens, const uint8_t* mask,
                      const float* logp_inf = nullptr) {
  if (d->T == 0) return JP_OK;
  // za == NULL with logp_inf: the policy tensor alone is streamed (sparse-actor forward)
  if ((!za && !logp_inf) || !zp || !tokens) return fail(c, JP_ERR_INVALID_ARG, "logits or tokens pointer is NULL");
  if (!aligned16(za) || !aligned16(zp)) return fail(c, JP_ERR_ALIGNMENT, "logit base pointers must be 16-byte aligned");
  StreamArgs a{};
  a.za = za; a.zp = zp; a.tokens = tokens; a.mask = mask; a.logp_inf = logp_inf;
  a.T = d->T; a.V = d->V; a.ld = ld; a.dtype = d->dtype; a.k = k_eff;
  a.record_offset = record_offset; a.rec = c->rec; a.sc = c->sc; a.list = c->list; a.spill = c->spill;
  const int slot = (int)(c->ev_count % jp_ctx::kEvRing);
  if (c->timing) {
    if (!c->ev0[slot]) { cudaEventCreate(&c->ev0[slot]); cudaEventCreate(&c->ev1[slot]); }
    cudaEventRecord(c->ev0[slot], c->stream);
  }
  cudaError_t e = launch_stream(a, c->stream, c->sms);
  if (c->timing) { cudaEventRecord(c->ev1[slot], c->stream); c->ev_count += 1; }
  if (e != cudaSuccess) return cuda_fail(c, e, "stream kernel launch");
  c->launches += 2;
  return JP_OK;
}

EpilogueArgs epilogue_args(jp_ctx* c, const jp_obrs_desc* d, int64_t T, int k_eff, uint64_t seed,
                           int64_t rng_base, float c1, uint8_t* out_accept, float* out_weight,
                           float* out_lq, float* out_lp, jp_stats* out_stats) {
  EpilogueArgs a{};
  a.T = T; a.k = k_eff; a.seed = seed; a.rng_base = rng_base; a.c1 = c1;
  a.rec = c->rec; a.sc = c->sc; a.part = c->part; a.solve = c->solve;
  int64_t np = (T + 7) / 8;
  a.n_part = (int32_t)(np < 1 ? 1 : (np > kMaxPartials ? kMaxPartials : np));
  a.out_accept = out_accept; a.out_weight = out_weight; a.out_lq = out_lq; a.out_lp = out_lp;
  a.out_stats = out_stats;
  a.have_kl = c->rec_kl ? 1 : 0;
  if (d) {
    a.aux_idx_a = d->topk_idx_actor; a.aux_idx_p = d->topk_idx_policy;
    a.aux_val_a = d->topk_val_actor; a.aux_val_p = d->topk_val_policy;
    a.aux_a = d->accept_prob; a.aux_u = d->uniform; a.aux_zk = d->z_approx; a.aux_zx = d->z_exact;
    a.aux_lse_a = d->lse_actor; a.aux_lse_p = d->lse_policy;
  }
  return a;
}

}  // namespace

extern "C" {

const char* jp_status_string(jp_status s) {
  switch (s) {
    case JP_OK: return "ok";
    case JP_ERR_INVALID_ARG: return "invalid argument";
    case JP_ERR_ALIGNMENT: return "misaligned pointer or row pitch";
    case JP_ERR_UNSUPPORTED: return "unsupported configuration";
    case JP_ERR_WORKSPACE: return "workspace allocation failed";
    case JP_ERR_CUDA: return "CUDA error";
    case JP_ERR_TIMEOUT: return "device wait timed out";
    case JP_ERR_STATE: return "call out of sequence";
    case JP_ERR_TOO_LARGE: return "size beyond the fixed maximum of this entry point";
  }
  return "unknown status";
}

const char* jp_last_error(jp_ctx* ctx) { return ctx ? ctx->err.c_str() : "context is NULL"; }

int64_t jp_launch_count(jp_ctx* ctx) { return ctx ? ctx->launches : 0; }

jp_status jp_create(jp_ctx** out_ctx, int device, void* cuda_stream) {
  if (!out_ctx) return JP_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  int n = 0;
  cudaError_t e = cudaGetDeviceCount(&n);
  if (e != cudaSuccess || device < 0 || device >= n) return JP_ERR_CUDA;
  e = cudaSetDevice(device);
  if (e != cudaSuccess) return JP_ERR_CUDA;
  jp_ctx* c = new (std::nothrow) jp_ctx();
  if (!c) return JP_ERR_WORKSPACE;
  c->device = device;
  c->stream = (cudaStream_t)cuda_stream;
  c->sms = stream_grid_size(device);
  *out_ctx = c;
  return JP_OK;
}

jp_status jp_destroy(jp_ctx* c) {
  if (!c) return JP_OK;
  cudaSetDevice(c->device);
  cudaStreamSynchronize(c->stream);
  if (c->ws) cudaFree(c->ws);
  if (c->stage) cudaFree(c->stage);
  if (c->lm_scratch) cudaFree(c->lm_scratch);
  for (int i = 0; i < jp_ctx::kEvRing; ++i) {
    if (c->ev0[i]) cudaEventDestroy(c->ev0[i]);
    if (c->ev1[i]) cudaEventDestroy(c->ev1[i]);
  }
  for (int i = 0; i < 2; ++i) {
    if (c->copy_done[i]) cudaEventDestroy(c->copy_done[i]);
    if (c->compute_done[i]) cudaEventDestroy(c->compute_done[i]);
  }
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  delete c;
  return JP_OK;
}

jp_status jp_set_stream(jp_ctx* c, void* cuda_stream) {
  if (!c) return JP_ERR_INVALID_ARG;
  c->stream = (cudaStream_t)cuda_stream;
  return JP_OK;
}

size_t jp_obrs_workspace_bytes(int64_t T_max, int64_t V, int k) {
  if (T_max < 0 || k < 1) return 0;
  int kk = (k > JP_MAX_TOPK || (int64_t)k >= V) ? 1 : k;
  return layout_for(T_max, kk).total;
}

jp_status jp_reserve(jp_ctx* c, int64_t T_max, int64_t V, int k) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (T_max < 0 || k < 1) return fail(c, JP_ERR_INVALID_ARG, "T_max < 0 or k < 1");
  cudaSetDevice(c->device);
  int kk = (k > JP_MAX_TOPK || (int64_t)k >= V) ? 1 : k;
  return ensure_workspace(c, T_max > 0 ? T_max : 1, kk);
}

jp_status jp_enable_kernel_timing(jp_ctx* c, int on) {
  if (!c) return JP_ERR_INVALID_ARG;
  c->timing = on != 0;
  c->ev_count = 0;
  return JP_OK;
}

int64_t jp_stream_kernel_times(jp_ctx* c, float* out_ms, int64_t n) {
  if (!c || !out_ms || n <= 0) return 0;
  int64_t have = c->ev_count < jp_ctx::kEvRing ? c->ev_count : jp_ctx::kEvRing;
  if (n > have) n = have;
  for (int64_t i = 0; i < n; ++i) {
    int slot = (int)((c->ev_count - n + i) % jp_ctx::kEvRing);
    out_ms[i] = -1.f;
    if (cudaEventSynchronize(c->ev1[slot]) != cudaSuccess) continue;
    cudaEventElapsedTime(&out_ms[i], c->ev0[slot], c->ev1[slot]);
  }
  return n;
}

jp_status jp_obrs_forward(jp_ctx* c, const jp_obrs_desc* d, const void* za, const void* zp,
                          const int32_t* tokens, const uint8_t* mask, float lambda_or_budget, int k,
                          uint64_t seed, uint8_t* out_accept, float* out_weight, float* out_lq,
                          float* out_lp, jp_stats* out_stats) {
  if (!c) return JP_ERR_INVALID_ARG;
  int64_t ld = 0;
  jp_status st = check_shape(c, d, &ld);
  if (st != JP_OK) return st;
  if ((st = check_k(c, k, d->V)) != JP_OK) return st;
  if ((st = check_lambda(c, lambda_or_budget, d->lambda_mode)) != JP_OK) return st;
  if (c->batch_open) return fail(c, JP_ERR_STATE, "a chunked batch is open: finalize it first");
  cudaSetDevice(c->device);
  const bool exact = (int64_t)k >= d->V;
  const int k_eff = exact ? 0 : k;
  const bool want_zx = d->z_exact != nullptr && !exact;
  if ((st = ensure_workspace(c, d->T > 0 ? d->T : 1, k_eff)) != JP_OK) return st;
  const bool budget = d->lambda_mode == JP_LAMBDA_FROM_BUDGET;
  const bool want_kl = (d->flags & JP_DESC_KL) != 0;
  cudaError_t e = launch_reset(c->sc, budget ? 1.0f : lambda_or_budget, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "reset launch");
  c->launches += 1;
  c->have_records = false;
  c->rec_kl = want_kl;
  c->rec_sparse = false;
  st = stream_rows(c, d, ld, k_eff, 0, za, zp, tokens, mask);
  if (st != JP_OK) return st;
  // the exact Z needs lambda: with a budget it has to wait for the solve; the divergence does not
  float* z_out = exact ? c->rec.zk : (want_zx ? c->rec.zx : nullptr);
  if ((st = extra_pass(c, d, ld, 0, za, zp, budget ? nullptr : z_out, want_kl)) != JP_OK) return st;
  EpilogueArgs ea = epilogue_args(c, d, d->T, k_eff, seed, d->token_offset, d->c1, out_accept,
                                  out_weight, out_lq, out_lp, out_stats);
  int nl = 0;
  if (budget) {
    e = launch_budget_solve(ea, (double)lambda_or_budget, c->stream, &nl);
    if (e != cudaSuccess) return cuda_fail(c, e, "budget solve launch");
    if ((st = extra_pass(c, d, ld, 0, za, zp, z_out, false)) != JP_OK) return st;
  }
  e = launch_epilogue(ea, c->stream, &nl);
  c->launches += nl;
  if (e != cudaSuccess) return cuda_fail(c, e, "epilogue launch");
  c->have_records = true;
  c->rec_rows = d->T; c->rec_V = d->V; c->rec_k = k_eff; c->rec_dtype = d->dtype;
  return JP_OK;
}

jp_status jp_obrs_forward_sparse_actor(jp_ctx* c, const jp_obrs_desc* d, const void* zp, const int32_t* tokens,
                                       const uint8_t* mask, const float* logp_inf_token, const int32_t* topk_inf_idx,
                                       const float* topk_inf_logp, int k_inf, float lambda_or_budget, int k,
                                       uint64_t seed, uint8_t* out_accept, float* out_weight, float* out_lp,
                                       float* out_z_lower, float* out_z_upper, jp_stats* out_stats) {
  if (!c) return JP_ERR_INVALID_ARG;
  int64_t ld = 0;
  jp_status st = check_shape(c, d, &ld);
  if (st != JP_OK) return st;
  if (k < 1 || k > JP_MAX_TOPK || (int64_t)k >= d->V)
    return fail(c, JP_ERR_UNSUPPORTED, "the sparse-actor forward takes 1 <= k <= JP_MAX_TOPK, k < V");
  if (k_inf < 1 || k_inf > JP_MAX_TOPK) return fail(c, JP_ERR_UNSUPPORTED, "1 <= k_inf <= JP_MAX_TOPK");
  if ((st = check_lambda(c, lambda_or_budget, d->lambda_mode)) != JP_OK) return st;
  if (c->batch_open) return fail(c, JP_ERR_STATE, "a chunked batch is open: finalize it first");
  if (d->flags & JP_DESC_KL) return fail(c, JP_ERR_UNSUPPORTED, "KL(p || q) needs the rollout model's full logits");
  if (d->topk_idx_actor || d->topk_val_actor || d->z_exact || d->lse_actor)
    return fail(c, JP_ERR_UNSUPPORTED, "actor-side optional outputs do not exist without the actor's logits");
  if (d->T > 0 && (!logp_inf_token || !topk_inf_idx || !topk_inf_logp))
    return fail(c, JP_ERR_INVALID_ARG, "a pointer of the rollout record is NULL");
  cudaSetDevice(c->device);
  if ((st = ensure_workspace(c, d->T > 0 ? d->T : 1, k)) != JP_OK) return st;
  const bool budget = d->lambda_mode == JP_LAMBDA_FROM_BUDGET;
  cudaError_t e = launch_reset(c->sc, budget ? 1.0f : lambda_or_budget, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "reset launch");
  c->launches += 1;
  c->have_records = false;
  c->rec_kl = false;
  c->rec_sparse = true;
  if ((st = stream_rows(c, d, ld, k, 0, nullptr, zp, tokens, mask, logp_inf_token)) != JP_OK) return st;
  // the epilogue takes Z_approx as given (k = 0): the kernel below has computed it from the record
  jp_obrs_desc dd = *d;
  dd.topk_idx_policy = nullptr; dd.topk_val_policy = nullptr;
  EpilogueArgs ea = epilogue_args(c, &dd, d->T, 0, seed, d->token_offset, d->c1, out_accept, out_weight, nullptr,
                                  out_lp, out_stats);
  int nl = 0;
  if (budget) {
    e = launch_budget_solve(ea, (double)lambda_or_budget, c->stream, &nl);
    if (e != cudaSuccess) return cuda_fail(c, e, "budget solve launch");
  }
  if (d->T > 0) {
    SparseZArgs z{};
    z.zp = zp; z.T = d->T; z.V = d->V; z.ld = ld; z.dtype = d->dtype; z.k = k; z.k_inf = k_inf;
    z.cap = (d->flags & JP_DESC_SPARSE_CAP) ? 1 : 0;
    z.inf_idx = topk_inf_idx; z.inf_logp = topk_inf_logp; z.rec = c->rec; z.sc = c->sc;
    z.out_z_lower = out_z_lower; z.out_z_upper = out_z_upper;
    z.out_idx_p = d->topk_idx_policy; z.out_val_p = d->topk_val_policy;
    e = launch_sparse_z(z, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "sparse Z launch");
    nl += 1;
  }
  e = launch_epilogue(ea, c->stream, &nl);
  c->launches += nl;
  if (e != cudaSuccess) return cuda_fail(c, e, "epilogue launch");
  c->have_records = true;
  c->rec_rows = d->T; c->rec_V = d->V; c->rec_k = k; c->rec_dtype = d->dtype;
  return JP_OK;
}

jp_status jp_lmhead_lse_topk(jp_ctx* c, const void* hidden, int64_t ld_hidden, const void* weight, int64_t ld_weight,
                             const int32_t* tokens, const uint8_t* mask, int64_t T, int64_t H, int64_t V, int k,
                             float* out_lse, float* out_logp_token, int32_t* out_topk_idx, float* out_topk_val,
                             int32_t* out_status) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (T < 0 || H < 1 || V < 1 || V > (int64_t)0x7fffffff) return fail(c, JP_ERR_INVALID_ARG, "T < 0, H < 1 or V out of range");
  if (k < 1 || k > kLmheadMaxK) return fail(c, JP_ERR_UNSUPPORTED, "the fused output-layer pass keeps lists of 1 <= k <= 64 entries");
  if (ld_hidden == 0) ld_hidden = H;
  if (ld_weight == 0) ld_weight = H;
  if (ld_hidden < H || ld_weight < H) return fail(c, JP_ERR_INVALID_ARG, "leading dimension < H");
  if ((ld_hidden * 2) % 16 != 0 || (ld_weight * 2) % 16 != 0)
    return fail(c, JP_ERR_ALIGNMENT, "row pitches of hidden and weight must be multiples of 16 bytes");
  if (T == 0) return JP_OK;
  if (!hidden || !weight || !tokens || !out_lse || !out_logp_token || !out_topk_idx || !out_topk_val)
    return fail(c, JP_ERR_INVALID_ARG, "a required pointer is NULL");
  if (!aligned16(hidden) || !aligned16(weight)) return fail(c, JP_ERR_ALIGNMENT, "hidden and weight must be 16-byte aligned");
  cudaSetDevice(c->device);
  const int splits = lmhead_splits(T, V, c->sms);
  const size_t need = lmhead_scratch_bytes(T, k, splits);
  cudaError_t e;
  if (need > c->lm_bytes) {
    cudaStreamSynchronize(c->stream);
    if (c->lm_scratch) cudaFree(c->lm_scratch);
    c->lm_scratch = nullptr; c->lm_bytes = 0;
    e = cudaMalloc((void**)&c->lm_scratch, need);
    if (e != cudaSuccess) return fail(c, JP_ERR_WORKSPACE, std::string("scratch cudaMalloc: ") + cudaGetErrorString(e));
    c->lm_bytes = need;
  }
  int32_t* status = out_status ? out_status : (int32_t*)(c->lm_scratch + need - 256);
  e = cudaMemsetAsync(status, 0, sizeof(int32_t), c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemsetAsync");
  e = launch_lmhead(hidden, ld_hidden, weight, ld_weight, tokens, mask, T, H, V, k, splits, c->lm_scratch, status,
                    out_lse, out_logp_token, out_topk_idx, out_topk_val, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "fused output-layer launch");
  c->launches += 2;
  return JP_OK;
}

jp_status jp_obrs_forward_lmhead(jp_ctx* c, const jp_obrs_desc* d, const void* hidden_actor, int64_t ld_ha,
                                 const void* weight_actor, int64_t ld_wa, int64_t H_actor, const void* hidden_policy,
                                 int64_t ld_hp, const void* weight_policy, int64_t ld_wp, int64_t H_policy,
                                 const int32_t* tokens, const uint8_t* mask, float lambda_or_budget, int k,
                                 uint64_t seed, uint8_t* out_accept, float* out_weight, float* out_lq, float* out_lp,
                                 jp_stats* out_stats) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!d) return fail(c, JP_ERR_INVALID_ARG, "desc is NULL");
  const int64_t T = d->T, V = d->V;
  if (T < 0 || V < 1 || V > (int64_t)0x7fffffff || H_actor < 1 || H_policy < 1)
    return fail(c, JP_ERR_INVALID_ARG, "T < 0, V out of range or a hidden size < 1");
  if (k < 1 || k > kLmheadMaxK || (int64_t)k >= V)
    return fail(c, JP_ERR_UNSUPPORTED, "the fused output-layer pass keeps lists of 1 <= k <= 64 entries, k < V");
  jp_status st = check_lambda(c, lambda_or_budget, d->lambda_mode);
  if (st != JP_OK) return st;
  if (c->batch_open) return fail(c, JP_ERR_STATE, "a chunked batch is open: finalize it first");
  if (d->flags & JP_DESC_KL) return fail(c, JP_ERR_UNSUPPORTED, "KL(p || q) needs whole rows of logits, which this path never forms");
  if (d->z_exact) return fail(c, JP_ERR_UNSUPPORTED, "the exact Z needs whole rows of logits, which this path never forms");
  if (ld_ha == 0) ld_ha = H_actor;
  if (ld_wa == 0) ld_wa = H_actor;
  if (ld_hp == 0) ld_hp = H_policy;
  if (ld_wp == 0) ld_wp = H_policy;
  if (ld_ha < H_actor || ld_wa < H_actor || ld_hp < H_policy || ld_wp < H_policy)
    return fail(c, JP_ERR_INVALID_ARG, "a leading dimension is smaller than the hidden size");
  if ((ld_ha * 2) % 16 || (ld_wa * 2) % 16 || (ld_hp * 2) % 16 || (ld_wp * 2) % 16)
    return fail(c, JP_ERR_ALIGNMENT, "row pitches of hidden states and output matrices must be multiples of 16 bytes");
  if (T > 0 && (!hidden_actor || !weight_actor || !hidden_policy || !weight_policy || !tokens))
    return fail(c, JP_ERR_INVALID_ARG, "a required pointer is NULL");
  if (!aligned16(hidden_actor) || !aligned16(weight_actor) || !aligned16(hidden_policy) || !aligned16(weight_policy))
    return fail(c, JP_ERR_ALIGNMENT, "hidden states and output matrices must be 16-byte aligned");
  cudaSetDevice(c->device);
  if ((st = ensure_workspace(c, T > 0 ? T : 1, k)) != JP_OK) return st;
  const bool budget = d->lambda_mode == JP_LAMBDA_FROM_BUDGET;
  cudaError_t e = launch_reset(c->sc, budget ? 1.0f : lambda_or_budget, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "reset launch");
  c->launches += 1;
  c->have_records = false;
  c->rec_kl = false;
  c->rec_sparse = true;                       // no logits behind these records either: no backward from them
  if (T > 0) {
    const int splits = lmhead_splits(T, V, c->sms);
    const size_t part = (lmhead_scratch_bytes(T, k, splits) + 255) / 256 * 256;
    const size_t per_model = ((size_t)T * (8 + 8 * (size_t)k) + 255) / 256 * 256;   // lse, logp, idx[k], val[k]
    const size_t need = part + 2 * per_model;
    if (need > c->lm_bytes) {
      cudaStreamSynchronize(c->stream);
      if (c->lm_scratch) cudaFree(c->lm_scratch);
      c->lm_scratch = nullptr; c->lm_bytes = 0;
      e = cudaMalloc((void**)&c->lm_scratch, need);
      if (e != cudaSuccess) return fail(c, JP_ERR_WORKSPACE, std::string("scratch cudaMalloc: ") + cudaGetErrorString(e));
      c->lm_bytes = need;
    }
    // the device status word of the row kernels doubles as the fused kernels' (JP_ERR_TIMEOUT lands in jp_stats.status)
    int32_t* status = &c->sc->status;
    float* res[2][4];
    for (int m = 0; m < 2; ++m) {
      char* b = c->lm_scratch + part + (size_t)m * per_model;
      res[m][0] = (float*)b;                                  // lse
      res[m][1] = (float*)(b + (size_t)T * 4);                // log-prob of the token
      res[m][2] = (float*)(b + (size_t)T * 8);                // idx (int32)
      res[m][3] = (float*)(b + (size_t)T * 8 + (size_t)T * k * 4);
    }
    e = launch_lmhead(hidden_actor, ld_ha, weight_actor, ld_wa, tokens, mask, T, H_actor, V, k, splits, c->lm_scratch,
                      status, res[0][0], res[0][1], (int32_t*)res[0][2], res[0][3], c->stream);
    if (e == cudaSuccess)
      e = launch_lmhead(hidden_policy, ld_hp, weight_policy, ld_wp, tokens, mask, T, H_policy, V, k, splits,
                        c->lm_scratch, status, res[1][0], res[1][1], (int32_t*)res[1][2], res[1][3], c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "fused output-layer launch");
    FusedRecordArgs fa{};
    fa.hidden_a = hidden_actor; fa.weight_a = weight_actor; fa.hidden_p = hidden_policy; fa.weight_p = weight_policy;
    fa.ld_ha = ld_ha; fa.ld_wa = ld_wa; fa.ld_hp = ld_hp; fa.ld_wp = ld_wp; fa.H_a = H_actor; fa.H_p = H_policy;
    fa.tokens = tokens; fa.mask = mask; fa.T = T; fa.V = V; fa.k = k;
    fa.lse_a = res[0][0]; fa.lq = res[0][1]; fa.idx_a = (const int32_t*)res[0][2]; fa.val_a = res[0][3];
    fa.lse_p = res[1][0]; fa.lp = res[1][1]; fa.idx_p = (const int32_t*)res[1][2]; fa.val_p = res[1][3];
    fa.rec = c->rec; fa.sc = c->sc;
    e = launch_fused_records(fa, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "fused records launch");
    c->launches += 5;
  }
  EpilogueArgs ea = epilogue_args(c, d, T, k, seed, d->token_offset, d->c1, out_accept, out_weight, out_lq, out_lp,
                                  out_stats);
  int nl = 0;
  if (budget) {
    e = launch_budget_solve(ea, (double)lambda_or_budget, c->stream, &nl);
    if (e != cudaSuccess) return cuda_fail(c, e, "budget solve launch");
  }
  e = launch_epilogue(ea, c->stream, &nl);
  c->launches += nl;
  if (e != cudaSuccess) return cuda_fail(c, e, "epilogue launch");
  c->have_records = true;
  c->rec_rows = T; c->rec_V = V; c->rec_k = k; c->rec_dtype = JP_BF16;
  return JP_OK;
}

jp_status jp_batch_begin(jp_ctx* c, int64_t T_total, int64_t V, int32_t dtype, int k,
                         float fixed_lambda_for_exact_mode) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (T_total < 0) return fail(c, JP_ERR_INVALID_ARG, "T_total < 0");
  if (V < 1) return fail(c, JP_ERR_INVALID_ARG, "V < 1");
  if (dtype != JP_BF16 && dtype != JP_F32) return fail(c, JP_ERR_INVALID_ARG, "unknown dtype");
  jp_status st = check_k(c, k, V);
  if (st != JP_OK) return st;
  const bool exact = (int64_t)k >= V;
  if (exact && !(fixed_lambda_for_exact_mode > 0.f))
    return fail(c, JP_ERR_UNSUPPORTED, "exact mode (k >= V) in a chunked batch needs a fixed lambda > 0 at begin");
  cudaSetDevice(c->device);
  const int k_eff = exact ? 0 : k;
  if ((st = ensure_workspace(c, T_total > 0 ? T_total : 1, k_eff)) != JP_OK) return st;
  cudaError_t e = launch_reset(c->sc, exact ? fixed_lambda_for_exact_mode : 1.0f, c->stream);
  if (e == cudaSuccess) e = launch_clear_flags(c->rec.flag, T_total, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "batch begin launch");
  c->launches += 2;
  c->batch_open = true;
  c->batch_exact = exact;
  c->have_records = false;
  c->rec_kl = T_total > 0;       // stays true only if every chunk asks for the divergence
  c->rec_sparse = false;
  c->rec_rows = T_total; c->rec_V = V; c->rec_k = k_eff; c->rec_dtype = dtype;
  return JP_OK;
}

jp_status jp_batch_chunk(jp_ctx* c, const jp_obrs_desc* d, const void* za, const void* zp,
                         const int32_t* tokens, const uint8_t* mask) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!c->batch_open) return fail(c, JP_ERR_STATE, "jp_batch_chunk without jp_batch_begin");
  int64_t ld = 0;
  jp_status st = check_shape(c, d, &ld);
  if (st != JP_OK) return st;
  if (d->V != c->rec_V || d->dtype != c->rec_dtype) return fail(c, JP_ERR_INVALID_ARG, "chunk V / dtype differ from jp_batch_begin");
  if (d->token_offset < 0 || d->token_offset + d->T > c->rec_rows)
    return fail(c, JP_ERR_INVALID_ARG, "chunk rows fall outside [0, T_total)");
  cudaSetDevice(c->device);
  // the row list restarts for every chunk; the other scalars accumulate
  cudaError_t e = cudaMemsetAsync(&c->sc->n_list, 0, 2 * sizeof(int32_t), c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemsetAsync");
  const bool want_kl = (d->flags & JP_DESC_KL) != 0;
  if (!want_kl && d->T > 0) c->rec_kl = false;
  if ((st = stream_rows(c, d, ld, c->rec_k, d->token_offset, za, zp, tokens, mask)) != JP_OK) return st;
  return extra_pass(c, d, ld, d->token_offset, za, zp, c->batch_exact ? c->rec.zk : nullptr, want_kl);
}

jp_status jp_batch_finalize(jp_ctx* c, const jp_obrs_desc* dout, float lambda_or_budget,
                            int32_t lambda_mode, uint64_t seed, uint8_t* out_accept,
                            float* out_weight, float* out_lq, float* out_lp, jp_stats* out_stats) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!c->batch_open) return fail(c, JP_ERR_STATE, "jp_batch_finalize without jp_batch_begin");
  jp_status st = check_lambda(c, lambda_or_budget, lambda_mode);
  if (st != JP_OK) return st;
  if (c->batch_exact && lambda_mode != JP_LAMBDA_FIXED)
    return fail(c, JP_ERR_UNSUPPORTED, "exact mode in a chunked batch supports a fixed lambda only");
  cudaSetDevice(c->device);
  float c1 = dout ? dout->c1 : 0.f;
  // record row 0 of this batch may sit at a global row index of its own (one shard of a larger batch)
  const int64_t rng_base = dout ? dout->token_offset : 0;
  EpilogueArgs ea = epilogue_args(c, dout, c->rec_rows, c->rec_k, seed, rng_base, c1, out_accept, out_weight,
                                  out_lq, out_lp, out_stats);
  ea.aux_zx = nullptr;
  int nl = 0;
  cudaError_t e;
  if (lambda_mode == JP_LAMBDA_FROM_BUDGET) {
    e = launch_budget_solve(ea, (double)lambda_or_budget, c->stream, &nl);
    if (e != cudaSuccess) return cuda_fail(c, e, "budget solve launch");
  } else if (!c->batch_exact) {
    e = cudaMemcpyAsync(&c->sc->lambda, &lambda_or_budget, sizeof(float), cudaMemcpyHostToDevice, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(lambda)");
  }
  e = launch_epilogue(ea, c->stream, &nl);
  c->launches += nl;
  if (e != cudaSuccess) return cuda_fail(c, e, "epilogue launch");
  c->batch_open = false;
  c->have_records = true;
  return JP_OK;
}

size_t jp_vshard_record_floats(int k) { return k < 1 ? 0 : (size_t)vshard_words(k); }

}  // extern "C"

namespace {
jp_status vshard_local_impl(jp_ctx* c, const jp_obrs_desc* d, const void* za, const void* zp, const int32_t* tokens,
                            const uint8_t* mask, int64_t vocab_offset, int64_t V_total, int k,
                            const VshardDests& dests, int64_t line0) {
  if (!c) return JP_ERR_INVALID_ARG;
  int64_t ld = 0;
  jp_status st = check_shape(c, d, &ld);
  if (st != JP_OK) return st;
  if (c->batch_open) return fail(c, JP_ERR_STATE, "a chunked batch is open: finalize it first");
  if (k < 1 || k > JP_MAX_TOPK) return fail(c, JP_ERR_UNSUPPORTED, "vocabulary shards support 1 <= k <= JP_MAX_TOPK (no exact mode)");
  if ((int64_t)k >= d->V) return fail(c, JP_ERR_UNSUPPORTED, "a vocabulary shard must be wider than k columns");
  if (vocab_offset < 0 || vocab_offset + d->V > V_total || V_total > (int64_t)0x7fffffff)
    return fail(c, JP_ERR_INVALID_ARG, "shard columns fall outside [0, V_total)");
  for (int p = 0; p < dests.n; ++p)
    if (d->T > 0 && !dests.dst[p]) return fail(c, JP_ERR_INVALID_ARG, "a destination of the packed records is NULL");
  cudaSetDevice(c->device);
  if ((st = ensure_workspace(c, d->T > 0 ? d->T : 1, k)) != JP_OK) return st;
  cudaError_t e = launch_reset(c->sc, 1.0f, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "reset launch");
  c->launches += 1;
  c->have_records = false;
  c->vshard_local_done = false;
  if (d->T > 0) {
    if (!tokens) return fail(c, JP_ERR_INVALID_ARG, "tokens pointer is NULL");
    e = launch_vshard_localize(d->T, tokens, mask, vocab_offset, d->V, V_total, 0, c->vtok, c->vmask, c->sc, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "shard token launch");
    c->launches += 1;
    if ((st = stream_rows(c, d, ld, k, 0, za, zp, c->vtok, c->vmask)) != JP_OK) return st;
    e = launch_vshard_export(d->T, k, c->rec, za, zp, ld, d->dtype, c->vtok, c->vmask, vocab_offset, dests, line0,
                             c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "shard export launch");
    c->launches += 1;
  }
  c->vshard_local_done = true;
  c->vshard_T = d->T;
  c->vshard_k = k;
  c->rec_dtype = d->dtype;
  return JP_OK;
}
}  // namespace

extern "C" {

jp_status jp_vshard_local(jp_ctx* c, const jp_obrs_desc* d, const void* za, const void* zp, const int32_t* tokens,
                          const uint8_t* mask, int64_t vocab_offset, int64_t V_total, int k, float* out_packed) {
  VshardDests dests{};
  dests.n = 1;
  dests.dst[0] = out_packed;
  return vshard_local_impl(c, d, za, zp, tokens, mask, vocab_offset, V_total, k, dests, 0);
}

jp_status jp_vshard_local_push(jp_ctx* c, const jp_obrs_desc* d, const void* za, const void* zp,
                               const int32_t* tokens, const uint8_t* mask, int64_t vocab_offset, int64_t V_total,
                               int k, int n_shards, int my_shard, float* const* gathered_of_shard) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!d) return fail(c, JP_ERR_INVALID_ARG, "desc is NULL");
  if (n_shards < 1 || n_shards > kVshardMaxDests) return fail(c, JP_ERR_TOO_LARGE, "at most 16 shards can be pushed to");
  if (my_shard < 0 || my_shard >= n_shards) return fail(c, JP_ERR_INVALID_ARG, "shard index out of range");
  if (!gathered_of_shard) return fail(c, JP_ERR_INVALID_ARG, "gathered_of_shard is NULL");
  VshardDests dests{};
  dests.n = n_shards;
  for (int p = 0; p < n_shards; ++p) dests.dst[p] = gathered_of_shard[p];
  return vshard_local_impl(c, d, za, zp, tokens, mask, vocab_offset, V_total, k, dests, (int64_t)my_shard * d->T);
}

jp_status jp_vshard_merge(jp_ctx* c, int n_shards, int my_shard, const float* gathered, int64_t T, int64_t V_total,
                          int k) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!c->vshard_local_done) return fail(c, JP_ERR_STATE, "jp_vshard_merge without jp_vshard_local");
  if (T != c->vshard_T || k != c->vshard_k) return fail(c, JP_ERR_INVALID_ARG, "T / k differ from jp_vshard_local");
  if (n_shards < 1 || my_shard < 0 || my_shard >= n_shards) return fail(c, JP_ERR_INVALID_ARG, "shard index out of range");
  if (n_shards > kVshardMaxShards) return fail(c, JP_ERR_TOO_LARGE, "the merge takes at most 128 shards");
  if ((int64_t)n_shards * k > kVshardMaxEntries)
    return fail(c, JP_ERR_TOO_LARGE, "n_shards * k beyond the 4096 entries per list the merge holds in shared memory");
  if (T > 0 && !gathered) return fail(c, JP_ERR_INVALID_ARG, "gathered is NULL");
  cudaSetDevice(c->device);
  cudaError_t e = launch_vshard_merge(n_shards, my_shard, gathered, T, k, c->rec, c->sc, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "shard merge launch");
  if (T > 0) c->launches += 1;
  // the records now describe the whole vocabulary: jp_batch_finalize completes the forward
  c->vshard_local_done = false;
  c->batch_open = true;
  c->batch_exact = false;
  c->rec_kl = false;             // the divergence needs whole rows
  c->rec_sparse = false;
  c->rec_rows = T; c->rec_V = V_total; c->rec_k = k;
  return JP_OK;
}

jp_status jp_obrs_row_lambda(jp_ctx* c, const jp_obrs_desc* d, const void* za, const void* zp, const uint8_t* mask,
                             float budget, float* out_lambda, float* out_kl_before, float* out_kl_after,
                             int32_t* out_iterations) {
  if (!c) return JP_ERR_INVALID_ARG;
  int64_t ld = 0;
  jp_status st = check_shape(c, d, &ld);
  if (st != JP_OK) return st;
  if (!(budget > 0.f) || budget > 1.f) return fail(c, JP_ERR_INVALID_ARG, "budget must lie in (0, 1]");
  if (d->T == 0) return JP_OK;
  if (!za || !zp || !out_lambda) return fail(c, JP_ERR_INVALID_ARG, "a required pointer is NULL");
  if (!aligned16(za) || !aligned16(zp)) return fail(c, JP_ERR_ALIGNMENT, "logit base pointers must be 16-byte aligned");
  cudaSetDevice(c->device);
  st = ensure_workspace(c, c->cap_rows > 0 ? c->cap_rows : 1, c->cap_k > 0 ? c->cap_k : 1);   // for the scalars
  if (st != JP_OK) return st;
  cudaError_t e = cudaMemsetAsync(&c->sc->row_counter2, 0, sizeof(int32_t), c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemsetAsync");
  RowLambdaArgs a{};
  a.za = za; a.zp = zp; a.mask = mask; a.T = d->T; a.V = d->V; a.ld = ld; a.dtype = d->dtype; a.budget = budget;
  a.sc = c->sc; a.out_lambda = out_lambda; a.out_kl_before = out_kl_before; a.out_kl_after = out_kl_after;
  a.out_iters = out_iterations;
  e = launch_row_lambda(a, c->stream, c->sms);
  if (e != cudaSuccess) return cuda_fail(c, e, "row lambda kernel launch");
  c->launches += 1;
  return JP_OK;
}

jp_status jp_batch_logprobs(jp_ctx* c, float* out_logp_actor, float* out_logp_policy, uint8_t* out_valid) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!c->batch_open) return fail(c, JP_ERR_STATE, "jp_batch_logprobs outside jp_batch_begin .. jp_batch_finalize");
  cudaSetDevice(c->device);
  cudaError_t e = launch_logprobs(c->rec_rows, c->rec, out_logp_actor, out_logp_policy, out_valid, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "log-prob copy launch");
  if (c->rec_rows > 0) c->launches += 1;
  return JP_OK;
}

jp_status jp_selftest_bounded_wait(jp_ctx* c, int64_t limit_cycles, int32_t* out_status) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (limit_cycles < 1 || limit_cycles > 2000000000ll) return fail(c, JP_ERR_INVALID_ARG, "limit_cycles must lie in [1, 2e9] (about a second at most)");
  if (!out_status) return fail(c, JP_ERR_INVALID_ARG, "out_status is NULL");
  cudaSetDevice(c->device);
  cudaError_t e = cudaMemsetAsync(out_status, 0, sizeof(int32_t), c->stream);
  if (e == cudaSuccess) e = launch_wait_selftest((long long)limit_cycles, out_status, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "self-test launch");
  c->launches += 1;
  return JP_OK;
}

jp_status jp_obrs_apply_kappa(jp_ctx* c, double kappa, float c1, float* out_weight) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!c->have_records) return fail(c, JP_ERR_STATE, "no forward records in this context: run the forward (or finalize the batch) first");
  if (!(kappa >= 0.0) || !(kappa < 1e300)) return fail(c, JP_ERR_INVALID_ARG, "kappa must be finite and >= 0");
  if (!out_weight && c->rec_rows > 0) return fail(c, JP_ERR_INVALID_ARG, "out_weight is NULL");
  cudaSetDevice(c->device);
  cudaError_t e = launch_reweight(c->rec_rows, c->rec, c->sc, kappa, c1, out_weight, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "reweight launch");
  if (c->rec_rows > 0) c->launches += 1;
  return JP_OK;
}

jp_status jp_batch_totals(jp_ctx* c, double* out_totals) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!c->have_records) return fail(c, JP_ERR_STATE, "no forward records in this context: run the forward (or finalize the batch) first");
  if (!out_totals) return fail(c, JP_ERR_INVALID_ARG, "out_totals is NULL");
  cudaSetDevice(c->device);
  cudaError_t e = cudaMemcpyAsync(out_totals, c->sc->totals, 4 * sizeof(double), cudaMemcpyDeviceToDevice, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(totals)");
  return JP_OK;
}

jp_status jp_obrs_apply_totals(jp_ctx* c, const double* totals, float c1, float* out_weight, jp_stats* out_stats) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (!c->have_records) return fail(c, JP_ERR_STATE, "no forward records in this context: run the forward (or finalize the batch) first");
  if (!totals) return fail(c, JP_ERR_INVALID_ARG, "totals is NULL");
  if (!out_weight && c->rec_rows > 0) return fail(c, JP_ERR_INVALID_ARG, "out_weight is NULL");
  cudaSetDevice(c->device);
  cudaError_t e = launch_reweight_totals(c->rec_rows, c->rec, c->sc, totals, c1, out_weight, out_stats, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "reweight launch");
  c->launches += 1;
  return JP_OK;
}

}  // extern "C"

namespace {
// slice_offset < 0: the rows are whole; otherwise they are the columns [slice_offset, slice_offset + V)
// of rows whose records describe rec_V columns.
jp_status backward_impl(jp_ctx* c, const jp_obrs_desc* d, const jp_obrs_bwd_desc* b,
                        const void* za, const void* zp, const int32_t* tokens,
                        const uint8_t* mask, const uint8_t* accept, const float* weight,
                        void* d_actor, void* d_policy, int64_t slice_offset) {
  if (!c) return JP_ERR_INVALID_ARG;
  int64_t ld = 0;
  jp_status st = check_shape(c, d, &ld);
  if (st != JP_OK) return st;
  if (!b) return fail(c, JP_ERR_INVALID_ARG, "bwd desc is NULL");
  if (!c->have_records) return fail(c, JP_ERR_STATE, "no forward records in this context: run the forward (or finalize the batch) first");
  if (c->rec_sparse) return fail(c, JP_ERR_STATE, "the records come from a forward without both logit tensors (sparse-actor or fused output layer): the gradients need the logits (run jp_obrs_forward)");
  const bool slice = slice_offset >= 0;
  if (!slice && (d->V != c->rec_V || d->dtype != c->rec_dtype)) return fail(c, JP_ERR_STATE, "V / dtype differ from the forward that left the records");
  if (slice && d->dtype != c->rec_dtype) return fail(c, JP_ERR_STATE, "dtype differs from the forward that left the records");
  if (slice && slice_offset + d->V > c->rec_V) return fail(c, JP_ERR_INVALID_ARG, "slice columns fall outside the vocabulary of the records");
  if (slice && (b->out_kl || b->out_loss)) return fail(c, JP_ERR_UNSUPPORTED, "the per-row KL and the loss value need whole rows");
  if (b->record_offset < 0 || b->record_offset + d->T > c->rec_rows)
    return fail(c, JP_ERR_INVALID_ARG, "rows fall outside the forward's records");
  if (b->lambda_distill < 0.f) return fail(c, JP_ERR_INVALID_ARG, "lambda_distill < 0");
  if (b->eps_lo < 0.f || b->eps_hi < 0.f || b->eps_lo >= 1.f) return fail(c, JP_ERR_INVALID_ARG, "clip range: need 0 <= eps_lo < 1 and eps_hi >= 0");
  if (b->out_loss && (!b->out_obj_policy || !b->out_obj_actor || !b->out_kl))
    return fail(c, JP_ERR_INVALID_ARG, "out_loss needs out_obj_policy, out_obj_actor and out_kl");
  if (d->T == 0) return JP_OK;
  if (!za || !zp || !tokens || !accept || !weight || !d_actor || !d_policy)
    return fail(c, JP_ERR_INVALID_ARG, "a required pointer is NULL");
  if (!aligned16(za) || !aligned16(zp) || !aligned16(d_actor) || !aligned16(d_policy))
    return fail(c, JP_ERR_ALIGNMENT, "logit and gradient base pointers must be 16-byte aligned");
  if ((ld * 2) % 16 != 0) return fail(c, JP_ERR_ALIGNMENT, "gradient row pitch (ld * 2 bytes) must be a multiple of 16 bytes");
  if (d->dtype == JP_F32 && (d_actor == za || d_policy == zp))
    return fail(c, JP_ERR_UNSUPPORTED, "in-place gradients need bf16 logits");
  cudaSetDevice(c->device);
  cudaError_t e = cudaMemsetAsync(&c->sc->row_counter2, 0, sizeof(int32_t), c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemsetAsync");
  if (slice) {
    e = launch_vshard_localize(d->T, tokens, mask, slice_offset, d->V, c->rec_V, -1, c->vtok, nullptr, nullptr, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "slice token launch");
    c->launches += 1;
    tokens = c->vtok;
  }
  GradArgs g{};
  g.za = za; g.zp = zp; g.tokens = tokens; g.mask = mask; g.accept = accept; g.weight = weight;
  g.adv = b->advantages; g.d_actor = d_actor; g.d_policy = d_policy;
  g.T = d->T; g.V = d->V; g.ld = ld; g.dtype = d->dtype; g.record_offset = b->record_offset;
  g.lambda_distill = b->lambda_distill; g.grad_out = b->grad_out == 0.f ? 1.f : b->grad_out;
  g.n_valid = b->n_valid; g.rec = c->rec; g.sc = c->sc;
  g.logp_ref = b->logp_ref; g.logp_actor_ref = b->logp_actor_ref; g.logp_inf = b->logp_inf;
  g.clip = (b->eps_lo > 0.f || b->eps_hi > 0.f) ? 1 : 0;
  g.eps_lo = b->eps_lo; g.eps_hi = b->eps_hi; g.c2 = b->c2; g.tis_cap = b->tis_cap;
  g.out_obj_policy = b->out_obj_policy; g.out_obj_actor = b->out_obj_actor; g.out_kl = b->out_kl;
  g.out_loss = b->out_loss;
  int n_launch = 0;
  e = launch_grad(g, c->stream, c->sms, &n_launch);
  if (e != cudaSuccess) return cuda_fail(c, e, "gradient kernel launch");
  c->launches += n_launch;
  return JP_OK;
}
}  // namespace

extern "C" {

jp_status jp_obrs_backward(jp_ctx* c, const jp_obrs_desc* d, const jp_obrs_bwd_desc* b,
                           const void* za, const void* zp, const int32_t* tokens,
                           const uint8_t* mask, const uint8_t* accept, const float* weight,
                           void* d_actor, void* d_policy) {
  return backward_impl(c, d, b, za, zp, tokens, mask, accept, weight, d_actor, d_policy, -1);
}

jp_status jp_vshard_backward(jp_ctx* c, const jp_obrs_desc* d, const jp_obrs_bwd_desc* b,
                             const void* za, const void* zp, const int32_t* tokens,
                             const uint8_t* mask, int64_t vocab_offset, const uint8_t* accept,
                             const float* weight, void* d_actor, void* d_policy) {
  if (!c) return JP_ERR_INVALID_ARG;
  if (vocab_offset < 0) return fail(c, JP_ERR_INVALID_ARG, "vocab_offset < 0");
  return backward_impl(c, d, b, za, zp, tokens, mask, accept, weight, d_actor, d_policy, vocab_offset);
}

jp_status jp_obrs_forward_host(jp_ctx* c, const jp_obrs_desc* d, const void* za, const void* zp,
                               const int32_t* tokens, const uint8_t* mask, float lambda_or_budget,
                               int k, uint64_t seed, uint8_t* out_accept, float* out_weight,
                               float* out_lq, float* out_lp, jp_stats* out_stats, int64_t chunk_rows) {
  if (!c) return JP_ERR_INVALID_ARG;
  int64_t ld = 0;
  jp_status st = check_shape(c, d, &ld);
  if (st != JP_OK) return st;
  if ((st = check_k(c, k, d->V)) != JP_OK) return st;
  if ((st = check_lambda(c, lambda_or_budget, d->lambda_mode)) != JP_OK) return st;
  if (d->topk_idx_actor || d->topk_idx_policy || d->topk_val_actor || d->topk_val_policy ||
      d->accept_prob || d->uniform || d->z_approx || d->z_exact || d->lse_actor || d->lse_policy)
    return fail(c, JP_ERR_UNSUPPORTED, "optional outputs are not supported with host buffers");
  const bool exact = (int64_t)k >= d->V;
  if (exact && d->lambda_mode != JP_LAMBDA_FIXED)
    return fail(c, JP_ERR_UNSUPPORTED, "exact mode with host buffers supports a fixed lambda only");
  if (d->T > 0 && (!za || !zp || !tokens)) return fail(c, JP_ERR_INVALID_ARG, "logits or tokens pointer is NULL");
  cudaSetDevice(c->device);
  const int es = d->dtype == JP_BF16 ? 2 : 4;
  const size_t row_bytes = (size_t)ld * es;
  if (chunk_rows <= 0) {
    chunk_rows = (int64_t)((size_t)256 << 20) / (int64_t)row_bytes;   // ~256 MiB per tensor per slot
    if (chunk_rows < 1) chunk_rows = 1;
  }
  if (chunk_rows > d->T) chunk_rows = d->T > 0 ? d->T : 1;
  // staging: 2 slots x (za, zp, tokens, mask) + outputs for all T rows
  const size_t slot_logits = align_up((size_t)chunk_rows * row_bytes, 256);
  const size_t slot_tok = align_up((size_t)chunk_rows * 4, 256);
  const size_t slot_mask = align_up((size_t)chunk_rows, 256);
  const size_t slot = 2 * slot_logits + slot_tok + slot_mask;
  const size_t Tn = (size_t)(d->T > 0 ? d->T : 1);
  const size_t out_bytes = align_up(Tn, 256) + 3 * align_up(Tn * 4, 256) + align_up(sizeof(jp_stats), 256);
  const size_t need = 2 * slot + out_bytes;
  cudaError_t e;
  if (need > c->stage_bytes) {
    cudaStreamSynchronize(c->stream);
    if (c->stage) cudaFree(c->stage);
  if (c->lm_scratch) cudaFree(c->lm_scratch);
    c->stage = nullptr; c->stage_bytes = 0;
    e = cudaMalloc((void**)&c->stage, need);
    if (e != cudaSuccess) return fail(c, JP_ERR_WORKSPACE, std::string("staging cudaMalloc: ") + cudaGetErrorString(e));
    c->stage_bytes = need;
  }
  if (!c->copy_stream) {
    e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamCreate");
    for (int i = 0; i < 2; ++i) {
      cudaEventCreateWithFlags(&c->copy_done[i], cudaEventDisableTiming);
      cudaEventCreateWithFlags(&c->compute_done[i], cudaEventDisableTiming);
    }
  }
  char* outs = c->stage + 2 * slot;
  uint8_t* d_acc = (uint8_t*)outs;
  float* d_w = (float*)(outs + align_up(Tn, 256));
  float* d_lq = (float*)((char*)d_w + align_up(Tn * 4, 256));
  float* d_lp = (float*)((char*)d_lq + align_up(Tn * 4, 256));
  jp_stats* d_stats = (jp_stats*)((char*)d_lp + align_up(Tn * 4, 256));

  st = jp_batch_begin(c, d->T, d->V, d->dtype, k, exact ? lambda_or_budget : 0.f);
  if (st != JP_OK) return st;
  // order the copy stream after whatever the compute stream did before
  cudaEventRecord(c->compute_done[0], c->stream);
  cudaEventRecord(c->compute_done[1], c->stream);
  int64_t n_chunks = (d->T + chunk_rows - 1) / chunk_rows;
  for (int64_t ci = 0; ci < n_chunks; ++ci) {
    const int s = (int)(ci & 1);
    const int64_t r0 = ci * chunk_rows;
    const int64_t rows = (d->T - r0) < chunk_rows ? (d->T - r0) : chunk_rows;
    char* base = c->stage + (size_t)s * slot;
    char* s_za = base;
    char* s_zp = base + slot_logits;
    int32_t* s_tok = (int32_t*)(base + 2 * slot_logits);
    uint8_t* s_mask = (uint8_t*)(base + 2 * slot_logits + slot_tok);
    cudaStreamWaitEvent(c->copy_stream, c->compute_done[s], 0);   // slot free again
    e = cudaMemcpyAsync(s_za, (const char*)za + (size_t)r0 * row_bytes, (size_t)rows * row_bytes, cudaMemcpyHostToDevice, c->copy_stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(s_zp, (const char*)zp + (size_t)r0 * row_bytes, (size_t)rows * row_bytes, cudaMemcpyHostToDevice, c->copy_stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(s_tok, tokens + r0, (size_t)rows * 4, cudaMemcpyHostToDevice, c->copy_stream);
    if (e == cudaSuccess && mask) e = cudaMemcpyAsync(s_mask, mask + r0, (size_t)rows, cudaMemcpyHostToDevice, c->copy_stream);
    if (e != cudaSuccess) { c->batch_open = false; return cuda_fail(c, e, "host-to-device copy"); }
    cudaEventRecord(c->copy_done[s], c->copy_stream);
    cudaStreamWaitEvent(c->stream, c->copy_done[s], 0);
    jp_obrs_desc cd = *d;
    cd.T = rows; cd.token_offset = r0;
    st = jp_batch_chunk(c, &cd, s_za, s_zp, s_tok, mask ? s_mask : nullptr);
    if (st != JP_OK) { c->batch_open = false; return st; }
    cudaEventRecord(c->compute_done[s], c->stream);
  }
  jp_obrs_desc fd = *d;
  st = jp_batch_finalize(c, &fd, lambda_or_budget, d->lambda_mode, seed, d_acc, d_w, d_lq, d_lp, d_stats);
  if (st != JP_OK) { c->batch_open = false; return st; }
  if (out_accept) cudaMemcpyAsync(out_accept, d_acc, (size_t)d->T, cudaMemcpyDeviceToHost, c->stream);
  if (out_weight) cudaMemcpyAsync(out_weight, d_w, (size_t)d->T * 4, cudaMemcpyDeviceToHost, c->stream);
  if (out_lq) cudaMemcpyAsync(out_lq, d_lq, (size_t)d->T * 4, cudaMemcpyDeviceToHost, c->stream);
  if (out_lp) cudaMemcpyAsync(out_lp, d_lp, (size_t)d->T * 4, cudaMemcpyDeviceToHost, c->stream);
  if (out_stats) cudaMemcpyAsync(out_stats, d_stats, sizeof(jp_stats), cudaMemcpyDeviceToHost, c->stream);
  e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamSynchronize");
  return JP_OK;
}

}  // extern "C"
