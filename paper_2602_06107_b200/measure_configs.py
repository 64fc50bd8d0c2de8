"""Times the workload shapes other than the headline one at their full sizes on one GPU:

  cfg3_batch  64 padded responses (131,072 rows, ~56 % valid) streamed in 16 chunks, lambda
              from an acceptance budget, k = 64;
  cfg4_sweep  16,384 rows at three actor/policy mismatches and k in {8, 32, 128, V}: Z_approx
              against the exact Z, and throughput per point;
  cfg5_train  32,768 rows in 4 chunks: chunked forward with a budget, then one fused backward
              per chunk.

Only the library calls are timed (CUDA events on the context's stream); input generation is
outside the timed regions.  One JSON line per measurement.

  row_lambda  the per-distribution budget of Theorem 3.4 on the headline shape (4096 rows);
  simulation  Dirichlet pairs at growing distance: acceptance rate and divergence before / after
              rejection (not run by default);
  vocab_shards  the headline batch split by columns over 2, 4 and 8 shards: one shard's local pass,
              the merge of all shards' records and the finalize, timed apart (not run by default).

    python -m paper_2602_06107_b200.measure_configs [cfg3_batch] [cfg4_sweep] [cfg5_train] [row_lambda] [simulation] [vocab_shards]
"""
from __future__ import annotations

import json
import sys

import torch

from . import binding as B
from . import build as jp_build
from . import runner
from .inputs import CONFIGS, LogitRecipe, make_lengths_mask, make_logits

DEV = "cuda:0"


def _recipe(r0: LogitRecipe, T: int, seed: int, sigma=None) -> LogitRecipe:
    return LogitRecipe(T=T, V=r0.V, dtype=r0.dtype, sigma0=r0.sigma0, peaks=r0.peaks, peak_lo=r0.peak_lo,
                       peak_hi=r0.peak_hi, sigma=r0.sigma if sigma is None else sigma, seed=seed)


class _Timer:
    """Sums the device time of the regions it brackets (events on the current stream,
    which is the stream the context was created on)."""

    def __init__(self):
        self.pairs = []

    def __enter__(self):
        self.e0 = torch.cuda.Event(enable_timing=True)
        self.e1 = torch.cuda.Event(enable_timing=True)
        self.e0.record()
        return self

    def __exit__(self, *a):
        self.e1.record()
        self.pairs.append((self.e0, self.e1))

    def ms(self) -> float:
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in self.pairs)


def _emit(**kw):
    print(json.dumps(kw), flush=True)


def cfg3_batch(ctx):
    cfg = CONFIGS["cfg3_batch"]
    r0, chunk = cfg["recipe"], cfg["chunk"]
    T, V, k = r0.T, r0.V, cfg["k"]
    mask, _ = make_lengths_mask(cfg["n_resp"], cfg["max_len"], cfg["min_len"], seed=cfg["seed"], device=DEV)
    n_valid = int(mask.sum().item())
    B.jp_reserve(ctx, T, V, k)
    out = runner._alloc_outputs(T, DEV)
    for rep in range(2):                      # the first pass warms up
        t = _Timer()
        B.jp_batch_begin(ctx, T, V, B.JP_BF16, k, 0.0)
        for c, off in enumerate(range(0, T, chunk)):
            za, zp, tok = make_logits(_recipe(r0, chunk, r0.seed + 17 * c), DEV)
            d = B.make_desc(za, token_offset=off)
            with t:
                B.jp_batch_chunk(ctx, d, za, zp, tok, mask[off:off + chunk])
            torch.cuda.synchronize()
            del za, zp, tok
        d = B.jp_obrs_desc()
        with t:
            B.jp_batch_finalize(ctx, d, cfg["budget"], B.JP_LAMBDA_FROM_BUDGET, cfg["seed"], out["accept"],
                                out["weight"], out["logp_actor"], out["logp_policy"], out["stats_buf"])
        ms = t.ms()
    st = B.read_stats(out["stats_buf"])
    gb = 2.0 * n_valid * V * 2 / 1e9
    _emit(workload="cfg3_batch", rows=T, valid=n_valid, k=k, budget=cfg["budget"], ms=ms,
          valid_tokens_per_s=n_valid / (ms * 1e-3), padded_rows_per_s=T / (ms * 1e-3), algorithmic_gb=gb,
          gb_per_s=gb / (ms * 1e-3), lambda_used=st["lambda_used"], alpha_hat=st["alpha_hat"],
          mean_accept_prob=st["mean_accept_prob"], kappa=st["kappa"], status=st["status"])


def cfg4_sweep(ctx):
    cfg = CONFIGS["cfg4_sweep"]
    r0 = cfg["recipe"]
    T, V, lam = r0.T, r0.V, cfg["lam"]
    B.jp_reserve(ctx, T, V, 128)
    for si, sigma in enumerate(cfg["sigmas"]):
        za, zp, tok = make_logits(_recipe(r0, T, r0.seed + si, sigma=sigma), DEV)
        exact = runner.forward(ctx, za, zp, tok, None, lam=lam, k=V, seed=cfg["seed"])
        zx = exact["z_approx"].double()
        for k in cfg["ks"]:
            out = runner._alloc_outputs(T, DEV)
            desc = B.make_desc(za)
            zk = torch.empty(T, dtype=torch.float32, device=DEV)
            desc.z_approx = zk.data_ptr()

            def fwd():
                B.jp_obrs_forward(ctx, desc, za, zp, tok, None, lam, k, cfg["seed"], out["accept"], out["weight"],
                                  out["logp_actor"], out["logp_policy"], out["stats_buf"])

            for _ in range(3):
                fwd()
            t = _Timer()
            reps = 20
            with t:
                for _ in range(reps):
                    fwd()
            ms = t.ms() / reps
            st = B.read_stats(out["stats_buf"])
            passes = 2 if k >= V else 1            # exact mode reads the rows a second time
            gb = passes * 2.0 * T * V * 2 / 1e9
            _emit(workload="cfg4_sweep", rows=T, sigma=sigma, k=int(k), ms=ms, tokens_per_s=T / (ms * 1e-3),
                  algorithmic_gb=gb, gb_per_s=gb / (ms * 1e-3),
                  mean_abs_zk_over_z_minus_1=float(((zk.double() / zx) - 1.0).abs().mean().item()),
                  kappa=st["kappa"], alpha_hat=st["alpha_hat"], status=st["status"])
        del za, zp, tok


def cfg5_train(ctx):
    cfg = CONFIGS["cfg5_train"]
    r0, chunk, k = cfg["recipe"], cfg["chunk"], cfg["k"]
    T, V = r0.T, r0.V
    B.jp_reserve(ctx, T, V, k)
    parts = [make_logits(_recipe(r0, chunk, r0.seed + 31 * c), DEV) for c in range(T // chunk)]
    grads = [(torch.empty_like(za), torch.empty_like(zp)) for za, zp, _ in parts]
    g = torch.Generator(device="cpu").manual_seed(cfg["seed"])
    adv = torch.randn(T // chunk, generator=g).repeat_interleave(chunk).to(DEV)   # one draw per response
    out = runner._alloc_outputs(T, DEV)
    for rep in range(3):                      # the first passes warm up
        tf, tb = _Timer(), _Timer()
        with tf:
            B.jp_batch_begin(ctx, T, V, B.JP_BF16, k, 0.0)
            for c, (za, zp, tok) in enumerate(parts):
                B.jp_batch_chunk(ctx, B.make_desc(za, token_offset=c * chunk), za, zp, tok, None)
            d = B.jp_obrs_desc()
            d.c1 = cfg["c1"]
            B.jp_batch_finalize(ctx, d, cfg["budget"], B.JP_LAMBDA_FROM_BUDGET, cfg["seed"], out["accept"],
                                out["weight"], out["logp_actor"], out["logp_policy"], out["stats_buf"])
        with tb:
            for c, (za, zp, tok) in enumerate(parts):
                sl = slice(c * chunk, (c + 1) * chunk)
                runner.backward(ctx, za, zp, tok, None, out["accept"][sl], out["weight"][sl], advantages=adv[sl],
                                lambda_distill=cfg["lambda_distill"], record_offset=c * chunk, d_actor=grads[c][0],
                                d_policy=grads[c][1])
        ms_f, ms_b = tf.ms(), tb.ms()
    st = B.read_stats(out["stats_buf"])
    gb_f, gb_b = 2.0 * T * V * 2 / 1e9, 4.0 * T * V * 2 / 1e9
    _emit(workload="cfg5_train", rows=T, k=k, budget=cfg["budget"], forward_ms=ms_f, backward_ms=ms_b,
          fwd_bwd_tokens_per_s=T / ((ms_f + ms_b) * 1e-3), forward_gb_per_s=gb_f / (ms_f * 1e-3),
          backward_gb_per_s=gb_b / (ms_b * 1e-3), lambda_used=st["lambda_used"], alpha_hat=st["alpha_hat"],
          kappa=st["kappa"], status=st["status"])


def row_lambda(ctx):
    """Theorem 3.4 per distribution on the headline shape: the lambda of every row for a budget,
    with KL(p||q) before and KL(p||kept) after (the quantities of the paper's simulation figure)."""
    cfg = CONFIGS["cfg2_qwen3"]
    za, zp, _ = make_logits(cfg["recipe"], DEV)
    T, V = za.shape
    lam = torch.empty(T, device=DEV)
    kb, ka = torch.empty(T, device=DEV), torch.empty(T, device=DEV)
    it = torch.empty(T, dtype=torch.int32, device=DEV)
    d = B.make_desc(za)
    for budget in (0.5, 0.7, 0.9):
        for _ in range(2):
            B.jp_obrs_row_lambda(ctx, d, za, zp, None, budget, lam, kb, ka, it)
        t = _Timer()
        reps = 5
        with t:
            for _ in range(reps):
                B.jp_obrs_row_lambda(ctx, d, za, zp, None, budget, lam, kb, ka, it)
        ms = t.ms() / reps
        steps = it.float().mean().item()
        _emit(workload="row_lambda", rows=T, budget=budget, ms=ms, rows_per_s=T / (ms * 1e-3),
              mean_newton_steps=steps, max_newton_steps=int(it.max().item()),
              passes_over_the_rows=4.0 + steps, mean_lambda=lam.mean().item(), mean_kl_before=kb.mean().item(),
              mean_kl_after=ka.mean().item())


def simulation(ctx):
    """The paper's numerical simulation, qualitatively: Dirichlet pairs at growing distance; acceptance
    rate of OBRS at lambda = 1 (the exact normaliser Z) and the divergence to the target before and after
    rejection at an acceptance budget of 0.9."""
    from .inputs import make_dirichlet_logits
    T, V = 2048, 32768
    for noise in (0.1, 0.25, 0.5, 1.0, 1.5):
        za, zp, tok = make_dirichlet_logits(T, V, 0.3, noise, seed=7, device=DEV)
        ex = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=V, seed=1)
        kb, ka = torch.empty(T, device=DEV), torch.empty(T, device=DEV)
        lam = torch.empty(T, device=DEV)
        B.jp_obrs_row_lambda(ctx, B.make_desc(za), za, zp, None, 0.9, lam, kb, ka, None)
        torch.cuda.synchronize()
        _emit(workload="simulation", rows=T, V=V, noise=noise, mean_kl_p_q=kb.mean().item(),
              acceptance_at_lambda_1=ex["z_approx"].mean().item(),
              mean_kl_after_budget_0p9=ka.mean().item(), kl_reduction_factor=(kb.mean() / ka.mean()).item(),
              mean_lambda_for_budget_0p9=lam.mean().item())


def vocab_shards(ctx):
    """One rank's share of the vocabulary-parallel forward on the headline shape.  The shards run one
    after the other here (a rank has one of them); every phase of shard 0 is timed on its own."""
    from . import parallel
    cfg = CONFIGS["cfg2_qwen3"]
    za, zp, tok = make_logits(cfg["recipe"], DEV)
    T, V = za.shape
    k, lam = cfg["k"], cfg["lam"]
    words = B.jp_vshard_record_floats(k)
    for n in (2, 4, 8):
        bounds = [parallel.shard_columns(V, n, s) for s in range(n)]
        gathered = torch.empty((n, T, words), device=DEV)
        for s, (lo, hi) in enumerate(bounds):
            zs, ps = za[:, lo:hi], zp[:, lo:hi]
            B.jp_vshard_local(ctx, B.make_desc(zs), zs, ps, tok, None, lo, V, k, gathered[s])
        lo, hi = bounds[0]
        zs, ps = za[:, lo:hi], zp[:, lo:hi]
        d0 = B.make_desc(zs)
        out = runner._alloc_outputs(T, DEV)
        tl, tm, tf = _Timer(), _Timer(), _Timer()
        reps = 20
        for i in range(reps + 3):
            if i == 3:
                tl, tm, tf = _Timer(), _Timer(), _Timer()
            with tl:
                B.jp_vshard_local(ctx, d0, zs, ps, tok, None, lo, V, k, gathered[0])
            with tm:
                B.jp_vshard_merge(ctx, n, 0, gathered, T, V, k)
            with tf:
                B.jp_batch_finalize(ctx, B.jp_obrs_desc(), lam, B.JP_LAMBDA_FIXED, cfg["seed"], out["accept"],
                                    out["weight"], out["logp_actor"], out["logp_policy"], out["stats_buf"])
        ms_l, ms_m, ms_f = tl.ms() / reps, tm.ms() / reps, tf.ms() / reps
        st = B.read_stats(out["stats_buf"])
        gb = 2.0 * T * (hi - lo) * 2 / 1e9
        _emit(workload="vocab_shards", rows=T, shards=n, shard_columns=hi - lo, k=k, local_ms=ms_l,
              local_gb_per_s=gb / (ms_l * 1e-3), merge_ms=ms_m, finalize_ms=ms_f,
              all_gather_bytes_per_rank=T * words * 4, rank_total_ms=ms_l + ms_m + ms_f,
              tokens_per_s=T / ((ms_l + ms_m + ms_f) * 1e-3), n_accept=st["n_accept"], kappa=st["kappa"],
              status=st["status"])


def main(argv):
    assert torch.cuda.is_available(), "needs a CUDA device"
    jp_build.build()
    torch.cuda.set_device(0)
    which = [a for a in argv if not a.startswith("-")] or ["cfg3_batch", "cfg4_sweep", "cfg5_train", "row_lambda"]
    ctx = B.Context(0)
    for name in which:
        {"cfg3_batch": cfg3_batch, "cfg4_sweep": cfg4_sweep, "cfg5_train": cfg5_train, "row_lambda": row_lambda, "simulation": simulation,
         "vocab_shards": vocab_shards}[name](ctx)
        torch.cuda.empty_cache()
    ctx.close()


if __name__ == "__main__":
    main(sys.argv[1:])
