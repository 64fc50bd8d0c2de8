"""GPU parity: libjackpot (through its C ABI) against the CPU oracle, element by
element on the same seeded inputs.

Bars (written here, as the task states them):
  * top-k indices, top-k logits, the uniforms and accept bits: bit-exact -- an
    accept bit may differ only on a token with |u - a| < 1e-6; such tokens are
    counted and reported;
  * log-sum-exps, log-probs, acceptance probabilities, Z_approx, exact Z, weights,
    kappa, lambda: rtol 1e-5 / atol 1e-6 against the oracle's double results.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200 import runner
from paper_2602_06107_b200.inputs import CONFIGS, LogitRecipe, make_logits, to_numpy_bits

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 1e-6


@pytest.fixture(scope="module")
def ctx():
    jp_build.build()
    c = B.Context(0)
    yield c
    c.close()


def close(a, b, rtol=RTOL, atol=ATOL):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    bad = np.abs(a - b) > atol + rtol * np.abs(b)
    assert not bad.any(), f"{bad.sum()} of {bad.size} differ; worst {np.abs(a - b).max():.3e} at {np.argmax(np.abs(a - b))}"


def check_forward(out, ref, k, V, mask=None, c1=0.0, exact_too=False):
    """out: runner.forward result (device tensors); ref: oracle.forward result."""
    T = ref["lq"].shape[0]
    valid = np.ones(T, bool) if mask is None else (mask != 0)
    valid &= ref["bad"] == 0
    g = {n: t.cpu().numpy() for n, t in out.items() if isinstance(t, torch.Tensor)}
    close(g["lse_actor"][valid], ref["lse_a"][valid])
    close(g["lse_policy"][valid], ref["lse_p"][valid])
    close(g["logp_actor"], ref["lq64"])
    close(g["logp_policy"], ref["lp64"])
    if k < V:
        assert np.array_equal(g["topk_idx_actor"][valid], ref["topk_idx_a"][valid])
        assert np.array_equal(g["topk_idx_policy"][valid], ref["topk_idx_p"][valid])
        assert np.all(g["topk_idx_actor"][~valid] == -1)
        # the published values are the rows' own logits at the published indices, widened exactly
        za_h, zp_h = ref.get("za_f32"), ref.get("zp_f32")
        if za_h is not None:
            rows = np.nonzero(valid)[0][:, None]
            assert np.array_equal(g["topk_val_actor"][valid], za_h[rows, ref["topk_idx_a"][valid]])
            assert np.array_equal(g["topk_val_policy"][valid], zp_h[rows, ref["topk_idx_p"][valid]])
    assert np.array_equal(g["uniform"], ref["u"])
    close(g["accept_prob"], ref["a"])
    diff = g["accept"] != ref["accept"]
    near = np.abs(ref["u"].astype(np.float64) - ref["a"].astype(np.float64)) < 1e-6
    assert not (diff & ~near).any(), "accept bits differ away from the threshold"
    n_flip = int(diff.sum())
    close(g["z_approx"], ref["zk"])
    if exact_too:
        close(g["z_exact"], ref["z_exact"])
    st, rs = out["stats"], ref["stats"]
    assert st["n_valid"] == rs["n_valid"] and st["n_bad_token"] == rs.get("n_bad_token", 0)
    assert st["n_accept"] == int(g["accept"].sum())
    close(st["lambda_used"], ref["lambda"])
    close(st["z_approx_mean"], rs["z_approx_mean"])
    close(st["mean_accept_prob"], rs["mean_accept_prob"])
    if st["n_valid"] > 0 and st["z_approx_mean"] > 0:
        close(st["kappa"] * st["z_approx_mean"], st["alpha_hat"])
    if n_flip == 0:
        assert st["n_accept"] == rs["n_accept"]
        close(st["kappa"], rs["kappa"])
        close(g["weight"], ref["w64"])
    elif c1 <= 0:
        close(g["weight"] / st["kappa"], ref["w64"] / rs["kappa"])
    assert np.all(g["weight"][~valid] == 0) and np.all(g["accept"][~valid] == 0)
    return n_flip


def run_case(ctx, za, zp, tok, mask=None, *, lam=None, budget=None, k, seed, c1=0.0, token_offset=0,
             exact_too=False):
    out = runner.forward(ctx, za, zp, tok, mask, lam=lam, budget=budget, k=k, seed=seed, c1=c1,
                         token_offset=token_offset, want_exact=exact_too)
    m = None if mask is None else mask.cpu().numpy()
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), m, lam=lam, budget=budget,
                         k=k, seed=seed, c1=c1, token_offset=token_offset, exact=exact_too)
    ref["za_f32"], ref["zp_f32"] = za.float().cpu().numpy(), zp.float().cpu().numpy()   # exact widening
    if budget is not None:
        # lambda parity first, then everything else with lambda forced to the oracle's value so
        # that a last-bit difference in lambda cannot leak into the accept bits
        close(out["stats"]["lambda_used"], ref["lambda"])
        out = runner.forward(ctx, za, zp, tok, mask, lam=ref["lambda"], k=k, seed=seed, c1=c1,
                             token_offset=token_offset, want_exact=exact_too)
    return check_forward(out, ref, k, za.shape[1], m, c1, exact_too), out, ref


def test_cfg1_tiny_exact(ctx):
    cfg = CONFIGS["cfg1_tiny"]
    za, zp, tok = make_logits(cfg["recipe"], "cuda")
    flips, out, ref = run_case(ctx, za, zp, tok, lam=cfg["lam"], k=cfg["k"], seed=cfg["seed"], exact_too=True)
    print("cfg1 near-threshold flips:", flips)
    # brute-force Z beside Z_approx: the estimate underestimates
    assert np.all(out["z_approx"].cpu().numpy() <= out["z_exact"].cpu().numpy() * (1 + 1e-5) + 1e-6)
    # k = V: exact mode through the same entry point
    V = za.shape[1]
    flips2, out2, ref2 = run_case(ctx, za, zp, tok, lam=cfg["lam"], k=V, seed=cfg["seed"])
    close(out2["z_approx"].cpu().numpy(), ref["z_exact"])


@pytest.mark.parametrize("k", [1, 8, 32, 128])
def test_qwen3_shape_small_T(ctx, k):
    r = LogitRecipe(T=48, V=151936, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0, peak_hi=15.0, sigma=1.0,
                    seed=100 + k)
    za, zp, tok = make_logits(r, "cuda")
    flips, _, _ = run_case(ctx, za, zp, tok, lam=2.0, k=k, seed=1, token_offset=12345)
    print("flips", flips)


def test_ragged_vocab_and_mask_bf16(ctx):
    V, ld, T = 5003, 5008, 300          # tail of 3 columns, padded pitch, several rows per CTA
    r = LogitRecipe(T=T, V=ld, dtype="bf16", sigma0=2.0, peaks=4, sigma=0.7, seed=7)
    za_full, zp_full, _ = make_logits(r, "cuda")
    za, zp = za_full[:, :V], zp_full[:, :V]
    g = torch.Generator(device="cuda").manual_seed(5)
    gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
    tok = (za.float() + gum).argmax(1).to(torch.int32)
    mask = (torch.arange(T, device="cuda") % 7 != 3).to(torch.uint8)
    za_c, zp_c = za.contiguous(), zp.contiguous()       # the oracle takes dense rows
    out = runner.forward(ctx, za, zp, tok, mask, lam=1.2, k=20, seed=3)
    ref = oracle.forward(to_numpy_bits(za_c), to_numpy_bits(zp_c), tok.cpu().numpy(), mask.cpu().numpy(),
                         lam=1.2, k=20, seed=3)
    check_forward(out, ref, 20, V, mask.cpu().numpy())


def test_ragged_vocab_f32(ctx):
    V, ld, T = 4099, 4100, 40
    r = LogitRecipe(T=T, V=ld, dtype="f32", sigma0=2.0, peaks=4, sigma=0.5, seed=8)
    za_full, zp_full, _ = make_logits(r, "cuda")
    za, zp = za_full[:, :V], zp_full[:, :V]
    tok = torch.randint(0, V, (T,), device="cuda", dtype=torch.int32)
    out = runner.forward(ctx, za, zp, tok, None, lam=0.8, k=16, seed=4)
    ref = oracle.forward(to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous()), tok.cpu().numpy(), None,
                         lam=0.8, k=16, seed=4)
    check_forward(out, ref, 16, V)


def test_adversarial_tie_rows(ctx):
    """all-equal rows, ramps, -inf entries, -0 vs +0, peaks at both ends, V barely above k."""
    V, k = 9000, 16
    rows = torch.zeros((8, V), dtype=torch.float32)
    rows[0, :] = 1.25
    rows[1, :] = torch.arange(V) * 0.001                  # ascending: every entry beats the list
    rows[2, :] = -torch.arange(V) * 0.001
    rows[3, [5, 4100, 8999]] = 2.0
    rows[4, :] = float("-inf")
    rows[4, [8999, 0, 17]] = torch.tensor([1.0, 1.0, 0.5])
    rows[5, 10::2] = -0.0
    rows[5, 3] = 1.0
    rows[6, :] = torch.randn(V).round()                   # massive ties
    rows[7, :] = torch.randn(V)
    for dt in (torch.bfloat16, torch.float32):
        za = rows.to(dt).cuda()
        zp = rows.flip(0).to(dt).cuda().contiguous()
        tok = torch.tensor([0, 8999, 0, 5, 0, 3, 1, 2], dtype=torch.int32, device="cuda")
        out = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=k, seed=0)
        ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), None, lam=1.0, k=k, seed=0)
        g_a, g_p = out["topk_idx_actor"].cpu().numpy(), out["topk_idx_policy"].cpu().numpy()
        assert np.array_equal(g_a, ref["topk_idx_a"]) and np.array_equal(g_p, ref["topk_idx_p"])
        assert g_a[0].tolist() == list(range(16))
        if dt == torch.float32:
            assert g_a[1].tolist() == list(range(V - 1, V - 17, -1))
        ok = np.isfinite(ref["lq64"]) & np.isfinite(ref["lp64"])
        close(out["logp_actor"].cpu().numpy()[ok], ref["lq64"][ok])
        close(out["z_approx"].cpu().numpy()[ok], ref["zk"][ok])


def test_rows_with_more_candidates_than_shared_memory_holds(ctx):
    """Rows built so that far more passes reach the running threshold than the CTA's
    buffer takes: a ramp over a fifth of the row (a few thousand candidates: they go
    to the workspace), a ramp over the whole row and a constant row (more than the
    workspace area takes as well: the row is read again), beside an ordinary row."""
    V = 151936
    for dt, k in ((torch.float32, 32), (torch.bfloat16, 64), (torch.float32, 128)):
        rows = torch.full((6, V), -5.0, dtype=torch.float32)
        n5 = V // 5
        rows[0, :n5] = torch.linspace(0.0, 8.0, n5)
        rows[1, :] = torch.linspace(-4.0, 9.0, V)
        rows[2, :] = 0.75
        rows[3, :] = torch.randn(V, generator=torch.Generator().manual_seed(5)) * 2.5
        rows[4, V - n5:] = torch.linspace(0.0, 8.0, n5)          # the ramp at the end of the row
        rows[5, :] = torch.linspace(9.0, -4.0, V)                # descending: the first passes win
        za = rows.to(dt).cuda()
        zp = rows.flip(0).to(dt).cuda().contiguous()
        tok = torch.tensor([7, V - 1, 100, 5, V - 3, 0], dtype=torch.int32, device="cuda")
        out = runner.forward(ctx, za, zp, tok, None, lam=1.5, k=k, seed=3)
        ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), None, lam=1.5, k=k, seed=3)
        assert out["stats"]["status"] == 0
        assert np.array_equal(out["topk_idx_actor"].cpu().numpy(), ref["topk_idx_a"])
        assert np.array_equal(out["topk_idx_policy"].cpu().numpy(), ref["topk_idx_p"])
        close(out["lse_actor"].cpu().numpy(), ref["lse_a"])
        close(out["lse_policy"].cpu().numpy(), ref["lse_p"])
        close(out["logp_actor"].cpu().numpy(), ref["lq64"])
        close(out["z_approx"].cpu().numpy(), ref["zk"])


def test_small_vocab_just_above_k(ctx):
    for V, k, dt in ((136, 128, "bf16"), (132, 128, "f32"), (24, 5, "bf16"), (8, 3, "f32")):
        r = LogitRecipe(T=33, V=V, dtype=dt, sigma0=2.0, peaks=2, sigma=0.6, seed=V)
        za, zp, tok = make_logits(r, "cuda")
        run_case(ctx, za, zp, tok, lam=1.0, k=k, seed=2)
        run_case(ctx, za, zp, tok, lam=1.3, k=V + 5, seed=2)       # exact mode


def test_bad_tokens_empty_and_all_masked(ctx):
    r = LogitRecipe(T=20, V=512, dtype="bf16", sigma0=2.0, peaks=2, sigma=0.6, seed=21)
    za, zp, tok = make_logits(r, "cuda")
    tok2 = tok.clone()
    tok2[3] = 512
    tok2[9] = -1
    out = runner.forward(ctx, za, zp, tok2, None, lam=1.0, k=8, seed=2)
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok2.cpu().numpy(), None, lam=1.0, k=8, seed=2)
    assert out["stats"]["n_bad_token"] == 2
    check_forward(out, ref, 8, 512)
    mask0 = torch.zeros(20, dtype=torch.uint8, device="cuda")
    out = runner.forward(ctx, za, zp, tok, mask0, lam=1.0, k=8, seed=2)
    assert out["stats"]["n_valid"] == 0 and out["stats"]["kappa"] == 1.0
    assert out["weight"].abs().sum().item() == 0 and out["accept"].sum().item() == 0
    out = runner.forward(ctx, za[:0], zp[:0], tok[:0], None, lam=1.0, k=8, seed=2)
    assert out["stats"]["n_valid"] == 0


def test_budget_lambda_and_clip(ctx):
    r = LogitRecipe(T=700, V=2048, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.5, seed=31)
    za, zp, tok = make_logits(r, "cuda")
    mask = (torch.arange(700, device="cuda") % 5 != 0).to(torch.uint8)
    for budget in (0.3, 0.6, 1.0):
        flips, out, ref = run_case(ctx, za, zp, tok, mask, budget=budget, k=12, seed=9, c1=3.0)
        out_b = runner.forward(ctx, za, zp, tok, mask, budget=budget, k=12, seed=9, c1=3.0)
        if budget < 1.0:
            assert abs(out_b["stats"]["mean_accept_prob"] - budget) < 5e-6
        assert out_b["weight"].max().item() <= 3.0


def test_chunked_batch_matches_monolithic_and_oracle(ctx):
    T, V, k = 640, 3000, 24
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.5, seed=41)
    za, zp, tok = make_logits(r, "cuda")
    from paper_2602_06107_b200.inputs import make_lengths_mask
    mask, _ = make_lengths_mask(10, 64, 8, seed=3, device="cuda")
    mono = runner.forward(ctx, za, zp, tok, mask, budget=0.6, k=k, seed=5)
    chunks = [(o, za[o:o + 128], zp[o:o + 128], tok[o:o + 128], mask[o:o + 128]) for o in range(0, T, 128)]
    ch = runner.forward_chunked(ctx, chunks, T, V, B.JP_BF16, budget=0.6, k=k, seed=5, aux=True)
    for n in ("accept", "weight", "logp_actor", "logp_policy", "z_approx", "uniform", "topk_idx_actor"):
        assert torch.equal(mono[n], ch[n]), n
    assert mono["stats"]["mean_kl_p_q"] is None            # not asked for
    assert mono["stats"] == ch["stats"]
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), mask.cpu().numpy(),
                         budget=0.6, k=k, seed=5)
    close(ch["stats"]["lambda_used"], ref["lambda"])
    # a chunk that is never streamed counts as masked
    ch2 = runner.forward_chunked(ctx, chunks[:-1], T, V, B.JP_BF16, lam=1.0, k=k, seed=5)
    assert ch2["stats"]["n_valid"] == int(mask[:512].sum().item())


def test_run_to_run_bitwise_determinism(ctx):
    r = LogitRecipe(T=200, V=30000, dtype="bf16", sigma=1.0, seed=51)
    za, zp, tok = make_logits(r, "cuda")
    outs = [runner.forward(ctx, za, zp, tok, None, budget=0.5, k=32, seed=1) for _ in range(3)]
    for o in outs[1:]:
        for n in ("accept", "weight", "logp_actor", "logp_policy", "z_approx", "lse_actor"):
            assert torch.equal(outs[0][n], o[n]), n
        assert outs[0]["stats"] == o["stats"]


def test_argument_errors_are_reported_not_trapped(ctx):
    r = LogitRecipe(T=4, V=64, dtype="bf16", seed=1)
    za, zp, tok = make_logits(r, "cuda")
    with pytest.raises(B.JackpotError, match="lambda"):
        runner.forward(ctx, za, zp, tok, None, lam=-1.0, k=4)
    with pytest.raises(B.JackpotError, match="budget"):
        runner.forward(ctx, za, zp, tok, None, budget=1.5, k=4)
    with pytest.raises(B.JackpotError, match="k < 1"):
        runner.forward(ctx, za, zp, tok, None, lam=1.0, k=0)
    zw = torch.zeros((4, 200 * 1000), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.JackpotError, match="unsupported"):
        runner.forward(ctx, zw, zw, tok, None, lam=1.0, k=129)
    with pytest.raises(B.JackpotError, match="pitch"):
        z63 = torch.zeros((4, 63), dtype=torch.bfloat16, device="cuda")
        runner.forward(ctx, z63, z63, tok, None, lam=1.0, k=4)
    with pytest.raises(B.JackpotError, match="sequence"):
        d = B.make_desc(za)
        B.jp_batch_chunk(ctx, d, za, zp, tok, None)
    # the context is still usable
    out = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=4)
    assert out["stats"]["n_valid"] == 4


def test_row_shards_with_a_batch_wide_kappa_match_the_undivided_batch(ctx):
    """Two shards of one batch (as two ranks would hold them): decisions are keyed on
    the global row index, and the weights rewritten with the all-shard kappa equal
    those of one call over the whole batch."""
    from paper_2602_06107_b200 import parallel
    T, V, k = 300, 6000, 12
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.2, seed=61)
    za, zp, tok = make_logits(r, "cuda")
    mask = (torch.arange(T, device="cuda") % 4 != 1).to(torch.uint8)
    whole = runner.forward(ctx, za, zp, tok, mask, lam=1.4, k=k, seed=3, c1=2.5)
    ctxs = [B.Context(0), B.Context(0)]
    outs, tot = [], torch.zeros(4, dtype=torch.float64, device="cuda")
    for rank, c in enumerate(ctxs):
        lo, hi = parallel.shard_rows(T, 2, rank)
        o = runner.forward(c, za[lo:hi], zp[lo:hi], tok[lo:hi], mask[lo:hi], lam=1.4, k=k, seed=3, c1=2.5,
                           token_offset=lo)
        outs.append(o)
        t = torch.empty(4, dtype=torch.float64, device="cuda")
        B.jp_batch_totals(c, t)
        tot += t                                  # what the all-reduce over the ranks does
    gstats = []
    for c, o in zip(ctxs, outs):
        sb = B.new_stats_buffer("cuda")
        B.jp_obrs_apply_totals(c, tot, 2.5, o["weight"], sb)
        gstats.append(sb)
    torch.cuda.synchronize()
    for sb in gstats:                             # every shard ends with the undivided batch's statistics
        gs = B.read_stats(sb)
        close(gs["kappa"], whole["stats"]["kappa"], rtol=1e-12)
        assert gs["n_valid"] == whole["stats"]["n_valid"] and gs["n_accept"] == whole["stats"]["n_accept"]
        close(gs["z_approx_mean"], whole["stats"]["z_approx_mean"], rtol=1e-12)
        close(gs["mean_accept_prob"], whole["stats"]["mean_accept_prob"], rtol=1e-12)
    kappa = B.read_stats(gstats[0])["kappa"]
    assert torch.equal(torch.cat([o["accept"] for o in outs]), whole["accept"])
    w = torch.cat([o["weight"] for o in outs])
    assert torch.equal(w, whole["weight"])
    for c in ctxs:
        c.close()
    fresh = B.Context(0)
    with pytest.raises(B.JackpotError, match="sequence"):
        B.jp_obrs_apply_kappa(fresh, 1.0, 0.0, w)
    fresh.close()


def test_row_shards_in_budget_mode_share_one_lambda(ctx):
    """Two shards of one batch in budget mode: each streams its rows once (chunked API), the
    log-probs are gathered, one lambda is solved for the whole batch and every shard is
    finalized with it; decisions, lambda and (after the kappa exchange) weights equal those
    of one budget-mode call over the whole batch."""
    from paper_2602_06107_b200 import parallel
    T, V, k, budget = 320, 6000, 12, 0.6
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.2, seed=62)
    za, zp, tok = make_logits(r, "cuda")
    mask = (torch.arange(T, device="cuda") % 5 != 2).to(torch.uint8)
    whole = runner.forward(ctx, za, zp, tok, mask, budget=budget, k=k, seed=3, c1=2.5)
    ctxs = [B.Context(0), B.Context(0)]
    shards = [parallel.shard_rows(T, 2, rank) for rank in range(2)]
    lqs, lps, vs = [], [], []
    for (lo, hi), c in zip(shards, ctxs):
        n = hi - lo
        B.jp_batch_begin(c, n, V, B.JP_BF16, k, 0.0)
        B.jp_batch_chunk(c, B.make_desc(za[lo:hi], token_offset=0), za[lo:hi], zp[lo:hi], tok[lo:hi], mask[lo:hi])
        lq, lp = torch.empty(n, device="cuda"), torch.empty(n, device="cuda")
        v = torch.empty(n, dtype=torch.uint8, device="cuda")
        B.jp_batch_logprobs(c, lq, lp, v)
        lqs.append(lq); lps.append(lp); vs.append(v)
    # what the all-gather would hand to every rank
    lam = parallel.solve_on_device(torch.cat(lqs), torch.cat(lps), torch.cat(vs), budget)
    close(lam, whole["stats"]["lambda_used"], rtol=1e-6)
    outs, tot = [], torch.zeros(4, dtype=torch.float64, device="cuda")
    for (lo, hi), c in zip(shards, ctxs):
        n = hi - lo
        o = runner._alloc_outputs(n, "cuda")
        d = B.jp_obrs_desc()
        d.c1 = 2.5
        d.token_offset = lo
        B.jp_batch_finalize(c, d, lam, B.JP_LAMBDA_FIXED, 3, o["accept"], o["weight"], o["logp_actor"],
                            o["logp_policy"], o["stats_buf"])
        torch.cuda.synchronize()
        o["stats"] = B.read_stats(o["stats_buf"])
        outs.append(o)
        t = torch.empty(4, dtype=torch.float64, device="cuda")
        B.jp_batch_totals(c, t)
        tot += t
    sb = B.new_stats_buffer("cuda")
    for c, o in zip(ctxs, outs):
        B.jp_obrs_apply_totals(c, tot, 2.5, o["weight"], sb)
    torch.cuda.synchronize()
    kappa = B.read_stats(sb)["kappa"]
    if float(np.float32(lam)) == float(np.float32(whole["stats"]["lambda_used"])):
        assert torch.equal(torch.cat([o["accept"] for o in outs]), whole["accept"])
        close(kappa, whole["stats"]["kappa"], rtol=1e-9)
        close(torch.cat([o["weight"] for o in outs]).cpu().numpy(), whole["weight"].cpu().numpy())
    for c in ctxs:
        c.close()


def test_wide_dynamic_range_rows(ctx):
    """Rows whose logits climb far beyond the headroom of a lane's reference exponent (64 binades =
    44 nats) in the middle of the row, in steps and as a ramp: the online sums must move their
    reference and still agree with the oracle.  (Magnitudes stay below ~60: see the next test.)"""
    V, k = 40000, 16
    g = torch.Generator().manual_seed(9)
    for dt in (torch.float32, torch.bfloat16):
        rows = torch.randn((8, V), generator=g)
        rows[0, : V // 2] -= 100.0                      # one jump of 100 nats half way
        rows[1, :] += torch.linspace(-400.0, 0.0, V)    # a ramp across many rescalings
        rows[2, :] += torch.linspace(0.0, -300.0, V)    # the maximum comes first
        rows[3, 123] = 45.0                             # one dominant entry
        rows[4, :] = rows[4, :] * 10.0 - 50.0           # a wide spread below zero
        rows[5, ::7] -= 150.0                           # entries far below the rest
        rows[6, :] *= 1e-3                              # nearly flat
        rows[7, : V - 5] -= 90.0                        # the jump in the last vectors
        za = rows.to(dt).cuda()
        zp = rows.flip(0).to(dt).cuda().contiguous()
        tok = torch.tensor([5, V - 1, 0, 123, 9, 7, 11, V - 2], dtype=torch.int32, device="cuda")
        # (the clip keeps the weights inside fp32: some tokens have p/q of e^150 here)
        run_case(ctx, za, zp, tok, lam=1.2, k=k, seed=4, c1=5.0)
        run_case(ctx, za, zp, tok, lam=1.2, k=V, seed=4, c1=5.0)    # exact mode


def test_large_magnitude_logits(ctx):
    """The exponent z log2(e) is formed with the fp32 constant log2(e), which is short by a factor
    1 - 1.335e-8; the kernel scales the finished log-sum-exp back, which leaves an error below
    1.335e-8 x (entropy of the row) < 2e-7.  So rows whose mass sits at logits of magnitude 100 to
    1500 must still give log-probs inside the usual bar (the log-sum-exp itself is published in
    fp32: half an ulp of its own magnitude), and exact top-k lists."""
    V, k = 20000, 8
    g = torch.Generator().manual_seed(10)
    rows = torch.randn((4, V), generator=g)
    offs = torch.tensor([500.0, -800.0, 1500.0, 120.0])
    rows += offs[:, None]
    za = rows.cuda()
    zp = rows.flip(1).contiguous().cuda()
    tok = torch.tensor([1, 2, 3, 4], dtype=torch.int32, device="cuda")
    out = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=k, seed=1)
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), None, lam=1.0, k=k, seed=1)
    close(out["logp_actor"].cpu().numpy(), ref["lq64"])
    close(out["logp_policy"].cpu().numpy(), ref["lp64"])
    assert np.all(np.abs(out["lse_actor"].cpu().numpy() - ref["lse_a"]) <= 1e-6 + 6e-8 * np.abs(ref["lse_a"]))
    assert np.all(np.abs(out["lse_policy"].cpu().numpy() - ref["lse_p"]) <= 1e-6 + 6e-8 * np.abs(ref["lse_p"]))
    assert np.array_equal(out["topk_idx_actor"].cpu().numpy(), ref["topk_idx_a"])
    assert np.array_equal(out["topk_idx_policy"].cpu().numpy(), ref["topk_idx_p"])
    close(out["z_approx"].cpu().numpy(), ref["zk"])
    # the normalisers and the weights hang on exp(z - lse): a log-sum-exp held in one fp32 word would
    # put ulp(1500)/2 = 6e-5 on every one of them
    flips, out, ref = run_case(ctx, za, zp, tok, lam=1.0, k=k, seed=1, exact_too=True)
    flips, out, ref = run_case(ctx, za, zp, tok, lam=0.7, k=V, seed=1)


def test_nonfinite_rows_are_counted_and_do_not_disturb_the_others(ctx):
    """+inf and NaN logits, and a sampled token of probability 0: the row is counted in n_nonfinite and
    treated as masked; nothing traps or waits, and every other row, the batch statistics, kappa, the
    weights and a budget-derived lambda are what they are with those rows masked out."""
    T, V, k = 64, 30000, 8
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.0, seed=63)
    za, zp, tok = make_logits(r, "cuda")
    za2, zp2 = za.clone(), zp.clone()
    za2[5, 100] = float("inf")
    zp2[9, 29999] = float("nan")
    za2[20, :] = float("nan")
    zp2[31, :] = float("nan")
    za2[31, 7] = float("nan")
    za2[40, int(tok[40])] = float("-inf")          # the sampled token has probability 0 under the actor
    bad_rows = [5, 9, 20, 31, 40]
    good = torch.ones(T, dtype=torch.bool, device="cuda")
    good[bad_rows] = False
    mask = good.to(torch.uint8)
    names = ("logp_actor", "logp_policy", "lse_actor", "lse_policy", "z_approx", "accept_prob", "uniform",
             "topk_idx_actor", "topk_idx_policy", "accept", "weight")
    for kw in (dict(lam=1.3), dict(budget=0.55)):
        for kk in (k, V):
            clean = runner.forward(ctx, za, zp, tok, mask, k=kk, seed=2, c1=4.0, **kw)
            out = runner.forward(ctx, za2, zp2, tok, None, k=kk, seed=2, c1=4.0, **kw)
            st, cs = out["stats"], clean["stats"]
            assert st["status"] == 0 and st["n_nonfinite"] == len(bad_rows) and cs["n_nonfinite"] == 0
            for n in ("n_valid", "n_accept", "alpha_hat", "mean_accept_prob", "z_approx_mean", "kappa", "lambda_used"):
                assert st[n] == cs[n], (n, st[n], cs[n])
            for n in names:
                if n in out:
                    assert torch.equal(out[n][good], clean[n][good]), n
            assert out["weight"][~good].abs().sum().item() == 0 and out["accept"][~good].sum().item() == 0
            assert out["accept_prob"][~good].abs().sum().item() == 0 and out["z_approx"][~good].abs().sum().item() == 0
    # and against the oracle with those rows masked
    out = runner.forward(ctx, za2, zp2, tok, None, lam=1.3, k=k, seed=2)
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), mask.cpu().numpy(), lam=1.3, k=k,
                         seed=2)
    check_forward(out, ref, k, V, mask.cpu().numpy())
    # the gradient rows of such a row are zero
    da, dp = runner.backward(ctx, za2, zp2, tok, None, out["accept"], out["weight"], lambda_distill=1.0)
    torch.cuda.synchronize()
    assert da[~good].float().abs().sum().item() == 0 and dp[~good].float().abs().sum().item() == 0
    assert torch.isfinite(da[good].float()).all() and torch.isfinite(dp[good].float()).all()


def test_mean_kl_statistic_on_request(ctx):
    """jp_stats.mean_kl_p_q: the batch mean of KL(p_target || p_inf) per row (the actor-policy divergence
    the paper tracks during training), computed by one more pass when the descriptor asks for it, NaN
    otherwise; monolithic, chunked, and in exact mode."""
    T, V, k = 300, 20008, 12
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.1, seed=65)
    za, zp, tok = make_logits(r, "cuda")
    mask = (torch.arange(T, device="cuda") % 6 != 2).to(torch.uint8)
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), mask.cpu().numpy(), lam=1.2, k=k,
                         seed=4, want_kl=True)
    o = runner._alloc_outputs(T, "cuda")

    def run(kk, flags, **kw):
        mode = B.JP_LAMBDA_FROM_BUDGET if "budget" in kw else B.JP_LAMBDA_FIXED
        d = B.make_desc(za, flags=flags, lambda_mode=mode)
        B.jp_obrs_forward(ctx, d, za, zp, tok, mask, kw.get("budget", kw.get("lam")), kk, 4, o["accept"], o["weight"],
                          o["logp_actor"], o["logp_policy"], o["stats_buf"])
        torch.cuda.synchronize()
        return B.read_stats(o["stats_buf"])

    assert run(k, 0, lam=1.2)["mean_kl_p_q"] is None
    for st in (run(k, B.JP_DESC_KL, lam=1.2), run(V, B.JP_DESC_KL, lam=1.2), run(k, B.JP_DESC_KL, budget=0.6),
               run(V, B.JP_DESC_KL, budget=0.6)):
        close(st["mean_kl_p_q"], ref["stats"]["mean_kl_p_q"], rtol=1e-4, atol=5e-6)
    # chunked: reported only if every chunk asked
    for flags_last, want in ((B.JP_DESC_KL, True), (0, False)):
        B.jp_batch_begin(ctx, T, V, B.JP_BF16, k, 0.0)
        for off in range(0, T, 100):
            fl = B.JP_DESC_KL if off < 200 else flags_last
            B.jp_batch_chunk(ctx, B.make_desc(za[off:off + 100], token_offset=off, flags=fl), za[off:off + 100],
                             zp[off:off + 100], tok[off:off + 100], mask[off:off + 100])
        B.jp_batch_finalize(ctx, B.jp_obrs_desc(), 1.2, B.JP_LAMBDA_FIXED, 4, o["accept"], o["weight"],
                            o["logp_actor"], o["logp_policy"], o["stats_buf"])
        torch.cuda.synchronize()
        got = B.read_stats(o["stats_buf"])["mean_kl_p_q"]
        if want:
            close(got, ref["stats"]["mean_kl_p_q"], rtol=1e-4, atol=5e-6)
        else:
            assert got is None


def test_host_buffer_entry_point_equals_the_device_path(ctx):
    """jp_obrs_forward_host stages host rows through device slots chunk by chunk: with a mask, a
    global row offset, several (uneven) chunks, pinned and pageable memory, fixed lambda and a
    budget, it must return the bits of the device-resident call."""
    T, V, k = 700, 12008, 16
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.1, seed=64)
    za, zp, tok = make_logits(r, "cuda")
    mask = (torch.arange(T, device="cuda") % 9 != 4).to(torch.uint8)
    for kw, lam_or_budget, mode in ((dict(lam=1.4), 1.4, B.JP_LAMBDA_FIXED), (dict(budget=0.55), 0.55, B.JP_LAMBDA_FROM_BUDGET)):
        dev = runner.forward(ctx, za, zp, tok, mask, k=k, seed=6, c1=2.0, token_offset=1000, **kw)
        for pinned in (True, False):
            def host(t):
                t = t.cpu()
                return t.pin_memory() if pinned else t
            hza, hzp, htok, hmask = host(za), host(zp), host(tok), host(mask)
            hacc = host(torch.empty(T, dtype=torch.uint8))
            hw, hlq, hlp = (host(torch.empty(T, dtype=torch.float32)) for _ in range(3))
            hst = host(torch.zeros(B.STATS_BYTES, dtype=torch.uint8))
            d = B.make_desc(hza, lambda_mode=mode, c1=2.0, token_offset=1000)
            B.jp_obrs_forward_host(ctx, d, hza, hzp, htok, hmask, lam_or_budget, k, 6, hacc, hw, hlq, hlp, hst, 300)
            assert torch.equal(hacc, dev["accept"].cpu())
            assert torch.equal(hw, dev["weight"].cpu())
            assert torch.equal(hlq, dev["logp_actor"].cpu()) and torch.equal(hlp, dev["logp_policy"].cpu())
            st = B.read_stats(hst)
            assert st["n_accept"] == dev["stats"]["n_accept"] and st["kappa"] == dev["stats"]["kappa"]
            assert st["lambda_used"] == dev["stats"]["lambda_used"]


def test_one_context_through_changing_shapes_equals_fresh_contexts(ctx):
    """A context re-lays its workspace out as shapes, dtypes and k change from call to call; nothing
    of an earlier call may leak into a later one."""
    cases = [("bf16", 300, 20000, 64), ("f32", 200, 4099 + 5, 8), ("bf16", 310, 151936, 128), ("bf16", 300, 20000, 20000),
             ("bf16", 64, 512, 4), ("bf16", 300, 20000, 64)]
    names = ("accept", "weight", "logp_actor", "logp_policy", "z_approx", "topk_idx_actor", "topk_idx_policy")
    for i, (dt, T, V, k) in enumerate(cases):
        r = LogitRecipe(T=T, V=V, dtype=dt, sigma0=2.5, peaks=4, sigma=1.0, seed=70 + i)
        za, zp, tok = make_logits(r, "cuda")
        mask = (torch.arange(T, device="cuda") % 5 != 1).to(torch.uint8)
        a = runner.forward(ctx, za, zp, tok, mask, lam=1.3, k=k, seed=i)
        fresh = B.Context(0)
        b = runner.forward(fresh, za, zp, tok, mask, lam=1.3, k=k, seed=i)
        for n in names:
            if k >= V and n.startswith("topk"):
                continue
            assert torch.equal(a[n], b[n]), (i, n)
        assert a["stats"] == b["stats"], i
        fresh.close()


def test_forward_on_a_side_stream():
    """The context enqueues on the stream it was given; results equal those of the default stream."""
    r = LogitRecipe(T=200, V=30000, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.0, seed=80)
    za, zp, tok = make_logits(r, "cuda")
    c0 = B.Context(0)
    ref = runner.forward(c0, za, zp, tok, None, lam=1.2, k=16, seed=3)
    c0.close()
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        c1 = B.Context(0)                       # binds torch's current stream: the side stream
        out = runner.forward(c1, za, zp, tok, None, lam=1.2, k=16, seed=3)
        side.synchronize()
        c1.close()
    for n in ("accept", "weight", "logp_actor", "topk_idx_policy"):
        assert torch.equal(out[n], ref[n]), n


def test_stream_probe_reports_a_plausible_rate():
    x = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    y = torch.empty_like(x)
    rd = B.jp_probe_stream(x, None, reps=5)
    cp = B.jp_probe_stream(x, y, reps=5)
    assert 1000.0 < rd < 12000.0 and 1000.0 < cp < 12000.0
    with pytest.raises(B.JackpotError):
        B.jp_probe_stream(x[1:], None, reps=1)          # not 16-byte aligned


def test_a_wait_that_nothing_completes_runs_out_and_leaves_the_context_usable(ctx):
    """The bounded wait of the kernels, against a barrier nobody arrives at, with a short limit (about
    50 ms of SM clock): the kernel ends by itself, the status word reads JP_ERR_TIMEOUT, and the next
    forward on the same context is unaffected."""
    import time
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    B.jp_selftest_bounded_wait(ctx, 100_000_000, st)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert st.item() == -6                                   # JP_ERR_TIMEOUT
    assert 0.01 < dt < 1.5, dt
    r = LogitRecipe(T=40, V=4096, dtype="bf16", sigma0=2.0, peaks=2, sigma=0.6, seed=77)
    za, zp, tok = make_logits(r, "cuda")
    run_case(ctx, za, zp, tok, lam=1.2, k=8, seed=1)
    with pytest.raises(B.JackpotError, match="limit_cycles"):
        B.jp_selftest_bounded_wait(ctx, 0, st)
