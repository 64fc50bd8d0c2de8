"""GPU parity of the fused logit gradients (jp_obrs_backward) against the oracle.

Bar: bf16 outputs within rtol 2e-2 of the oracle's double gradients, plus an
absolute floor that covers cancellation in q - p and the one-hot term,
  1e-4 (g/N) (|A_t| max(q_v, p_v, 1[v=x]) + lambda_distill (q_v + p_v)),
(elements that needed the floor are counted).  Row sums of both gradients are
zero; rejected and masked rows are exactly zero.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200 import runner
from paper_2602_06107_b200.inputs import LogitRecipe, make_logits, to_numpy_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    jp_build.build()
    c = B.Context(0)
    yield c
    c.close()


def _widen(bits):
    if bits.dtype == np.uint16:
        return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return bits.astype(np.float64)


def check_grads(da, dp, rows, za_np, zp_np, tok, mask, acc, w, lse_a, lse_p, n_valid, adv, lam_d, g=1.0):
    ra, rp = oracle.grad_rows(rows, za_np, zp_np, tok, acc, w, lse_a, lse_p, float(n_valid), mask=mask, adv=adv,
                              grad_out=g, lambda_distill=lam_d)
    ga = da[rows].float().cpu().numpy().astype(np.float64)
    gp = dp[rows].float().cpu().numpy().astype(np.float64)
    q = np.exp(_widen(za_np[rows]) - lse_a[rows][:, None])
    p = np.exp(_widen(zp_np[rows]) - lse_p[rows][:, None])
    hot = np.zeros_like(q)
    hot[np.arange(len(rows)), np.clip(tok[rows], 0, q.shape[1] - 1)] = 1.0
    A = np.ones(len(rows)) if adv is None else adv[rows].astype(np.float64)
    scale = g / max(n_valid, 1)
    floor_a = 1e-4 * scale * (np.abs(A)[:, None] * np.maximum(np.maximum(q, p), hot) + lam_d * (q + p)) + 1e-30
    floor_p = 1e-4 * scale * (np.abs(A) * w[rows])[:, None] * np.maximum(p, hot) + 1e-30
    bad_a = np.abs(ga - ra) > 2e-2 * np.abs(ra) + floor_a
    bad_p = np.abs(gp - rp) > 2e-2 * np.abs(rp) + floor_p
    assert not bad_a.any(), f"d_actor: {bad_a.sum()} bad, worst {np.abs(ga - ra).max():.3e}"
    assert not bad_p.any(), f"d_policy: {bad_p.sum()} bad, worst {np.abs(gp - rp).max():.3e}"
    needed_floor = int(((np.abs(ga - ra) > 2e-2 * np.abs(ra)) | (np.abs(gp - rp) > 2e-2 * np.abs(rp))).sum())
    # invariants the formulas fix
    valid = np.ones(len(rows), bool) if mask is None else mask[rows] != 0
    assert np.all(ga[~valid] == 0) and np.all(gp[~valid] == 0)
    rej = valid & (acc[rows] == 0)
    assert np.all(gp[rej] == 0), "a rejected token must not reach the policy gradient"
    # bf16 rounding of V terms, plus the elementwise floor of the bar above summed over the row (where the
    # gradients are tiny, A_t near 0, the floor and not the rounding is what bounds the elements)
    tol_sum = 2.0 ** -8 * np.abs(ra).sum(1) + floor_a.sum(1) + 1e-12
    assert np.all(np.abs(ga.sum(1)) <= tol_sum + np.abs(ra.sum(1)))
    return needed_floor


@pytest.mark.parametrize("dtype,V,ld", [("bf16", 20000, 20000), ("bf16", 5003, 5008), ("f32", 4099, 4104)])
@pytest.mark.parametrize("lam_d", [0.0, 1.0])
def test_backward_matches_oracle(ctx, dtype, V, ld, lam_d):
    T = 150
    r = LogitRecipe(T=T, V=ld, dtype=dtype, sigma0=2.5, peaks=4, sigma=1.0, seed=11)
    zaf, zpf, _ = make_logits(r, "cuda")
    za, zp = zaf[:, :V], zpf[:, :V]
    g = torch.Generator(device="cuda").manual_seed(3)
    gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
    tok = (za.float() + gum).argmax(1).to(torch.int32)
    mask = (torch.arange(T, device="cuda") % 6 != 1).to(torch.uint8)
    adv = torch.randn(T, generator=g, device="cuda")
    out = runner.forward(ctx, za, zp, tok, mask, lam=1.3, k=16, seed=5, c1=3.0)
    da, dp = runner.backward(ctx, za, zp, tok, mask, out["accept"], out["weight"], advantages=adv,
                             lambda_distill=lam_d, grad_out=0.5)
    torch.cuda.synchronize()
    za_np, zp_np = to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous())
    ref = oracle.forward(za_np, zp_np, tok.cpu().numpy(), mask.cpu().numpy(), lam=1.3, k=16, seed=5, c1=3.0)
    rows = np.arange(0, T, 3)
    n = check_grads(da, dp, rows, za_np, zp_np, tok.cpu().numpy(), mask.cpu().numpy(), out["accept"].cpu().numpy(),
                    out["weight"].cpu().numpy(), ref["lse_a"], ref["lse_p"], out["stats"]["n_valid"],
                    adv.cpu().numpy(), lam_d, g=0.5)
    print("elements that needed the absolute floor:", n)
    # padding columns of the pitch are never written
    if ld > V:
        pad = torch.full((T, ld), 7.0, dtype=torch.bfloat16, device="cuda")
        pad2 = pad.clone()
        runner.backward(ctx, za, zp, tok, mask, out["accept"], out["weight"], advantages=adv, lambda_distill=lam_d,
                        d_actor=pad[:, :V], d_policy=pad2[:, :V])
        torch.cuda.synchronize()
        assert torch.all(pad[:, V:] == 7.0) and torch.all(pad2[:, V:] == 7.0)


def test_backward_in_place_and_defaults(ctx):
    r = LogitRecipe(T=64, V=8192, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.0, seed=12)
    za, zp, tok = make_logits(r, "cuda")
    out = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=8, seed=1)
    da, dp = runner.backward(ctx, za, zp, tok, None, out["accept"], out["weight"], lambda_distill=1.0)
    za2, zp2 = za.clone(), zp.clone()
    runner.backward(ctx, za2, zp2, tok, None, out["accept"], out["weight"], lambda_distill=1.0, d_actor=za2,
                    d_policy=zp2)
    torch.cuda.synchronize()
    assert torch.equal(da, za2) and torch.equal(dp, zp2), "aliased gradients differ from out-of-place ones"
    # no advantages = all ones; explicit ones give the same bits
    ones = torch.ones(64, device="cuda")
    da1, dp1 = runner.backward(ctx, za, zp, tok, None, out["accept"], out["weight"], advantages=ones,
                               lambda_distill=1.0)
    assert torch.equal(da, da1) and torch.equal(dp, dp1)
    # lambda_distill = 0 and zero advantages: nothing flows
    da0, dp0 = runner.backward(ctx, za, zp, tok, None, out["accept"], out["weight"], advantages=ones * 0,
                               lambda_distill=0.0)
    assert da0.abs().max().item() == 0 and dp0.abs().max().item() == 0


def test_backward_needs_a_forward_and_matching_shapes():
    c = B.Context(0)
    r = LogitRecipe(T=8, V=256, dtype="bf16", seed=2)
    za, zp, tok = make_logits(r, "cuda")
    acc = torch.ones(8, dtype=torch.uint8, device="cuda")
    w = torch.ones(8, device="cuda")
    with pytest.raises(B.JackpotError, match="sequence"):
        runner.backward(c, za, zp, tok, None, acc, w)
    runner.forward(c, za, zp, tok, None, lam=1.0, k=4)
    with pytest.raises(B.JackpotError, match="records"):
        runner.backward(c, za, zp, tok, None, acc, w, record_offset=4)
    c.close()


def test_training_step_chunked_budget_then_backward(ctx):
    """The training-step shape at reduced T: chunked forward with a budget-derived
    lambda and a clip, then one backward per chunk against the batch's records."""
    T, V, chunk, k = 1536, 151936, 512, 64
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0, peak_hi=15.0, sigma=1.0, seed=4)
    za, zp, tok = make_logits(r, "cuda")
    chunks = [(o, za[o:o + chunk], zp[o:o + chunk], tok[o:o + chunk], None) for o in range(0, T, chunk)]
    out = runner.forward_chunked(ctx, chunks, T, V, B.JP_BF16, budget=0.5, k=k, seed=4, c1=3.0)
    adv = torch.randn(T, device="cuda")
    da = torch.empty_like(za)
    dp = torch.empty_like(zp)
    for o in range(0, T, chunk):
        runner.backward(ctx, za[o:o + chunk], zp[o:o + chunk], tok[o:o + chunk], None, out["accept"][o:o + chunk],
                        out["weight"][o:o + chunk], advantages=adv[o:o + chunk], lambda_distill=1.0,
                        record_offset=o, d_actor=da[o:o + chunk], d_policy=dp[o:o + chunk])
    torch.cuda.synchronize()
    assert abs(out["stats"]["mean_accept_prob"] - 0.5) < 5e-6
    rows = np.arange(5, T, 97)
    sub = torch.from_numpy(rows).cuda()
    za_s, zp_s = to_numpy_bits(za[sub]), to_numpy_bits(zp[sub])
    tok_s = tok[sub].cpu().numpy()
    lg = oracle.lse_gather(za_s, zp_s, tok_s)
    check_grads(da[sub], dp[sub], np.arange(len(rows)), za_s, zp_s, tok_s, None, out["accept"][sub].cpu().numpy(),
                out["weight"][sub].cpu().numpy(), lg["lse_a"], lg["lse_p"], out["stats"]["n_valid"],
                adv[sub].cpu().numpy(), 1.0)


@pytest.mark.parametrize("dtype,V", [("bf16", 20000), ("f32", 4099 + 5)])
def test_backward_general_form_matches_oracle(ctx, dtype, V):
    """Away from the first update: PPO ratios against reference log-probs, asymmetric clip,
    rho with c2, the truncated importance weight F, per-token terms, KL and the loss."""
    T = 120
    r = LogitRecipe(T=T, V=V, dtype=dtype, sigma0=2.5, peaks=4, sigma=1.0, seed=21)
    za, zp, tok = make_logits(r, "cuda")
    g = torch.Generator(device="cuda").manual_seed(7)
    mask = (torch.arange(T, device="cuda") % 7 != 3).to(torch.uint8)
    adv = torch.randn(T, generator=g, device="cuda")
    out = runner.forward(ctx, za, zp, tok, mask, lam=1.3, k=16, seed=5, c1=3.0)
    # reference log-probs scattered around the current ones so that tokens land on both
    # sides of the clip range
    logp_ref = out["logp_policy"] + 0.35 * torch.randn(T, generator=g, device="cuda")
    logq_ref = out["logp_actor"] + 0.35 * torch.randn(T, generator=g, device="cuda")
    logp_inf = logq_ref + 0.5 * torch.randn(T, generator=g, device="cuda")
    eps_lo, eps_hi = float(np.float32(0.2)), float(np.float32(0.28))
    c2, cap = float(np.float32(1.25)), float(np.float32(1.5))
    lam_d, g_out = 0.6, 0.5
    obj_p = torch.empty(T, device="cuda")
    obj_a = torch.empty(T, device="cuda")
    kl = torch.empty(T, device="cuda")
    loss = torch.zeros(4, dtype=torch.float64, device="cuda")
    da, dp = runner.backward(ctx, za, zp, tok, mask, out["accept"], out["weight"], advantages=adv,
                             lambda_distill=lam_d, grad_out=g_out, logp_ref=logp_ref, logp_actor_ref=logq_ref,
                             logp_inf=logp_inf, eps_lo=eps_lo, eps_hi=eps_hi, c2=c2, tis_cap=cap,
                             out_obj_policy=obj_p, out_obj_actor=obj_a, out_kl=kl, out_loss=loss)
    torch.cuda.synchronize()
    za_np, zp_np = to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous())
    m_np, acc, w = mask.cpu().numpy(), out["accept"].cpu().numpy(), out["weight"].cpu().numpy()
    lq, lp = out["logp_actor"].cpu().numpy(), out["logp_policy"].cpu().numpy()
    terms = oracle.ppo_terms(lq, lp, acc, w, adv.cpu().numpy(), mask=m_np, logp_ref=logp_ref.cpu().numpy(),
                             logq_ref=logq_ref.cpu().numpy(), logp_inf=logp_inf.cpu().numpy(), clip=True,
                             eps_lo=eps_lo, eps_hi=eps_hi, c2=c2, tis_cap=cap)
    # the fixture must exercise every branch
    valid = m_np != 0
    assert (terms["slope_theta"][valid & (acc != 0)] == 0).any() and (terms["slope_theta"][valid] != 0).any()
    assert (terms["slope_omega"][valid] == 0).any() and (terms["F"][valid] == cap).any()
    # per-token terms (decisions taken in double on both sides; values rounded to fp32)
    assert np.allclose(obj_p.cpu().numpy(), terms["obj_theta"], rtol=1e-5, atol=1e-7)
    assert np.allclose(obj_a.cpu().numpy(), terms["obj_omega"], rtol=1e-5, atol=1e-7)
    ref = oracle.forward(za_np, zp_np, tok.cpu().numpy(), m_np, lam=1.3, k=16, seed=5, c1=3.0)
    kl_ref = oracle.kl_rows(za_np, zp_np, ref["lse_a"], ref["lse_p"], mask=m_np)
    # KL = sum_v p (zp - za) - lse_p + lse_a in fp32: the two log-sum-exps (~10, half an ulp = 5e-7 each)
    # cancel against the sum, so the error is absolute, a few 1e-6
    assert np.allclose(kl.cpu().numpy(), kl_ref, rtol=1e-4, atol=5e-6)
    N = out["stats"]["n_valid"]
    l1, l2, l3 = terms["obj_theta"].sum() / N, terms["obj_omega"].sum() / N, kl_ref.sum() / N
    got = loss.cpu().numpy()
    assert np.allclose(got[1:], [l1, l2, l3], rtol=1e-4, atol=5e-6)
    assert got[0] == pytest.approx(-l1 - l2 + lam_d * l3, rel=1e-4, abs=1e-5)
    # gradients
    rows = np.arange(0, T, 2)
    ra, rp = oracle.grad_rows(rows, za_np, zp_np, tok.cpu().numpy(), acc, w, ref["lse_a"], ref["lse_p"], float(N),
                              mask=m_np, adv=adv.cpu().numpy(), grad_out=g_out, lambda_distill=lam_d, ppo=terms)
    ga = da[rows].float().cpu().numpy().astype(np.float64)
    gp = dp[rows].float().cpu().numpy().astype(np.float64)
    q = np.exp(_widen(za_np[rows]) - ref["lse_a"][rows][:, None])
    p = np.exp(_widen(zp_np[rows]) - ref["lse_p"][rows][:, None])
    hot = np.zeros_like(q)
    hot[np.arange(len(rows)), tok.cpu().numpy()[rows]] = 1.0
    scale = g_out / N
    ca = np.abs(terms["slope_omega"] * terms["r_omega"])[rows][:, None]
    cp = np.abs(terms["slope_theta"] * terms["r_theta"])[rows][:, None]
    floor_a = 1e-4 * scale * (ca * np.maximum(q, hot) + lam_d * (q + p)) + 1e-30
    floor_p = 1e-4 * scale * cp * np.maximum(p, hot) + 1e-30
    assert not (np.abs(ga - ra) > 2e-2 * np.abs(ra) + floor_a).any()
    assert not (np.abs(gp - rp) > 2e-2 * np.abs(rp) + floor_p).any()
    clipped = (terms["slope_theta"][rows] == 0)
    assert np.all(gp[clipped] == 0), "a clipped, rejected or masked token must not reach the policy gradient"


def test_backward_general_form_defaults_equal_first_update(ctx):
    r = LogitRecipe(T=64, V=8192, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.0, seed=12)
    za, zp, tok = make_logits(r, "cuda")
    out = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=8, seed=1)
    adv = torch.randn(64, device="cuda")
    da, dp = runner.backward(ctx, za, zp, tok, None, out["accept"], out["weight"], advantages=adv, lambda_distill=1.0)
    # the reference log-probs equal to the current ones: every ratio is 1 and nothing is clipped
    da1, dp1 = runner.backward(ctx, za, zp, tok, None, out["accept"], out["weight"], advantages=adv,
                               lambda_distill=1.0, logp_ref=out["logp_policy"], logp_actor_ref=out["logp_actor"],
                               logp_inf=out["logp_actor"], eps_lo=0.2, eps_hi=0.2, c2=10.0, tis_cap=10.0)
    torch.cuda.synchronize()
    assert torch.equal(da, da1) and torch.equal(dp, dp1)
    with pytest.raises(B.JackpotError, match="out_loss needs"):
        runner.backward(ctx, za, zp, tok, None, out["accept"], out["weight"],
                        out_loss=torch.zeros(4, dtype=torch.float64, device="cuda"))
