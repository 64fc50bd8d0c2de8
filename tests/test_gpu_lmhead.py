"""GPU parity of the output-layer-fused row pass (jp_lmhead_lse_topk) against the oracle.

The fused kernel forms logits z = hidden x weight^T on the tensor cores (bf16 operands, fp32
accumulation) and never stores them; the oracle forms the same logits in double and rounds them once
to fp32, then takes log-sum-exp, the token's log-prob and the top-k by its usual routines.

Bars.  A logit is a sum of H exact products accumulated in fp32 in an order the hardware chooses, so
it differs from the oracle's by up to ~ sqrt(H) ulps of the partial sums: a few 1e-6 in absolute terms
for logits of magnitude 10.  Log-sum-exp and log-prob: rtol 1e-5 / atol 2e-5 (the atol is that logit
error, not the summation's).  Top-k: the values within the same bar; the index lists must be equal
except where two logits are closer than the bar (then either order is right: what is compared is
that the list is a valid top-k of the oracle's logits within the bar)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200.inputs import to_numpy_bits

pytestmark = pytest.mark.gpu
RTOL, ATOL = 1e-5, 2e-5


@pytest.fixture(scope="module")
def ctx():
    jp_build.build()
    c = B.Context(0)
    yield c
    c.close()


def make(T, H, V, seed, sigma=3.0, ldh=None, ldw=None):
    g = torch.Generator(device="cuda").manual_seed(seed)
    ldh, ldw = ldh or H, ldw or H
    h = torch.zeros((T, ldh), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((V, ldw), dtype=torch.bfloat16, device="cuda")
    h[:, :H] = torch.randn((T, H), generator=g, device="cuda").to(torch.bfloat16)
    w[:, :H] = (torch.randn((V, H), generator=g, device="cuda") * (sigma / H ** 0.5)).to(torch.bfloat16)
    tok = torch.randint(0, V, (T,), generator=g, device="cuda", dtype=torch.int32)
    return h[:, :H], w[:, :H], tok


def run(ctx, h, w, tok, mask, k):
    T = h.shape[0]
    lse = torch.empty(T, device="cuda")
    lp = torch.empty(T, device="cuda")
    idx = torch.empty((T, k), dtype=torch.int32, device="cuda")
    val = torch.empty((T, k), device="cuda")
    st = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    B.jp_lmhead_lse_topk(ctx, h, w, tok, mask, k, lse, lp, idx, val, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    return lse.cpu().numpy(), lp.cpu().numpy(), idx.cpu().numpy(), val.cpu().numpy()


def check(ctx, h, w, tok, mask, k, rows):
    lse, lp, idx, val = run(ctx, h, w, tok, mask, k)
    hb, wb = to_numpy_bits(h.contiguous()), to_numpy_bits(w.contiguous())
    z = oracle.lmhead_rows(rows, hb, wb)
    tok_h = tok.cpu().numpy()[rows]
    m = None if mask is None else mask.cpu().numpy()[rows]
    ref = oracle.lse_gather(z, z, tok_h, m)
    ref_idx = oracle.topk(z, k, m)
    valid = (np.ones(len(rows), bool) if m is None else m != 0) & (ref["bad"] == 0)
    tol = lambda x: ATOL + RTOL * np.abs(x)
    assert np.all(np.abs(lse[rows][valid] - ref["lse_a"][valid]) <= tol(ref["lse_a"][valid]))
    assert np.all(np.abs(lp[rows][valid] - ref["lq64"][valid]) <= tol(ref["lq64"][valid]))
    assert np.all(lse[rows][~valid] == 0) and np.all(idx[rows][~valid] == -1)
    n_swapped = 0
    for i, r in enumerate(rows):
        if not valid[i]:
            continue
        zi = z[i].astype(np.float64)
        gi, gv = idx[r], val[r].astype(np.float64)
        assert len(set(gi.tolist())) == k and gi.min() >= 0 and gi.max() < z.shape[1]
        assert np.all(np.abs(gv - zi[gi]) <= tol(zi[gi]))                 # the values are the logits at the indices
        assert np.all(gv[:-1] >= gv[1:])                                  # best first
        kth = zi[ref_idx[i][-1]]
        assert np.all(zi[gi] >= kth - tol(kth))                           # nothing in the list is clearly outside the top k
        outside = np.setdiff1d(ref_idx[i], gi)
        assert np.all(zi[outside] <= kth + tol(kth))                      # and nothing clearly inside is missing
        n_swapped += int(not np.array_equal(gi, ref_idx[i]))
    return n_swapped


def test_fused_output_layer_small(ctx):
    for (T, H, V, k) in ((200, 256, 1000, 8), (129, 192, 777, 32), (64, 64, 256, 1), (300, 520, 5003, 20), (260, 128, 2000, 40),
                         (100, 256, 900, 64)):
        h, w, tok = make(T, H, V, seed=T + V, ldh=H + 8, ldw=H + 24)
        tok[3] = V + 1
        mask = (torch.arange(T, device="cuda") % 5 != 2).to(torch.uint8)
        swapped = check(ctx, h, w, tok, mask, k, np.arange(T))
        assert swapped <= T // 20, swapped
        check(ctx, h, w, tok, None, k, np.arange(0, T, 3))


def test_fused_output_layer_full_vocabulary(ctx):
    T, H, V, k = 1024, 2048, 151936, 20
    h, w, tok = make(T, H, V, seed=7)
    rows = np.concatenate([np.arange(0, 8), np.arange(500, 508), np.arange(T - 8, T)])
    swapped = check(ctx, h, w, tok, None, k, rows)
    print("rows whose list differs from the oracle's inside the bar:", swapped, "of", len(rows))
    # the same call again gives the same bits
    a = run(ctx, h, w, tok, None, k)
    b = run(ctx, h, w, tok, None, k)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_fused_output_layer_arguments(ctx):
    h, w, tok = make(16, 64, 300, seed=1)
    with pytest.raises(B.JackpotError, match="64"):
        run(ctx, h, w, tok, None, 65)
    hp = torch.zeros((16, 68), dtype=torch.bfloat16, device="cuda")[:, :64]       # pitch 136 bytes
    with pytest.raises(B.JackpotError, match="16 bytes"):
        run(ctx, hp, w, tok, None, 4)


# ---- the whole forward with both models' output layers fused ------------------------------------

def _two_models(T, V, Ha, Hp, seed, noise=1.0):
    """Actor and policy as hidden states and output matrices whose logits are N(0, 9) and differ by
    N(0, noise^2) (same hidden states, perturbed matrix) when the hidden sizes agree, unrelated otherwise."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    ha = torch.randn((T, Ha), generator=g, device="cuda").to(torch.bfloat16)
    wa = (torch.randn((V, Ha), generator=g, device="cuda") * (3.0 / Ha ** 0.5)).to(torch.bfloat16)
    if Hp == Ha:
        hp = ha.clone()
        wp = (wa.float() + torch.randn((V, Ha), generator=g, device="cuda") * (noise / Ha ** 0.5)).to(torch.bfloat16)
    else:
        hp = torch.randn((T, Hp), generator=g, device="cuda").to(torch.bfloat16)
        wp = (torch.randn((V, Hp), generator=g, device="cuda") * (3.0 / Hp ** 0.5)).to(torch.bfloat16)
    za = ha.float() @ wa.float().t()
    gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
    tok = (za + gum).argmax(1).to(torch.int32)               # a draw from (about) the actor's distribution
    return ha, wa, hp, wp, tok


def _check_fused_forward(ctx, ha, wa, hp, wp, tok, mask, rows, k, seed, lam=None, budget=None, c1=0.0, whole_batch=True):
    from paper_2602_06107_b200 import runner
    out = runner.forward_lmhead(ctx, ha, wa, hp, wp, tok, mask, lam=lam, budget=budget, k=k, seed=seed, c1=c1)
    assert out["stats"]["status"] == 0
    za = oracle.lmhead_rows(rows, to_numpy_bits(ha.contiguous()), to_numpy_bits(wa.contiguous()))
    zp = oracle.lmhead_rows(rows, to_numpy_bits(hp.contiguous()), to_numpy_bits(wp.contiguous()))
    m = None if mask is None else mask.cpu().numpy()[rows]
    lam_used = float(np.float32(out["stats"]["lambda_used"]))
    if budget is not None and whole_batch:
        ref_b = oracle.forward(za, zp, tok.cpu().numpy()[rows], m, budget=budget, k=k, seed=seed, c1=c1)
        assert abs(lam_used - ref_b["lambda"]) <= 2e-4 * ref_b["lambda"]      # the ratios carry the logits' 2e-5
    # everything else with lambda forced to the library's value; rows are consecutive from rows[0]
    ref = oracle.forward(za, zp, tok.cpu().numpy()[rows], m, lam=lam_used, k=k, seed=seed, c1=c1, token_offset=int(rows[0]))
    valid = (np.ones(len(rows), bool) if m is None else m != 0) & (ref["bad"] == 0)
    g = {n: t.cpu().numpy()[rows] for n, t in out.items() if isinstance(t, torch.Tensor) and t.shape[:1] == tok.shape}
    tol = lambda x, r=RTOL, a=ATOL: a + r * np.abs(x)
    for got, want in ((g["logp_actor"], ref["lq64"]), (g["logp_policy"], ref["lp64"]), (g["lse_actor"], ref["lse_a"]),
                      (g["lse_policy"], ref["lse_p"])):
        assert np.all(np.abs(got[valid] - want[valid]) <= tol(want[valid]))
    assert np.array_equal(g["uniform"], ref["u"])
    assert np.all(np.abs(g["accept_prob"] - ref["a"]) <= 1e-4 * np.maximum(ref["a"], 1e-3))
    flips = g["accept"] != ref["accept"]
    near = np.abs(ref["u"].astype(np.float64) - ref["a"]) < 1e-4
    assert not (flips & ~near).any()
    assert np.all(np.abs(g["z_approx"] - ref["zk"]) <= 1e-6 + 3e-4 * ref["zk"])
    same_lists = sum(int(np.array_equal(g["topk_idx_actor"][i], ref["topk_idx_a"][i]) and
                         np.array_equal(g["topk_idx_policy"][i], ref["topk_idx_p"][i])) for i in range(len(rows)) if valid[i])
    assert same_lists >= 0.9 * valid.sum(), (same_lists, valid.sum())
    assert np.all(g["weight"][~valid] == 0) and np.all(g["accept"][~valid] == 0)
    if whole_batch:
        st, rs = out["stats"], ref["stats"]
        assert st["n_valid"] == rs["n_valid"] and st["n_bad_token"] == rs["n_bad_token"]
        assert abs(st["z_approx_mean"] - rs["z_approx_mean"]) <= 3e-4 * rs["z_approx_mean"]
        assert abs(st["mean_accept_prob"] - rs["mean_accept_prob"]) <= 1e-4
        if not flips.any():
            assert abs(st["kappa"] - rs["kappa"]) <= 5e-4 * rs["kappa"]
            assert np.all(np.abs(g["weight"] - ref["w64"]) <= 1e-6 + 6e-4 * np.abs(ref["w64"]))
    return out


def test_fused_forward_small(ctx):
    for (T, V, Ha, Hp, k) in ((160, 3000, 256, 256, 16), (100, 777, 128, 192, 8), (200, 2000, 128, 128, 40)):
        ha, wa, hp, wp, tok = _two_models(T, V, Ha, Hp, seed=T)
        tok[5] = V + 2
        mask = (torch.arange(T, device="cuda") % 6 != 1).to(torch.uint8)
        rows = np.arange(T)
        _check_fused_forward(ctx, ha, wa, hp, wp, tok, mask, rows, k, seed=3, lam=1.3, c1=3.0)
        _check_fused_forward(ctx, ha, wa, hp, wp, tok, None, rows, k, seed=3, budget=0.6)
    # its records do not serve the backward
    from paper_2602_06107_b200 import runner
    ha, wa, hp, wp, tok = _two_models(32, 1024, 64, 64, seed=1)
    out = runner.forward_lmhead(ctx, ha, wa, hp, wp, tok, None, lam=1.0, k=8)
    z = torch.zeros((ha.shape[0], wa.shape[0]), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.JackpotError, match="without both logit tensors"):
        runner.backward(ctx, z, z, tok, None, out["accept"], out["weight"])


def test_fused_forward_full_vocabulary(ctx):
    T, V, H, k = 512, 151936, 1024, 20
    ha, wa, hp, wp, tok = _two_models(T, V, H, H, seed=9)
    rows = np.arange(200, 216)
    out = _check_fused_forward(ctx, ha, wa, hp, wp, tok, None, rows, k, seed=4, lam=1.0, whole_batch=False)
    st = out["stats"]
    assert st["n_valid"] == T and abs(st["kappa"] * st["z_approx_mean"] - st["alpha_hat"]) < 1e-12
