"""GPU parity of jp_obrs_forward_sparse_actor against the oracle: the forward with the rollout model
known only through the record Algorithm 1 Phase 1 stores (log p_inf(a_t) and the top-k_inf
log-probabilities), Phase 2 step 2's Z_approx over TopK_inf U TopK_new in both readings of the
entries the record does not hold.  Bars as for the dense path: lists, uniforms and accept bits
bit-exact (accept bits may differ only where |u - a| < 1e-6), everything else rtol 1e-5 / atol 1e-6."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200 import runner
from paper_2602_06107_b200.inputs import LogitRecipe, make_logits, to_numpy_bits

pytestmark = pytest.mark.gpu
RTOL, ATOL = 1e-5, 1e-6


@pytest.fixture(scope="module")
def ctx():
    jp_build.build()
    c = B.Context(0)
    yield c
    c.close()


def close(a, b, rtol=RTOL, atol=ATOL):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    bad = np.abs(a - b) > atol + rtol * np.abs(b)
    assert not bad.any(), f"{bad.sum()} of {bad.size} differ; worst {np.abs(a - b).max():.3e}"


def record_of(za, tok, k_inf, mask=None):
    """The rollout record, made on the CPU by the oracle from the actor's logits, then handed to both sides."""
    m = None if mask is None else mask.cpu().numpy()
    lq, idx, logp = oracle.rollout_record(to_numpy_bits(za), tok.cpu().numpy(), k_inf, m)
    dev = za.device
    return (lq, idx, logp), (torch.from_numpy(lq).to(dev), torch.from_numpy(idx).to(dev), torch.from_numpy(logp).to(dev))


def check(ctx, za, zp, tok, mask, k, k_inf, seed, cap, c1=0.0, lam=None, budget=None, token_offset=0):
    (lq, idx, logp), (d_lq, d_idx, d_logp) = record_of(za, tok, k_inf, mask)
    zp_h, tok_h = to_numpy_bits(zp.contiguous()), tok.cpu().numpy()
    m = None if mask is None else mask.cpu().numpy()
    ref = oracle.forward_sparse(zp_h, tok_h, lq, idx, logp, m, lam=lam, budget=budget, k=k, seed=seed, c1=c1, cap=cap,
                                token_offset=token_offset)
    if budget is not None:
        out = runner.forward_sparse_actor(ctx, zp, tok, mask, d_lq, d_idx, d_logp, budget=budget, k=k, seed=seed, c1=c1,
                                          cap=cap, token_offset=token_offset)
        close(out["stats"]["lambda_used"], ref["lambda"])
        lam = ref["lambda"]                   # then everything else with lambda forced to the oracle's value
    out = runner.forward_sparse_actor(ctx, zp, tok, mask, d_lq, d_idx, d_logp, lam=lam, k=k, seed=seed, c1=c1, cap=cap,
                                      token_offset=token_offset)
    T = zp.shape[0]
    valid = (np.ones(T, bool) if m is None else m != 0) & (ref["bad"] == 0)
    g = {n: t.cpu().numpy() for n, t in out.items() if isinstance(t, torch.Tensor)}
    assert np.array_equal(g["topk_idx_policy"][valid], ref["topk_idx_p"][valid])
    assert np.all(g["topk_idx_policy"][~valid] == -1)
    zp_f = zp.float().cpu().numpy()
    assert np.array_equal(g["topk_val_policy"][valid], zp_f[np.nonzero(valid)[0][:, None], ref["topk_idx_p"][valid]])
    close(g["lse_policy"][valid], ref["lse_p"][valid])
    close(g["logp_policy"], ref["lp64"])
    assert np.array_equal(g["uniform"], ref["u"])
    close(g["accept_prob"], ref["a"])
    diff = g["accept"] != ref["accept"]
    near = np.abs(ref["u"].astype(np.float64) - ref["a"].astype(np.float64)) < 1e-6
    assert not (diff & ~near).any()
    close(g["z_lower"], ref["z_lo"])
    close(g["z_upper"], ref["z_hi"])
    close(g["z_approx"], ref["zk"])
    assert np.all(g["z_lower"] <= g["z_upper"] * (1 + 1e-6))
    st, rs = out["stats"], ref["stats"]
    assert st["n_valid"] == rs["n_valid"] and st["n_bad_token"] == rs["n_bad_token"] and st["status"] == 0
    close(st["z_approx_mean"], rs["z_approx_mean"])
    close(st["mean_accept_prob"], rs["mean_accept_prob"])
    if not diff.any():
        close(st["kappa"], rs["kappa"])
        close(g["weight"], ref["w64"])
    assert np.all(g["weight"][~valid] == 0) and np.all(g["accept"][~valid] == 0)
    return out, ref


@pytest.mark.parametrize("cap", [False, True])
def test_sparse_actor_small_shapes(ctx, cap):
    for dt, V, ld, k, k_inf in (("bf16", 20000, 20000, 12, 20), ("f32", 4099, 4100, 40, 7), ("bf16", 5003, 5008, 100, 128)):
        T = 120
        r = LogitRecipe(T=T, V=ld, dtype=dt, sigma0=2.5, peaks=4, sigma=1.1, seed=81)
        zaf, zpf, _ = make_logits(r, "cuda")
        za, zp = zaf[:, :V].contiguous(), zpf[:, :V]
        g = torch.Generator(device="cuda").manual_seed(6)
        gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
        tok = (za.float() + gum).argmax(1).to(torch.int32)
        tok[7] = V + 3                                       # a token id outside the vocabulary
        mask = (torch.arange(T, device="cuda") % 6 != 2).to(torch.uint8)
        check(ctx, za, zp, tok, mask, k, k_inf, seed=3, cap=cap, lam=1.3, c1=3.0, token_offset=500)
        check(ctx, za, zp, tok, None, k, k_inf, seed=3, cap=cap, budget=0.6)


@pytest.mark.parametrize("k,k_inf", [(20, 20), (64, 32), (128, 128)])
def test_sparse_actor_full_vocabulary(ctx, k, k_inf):
    r = LogitRecipe(T=64, V=151936, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0, peak_hi=15.0, sigma=1.0, seed=82 + k)
    za, zp, tok = make_logits(r, "cuda")
    out, ref = check(ctx, za, zp, tok, None, k, k_inf, seed=9, cap=False, lam=1.0)
    # against the dense forward on the same rows: same decisions whenever the stored log p_inf(a_t) rounds like
    # the dense path's, and a Z that the dense estimate brackets
    dense = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=max(k, k_inf), seed=9)
    assert np.all(out["z_lower"].cpu().numpy() <= dense["z_approx"].cpu().numpy() * (1 + 1e-5) + 1e-6)


def test_sparse_actor_with_everything_stored_is_the_exact_forward(ctx):
    T, V = 90, 128
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.0, peaks=3, sigma=0.8, seed=83)
    za, zp, tok = make_logits(r, "cuda")
    (lq, idx, logp), (d_lq, d_idx, d_logp) = record_of(za, tok, V)
    dense = runner.forward(ctx, za, zp, tok, None, lam=1.4, k=V, seed=2)
    for cap in (False, True):
        sp = runner.forward_sparse_actor(ctx, zp, tok, None, d_lq, d_idx, d_logp, lam=1.4, k=16, seed=2, cap=cap)
        close(sp["z_approx"].cpu().numpy(), dense["z_approx"].cpu().numpy(), rtol=3e-6)
        assert torch.equal(sp["uniform"], dense["uniform"])
        close(sp["accept_prob"].cpu().numpy(), dense["accept_prob"].cpu().numpy(), rtol=3e-6)
    # the records of this call do not serve the backward
    with pytest.raises(B.JackpotError, match="sparse"):
        runner.backward(ctx, za, zp, tok, None, sp["accept"], sp["weight"])
    # argument checks
    with pytest.raises(B.JackpotError, match="k_inf"):
        runner.forward_sparse_actor(ctx, zp, tok, None, d_lq, d_idx[:, :0].contiguous(), d_logp[:, :0].contiguous(),
                                    lam=1.0, k=8)
    with pytest.raises(B.JackpotError, match="k < V"):
        runner.forward_sparse_actor(ctx, zp, tok, None, d_lq, d_idx, d_logp, lam=1.0, k=V)
