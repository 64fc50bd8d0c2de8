"""GPU parity of jp_obrs_row_lambda (Theorem 3.4 per distribution) against the oracle.

Bars: lambda_t within rtol 1e-5 of the oracle's exact sort-based solve, the bar of every other
lambda in this library (the root is ill-conditioned at budgets near 1, where most of the accepted
mass sits on capped entries, so the kernel takes its normalisers and its last step in double);
both KL values within rtol 1e-4 / atol 5e-6 (sums of V fp32 terms with cancellation against the
log-sum-exps)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200.inputs import LogitRecipe, make_logits, to_numpy_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    jp_build.build()
    c = B.Context(0)
    yield c
    c.close()


def run(ctx, za, zp, mask, budget):
    T = za.shape[0]
    lam = torch.empty(T, device="cuda")
    kb = torch.empty(T, device="cuda")
    ka = torch.empty(T, device="cuda")
    it = torch.empty(T, dtype=torch.int32, device="cuda")
    B.jp_obrs_row_lambda(ctx, B.make_desc(za), za, zp, mask, budget, lam, kb, ka, it)
    torch.cuda.synchronize()
    return lam.cpu().numpy(), kb.cpu().numpy(), ka.cpu().numpy(), it.cpu().numpy()


@pytest.mark.parametrize("dtype,V", [("bf16", 20000), ("f32", 4099), ("bf16", 151936)])
@pytest.mark.parametrize("budget", [0.3, 0.7, 0.95, 0.995])
def test_row_lambda_matches_oracle(ctx, dtype, V, budget):
    T = 24 if V > 100000 else 96
    ld = (V + 7) // 8 * 8
    r = LogitRecipe(T=T, V=ld, dtype=dtype, sigma0=2.5, peaks=4, sigma=1.2, seed=41)
    zaf, zpf, _ = make_logits(r, "cuda")
    za, zp = zaf[:, :V], zpf[:, :V]
    mask = (torch.arange(T, device="cuda") % 6 != 4).to(torch.uint8)
    lam, kb, ka, it = run(ctx, za, zp, mask, budget)
    ref = oracle.row_lambda(to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous()), budget,
                            mask=mask.cpu().numpy())
    assert np.allclose(lam, ref["lam"], rtol=1e-5, atol=0), np.abs(lam / np.maximum(ref["lam"], 1e-30) - 1).max()
    assert np.allclose(kb, ref["kl_before"], rtol=1e-4, atol=5e-6)
    assert np.allclose(ka, ref["kl_after"], rtol=1e-4, atol=5e-6)
    valid = mask.cpu().numpy() != 0
    assert np.all(lam[~valid] == 0) and np.all(it[~valid] == 0)
    assert it[valid].max() < 24, "Newton must end well inside its limit of 48 steps (0 steps: no entry reaches its cap)"
    assert np.all(ka[valid] <= kb[valid] + 1e-5)              # Theorem 3.3


def test_row_lambda_special_cases(ctx):
    r = LogitRecipe(T=16, V=4096, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.0, seed=42)
    za, zp, _ = make_logits(r, "cuda")
    # p == q: Z(lambda) = min(1, 1/lambda), so lambda = 1 / budget and nothing changes
    lam, kb, ka, _ = run(ctx, za, za, None, 0.4)
    assert np.allclose(lam, 2.5, rtol=1e-5) and np.allclose(kb, 0, atol=5e-6) and np.allclose(ka, 0, atol=5e-6)
    # budget 1: the smallest ratio p/q
    lam, _, _, _ = run(ctx, za, zp, None, 1.0)
    ref = oracle.row_lambda(to_numpy_bits(za), to_numpy_bits(zp), 1.0)
    assert np.allclose(lam, ref["lam"], rtol=1e-5)
    with pytest.raises(B.JackpotError, match="budget"):
        run(ctx, za, zp, None, 0.0)
    with pytest.raises(B.JackpotError, match="budget"):
        run(ctx, za, zp, None, 1.5)
