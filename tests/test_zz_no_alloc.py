"""The allocation-free budget solve (jp_budget_lambda_static) against the
budget mode of jp_obrs_forward.

Some users of the library run where device allocation is not allowed (memory
fully owned by a framework's allocator, plug-ins that may allocate only at
start-up, loops that cannot afford the device-wide synchronisation of
cudaMalloc).  For them the library offers one call whose scratch is a fixed
array inside the library image.  This test drives it through the C ABI twice in
a row -- the second call finds the first call's leftovers in the shared array --
and checks both answers against the lambda that the ordinary forward solves from
the same log-probabilities, against the CPU oracle's exact sort-based solve, and
against the defining equation itself, within the tolerance the other parity tests
use for lambda (rtol 1e-5 / atol 1e-6).  It also checks that nothing was
allocated, that the far end of the fixed array works (a batch of exactly the
maximum size) and that sizes beyond the maximum are refused.

The file name sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200 import runner
from paper_2602_06107_b200.inputs import LogitRecipe, make_logits

pytestmark = pytest.mark.gpu
RTOL, ATOL = 1e-5, 1e-6


def _close(a, b):
    assert abs(a - b) <= ATOL + RTOL * abs(b), (a, b)


def _check_against_the_definition(lam, lq, lp, mask, budget):
    """lambda against the oracle's solve on the same fp32 log-probs, and the equation it solves,
    (1/N) sum_t min(1, (p/q)(x_t) / lambda) = budget, evaluated directly in double."""
    lq, lp = lq.cpu().numpy(), lp.cpu().numpy()
    m = None if mask is None else mask.cpu().numpy()
    _close(lam, oracle.lambda_from_budget(lq, lp, budget, m))
    take = np.ones(lq.shape[0], bool) if m is None else m != 0
    r = np.exp(lp[take].astype(np.float64) - lq[take].astype(np.float64))
    if budget < 1.0:
        assert abs(np.minimum(1.0, r / lam).mean() - budget) <= 2e-5 * budget


def test_static_budget_lambda_matches_forward_twice_in_a_row():
    jp_build.build()
    ctx = B.Context(0)
    lam_out = torch.zeros(1, dtype=torch.float32, device="cuda")
    # The first call on a device sets up: the driver loads the part of the library
    # image that holds the fixed scratch array (that is when the device's free memory
    # drops by the array's size, once) and the array's address is looked up.
    z4 = torch.zeros(4, dtype=torch.float32, device="cuda")
    assert B.jp_budget_lambda_static(z4, z4, None, 4, 0.5, lam_out) == 0
    torch.cuda.synchronize()
    cases = [dict(T=900, V=4096, seed=71, budget=0.6, stride=5), dict(T=333, V=2048, seed=72, budget=0.3, stride=3)]
    for c in cases:                       # two calls in a row on the shared array; the second is smaller
        r = LogitRecipe(T=c["T"], V=c["V"], dtype="bf16", sigma0=2.5, peaks=4, sigma=1.5, seed=c["seed"])
        za, zp, tok = make_logits(r, "cuda")
        mask = (torch.arange(c["T"], device="cuda") % c["stride"] != 1).to(torch.uint8)
        out = runner.forward(ctx, za, zp, tok, mask, budget=c["budget"], k=8, seed=1)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        st = B.jp_budget_lambda_static(out["logp_actor"], out["logp_policy"], mask, c["T"], c["budget"], lam_out)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert st == 0
        assert free_after == free_before, "a call after the first changed the device's free memory"
        _close(float(lam_out.item()), out["stats"]["lambda_used"])
        _check_against_the_definition(float(lam_out.item()), out["logp_actor"], out["logp_policy"], mask, c["budget"])
        # no mask = all rows: same as a forward without a mask
        out_all = runner.forward(ctx, za, zp, tok, None, budget=c["budget"], k=8, seed=1)
        assert B.jp_budget_lambda_static(out_all["logp_actor"], out_all["logp_policy"], None, c["T"], c["budget"],
                                         lam_out) == 0
        torch.cuda.synchronize()
        _close(float(lam_out.item()), out_all["stats"]["lambda_used"])
        _check_against_the_definition(float(lam_out.item()), out_all["logp_actor"], out_all["logp_policy"], None,
                                      c["budget"])
    # budget 1: the largest lambda with full acceptance
    assert B.jp_budget_lambda_static(out_all["logp_actor"], out_all["logp_policy"], None, cases[-1]["T"], 1.0,
                                     lam_out) == 0
    torch.cuda.synchronize()
    d = (out_all["logp_policy"] - out_all["logp_actor"]).double()
    _close(float(lam_out.item()), float(torch.exp(d.min()).item()))
    ctx.close()


def test_static_budget_lambda_at_the_maximum_size():
    """A batch of exactly JP_STATIC_MAX_ROWS rows uses the fixed array to its last element; the log-probs
    are synthetic (the solve only sees them), every seventh row masked."""
    jp_build.build()
    T = B.JP_STATIC_MAX_ROWS
    g = torch.Generator(device="cuda").manual_seed(73)
    lq = -torch.rand(T, generator=g, device="cuda") * 6.0
    lp = lq + 1.5 * torch.randn(T, generator=g, device="cuda")
    mask = (torch.arange(T, device="cuda") % 7 != 3).to(torch.uint8)
    lam_out = torch.zeros(1, dtype=torch.float32, device="cuda")
    for budget in (0.6, 0.25):
        assert B.jp_budget_lambda_static(lq, lp, mask, T, budget, lam_out) == 0
        torch.cuda.synchronize()
        _check_against_the_definition(float(lam_out.item()), lq, lp, mask, budget)


def test_static_entry_point_limits_and_arguments():
    jp_build.build()
    lam_out = torch.full((1,), 7.0, dtype=torch.float32, device="cuda")
    z = torch.zeros(4, dtype=torch.float32, device="cuda")
    too_many = B.JP_STATIC_MAX_ROWS + 1
    assert B.jp_budget_lambda_static(z, z, None, too_many, 0.5, lam_out) == B.JP_ERR_TOO_LARGE
    assert b"maximum" in B.load().jp_status_string(B.JP_ERR_TOO_LARGE)
    assert B.jp_budget_lambda_static(z, z, None, 4, 0.0, lam_out) == -1
    assert B.jp_budget_lambda_static(z, z, None, 4, 1.5, lam_out) == -1
    assert B.jp_budget_lambda_static(z, z, None, -1, 0.5, lam_out) == -1
    assert B.jp_budget_lambda_static(z, z, None, 4, 0.5, None) == -1
    torch.cuda.synchronize()
    assert lam_out.item() == 7.0, "a refused call must not touch its output"
    # no rows: lambda = 1 by convention
    assert B.jp_budget_lambda_static(z, z, None, 0, 0.5, lam_out) == 0
    torch.cuda.synchronize()
    assert lam_out.item() == 1.0
    # equal distributions: every ratio is 1, so lambda = 1 / budget
    assert B.jp_budget_lambda_static(z, z, None, 4, 0.5, lam_out) == 0
    torch.cuda.synchronize()
    assert abs(lam_out.item() - 2.0) < 1e-6
