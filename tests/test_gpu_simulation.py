"""The paper's numerical simulation as a tested workload (Section 3.2, Theorems 3.3 and 3.4): pairs of
distributions drawn from a Dirichlet at growing distance go through the forward pass (fixed
lambda = 1, exact mode and top-k mode) and through the per-distribution budget solve, on the GPU and in
the oracle, at the usual bars.  The paper gives no parameters for its figure, so these are free; what
is asserted beside parity are the trends the figure shows, on the oracle's numbers: the acceptance
rate falls as the divergence grows, and rejection never increases the divergence to the target."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200 import runner
from paper_2602_06107_b200.inputs import make_dirichlet_logits, to_numpy_bits

pytestmark = pytest.mark.gpu
RTOL, ATOL = 1e-5, 1e-6
NOISES = (0.1, 0.25, 0.5, 1.0, 1.5)


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


@pytest.mark.parametrize("dtype,V", [("f32", 8192), ("bf16", 32768)])
def test_dirichlet_pairs_forward_and_row_budget(ctx, dtype, V):
    T, k, budget = 96, 20, 0.9
    acc_rate, kl_before, kl_after = [], [], []
    for i, noise in enumerate(NOISES):
        za, zp, tok = make_dirichlet_logits(T, V, 0.3, noise, seed=7 + i, dtype=dtype, device="cuda")
        za_h, zp_h, tok_h = to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy()
        # forward at the paper's default lambda = 1: exact normaliser beside the top-k estimate
        out = runner.forward(ctx, za, zp, tok, None, lam=1.0, k=k, seed=11, want_exact=True)
        ref = oracle.forward(za_h, zp_h, tok_h, None, lam=1.0, k=k, seed=11, exact=True)
        assert np.array_equal(out["topk_idx_actor"].cpu().numpy(), ref["topk_idx_a"])
        assert np.array_equal(out["topk_idx_policy"].cpu().numpy(), ref["topk_idx_p"])
        close(out["logp_actor"].cpu().numpy(), ref["lq64"])
        close(out["logp_policy"].cpu().numpy(), ref["lp64"])
        close(out["accept_prob"].cpu().numpy(), ref["a"])
        close(out["z_approx"].cpu().numpy(), ref["zk"])
        close(out["z_exact"].cpu().numpy(), ref["z_exact"])
        assert np.array_equal(out["uniform"].cpu().numpy(), ref["u"])
        diff = out["accept"].cpu().numpy() != ref["accept"]
        near = np.abs(ref["u"].astype(np.float64) - ref["a"]) < 1e-6
        assert not (diff & ~near).any()
        # the per-distribution budget (Theorem 3.4) and the divergences before / after (Theorem 3.3)
        lam = torch.empty(T, device="cuda")
        kb, ka = torch.empty(T, device="cuda"), torch.empty(T, device="cuda")
        B.jp_obrs_row_lambda(ctx, B.make_desc(za), za, zp, None, budget, lam, kb, ka, None)
        torch.cuda.synchronize()
        rl = oracle.row_lambda(za_h, zp_h, budget)
        close(lam.cpu().numpy(), rl["lam"], rtol=1e-5, atol=0)
        close(kb.cpu().numpy(), rl["kl_before"], rtol=1e-4, atol=5e-6)
        close(ka.cpu().numpy(), rl["kl_after"], rtol=1e-4, atol=5e-6)
        acc_rate.append(ref["z_exact"].mean())          # Z = expected acceptance rate (Section 4.4.2)
        kl_before.append(rl["kl_before"].mean())
        kl_after.append(rl["kl_after"].mean())
        assert np.all(rl["kl_after"] <= rl["kl_before"] + 1e-12)          # Theorem 3.3, row by row
    # the figure's trends, on the oracle's numbers
    assert all(a < b for a, b in zip(kl_before, kl_before[1:])), kl_before   # the pairs do move apart
    assert all(a > b for a, b in zip(acc_rate, acc_rate[1:])), acc_rate      # acceptance falls as KL grows
    assert all(a < b for a, b in zip(kl_after, kl_before)), (kl_after, kl_before)
    print("KL(p||q)", [f"{x:.4f}" for x in kl_before], "acceptance at lambda=1", [f"{x:.3f}" for x in acc_rate],
          "KL(p||kept) at budget 0.9", [f"{x:.4f}" for x in kl_after])
