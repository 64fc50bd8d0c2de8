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
    for (T, H, V, k) in ((200, 256, 1000, 8), (129, 192, 777, 32), (64, 64, 256, 1), (300, 520, 5003, 20)):
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
    with pytest.raises(B.JackpotError, match="32"):
        run(ctx, h, w, tok, None, 33)
    hp = torch.zeros((16, 68), dtype=torch.bfloat16, device="cuda")[:, :64]       # pitch 136 bytes
    with pytest.raises(B.JackpotError, match="16 bytes"):
        run(ctx, hp, w, tok, None, 4)
