"""Seeded random sweep over the forward's parameter space: vocabulary widths from 40 to 70,000 columns
(ragged, padded pitch), both dtypes, k from 1 to 128, masks, out-of-range tokens, fixed lambda and
budget, weight clip, row offsets; every case element by element against the oracle at the usual bars
(dense forward; every fourth case also the sparse-actor forward; a dozen shapes of the fused output
layer).  It complements the hand-picked cases of the other files: whatever combination of tile
geometry, tail handling and list length a case lands on must agree with the oracle."""
import random

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


@pytest.mark.parametrize("seed", [11, 12])
def test_random_forward_cases_against_the_oracle(ctx, seed):
    from test_gpu_parity import check_forward, close
    import test_gpu_sparse_actor as sparse
    rng = random.Random(seed)
    done = 0
    for it in range(60):
        dt = rng.choice(["bf16", "f32"])
        al = 8 if dt == "bf16" else 4
        V = rng.choice([rng.randint(40, 300), rng.randint(300, 9000), rng.randint(9000, 70000)])
        ld = -(-V // al) * al + al * rng.choice([0, 0, 1, 3])
        T = rng.randint(1, 400 if V < 20000 else 60)
        k = min(rng.choice([1, 3, 8, 20, 32, 33, 64, 100, 128]), V - 1)
        r = LogitRecipe(T=T, V=ld, dtype=dt, sigma0=rng.choice([0.5, 2.0, 3.0]), peaks=rng.choice([0, 2, 8]), peak_lo=4.0,
                        peak_hi=12.0, sigma=rng.choice([0.1, 1.0, 2.0]), seed=rng.randint(0, 10 ** 6))
        zaf, zpf, _ = make_logits(r, "cuda")
        za, zp = zaf[:, :V], zpf[:, :V]
        g = torch.Generator(device="cuda").manual_seed(it)
        gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
        tok = (za.float() + gum).argmax(1).to(torch.int32)
        if rng.random() < 0.3 and T > 2:
            tok[rng.randrange(T)] = V + rng.randint(0, 5)
        mask = None if rng.random() < 0.4 else (torch.rand(T, generator=g, device="cuda") > 0.3).to(torch.uint8)
        kw = dict(lam=rng.choice([0.5, 1.0, 1.7])) if rng.random() < 0.6 else dict(budget=rng.choice([0.3, 0.6, 0.9, 1.0]))
        c1, rseed, off = rng.choice([0.0, 2.5]), rng.randint(0, 2 ** 40), rng.choice([0, 12345])
        m = None if mask is None else mask.cpu().numpy()
        ref = oracle.forward(to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous()), tok.cpu().numpy(), m, k=k,
                             seed=rseed, c1=c1, token_offset=off, **kw)
        if ref["stats"]["n_valid"] == 0 and "budget" in kw:
            continue
        lam = ref["lambda"]
        if "budget" in kw:                       # lambda first, then everything else with lambda forced to the oracle's
            o1 = runner.forward(ctx, za, zp, tok, mask, k=k, seed=rseed, c1=c1, token_offset=off, **kw)
            close(o1["stats"]["lambda_used"], lam)
        out = runner.forward(ctx, za, zp, tok, mask, lam=lam, k=k, seed=rseed, c1=c1, token_offset=off)
        ref["za_f32"], ref["zp_f32"] = za.float().cpu().numpy(), zp.float().cpu().numpy()
        check_forward(out, ref, k, V, m, c1)
        if it % 4 == 0 and V * (2 if dt == "bf16" else 4) % 16 == 0:
            k_inf = min(rng.choice([5, 20, 64, 128]), V)
            sparse.check(ctx, za.contiguous(), zp, tok, mask, k, k_inf, seed=rseed, cap=bool(it % 8), lam=lam, c1=c1)
        done += 1
    assert done >= 50


def test_random_fused_output_layer_cases_against_the_oracle(ctx):
    import test_gpu_lmhead as fused
    rng = random.Random(21)
    for it in range(12):
        T, H, V = rng.randint(1, 300), rng.choice([64, 72, 128, 200, 320]), rng.randint(70, 3000)
        k = min(rng.choice([1, 8, 20, 40, 64]), V - 1)
        h, w, tok = fused.make(T, H, V, seed=it, ldh=H + 8 * rng.randint(0, 2), ldw=H + 8 * rng.randint(0, 2))
        mask = None if it % 2 else (torch.arange(T, device="cuda") % 3 != 1).to(torch.uint8)
        fused.check(ctx, h, w, tok, mask, k, np.arange(T))


def test_random_backward_cases_against_the_oracle(ctx):
    """The fused gradients on random shapes (both dtypes, ragged widths, padded pitches, masks, in-place or
    not, with and without the distillation term) against the oracle's double gradients at the backward's bar."""
    from test_gpu_backward import check_grads
    rng = random.Random(31)
    for it in range(24):
        dt = rng.choice(["bf16", "f32"])
        V = rng.choice([rng.randint(40, 600), rng.randint(600, 20000)])
        ld = -(-V // 8) * 8 + 8 * rng.choice([0, 0, 2])                  # gradients are bf16: pitch in units of 8
        T = rng.randint(1, 120)
        k = min(rng.choice([4, 16, 32]), V - 1)
        r = LogitRecipe(T=T, V=ld, dtype=dt, sigma0=rng.choice([1.0, 2.5]), peaks=rng.choice([0, 4]), peak_lo=4.0, peak_hi=10.0,
                        sigma=rng.choice([0.3, 1.0]), seed=rng.randint(0, 10 ** 6))
        zaf, zpf, _ = make_logits(r, "cuda")
        za, zp = zaf[:, :V], zpf[:, :V]
        g = torch.Generator(device="cuda").manual_seed(100 + it)
        gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
        tok = (za.float() + gum).argmax(1).to(torch.int32)
        mask = None if rng.random() < 0.4 else (torch.rand(T, generator=g, device="cuda") > 0.25).to(torch.uint8)
        adv = None if rng.random() < 0.3 else torch.randn(T, generator=g, device="cuda")
        lam_d, gout = rng.choice([0.0, 1.0, 0.3]), rng.choice([1.0, 2.5])
        out = runner.forward(ctx, za, zp, tok, mask, lam=rng.choice([0.7, 1.3]), k=k, seed=it, c1=rng.choice([0.0, 3.0]))
        if out["stats"]["n_valid"] == 0:
            continue
        za_np, zp_np = to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous())
        in_place = dt == "bf16" and rng.random() < 0.3
        za_in = za.clone() if in_place else za                       # the in-place call overwrites its logits
        zp_in = zp.clone() if in_place else zp
        if in_place:
            zfa, zfp = zaf.clone(), zpf.clone()
            za_in, zp_in = zfa[:, :V], zfp[:, :V]
        da, dp = runner.backward(ctx, za_in, zp_in, tok, mask, out["accept"], out["weight"], advantages=adv,
                                 lambda_distill=lam_d, grad_out=gout, d_actor=za_in if in_place else None,
                                 d_policy=zp_in if in_place else None)
        torch.cuda.synchronize()
        m = None if mask is None else mask.cpu().numpy()
        lg = oracle.lse_gather(za_np, zp_np, tok.cpu().numpy(), m)
        rows = np.arange(T)
        check_grads(da, dp, rows, za_np, zp_np, tok.cpu().numpy(), m, out["accept"].cpu().numpy(),
                    out["weight"].cpu().numpy(), lg["lse_a"], lg["lse_p"], out["stats"]["n_valid"],
                    None if adv is None else adv.cpu().numpy(), lam_d, g=gout)
