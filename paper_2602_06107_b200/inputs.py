"""Seeded synthetic LLM-shaped logits: the only module shared by the CUDA path's
tests/benchmark and the CPU oracle's tests.  It holds none of the method's
arithmetic: it draws numbers, adds them, rounds them to the storage dtype and
picks tokens with the Gumbel-max trick (an argmax over perturbed logits, which
samples from the softmax without computing it).

Recipe (one row = one token position):
  policy  zp = N(0, sigma0^2) i.i.d. over the vocabulary, plus ``peaks`` distinct
          columns per row (one per equal-width stratum of the vocabulary) boosted
          by U(peak_lo, peak_hi) -- a heavy head over a broad Gaussian body, the
          shape of a language model's next-token logits;
  actor   za = zp + N(0, sigma^2)   (the rollout model disagrees with the policy;
          peaks are inherited);
  both are rounded to the storage dtype before anything reads them;
  tokens  x_t ~ softmax(za[t, :]) by Gumbel-max on the rounded actor logits.
Rows are generated in blocks so a [T, 151936] tensor never needs fp32 temporaries
larger than ``block_rows`` rows.  CPU and CUDA generators give different bits
for the same seed; a test always hands the *same bits* to both sides.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class LogitRecipe:
    T: int
    V: int
    dtype: str = "bf16"          # "bf16" | "f32"
    sigma0: float = 3.0          # std of the policy's Gaussian body
    peaks: int = 8               # boosted columns per row
    peak_lo: float = 8.0
    peak_hi: float = 15.0
    sigma: float = 1.0           # std of actor - policy noise
    seed: int = 0


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[name]


def make_logits(r: LogitRecipe, device="cpu", block_rows: int = 256, rows=None):
    """Returns (actor_logits, policy_logits, tokens) on ``device``.

    ``rows`` = (start, stop) generates only that row range of the T-row problem
    with the bits the full call would give for those rows when the range is a
    whole number of blocks (each block draws from its own seeded stream).
    """
    dt = torch_dtype(r.dtype)
    lo, hi = (0, r.T) if rows is None else rows
    n = hi - lo
    za = torch.empty((n, r.V), dtype=dt, device=device)
    zp = torch.empty((n, r.V), dtype=dt, device=device)
    tok = torch.empty((n,), dtype=torch.int32, device=device)
    assert lo % block_rows == 0 or n <= block_rows
    for b0 in range(lo, hi, block_rows):
        b1 = min(b0 + block_rows, hi)
        m = b1 - b0
        g = torch.Generator(device=device)
        g.manual_seed((r.seed * 1_000_003 + b0) & 0x7FFFFFFFFFFFFFFF)
        pol = torch.randn((m, r.V), generator=g, device=device, dtype=torch.float32) * r.sigma0
        if r.peaks > 0:
            strata = torch.arange(r.peaks, device=device, dtype=torch.float32)
            frac = torch.rand((m, r.peaks), generator=g, device=device)
            cols = ((strata + frac) * (r.V / r.peaks)).long().clamp_(0, r.V - 1)
            boost = r.peak_lo + (r.peak_hi - r.peak_lo) * torch.rand((m, r.peaks), generator=g, device=device)
            pol.scatter_add_(1, cols, boost)
        act = pol + torch.randn((m, r.V), generator=g, device=device, dtype=torch.float32) * r.sigma
        zp[b0 - lo:b1 - lo] = pol.to(dt)
        za_blk = act.to(dt)
        za[b0 - lo:b1 - lo] = za_blk
        u = torch.rand((m, r.V), generator=g, device=device, dtype=torch.float32).clamp_(1e-30, 1.0 - 1e-7)
        gumbel = -torch.log(-torch.log(u))
        tok[b0 - lo:b1 - lo] = (za_blk.float() + gumbel).argmax(dim=1).to(torch.int32)
    return za, zp, tok


def make_dirichlet_logits(T: int, V: int, concentration: float, noise: float, seed: int, dtype="f32", device="cpu"):
    """Simulated distribution pairs in the manner of the paper's numerical simulation: every row of the
    policy is a draw from a symmetric Dirichlet (as log-probabilities, from Gamma draws), the actor is the
    same row with Gaussian noise of scale ``noise`` added to the log-probabilities, which sets how far the
    two distributions are apart.  The paper states no parameters for its figure; these are free."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    conc = torch.full((T, V), float(concentration), device=device)
    gam = torch._standard_gamma(conc, generator=g).clamp_min_(1e-30)
    logp = torch.log(gam)
    logp = logp - torch.logsumexp(logp, dim=1, keepdim=True)
    act = logp + noise * torch.randn((T, V), generator=g, device=device)
    dt = torch_dtype(dtype)
    zp, za = logp.to(dt), act.to(dt)
    u = torch.rand((T, V), generator=g, device=device).clamp_(1e-30, 1.0 - 1e-7)
    tok = (za.float() - torch.log(-torch.log(u))).argmax(dim=1).to(torch.int32)
    return za, zp, tok


def make_lengths_mask(n_resp: int, max_len: int, min_len: int, seed: int, device="cpu"):
    """Padded batch layout: ``n_resp`` responses with lengths U{min_len..max_len},
    each padded to ``max_len``; returns (mask[n_resp*max_len] uint8, lengths)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    lengths = torch.randint(min_len, max_len + 1, (n_resp,), generator=g)
    pos = torch.arange(max_len).unsqueeze(0)
    mask = (pos < lengths.unsqueeze(1)).to(torch.uint8).reshape(-1)
    return mask.to(device), lengths


def to_numpy_bits(z: torch.Tensor):
    """Host copy in the form the oracle takes: bf16 as uint16 bit patterns, fp32 as is."""
    z = z.detach().cpu().contiguous()
    if z.dtype == torch.bfloat16:
        return z.view(torch.int16).numpy().view("uint16")
    return z.numpy()


# The five workload shapes this build is measured and tested on.  "full" sizes are
# those of the benchmark; tests also use scaled-down T with the same V / dtype / k.
CONFIGS = {
    "cfg1_tiny": dict(recipe=LogitRecipe(T=256, V=4096, dtype="f32", sigma0=2.0, peaks=4, peak_lo=6.0,
                                         peak_hi=12.0, sigma=0.5, seed=0), k=16, lam=1.5, seed=0),
    "cfg2_qwen3": dict(recipe=LogitRecipe(T=4096, V=151936, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0,
                                          peak_hi=15.0, sigma=1.0, seed=1), k=32, lam=2.0, seed=1),
    "cfg3_batch": dict(recipe=LogitRecipe(T=131072, V=151936, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0,
                                          peak_hi=15.0, sigma=1.5, seed=2), k=64, budget=0.6, seed=2,
                       n_resp=64, max_len=2048, min_len=256, chunk=8192),
    "cfg4_sweep": dict(recipe=LogitRecipe(T=16384, V=151936, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0,
                                          peak_hi=15.0, sigma=1.0, seed=3), ks=(8, 32, 128, 151936),
                       sigmas=(0.25, 1.0, 2.0), lam=1.0, seed=3),
    "cfg5_train": dict(recipe=LogitRecipe(T=32768, V=151936, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0,
                                          peak_hi=15.0, sigma=1.0, seed=4), k=64, budget=0.5, seed=4,
                       chunk=8192, lambda_distill=1.0, c1=3.0),
}
