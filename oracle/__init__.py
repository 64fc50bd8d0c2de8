"""CPU oracle for the OBRS token pass (TEST INFRASTRUCTURE ONLY).

A thin ctypes loader around ``obrs_oracle.cpp`` plus :func:`forward`, which
strings the oracle's steps together in the paper's order (log-softmax and
gathers, the two top-k lists, lambda, acceptance and decision, Z_approx and
exact Z, batch correction, weights).  Only tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the product path never
does, and this package never imports the CUDA path.

Arrays are numpy.  bf16 logits travel as ``uint16`` bit patterns
(``dtype="bf16"``); fp32 logits as ``float32``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "obrs_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

BF16, F32 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math: summation order is part of it)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC]
    subprocess.run(cmd, check=True)
    return _LIB


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _vp(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.jo_uniform.restype = ctypes.c_float
        _lib.jo_uniform.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        _lib.jo_lambda_from_budget.restype = ctypes.c_double
        _lib.jo_loss.restype = ctypes.c_double
        _lib.jo_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().jo_num_threads())


def set_num_threads(n: int) -> None:
    lib().jo_set_num_threads(ctypes.c_int(n))


def _dtype_code(z: np.ndarray) -> int:
    if z.dtype == np.uint16:
        return BF16
    if z.dtype == np.float32:
        return F32
    raise TypeError("logits must be uint16 (bf16 bits) or float32")


def _check2d(z):
    assert z.ndim == 2 and z.flags.c_contiguous
    return z.shape[0], z.shape[1]


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().jo_philox4x32_10(_p(c, ctypes.c_uint32), _p(k, ctypes.c_uint32), _p(out, ctypes.c_uint32))
    return out


def uniform(seed: int, g: int) -> float:
    return float(lib().jo_uniform(ctypes.c_uint64(seed), ctypes.c_uint64(g)))


def lse_gather(za, zp, tokens, mask=None):
    T, V = _check2d(za)
    dt = _dtype_code(za)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    out = dict(lse_a=np.zeros(T), lse_p=np.zeros(T), lq64=np.zeros(T), lp64=np.zeros(T),
               lq=np.zeros(T, np.float32), lp=np.zeros(T, np.float32), bad=np.zeros(T, np.uint8))
    lib().jo_lse_gather(ctypes.c_int64(T), ctypes.c_int64(V), ctypes.c_int64(V), ctypes.c_int(dt),
                        _vp(za), _vp(zp), _p(tokens, ctypes.c_int32), _p(mask, ctypes.c_uint8),
                        _p(out["lse_a"], ctypes.c_double), _p(out["lse_p"], ctypes.c_double),
                        _p(out["lq64"], ctypes.c_double), _p(out["lp64"], ctypes.c_double),
                        _p(out["lq"], ctypes.c_float), _p(out["lp"], ctypes.c_float),
                        _p(out["bad"], ctypes.c_uint8))
    return out


def topk(z, k, mask=None):
    T, V = _check2d(z)
    idx = np.zeros((T, k), dtype=np.int32)
    lib().jo_topk(ctypes.c_int64(T), ctypes.c_int64(V), ctypes.c_int64(V), ctypes.c_int(_dtype_code(z)),
                  _vp(z), _p(mask, ctypes.c_uint8), ctypes.c_int(k), _p(idx, ctypes.c_int32))
    return idx


def lambda_from_budget(lq, lp, budget, mask=None, bad=None):
    lq = np.ascontiguousarray(lq, np.float32)
    lp = np.ascontiguousarray(lp, np.float32)
    return float(lib().jo_lambda_from_budget(ctypes.c_int64(lq.shape[0]), _p(lq, ctypes.c_float),
                                             _p(lp, ctypes.c_float), _p(mask, ctypes.c_uint8),
                                             _p(bad, ctypes.c_uint8), ctypes.c_double(budget)))


def accept(lq, lp, lam, seed, token_offset=0, mask=None, bad=None):
    T = lq.shape[0]
    a = np.zeros(T, np.float32)
    u = np.zeros(T, np.float32)
    acc = np.zeros(T, np.uint8)
    lib().jo_accept(ctypes.c_int64(T), _p(lq, ctypes.c_float), _p(lp, ctypes.c_float),
                    _p(mask, ctypes.c_uint8), _p(bad, ctypes.c_uint8), ctypes.c_float(lam),
                    ctypes.c_uint64(seed), ctypes.c_int64(token_offset),
                    _p(a, ctypes.c_float), _p(u, ctypes.c_float), _p(acc, ctypes.c_uint8))
    return a, u, acc


def z_topk(za, zp, idx_a, idx_p, lse_a, lse_p, lam, mask=None, bad=None):
    T, V = _check2d(za)
    k = idx_a.shape[1]
    zk = np.zeros(T)
    lib().jo_z_topk(ctypes.c_int64(T), ctypes.c_int64(V), ctypes.c_int64(V), ctypes.c_int(_dtype_code(za)),
                    _vp(za), _vp(zp), _p(mask, ctypes.c_uint8), _p(bad, ctypes.c_uint8), ctypes.c_int(k),
                    _p(np.ascontiguousarray(idx_a), ctypes.c_int32),
                    _p(np.ascontiguousarray(idx_p), ctypes.c_int32),
                    _p(lse_a, ctypes.c_double), _p(lse_p, ctypes.c_double), ctypes.c_double(lam),
                    _p(zk, ctypes.c_double))
    return zk


def z_exact(za, zp, lse_a, lse_p, lam, mask=None, bad=None):
    T, V = _check2d(za)
    z = np.zeros(T)
    lib().jo_z_exact(ctypes.c_int64(T), ctypes.c_int64(V), ctypes.c_int64(V), ctypes.c_int(_dtype_code(za)),
                     _vp(za), _vp(zp), _p(mask, ctypes.c_uint8), _p(bad, ctypes.c_uint8),
                     _p(lse_a, ctypes.c_double), _p(lse_p, ctypes.c_double), ctypes.c_double(lam),
                     _p(z, ctypes.c_double))
    return z


def z_sparse(zp, inf_idx, inf_logp, new_idx, lse_p, lam, mask=None, bad=None):
    """Z_approx when the rollout model is known only through its stored top-k log-probs
    (Algorithm 1 Phase 1 / Phase 2 step 2): returns (z_lo, z_hi), see jo_z_sparse."""
    T, V = _check2d(zp)
    inf_idx = np.ascontiguousarray(inf_idx, np.int32)
    inf_logp = np.ascontiguousarray(inf_logp, np.float32)
    new_idx = np.ascontiguousarray(new_idx, np.int32)
    lo, hi = np.zeros(T), np.zeros(T)
    lib().jo_z_sparse(ctypes.c_int64(T), ctypes.c_int64(V), ctypes.c_int64(V), ctypes.c_int(_dtype_code(zp)),
                      _vp(zp), _p(mask, ctypes.c_uint8), _p(bad, ctypes.c_uint8), ctypes.c_int(inf_idx.shape[1]),
                      _p(inf_idx, ctypes.c_int32), _p(inf_logp, ctypes.c_float), ctypes.c_int(new_idx.shape[1]),
                      _p(new_idx, ctypes.c_int32), _p(lse_p, ctypes.c_double), ctypes.c_double(lam),
                      _p(lo, ctypes.c_double), _p(hi, ctypes.c_double))
    return lo, hi


def rollout_record(za, tokens, k_inf, mask=None):
    """What Algorithm 1 Phase 1 stores per token from the rollout model's forward: log p_inf(a_t) and
    the k_inf most likely tokens with their log-probabilities (fp32, best first)."""
    T, V = _check2d(za)
    r = lse_gather(za, za, tokens, mask)
    idx = topk(za, k_inf, mask)
    if za.dtype == np.uint16:
        zf = (za.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    else:
        zf = za.astype(np.float64)
    safe = np.maximum(idx, 0)
    logp = (np.take_along_axis(zf, safe, axis=1) - r["lse_a"][:, None]).astype(np.float32)
    logp[idx < 0] = 0.0
    return r["lq"], idx, logp


def forward_sparse(zp, tokens, logp_inf_token, inf_idx, inf_logp, mask=None, *, lam=None, budget=None, k=20, seed=0,
                   token_offset=0, c1=0.0, cap=False):
    """The forward steps with the rollout model known only through the stored record: the policy's
    log-softmax and top-k from its logits, acceptance from the stored log p_inf(a_t), Z from
    jo_z_sparse (z_lo, or z_hi with cap=True), then the batch correction and weights as usual."""
    assert (lam is None) != (budget is None)
    T, V = _check2d(zp)
    mask = None if mask is None else np.ascontiguousarray(mask, np.uint8)
    r = lse_gather(zp, zp, tokens, mask)
    bad = r["bad"]
    r["lq"] = np.ascontiguousarray(logp_inf_token, np.float32).copy()
    r["lq"][(bad != 0) | (np.zeros(T, bool) if mask is None else mask == 0)] = 0.0
    r["lq64"] = r["lq"].astype(np.float64)
    r["topk_idx_p"] = topk(zp, k, mask)
    if budget is not None:
        lam = float(np.float32(lambda_from_budget(r["lq"], r["lp"], budget, mask, bad)))
    lam = float(np.float32(lam))
    r["lambda"] = lam
    r["a"], r["u"], r["accept"] = accept(r["lq"], r["lp"], lam, seed, token_offset, mask, bad)
    r["z_lo"], r["z_hi"] = z_sparse(zp, inf_idx, inf_logp, r["topk_idx_p"], r["lse_p"], lam, mask, bad)
    r["zk"] = r["z_hi"] if cap else r["z_lo"]
    r["w"], r["w64"], r["stats"] = batch_weights(r["lq"], r["lp"], r["accept"], r["a"], r["zk"], lam, c1, mask, bad)
    r["stats"]["n_bad_token"] = int(bad.sum())
    return r


def lmhead_rows(rows, hidden, weight):
    """fp32 logits of the given rows of an output layer: hidden [T, H] and weight [V, H] as bf16 bit
    patterns (uint16); products and sums in double, one rounding."""
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    assert hidden.dtype == np.uint16 and weight.dtype == np.uint16 and hidden.shape[1] == weight.shape[1]
    hidden, weight = np.ascontiguousarray(hidden), np.ascontiguousarray(weight)
    H, V = hidden.shape[1], weight.shape[0]
    out = np.zeros((rows.shape[0], V), dtype=np.float32)
    lib().jo_lmhead_rows(ctypes.c_int64(rows.shape[0]), _p(rows, ctypes.c_int64), ctypes.c_int64(H), ctypes.c_int64(V),
                         _p(hidden, ctypes.c_uint16), ctypes.c_int64(H), _p(weight, ctypes.c_uint16),
                         ctypes.c_int64(H), _p(out, ctypes.c_float))
    return out


_STAT_KEYS = ("n_valid", "n_accept", "alpha_hat", "mean_accept_prob", "z_approx_mean", "kappa",
              "lambda_used")


def batch_weights(lq, lp, acc, a, zk, lam, c1=0.0, mask=None, bad=None):
    T = lq.shape[0]
    w = np.zeros(T, np.float32)
    w64 = np.zeros(T)
    st = np.zeros(8)
    lib().jo_batch_weights(ctypes.c_int64(T), _p(lq, ctypes.c_float), _p(lp, ctypes.c_float),
                           _p(mask, ctypes.c_uint8), _p(bad, ctypes.c_uint8), _p(acc, ctypes.c_uint8),
                           _p(a, ctypes.c_float), _p(zk, ctypes.c_double), ctypes.c_double(lam),
                           ctypes.c_double(c1), _p(w, ctypes.c_float), _p(w64, ctypes.c_double),
                           _p(st, ctypes.c_double))
    stats = {k: float(st[i]) for i, k in enumerate(_STAT_KEYS)}
    stats["n_valid"] = int(stats["n_valid"])
    stats["n_accept"] = int(stats["n_accept"])
    return w, w64, stats


def ppo_terms(lq, lp, acc, weight, adv=None, mask=None, logp_ref=None, logq_ref=None, logp_inf=None,
              clip=False, eps_lo=0.0, eps_hi=0.0, c2=0.0, tis_cap=0.0):
    """Per-token PPO / Jackpot terms (Algorithm 1 steps 1, 3, 4; Eq. ppo_rollout): a dict of
    rho, r_theta, slope_theta, obj_theta, F, r_omega, slope_omega, obj_omega, plus the raw [T, 8]."""
    T = len(lq)
    f32 = lambda a: None if a is None else np.ascontiguousarray(a, np.float32)
    out = np.zeros((T, 8))
    lib().jo_ppo_terms(ctypes.c_int64(T), _p(f32(lq), ctypes.c_float), _p(f32(lp), ctypes.c_float),
                       _p(mask, ctypes.c_uint8), _p(np.ascontiguousarray(acc, np.uint8), ctypes.c_uint8),
                       _p(f32(weight), ctypes.c_float), _p(f32(adv), ctypes.c_float),
                       _p(f32(logp_ref), ctypes.c_float), _p(f32(logq_ref), ctypes.c_float),
                       _p(f32(logp_inf), ctypes.c_float), ctypes.c_int(1 if clip else 0),
                       ctypes.c_double(eps_lo), ctypes.c_double(eps_hi), ctypes.c_double(c2),
                       ctypes.c_double(tis_cap), _p(out, ctypes.c_double))
    names = ("rho", "r_theta", "slope_theta", "obj_theta", "F", "r_omega", "slope_omega", "obj_omega")
    d = {n: out[:, i].copy() for i, n in enumerate(names)}
    d["raw"] = out
    return d


def grad_rows(rows, za, zp, tokens, acc, weight, lse_a, lse_p, n_valid, mask=None, adv=None,
              grad_out=1.0, lambda_distill=0.0, ppo=None):
    T, V = _check2d(za)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    da = np.zeros((rows.shape[0], V))
    dp = np.zeros((rows.shape[0], V))
    adv32 = None if adv is None else np.ascontiguousarray(adv, np.float32)
    lib().jo_grad_rows(ctypes.c_int64(rows.shape[0]), _p(rows, ctypes.c_int64), ctypes.c_int64(V),
                       ctypes.c_int64(V), ctypes.c_int(_dtype_code(za)), _vp(za), _vp(zp),
                       _p(tokens, ctypes.c_int32), _p(mask, ctypes.c_uint8), _p(acc, ctypes.c_uint8),
                       _p(np.ascontiguousarray(weight, np.float32), ctypes.c_float),
                       _p(adv32, ctypes.c_float), _p(lse_a, ctypes.c_double), _p(lse_p, ctypes.c_double),
                       ctypes.c_double(n_valid), ctypes.c_double(grad_out), ctypes.c_double(lambda_distill),
                       _p(None if ppo is None else np.ascontiguousarray(ppo["raw"], np.float64), ctypes.c_double),
                       _p(da, ctypes.c_double), _p(dp, ctypes.c_double))
    return da, dp


def loss(za64, zp64, tokens, acc, weight64, adv64, logp_ref, logq_ref, pfix, lambda_distill, mask=None,
         f_actor=None, clip=False, eps_lo=0.0, eps_hi=0.0):
    T, V = za64.shape
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    args = [np.ascontiguousarray(x, np.float64) for x in (za64, zp64)]
    return float(lib().jo_loss(ctypes.c_int64(T), ctypes.c_int64(V), _p(args[0], ctypes.c_double),
                               _p(args[1], ctypes.c_double), _p(tokens, ctypes.c_int32),
                               _p(mask, ctypes.c_uint8), _p(acc, ctypes.c_uint8),
                               _p(np.ascontiguousarray(weight64, np.float64), ctypes.c_double),
                               _p(None if adv64 is None else np.ascontiguousarray(adv64, np.float64),
                                  ctypes.c_double),
                               _p(np.ascontiguousarray(logp_ref, np.float64), ctypes.c_double),
                               _p(np.ascontiguousarray(logq_ref, np.float64), ctypes.c_double),
                               _p(np.ascontiguousarray(pfix, np.float64), ctypes.c_double),
                               ctypes.c_double(lambda_distill),
                               _p(None if f_actor is None else np.ascontiguousarray(f_actor, np.float64),
                                  ctypes.c_double),
                               ctypes.c_int(1 if clip else 0), ctypes.c_double(eps_lo), ctypes.c_double(eps_hi)))


def row_lambda(za, zp, budget, mask=None):
    """Per-row lambda meeting an acceptance budget (Theorem 3.4), with KL(p||q) and KL(p||q~)."""
    T, V = _check2d(za)
    lam, kb, ka = np.zeros(T), np.zeros(T), np.zeros(T)
    lib().jo_row_lambda(ctypes.c_int64(T), ctypes.c_int64(V), ctypes.c_int64(V), ctypes.c_int(_dtype_code(za)),
                        _vp(za), _vp(zp), _p(mask, ctypes.c_uint8), ctypes.c_double(budget),
                        _p(lam, ctypes.c_double), _p(kb, ctypes.c_double), _p(ka, ctypes.c_double))
    return dict(lam=lam, kl_before=kb, kl_after=ka)


def kl_rows(za, zp, lse_a, lse_p, mask=None):
    T, V = _check2d(za)
    kl = np.zeros(T)
    lib().jo_kl_rows(ctypes.c_int64(T), ctypes.c_int64(V), ctypes.c_int64(V), ctypes.c_int(_dtype_code(za)),
                     _vp(za), _vp(zp), _p(mask, ctypes.c_uint8), _p(lse_a, ctypes.c_double),
                     _p(lse_p, ctypes.c_double), _p(kl, ctypes.c_double))
    return kl


def forward(za, zp, tokens, mask=None, *, lam=None, budget=None, k=20, seed=0, token_offset=0,
            c1=0.0, exact=False, want_kl=False):
    """All forward steps in the paper's order on whole arrays.

    Exactly one of ``lam`` (fixed lambda) and ``budget`` (acceptance budget) is
    given.  ``k >= V`` makes Z_approx the exact Z.  ``exact=True`` also returns
    the brute-force full-vocabulary Z beside Z_approx.
    """
    assert (lam is None) != (budget is None)
    T, V = _check2d(za)
    mask = None if mask is None else np.ascontiguousarray(mask, np.uint8)
    r = lse_gather(za, zp, tokens, mask)
    bad = r["bad"]
    kk = min(k, V)
    if kk < V:
        r["topk_idx_a"] = topk(za, kk, mask)
        r["topk_idx_p"] = topk(zp, kk, mask)
    if budget is not None:
        lam = float(np.float32(lambda_from_budget(r["lq"], r["lp"], budget, mask, bad)))
    lam = float(np.float32(lam))
    r["lambda"] = lam
    r["a"], r["u"], r["accept"] = accept(r["lq"], r["lp"], lam, seed, token_offset, mask, bad)
    if exact or kk >= V:
        r["z_exact"] = z_exact(za, zp, r["lse_a"], r["lse_p"], lam, mask, bad)
    if kk < V:
        r["zk"] = z_topk(za, zp, r["topk_idx_a"], r["topk_idx_p"], r["lse_a"], r["lse_p"], lam, mask, bad)
    else:
        r["zk"] = r["z_exact"]
    r["w"], r["w64"], r["stats"] = batch_weights(r["lq"], r["lp"], r["accept"], r["a"], r["zk"], lam,
                                                 c1, mask, bad)
    r["stats"]["n_bad_token"] = int(bad.sum())
    if want_kl:
        kl = kl_rows(za, zp, r["lse_a"], r["lse_p"], mask)
        n = max(r["stats"]["n_valid"], 1)
        r["stats"]["mean_kl_p_q"] = float(kl.sum() / n)
    return r
