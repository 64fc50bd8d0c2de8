"""Output allocation around the libjackpot calls (no arithmetic of the method here)."""
from __future__ import annotations

import torch

from . import binding as B

AUX_F32 = ("accept_prob", "uniform", "z_approx", "lse_actor", "lse_policy")


def _alloc_outputs(T, dev):
    return dict(accept=torch.empty(T, dtype=torch.uint8, device=dev),
                weight=torch.empty(T, dtype=torch.float32, device=dev),
                logp_actor=torch.empty(T, dtype=torch.float32, device=dev),
                logp_policy=torch.empty(T, dtype=torch.float32, device=dev),
                stats_buf=B.new_stats_buffer(dev))


def _alloc_aux(T, k, V, dev, want_exact):
    aux = {n: torch.empty(T, dtype=torch.float32, device=dev) for n in AUX_F32}
    if k < V:
        aux["topk_idx_actor"] = torch.empty((T, k), dtype=torch.int32, device=dev)
        aux["topk_idx_policy"] = torch.empty((T, k), dtype=torch.int32, device=dev)
        aux["topk_val_actor"] = torch.empty((T, k), dtype=torch.float32, device=dev)
        aux["topk_val_policy"] = torch.empty((T, k), dtype=torch.float32, device=dev)
    if want_exact:
        aux["z_exact"] = torch.empty(T, dtype=torch.float32, device=dev)
    return aux


def forward(ctx: B.Context, za, zp, tokens, mask=None, *, lam=None, budget=None, k=20, seed=0,
            token_offset=0, c1=0.0, aux=True, want_exact=False, sync=True):
    """One jp_obrs_forward call; returns a dict of device tensors plus ``stats``."""
    assert (lam is None) != (budget is None)
    T, V = za.shape
    dev = za.device
    out = _alloc_outputs(T, dev)
    auxd = _alloc_aux(T, k, V, dev, want_exact) if aux else {}
    mode = B.JP_LAMBDA_FIXED if budget is None else B.JP_LAMBDA_FROM_BUDGET
    desc = B.make_desc(za, lambda_mode=mode, c1=c1, token_offset=token_offset, aux=auxd)
    B.jp_obrs_forward(ctx, desc, za, zp, tokens, mask, lam if budget is None else budget, k, seed,
                      out["accept"], out["weight"], out["logp_actor"], out["logp_policy"], out["stats_buf"])
    out.update(auxd)
    if sync:
        torch.cuda.synchronize(dev)
        out["stats"] = B.read_stats(out["stats_buf"])
    return out


def forward_chunked(ctx: B.Context, chunks, T_total, V, dtype_code, *, lam=None, budget=None, k=20, seed=0,
                    c1=0.0, device="cuda", aux=False):
    """``chunks`` yields (token_offset, za, zp, tokens, mask_or_None) blocks of rows."""
    assert (lam is None) != (budget is None)
    exact = k >= V
    B.jp_batch_begin(ctx, T_total, V, dtype_code, k, lam if (exact and lam is not None) else 0.0)
    for off, za, zp, tok, m in chunks:
        d = B.make_desc(za, token_offset=off)
        B.jp_batch_chunk(ctx, d, za, zp, tok, m)
    out = _alloc_outputs(T_total, device)
    auxd = {}
    d = B.jp_obrs_desc()
    d.c1 = c1
    if aux:
        auxd = _alloc_aux(T_total, k, V, device, False)
        for n, t in auxd.items():
            setattr(d, n, t.data_ptr())
    mode = B.JP_LAMBDA_FIXED if budget is None else B.JP_LAMBDA_FROM_BUDGET
    B.jp_batch_finalize(ctx, d, lam if budget is None else budget, mode, seed, out["accept"], out["weight"],
                        out["logp_actor"], out["logp_policy"], out["stats_buf"])
    out.update(auxd)
    torch.cuda.synchronize()
    out["stats"] = B.read_stats(out["stats_buf"])
    return out


def backward(ctx: B.Context, za, zp, tokens, mask, accept, weight, *, advantages=None, lambda_distill=0.0,
             grad_out=1.0, n_valid=0, record_offset=0, d_actor=None, d_policy=None, vocab_offset=None, **general):
    """``general``: the optional fields of jp_obrs_bwd_desc (logp_ref, logp_actor_ref, logp_inf, eps_lo,
    eps_hi, c2, tis_cap, out_obj_policy, out_obj_actor, out_kl, out_loss).  ``vocab_offset``: the logits are
    the columns from there on of rows whose records a vocabulary-parallel forward left (jp_vshard_backward)."""
    T, V = za.shape
    if d_actor is None:
        d_actor = torch.empty((T, za.stride(0)), dtype=torch.bfloat16, device=za.device)[:, :V]
    if d_policy is None:
        d_policy = torch.empty((T, zp.stride(0)), dtype=torch.bfloat16, device=za.device)[:, :V]
    desc = B.make_desc(za)
    bwd = B.make_bwd_desc(advantages, lambda_distill, grad_out, n_valid, record_offset, **general)
    if vocab_offset is None:
        B.jp_obrs_backward(ctx, desc, bwd, za, zp, tokens, mask, accept, weight, d_actor, d_policy)
    else:
        B.jp_vshard_backward(ctx, desc, bwd, za, zp, tokens, mask, vocab_offset, accept, weight, d_actor, d_policy)
    return d_actor, d_policy


def forward_sparse_actor(ctx: B.Context, zp, tokens, mask, logp_inf_token, topk_inf_idx, topk_inf_logp, *, lam=None,
                         budget=None, k=20, seed=0, token_offset=0, c1=0.0, cap=False, aux=True):
    """One jp_obrs_forward_sparse_actor call; returns a dict of device tensors plus ``stats``."""
    assert (lam is None) != (budget is None)
    T, V = zp.shape
    dev = zp.device
    out = _alloc_outputs(T, dev)
    del out["logp_actor"]
    out["z_lower"] = torch.empty(T, dtype=torch.float32, device=dev)
    out["z_upper"] = torch.empty(T, dtype=torch.float32, device=dev)
    auxd = {}
    if aux:
        auxd = {n: torch.empty(T, dtype=torch.float32, device=dev) for n in ("accept_prob", "uniform", "z_approx",
                                                                              "lse_policy")}
        auxd["topk_idx_policy"] = torch.empty((T, k), dtype=torch.int32, device=dev)
        auxd["topk_val_policy"] = torch.empty((T, k), dtype=torch.float32, device=dev)
    mode = B.JP_LAMBDA_FIXED if budget is None else B.JP_LAMBDA_FROM_BUDGET
    desc = B.make_desc(zp, lambda_mode=mode, c1=c1, token_offset=token_offset, aux=auxd,
                       flags=B.JP_DESC_SPARSE_CAP if cap else 0)
    B.jp_obrs_forward_sparse_actor(ctx, desc, zp, tokens, mask, logp_inf_token, topk_inf_idx, topk_inf_logp,
                                   topk_inf_idx.shape[1], lam if budget is None else budget, k, seed, out["accept"],
                                   out["weight"], out["logp_policy"], out["z_lower"], out["z_upper"], out["stats_buf"])
    out.update(auxd)
    torch.cuda.synchronize(dev)
    out["stats"] = B.read_stats(out["stats_buf"])
    return out


def forward_lmhead(ctx: B.Context, h_actor, w_actor, h_policy, w_policy, tokens, mask=None, *, lam=None, budget=None, k=20,
                   seed=0, token_offset=0, c1=0.0):
    """One jp_obrs_forward_lmhead call; returns a dict of device tensors plus ``stats``."""
    assert (lam is None) != (budget is None)
    T, V = h_actor.shape[0], w_actor.shape[0]
    dev = h_actor.device
    out = _alloc_outputs(T, dev)
    auxd = _alloc_aux(T, k, V, dev, False)
    d = B.jp_obrs_desc()
    d.T, d.V = T, V
    d.lambda_mode = B.JP_LAMBDA_FIXED if budget is None else B.JP_LAMBDA_FROM_BUDGET
    d.c1, d.token_offset = c1, token_offset
    for n, t in auxd.items():
        setattr(d, n, t.data_ptr())
    B.jp_obrs_forward_lmhead(ctx, d, h_actor, w_actor, h_policy, w_policy, tokens, mask,
                             lam if budget is None else budget, k, seed, out["accept"], out["weight"],
                             out["logp_actor"], out["logp_policy"], out["stats_buf"])
    out.update(auxd)
    torch.cuda.synchronize(dev)
    out["stats"] = B.read_stats(out["stats_buf"])
    return out
