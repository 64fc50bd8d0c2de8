"""Rows over several GPUs: one process per GPU, `torch.distributed` for the plumbing.

Token rows are independent (rejection is per token), so a batch shards over
ranks by contiguous row ranges and every rank streams its own rows.  The
accept draw of a row is keyed on its global index (desc.token_offset), so the
decisions do not depend on how the batch was split.  The one batch-wide
quantity is the calibration factor kappa (Section 4.4.2): the library writes a
shard's four batch sums to device memory (jp_batch_totals), one all-reduce adds
them up (32 bytes per rank), and the library forms kappa from the sums and
rewrites the shard's weights (jp_obrs_apply_totals).  Nothing here does any of
the method's arithmetic.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(T: int, world: int, rank: int):
    """Contiguous, balanced row range [lo, hi) of rank `rank` (the first T % world ranks get one row more)."""
    if world < 1 or not (0 <= rank < world) or T < 0:
        raise ValueError("need world >= 1, 0 <= rank < world, T >= 0")
    q, r = divmod(T, world)
    lo = rank * q + min(rank, r)
    return lo, lo + q + (1 if rank < r else 0)


def all_reduce_totals(totals: torch.Tensor, group=None) -> torch.Tensor:
    """Sums the shards' batch totals (the four doubles jp_batch_totals writes) over the ranks, in place."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(totals, op=dist.ReduceOp.SUM, group=group)
    return totals


def apply_global_kappa(ctx, out_weight: torch.Tensor, c1: float = 0.0, group=None, out_stats=None) -> torch.Tensor:
    """After every rank's forward on its shard: exchanges the batch totals (32 bytes, one all-reduce on
    device memory) and lets the library form the batch-wide kappa and rewrite this shard's weights
    (jp_batch_totals -> all-reduce -> jp_obrs_apply_totals).  Returns the summed totals (device)."""
    from . import binding as B
    totals = torch.empty(4, dtype=torch.float64, device=out_weight.device)
    B.jp_batch_totals(ctx, totals)
    all_reduce_totals(totals, group)
    B.jp_obrs_apply_totals(ctx, totals, c1, out_weight, out_stats)
    return totals


def max_over_ranks(value: float, group=None, device=None) -> float:
    """A timing is the slowest rank's."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def gather_rows(x: torch.Tensor, group=None) -> torch.Tensor:
    """All ranks' 1-D shards of a row-indexed array, concatenated in rank order (shards may differ in length)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return x
    world = dist.get_world_size(group)
    n = torch.tensor([x.numel()], dtype=torch.int64, device=x.device)
    sizes = [torch.zeros_like(n) for _ in range(world)]
    dist.all_gather(sizes, n, group=group)
    sizes = [int(s.item()) for s in sizes]
    pad = torch.zeros(max(sizes), dtype=x.dtype, device=x.device)
    pad[: x.numel()] = x
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad, group=group)
    return torch.cat([p[:s] for p, s in zip(parts, sizes)])


def global_lambda_from_budget(logp_actor, logp_policy, valid, budget: float, solve, group=None) -> float:
    """One lambda for a batch whose rows are spread over the ranks (budget mode).

    Every rank passes its shard's log-probs of the sampled tokens and validity flags (from
    jp_batch_logprobs); they are all-gathered (12 bytes a token: at most 1.5 MB for the largest
    workload) and every rank solves the same system with `solve(logp_actor, logp_policy, valid,
    budget) -> float`, on a GPU `solve_on_device` below.  The result is the same on all ranks
    because the inputs are."""
    lq = gather_rows(logp_actor, group)
    lp = gather_rows(logp_policy, group)
    v = gather_rows(valid, group)
    return float(solve(lq, lp, v, budget))


def solve_on_device(logp_actor, logp_policy, valid, budget: float) -> float:
    """The library's batch-level budget solve on device arrays (jp_budget_lambda_static: no allocation
    inside the library, at most JP_STATIC_MAX_ROWS rows)."""
    from . import binding as B
    out = torch.zeros(1, dtype=torch.float32, device=logp_actor.device)
    st = B.jp_budget_lambda_static(logp_actor.contiguous(), logp_policy.contiguous(), valid.contiguous(),
                                   logp_actor.numel(), budget, out)
    if st != 0:
        raise B.JackpotError(f"jp_budget_lambda_static: status {st}")
    return float(out.item())


# ---- vocabulary shards: every rank holds a slice of the vocabulary's columns of all rows ------------

def shard_columns(V: int, world: int, rank: int, align: int = 8):
    """Column range [lo, hi) of rank `rank`: balanced, every boundary but the last a multiple of
    `align` elements (a slice of a row-major tensor must start on a 16-byte boundary: 8 bf16 / 4 fp32)."""
    if world < 1 or not (0 <= rank < world) or V < 1 or align < 1:
        raise ValueError("need world >= 1, 0 <= rank < world, V >= 1, align >= 1")
    units = -(-V // align)
    q, r = divmod(units, world)
    lo_u = rank * q + min(rank, r)
    hi_u = lo_u + q + (1 if rank < r else 0)
    return min(lo_u * align, V), min(hi_u * align, V)


def gather_shard_records(packed: torch.Tensor, group=None) -> torch.Tensor:
    """[T, words] of every rank -> [world, T, words] in rank order (= ascending column offset)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return packed.unsqueeze(0).contiguous()
    world = dist.get_world_size(group)
    out = torch.empty((world * packed.shape[0],) + tuple(packed.shape[1:]), dtype=packed.dtype, device=packed.device)
    dist.all_gather_into_tensor(out, packed.contiguous(), group=group)       # concatenated along the rows
    return out.view((world,) + tuple(packed.shape))


def forward_vocab_parallel(ctx, za, zp, tokens, mask, vocab_offset: int, V_total: int, *, lam=None, budget=None,
                           k=20, seed=0, c1=0.0, aux=False, group=None, gather=gather_shard_records, shard_index=None, push_to=None,
                           own_gathered=None):
    """The forward over column slices: local pass, one all-gather of the packed records
    (T x (8 + 6k) words per rank), merge, finalize.  Every rank returns the outputs of all T rows.
    ``push_to``: per shard, that shard's gathered buffer [world, T, words] as this device addresses it
    (tensors, or raw peer-mapped pointers with this rank's own buffer in ``own_gathered``); the local
    pass then pushes its lines there itself and no collective runs."""
    from . import binding as B
    from . import runner
    assert (lam is None) != (budget is None)
    T = za.shape[0]
    if shard_index is None:
        shard_index = dist.get_rank(group) if dist.is_available() and dist.is_initialized() else 0
    if push_to is not None:
        # the export kernel stores this shard's lines into every shard's gathered buffer (peer-mapped
        # memory); all that is left of the exchange is to wait until every shard has done so
        gathered = push_to[shard_index] if isinstance(push_to[shard_index], torch.Tensor) else own_gathered
        B.jp_vshard_local_push(ctx, B.make_desc(za), za, zp, tokens, mask, vocab_offset, V_total, k, shard_index,
                               push_to)
        torch.cuda.synchronize()
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.barrier(group)
    else:
        packed = torch.empty((T, B.jp_vshard_record_floats(k)), dtype=torch.float32, device=za.device)
        B.jp_vshard_local(ctx, B.make_desc(za), za, zp, tokens, mask, vocab_offset, V_total, k, packed)
        gathered = gather(packed, group)
    B.jp_vshard_merge(ctx, gathered.shape[0], shard_index, gathered, T, V_total, k)
    out = runner._alloc_outputs(T, za.device)
    d = B.jp_obrs_desc()
    d.c1 = c1
    auxd = {}
    if aux:
        auxd = runner._alloc_aux(T, k, V_total, za.device, False)
        for n, t in auxd.items():
            setattr(d, n, t.data_ptr())
    mode = B.JP_LAMBDA_FIXED if budget is None else B.JP_LAMBDA_FROM_BUDGET
    B.jp_batch_finalize(ctx, d, lam if budget is None else budget, mode, seed, out["accept"], out["weight"],
                        out["logp_actor"], out["logp_policy"], out["stats_buf"])
    out.update(auxd)
    torch.cuda.synchronize()
    out["stats"] = B.read_stats(out["stats_buf"])
    return out
