"""GPU parity of the vocabulary-parallel forward (jp_vshard_local / jp_vshard_merge /
jp_batch_finalize) against the oracle on the whole vocabulary.

The shards of one batch are run one after the other on the one GPU, each through a
context of its own as a rank would; no kernel waits for another.  What every rank ends with
must be what the oracle gives for the unsplit rows -- same bars as the single-device
forward: indices, uniforms and accept bits bit-exact, floating point within rtol 1e-5 /
atol 1e-6 -- and identical, bit for bit, on every rank.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06107_b200 import binding as B
from paper_2602_06107_b200 import build as jp_build
from paper_2602_06107_b200 import parallel, runner
from paper_2602_06107_b200.inputs import LogitRecipe, make_logits, to_numpy_bits
from test_gpu_parity import check_forward, close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ranks():
    jp_build.build()
    cs = [B.Context(0) for _ in range(17)]
    yield cs
    for c in cs:
        c.close()


def run_shards(ctxs, za, zp, tok, mask, bounds, *, lam=None, budget=None, k, seed, c1=0.0, finish=(0, -1)):
    """Local pass of every shard, the gather (a stack), then merge + finalize on the ranks in `finish`."""
    T, V = za.shape
    n = len(bounds)
    words = B.jp_vshard_record_floats(k)
    assert words == 8 + 6 * k
    gathered = torch.empty((n, T, words), dtype=torch.float32, device=za.device)
    for s, (lo, hi) in enumerate(bounds):
        zs, ps = za[:, lo:hi], zp[:, lo:hi]
        B.jp_vshard_local(ctxs[s % len(ctxs)], B.make_desc(zs), zs, ps, tok, mask, lo, V, k, gathered[s])
    outs = []
    for s in finish:
        s = s % n
        got = {}

        def gather(packed, group, got=got):
            got["packed"] = packed
            return gathered

        # the rank's own local pass runs again inside (same bits), then the merge over all shards
        lo, hi = bounds[s]
        out = parallel.forward_vocab_parallel(ctxs[s % len(ctxs)], za[:, lo:hi], zp[:, lo:hi], tok, mask, lo, V, lam=lam,
                                              budget=budget, k=k, seed=seed, c1=c1, aux=True, gather=gather,
                                              shard_index=s)
        assert torch.equal(got["packed"].view(torch.int32), gathered[s].view(torch.int32))
        outs.append(out)
    return outs


def same_bits(a, b):
    for n, t in a.items():
        if isinstance(t, torch.Tensor) and n != "stats_buf":
            assert torch.equal(t.view(torch.uint8) if t.dtype != torch.uint8 else t,
                               b[n].view(torch.uint8) if b[n].dtype != torch.uint8 else b[n]), n
    assert a["stats"] == b["stats"]


@pytest.mark.parametrize("dtype,T,V,n,k", [("bf16", 300, 20000, 4, 16), ("bf16", 96, 151936, 8, 32),
                                           ("f32", 130, 4099, 3, 8), ("bf16", 64, 50001, 2, 128),
                                           ("bf16", 24, 16 * 1024, 16, 128),
                                           ("bf16", 40, 8 * 1024, 40, 12),       # more shards than lanes in the merge's warp
                                           ("f32", 20, 128 * 40, 128, 5)])       # the most shards the merge takes
def test_shards_match_oracle_on_the_whole_vocabulary(ranks, dtype, T, V, n, k):
    align = 8 if dtype == "bf16" else 4
    ld = -(-V // align) * align
    r = LogitRecipe(T=T, V=ld, dtype=dtype, sigma0=2.5, peaks=6, peak_lo=6.0, peak_hi=14.0, sigma=1.0, seed=21)
    zaf, zpf, _ = make_logits(r, "cuda")
    za, zp = zaf[:, :V], zpf[:, :V]
    g = torch.Generator(device="cuda").manual_seed(5)
    gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
    tok = (za.float() + gum).argmax(1).to(torch.int32)
    tok[3] = V                                   # out of range: the row is invalid on every shard
    tok[5] = V - 1                               # the last column, owned by the last shard
    tok[6] = 0
    mask = (torch.arange(T, device="cuda") % 7 != 2).to(torch.uint8)
    bounds = [parallel.shard_columns(V, n, s, align) for s in range(n)]
    assert bounds[0][0] == 0 and bounds[-1][1] == V and all(bounds[i][1] == bounds[i + 1][0] for i in range(n - 1))
    lam, seed = 1.4, 9
    a, b = run_shards(ranks, za, zp, tok, mask, bounds, lam=lam, k=k, seed=seed, c1=4.0)
    same_bits(a, b)
    ref = oracle.forward(to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous()), tok.cpu().numpy(),
                         mask.cpu().numpy(), lam=lam, k=k, seed=seed, c1=4.0)
    flips = check_forward(a, ref, k, V, mask.cpu().numpy(), 4.0)
    print("near-threshold accept flips:", flips)
    # against the single-device forward of the same rows: same lists, same draws
    one = runner.forward(ranks[0], za, zp, tok, mask, lam=lam, k=k, seed=seed, c1=4.0)
    for name in ("topk_idx_actor", "topk_idx_policy", "topk_val_actor", "topk_val_policy", "uniform"):
        assert torch.equal(one[name], a[name]), name
    close(a["logp_actor"].cpu().numpy(), one["logp_actor"].cpu().numpy())
    close(a["z_approx"].cpu().numpy(), one["z_approx"].cpu().numpy())


def test_shards_with_a_budget(ranks):
    T, V, n, k = 512, 32768, 4, 20
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=3.0, peaks=8, peak_lo=8.0, peak_hi=15.0, sigma=1.5, seed=33)
    za, zp, tok = make_logits(r, "cuda")
    bounds = [parallel.shard_columns(V, n, s) for s in range(n)]
    a, b = run_shards(ranks, za, zp, tok, None, bounds, budget=0.6, k=k, seed=2)
    same_bits(a, b)
    assert abs(a["stats"]["mean_accept_prob"] - 0.6) < 5e-6
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), None, budget=0.6, k=k, seed=2)
    close(a["stats"]["lambda_used"], ref["lambda"])
    a2, = run_shards(ranks, za, zp, tok, None, bounds, lam=ref["lambda"], k=k, seed=2, finish=(1,))
    check_forward(a2, ref, k, V, None, 0.0)


def test_one_shard_is_the_plain_forward(ranks):
    T, V, k = 200, 30000, 32
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=3.0, peaks=8, sigma=1.0, seed=34)
    za, zp, tok = make_logits(r, "cuda")
    a = parallel.forward_vocab_parallel(ranks[0], za, zp, tok, None, 0, V, lam=2.0, k=k, seed=4, aux=True)
    one = runner.forward(ranks[1], za, zp, tok, None, lam=2.0, k=k, seed=4)
    for name in ("accept", "uniform", "topk_idx_actor", "topk_idx_policy", "topk_val_actor", "topk_val_policy"):
        assert torch.equal(one[name], a[name]), name
    for name in ("weight", "logp_actor", "logp_policy", "lse_actor", "lse_policy", "z_approx", "accept_prob"):
        close(a[name].cpu().numpy(), one[name].cpu().numpy(), rtol=1e-6, atol=1e-7)


def test_non_finite_row_in_one_shard_invalidates_the_row_everywhere(ranks):
    T, V, n, k = 40, 16384, 4, 8
    r = LogitRecipe(T=T, V=V, dtype="f32", sigma0=2.0, peaks=4, sigma=1.0, seed=35)
    za, zp, tok = make_logits(r, "cuda")
    za[7, 9000] = float("nan")                  # shard 2 only
    bounds = [parallel.shard_columns(V, n, s, 4) for s in range(n)]
    a, b = run_shards(ranks, za, zp, tok, None, bounds, lam=1.0, k=k, seed=1, finish=(0, 2))
    one = runner.forward(ranks[0], za, zp, tok, None, lam=1.0, k=k, seed=1)
    for o in (a, b):
        assert o["stats"]["n_nonfinite"] == one["stats"]["n_nonfinite"] == 1
        assert o["stats"]["n_valid"] == one["stats"]["n_valid"]
        assert torch.equal(o["accept"], one["accept"])
        close(o["weight"].cpu().numpy(), one["weight"].cpu().numpy())


def test_shard_call_sequence_and_limits(ranks):
    c = ranks[0]
    r = LogitRecipe(T=8, V=4096, dtype="bf16", seed=2)
    za, zp, tok = make_logits(r, "cuda")
    buf = torch.empty((8, B.jp_vshard_record_floats(16)), device="cuda")
    with pytest.raises(B.JackpotError, match="jp_vshard_local"):
        B.jp_vshard_merge(c, 1, 0, buf, 8, 4096, 16)
    with pytest.raises(B.JackpotError, match="wider"):
        B.jp_vshard_local(c, B.make_desc(za[:, :16]), za[:, :16], zp[:, :16], tok, None, 0, 4096, 16, buf)
    with pytest.raises(B.JackpotError, match="outside"):
        B.jp_vshard_local(c, B.make_desc(za), za, zp, tok, None, 8, 4096, 16, buf)
    B.jp_vshard_local(c, B.make_desc(za), za, zp, tok, None, 0, 4096, 16, buf)
    with pytest.raises(B.JackpotError, match="128 shards"):
        B.jp_vshard_merge(c, 129, 0, buf, 8, 4096, 16)
    with pytest.raises(B.JackpotError, match="differ"):
        B.jp_vshard_merge(c, 1, 0, buf, 8, 4096, 8)
    B.jp_vshard_merge(c, 1, 0, buf, 8, 4096, 16)
    out = runner._alloc_outputs(8, "cuda")
    B.jp_batch_finalize(c, B.jp_obrs_desc(), 1.0, B.JP_LAMBDA_FIXED, 0, out["accept"], out["weight"],
                        out["logp_actor"], out["logp_policy"], out["stats_buf"])
    torch.cuda.synchronize()
    assert B.read_stats(out["stats_buf"])["n_valid"] == 8


@pytest.mark.parametrize("dtype,V,n", [("bf16", 20000, 3), ("f32", 4099, 2)])
def test_slice_gradients_match_oracle_on_whole_rows(ranks, dtype, V, n):
    """Every rank writes the gradient of its own columns from the merged records; side by side
    the slices are the oracle's gradient of the whole rows (general form: ratios, clip, c2, F)."""
    from test_gpu_backward import check_grads
    T, k, lam, seed = 90, 16, 1.3, 5
    align = 8                                    # gradients are bf16: slices start on 8 elements
    ld = -(-V // align) * align
    r = LogitRecipe(T=T, V=ld, dtype=dtype, sigma0=2.5, peaks=4, sigma=1.0, seed=41)
    zaf, zpf, _ = make_logits(r, "cuda")
    za, zp = zaf[:, :V], zpf[:, :V]
    g = torch.Generator(device="cuda").manual_seed(6)
    gum = -torch.log(-torch.log(torch.rand((T, V), generator=g, device="cuda").clamp_(1e-30, 1 - 1e-7)))
    tok = (za.float() + gum).argmax(1).to(torch.int32)
    tok[4], tok[5] = V - 1, 0
    mask = (torch.arange(T, device="cuda") % 6 != 1).to(torch.uint8)
    adv = torch.randn(T, generator=g, device="cuda")
    bounds = [parallel.shard_columns(V, n, s, align) for s in range(n)]
    outs = run_shards(ranks, za, zp, tok, mask, bounds, lam=lam, k=k, seed=seed, c1=3.0, finish=tuple(range(n)))
    out = outs[0]
    da = torch.full((T, ld), 7.0, dtype=torch.bfloat16, device="cuda")
    dp = torch.full((T, ld), 7.0, dtype=torch.bfloat16, device="cuda")
    for s, (lo, hi) in enumerate(bounds):
        runner.backward(ranks[s], za[:, lo:hi], zp[:, lo:hi], tok, mask, out["accept"], out["weight"], advantages=adv,
                        lambda_distill=1.0, grad_out=0.5, d_actor=da[:, lo:hi], d_policy=dp[:, lo:hi], vocab_offset=lo)
    torch.cuda.synchronize()
    assert torch.all(da[:, V:] == 7.0) and torch.all(dp[:, V:] == 7.0)
    za_np, zp_np = to_numpy_bits(za.contiguous()), to_numpy_bits(zp.contiguous())
    ref = oracle.forward(za_np, zp_np, tok.cpu().numpy(), mask.cpu().numpy(), lam=lam, k=k, seed=seed, c1=3.0)
    rows = np.arange(0, T, 2)
    check_grads(da[:, :V], dp[:, :V], rows, za_np, zp_np, tok.cpu().numpy(), mask.cpu().numpy(),
                out["accept"].cpu().numpy(), out["weight"].cpu().numpy(), ref["lse_a"], ref["lse_p"],
                out["stats"]["n_valid"], adv.cpu().numpy(), 1.0, g=0.5)
    # and the same bits as the single-device backward of the whole rows
    one = runner.forward(ranks[n], za, zp, tok, mask, lam=lam, k=k, seed=seed, c1=3.0)
    da1, dp1 = runner.backward(ranks[n], za, zp, tok, mask, out["accept"], out["weight"], advantages=adv,
                               lambda_distill=1.0, grad_out=0.5)
    torch.cuda.synchronize()
    same = (da[:, :V] == da1).float().mean().item(), (dp[:, :V] == dp1).float().mean().item()
    print("share of gradient elements bit-identical to the single-device backward:", same)
    assert min(same) > 0.999
    # whole-row outputs are refused on a slice
    lo, hi = bounds[0]
    with pytest.raises(B.JackpotError, match="whole rows"):
        runner.backward(ranks[0], za[:, lo:hi], zp[:, lo:hi], tok, mask, out["accept"], out["weight"],
                        d_actor=da[:, lo:hi], d_policy=dp[:, lo:hi], vocab_offset=lo,
                        out_kl=torch.empty(T, device="cuda"))


def test_pushed_lines_equal_the_gathered_ones(ranks):
    """The export that stores into every shard's gathered buffer (here all of them on the one GPU,
    standing in for peer-mapped memory) leaves in each what the all-gather leaves."""
    T, V, n, k = 150, 24000, 4, 16
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=3.0, peaks=6, sigma=1.0, seed=51)
    za, zp, tok = make_logits(r, "cuda")
    mask = (torch.arange(T, device="cuda") % 5 != 0).to(torch.uint8)
    bounds = [parallel.shard_columns(V, n, s) for s in range(n)]
    words = B.jp_vshard_record_floats(k)
    stacked = torch.empty((n, T, words), device="cuda")
    bufs = [torch.full((n, T, words), float("nan"), device="cuda") for _ in range(n)]
    for s, (lo, hi) in enumerate(bounds):
        zs, ps = za[:, lo:hi], zp[:, lo:hi]
        B.jp_vshard_local(ranks[s], B.make_desc(zs), zs, ps, tok, mask, lo, V, k, stacked[s])
        B.jp_vshard_local_push(ranks[s], B.make_desc(zs), zs, ps, tok, mask, lo, V, k, s, bufs)
    torch.cuda.synchronize()
    for b in bufs:
        assert torch.equal(b.view(torch.int32), stacked.view(torch.int32))
    # through the glue: push, then merge and finalize from the rank's own buffer
    lo, hi = bounds[2]
    out = parallel.forward_vocab_parallel(ranks[2], za[:, lo:hi], zp[:, lo:hi], tok, mask, lo, V, lam=1.5, k=k, seed=3,
                                          aux=True, shard_index=2, push_to=bufs)
    ref = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), mask.cpu().numpy(), lam=1.5, k=k,
                         seed=3)
    check_forward(out, ref, k, V, mask.cpu().numpy(), 0.0)
    with pytest.raises(B.JackpotError, match="16"):
        B.jp_vshard_local_push(ranks[0], B.make_desc(za[:, :hi]), za[:, :hi], zp[:, :hi], tok, mask, 0, V, k, 0,
                               [bufs[0]] * 17)


def test_shards_of_an_empty_batch(ranks):
    c = ranks[0]
    za = torch.empty((0, 4096), dtype=torch.bfloat16, device="cuda")
    tok = torch.empty(0, dtype=torch.int32, device="cuda")
    buf = torch.empty((0, B.jp_vshard_record_floats(8)), device="cuda")
    d = B.jp_obrs_desc()
    d.T, d.V, d.ld, d.dtype = 0, 4096, 4096, B.JP_BF16
    B.jp_vshard_local(c, d, za, za, tok, None, 0, 8192, 8, buf)
    B.jp_vshard_merge(c, 2, 0, buf, 0, 8192, 8)
    out = runner._alloc_outputs(1, "cuda")
    B.jp_batch_finalize(c, B.jp_obrs_desc(), 1.0, B.JP_LAMBDA_FIXED, 0, out["accept"], out["weight"],
                        out["logp_actor"], out["logp_policy"], out["stats_buf"])
    torch.cuda.synchronize()
    st = B.read_stats(out["stats_buf"])
    assert st["n_valid"] == 0 and st["status"] == 0
