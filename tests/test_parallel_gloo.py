"""The multi-rank path on CPU: two gloo ranks each take a contiguous share of a
batch's rows, run the oracle on their share (standing in for the GPU forward of
that shard), all-reduce the batch totals and form the batch-wide kappa.
It must equal the kappa of the undivided batch, and the accept decisions must
not depend on the split (they are keyed on the global row index)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2602_06107_b200 import parallel
from paper_2602_06107_b200.inputs import LogitRecipe, make_logits, to_numpy_bits


def test_shard_rows_partitions_exactly():
    for T in (0, 1, 7, 4096, 131072 + 3):
        for world in (1, 2, 3, 8):
            spans = [parallel.shard_rows(T, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        parallel.shard_rows(10, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, T, V, out_q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.2, seed=9)
        za, zp, tok = make_logits(r, "cpu", block_rows=T)
        mask = (torch.arange(T) % 5 != 2).to(torch.uint8).numpy()
        lo, hi = parallel.shard_rows(T, world, rank)
        ref = oracle.forward(to_numpy_bits(za[lo:hi]), to_numpy_bits(zp[lo:hi]), tok[lo:hi].numpy(), mask[lo:hi],
                             lam=1.4, k=8, seed=3, token_offset=lo)
        # the shard's batch totals as the library writes them (N, accepted, sum of Z_approx, sum of a);
        # the product path hands the summed totals back to the library, which forms kappa; here the
        # test forms it, to compare with the undivided batch
        st = ref["stats"]
        valid_rows = mask[lo:hi] != 0
        tot = torch.tensor([float(st["n_valid"]), float(st["n_accept"]), float(ref["zk"][valid_rows].sum()),
                            float(ref["a"][valid_rows].astype(np.float64).sum())], dtype=torch.float64)
        parallel.all_reduce_totals(tot)
        kappa = (float(tot[1]) / float(tot[0])) / (float(tot[2]) / float(tot[0]))
        slow = parallel.max_over_ranks(float(rank + 1))
        # budget mode: one lambda for the whole batch from the gathered log-probs of the shards
        valid = torch.from_numpy((mask[lo:hi] != 0).astype(np.uint8))
        lam_b = parallel.global_lambda_from_budget(
            torch.from_numpy(ref["lq"]), torch.from_numpy(ref["lp"]), valid, 0.55,
            lambda a, b, v, bud: oracle.lambda_from_budget(a.numpy(), b.numpy(), bud, v.numpy()))
        out_q.put((rank, lo, hi, kappa, tot.tolist(), slow, ref["accept"].tolist(), ref["zk"].tolist(), lam_b))
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_with_the_undivided_batch():
    T, V, world = 96, 2048, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, T, V, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.2, seed=9)
    za, zp, tok = make_logits(r, "cpu", block_rows=T)
    mask = (torch.arange(T) % 5 != 2).to(torch.uint8).numpy()
    whole = oracle.forward(to_numpy_bits(za), to_numpy_bits(zp), tok.numpy(), mask, lam=1.4, k=8, seed=3)
    assert got[0][3] == got[1][3], "ranks disagree on kappa"
    assert got[0][3] == pytest.approx(whole["stats"]["kappa"], rel=1e-12)
    assert got[0][4][0] == whole["stats"]["n_valid"] and got[0][4][1] == whole["stats"]["n_accept"]
    assert got[0][5] == got[1][5] == 2.0
    acc = np.concatenate([np.asarray(g[6], np.uint8) for g in got])
    zk = np.concatenate([np.asarray(g[7]) for g in got])
    assert np.array_equal(acc, whole["accept"]), "decisions depend on the split"
    assert np.array_equal(zk, whole["zk"])
    lam_whole = oracle.lambda_from_budget(whole["lq"], whole["lp"], 0.55, mask)
    assert got[0][8] == got[1][8] == lam_whole, "the gathered solve must equal the undivided batch's"


def test_shard_columns_tiles_the_vocabulary_on_aligned_boundaries():
    for V in (1, 7, 4099, 50001, 151936):
        for world in (1, 2, 3, 8):
            for align in (4, 8):
                spans = [parallel.shard_columns(V, world, r, align) for r in range(world)]
                assert spans[0][0] == 0 and spans[-1][1] == V
                assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
                assert all(lo % align == 0 or lo == V for lo, _ in spans)
                widths = [hi - lo for lo, hi in spans if hi > lo]
                assert max(widths) - min(widths) < 2 * align or V < world * align
    with pytest.raises(ValueError):
        parallel.shard_columns(10, 2, 2)


def _vocab_worker(rank, world, port, T, V, out_q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank holds a slice of the columns; what it would publish per row is the slice's
        # log-sum-exp (the oracle's, of the slice alone, standing in for the GPU pass of the shard)
        r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.2, seed=10)
        za, zp, tok = make_logits(r, "cpu", block_rows=T)
        lo, hi = parallel.shard_columns(V, world, rank)
        part = oracle.lse_gather(to_numpy_bits(za[:, lo:hi].contiguous()), to_numpy_bits(zp[:, lo:hi].contiguous()),
                                 np.zeros(T, np.int32))
        packed = torch.from_numpy(np.stack([part["lse_a"], part["lse_p"], np.full(T, float(rank))], 1))
        gathered = parallel.gather_shard_records(packed)
        out_q.put((rank, gathered.numpy()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gather_shard_records_in_column_order():
    T, V, world = 12, 4096, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_vocab_worker, args=(r, world, port, T, V, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert np.array_equal(res[0], res[1]) and res[0].shape == (world, T, 3)
    assert np.all(res[0][0, :, 2] == 0) and np.all(res[0][1, :, 2] == 1)
    # the merge identity the device kernel uses: log sum_s exp(lse_s) is the row's log-sum-exp
    r = LogitRecipe(T=T, V=V, dtype="bf16", sigma0=2.5, peaks=4, sigma=1.2, seed=10)
    za, zp, tok = make_logits(r, "cpu", block_rows=T)
    whole = oracle.lse_gather(to_numpy_bits(za), to_numpy_bits(zp), np.zeros(T, np.int32))
    merged = np.logaddexp(res[0][0, :, 0], res[0][1, :, 0])
    assert np.allclose(merged, whole["lse_a"], rtol=0, atol=1e-12)
