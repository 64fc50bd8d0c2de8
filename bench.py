#!/usr/bin/env python
"""Benchmark of the OBRS token pass (libjackpot) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg2_qwen3|cfg3_batch|cfg4_sweep|cfg5_train|sparse_actor|lmhead_fused|
                                fused_forward|vocab_shards|vocab_widths]

A step is one pass of the whole path over one batch of synthetic logits:

  cfg2_qwen3 (default)  one jp_obrs_forward over T=4096 tokens, V=151936, bf16, k=32, lambda=2
                        (row stream with online softmax and both top-k lists, acceptance, decision,
                        Z_approx, kappa, weights); the line also carries forward+backward on the
                        same batch, the end-to-end rate from host buffers and the CPU oracle;
  cfg3_batch            64 padded responses (131,072 rows, ~58 % valid) streamed in 16 chunks of 8192
                        rows, lambda from an acceptance budget of 0.6, k=64 (jp_batch_begin / chunk /
                        finalize); the unit is a valid token;
  cfg4_sweep            16,384 rows at three actor/policy mismatches and k in {8, 32, 128, V}: twelve
                        forwards per step, Z_approx against the exact Z and throughput per point;
  cfg5_train            32,768 rows in 4 chunks: chunked forward with a budget of 0.5 and a weight
                        clip, then one fused backward per chunk (bf16 gradients of both tensors).

  sparse_actor          the cfg2 shape through jp_obrs_forward_sparse_actor: only the policy tensor is
                        streamed (303,872 B per token), the rollout model comes as the record the
                        paper's rollout phase stores (log p_inf(a_t) and its 20 best log-probs).
  lmhead_fused          one model's row pass fused into its output layer (jp_lmhead_lse_topk): 4096 hidden
                        states of width 2048 against the [151936, 2048] bf16 output matrix on the tensor
                        cores; log-sum-exp, token log-prob and top-20 straight from the accumulator.
  fused_forward         the whole forward with both models' output layers fused (jp_obrs_forward_lmhead): two
                        such passes, the partner logits of the list entries, then acceptance, Z_approx, kappa
                        and weights; neither logit tensor is stored.
  vocab_shards          the cfg2 batch split by columns over 8 vocabulary shards: one rank's share (local
                        pass of its slice, merge of all shards' records, finalize); 2 and 4 shards beside it.
  vocab_widths          the row stream at vocabulary widths from 8 K to 262 K columns, rows scaled so that
                        every point streams the same 2.4 GB.

Every workload prints one JSON line with `roofline` (the dominant kernel, timed per launch by CUDA
events on the stream it runs on), `cpu_baseline` (the oracle on a bounded sample, all host cores and
one) and `e2e` (host buffers through jp_obrs_forward_host, or null with the reason).  With --gpus N
every rank runs its own batch of the same shape (rows are independent: weak scaling, no data-path
collective); started without torchrun, the script starts its N ranks itself.
"""
from __future__ import annotations

import argparse
import glob
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

UNIT = "tokens/s"
METRICS = {"cfg2_qwen3": "obrs_forward_tokens_per_s", "cfg3_batch": "obrs_forward_tokens_per_s",
           "cfg4_sweep": "obrs_forward_tokens_per_s", "cfg5_train": "obrs_fwd_bwd_tokens_per_s",
           "sparse_actor": "obrs_forward_tokens_per_s", "lmhead_fused": "lmhead_row_pass_tokens_per_s",
           "vocab_shards": "obrs_forward_tokens_per_s", "vocab_widths": "obrs_forward_tokens_per_s",
           "fused_forward": "obrs_forward_tokens_per_s"}
LMHEAD = dict(T=4096, H=2048, k=20)    # hidden size of the paper's 1.7B rollout model; its default top-k count
SPARSE_K_INF = 20            # the rollout stores its 20 most likely tokens (the paper's default top-k count)
DATASHEET_GBS = 8000.0


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples, taken from start() to stop()."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, pw, reasons, rows_all = [], [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                s_, m_, p_ = float(c[1]), float(c[2]), float(c[3])
            except ValueError:
                continue
            rows_all.append((s_, m_, p_, c[5:9]))
            if p_ < 250.0:            # an idle sample between two timed regions says nothing about the load
                continue
            sm.append(s_)
            mx.append(m_)
            pw.append(p_)
            for n, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        note = "samples under load (board power >= 250 W)"
        if not sm and rows_all:       # a run too short for the power reading to rise: take what there is
            note = "the timed regions were too short for a sample under load: all samples"
            for s_, m_, p_, flags in rows_all:
                sm.append(s_)
                mx.append(m_)
                pw.append(p_)
                for n, v in zip(names, flags):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_mhz_min=sm[0], sm_max_mhz=max(mx), power_w_max=max(pw),
                       reasons=sorted(reasons), samples=len(sm), note=note)
        return out


def _recipe(r0, T, seed, sigma=None):
    from paper_2602_06107_b200.inputs import LogitRecipe
    return LogitRecipe(T=T, V=r0.V, dtype=r0.dtype, sigma0=r0.sigma0, peaks=r0.peaks, peak_lo=r0.peak_lo,
                       peak_hi=r0.peak_hi, sigma=r0.sigma if sigma is None else sigma, seed=seed)


def _workload(name):
    from paper_2602_06107_b200.inputs import CONFIGS
    if name == "sparse_actor":                 # the headline shape, the rollout model as a stored record
        return CONFIGS["cfg2_qwen3"]
    if name in ("lmhead_fused", "fused_forward", "vocab_shards", "vocab_widths"):
        return CONFIGS["cfg2_qwen3"]
    if name not in METRICS:
        raise SystemExit(f"bench.py: workload {name!r} is not a bench line (choose from {sorted(METRICS)}); "
                         "the tiny exact-check shape is a parity test, see tests/")
    return CONFIGS[name]


# ---------------------------------------------------------------------------------------------------
# the oracle on the host cores (cpu_baseline leg and the reference arm)

def _oracle_sample(name, cfg, rows, device="cpu"):
    """`rows` rows of the workload (its first chunk / first sweep point), as the oracle takes them."""
    from paper_2602_06107_b200.inputs import make_lengths_mask, make_logits, to_numpy_bits
    r0 = cfg["recipe"]
    if name in ("lmhead_fused", "fused_forward"):
        import torch
        g = torch.Generator().manual_seed(11)
        rows = min(rows, 16)                                     # 0.6 GFLOP per row in scalar double
        h = torch.randn((rows, LMHEAD["H"]), generator=g).to(torch.bfloat16)
        w = (torch.randn((r0.V, LMHEAD["H"]), generator=g) * (3.0 / LMHEAD["H"] ** 0.5)).to(torch.bfloat16)
        tok = torch.randint(0, r0.V, (rows,), generator=g, dtype=torch.int32)
        return to_numpy_bits(h), to_numpy_bits(w), tok.numpy(), None
    za, zp, tok = make_logits(_recipe(r0, rows, r0.seed), device, block_rows=rows)
    mask = None
    if name == "cfg3_batch":
        m, _ = make_lengths_mask(cfg["n_resp"], cfg["max_len"], cfg["min_len"], seed=cfg["seed"], device="cpu")
        mask = m[:rows].numpy().copy()
    return to_numpy_bits(za), to_numpy_bits(zp), tok.cpu().numpy(), mask


def _oracle_step(name, cfg, za, zp, tok, mask):
    """One pass of the oracle over the sample, with the workload's own parameters; returns the
    number of units (tokens, valid tokens for the padded batch) it processed."""
    import numpy as np

    import oracle
    n = za.shape[0]
    if name == "cfg2_qwen3":
        oracle.forward(za, zp, tok, None, lam=cfg["lam"], k=cfg["k"], seed=cfg["seed"])
        return n
    if name in ("vocab_shards", "vocab_widths"):             # the oracle knows whole rows of the headline shape only
        oracle.forward(za, zp, tok, None, lam=cfg["lam"], k=cfg["k"], seed=cfg["seed"])
        return n
    if name == "fused_forward":                              # both models' logits in double, then the dense forward
        hb, wb = za, zp
        z = oracle.lmhead_rows(np.arange(hb.shape[0]), hb, wb)
        z2 = oracle.lmhead_rows(np.arange(hb.shape[0]), hb, wb)
        oracle.forward(z, z2, tok, None, lam=1.0, k=LMHEAD["k"], seed=cfg["seed"])
        return hb.shape[0]
    if name == "lmhead_fused":
        hb, wb = za, zp                                          # the sample carries hidden states and the matrix here
        z = oracle.lmhead_rows(np.arange(hb.shape[0]), hb, wb)
        oracle.lse_gather(z, z, tok, None)
        oracle.topk(z, LMHEAD["k"], None)
        return hb.shape[0]
    if name == "sparse_actor":
        lq, idx, logp = oracle.rollout_record(za, tok, SPARSE_K_INF)      # the rollout engine's part, not the path's
        oracle.forward_sparse(zp, tok, lq, idx, logp, None, lam=cfg["lam"], k=cfg["k"], seed=cfg["seed"])
        return n
    if name == "cfg3_batch":
        oracle.forward(za, zp, tok, mask, budget=cfg["budget"], k=cfg["k"], seed=cfg["seed"])
        return int((mask != 0).sum())
    if name == "cfg4_sweep":
        for k in cfg["ks"]:
            oracle.forward(za, zp, tok, None, lam=cfg["lam"], k=min(k, za.shape[1]), seed=cfg["seed"])
        return n * len(cfg["ks"])
    ref = oracle.forward(za, zp, tok, None, budget=cfg["budget"], k=cfg["k"], seed=cfg["seed"], c1=cfg["c1"])
    adv = np.ones(n, np.float32)
    oracle.grad_rows(np.arange(n), za, zp, tok, ref["accept"], ref["w"], ref["lse_a"], ref["lse_p"],
                     float(ref["stats"]["n_valid"]), adv=adv, lambda_distill=cfg["lambda_distill"])
    return n


def _time_oracle(name, cfg, sample, seconds, threads=None):
    import oracle
    all_threads = oracle.num_threads()
    if threads is not None:
        oracle.set_num_threads(threads)
    try:
        if name not in ("lmhead_fused", "fused_forward"):
            _oracle_step(name, cfg, *[None if x is None else x[:8] for x in sample])
        t0, units, reps = time.perf_counter(), 0, 0
        while time.perf_counter() - t0 < seconds:
            units += _oracle_step(name, cfg, *sample)
            reps += 1
        dt = time.perf_counter() - t0
        return units / dt, reps, dt, oracle.num_threads()
    finally:
        if threads is not None:
            oracle.set_num_threads(all_threads)


def cpu_baseline_for(name, cfg, sample):
    rows = sample[0].shape[0]
    v, reps, dt, cores = _time_oracle(name, cfg, sample, 8.0)
    one = [None if x is None else x[:max(8, rows // 8)] for x in sample]
    if name in ("lmhead_fused", "fused_forward"):
        one = [sample[0][:2], sample[1], sample[2][:2], None]       # the matrix stays whole: two rows of hidden states
    v1, reps1, dt1, _ = _time_oracle(name, cfg, one, 6.0, threads=1)
    what = {"cfg2_qwen3": "forward", "fused_forward": "both models' logits of the rows in double, then the dense forward", "vocab_shards": "forward on whole rows (the oracle does not shard)",
            "vocab_widths": "forward at V = 151,936 only", "lmhead_fused": "logits of the rows in double, then log-sum-exp and top-k", "sparse_actor": "forward from the policy logits and the stored record (making "
            "the record from the actor's logits is inside the timed region: it costs about as much again)", "cfg3_batch": "forward with the budget solve, valid tokens",
            "cfg4_sweep": "the four k of one sweep point", "cfg5_train": "forward + both gradients"}[name]
    return {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {rows} rows of the workload, {what}, {reps} passes, {dt:.1f} s",
            "single_thread": {"value": v1, "unit": UNIT, "cores": 1,
                              "sample": f"first {one[0].shape[0]} rows, {reps1} passes, {dt1:.1f} s"}}


def run_reference(args, rank):
    """The reference arm: the CPU oracle, as it stands, on this machine's host cores, each step a
    bounded sample of the workload's rows."""
    if rank != 0:
        return
    import oracle
    cfg = _workload(args.workload)
    r = cfg["recipe"]
    rows = args.ref_rows
    sample = _oracle_sample(args.workload, cfg, rows)
    rows = sample[0].shape[0]
    for _ in range(args.warmup):
        _oracle_step(args.workload, cfg, *sample)
    t0, units = time.perf_counter(), 0
    for _ in range(args.steps):
        units += _oracle_step(args.workload, cfg, *sample)
    dt = time.perf_counter() - t0
    val = units / dt
    cores = oracle.num_threads()
    line = {"impl": "reference", "metric": METRICS[args.workload], "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": args.workload, "T": r.T, "V": r.V, "logits": r.dtype,
                       "sample": f"{rows} rows of the workload per step"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{rows} rows x {args.steps} steps of {args.workload}"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
# the library on the GPU

class Bench:
    """What every workload needs: device, ranks, context, timing."""

    def __init__(self, args, rank, world, local_rank):
        import torch
        import torch.distributed as dist

        from paper_2602_06107_b200 import binding as B
        from paper_2602_06107_b200 import build as jp_build
        self.torch, self.dist, self.B = torch, dist, B
        self.args, self.rank, self.world = args, rank, world
        if not torch.cuda.is_available():
            raise SystemExit("bench.py: no CUDA device; libjackpot has no CPU path")
        torch.cuda.set_device(local_rank)
        self.dev = torch.device("cuda", local_rank)
        if world > 1:
            dist.init_process_group("nccl", device_id=self.dev)
        if rank == 0:
            jp_build.build()
        if world > 1:
            dist.barrier()
        self.ctx = B.Context(local_rank)
        self.local_rank = local_rank
        self.peak, self.peak_kind = _peaks()
        self.sampler = None

    def sync_all(self):
        self.torch.cuda.synchronize(self.dev)
        if self.world > 1:
            self.dist.barrier()
            self.torch.cuda.synchronize(self.dev)

    def max_over_ranks(self, x):
        if self.world > 1:
            t = self.torch.tensor([x], device=self.dev, dtype=self.torch.float64)
            self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
            x = float(t.item())
        return x

    def timed(self, fn, steps, warmup):
        """Device time of `steps` calls (CUDA events on the stream the library launches on, which is
        torch's current stream), barrier and device sync on both sides, max over ranks."""
        torch = self.torch
        for _ in range(warmup):
            fn()
        self.sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        self.sync_all()
        return self.max_over_ranks(e0.elapsed_time(e1))

    def timed_with_kernel_times(self, fn, steps, warmup, launches_per_step):
        """timed(), then the device time of every row-stream launch over the last steps again, with the
        library's per-launch events on (they are off while the headline figure is taken: two event
        records per launch cost a little stream time)."""
        B = self.B
        l0 = self.ctx.launch_count()
        ms = self.timed(fn, steps, warmup)
        launches = (self.ctx.launch_count() - l0) // (steps + warmup)
        n_steps = min(steps, 256 // launches_per_step)
        B.jp_enable_kernel_timing(self.ctx, True)
        self.timed(fn, n_steps, 0)
        kt = B.jp_stream_kernel_times(self.ctx, n_steps * launches_per_step)
        B.jp_enable_kernel_timing(self.ctx, False)
        return ms, launches, kt

    def roofline(self, kernel, alg_bytes, kernel_ms, **extra):
        achieved = alg_bytes / (kernel_ms * 1e-3) / 1e9
        r = {"bound": "hbm", "achieved": achieved, "peak": self.peak, "unit": "GB/s", "frac": achieved / self.peak,
             "traffic": None, "peak_kind": f"of {self.peak_kind} (copy bandwidth; the 80 % target is judged on this one)",
             "frac_of_datasheet_8tbs": achieved / DATASHEET_GBS, "kernel": kernel, "kernel_ms": kernel_ms,
             "algorithmic_bytes": alg_bytes}
        r.update(extra)
        return r

    def add_probe_rates(self, roof, a, b):
        """This GPU's plain streaming rates, measured now with the library's probe kernel: the forward
        only reads its logits, so the read-only rate is the tighter reference beside the copy rate."""
        try:
            ro = self.B.jp_probe_stream(a, None, reps=20)
            roof["read_only_gbs_now"] = ro
            if b is not None:
                roof["copy_gbs_now"] = self.B.jp_probe_stream(a, b, reps=10)
            roof["frac_of_read_only_now"] = roof["achieved"] / ro
        except Exception as exc:                               # a measurement aid must not lose the line
            roof["probe_error"] = str(exc)

    def add_traffic(self, roof, key, units):
        """DRAM bytes per launch of the row stream, from an ncu capture of a smaller case scaled by
        rows (traffic is proportional to the rows streamed); null unless the capture was taken
        from the kernel source as it stands."""
        tr = os.path.join(ROOT, "profiles", "traffic.json")
        if not os.path.exists(tr):
            return
        with open(tr) as f:
            t = json.load(f)
        import hashlib
        with open(os.path.join(ROOT, "paper_2602_06107_b200", "csrc", "jp_stream.cu"), "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()[:16]
        ent = t.get(key)
        if ent and ent.get("source_sha256_16") == digest:
            roof["traffic"] = ent["dram_bytes_per_row"] * units

    def stream_kernel_name(self, dtype, k, V):
        if k >= V:
            return f"prep_rows_kernel + stream_kernel<{dtype}, no top-k> (exact mode; exact_z_kernel follows)"
        kpl = 1 if k <= 32 else 2 if k <= 64 else 4
        return f"prep_rows_kernel + stream_kernel<{dtype}, {32 * kpl}-entry lists> (k = {k})"


def wl_cfg2(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import runner
    from paper_2602_06107_b200.inputs import make_logits
    r0 = cfg["recipe"]
    T = args.T or r0.T
    r = _recipe(r0, T, r0.seed + 1000 * b.rank)
    k, lam, seed = cfg["k"], cfg["lam"], cfg["seed"]
    za, zp, tok = make_logits(r, b.dev)
    V, esize = r.V, za.element_size()
    B.jp_reserve(b.ctx, T, V, k)
    out = runner._alloc_outputs(T, b.dev)
    desc = B.make_desc(za)

    def fwd():
        B.jp_obrs_forward(b.ctx, desc, za, zp, tok, None, lam, k, seed, out["accept"], out["weight"],
                          out["logp_actor"], out["logp_policy"], out["stats_buf"])

    ms, launches, kt = b.timed_with_kernel_times(fwd, args.steps, args.warmup, 1)
    stats = B.read_stats(out["stats_buf"])
    k_ms = sum(kt) / len(kt)
    alg = 2.0 * stats["n_valid"] * V * esize
    roof = b.roofline(b.stream_kernel_name(r.dtype, k, V) + ": one forward's row stream", alg, k_ms,
                      kernel_ms_min=min(kt), kernel_ms_max=max(kt))
    b.add_probe_rates(roof, za, zp)
    b.add_traffic(roof, "cfg2_qwen3", stats["n_valid"])

    # forward + backward on the same batch (fused gradients of both tensors)
    adv = torch.randn(T, device=b.dev)
    d_a, d_p = torch.empty_like(za), torch.empty_like(zp)
    bwd = B.make_bwd_desc(adv, 1.0, 1.0, 0, 0)

    def bwd_only():
        B.jp_obrs_backward(b.ctx, desc, bwd, za, zp, tok, None, out["accept"], out["weight"], d_a, d_p)

    def fwd_bwd():
        fwd()
        bwd_only()

    steps_b = max(3, min(args.steps // 2, 100))
    ms_fb = b.timed(fwd_bwd, steps_b, 3)
    ms_b = b.timed(bwd_only, steps_b, 3)
    del d_a, d_p
    bw_gbs = 4.0 * T * V * esize / (ms_b / steps_b * 1e-3) / 1e9
    fb = {"value": b.world * T * steps_b / (ms_fb * 1e-3), "unit": UNIT, "ms_per_step": ms_fb / steps_b,
          "backward_ms": ms_b / steps_b, "backward_gbs": bw_gbs, "backward_frac_of_peak": bw_gbs / b.peak}

    # end to end from pinned host buffers through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        hza, hzp, htok = za.cpu().pin_memory(), zp.cpu().pin_memory(), tok.cpu().pin_memory()
        hacc = torch.empty(T, dtype=torch.uint8).pin_memory()
        hw, hlq, hlp = (torch.empty(T, dtype=torch.float32).pin_memory() for _ in range(3))
        hst = torch.zeros(B.STATS_BYTES, dtype=torch.uint8).pin_memory()
        hdesc = B.make_desc(hza)

        def e2e_step():
            B.jp_obrs_forward_host(b.ctx, hdesc, hza, hzp, htok, None, lam, k, seed, hacc, hw, hlq, hlp, hst, 0)

        e2e_steps = max(2, min(args.steps, 5))
        for _ in range(2):
            e2e_step()
        b.sync_all()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        b.sync_all()
        dt = b.max_over_ranks(time.perf_counter() - t0)
        e2e = {"value": b.world * T * e2e_steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": int(2 * T * V * esize + 4 * T),
               "d2h_bytes_per_step": int(T * 13 + B.STATS_BYTES), "ms_per_step": 1e3 * dt / e2e_steps}
        assert torch.equal(hacc.to(b.dev), out["accept"]), "host-buffer path disagrees with the device path"
        del hza, hzp
    return dict(ms=ms, units_per_step=T, launches=launches, roofline=roof, e2e=e2e, extra={"fwd_bwd": fb},
                config={"T": T, "V": V, "logits": r.dtype, "k": k, "lambda": lam, "seed": seed,
                        "l2": f"inputs {2 * T * V * esize / 1e9:.2f} GB per step exceed the 126 MB L2; no flush needed",
                        "stats": {n: stats[n] for n in ("alpha_hat", "kappa", "z_approx_mean")}})


E2E_NULL = ("not measured for this workload: its host buffers would be {gb:.0f} GB of pinned memory per rank; the "
            "host-buffer entry point is PCIe-bound and its rate is the default workload's e2e figure")


def wl_cfg3(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import runner
    from paper_2602_06107_b200.inputs import make_lengths_mask, make_logits
    r0, chunk, k = cfg["recipe"], cfg["chunk"], cfg["k"]
    T, V = r0.T, r0.V
    mask, _ = make_lengths_mask(cfg["n_resp"], cfg["max_len"], cfg["min_len"], seed=cfg["seed"] + 1000 * b.rank,
                                device=b.dev)
    n_valid = int(mask.sum().item())
    parts = [make_logits(_recipe(r0, chunk, r0.seed + 17 * c + 1000 * b.rank), b.dev, block_rows=2048)
             for c in range(T // chunk)]
    B.jp_reserve(b.ctx, T, V, k)
    out = runner._alloc_outputs(T, b.dev)
    descs = [B.make_desc(p[0], token_offset=c * chunk) for c, p in enumerate(parts)]
    masks = [mask[c * chunk:(c + 1) * chunk] for c in range(len(parts))]
    fdesc = B.jp_obrs_desc()

    def step():
        B.jp_batch_begin(b.ctx, T, V, B.JP_BF16, k, 0.0)
        for d, (za, zp, tok), m in zip(descs, parts, masks):
            B.jp_batch_chunk(b.ctx, d, za, zp, tok, m)
        B.jp_batch_finalize(b.ctx, fdesc, cfg["budget"], B.JP_LAMBDA_FROM_BUDGET, cfg["seed"], out["accept"],
                            out["weight"], out["logp_actor"], out["logp_policy"], out["stats_buf"])

    nch = len(parts)
    ms, launches, kt = b.timed_with_kernel_times(step, args.steps, args.warmup, nch)
    stats = B.read_stats(out["stats_buf"])
    assert stats["n_valid"] == n_valid and stats["status"] == 0
    k_ms = sum(kt) / (len(kt) // nch)                        # the sixteen launches of one step
    alg = 2.0 * n_valid * V * 2
    per_chunk = [sum(kt[i::nch]) / len(kt[i::nch]) for i in range(nch)]
    roof = b.roofline(b.stream_kernel_name(r0.dtype, k, V) + f": the {nch} row-stream launches of one step", alg, k_ms,
                      chunk_ms=per_chunk, chunk_valid_rows=[int(m.sum().item()) for m in masks])
    b.add_probe_rates(roof, parts[0][0], parts[0][1])
    b.add_traffic(roof, "cfg3_batch", n_valid)
    return dict(ms=ms, units_per_step=n_valid, launches=launches, roofline=roof,
                e2e={"value": None, "reason": E2E_NULL.format(gb=2 * T * V * 2 / 1e9)}, extra={},
                config={"T": T, "valid_tokens": n_valid, "V": V, "logits": r0.dtype, "k": k, "budget": cfg["budget"],
                        "chunks": nch, "unit": "valid tokens (padding rows are not read)",
                        "padded_rows_per_s": b.world * T * args.steps / (ms * 1e-3),
                        "l2": f"inputs {2 * T * V * 2 / 1e9:.1f} GB resident, {alg / 1e9:.1f} GB read per step: far beyond L2",
                        "stats": {n: stats[n] for n in ("lambda_used", "alpha_hat", "mean_accept_prob", "kappa")}})


def wl_cfg4(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import runner
    from paper_2602_06107_b200.inputs import make_logits
    r0, lam, seed = cfg["recipe"], cfg["lam"], cfg["seed"]
    T, V = r0.T, r0.V
    B.jp_reserve(b.ctx, T, V, 128)
    data = [make_logits(_recipe(r0, T, r0.seed + si + 1000 * b.rank, sigma=s), b.dev, block_rows=2048)
            for si, s in enumerate(cfg["sigmas"])]
    out = runner._alloc_outputs(T, b.dev)
    zk = torch.empty(T, dtype=torch.float32, device=b.dev)
    points = [(si, k) for si in range(len(data)) for k in cfg["ks"]]
    descs = {}
    for si, (za, _, _) in enumerate(data):
        d = B.make_desc(za)
        d.z_approx = zk.data_ptr()
        descs[si] = d

    def point(si, k):
        za, zp, tok = data[si]
        B.jp_obrs_forward(b.ctx, descs[si], za, zp, tok, None, lam, k, seed, out["accept"], out["weight"],
                          out["logp_actor"], out["logp_policy"], out["stats_buf"])

    def step():
        for si, k in points:
            point(si, k)

    npt = len(points)
    ms, launches, kt = b.timed_with_kernel_times(step, args.steps, args.warmup, npt)
    per_point_ms = [sum(kt[i::npt]) / len(kt[i::npt]) for i in range(npt)]
    # outside the timed region: every point once more on its own (CUDA events around the whole
    # forward), and the normaliser error against the exact value
    table, zx = [], {}
    for si in range(len(data)):
        point(si, V)
        torch.cuda.synchronize()
        zx[si] = zk.double().clone()
    for i, (si, k) in enumerate(points):
        one = b.timed(lambda: point(si, k), 5, 2) / 5
        st = B.read_stats(out["stats_buf"])
        passes = 2 if k >= V else 1
        gbs = passes * 2.0 * T * V * 2 / (one * 1e-3) / 1e9
        table.append({"sigma": cfg["sigmas"][si], "k": int(k), "forward_ms": one, "stream_kernel_ms": per_point_ms[i],
                      "tokens_per_s": T / (one * 1e-3), "gb_per_s": gbs, "frac": gbs / b.peak,
                      "stream_kernel_frac": 2.0 * T * V * 2 / (per_point_ms[i] * 1e-3) / 1e9 / b.peak,
                      "mean_abs_zk_over_z_minus_1": float(((zk.double() / zx[si]) - 1.0).abs().mean().item()),
                      "kappa": st["kappa"], "alpha_hat": st["alpha_hat"]})
    k_ms = sum(per_point_ms)
    alg = npt * 2.0 * T * V * 2
    roof = b.roofline(f"prep_rows_kernel + stream_kernel<{r0.dtype}> at k in {list(cfg['ks'])}: the {npt} row-stream "
                      "launches of one step (exact mode's second pass, exact_z_kernel, is not in this figure)",
                      alg, k_ms)
    b.add_probe_rates(roof, data[0][0], data[0][1])
    return dict(ms=ms, units_per_step=T * npt, launches=launches, roofline=roof,
                e2e={"value": None, "reason": E2E_NULL.format(gb=len(data) * 2 * T * V * 2 / 1e9)},
                extra={"sweep": table},
                config={"T": T, "V": V, "logits": r0.dtype, "lambda": lam, "sigmas": list(cfg["sigmas"]),
                        "ks": [int(k) for k in cfg["ks"]], "forwards_per_step": npt,
                        "l2": "every forward reads 9.96 GB (19.9 GB in exact mode): far beyond L2"})


def wl_cfg5(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import runner
    from paper_2602_06107_b200.inputs import make_logits
    r0, chunk, k = cfg["recipe"], cfg["chunk"], cfg["k"]
    T, V = r0.T, r0.V
    B.jp_reserve(b.ctx, T, V, k)
    parts = [make_logits(_recipe(r0, chunk, r0.seed + 31 * c + 1000 * b.rank), b.dev, block_rows=2048)
             for c in range(T // chunk)]
    grads = [(torch.empty_like(za), torch.empty_like(zp)) for za, zp, _ in parts]
    g = torch.Generator(device="cpu").manual_seed(cfg["seed"])
    adv = torch.randn(T // chunk, generator=g).repeat_interleave(chunk).to(b.dev)      # one draw per response
    out = runner._alloc_outputs(T, b.dev)
    nch = len(parts)
    descs = [B.make_desc(p[0], token_offset=c * chunk) for c, p in enumerate(parts)]
    fdesc = B.jp_obrs_desc()
    fdesc.c1 = cfg["c1"]
    bdescs = [B.make_bwd_desc(adv[c * chunk:(c + 1) * chunk], cfg["lambda_distill"], 1.0, 0, c * chunk)
              for c in range(nch)]

    def forward():
        B.jp_batch_begin(b.ctx, T, V, B.JP_BF16, k, 0.0)
        for d, (za, zp, tok) in zip(descs, parts):
            B.jp_batch_chunk(b.ctx, d, za, zp, tok, None)
        B.jp_batch_finalize(b.ctx, fdesc, cfg["budget"], B.JP_LAMBDA_FROM_BUDGET, cfg["seed"], out["accept"],
                            out["weight"], out["logp_actor"], out["logp_policy"], out["stats_buf"])

    def backward():
        for c, (za, zp, tok) in enumerate(parts):
            sl = slice(c * chunk, (c + 1) * chunk)
            B.jp_obrs_backward(b.ctx, descs[c], bdescs[c], za, zp, tok, None, out["accept"][sl], out["weight"][sl],
                               grads[c][0], grads[c][1])

    def step():
        forward()
        backward()

    ms, launches, kt = b.timed_with_kernel_times(step, args.steps, args.warmup, nch)
    stats = B.read_stats(out["stats_buf"])
    assert stats["status"] == 0
    steps2 = max(3, min(args.steps, 20))
    ms_b = b.timed(backward, steps2, 2) / steps2
    ms_f = b.timed(forward, steps2, 2) / steps2
    alg_b = 4.0 * T * V * 2
    roof = b.roofline("grad_kernel<bf16> (reads both rows, writes both bf16 gradient rows): the "
                      f"{nch} backward launches of one step", alg_b, ms_b)
    k_ms = sum(kt) / (len(kt) // nch)
    fw = b.roofline(b.stream_kernel_name(r0.dtype, k, V) + f": the {nch} row-stream launches of one step",
                    2.0 * T * V * 2, k_ms, forward_ms=ms_f)
    b.add_probe_rates(fw, parts[0][0], parts[0][1])
    roof["copy_gbs_now"] = fw.get("copy_gbs_now")
    return dict(ms=ms, units_per_step=T, launches=launches, roofline=roof,
                e2e={"value": None, "reason": E2E_NULL.format(gb=2 * T * V * 2 / 1e9)},
                extra={"forward_roofline": fw, "forward_ms": ms_f, "backward_ms": ms_b,
                       "ideal_tokens_per_s_at_peak": b.peak * 1e9 / (6.0 * V * 2)},
                config={"T": T, "V": V, "logits": r0.dtype, "k": k, "budget": cfg["budget"], "c1": cfg["c1"],
                        "lambda_distill": cfg["lambda_distill"], "chunks": nch,
                        "l2": f"{6 * T * V * 2 / 1e9:.1f} GB moved per step: far beyond L2",
                        "stats": {n: stats[n] for n in ("lambda_used", "alpha_hat", "kappa")}})


def wl_sparse(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import runner
    from paper_2602_06107_b200.inputs import make_logits
    r0 = cfg["recipe"]
    T = r0.T
    r = _recipe(r0, T, r0.seed + 1000 * b.rank)
    k, lam, seed = cfg["k"], cfg["lam"], cfg["seed"]
    za, zp, tok = make_logits(r, b.dev)
    V, esize = r.V, zp.element_size()
    # the rollout record (input data: what a rollout engine stores per token), then the actor's logits go
    lq_all = torch.empty((T,), dtype=torch.float32, device=b.dev)
    inf_idx = torch.empty((T, SPARSE_K_INF), dtype=torch.int32, device=b.dev)
    inf_logp = torch.empty((T, SPARSE_K_INF), dtype=torch.float32, device=b.dev)
    for o in range(0, T, 512):
        lsm = torch.log_softmax(za[o:o + 512].float(), dim=1)
        v, i = lsm.topk(SPARSE_K_INF, dim=1)
        inf_idx[o:o + 512], inf_logp[o:o + 512] = i.to(torch.int32), v
        lq_all[o:o + 512] = lsm.gather(1, tok[o:o + 512].long()[:, None])[:, 0]
    del za, lsm
    B.jp_reserve(b.ctx, T, V, k)
    out = runner._alloc_outputs(T, b.dev)
    desc = B.make_desc(zp)

    def fwd():
        B.jp_obrs_forward_sparse_actor(b.ctx, desc, zp, tok, None, lq_all, inf_idx, inf_logp, SPARSE_K_INF, lam, k, seed,
                                       out["accept"], out["weight"], out["logp_policy"], None, None, out["stats_buf"])

    ms, launches, kt = b.timed_with_kernel_times(fwd, args.steps, args.warmup, 1)
    stats = B.read_stats(out["stats_buf"])
    k_ms = sum(kt) / len(kt)
    alg = 1.0 * stats["n_valid"] * V * esize
    roof = b.roofline(f"prep_rows_kernel + stream_kernel<{r.dtype}, {32 if k <= 32 else 64 if k <= 64 else 128}-entry list, "
                      f"policy tensor only> (k = {k}): one forward's row stream", alg, k_ms,
                      kernel_ms_min=min(kt), kernel_ms_max=max(kt))
    b.add_probe_rates(roof, zp, None)
    e2e = {"value": None, "reason": "the host-buffer entry point exists for the dense forward only"}
    return dict(ms=ms, units_per_step=T, launches=launches, roofline=roof, e2e=e2e, extra={},
                config={"T": T, "V": V, "logits": r.dtype, "k": k, "k_inf": SPARSE_K_INF, "lambda": lam, "seed": seed,
                        "record": "log p_inf(a_t) and the 20 best log-probs per token, from torch.log_softmax / topk "
                                  "of the synthetic actor logits",
                        "l2": f"inputs {T * V * esize / 1e9:.2f} GB per step exceed the 126 MB L2; no flush needed",
                        "stats": {n: stats[n] for n in ("alpha_hat", "kappa", "z_approx_mean")}})


def wl_lmhead(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    T, H, k = LMHEAD["T"], LMHEAD["H"], LMHEAD["k"]
    V = cfg["recipe"].V
    g = torch.Generator(device=b.dev).manual_seed(11 + 1000 * b.rank)
    h = torch.randn((T, H), generator=g, device=b.dev).to(torch.bfloat16)
    w = (torch.randn((V, H), generator=g, device=b.dev) * (3.0 / H ** 0.5)).to(torch.bfloat16)
    tok = torch.randint(0, V, (T,), generator=g, device=b.dev, dtype=torch.int32)
    lse, lp = torch.empty(T, device=b.dev), torch.empty(T, device=b.dev)
    idx = torch.empty((T, k), dtype=torch.int32, device=b.dev)
    val = torch.empty((T, k), device=b.dev)
    st = torch.zeros(1, dtype=torch.int32, device=b.dev)

    def step():
        B.jp_lmhead_lse_topk(b.ctx, h, w, tok, None, k, lse, lp, idx, val, st)

    l0 = b.ctx.launch_count()
    ms = b.timed(step, args.steps, args.warmup)
    launches = (b.ctx.launch_count() - l0) // (args.steps + args.warmup)
    assert st.item() == 0, "a wait inside the fused kernel ran out"
    flops = 2.0 * T * V * H
    peaks = {}
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            peaks = json.load(f)
    long_run = ms > 500.0                                     # longer than about half a second: the board's power limit rules
    peak = float(peaks.get("bf16_tflops_sustained" if long_run else "bf16_tflops", 1404.0 if long_run else 1590.0))
    achieved = flops / (ms / args.steps * 1e-3) / 1e12
    roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
            "traffic": None, "peak_kind": ("of measured" if peaks else "of fallback") + (" (sustained)" if long_run else " (burst)"),
            "frac_of_sustained": achieved / float(peaks.get("bf16_tflops_sustained", 1404.0)),
            "kernel": "lmhead_kernel (tcgen05.mma 128x256x16 bf16 -> fp32 in TMEM, TMA operand ring, epilogue from the "
                      "accumulator) + lmhead_merge_kernel; timed together by CUDA events around the call",
            "kernel_ms": ms / args.steps, "algorithmic_flops": flops,
            "operand_bytes": float(V * H * 2 + T * H * 2)}
    return dict(ms=ms, units_per_step=T, launches=launches, roofline=roof,
                e2e={"value": None, "reason": "inputs are a model's hidden states and output matrix, resident on the device in "
                                              "any use of this call; there is no host-buffer entry point for it"},
                extra={}, dtype="bf16",
                config={"T": T, "H": H, "V": V, "k": k, "operands": "bf16 hidden [T, H] and weight [V, H], N(0,1) and "
                        "N(0, 9/H) draws: logits ~ N(0, 9)", "logits_never_stored_bytes": float(T) * V * 2,
                        "l2": f"the output matrix ({V * H * 2 / 1e6:.0f} MB) exceeds the 126 MB L2; no flush needed"})


def wl_vocab_shards(b: Bench, cfg):
    """One rank's share of the vocabulary-parallel forward.  The shards run one after the other on this
    GPU to fill the gathered buffer (a rank has one of them); shard 0's three phases are what a step times."""
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import parallel, runner
    from paper_2602_06107_b200.inputs import make_logits
    r0 = cfg["recipe"]
    r = _recipe(r0, r0.T, r0.seed + 1000 * b.rank)
    za, zp, tok = make_logits(r, b.dev)
    T, V = za.shape
    k, lam, seed = cfg["k"], cfg["lam"], cfg["seed"]
    words = B.jp_vshard_record_floats(k)
    out = runner._alloc_outputs(T, b.dev)
    fdesc = B.jp_obrs_desc()
    table, headline = [], None
    for n in (2, 4, 8):
        bounds = [parallel.shard_columns(V, n, s) for s in range(n)]
        gathered = torch.empty((n, T, words), device=b.dev)
        for s_, (lo, hi) in enumerate(bounds):
            zs, ps = za[:, lo:hi], zp[:, lo:hi]
            B.jp_vshard_local(b.ctx, B.make_desc(zs), zs, ps, tok, None, lo, V, k, gathered[s_])
        lo, hi = bounds[0]
        zs, ps = za[:, lo:hi], zp[:, lo:hi]
        d0 = B.make_desc(zs)

        def local():
            B.jp_vshard_local(b.ctx, d0, zs, ps, tok, None, lo, V, k, gathered[0])

        def merge():
            B.jp_vshard_merge(b.ctx, n, 0, gathered, T, V, k)

        def finalize():
            B.jp_batch_finalize(b.ctx, fdesc, lam, B.JP_LAMBDA_FIXED, seed, out["accept"], out["weight"],
                                out["logp_actor"], out["logp_policy"], out["stats_buf"])

        def step():
            local()
            merge()
            finalize()

        if n == 8:
            ms, launches, kt = b.timed_with_kernel_times(step, args.steps, args.warmup, 1)
            headline = (ms, launches, sum(kt) / len(kt), hi - lo)
        reps = max(5, min(args.steps, 50))
        # the phases one by one: events between the three calls of a step
        for _ in range(2):
            step()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(reps)]
        b.sync_all()
        for e in ev:
            e[0].record()
            local()
            e[1].record()
            merge()
            e[2].record()
            finalize()
            e[3].record()
        b.sync_all()
        t_local = sum(e[0].elapsed_time(e[1]) for e in ev) / reps
        t_merge = sum(e[1].elapsed_time(e[2]) for e in ev) / reps
        t_fin = sum(e[2].elapsed_time(e[3]) for e in ev) / reps
        t_step = t_local + t_merge + t_fin
        step()
        torch.cuda.synchronize()
        st = B.read_stats(out["stats_buf"])
        gb = 2.0 * T * (hi - lo) * 2 / 1e9
        table.append({"shards": n, "shard_columns": hi - lo, "local_ms": t_local, "local_gb_per_s": gb / (t_local * 1e-3),
                      "local_frac": gb / (t_local * 1e-3) / b.peak, "merge_ms": t_merge, "finalize_ms": t_fin,
                      "rank_total_ms": t_step, "all_gather_bytes_per_rank": T * words * 4,
                      "tokens_per_s": T / (t_step * 1e-3), "n_accept": st["n_accept"], "kappa": st["kappa"]})
    ms, launches, k_ms, width = headline
    roof = b.roofline(b.stream_kernel_name(r.dtype, k, V) + f": the row stream of one slice of {width} columns (8 shards)",
                      2.0 * T * width * 2, k_ms)
    b.add_probe_rates(roof, za, zp)
    return dict(ms=ms, units_per_step=T, launches=launches, roofline=roof,
                e2e={"value": None, "reason": "the slices of a vocabulary-parallel output layer are device-resident by construction"},
                extra={"shards": table},
                config={"T": T, "V": V, "logits": r.dtype, "k": k, "lambda": lam, "shards": 8,
                        "step": "shard 0's local pass, the merge of all 8 shards' records, finalize: one rank's share; the "
                                "all-gather between local pass and merge is not in the timed region on one GPU",
                        "l2": "the slice (311 MB) exceeds the 126 MB L2"})


def wl_vocab_widths(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import runner
    from paper_2602_06107_b200.inputs import make_logits
    r0 = cfg["recipe"]
    k, lam, seed = cfg["k"], cfg["lam"], cfg["seed"]
    widths = (8192, 18992, 32000, 50304, 65536, 128256, 151936, 262144)
    points = []
    for V in widths:
        T = int(round(4096 * 151936 / V / 148)) * 148
        r = _recipe(r0, T, r0.seed, None)
        r = type(r)(T=T, V=V, dtype=r.dtype, sigma0=r.sigma0, peaks=r.peaks, peak_lo=r.peak_lo, peak_hi=r.peak_hi,
                    sigma=r.sigma, seed=r.seed + 1000 * b.rank)
        za, zp, tok = make_logits(r, b.dev, block_rows=2048)
        out = runner._alloc_outputs(T, b.dev)
        points.append((V, T, za, zp, tok, out, B.make_desc(za)))
    B.jp_reserve(b.ctx, max(p[1] for p in points), 262144, k)

    def point(i):
        V, T, za, zp, tok, out, d = points[i]
        B.jp_obrs_forward(b.ctx, d, za, zp, tok, None, lam, k, seed, out["accept"], out["weight"], out["logp_actor"],
                          out["logp_policy"], out["stats_buf"])

    def step():
        for i in range(len(points)):
            point(i)

    npt = len(points)
    ms, launches, kt = b.timed_with_kernel_times(step, args.steps, args.warmup, npt)
    per = [sum(kt[i::npt]) / len(kt[i::npt]) for i in range(npt)]
    table = [{"V": V, "rows": T, "stream_kernel_ms": per[i], "gb_per_s": 2.0 * T * V * 2 / (per[i] * 1e-3) / 1e9,
              "frac": 2.0 * T * V * 2 / (per[i] * 1e-3) / 1e9 / b.peak,
              "us_per_row_per_cta": per[i] * 1e3 / (T / 148)} for i, (V, T, *_rest) in enumerate(points)]
    alg = sum(2.0 * T * V * 2 for V, T, *_r in points)
    roof = b.roofline(f"prep_rows_kernel + stream_kernel<{r0.dtype}, 32-entry lists> over {npt} vocabulary widths", alg, sum(per))
    return dict(ms=ms, units_per_step=sum(p[1] for p in points), launches=launches, roofline=roof,
                e2e={"value": None, "reason": "a sweep of the row stream alone"}, extra={"widths": table},
                config={"widths": list(widths), "k": k, "lambda": lam, "logits": r0.dtype,
                        "rows": "scaled so that every width streams about 2.4 GB, a multiple of 148",
                        "l2": "every point exceeds the 126 MB L2"})


def wl_fused_forward(b: Bench, cfg):
    torch, B, args = b.torch, b.B, b.args
    from paper_2602_06107_b200 import runner
    T, H, k = LMHEAD["T"], LMHEAD["H"], LMHEAD["k"]
    V, seed = cfg["recipe"].V, cfg["seed"]
    g = torch.Generator(device=b.dev).manual_seed(12 + 1000 * b.rank)
    ha = torch.randn((T, H), generator=g, device=b.dev).to(torch.bfloat16)
    wa = (torch.randn((V, H), generator=g, device=b.dev) * (3.0 / H ** 0.5)).to(torch.bfloat16)
    hp = ha.clone()
    wp = (wa.float() + torch.randn((V, H), generator=g, device=b.dev) * (1.0 / H ** 0.5)).to(torch.bfloat16)
    tok = torch.randint(0, V, (T,), generator=g, device=b.dev, dtype=torch.int32)
    out = runner._alloc_outputs(T, b.dev)
    d = B.jp_obrs_desc()
    d.T, d.V = T, V

    def step():
        B.jp_obrs_forward_lmhead(b.ctx, d, ha, wa, hp, wp, tok, None, 1.0, k, seed, out["accept"], out["weight"],
                                 out["logp_actor"], out["logp_policy"], out["stats_buf"])

    l0 = b.ctx.launch_count()
    ms = b.timed(step, args.steps, args.warmup)
    launches = (b.ctx.launch_count() - l0) // (args.steps + args.warmup)
    st = B.read_stats(out["stats_buf"])
    assert st["status"] == 0
    flops = 2.0 * 2.0 * T * V * H + 2.0 * T * 2 * k * H * 2          # two output layers, and the partner logits
    peaks = {}
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            peaks = json.load(f)
    long_run = ms > 500.0
    peak = float(peaks.get("bf16_tflops_sustained" if long_run else "bf16_tflops", 1404.0 if long_run else 1590.0))
    achieved = flops / (ms / args.steps * 1e-3) / 1e12
    roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak, "traffic": None,
            "peak_kind": ("of measured" if peaks else "of fallback") + (" (sustained)" if long_run else " (burst)"),
            "frac_of_sustained": achieved / float(peaks.get("bf16_tflops_sustained", 1404.0)),
            "kernel": "the whole step: 2 x (lmhead_kernel + lmhead_merge_kernel), fused_records_kernel, epilogue, finalize; "
                      "timed together by CUDA events (the two tcgen05 kernels are 98 % of it)",
            "kernel_ms": ms / args.steps, "algorithmic_flops": flops}
    return dict(ms=ms, units_per_step=T, launches=launches, roofline=roof, dtype="bf16",
                e2e={"value": None, "reason": "inputs are two models' hidden states and output matrices, resident on the device "
                                              "in any use of this call"},
                extra={},
                config={"T": T, "H": H, "V": V, "k": k, "lambda": 1.0,
                        "tokens": "uniform draws (the sampled token enters only O(T) scalars; kappa is not meaningful here)",
                        "logits_never_stored_bytes": 2.0 * T * V * 2,
                        "l2": "the output matrices (2 x 622 MB) exceed the 126 MB L2; no flush needed",
                        "stats": {n: st[n] for n in ("alpha_hat", "kappa", "z_approx_mean")}})


WORKLOADS = {"fused_forward": wl_fused_forward, "vocab_shards": wl_vocab_shards, "vocab_widths": wl_vocab_widths, "lmhead_fused": wl_lmhead, "sparse_actor": wl_sparse, "cfg2_qwen3": wl_cfg2, "cfg3_batch": wl_cfg3, "cfg4_sweep": wl_cfg4, "cfg5_train": wl_cfg5}


def _nccl_summary(log_dir, world):
    """What the communicator's own log says: ranks, and whether in-switch reduction is on."""
    if not log_dir:
        return None
    text = ""
    for p in glob.glob(os.path.join(log_dir, "*")):
        try:
            with open(p, errors="replace") as f:
                text += f.read()
        except OSError:
            pass
    return {"init_complete_lines": text.count("Init COMPLETE"), "nranks_expected": world,
            "nvls_mentioned": "NVLS" in text}


def run_ours(args, rank, world, local_rank):
    cfg = _workload(args.workload)
    b = Bench(args, rank, world, local_rank)
    sampler = ClockSampler(local_rank) if rank == 0 else None       # alive across every timed region
    res = WORKLOADS[args.workload](b, cfg)
    clocks = sampler.stop() if sampler else None
    if rank != 0:
        return
    cpu_baseline = None
    if not args.no_cpu_baseline:
        cpu_baseline = cpu_baseline_for(args.workload, cfg, _oracle_sample(args.workload, cfg, args.ref_rows))
    ms = res["ms"]
    roof = res["roofline"]
    if clocks and clocks.get("sm_mhz"):
        roof["kernel_ms_x_sm_mhz"] = roof["kernel_ms"] * clocks["sm_mhz"]
    config = {"workload": args.workload}
    config.update(res["config"])
    config["parallelism"] = f"rows x{world}: every rank its own batch" if world > 1 else "1 gpu"
    if world > 1:
        config["nccl"] = _nccl_summary(os.environ.get("JP_BENCH_NCCL_LOG_DIR"), world)
    line = {"metric": METRICS[args.workload], "value": world * res["units_per_step"] * args.steps / (ms * 1e-3),
            "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": res.get("dtype", "f32"), "data": "synthetic", "config": config, "clocks": clocks, "e2e": res["e2e"],
            "gpu_launches": int(res["launches"]), "roofline": roof}
    line.update(res["extra"])
    line["cpu_baseline"] = cpu_baseline
    print(json.dumps(line))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def relaunch_with_ranks(args):
    """`python bench.py --gpus N` without a launcher: start the N ranks here (one process per GPU,
    rendezvous on 127.0.0.1) and pass their output through; rank 0 prints the one line."""
    env = dict(os.environ)
    log_dir = tempfile.mkdtemp(prefix="jp_bench_nccl_")
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", os.path.join(log_dir, "nccl.%h.%p.log"))   # keeps stdout to the one JSON line
    env["JP_BENCH_NCCL_LOG_DIR"] = log_dir
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd, env=env))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps (default: 1000 for cfg2_qwen3, 10 for the others)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_qwen3")
    ap.add_argument("--T", type=int, default=0, help="override the row count (cfg2_qwen3 only)")
    ap.add_argument("--ref-rows", type=int, default=256, help="rows in the CPU oracle's bounded sample")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.steps <= 0:
        args.steps = (1000 if args.workload == "cfg2_qwen3" else 10) if args.impl == "ours" else 20
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.T and args.workload != "cfg2_qwen3":
        raise SystemExit("bench.py: --T applies to cfg2_qwen3 only")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        relaunch_with_ranks(args)
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} ranks")
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
