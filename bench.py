#!/usr/bin/env python
"""Benchmark of the OBRS token pass (libjackpot) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2_qwen3]

A step is one forward pass of the whole path (row stream with online softmax and
both top-k lists, acceptance, decision, Z_approx, kappa, weights) over one batch
of synthetic logits of the Qwen3 shape: T=4096 tokens, V=151936, bf16, k=32,
lambda=2.0.  The same JSON line also reports the forward+backward step on the
same batch (fused logit gradients for both tensors), the roofline of the row
stream kernel, the end-to-end rate from host buffers, and the CPU oracle timed
on the machine's host cores.  With --gpus N (torchrun) each rank runs its own batch
(rows are independent; weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "obrs_forward_tokens_per_s"
UNIT = "tokens/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "50"],
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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for n, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def _workload(name):
    from paper_2602_06107_b200.inputs import CONFIGS
    cfg = CONFIGS[name]
    return cfg


def run_reference(args, rank):
    """The reference arm: the CPU oracle, as it stands, on this machine's host cores,
    each step a bounded sample of the workload's rows."""
    if rank != 0:
        return
    import numpy as np
    import torch

    import oracle
    from paper_2602_06107_b200.inputs import LogitRecipe, make_logits, to_numpy_bits
    cfg = _workload(args.workload)
    r = cfg["recipe"]
    rows = args.ref_rows
    sample = LogitRecipe(T=rows, V=r.V, dtype=r.dtype, sigma0=r.sigma0, peaks=r.peaks, peak_lo=r.peak_lo,
                         peak_hi=r.peak_hi, sigma=r.sigma, seed=r.seed)
    za, zp, tok = make_logits(sample, "cpu", block_rows=rows)
    za, zp, tok = to_numpy_bits(za), to_numpy_bits(zp), tok.numpy()
    k, lam = cfg.get("k", 32), cfg.get("lam", 2.0)
    for _ in range(args.warmup):
        oracle.forward(za, zp, tok, None, lam=lam, k=k, seed=cfg["seed"])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward(za, zp, tok, None, lam=lam, k=k, seed=cfg["seed"])
    dt = time.perf_counter() - t0
    val = rows * args.steps / dt
    cores = oracle.num_threads()
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": args.workload, "T": r.T, "V": r.V, "logits": r.dtype, "k": k, "lambda": lam,
                       "sample": f"{rows} rows of the workload per step"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{rows} rows x {args.steps} steps of {args.workload}"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist

    from paper_2602_06107_b200 import binding as B
    from paper_2602_06107_b200 import build as jp_build
    from paper_2602_06107_b200 import runner
    from paper_2602_06107_b200.inputs import LogitRecipe, make_logits

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; libjackpot has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        jp_build.build()
    if world > 1:
        dist.barrier()
    cfg = _workload(args.workload)
    r0 = cfg["recipe"]
    T = args.T or r0.T
    r = LogitRecipe(T=T, V=r0.V, dtype=r0.dtype, sigma0=r0.sigma0, peaks=r0.peaks, peak_lo=r0.peak_lo,
                    peak_hi=r0.peak_hi, sigma=r0.sigma, seed=r0.seed + 1000 * rank)
    k, lam, seed = cfg.get("k", 32), cfg.get("lam", 2.0), cfg["seed"]
    za, zp, tok = make_logits(r, dev)
    V = r.V
    esize = za.element_size()
    ctx = B.Context(local_rank)
    B.jp_reserve(ctx, T, V, k)
    out = runner._alloc_outputs(T, dev)
    desc = B.make_desc(za)

    def fwd():
        B.jp_obrs_forward(ctx, desc, za, zp, tok, None, lam, k, seed, out["accept"], out["weight"],
                          out["logp_actor"], out["logp_policy"], out["stats_buf"])

    def sync_all():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        sync_all()
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    # ---- forward (the headline): device-resident inputs, per-launch stream-kernel times
    B.jp_enable_kernel_timing(ctx, True)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    l0 = ctx.launch_count()
    ms = timed(fwd, args.steps, args.warmup)
    launches = (ctx.launch_count() - l0) * args.steps // (args.steps + args.warmup)
    clocks = sampler.stop() if sampler else None
    kt = B.jp_stream_kernel_times(ctx, min(args.steps, 256))
    B.jp_enable_kernel_timing(ctx, False)
    stats = B.read_stats(out["stats_buf"])
    ms_per_step = ms / args.steps
    value = world * T * args.steps / (ms * 1e-3)
    peak, peak_kind = _peaks()
    k_ms = sum(kt) / len(kt)
    alg_bytes = 2.0 * stats["n_valid"] * V * esize
    achieved = alg_bytes / (k_ms * 1e-3) / 1e9

    # ---- forward + backward on the same batch (fused gradients of both tensors)
    adv = torch.randn(T, device=dev)
    d_a = torch.empty_like(za)
    d_p = torch.empty_like(zp)
    bwd = B.make_bwd_desc(adv, 1.0, 1.0, 0, 0)

    def fwd_bwd():
        fwd()
        B.jp_obrs_backward(ctx, desc, bwd, za, zp, tok, None, out["accept"], out["weight"], d_a, d_p)

    def bwd_only():
        B.jp_obrs_backward(ctx, desc, bwd, za, zp, tok, None, out["accept"], out["weight"], d_a, d_p)

    steps_b = max(3, min(args.steps // 2, 100))
    ms_fb = timed(fwd_bwd, steps_b, 3)
    ms_b = timed(bwd_only, steps_b, 3)
    del d_a, d_p
    fb = {"value": world * T * steps_b / (ms_fb * 1e-3), "unit": UNIT, "ms_per_step": ms_fb / steps_b,
          "backward_ms": ms_b / steps_b,
          "backward_gbs": 4.0 * T * V * esize / (ms_b / steps_b * 1e-3) / 1e9,
          "backward_frac_of_peak": 4.0 * T * V * esize / (ms_b / steps_b * 1e-3) / 1e9 / peak}

    # ---- end to end from pinned host buffers through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        hza = za.cpu().pin_memory()
        hzp = zp.cpu().pin_memory()
        htok = tok.cpu().pin_memory()
        hacc = torch.empty(T, dtype=torch.uint8).pin_memory()
        hw = torch.empty(T, dtype=torch.float32).pin_memory()
        hlq = torch.empty(T, dtype=torch.float32).pin_memory()
        hlp = torch.empty(T, dtype=torch.float32).pin_memory()
        hst = torch.zeros(B.STATS_BYTES, dtype=torch.uint8).pin_memory()
        hdesc = B.make_desc(hza)

        def e2e_step():
            B.jp_obrs_forward_host(ctx, hdesc, hza, hzp, htok, None, lam, k, seed, hacc, hw, hlq, hlp, hst, 0)

        e2e_steps = max(2, min(args.steps, 5))
        for _ in range(2):
            e2e_step()
        sync_all()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        sync_all()
        dt = time.perf_counter() - t0
        if world > 1:
            t = torch.tensor([dt], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            dt = float(t.item())
        e2e = {"value": world * T * e2e_steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": int(2 * T * V * esize + 4 * T),
               "d2h_bytes_per_step": int(T * 13 + B.STATS_BYTES), "ms_per_step": 1e3 * dt / e2e_steps}
        assert torch.equal(hacc.to(dev), out["accept"]), "host-buffer path disagrees with the device path"
        del hza, hzp

    if rank != 0:
        return
    # ---- the oracle on this machine's host cores, on a bounded sample of the same workload
    cpu_baseline = None
    if not args.no_cpu_baseline:
        import oracle
        from paper_2602_06107_b200.inputs import to_numpy_bits
        n = min(args.ref_rows, T)
        hz_a, hz_p, ht = to_numpy_bits(za[:n]), to_numpy_bits(zp[:n]), tok[:n].cpu().numpy()
        oracle.forward(hz_a[:8], hz_p[:8], ht[:8], None, lam=lam, k=k, seed=seed)
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 10.0:
            oracle.forward(hz_a, hz_p, ht, None, lam=lam, k=k, seed=seed)
            reps += 1
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": n * reps / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"first {n} rows of the batch, {reps} passes, {dt:.1f} s"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "T": T, "V": V, "logits": r.dtype, "k": k, "lambda": lam,
                   "seed": seed, "parallelism": f"rows x{world}" if world > 1 else "1 gpu",
                   "l2": f"inputs {2 * T * V * esize / 1e9:.2f} GB per step exceed the 126 MB L2; no flush needed",
                   "stats": {"alpha_hat": stats["alpha_hat"], "kappa": stats["kappa"],
                             "z_approx_mean": stats["z_approx_mean"]}},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "peak_kind": f"of {peak_kind}", "kernel": "prep_rows_kernel + stream_kernel<bf16,k<=32> (one forward's row stream)",
                     "kernel_ms": k_ms, "kernel_ms_min": min(kt), "kernel_ms_max": max(kt),
                     "algorithmic_bytes": alg_bytes},
        "fwd_bwd": fb,
        "cpu_baseline": cpu_baseline,
    }
    # this GPU's plain streaming rates, measured now with the library's probe kernel: the forward
    # only reads its logits, so the read-only rate is the tighter reference beside the copy rate
    try:
        line["roofline"]["read_only_gbs_now"] = B.jp_probe_stream(za, None, reps=20)
        line["roofline"]["copy_gbs_now"] = B.jp_probe_stream(za, zp, reps=10)
    except Exception as exc:                                   # a measurement aid must not lose the line
        line["roofline"]["probe_error"] = str(exc)
    # DRAM bytes per launch of the row stream, from an ncu capture of a smaller case
    # scaled by rows (traffic is proportional to the rows streamed); null unless the
    # capture was taken from the kernel source as it stands
    tr = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tr):
        with open(tr) as f:
            t = json.load(f)
        src = os.path.join(ROOT, "paper_2602_06107_b200", "csrc", "jp_stream.cu")
        import hashlib
        with open(src, "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()[:16]
        ent = t.get(args.workload)
        if ent and ent.get("source_sha256_16") == digest:
            line["roofline"]["traffic"] = ent["dram_bytes_per_row"] * stats["n_valid"]
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_qwen3")
    ap.add_argument("--T", type=int, default=0, help="override the workload's row count")
    ap.add_argument("--ref-rows", type=int, default=256, help="rows in the CPU oracle's bounded sample")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if world != args.gpus and world == 1 and args.gpus > 1:
        raise SystemExit("bench.py: launch with torch.distributed.run for --gpus > 1")
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
