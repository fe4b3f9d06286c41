#!/usr/bin/env python
"""Benchmark of the operator-split linear layer (forward + backward) on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--k-split 8] [--split out|red]

A step is one pass of the whole hot path over one batch of synthetic input: forward
Y = X W^T, then backward dX, dW, db, all k slices in slice-major order.  The workload is the
"split sweep" shape (M = 16384 tokens, N = K = 8192, bf16, fp32 accumulate) at k = 8 along the
output dimension: the configuration on which the metric's three parts (TFLOP/s, fraction of the
bf16 tensor peak, overhead versus the unsplit layer) are defined.  One JSON line is printed by
rank 0.  The path does not shard (single-GPU operator, no collective): with --gpus N each rank
runs an independent replica and the value is the aggregate ("replicas only", weak scaling).

The reference arm (--impl reference) times the fp64 CPU oracle on a bounded sample of the same
workload on the host cores; it is a deliberately slow program, a reported baseline only.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = {"name": "split sweep GEMM M=16384 N=K=8192 bf16", "M": 16384, "N": 8192, "K": 8192,
            "x_std": 1.0, "w_std": 0.02, "dy_std": 1.0}
METRIC = "split-linear fwd+bwd TFLOP/s"
UNIT = "TFLOP/s"

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture of this
# very command at full size, summarised in profiles/bench_split_sweep_k8_launch_list.md.
NCU_TRAFFIC_BYTES = {
    ("fwd", 8, "out"): 2711566336 + 255925504,
    ("dx", 8, "out"): 5495490304 + 4003963648,
    ("dw", 8, "out"): 2611305472 + 118412032,
}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def flops_per_step(M, N, K):
    return 3 * 2.0 * M * N * K     # forward, dX, dW; bias, db and activation work not counted


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.stop_flag = threading.Event()
        self.proc = None

    def run(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                if self.stop_flag.is_set():
                    break
                parts = [p.strip() for p in line.split(",")]
                if len(parts) >= 6:
                    self.samples.append(parts)
        except Exception:
            pass

    def stop(self):
        self.stop_flag.set()
        if self.proc is not None:
            try:
                self.proc.terminate()     # the exact child started above
            except Exception:
                pass

    def summary(self):
        sm = []
        reasons = set()
        mx = None
        for p in self.samples:
            try:
                sm.append(float(p[0]))
                mx = float(p[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(value, world, device=None):
    """Max of a float over all ranks (identity for one rank)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(flops_per_rank_step, steps, world, max_ms_total):
    """Whole-job TFLOP/s: work of all ranks over the slowest rank's time."""
    return flops_per_rank_step * steps * world / (max_ms_total * 1e-3) / 1e12


# ---------------------------------------------------------------------------------------------
# CPU oracle legs

_SAMPLE_CACHE = {}


def oracle_sample_run(k, split_name, rows):
    """One fwd+bwd of the oracle on `rows` tokens of the workload (same N, K, k, split).
    Input generation and widening to fp64 are outside the timed part.
    Returns (seconds, flops, cores)."""
    import oracle
    from paper_2209_13258_b200 import inputs
    N, K = WORKLOAD["N"], WORKLOAD["K"]
    if rows not in _SAMPLE_CACHE:
        c = inputs.linear_case(rows, N, K, w_std=WORKLOAD["w_std"])
        _SAMPLE_CACHE[rows] = (oracle.as_f64(c["x"]), oracle.as_f64(c["w"]), oracle.as_f64(c["dy"]))
    X, W, DY = _SAMPLE_CACHE[rows]
    split = oracle.SPLIT_OUT if split_name == "out" else oracle.SPLIT_RED
    t0 = time.perf_counter()
    z, y = oracle.linear_fwd(X, W, None, oracle.ACT_NONE, k, split)
    oracle.linear_bwd(DY, X, W, None, oracle.ACT_NONE, k, split)
    dt = time.perf_counter() - t0
    return dt, flops_per_step(rows, N, K), oracle.num_threads()


def run_reference(args):
    rank, world, _ = dist_setup(args.gpus)
    if rank != 0:
        return 0
    rows = args.ref_rows
    for _ in range(max(min(args.warmup, 1), 0)):
        oracle_sample_run(args.k_split, args.split, rows)
    fl = 0.0
    total = 0.0
    cores = 1
    for _ in range(args.steps):
        dt, f, cores = oracle_sample_run(args.k_split, args.split, rows)
        fl += f
        total += dt
    value = fl / total / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "%d of %d token rows, full N and K, k=%d %s, fwd+bwd per step" % (
                             rows, WORKLOAD["M"], args.k_split, args.split)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def config_dict(args):
    return {"workload": WORKLOAD["name"], "M": WORKLOAD["M"], "N": WORKLOAD["N"], "K": WORKLOAD["K"],
            "k_split": args.k_split, "split_dim": args.split, "act": "none", "accumulate": "fp32 (TMEM)",
            "carry": "fp32 running sum in the workspace (exact)",
            "l2": "inputs larger than L2 (X, W, dY, outputs total 1.07 GB per step)",
            "parallelism": "replicas only" if args.gpus > 1 else "single GPU"}


# ---------------------------------------------------------------------------------------------
# CUDA arm

def run_ours(args):
    import numpy as np
    import torch
    import paper_2209_13258_b200 as P
    from paper_2209_13258_b200 import inputs

    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the split-linear path has no CPU fallback")
    if rank == 0:
        from paper_2209_13258_b200.build import build as build_osdp
        build_osdp()          # no-op when the in-tree library is up to date
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    P.lib()

    M, N, K = WORKLOAD["M"], WORKLOAD["N"], WORKLOAD["K"]
    k = args.k_split
    split = P.SPLIT_OUT if args.split == "out" else P.SPLIT_RED
    case = inputs.linear_case(M, N, K, w_std=WORKLOAD["w_std"], layer=rank)

    def pinned(bits):
        t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
        return t.pin_memory()

    h_x, h_dy, h_w = pinned(case["x"]), pinned(case["dy"]), pinned(case["w_flat"])
    x = h_x.to(dev); dy = h_dy.to(dev); w_flat = h_w.to(dev)
    out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    dx = torch.empty(M, K, dtype=torch.bfloat16, device=dev)
    dw_flat = torch.empty(N * K, dtype=torch.bfloat16, device=dev)
    db = torch.empty(N, dtype=torch.float32, device=dev)
    h_out = torch.empty(M, N, dtype=torch.bfloat16).pin_memory()
    h_dx = torch.empty(M, K, dtype=torch.bfloat16).pin_memory()
    h_dw = torch.empty(N * K, dtype=torch.bfloat16).pin_memory()
    h_db = torch.empty(N, dtype=torch.float32).pin_memory()

    def workspace(kk, sp, fl=0):
        _, a = P.osdp_split_linear_workspace_bytes(M, N, K, kk, sp, P.ACT_NONE, P.OP_LINEAR_FWD, fl)
        _, b = P.osdp_split_linear_workspace_bytes(M, N, K, kk, sp, P.ACT_NONE, P.OP_LINEAR_BWD, fl)
        return max(a, b)

    ws_bytes = workspace(k, split)
    ws = P.new_workspace(ws_bytes, dev)
    stream = torch.cuda.current_stream()

    def fwd(kk=k, sp=split, w=ws, fl=0):
        P.osdp_split_linear_fwd(x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, out, None, w, check=True, flags=fl)

    def bwd_dx(kk=k, sp=split, w=ws, fl=0):
        P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, dx, None, 0, P.DTYPE_BF16, fl,
                                None, w, check=True)

    def bwd_dw(kk=k, sp=split, w=ws):
        P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, None, dw_flat, 0,
                                P.DTYPE_BF16, 0, None, w, check=True)

    def bwd_db(kk=k, sp=split, w=ws):
        P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, None, None, 0, P.DTYPE_BF16, 0,
                                db, w, check=True)

    def step(kk=k, sp=split, w=ws, fl=0):
        fwd(kk, sp, w, fl); bwd_dx(kk, sp, w, fl); bwd_dw(kk, sp, w); bwd_db(kk, sp, w)

    launches_per_step = 5     # fwd GEMM, dX GEMM, dW GEMM, column-sum partial + final

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    # ---- headline: device-resident inputs, K steps, per-GEMM launch durations measured live
    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(args.warmup):
        step()
    barrier()
    if sampler:
        sampler.start()
        time.sleep(0.3)
    names = ("fwd", "dx", "dw", "db")
    fns = (fwd, bwd_dx, bwd_dw, bwd_db)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(fns) + 1)] for _ in range(args.steps)]
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for s in range(args.steps):
        evs[s][0].record(stream)
        for i, fn in enumerate(fns):
            fn()
            evs[s][i + 1].record(stream)
    e1.record(stream)
    barrier()
    if sampler:
        time.sleep(0.2)
        sampler.stop()
    ms_total = e0.elapsed_time(e1)
    per_kernel_ms = {n: sum(evs[s][i].elapsed_time(evs[s][i + 1]) for s in range(args.steps)) / args.steps
                     for i, n in enumerate(names)}
    ms_total = max_over_ranks(ms_total, world, dev)
    fl = flops_per_step(M, N, K)
    value = aggregate_value(fl, args.steps, world, ms_total)
    rc, st = P.osdp_read_device_status(ws)
    if rc != 0 or st != 0:
        raise SystemExit("device status %d/%d after the timed region" % (rc, st))

    # ---- overhead versus the unsplit layer and the other split dimension, same process
    # The configurations are run round-robin (one timed step each per round) so that clock and
    # power drift over the measurement hits all of them alike; medians are reported.
    sweep = {}
    if rank == 0 and not args.no_sweep:
        cfgs = [(1, P.SPLIT_OUT, 0, "k1"), (k, P.SPLIT_OUT, 0, "k%d_out" % k), (k, P.SPLIT_RED, 0, "k%d_red" % k),
                (k, P.SPLIT_OUT, P.FLAG_CARRY_BF16, "k%d_out_bf16_running_sum" % k),
                (k, P.SPLIT_RED, P.FLAG_CARRY_BF16, "k%d_red_bf16_running_sum" % k),
                (k, P.SPLIT_OUT, P.FLAG_PAIR_SLICES, "k%d_out_paired_slices" % k),
                (k, P.SPLIT_RED, P.FLAG_PAIR_SLICES, "k%d_red_paired_slices" % k)]
        need = max(workspace(kk, sp, f) for kk, sp, f, _ in cfgs)
        w2 = ws if need <= ws_bytes else P.new_workspace(need, dev)
        times = {label: [] for _, _, _, label in cfgs}
        for rnd in range(2 + max(args.steps // 2, 5)):
            for kk, sp, f, label in cfgs:
                a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
                a.record(stream); step(kk, sp, w2, f); b.record(stream); torch.cuda.synchronize()
                if rnd >= 2:
                    times[label].append(a.elapsed_time(b))
        for kk, sp, f, label in cfgs:
            ms = sorted(times[label])[len(times[label]) // 2]
            sweep[label] = {"ms_per_step": ms, "tflops": fl / ms / 1e9, "staging_bytes": workspace(kk, sp, f)}
        for label in list(sweep):
            sweep[label]["overhead_vs_k1"] = sweep[label]["ms_per_step"] / sweep["k1"]["ms_per_step"] - 1.0
        del w2

    # ---- the transformer MLP block of the small model configuration (hidden 1024, ffn 4096, 8 x 512
    # tokens, Linear -> GeLU -> Linear split along ffn, k = 1, 2, 4, 8): forward + backward, same round-robin
    # timing.  Secondary figures; the headline above is the split-sweep operator.
    mlp_block = {}
    if rank == 0 and not args.no_sweep:
        Mm, Hh, Ff = 4096, 1024, 4096
        xm = torch.randn(Mm, Hh, device=dev).bfloat16()
        dym = torch.randn(Mm, Hh, device=dev).bfloat16()
        off1, off2 = 0, Ff * Hh
        wfm = (torch.randn(2 * Ff * Hh, device=dev) * 0.02).bfloat16()
        b1m = torch.zeros(Ff, device=dev); b2m = torch.zeros(Hh, device=dev)
        outm = torch.empty(Mm, Hh, device=dev, dtype=torch.bfloat16); dxm = torch.empty_like(outm)
        z1m = torch.empty(Mm, Ff, device=dev, dtype=torch.bfloat16)
        dwm = torch.empty(2 * Ff * Hh, device=dev, dtype=torch.bfloat16)
        db1m = torch.empty(Ff, device=dev); db2m = torch.empty(Hh, device=dev)
        ks = (1, 2, 4, 8)
        wsm = {}
        for kk in ks:
            n1 = P.osdp_split_linear_workspace_bytes(Mm, Ff, Hh, kk, P.SPLIT_OUT, P.ACT_GELU_TANH, P.OP_MLP_FWD)[1]
            n2 = P.osdp_split_linear_workspace_bytes(Mm, Ff, Hh, kk, P.SPLIT_OUT, P.ACT_GELU_TANH, P.OP_MLP_BWD)[1]
            wsm[kk] = (P.new_workspace(max(n1, n2), dev), max(n1, n2))

        def mlp_step(kk):
            P.osdp_split_mlp_fwd(xm, wfm, off1, b1m, off2, b2m, Mm, Hh, Ff, kk, P.ACT_GELU_TANH, outm, z1m, wsm[kk][0],
                                 stream=stream, check=True)
            P.osdp_split_mlp_bwd(dym, xm, wfm, off1, off2, z1m, Mm, Hh, Ff, kk, P.ACT_GELU_TANH, dxm, dwm, off1, off2,
                                 P.DTYPE_BF16, 0, db1m, db2m, wsm[kk][0], stream=stream, check=True)
        tm = {kk: [] for kk in ks}
        reps = 6          # steps per sample, issued back to back: a step is shorter than the host needs to issue it
        for rnd in range(12):
            for kk in ks:
                a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(reps):
                    mlp_step(kk)
                b.record(stream); torch.cuda.synchronize()
                if rnd >= 2:
                    tm[kk].append(a.elapsed_time(b) / reps)
        flm = 6 * 2.0 * Mm * Hh * Ff
        for kk in ks:
            ms = sorted(tm[kk])[len(tm[kk]) // 2]
            mlp_block["k%d" % kk] = {"ms_per_step": ms, "tflops": flm / ms / 1e9, "staging_bytes": wsm[kk][1]}
        for kk in ks:
            mlp_block["k%d" % kk]["overhead_vs_k1"] = mlp_block["k%d" % kk]["ms_per_step"] / mlp_block["k1"]["ms_per_step"] - 1.0
        del wsm
    # ---- the same operator with fp8 (e4m3) operands, k = 1 and the headline split (secondary figures)
    fp8 = {}
    if rank == 0 and not args.no_sweep:
        x8 = torch.randn(M, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
        w8 = torch.randn(N * K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
        dy8 = torch.randn(M, N, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
        need = max(workspace(1, P.SPLIT_OUT), workspace(k, P.SPLIT_OUT))
        w8s = P.new_workspace(need, dev)

        def f8_step(kk):
            P.osdp_split_linear_fwd_f8(x8, w8, 0, 1.0, None, M, N, K, kk, P.SPLIT_OUT, 0, out, None, w8s, stream=stream,
                                       check=True)
            P.osdp_split_linear_bwd_f8(dy8, x8, w8, 0, 1.0, 1.0, M, N, K, kk, P.SPLIT_OUT, dx, dw_flat, 0,
                                       P.DTYPE_BF16, 0, w8s, stream=stream, check=True)
        t8 = {1: [], k: []}
        for rnd in range(10):
            for kk in t8:
                a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
                a.record(stream); f8_step(kk); b.record(stream); torch.cuda.synchronize()
                if rnd >= 2:
                    t8[kk].append(a.elapsed_time(b))
        for kk in t8:
            ms = sorted(t8[kk])[len(t8[kk]) // 2]
            fp8["k%d_out" % kk] = {"ms_per_step": ms, "tflops": fl / ms / 1e9,
                                   "frac_of_2x_measured_bf16_burst": fl / ms / 1e9 / (2 * peaks()["bf16_tflops"])}
        del w8s, x8, w8, dy8
    if world > 1:
        barrier()

    # ---- end to end: every step copies its inputs in from pinned host memory and all its results
    # out to pinned host memory.  Three streams (copy-in, compute, copy-out) and two sets of device
    # buffers, so that step i+1's inputs arrive and step i-1's results leave while step i computes.
    # The library calls are the same C-ABI calls, issued on the compute stream.
    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    bufs = []
    for _ in range(2):
        bufs.append({"x": torch.empty_like(x), "dy": torch.empty_like(dy), "out": torch.empty_like(out),
                     "dx": torch.empty_like(dx), "dw": torch.empty_like(dw_flat), "db": torch.empty_like(db),
                     "in_done": torch.cuda.Event(), "cmp_done": torch.cuda.Event(), "out_done": torch.cuda.Event()})
    ws_e2e = [ws, P.new_workspace(ws_bytes, dev)]

    def e2e_run(n):
        for i in range(n):
            b = bufs[i % 2]
            with torch.cuda.stream(s_in):
                s_in.wait_event(b["cmp_done"])          # the step that last read these inputs has finished
                b["x"].copy_(h_x, non_blocking=True); b["dy"].copy_(h_dy, non_blocking=True)
                b["in_done"].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(b["in_done"])
                s_cmp.wait_event(b["out_done"])         # its previous results have been copied out
                w = ws_e2e[i % 2]
                P.osdp_split_linear_fwd(b["x"], w_flat, 0, None, M, N, K, k, split, P.ACT_NONE, b["out"], None, w,
                                        check=True)
                P.osdp_split_linear_bwd(b["dy"], b["x"], w_flat, 0, None, M, N, K, k, split, P.ACT_NONE, b["dx"],
                                        b["dw"], 0, P.DTYPE_BF16, 0, b["db"], w, check=True)
                b["cmp_done"].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(b["cmp_done"])
                h_out.copy_(b["out"], non_blocking=True); h_dx.copy_(b["dx"], non_blocking=True)
                h_dw.copy_(b["dw"], non_blocking=True); h_db.copy_(b["db"], non_blocking=True)
                b["out_done"].record(s_out)

    e2e_steps = max(min(args.steps, 10), 2)
    e2e_run(2)
    barrier()
    t0 = time.perf_counter()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record(s_in)
    e2e_run(e2e_steps)
    for st in (s_in, s_cmp):
        s_out.wait_stream(st)
    e1.record(s_out)
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev)
    e2e_value = aggregate_value(fl, e2e_steps, world, ms_e2e)
    h2d = (h_x.numel() + h_dy.numel()) * 2
    d2h = (h_out.numel() + h_dx.numel() + h_dw.numel()) * 2 + h_db.numel() * 4

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel (the slowest of the three GEMM launches)
    pk = peaks()
    dom = max(("fwd", "dx", "dw"), key=lambda n: per_kernel_ms[n])
    gemm_flops = 2.0 * M * N * K
    achieved = gemm_flops / (per_kernel_ms[dom] * 1e-3) / 1e12
    timed_seconds = ms_total * 1e-3
    peak_kind = "bf16_tflops_sustained" if timed_seconds >= 1.0 else "bf16_tflops"
    roofline = {"bound": "tensor", "kernel": "gemm_kernel (%s GEMM)" % dom, "achieved": achieved,
                "peak": pk[peak_kind], "unit": "TFLOP/s", "frac": achieved / pk[peak_kind],
                "peak_kind": "%s, %s" % (peak_kind, pk["source"]),
                "frac_of_burst_peak": achieved / pk["bf16_tflops"],
                "per_launch_ms": per_kernel_ms, "traffic": NCU_TRAFFIC_BYTES.get((dom, k, args.split))}
    # Both floors of that launch: tensor time of its flops, and HBM time of its algorithmic bytes (operands once per
    # slice that re-reads them, plus 2 x 4 bytes x (k - 1) per element of a summed output for the fp32 carry).
    carried = (dom == "dx" and args.split == "out") or (dom == "fwd" and args.split == "red")
    alg_bytes = {"fwd": 2.0 * ((k if args.split == "out" else 1) * M * K + N * K + M * N),
                 "dx": 2.0 * ((k if args.split == "red" else 1) * M * N + N * K + M * K),
                 "dw": 2.0 * (M * N + N * K + M * K + (k - 1) * (M * K if args.split == "out" else M * N))}[dom]
    if carried:
        alg_bytes += 8.0 * (k - 1) * (M * K if dom == "dx" else M * N)
    roofline["algorithmic_bytes"] = alg_bytes
    roofline["tensor_floor_ms"] = gemm_flops / (pk[peak_kind] * 1e12) * 1e3
    roofline["hbm_floor_ms"] = alg_bytes / (pk["hbm_gbs"] * 1e9) * 1e3

    # ---- CPU baseline: the oracle, as it stands, on a bounded sample of the same workload
    cpu = None
    if not args.no_cpu_baseline:
        dt, f, cores = oracle_sample_run(k, args.split, args.ref_rows)
        cpu = {"value": f / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dt,
               "sample": "%d of %d token rows, full N and K, k=%d %s, one fwd+bwd" % (args.ref_rows, M, k, args.split)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": config_dict(args),
        "frac_of_bf16_peak": {"measured_burst_1658": value / world / pk["bf16_tflops"],
                              "measured_sustained_1378": value / world / pk["bf16_tflops_sustained"],
                              "datasheet_2250": value / world / 2250.0},
        "sweep": sweep, "mlp_block_hidden1024_ffn4096_tokens4096": mlp_block,
        "fp8_e4m3_operands": fp8, "staging_bytes": ws_bytes,
        "roofline": roofline, "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / e2e_steps,
                "how": "pinned host -> device copies, C-ABI fwd+bwd, device -> pinned host copies, every step; "
                       "copy-in / compute / copy-out on three streams over two buffer sets"},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": sampler.summary() if sampler else None,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--k-split", type=int, default=8)
    ap.add_argument("--split", default="out", choices=["out", "red"])
    ap.add_argument("--ref-rows", type=int, default=1024,
                    help="token rows in the oracle's bounded sample (1024 rows = 4.1e11 flop, about 8 s on 16 cores)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
