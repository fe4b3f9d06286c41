#!/usr/bin/env python
"""Benchmark of the operator-split linear layer (forward + backward) on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--k-split 8] [--split out|red]
    python bench.py --case linear:M:N:K:k:out|red[:flags]     one fwd+bwd, twice (a small run for profilers)
    python bench.py --case f8:M:N:K:k:out|red | --case mlp:M:hidden:ffn:k

A step is one pass of the whole hot path over one batch of synthetic input: one forward call
(Y = X W^T) and one backward call (dX, dW, db), all k slices.  The workload is the "split sweep"
shape (M = 16384 tokens, N = K = 8192, bf16, fp32 accumulate) at k = 8 along the output dimension:
the configuration on which the metric's three parts (TFLOP/s, fraction of the bf16 tensor peak,
overhead versus the unsplit layer) are defined.  One JSON line is printed by rank 0; besides the
headline it carries the whole split sweep, the sustained figures, the other workload
configurations (decoder-layer linears, wide MLP block, small MLP block, the skinny single layer)
and cuBLAS (torch.matmul) measured in the same process as the like-for-like bar.
The path does not shard (single-GPU operator, no collective): with --gpus N each rank runs an
independent replica and the value is the aggregate ("replicas only", weak scaling).

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

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the three GEMM launches of a
# step at this workload's full size, k = 8, output split, from one ncu capture of
# `bench.py --case linear:16384:8192:8192:8:out`.  Refreshed whenever the kernel or its tile choice changes.
NCU_TRAFFIC_BYTES = {
    ("fwd", 8, "out"): 2709627000 + 257286400,
    ("dx", 8, "out"): 1851115000 + 258307840,
    ("dw", 8, "out"): 2350985000 + 121548544,
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
            "slice_sum": "fp32; all-slices call: kept in tensor memory across the slices of a tile (flags = 0)",
            "l2": "inputs larger than L2 (X, W, dY, outputs total 1.07 GB per step)",
            "preheat": "untimed back-to-back steps for %.1f s before the warm-up steps, so that the timed steps run "
                       "at the clocks of a long job (power cap reached)" % args.preheat,
            "parallelism": "replicas only" if args.gpus > 1 else "single GPU"}


# ---------------------------------------------------------------------------------------------
# small runs for profilers

def run_case(spec):
    import torch
    import paper_2209_13258_b200 as P
    from paper_2209_13258_b200.build import build as build_osdp
    build_osdp()
    parts = spec.split(":")
    kind = parts[0]
    dev = "cuda"
    if kind in ("linear", "f8"):
        M, N, K, k = (int(v) for v in parts[1:5])
        split = P.SPLIT_OUT if parts[5] == "out" else P.SPLIT_RED
        flags = int(parts[6]) if len(parts) > 6 else 0
        out = torch.empty(M, N, device=dev, dtype=torch.bfloat16)
        dx = torch.empty(M, K, device=dev, dtype=torch.bfloat16)
        dw = torch.empty(N, K, device=dev, dtype=torch.bfloat16)
        db = torch.empty(N, device=dev, dtype=torch.float32)
        _, a = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, 0, P.OP_LINEAR_FWD, flags)
        _, b = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, 0, P.OP_LINEAR_BWD, flags)
        ws = P.new_workspace(max(a, b))
        if kind == "linear":
            x = torch.randn(M, K, device=dev).bfloat16()
            w = (torch.randn(N, K, device=dev) * 0.02).bfloat16()
            dy = torch.randn(M, N, device=dev).bfloat16()
            for _ in range(2):
                P.osdp_split_linear_fwd(x, w, 0, None, M, N, K, k, split, 0, out, None, ws, check=True, flags=flags)
                # the three parts of the backward as launches of their own, one after another
                P.osdp_split_linear_bwd(dy, x, w, 0, None, M, N, K, k, split, 0, dx, None, 0, 0, flags, None, ws, check=True)
                P.osdp_split_linear_bwd(dy, x, w, 0, None, M, N, K, k, split, 0, None, dw, 0, 0, flags, db, ws, check=True)
                torch.cuda.synchronize()
        else:
            x8 = torch.randn(M, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
            w8 = torch.randn(N, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
            dy8 = torch.randn(M, N, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
            for _ in range(2):
                P.osdp_split_linear_fwd_f8(x8, w8, 0, 1.0, None, M, N, K, k, split, 0, out, None, ws, check=True, flags=flags)
                P.osdp_split_linear_bwd_f8(dy8, x8, w8, 0, 1.0, 1.0, M, N, K, k, split, dx, dw, 0, P.DTYPE_BF16, flags, ws,
                                           check=True)
                torch.cuda.synchronize()
    elif kind == "mlp":
        M, H, F, k = (int(v) for v in parts[1:5])
        t = _mlp_tensors(torch, dev, M, H, F)
        _, n1 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_FWD, 0)
        _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_BWD, 0)
        ws = P.new_workspace(max(n1, n2))
        for _ in range(2):
            _mlp_step(P, t, M, H, F, k, ws, None)
            torch.cuda.synchronize()
    else:
        raise SystemExit("unknown --case kind %r" % kind)
    print("device status", P.osdp_read_device_status(ws))
    return 0


def _mlp_tensors(torch, dev, M, H, F):
    return {"x": torch.randn(M, H, device=dev).bfloat16(), "dy": torch.randn(M, H, device=dev).bfloat16(),
            "wf": (torch.randn(2 * F * H, device=dev) * 0.02).bfloat16(),
            "b1": torch.zeros(F, device=dev), "b2": torch.zeros(H, device=dev),
            "out": torch.empty(M, H, device=dev, dtype=torch.bfloat16), "dx": torch.empty(M, H, device=dev, dtype=torch.bfloat16),
            "z1": torch.empty(M, F, device=dev, dtype=torch.bfloat16),
            "dw": torch.empty(2 * F * H, device=dev, dtype=torch.bfloat16),
            "db1": torch.empty(F, device=dev), "db2": torch.empty(H, device=dev)}


def _mlp_step(P, t, M, H, F, k, ws, stream):
    P.osdp_split_mlp_fwd(t["x"], t["wf"], 0, t["b1"], F * H, t["b2"], M, H, F, k, P.ACT_GELU_TANH, t["out"], t["z1"], ws,
                         stream=stream, check=True)
    P.osdp_split_mlp_bwd(t["dy"], t["x"], t["wf"], 0, F * H, t["z1"], M, H, F, k, P.ACT_GELU_TANH, t["dx"], t["dw"], 0,
                         F * H, P.DTYPE_BF16, 0, t["db1"], t["db2"], ws, stream=stream, check=True)


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
    pk = peaks()

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

    def workspace(kk, sp, fl=0, m=M, n=N, kd=K):
        _, a = P.osdp_split_linear_workspace_bytes(m, n, kd, kk, sp, P.ACT_NONE, P.OP_LINEAR_FWD, fl)
        _, b = P.osdp_split_linear_workspace_bytes(m, n, kd, kk, sp, P.ACT_NONE, P.OP_LINEAR_BWD, fl)
        return max(a, b)

    ws_bytes = workspace(k, split)
    ws = P.new_workspace(ws_bytes, dev)
    stream = torch.cuda.current_stream()

    def fwd(kk=k, sp=split, w=ws, fl=0):
        P.osdp_split_linear_fwd(x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, out, None, w, check=True, flags=fl)

    def bwd(kk=k, sp=split, w=ws, fl=0):
        P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, dx, dw_flat, 0, P.DTYPE_BF16, fl,
                                db, w, check=True)

    def bwd_dx(kk=k, sp=split, w=ws, fl=0):
        P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, dx, None, 0, P.DTYPE_BF16, fl,
                                None, w, check=True)

    def bwd_dw(kk=k, sp=split, w=ws, fl=0):
        P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, None, dw_flat, 0,
                                P.DTYPE_BF16, fl, None, w, check=True)

    def bwd_db(kk=k, sp=split, w=ws, fl=0):
        P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, sp, P.ACT_NONE, None, None, 0, P.DTYPE_BF16, fl,
                                db, w, check=True)

    def step(kk=k, sp=split, w=ws, fl=0):
        fwd(kk, sp, w, fl); bwd(kk, sp, w, fl)

    launches_per_step = 5     # fwd GEMM, dX GEMM, dW GEMM, column-sum partial + final

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def interleaved(fns, rounds=10, warm=2, reps=1):
        """Median ms per call of each callable in `fns` (label -> callable), run round-robin (one timed sample
        of `reps` back-to-back calls each per round) so that clock and power drift hits all of them alike."""
        ts = {label: [] for label in fns}
        for rnd in range(warm + rounds):
            for label, fn in fns.items():
                a, b = ev(), ev()
                a.record(stream)
                for _ in range(reps):
                    fn()
                b.record(stream)
                torch.cuda.synchronize()
                if rnd >= warm:
                    ts[label].append(a.elapsed_time(b) / reps)
        return {label: sorted(v)[len(v) // 2] for label, v in ts.items()}

    fl = flops_per_step(M, N, K)

    # ---- cold start: the first K steps after the warm-up, GPU not yet at its power cap (burst clocks)
    for _ in range(args.warmup):
        step()
    barrier()
    a, b = ev(), ev()
    a.record(stream)
    for _ in range(args.steps):
        step()
    b.record(stream)
    barrier()
    burst_ms = a.elapsed_time(b)

    # ---- pre-heat: untimed back-to-back steps until the GPU has been under load for `preheat` seconds
    t0 = time.perf_counter()
    n_pre = 0
    while time.perf_counter() - t0 < args.preheat:
        for _ in range(20):
            step()
        torch.cuda.synchronize()
        n_pre += 20

    # ---- headline: W warm-up steps, then exactly K timed steps, device-resident inputs
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    e0, e1 = ev(), ev()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    value = aggregate_value(fl, args.steps, world, ms_total)

    # ---- the same steps with every launch of the backward issued on its own (dX, dW, db one after another)
    # and an event between them: per-GEMM durations for the roofline of the dominant kernel
    names = ("fwd", "dx", "dw", "db")
    fns = (fwd, bwd_dx, bwd_dw, bwd_db)
    evs = [[ev() for _ in range(len(fns) + 1)] for _ in range(args.steps)]
    for s in range(args.steps):
        evs[s][0].record(stream)
        for i, fn in enumerate(fns):
            fn()
            evs[s][i + 1].record(stream)
    barrier()
    per_kernel_ms = {n: sum(evs[s][i].elapsed_time(evs[s][i + 1]) for s in range(args.steps)) / args.steps
                     for i, n in enumerate(names)}

    # ---- sustained: >= 2 s of back-to-back steps, unsplit and the headline split
    sustained = {}
    if rank == 0 and not args.no_sweep:
        w_k1 = P.new_workspace(workspace(1, P.SPLIT_OUT), dev)
        for label, kk, sp, w in (("k1", 1, P.SPLIT_OUT, w_k1), ("k%d_%s" % (k, args.split), k, split, ws)):
            n = max(50, int(2200.0 / (ms_total / args.steps)) + 1)
            a, b = ev(), ev()
            a.record(stream)
            for _ in range(n):
                step(kk, sp, w)
            b.record(stream)
            torch.cuda.synchronize()
            t = a.elapsed_time(b)
            sustained[label] = {"steps": n, "seconds": t / 1e3, "ms_per_step": t / n, "tflops": fl * n / t / 1e9,
                                "frac_of_measured_sustained_peak": fl * n / t / 1e9 / pk["bf16_tflops_sustained"]}
        sustained["k%d_%s" % (k, args.split)]["overhead_vs_k1"] = (
            sustained["k%d_%s" % (k, args.split)]["ms_per_step"] / sustained["k1"]["ms_per_step"] - 1.0)
        del w_k1
    if sampler:
        time.sleep(0.2)
        sampler.stop()
    rc, st = P.osdp_read_device_status(ws)
    if rc != 0 or st != 0:
        raise SystemExit("device status %d/%d after the timed region" % (rc, st))

    # ---- the split sweep: k in {1, 2, 4, 8, 16, 32} x {output, reduction}, default flags; then, labelled, the
    # slice-major order (the operator swept once per slice, fp32 carry through the workspace: what a sequence of
    # per-slice calls does) and its two carry options
    sweep = {}
    if rank == 0 and not args.no_sweep:
        SM = P.FLAG_SLICE_MAJOR
        cfgs = [(1, P.SPLIT_OUT, 0, "k1")]
        for kk in (2, 4, 8, 16, 32):
            cfgs += [(kk, P.SPLIT_OUT, 0, "k%d_out" % kk), (kk, P.SPLIT_RED, 0, "k%d_red" % kk)]
        for kk in (4, 8, 16):
            cfgs += [(kk, P.SPLIT_OUT, SM, "k%d_out_slice_major" % kk), (kk, P.SPLIT_RED, SM, "k%d_red_slice_major" % kk)]
        cfgs += [(8, P.SPLIT_OUT, SM | P.FLAG_CARRY_BF16, "k8_out_slice_major_bf16_running_sum"),
                 (8, P.SPLIT_OUT, P.FLAG_PAIR_SLICES, "k8_out_slice_major_paired_slices")]
        need = max(workspace(kk, sp, f) for kk, sp, f, _ in cfgs)
        w2 = P.new_workspace(need, dev)
        med = interleaved({label: (lambda kk=kk, sp=sp, f=f: step(kk, sp, w2, f)) for kk, sp, f, label in cfgs},
                          rounds=9, warm=2)
        for kk, sp, f, label in cfgs:
            ms = med[label]
            sweep[label] = {"ms_per_step": ms, "tflops": fl / ms / 1e9, "staging_bytes": workspace(kk, sp, f),
                            "overhead_vs_k1": ms / med["k1"] - 1.0,
                            "frac_of_measured_sustained_peak": fl / ms / 1e9 / pk["bf16_tflops_sustained"]}
        del w2

    # ---- cuBLAS (torch.matmul) on the same shape in the same process: the like-for-like bar
    like_for_like = {}
    if rank == 0 and not args.no_sweep:
        W2d = w_flat[:N * K].view(N, K)

        def torch_step():
            torch.matmul(x, W2d.t(), out=out); torch.matmul(dy, W2d, out=dx); torch.matmul(dy.t(), x, out=dw_flat.view(N, K))

        def ours_no_db(kk):
            fwd(kk, split, ws)
            P.osdp_split_linear_bwd(dy, x, w_flat, 0, None, M, N, K, kk, split, P.ACT_NONE, dx, dw_flat, 0, P.DTYPE_BF16, 0,
                                    None, ws, check=True)
        med = interleaved({"torch": torch_step, "ours_k1": lambda: ours_no_db(1), "ours_k%d" % k: lambda: ours_no_db(k)},
                          rounds=9, warm=2)
        like_for_like = {"what": "fwd + dX + dW, no bias gradient, same process, interleaved medians",
                         "torch_matmul_ms": med["torch"], "torch_matmul_tflops": fl / med["torch"] / 1e9,
                         "ours_k1_ms": med["ours_k1"], "ours_k%d_ms" % k: med["ours_k%d" % k],
                         "ours_k1_over_torch": med["ours_k1"] / med["torch"],
                         "ours_k%d_over_torch" % k: med["ours_k%d" % k] / med["torch"]}

    # ---- decoder-stack layer (hidden 2048, ffn 8192, 8 x 1024 tokens): its four linears, k = 1 and k = 4 along
    # the output dimension, next to torch.matmul on the same shapes
    decoder_layer = {}
    if rank == 0 and not args.no_sweep:
        Mm = 8192
        tot = {"k1": 0.0, "k4": 0.0, "torch": 0.0}
        tot_fl = 0.0
        for name, (Nn, Kk) in (("qkv_6144x2048", (6144, 2048)), ("proj_2048x2048", (2048, 2048)),
                               ("fc1_8192x2048", (8192, 2048)), ("fc2_2048x8192", (2048, 8192))):
            xm = torch.randn(Mm, Kk, device=dev).bfloat16(); dym = torch.randn(Mm, Nn, device=dev).bfloat16()
            wm = (torch.randn(Nn * Kk, device=dev) * 0.02).bfloat16(); W2d = wm.view(Nn, Kk)
            om = torch.empty(Mm, Nn, device=dev, dtype=torch.bfloat16); dxm = torch.empty(Mm, Kk, device=dev, dtype=torch.bfloat16)
            dwm = torch.empty(Nn * Kk, device=dev, dtype=torch.bfloat16); dbm = torch.empty(Nn, device=dev)
            wsm = P.new_workspace(max(workspace(kk, P.SPLIT_OUT, 0, Mm, Nn, Kk) for kk in (1, 4)), dev)

            def ours(kk, with_db=True):
                P.osdp_split_linear_fwd(xm, wm, 0, None, Mm, Nn, Kk, kk, P.SPLIT_OUT, 0, om, None, wsm, check=True)
                P.osdp_split_linear_bwd(dym, xm, wm, 0, None, Mm, Nn, Kk, kk, P.SPLIT_OUT, 0, dxm, dwm, 0, P.DTYPE_BF16, 0,
                                        dbm if with_db else None, wsm, check=True)

            def tm():
                torch.matmul(xm, W2d.t(), out=om); torch.matmul(dym, W2d, out=dxm); torch.matmul(dym.t(), xm, out=dwm.view(Nn, Kk))
            med = interleaved({"k1": lambda: ours(1), "k4": lambda: ours(4), "k1_no_db": lambda: ours(1, False), "torch": tm},
                              rounds=9, warm=2, reps=4)
            f3 = flops_per_step(Mm, Nn, Kk)
            decoder_layer[name] = {"k1_ms": med["k1"], "k4_ms": med["k4"], "k1_tflops": f3 / med["k1"] / 1e9,
                                   "k4_tflops": f3 / med["k4"] / 1e9, "k4_overhead_vs_k1": med["k4"] / med["k1"] - 1.0,
                                   "torch_matmul_ms": med["torch"], "torch_matmul_tflops": f3 / med["torch"] / 1e9,
                                   "k1_no_db_over_torch": med["k1_no_db"] / med["torch"]}
            for key in tot:
                tot[key] += med[key]
            tot_fl += f3
            del xm, dym, wm, om, dxm, dwm, dbm, wsm
        decoder_layer["layer_total"] = {"k1_ms": tot["k1"], "k4_ms": tot["k4"], "torch_matmul_ms": tot["torch"],
                                        "k4_tflops": tot_fl / tot["k4"] / 1e9,
                                        "k4_frac_of_measured_sustained_peak": tot_fl / tot["k4"] / 1e9 / pk["bf16_tflops_sustained"],
                                        "k4_frac_of_measured_burst_peak": tot_fl / tot["k4"] / 1e9 / pk["bf16_tflops"],
                                        "k4_overhead_vs_k1": tot["k4"] / tot["k1"] - 1.0}

    # ---- MLP blocks split along ffn (Linear -> GeLU -> Linear, fc1 output-split + fc2 reduction-split):
    # the wide-layer stress (hidden 8192, ffn 32768, 4 x 2048 tokens; k = 1, 8) and the small block
    # (hidden 1024, ffn 4096, 8 x 512 tokens; k = 1, 2, 4, 8)
    def mlp_block(Mm, Hh, Ff, ks, reps, rounds, graphs=False):
        t = _mlp_tensors(torch, dev, Mm, Hh, Ff)
        wsm = {}
        for kk in ks:
            n1 = P.osdp_split_linear_workspace_bytes(Mm, Ff, Hh, kk, P.SPLIT_OUT, P.ACT_GELU_TANH, P.OP_MLP_FWD)[1]
            n2 = P.osdp_split_linear_workspace_bytes(Mm, Ff, Hh, kk, P.SPLIT_OUT, P.ACT_GELU_TANH, P.OP_MLP_BWD)[1]
            wsm[kk] = (P.new_workspace(max(n1, n2), dev), n1, n2)
        fns = {kk: (lambda kk=kk: _mlp_step(P, t, Mm, Hh, Ff, kk, wsm[kk][0], stream)) for kk in ks}
        if graphs:
            # the same calls captured once into a CUDA graph and replayed: what a launch-bound loop of small
            # operators does in production (the calls are plain stream work, internal fork / join included)
            side = torch.cuda.Stream(dev)
            for kk in ks:
                fns[kk]()                                   # first use outside the capture
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(g, stream=side):
                        _mlp_step(P, t, Mm, Hh, Ff, kk, wsm[kk][0], torch.cuda.current_stream())
                fns["graph_k%d" % kk] = g.replay
        med = interleaved(fns, rounds=rounds, warm=2, reps=reps)
        flm = 6 * 2.0 * Mm * Hh * Ff
        res = {}
        for kk in ks:
            res["k%d" % kk] = {"ms_per_step": med[kk], "tflops": flm / med[kk] / 1e9,
                               "frac_of_measured_sustained_peak": flm / med[kk] / 1e9 / pk["bf16_tflops_sustained"],
                               "staging_fwd_bytes": wsm[kk][1], "staging_bwd_bytes": wsm[kk][2],
                               "overhead_vs_k1": med[kk] / med[ks[0]] - 1.0}
            if graphs:
                g = med["graph_k%d" % kk]
                res["k%d" % kk].update({"graph_replay_ms_per_step": g, "graph_replay_tflops": flm / g / 1e9,
                                        "graph_replay_overhead_vs_k1": g / med["graph_k%d" % ks[0]] - 1.0})
        return res

    mlp_wide, mlp_small = {}, {}
    if rank == 0 and not args.no_sweep:
        mlp_wide = mlp_block(8192, 8192, 32768, (1, 8), 1, 7)
        mlp_small = mlp_block(4096, 1024, 4096, (1, 2, 4, 8), 6, 10, graphs=True)

    # ---- the skinny single layer (X [256,512], W [2048,512], k = 4 along the output dimension): latency of one
    # forward + backward issued to an idle GPU, with the operands left in L2 by the previous step and after a flush
    # (a 256 MB buffer overwritten), and the device-side time of a step when steps are issued back to back
    skinny = {}
    if rank == 0 and not args.no_sweep:
        Ms, Ns, Ks, kk = 256, 2048, 512, 4
        xs = torch.randn(Ms, Ks, device=dev).bfloat16(); dys = torch.randn(Ms, Ns, device=dev).bfloat16()
        wsk = (torch.randn(Ns * Ks, device=dev) * 0.02).bfloat16()
        os_ = torch.empty(Ms, Ns, device=dev, dtype=torch.bfloat16); dxs = torch.empty(Ms, Ks, device=dev, dtype=torch.bfloat16)
        dws = torch.empty(Ns * Ks, device=dev, dtype=torch.bfloat16); dbs = torch.empty(Ns, device=dev)
        wss = P.new_workspace(workspace(kk, P.SPLIT_OUT, 0, Ms, Ns, Ks), dev)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

        def sstep():
            P.osdp_split_linear_fwd(xs, wsk, 0, None, Ms, Ns, Ks, kk, P.SPLIT_OUT, 0, os_, None, wss, check=True)
            P.osdp_split_linear_bwd(dys, xs, wsk, 0, None, Ms, Ns, Ks, kk, P.SPLIT_OUT, 0, dxs, dws, 0, P.DTYPE_BF16, 0, dbs,
                                    wss, check=True)
        alg_bytes = 2.0 * 3 * (Ms * Ks + Ns * Ks + Ms * Ns)
        for name, cold in (("warm_l2", False), ("cold_l2", True)):
            ts = []
            for i in range(40):
                if cold:
                    flush.fill_(i & 255)
                a, b = ev(), ev()
                torch.cuda.synchronize()
                a.record(stream); sstep(); b.record(stream)
                torch.cuda.synchronize()
                if i >= 10:
                    ts.append(a.elapsed_time(b) * 1e3)
            ts.sort()
            skinny[name] = {"median_us": ts[len(ts) // 2], "best_us": ts[0],
                            "achieved_gbs_at_median": alg_bytes / (ts[len(ts) // 2] * 1e-6) / 1e9}
        a, b = ev(), ev()
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(200):
            sstep()
        b.record(stream)
        torch.cuda.synchronize()
        us = a.elapsed_time(b) * 1e3 / 200
        skinny["back_to_back"] = {"us_per_step": us, "achieved_gbs": alg_bytes / (us * 1e-6) / 1e9,
                                  "frac_of_measured_hbm": alg_bytes / (us * 1e-6) / 1e9 / pk["hbm_gbs"]}
        # the same step captured once into a CUDA graph and replayed: the device-side time without the host's issue cost
        side = torch.cuda.Stream(dev)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                cur = torch.cuda.current_stream()
                P.osdp_split_linear_fwd(xs, wsk, 0, None, Ms, Ns, Ks, kk, P.SPLIT_OUT, 0, os_, None, wss, stream=cur, check=True)
                P.osdp_split_linear_bwd(dys, xs, wsk, 0, None, Ms, Ns, Ks, kk, P.SPLIT_OUT, 0, dxs, dws, 0, P.DTYPE_BF16, 0, dbs,
                                        wss, stream=cur, check=True)
        g.replay(); torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(200):
            g.replay()
        b.record(stream)
        torch.cuda.synchronize()
        us = a.elapsed_time(b) * 1e3 / 200
        skinny["graph_replay"] = {"us_per_step": us, "achieved_gbs": alg_bytes / (us * 1e-6) / 1e9,
                                  "frac_of_measured_hbm": alg_bytes / (us * 1e-6) / 1e9 / pk["hbm_gbs"]}
        skinny["algorithmic_bytes_per_step"] = alg_bytes
        skinny["shape"] = "M=256 N=2048 K=512 k=4 out"
        del flush

    # ---- the same operator with fp8 (e4m3) operands, k = 1 and the headline split (secondary figures)
    fp8 = {}
    if rank == 0 and not args.no_sweep:
        x8 = torch.randn(M, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
        w8 = torch.randn(N * K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
        dy8 = torch.randn(M, N, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
        SM = P.FLAG_SLICE_MAJOR
        w8s = P.new_workspace(max(workspace(1, P.SPLIT_OUT), workspace(k, P.SPLIT_OUT, SM)), dev)

        def f8_step(kk, f=0):
            P.osdp_split_linear_fwd_f8(x8, w8, 0, 1.0, None, M, N, K, kk, P.SPLIT_OUT, 0, out, None, w8s, stream=stream,
                                       check=True, flags=f)
            P.osdp_split_linear_bwd_f8(dy8, x8, w8, 0, 1.0, 1.0, M, N, K, kk, P.SPLIT_OUT, dx, dw_flat, 0,
                                       P.DTYPE_BF16, f, w8s, stream=stream, check=True)
        med = interleaved({"k1_out": lambda: f8_step(1), "k%d_out" % k: lambda: f8_step(k),
                           "k%d_out_slice_major" % k: lambda: f8_step(k, SM)}, rounds=8, warm=2)
        for label, ms in med.items():
            fp8[label] = {"ms_per_step": ms, "tflops": fl / ms / 1e9, "overhead_vs_k1": ms / med["k1_out"] - 1.0,
                          "frac_of_2x_measured_bf16_burst": fl / ms / 1e9 / (2 * pk["bf16_tflops"])}
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

    # ---- roofline of the dominant kernel (the slowest of the three GEMM launches), measured in the
    # sustained state, so against the sustained peak; the burst figures are given beside it
    dom = max(("fwd", "dx", "dw"), key=lambda n: per_kernel_ms[n])
    gemm_flops = 2.0 * M * N * K
    achieved = gemm_flops / (per_kernel_ms[dom] * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "gemm_kernel (%s GEMM)" % dom, "achieved": achieved,
                "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": achieved / pk["bf16_tflops_sustained"],
                "peak_kind": "bf16_tflops_sustained (the launches are timed after %.1f s under load), %s" % (
                    args.preheat, pk["source"]),
                "frac_of_burst_peak": achieved / pk["bf16_tflops"],
                "per_launch_ms": per_kernel_ms, "traffic": NCU_TRAFFIC_BYTES.get((dom, k, args.split))}
    # Both floors of that launch: tensor time of its flops, and HBM time of its algorithmic bytes (operands once
    # per slice that re-reads them; the default order carries nothing through memory).
    alg_bytes = {"fwd": 2.0 * ((k if args.split == "out" else 1) * M * K + N * K + M * N),
                 "dx": 2.0 * ((k if args.split == "red" else 1) * M * N + N * K + M * K),
                 "dw": 2.0 * (M * N + N * K + M * K + (k - 1) * (M * K if args.split == "out" else M * N))}[dom]
    roofline["algorithmic_bytes"] = alg_bytes
    roofline["tensor_floor_ms"] = gemm_flops / (pk["bf16_tflops_sustained"] * 1e12) * 1e3
    roofline["hbm_floor_ms"] = alg_bytes / (pk["hbm_gbs"] * 1e9) * 1e3

    # ---- CPU baseline: the oracle, as it stands, on a bounded sample of the same workload
    cpu = None
    if not args.no_cpu_baseline:
        dt, f, cores = oracle_sample_run(k, args.split, args.ref_rows)
        cpu = {"value": f / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dt,
               "sample": "%d of %d token rows, full N and K, k=%d %s, one fwd+bwd" % (args.ref_rows, M, k, args.split)}

    burst_value = aggregate_value(fl, args.steps, 1, burst_ms)
    clocks = sampler.summary() if sampler else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": config_dict(args),
        "value_kind": "sustained state: the K timed steps follow %.1f s of untimed load (%d steps); divide by the "
                      "sustained peak" % (args.preheat, n_pre),
        "frac_of_bf16_peak": {"of_measured_sustained_%d" % round(pk["bf16_tflops_sustained"]): value / world / pk["bf16_tflops_sustained"],
                              "of_measured_burst_%d" % round(pk["bf16_tflops"]): value / world / pk["bf16_tflops"],
                              "of_datasheet_2250": value / world / 2250.0},
        "cold_start": {"what": "the first K steps after the warm-up, before the pre-heat (rank 0; burst clocks)",
                       "ms_per_step": burst_ms / args.steps, "tflops": burst_value,
                       "frac_of_measured_burst_peak": burst_value / pk["bf16_tflops"]},
        "sustained": sustained, "sweep": sweep, "torch_matmul_same_shape": like_for_like,
        "decoder_layer_hidden2048_tokens8192": decoder_layer,
        "mlp_block_hidden8192_ffn32768_tokens8192": mlp_wide,
        "mlp_block_hidden1024_ffn4096_tokens4096": mlp_small,
        "skinny_layer_latency": skinny,
        "fp8_e4m3_operands": fp8, "staging_bytes": ws_bytes,
        "roofline": roofline, "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / e2e_steps,
                "how": "every step: X and dY copied pinned host -> device, C-ABI fwd+bwd, Y, dX, dW, db copied device -> "
                       "pinned host; copy-in / compute / copy-out on three streams over two buffer sets; the flat "
                       "weight buffer stays resident on the device (parameters are not an input of a step)"},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
        # time x clock: what is left of a comparison between runs once the power cap's clock is divided out
        "clock_normalised": ({"ms_per_step_x_sm_ghz": ms_total / args.steps * clocks["sm_mhz"] / 1e3,
                              "tflops_per_sm_ghz": value / world / (clocks["sm_mhz"] / 1e3)}
                             if clocks and clocks.get("sm_mhz") else None),
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
    ap.add_argument("--preheat", type=float, default=1.5,
                    help="seconds of untimed back-to-back steps before the warm-up (sustained clocks)")
    ap.add_argument("--ref-rows", type=int, default=1024,
                    help="token rows in the oracle's bounded sample (1024 rows = 4.1e11 flop, about 8 s on 16 cores)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--case", default=None, help="run one small case twice and exit (for profilers)")
    args = ap.parse_args()
    if args.case:
        return run_case(args.case)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
