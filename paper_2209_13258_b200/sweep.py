"""Command-line runs of the split-linear path on synthetic tensors (device-side random data).

    python -m paper_2209_13258_b200.sweep case M N K k split        one fwd+bwd (twice), for profilers
    python -m paper_2209_13258_b200.sweep case-mlp M hidden ffn k   one MLP-block fwd+bwd (twice), for profilers
    python -m paper_2209_13258_b200.sweep case-f8 M N K k split     one fwd+bwd with fp8 operands (twice), for profilers
    python -m paper_2209_13258_b200.sweep latency M N K k split     small operators: one fwd+bwd with a warm and with
                                                                    a flushed L2 (median and best of 50 after 10 warm-ups)
    python -m paper_2209_13258_b200.sweep sustained M N K k split [seconds]   fwd+bwd back to back for >= `seconds`
                                                                    (default 2): the power-limited figure
    python -m paper_2209_13258_b200.sweep linear M N K [ks]         time vs slice granularity, both split dims
    python -m paper_2209_13258_b200.sweep linear-f8 M N K [ks]      the same with fp8 (e4m3) operands
    python -m paper_2209_13258_b200.sweep mlp M hidden ffn [ks]     MLP block split along ffn: time and staging
    python -m paper_2209_13258_b200.sweep zdp M N K [ks]            sharded slice loop (gather / compute /
                                                                    reduce-scatter per slice) against the resident-
                                                                    weight path; also under torchrun, M tokens per rank

    python -m paper_2209_13258_b200.sweep plan hidden layers tokens world mem_GB [ks]
                                                                    execution plan (DP / ZDP per operator or per
                                                                    slice, batch size) for a GPT-like stack of
                                                                    linears, from compute times measured here

The `linear` and `mlp` modes reproduce in kind the paper's Figure 7 (time and memory of an operator
against slice granularity) for this single-GPU path: TFLOP/s, overhead versus k = 1, staging bytes.
Timing: CUDA events on the current stream, median of `iters` runs after warm-up.
"""
from __future__ import annotations

import json
import sys

import torch

from . import binding as P


def _time_interleaved(fns, rounds=12, warm=2):
    """Median time (ms) of each callable.  The callables are run round-robin, one timed run each
    per round, so that clock / power drift over the measurement hits every configuration alike."""
    for _ in range(warm):
        for fn in fns:
            fn()
    torch.cuda.synchronize()
    ts = [[] for _ in fns]
    for _ in range(rounds):
        for i, fn in enumerate(fns):
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts[i].append(a.elapsed_time(b))
    return [sorted(t)[len(t) // 2] for t in ts]


def _linear_tensors(M, N, K):
    dev = "cuda"
    x = torch.randn(M, K, device=dev).bfloat16()
    w = (torch.randn(N, K, device=dev) * 0.02).bfloat16()
    dy = torch.randn(M, N, device=dev).bfloat16()
    out = torch.empty(M, N, device=dev, dtype=torch.bfloat16)
    dx = torch.empty(M, K, device=dev, dtype=torch.bfloat16)
    dw = torch.empty(N, K, device=dev, dtype=torch.bfloat16)
    db = torch.empty(N, device=dev, dtype=torch.float32)
    return x, w, dy, out, dx, dw, db


def _ws_linear(M, N, K, k, split, flags=0):
    _, a = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, 0, P.OP_LINEAR_FWD, flags)
    _, b = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, 0, P.OP_LINEAR_BWD, flags)
    return max(a, b)


def run_case(M, N, K, k, split):
    x, w, dy, out, dx, dw, db = _linear_tensors(M, N, K)
    ws = P.new_workspace(_ws_linear(M, N, K, k, split))
    for _ in range(2):
        P.osdp_split_linear_fwd(x, w, 0, None, M, N, K, k, split, 0, out, None, ws, check=True)
        P.osdp_split_linear_bwd(dy, x, w, 0, None, M, N, K, k, split, 0, dx, dw, 0, 0, 0, None, ws, check=True)
        torch.cuda.synchronize()
    print("device status", P.osdp_read_device_status(ws))


def run_case_f8(M, N, K, k, split):
    dev = "cuda"
    x8 = torch.randn(M, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
    w8 = torch.randn(N, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
    dy8 = torch.randn(M, N, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
    out = torch.empty(M, N, device=dev, dtype=torch.bfloat16)
    dx = torch.empty(M, K, device=dev, dtype=torch.bfloat16)
    dw = torch.empty(N, K, device=dev, dtype=torch.bfloat16)
    ws = P.new_workspace(_ws_linear(M, N, K, k, split))
    for _ in range(2):
        P.osdp_split_linear_fwd_f8(x8, w8, 0, 1.0, None, M, N, K, k, split, 0, out, None, ws, check=True)
        P.osdp_split_linear_bwd_f8(dy8, x8, w8, 0, 1.0, 1.0, M, N, K, k, split, dx, dw, 0, P.DTYPE_BF16, 0, ws,
                                   check=True)
        torch.cuda.synchronize()
    print("device status", P.osdp_read_device_status(ws))


def run_case_mlp(M, H, F, k, flags=0):
    dev = "cuda"
    x = torch.randn(M, H, device=dev).bfloat16()
    dy = torch.randn(M, H, device=dev).bfloat16()
    wf = (torch.randn(2 * F * H, device=dev) * 0.02).bfloat16()
    b1 = torch.zeros(F, device=dev)
    b2 = torch.zeros(H, device=dev)
    out = torch.empty(M, H, device=dev, dtype=torch.bfloat16)
    z1 = torch.empty(M, F, device=dev, dtype=torch.bfloat16)
    dx = torch.empty(M, H, device=dev, dtype=torch.bfloat16)
    dwf = torch.empty(2 * F * H, device=dev, dtype=torch.bfloat16)
    db1 = torch.empty(F, device=dev)
    db2 = torch.empty(H, device=dev)
    _, n1 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_FWD, flags)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_BWD, flags)
    ws = P.new_workspace(max(n1, n2))
    for _ in range(2):
        P.osdp_split_mlp_fwd(x, wf, 0, b1, F * H, b2, M, H, F, k, 1, out, z1, ws, check=True, flags=flags)
        P.osdp_split_mlp_bwd(dy, x, wf, 0, F * H, z1, M, H, F, k, 1, dx, dwf, 0, F * H, 0, flags, db1, db2, ws,
                             check=True)
        torch.cuda.synchronize()
    print("device status", P.osdp_read_device_status(ws))


def run_latency(M, N, K, k, split, iters=50, warm=10):
    """Forward + backward of a small operator, timed one step at a time: with the operands left in L2 by the
    previous step, and after the L2 has been flushed (a 256 MB buffer is overwritten between steps)."""
    x, w, dy, out, dx, dw, db = _linear_tensors(M, N, K)
    ws = P.new_workspace(_ws_linear(M, N, K, k, split))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def step():
        P.osdp_split_linear_fwd(x, w, 0, None, M, N, K, k, split, 0, out, None, ws, check=True)
        P.osdp_split_linear_bwd(dy, x, w, 0, None, M, N, K, k, split, 0, dx, dw, 0, 0, 0, db, ws, check=True)
    res = {}
    for name, cold in (("warm_l2", False), ("cold_l2", True)):
        ts = []
        for i in range(warm + iters):
            if cold:
                flush.fill_(i & 255)
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            step()
            b.record()
            torch.cuda.synchronize()
            if i >= warm:
                ts.append(a.elapsed_time(b) * 1e3)
        ts.sort()
        res[name] = {"median_us": ts[len(ts) // 2], "best_us": ts[0]}
    # several steps issued back to back (the host runs ahead): the device-side time of a step
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True)
    b = torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(200):
        step()
    b.record()
    torch.cuda.synchronize()
    res["back_to_back_us"] = a.elapsed_time(b) * 1e3 / 200
    res.update({"M": M, "N": N, "K": K, "k": k, "split": "out" if split == P.SPLIT_OUT else "red",
                "flops": 3 * 2.0 * M * N * K, "bytes_min": 2 * 3 * (M * K + N * K + M * N)})
    print(json.dumps(res), flush=True)
    return res


def run_sustained(M, N, K, k, split, seconds=2.0):
    """Forward + backward issued back to back for at least `seconds`: the figure a long training loop sees
    under the power cap, next to the median and best of 50 single steps."""
    x, w, dy, out, dx, dw, db = _linear_tensors(M, N, K)
    ws = P.new_workspace(_ws_linear(M, N, K, k, split))
    flops = 3 * 2.0 * M * N * K

    def step():
        P.osdp_split_linear_fwd(x, w, 0, None, M, N, K, k, split, 0, out, None, ws, check=True)
        P.osdp_split_linear_bwd(dy, x, w, 0, None, M, N, K, k, split, 0, dx, dw, 0, 0, 0, db, ws, check=True)
    for _ in range(10):
        step()
    torch.cuda.synchronize()
    ts = []
    for _ in range(50):
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record()
        step()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ts.sort()
    n = max(50, int(seconds * 1e3 / ts[len(ts) // 2]) + 1)
    a = torch.cuda.Event(enable_timing=True)
    b = torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(n):
        step()
    b.record()
    torch.cuda.synchronize()
    total = a.elapsed_time(b)
    row = {"M": M, "N": N, "K": K, "k": k, "split": "out" if split == P.SPLIT_OUT else "red",
           "median_ms": ts[len(ts) // 2], "best_ms": ts[0], "median_tflops": flops / ts[len(ts) // 2] / 1e9,
           "best_tflops": flops / ts[0] / 1e9, "sustained_steps": n, "sustained_seconds": total / 1e3,
           "sustained_ms": total / n, "sustained_tflops": flops * n / total / 1e9}
    print(json.dumps(row), flush=True)
    return row


def sweep_linear(M, N, K, ks):
    x, w, dy, out, dx, dw, db = _linear_tensors(M, N, K)
    flops = 3 * 2.0 * M * N * K
    cfgs = []
    for k in ks:
        for split, name in ((P.SPLIT_OUT, "out"), (P.SPLIT_RED, "red")):
            if k == 1 and split == P.SPLIT_RED:
                continue
            if P.osdp_slice_range(N if split == P.SPLIT_OUT else K, k, 0)[0] != 0:
                continue
            cfgs.append((k, split, name, 0, _ws_linear(M, N, K, k, split)))
            if k > 1:   # the summed output carried in bf16 in the output buffer instead of fp32 in the workspace
                cfgs.append((k, split, name, P.FLAG_CARRY_BF16, _ws_linear(M, N, K, k, split, P.FLAG_CARRY_BF16)))
            if k > 2:   # exact fp32 carry, adjacent slices accumulated in pairs (two slices live)
                cfgs.append((k, split, name, P.FLAG_PAIR_SLICES, _ws_linear(M, N, K, k, split, P.FLAG_PAIR_SLICES)))
    ws = P.new_workspace(max(c[4] for c in cfgs))     # one workspace, large enough for every configuration
    fns = []
    for k, split, name, fl, _ in cfgs:
        fns.append(lambda k=k, split=split, fl=fl: P.osdp_split_linear_fwd(
            x, w, 0, None, M, N, K, k, split, 0, out, None, ws, check=True, flags=fl))
        fns.append(lambda k=k, split=split, fl=fl: P.osdp_split_linear_bwd(
            dy, x, w, 0, None, M, N, K, k, split, 0, dx, dw, 0, 0, fl, db, ws, check=True))
    ts = _time_interleaved(fns)
    rows = []
    base = ts[0] + ts[1]
    for i, (k, split, name, fl, nbytes) in enumerate(cfgs):
        tf, tb = ts[2 * i], ts[2 * i + 1]
        t = tf + tb
        rows.append({"k": k, "split": name,
                     "carry": {0: "fp32", P.FLAG_CARRY_BF16: "bf16", P.FLAG_PAIR_SLICES: "fp32-paired"}[fl],
                     "fwd_ms": tf, "bwd_ms": tb, "ms": t,
                     "tflops": flops / t / 1e9, "overhead_vs_k1": t / base - 1.0, "staging_bytes": nbytes})
        print(json.dumps(rows[-1]), flush=True)
    return rows


def sweep_linear_f8(M, N, K, ks):
    """fp8 (e4m3) operands: forward + backward (dX, dW) per granularity and split dimension."""
    dev = "cuda"
    x8 = torch.randn(M, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
    w8 = torch.randn(N, K, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
    dy8 = torch.randn(M, N, device=dev).to(torch.float8_e4m3fn).view(torch.uint8)
    out = torch.empty(M, N, device=dev, dtype=torch.bfloat16)
    dx = torch.empty(M, K, device=dev, dtype=torch.bfloat16)
    dw = torch.empty(N, K, device=dev, dtype=torch.bfloat16)
    flops = 3 * 2.0 * M * N * K
    cfgs = []
    for k in ks:
        for split, name in ((P.SPLIT_OUT, "out"), (P.SPLIT_RED, "red")):
            if k == 1 and split == P.SPLIT_RED:
                continue
            rc, b, e = P.osdp_slice_range(N if split == P.SPLIT_OUT else K, k, 0)
            if rc != 0 or (k > 1 and (e - b) % 16):
                continue
            cfgs.append((k, split, name, _ws_linear(M, N, K, k, split)))
    ws = P.new_workspace(max(c[3] for c in cfgs))
    fns = []
    for k, split, name, _ in cfgs:
        fns.append(lambda k=k, split=split: P.osdp_split_linear_fwd_f8(
            x8, w8, 0, 1.0, None, M, N, K, k, split, 0, out, None, ws, check=True))
        fns.append(lambda k=k, split=split: P.osdp_split_linear_bwd_f8(
            dy8, x8, w8, 0, 1.0, 1.0, M, N, K, k, split, dx, dw, 0, P.DTYPE_BF16, 0, ws, check=True))
    ts = _time_interleaved(fns)
    rows = []
    base = ts[0] + ts[1]
    for i, (k, split, name, nbytes) in enumerate(cfgs):
        t = ts[2 * i] + ts[2 * i + 1]
        rows.append({"operands": "fp8 e4m3", "k": k, "split": name, "fwd_ms": ts[2 * i], "bwd_ms": ts[2 * i + 1], "ms": t,
                     "tflops": flops / t / 1e9, "overhead_vs_k1": t / base - 1.0, "staging_bytes": nbytes})
        print(json.dumps(rows[-1]), flush=True)
    return rows


def sweep_mlp(M, H, F, ks):
    dev = "cuda"
    x = torch.randn(M, H, device=dev).bfloat16()
    dy = torch.randn(M, H, device=dev).bfloat16()
    wf = (torch.randn(2 * F * H, device=dev) * 0.02).bfloat16()
    b1 = torch.zeros(F, device=dev)
    b2 = torch.zeros(H, device=dev)
    out = torch.empty(M, H, device=dev, dtype=torch.bfloat16)
    z1 = torch.empty(M, F, device=dev, dtype=torch.bfloat16)
    dx = torch.empty(M, H, device=dev, dtype=torch.bfloat16)
    dwf = torch.empty(2 * F * H, device=dev, dtype=torch.bfloat16)
    db1 = torch.empty(F, device=dev)
    db2 = torch.empty(H, device=dev)
    flops = 2 * 3 * 2.0 * M * H * F
    cfgs = []
    for k in ks:
        if P.osdp_slice_range(F, k, 0)[0] != 0:
            continue
        for fl in ((0, P.FLAG_RECOMPUTE) if k == 1 else (0, P.FLAG_CARRY_BF16, P.FLAG_RECOMPUTE)):
            _, n1 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_FWD, fl & P.FLAG_CARRY_BF16)
            _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_BWD, fl)
            cfgs.append((k, n1, n2, fl))
    ws = P.new_workspace(max(max(c[1], c[2]) for c in cfgs))
    fns = []
    for k, _, _, fl in cfgs:
        fns.append(lambda k=k, fl=fl: P.osdp_split_mlp_fwd(x, wf, 0, b1, F * H, b2, M, H, F, k, 1, out, z1, ws,
                                                           check=True, flags=fl & P.FLAG_CARRY_BF16))
        fns.append(lambda k=k, fl=fl: P.osdp_split_mlp_bwd(dy, x, wf, 0, F * H, z1, M, H, F, k, 1, dx, dwf, 0, F * H,
                                                           0, fl, db1, db2, ws, check=True, b1=b1))
    ts = _time_interleaved(fns)
    rows = []
    base = ts[0] + ts[1]
    for i, (k, n1, n2, fl) in enumerate(cfgs):
        tf, tb = ts[2 * i], ts[2 * i + 1]
        t = tf + tb
        rows.append({"k": k, "carry": "bf16" if fl & P.FLAG_CARRY_BF16 else "fp32",
                     "recompute": bool(fl & P.FLAG_RECOMPUTE), "fwd_ms": tf, "bwd_ms": tb, "ms": t,
                     "tflops": flops / t / 1e9,
                     "overhead_vs_k1": t / base - 1.0, "staging_fwd_bytes": n1, "staging_bwd_bytes": n2})
        print(json.dumps(rows[-1]), flush=True)
    return rows


def sweep_zdp(M, N, K, ks):
    """Time and staging of the sharded slice loop per granularity.  Stand-alone it forms a one-rank NCCL
    group (every collective still runs, as a device copy); under torchrun every rank works on M tokens."""
    import os
    import torch.distributed as dist
    from .zdp import ZdpSplitLinear
    own_group = not dist.is_initialized()
    if own_group:
        if "RANK" in os.environ:
            torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
            dist.init_process_group("nccl")
        else:
            dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29755", rank=0, world_size=1)
    rank, world = dist.get_rank(), dist.get_world_size()
    x, w, dy, out, dx, _, db = _linear_tensors(M, N, K)
    dw = torch.empty(N, K, device="cuda", dtype=torch.float32)
    flops = 3 * 2.0 * M * N * K
    cfgs, fns, layers, fused_ok = [], [], [], True
    for k in ks:
        for split, name in ((P.SPLIT_OUT, "out"), (P.SPLIT_RED, "red")):
            if k == 1 and split == P.SPLIT_RED:
                continue
            if P.osdp_slice_range(N if split == P.SPLIT_OUT else K, k, 0)[0] != 0:
                continue
            cfgs.append((k, split, name))
    ws = P.new_workspace(max(_ws_linear(M, N, K, k, split) for k, split, _ in cfgs))
    for k, split, name in cfgs:
        layer = ZdpSplitLinear(N, K, k, split, dw_dtype=P.DTYPE_FP32)
        layer.load_full_weight(w)
        layers.append(layer)

        def resident(k=k, split=split):
            P.osdp_split_linear_fwd(x, w, 0, None, M, N, K, k, split, 0, out, None, ws, check=True)
            P.osdp_split_linear_bwd(dy, x, w, 0, None, M, N, K, k, split, 0, dx, dw, 0, P.DTYPE_FP32, 0, db, ws,
                                    check=True)

        def sharded(layer=layer):
            layer.forward(x, out=out)
            layer.backward(dy, x, dx=dx, dbias=db)
        fns += [resident, sharded]
        # the same loop with the reduce-scatter done by the backward GEMM's epilogue (peer-mapped gradient shards)
        try:
            fl = ZdpSplitLinear(N, K, k, split, dw_dtype=P.DTYPE_FP32, fused_scatter=True) if fused_ok else None
        except Exception:
            fused_ok, fl = False, None
        if fl is not None:
            fl.load_full_weight(w)

            def fused(fl=fl):
                fl.forward(x, out=out)
                fl.backward(dy, x, dx=dx, dbias=db)
            fns.append(fused)
        else:
            fns.append(sharded)
        layers[-1] = (layer, fl)
    ts = _time_interleaved(fns, rounds=8)
    tt = torch.tensor(ts, device="cuda", dtype=torch.float64)
    if world > 1:
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)     # a step is as slow as its slowest rank
    ts = tt.tolist()
    rows = []
    for i, (k, split, name) in enumerate(cfgs):
        st = layers[i][0].staging_bytes(M)
        rows.append({"k": k, "split": name, "world": world, "resident_ms": ts[3 * i], "sharded_ms": ts[3 * i + 1],
                     "sharded_fused_scatter_ms": ts[3 * i + 2] if layers[i][1] is not None else None,
                     "sharded_tflops_all_ranks": world * flops / ts[3 * i + 1] / 1e9,
                     "loop_overhead": ts[3 * i + 1] / ts[3 * i] - 1.0,
                     "weight_staging_bytes": st["weight_staging"], "grad_staging_bytes": st["grad_staging"],
                     "workspace_bytes": st["workspace"], "full_gather_bytes": N * K * 2, "full_grad_bytes": N * K * 4})
        if rank == 0:
            print(json.dumps(rows[-1]), flush=True)
    if own_group:
        dist.destroy_process_group()
    return rows


def plan_from_measurements(hidden, layers, tokens, world, mem_gb, ks, alpha=10e-6, beta=1.0 / 770e9):
    """Section 3.1 / Algorithm 1 fed with this GPU's kernel times: gamma_i of each linear of a GPT-like layer
    (QKV, out-projection, the two MLP layers; `tokens` tokens per sample) is measured per slice granularity,
    then the plan search runs on whole operators and on operators cut into k slices (Section 3.3, last
    paragraph).  States: 16 bytes per parameter; wire: bf16 parameters; activations: the bf16 input and
    output of each linear; alpha / beta default to 10 us per step and the 770 GB/s peer-copy figure."""
    shapes = [("qkv", 3 * hidden, hidden), ("proj", hidden, hidden), ("fc1", 4 * hidden, hidden),
              ("fc2", hidden, 4 * hidden)]
    split_of = {"qkv": P.SPLIT_OUT, "proj": P.SPLIT_RED, "fc1": P.SPLIT_OUT, "fc2": P.SPLIT_RED}
    gamma = {}
    for name, N, K in shapes:
        x, w, dy, out, dx, dw, db = _linear_tensors(tokens, N, K)
        split = split_of[name]
        valid = [k for k in ks if P.osdp_slice_range(N if split == P.SPLIT_OUT else K, k, 0)[0] == 0]
        ws = P.new_workspace(max(_ws_linear(tokens, N, K, k, split) for k in valid))
        fns = []
        for k in valid:
            def step(k=k):
                P.osdp_split_linear_fwd(x, w, 0, None, tokens, N, K, k, split, 0, out, None, ws, check=True)
                P.osdp_split_linear_bwd(dy, x, w, 0, None, tokens, N, K, k, split, 0, dx, dw, 0, 0, 0, db, ws,
                                        check=True)
            fns.append(step)
        for k, t in zip(valid, _time_interleaved(fns)):
            gamma[(name, k)] = t * 1e-3
    limit = mem_gb * 1e9
    rows = []
    for k in ks:
        if any((name, k) not in gamma for name, _, _ in shapes):
            continue
        ops = []
        for _ in range(layers):
            for name, N, K in shapes:
                params = float(N * K)
                op = (16.0 * params, 2.0 * tokens * (N + K), 0.0, 2.0 * params, gamma[(name, 1)])
                rc, sl = P.osdp_plan_expand_slices(op, k, gamma[(name, k)] / gamma[(name, 1)] - 1.0)
                ops += sl
        rc, modes, b, t, nodes = P.osdp_plan_search(ops, world, alpha, beta, limit, 4096)
        row = {"k": k, "status": rc, "operators": len(ops), "batch": b, "dp": modes.count(0) if b else 0,
               "zdp": modes.count(1) if b else 0, "time_per_sample_ms": t * 1e3 if b else None,
               "samples_per_s_per_gpu": 1.0 / t if b else 0.0, "nodes": nodes,
               "gamma_ms": {name: gamma[(name, k)] * 1e3 for name, _, _ in shapes}}
        rows.append(row)
        print(json.dumps(row), flush=True)
    # every operator free to take any of the measured granularities, its slices planned one by one
    ops, cands, names = [], [], []
    for _ in range(layers):
        for name, N, K in shapes:
            params = float(N * K)
            ops.append((16.0 * params, 2.0 * tokens * (N + K), 0.0, 2.0 * params, gamma[(name, 1)]))
            cands.append([(k, gamma[(name, k)] / gamma[(name, 1)] - 1.0) for k in ks if (name, k) in gamma])
            names.append(name)
    # surge 0: the memory model of Section 3.1 as it stands; surge 2: the double-buffered gathered slice of the
    # sharded slice loop counted as well (what Section 3.3 says splitting divides by the granularity)
    for surge in ((0.0, 2.0) if all(cands) else ()):
        rc, kk, dps, b, t, nodes = P.osdp_plan_search_granularity(ops, cands, world, alpha, beta, limit, 4096,
                                                                  surge_factor=surge)
        chosen = {}
        for name, k, d in zip(names, kk, dps):
            if b:
                key = "k=%d dp=%d" % (k, d)
                chosen.setdefault(name, {})[key] = chosen.setdefault(name, {}).get(key, 0) + 1
        row = {"k": "free", "surge_factor": surge, "status": rc, "operators": len(ops), "batch": b, "chosen": chosen,
               "time_per_sample_ms": t * 1e3 if b else None, "samples_per_s_per_gpu": 1.0 / t if b else 0.0,
               "nodes": nodes}
        rows.append(row)
        print(json.dumps(row), flush=True)
    return rows


def main(argv):
    if len(argv) < 2:
        print(__doc__)
        return 2
    mode = argv[1]
    ks = [int(v) for v in argv[5].split(",")] if len(argv) > 5 and not mode.startswith("case") else [1, 2, 4, 8, 16, 32]
    if mode == "case":
        run_case(*[int(v) for v in argv[2:7]])
    elif mode == "case-f8":
        run_case_f8(*[int(v) for v in argv[2:7]])
    elif mode == "case-mlp":
        run_case_mlp(*[int(v) for v in argv[2:6]])
    elif mode == "sustained":
        run_sustained(*[int(v) for v in argv[2:7]], seconds=float(argv[7]) if len(argv) > 7 else 2.0)
    elif mode == "latency":
        run_latency(*[int(v) for v in argv[2:7]])
    elif mode == "linear":
        sweep_linear(int(argv[2]), int(argv[3]), int(argv[4]), ks)
    elif mode == "linear-f8":
        sweep_linear_f8(int(argv[2]), int(argv[3]), int(argv[4]), ks)
    elif mode == "mlp":
        sweep_mlp(int(argv[2]), int(argv[3]), int(argv[4]), ks)
    elif mode == "zdp":
        sweep_zdp(int(argv[2]), int(argv[3]), int(argv[4]), ks)
    elif mode == "plan":
        ks = [int(v) for v in argv[7].split(",")] if len(argv) > 7 else [1, 2, 4, 8]
        plan_from_measurements(int(argv[2]), int(argv[3]), int(argv[4]), int(argv[5]), float(argv[6]), ks)
    else:
        print(__doc__)
        return 2
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
