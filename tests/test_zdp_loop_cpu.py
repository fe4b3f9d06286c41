"""The sharded slice loops themselves (paper_2209_13258_b200/zdp.py: ZdpSplitLinear, ZdpSplitMLP) run on CPU
by two gloo ranks: which slice is gathered when, which gradient goes through a reduce-scatter (ZDP
slice) and which through an all-reduce (DP slice), where each lands in the rank's shard buffers.

The loop code is the product's; what this test replaces is (a) the CUDA streams and events it orders its
work with (no-op stand-ins: a CPU run is sequential) and (b) the per-slice CUDA entry points it calls,
which are stood in for by the fp64 oracle on the slice's compact matrices (this is a test; the product's
arithmetic runs only in the CUDA kernels).  Plus, host only: the order of the steps of a gradient step with
the epilogue-fused scatter (zero, barrier, backward, barrier) as seen by a communicator that records calls.
"""
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

torch = pytest.importorskip("torch")

# Shared by the gloo workers and by the in-process protocol test: stand-ins for torch.cuda and for the
# per-slice entry points.
SHIM = textwrap.dedent('''
    import contextlib
    import numpy as np, torch
    import oracle
    from paper_2209_13258_b200 import binding as B

    class FakeStream:
        def __init__(self, log=None): self.log = log
        def wait_stream(self, s): pass
        def wait_event(self, e): pass
        def synchronize(self):
            if self.log is not None: self.log.append("stream.synchronize")

    class FakeEvent:
        def __init__(self, *a, **k): pass
        def record(self, s=None): pass

    def install_fake_cuda(log=None):
        cur = FakeStream(log)
        torch.cuda.is_available = lambda: True
        torch.cuda.Stream = lambda device=None: FakeStream()
        torch.cuda.Event = FakeEvent
        torch.cuda.current_stream = lambda device=None: cur
        torch.cuda.stream = lambda s: contextlib.nullcontext()

    def bits(t):                         # bf16 torch tensor -> the oracle's input (bf16 bit patterns)
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)

    def put(dst, a):                     # fp64 result -> the caller's tensor (rounded to its dtype by torch)
        dst.copy_(torch.from_numpy(np.ascontiguousarray(a)).to(dst.dtype))

    CARRY = {}                           # running sums of summed outputs, per workspace (the kernels keep them there)

    def lin_fwd_slice(x, w, ld, bias, M, N, K, k, split, act, s, out, z_save, ws, stream=None, check=False, flags=0):
        LOG.append(("fwd_slice", s))
        b, e = oracle.slice_range(N if split == 0 else K, k, s)
        wb = bits(w)[:(e - b) * K if split == 0 else N * (e - b)]
        bb = None if bias is None else bias.numpy()
        if split == 0:
            z, y = oracle.linear_fwd(bits(x), wb.reshape(e - b, K), None if bb is None else bb[b:e], act, 1)
            put(out[:, b:e], y)
            if z_save is not None: put(z_save[:, b:e], z)
        else:
            z, _ = oracle.linear_fwd(bits(x)[:, b:e], wb.reshape(N, e - b), None, 0, 1)
            acc = z if s == 0 else CARRY[("y", ws.data_ptr())] + z
            CARRY[("y", ws.data_ptr())] = acc
            if s == k - 1:
                if bb is not None: acc = acc + bb[None, :]
                if z_save is not None: put(z_save, acc)
                put(out, acc if act == 0 else np.vectorize(lambda v: oracle.gelu(v, act))(acc))
        return 0

    def lin_bwd_slice(dy, x, w, ld, z, M, N, K, k, split, act, s, dx, dw, ld_dw, dw_dtype, flags, dbias, ws,
                      stream=None, check=False):
        LOG.append(("bwd_slice", s, dx is not None, dw is not None))
        b, e = oracle.slice_range(N if split == 0 else K, k, s)
        wb = bits(w)[:(e - b) * K if split == 0 else N * (e - b)]
        zz = None if z is None else oracle.as_f64(bits(z))
        if split == 0:
            dX, dW, db = oracle.linear_bwd(bits(dy)[:, b:e], bits(x), wb.reshape(e - b, K),
                                           None if zz is None else np.ascontiguousarray(zz[:, b:e]), act, 1)
            if dx is not None:
                acc = dX if s == 0 else CARRY[("dx", ws.data_ptr())] + dX
                CARRY[("dx", ws.data_ptr())] = acc
                if s == k - 1: put(dx, acc)
            if dbias is not None: put(dbias[b:e], db)
        else:
            dX, dW, db = oracle.linear_bwd(bits(dy), np.ascontiguousarray(bits(x)[:, b:e]), wb.reshape(N, e - b), zz, act, 1)
            if dx is not None: put(dx[:, b:e], dX)
            if dbias is not None and s == 0: put(dbias, db)
        if dw is not None: put(dw[:dW.size], dW.reshape(-1))
        return 0

    def mlp_fwd_slice(x, w1, w2, ld2, b1, b2, M, H, F, k, act, s, out, z1_save, ws, stream=None, check=False, flags=0):
        LOG.append(("mlp_fwd_slice", s))
        b, e = oracle.slice_range(F, k, s)
        w1b, w2b = bits(w1)[:(e - b) * H].reshape(e - b, H), bits(w2)[:H * (e - b)].reshape(H, e - b)
        z1, y = oracle.mlp_fwd(bits(x), w1b, None if b1 is None else b1.numpy()[b:e], w2b, None, act, None)
        acc = y if s == 0 else CARRY[("y", ws.data_ptr())] + y
        CARRY[("y", ws.data_ptr())] = acc
        if z1_save is not None: put(z1_save[:, b:e], z1)
        if s == k - 1:
            put(out, acc if b2 is None else acc + b2.numpy()[None, :])
        return 0

    def mlp_bwd_slice(dy, x, w1, w2, ld2, b1, z1, M, H, F, k, act, s, dx, dw1, dw2, ld_dw2, p1, p2, dw_dtype, flags,
                      db1, db2, ws, stream=None, check=False):
        LOG.append(("mlp_bwd_slice", s, p1 is not None))
        b, e = oracle.slice_range(F, k, s)
        w1b, w2b = bits(w1)[:(e - b) * H].reshape(e - b, H), bits(w2)[:H * (e - b)].reshape(H, e - b)
        dX, dW1, d1, dW2, d2 = oracle.mlp_bwd(bits(dy), bits(x), w1b, None if b1 is None else b1.numpy()[b:e], w2b, act, None)
        acc = dX if s == 0 else CARRY[("dx", ws.data_ptr())] + dX
        CARRY[("dx", ws.data_ptr())] = acc
        if s == k - 1: put(dx, acc)
        if db1 is not None: put(db1[b:e], d1)
        if db2 is not None and s == 0: put(db2, d2)
        if p1 is not None:               # the epilogue's scatter: every rank's part is added where its owner keeps it
            for peers, g in ((p1, dW1), (p2, dW2)):
                flat = torch.from_numpy(np.ascontiguousarray(g).reshape(-1))
                n = -(-flat.numel() // (8 * len(peers))) * 8
                for q, addr in enumerate(peers):     # the loop passes addresses: rank q's shard + the slice's offset
                    t, off = PEER_TENSORS[addr]
                    part = flat[q * n:(q + 1) * n]
                    t[off:off + part.numel()] += part.to(t.dtype)
        else:
            put(dw1[:dW1.size], dW1.reshape(-1)); put(dw2[:dW2.size], dW2.reshape(-1))
        return 0

    LOG = []
    PEER_TENSORS = {}                    # address -> (tensor, element offset): what the fake scatter writes to

    def register_peers(layer):
        for m, peers in enumerate(layer.peer_grad_shards):
            for t in peers:
                for s in layer.zdp_slices:
                    PEER_TENSORS[int(t.data_ptr()) + layer._zoff[m][s] * t.element_size()] = (t, layer._zoff[m][s])

    def install_fake_kernels():
        B.osdp_zdp_linear_fwd_slice = lin_fwd_slice
        B.osdp_zdp_linear_bwd_slice = lin_bwd_slice
        B.osdp_zdp_mlp_fwd_slice = mlp_fwd_slice
        B.osdp_zdp_mlp_bwd_slice = mlp_bwd_slice
''')

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    exec(%r)
    import torch.distributed as dist
    from paper_2209_13258_b200 import inputs
    from paper_2209_13258_b200.zdp import ZdpSplitLinear, ZdpSplitMLP, DistComm, DP, ZDP
    install_fake_cuda(); install_fake_kernels()
    dist.init_process_group("gloo")
    comm = DistComm()
    rank, world = comm.rank, comm.world

    def t16(a): return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    def rel(a, b): return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))
    def gather_full(t):                       # every rank's copy of a 1-D tensor, in rank order
        parts = [torch.empty_like(t) for _ in range(world)]
        dist.all_gather(parts, t.contiguous())
        return parts
    worst = {}

    # ---- the MLP block: all ZDP, and mixed patterns (DP slices all-reduced, ZDP slices reduce-scattered)
    M, H, F = 48, 64, 256
    for k, modes in ((4, None), (4, [DP, ZDP, ZDP, DP]), (3, [ZDP, DP, ZDP]), (2, [DP, DP])):
        c = inputs.mlp_case(M, H, F, w_std=0.1, bias_std=0.1, layer=k)
        layer = ZdpSplitMLP(H, F, k, comm=comm, device="cpu", slice_modes=modes)
        layer.load_full_weights(t16(c["w1"]), t16(c["w2"]))
        # every ZDP slice gathers to exactly the slice of W1 / W2 (checked through the loop's own staging)
        rows = np.arange(rank, M, world)
        x, dy = t16(c["x"][rows]), t16(c["dy"][rows])
        b1, b2 = torch.from_numpy(c["b1"]), torch.from_numpy(c["b2"])
        z1 = torch.empty(len(rows), F, dtype=torch.bfloat16)
        LOG.clear()
        y = layer.forward(x, b1=b1, b2=b2, z1_save=z1)
        assert [e for e in LOG if e[0] == "mlp_fwd_slice"] == [("mlp_fwd_slice", s) for s in range(k)]
        db1, db2 = torch.zeros(F), torch.zeros(H)
        dx = layer.backward(dy, x, z1_saved=z1, b1=b1, db1=db1, db2=db2)
        _, yo = oracle.mlp_fwd(c["x"][rows], c["w1"], c["b1"], c["w2"], c["b2"], 1, k)
        dXo, _, _, _, _ = oracle.mlp_bwd(c["dy"][rows], c["x"][rows], c["w1"], c["b1"], c["w2"], 1, k)
        worst["mlp y k%%d %%s" %% (k, modes)] = rel(y.double().numpy(), yo)
        worst["mlp dx k%%d %%s" %% (k, modes)] = rel(dx.double().numpy(), dXo)
        # weight gradients summed over ranks = the full batch's gradients, laid out as the loop keeps them
        _, dW1o, db1o, dW2o, db2o = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], 1, k)
        for m, want in ((0, dW1o), (1, dW2o)):
            shards = gather_full(layer.grad_shard[m])
            full = layer.full_from_parts(m, shards, layer.dp_grad[m])
            worst["mlp dW%%d k%%d %%s" %% (m + 1, k, modes)] = rel(full.double().numpy(), want)
            for s, t in layer.dp_grad[m].items():       # an all-reduced DP gradient is the same on every rank
                copies = gather_full(t)
                assert all(torch.equal(copies[0], cq) for cq in copies)

    # ---- the linear loop with mixed modes, both split dimensions
    M, N, K = 64, 256, 128
    for split in (0, 1):
        for k, modes in ((4, [ZDP, DP, DP, ZDP]), (4, None)):
            c = inputs.linear_case(M, N, K, w_std=0.1, bias_std=0.1, layer=10 + split)
            layer = ZdpSplitLinear(N, K, k, split, comm=comm, device="cpu", slice_modes=modes)
            layer.load_full_weight(t16(c["w"]))
            rows = np.arange(rank, M, world)
            x, dy = t16(c["x"][rows]), t16(c["dy"][rows])
            y = layer.forward(x, bias=torch.from_numpy(c["bias"]))
            dx = layer.backward(dy, x)
            _, yo = oracle.linear_fwd(c["x"][rows], c["w"], c["bias"], 0, k, split)
            dXo, _, _ = oracle.linear_bwd(c["dy"][rows], c["x"][rows], c["w"], None, 0, k, split)
            _, dWo, _ = oracle.linear_bwd(c["dy"], c["x"], c["w"], None, 0, k, split)
            full = layer.full_from_parts(gather_full(layer.grad_shard), layer.dp_grad)
            tag = "lin split%%d %%s" %% (split, modes)
            worst[tag + " y"] = rel(y.double().numpy(), yo)
            worst[tag + " dx"] = rel(dx.double().numpy(), dXo)
            worst[tag + " dW"] = rel(full.double().numpy(), dWo)
    dist.barrier()
    print(json.dumps({"rank": rank, "world": world, "worst": worst}))
    dist.destroy_process_group()
""") % (ROOT, SHIM)


def test_two_gloo_ranks_run_the_sharded_loops_with_mixed_slice_modes():
    import json
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29751", OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=600) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-4000:]
    for o, _ in outs:
        line = json.loads(o.strip().splitlines()[-1])
        assert line["world"] == 2
        for name, err in line["worst"].items():
            # outputs pass through bf16 tensors (Y, dX: one rounding, 2^-8 relative to the largest element at worst)
            # or fp32 gradient buffers summed by the collectives
            tol = 5e-3 if (" y" in name or " dx" in name) else 1e-5
            assert err < tol, (name, err)


PROTOCOL = textwrap.dedent("""
    import sys, json
    sys.path.insert(0, %r)
    exec(%r)
    from paper_2209_13258_b200 import inputs
    from paper_2209_13258_b200.zdp import ZdpSplitMLP, ZdpSplitLinear

    class RecordingComm:
        rank, world = 0, 1
        def __init__(self, log): self.log = log
        def all_gather_slice(self, dst, shard, off, n): self.log.append("all_gather"); dst[:n].copy_(shard[off:off + n])
        def reduce_scatter_slice(self, shard, off, n, src): self.log.append("reduce_scatter"); shard[off:off + n].copy_(src[:n])
        def all_reduce(self, t, tag=None): self.log.append("all_reduce")
        def barrier(self): self.log.append("barrier")
        def peer_buffers(self, numel, dtype, device): return [torch.zeros(numel, dtype=dtype)]

    install_fake_cuda(LOG); install_fake_kernels()
    def t16(a): return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    M, H, F, k = 32, 64, 256, 4
    c = inputs.mlp_case(M, H, F, w_std=0.1)
    res = {}
    for fused in (True, False):
        layer = ZdpSplitMLP(H, F, k, comm=RecordingComm(LOG), device="cpu", fused_scatter=fused)
        layer.load_full_weights(t16(c["w1"]), t16(c["w2"]))
        if fused:
            register_peers(layer)
        x, dy = t16(c["x"]), t16(c["dy"])
        z1 = torch.empty(M, F, dtype=torch.bfloat16)
        layer.forward(x, z1_save=z1)
        zero = layer.zero_grad
        layer.zero_grad = lambda: (LOG.append("zero_grad"), zero())[1]
        for t in layer.grad_shard: t.fill_(7.0)            # stale contents that the step must not keep
        LOG.clear()
        layer.backward_step(dy, x, z1_saved=z1)
        _, dW1o, _, dW2o, _ = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], None, c["w2"], 1, k)     # the step ran without biases
        got = layer.full_from_parts(0, [layer.grad_shard[0]], {})
        res[str(fused)] = {"log": [e if isinstance(e, str) else e[0] + (":scatter" if e[-1] is True else "") for e in LOG],
                           "err": float((got.double() - torch.from_numpy(dW1o)).abs().max())}
    print(json.dumps(res))
""") % (ROOT, SHIM)


def test_fused_scatter_step_protocol_order():
    """zero -> (device idle) -> barrier -> backward of every slice -> (device idle) -> barrier; the staged form needs
    neither the zeroing nor the barriers (its collectives order the ranks)."""
    import json
    r = subprocess.run([sys.executable, "-c", PROTOCOL], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-4000:]
    res = json.loads(r.stdout.strip().splitlines()[-1])
    log = res["True"]["log"]
    kernels = [e for e in log if e.startswith("mlp_bwd_slice")]
    assert kernels == ["mlp_bwd_slice:scatter"] * 4                       # every slice through the epilogue's scatter
    assert "reduce_scatter" not in log and "all_reduce" not in log
    i0, i1 = log.index("zero_grad"), log.index("barrier")
    first_k = log.index("mlp_bwd_slice:scatter")
    last_k = len(log) - 1 - log[::-1].index("mlp_bwd_slice:scatter")
    b2 = len(log) - 1 - log[::-1].index("barrier")
    assert i0 < i1 < first_k and last_k < b2 and log.count("barrier") == 2
    assert "stream.synchronize" in log[i0:i1] and "stream.synchronize" in log[last_k:b2]
    assert res["True"]["err"] < 1e-4                                       # stale shard contents were cleared
    staged = res["False"]["log"]
    assert "barrier" not in staged and "zero_grad" not in staged
    assert staged.count("reduce_scatter") == 8 and [e for e in staged if e.startswith("mlp_bwd")] == ["mlp_bwd_slice"] * 4
    assert res["False"]["err"] < 1e-4
