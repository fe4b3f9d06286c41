"""GPU parity of the sharded MLP block (Section 3.3 with zero-redundancy data parallelism, applied to the
Linear -> GeLU -> Linear pair split along ffn): the per-slice entry points with gathered compact weights
against the flat-buffer calls, and the slice loop over emulated ranks (one after another in this process,
their "peer" buffers on this GPU) against the fp64 oracle on the whole batch."""
import numpy as np
import pytest

import oracle
from paper_2209_13258_b200 import inputs
from util import Guarded, assert_close, to_dev, to_f64

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2209_13258_b200 as pkg
    pkg.lib()
    return pkg


def bits(t):
    return t.view(torch.int32 if t.dtype == torch.float32 else torch.int16)


@pytest.mark.parametrize("shape,k", [((256, 512, 2048), 4), ((300, 264, 520), 3), ((512, 1024, 4096), 1),
                                     ((130, 136, 392), 5)])
@pytest.mark.parametrize("recompute", [False, True])
def test_compact_slice_entry_points_match_the_flat_buffer_block_bit_for_bit(P, shape, k, recompute):
    M, H, F = shape
    if P.osdp_slice_range(F, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c = inputs.mlp_case(M, H, F, w_std=0.05, bias_std=0.1, layer=6)
    x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
    b1, b2 = to_dev(c["b1"]), to_dev(c["b2"])
    W1 = wf[c["off_w1"]:c["off_w1"] + F * H].view(F, H)
    W2 = wf[c["off_w2"]:c["off_w2"] + H * F].view(H, F)
    fl = P.FLAG_RECOMPUTE if recompute else 0
    _, n1 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_FWD, 0)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_BWD, fl)
    res = {}
    for compact in (False, True):
        ws = P.new_workspace(max(n1, n2))
        out, z1, dx = Guarded((M, H), torch.bfloat16), Guarded((M, F), torch.bfloat16), Guarded((M, H), torch.bfloat16)
        dwf = torch.zeros(wf.numel(), dtype=torch.float32, device="cuda")
        db1, db2 = Guarded((F,), torch.float32), Guarded((H,), torch.float32)
        zs = None if recompute else z1.t
        if not compact:
            P.osdp_split_mlp_fwd(x, wf, c["off_w1"], b1, c["off_w2"], b2, M, H, F, k, 1, out.t, z1.t, ws, check=True)
            P.osdp_split_mlp_bwd(dy, x, wf, c["off_w1"], c["off_w2"], zs, M, H, F, k, 1, dx.t, dwf, c["off_w1"],
                                 c["off_w2"], P.DTYPE_FP32, fl, db1.t, db2.t, ws, check=True, b1=b1)
            dw1 = dwf[c["off_w1"]:c["off_w1"] + F * H].view(F, H).clone()
            dw2 = dwf[c["off_w2"]:c["off_w2"] + H * F].view(H, F).clone()
        else:
            dw1 = torch.zeros(F, H, dtype=torch.float32, device="cuda")
            dw2 = torch.zeros(H, F, dtype=torch.float32, device="cuda")
            sl = [P.osdp_slice_range(F, k, s)[1:] for s in range(k)]
            for s, (b, e) in enumerate(sl):
                w1s, w2s = W1[b:e].contiguous(), W2[:, b:e].contiguous()
                P.osdp_zdp_mlp_fwd_slice(x, w1s, w2s, e - b, b1, b2, M, H, F, k, 1, s, out.t, z1.t, ws, check=True)
            for s, (b, e) in enumerate(sl):
                w1s, w2s = W1[b:e].contiguous(), W2[:, b:e].contiguous()
                g1, g2 = Guarded((e - b, H), torch.float32), Guarded((H, e - b), torch.float32)
                P.osdp_zdp_mlp_bwd_slice(dy, x, w1s, w2s, e - b, b1, zs, M, H, F, k, 1, s, dx.t, g1.t, g2.t, e - b, None,
                                         None, P.DTYPE_FP32, fl, db1.t, db2.t, ws, check=True)
                g1.check(); g2.check()
                dw1[b:e] = g1.t
                dw2[:, b:e] = g2.t
        rc, st = P.osdp_read_device_status(ws)
        assert rc == 0 and st == 0
        for g in (out, z1, dx, db1, db2):
            g.check()
        res[compact] = {"y": out.t.clone(), "z1": z1.t.clone(), "dx": dx.t.clone(), "dw1": dw1, "dw2": dw2,
                        "db1": db1.t.clone(), "db2": db2.t.clone()}
    for name in res[True]:
        assert torch.equal(bits(res[True][name]), bits(res[False][name])), name


class EmulatedComm:
    """Collectives of the loop for ranks that run one after another in this process (see test_gpu_zdp.py); the
    shard buffers of every rank are registered under the operator they belong to."""

    def __init__(self, rank, world, shared):
        self.rank, self.world, self.shared = rank, world, shared

    def _which(self, kind, buf):
        for i, per_rank in enumerate(self.shared[kind]):
            if per_rank[self.rank] is not None and per_rank[self.rank].data_ptr() == buf.data_ptr():
                return i
        raise AssertionError("unregistered shard buffer")

    def all_gather_slice(self, dst, shard_buf, off, n):
        i = self._which("param", shard_buf)
        for q in range(self.world):
            dst[q * n:(q + 1) * n].copy_(self.shared["param"][i][q][off:off + n])

    def reduce_scatter_slice(self, shard_buf, off, n, src):
        i = self._which("grad", shard_buf)
        for q in range(self.world):
            self.shared["acc"][i][q][off:off + n] += src[q * n:(q + 1) * n].double()

    def all_reduce(self, t, tag=None):
        acc = self.shared.setdefault("dp_acc", {})
        acc[tag] = t.double().clone() if tag not in acc else acc[tag] + t.double()

    def barrier(self):
        pass

    def peer_buffers(self, numel, dtype, device):
        # the i-th request of every rank returns the same list: one buffer per rank, all on this GPU
        lst = self.shared.setdefault("peer_lists", [])
        idx = self.shared["peer_next"][self.rank]
        self.shared["peer_next"][self.rank] += 1
        if idx >= len(lst):
            lst.append([torch.zeros(numel, dtype=dtype, device=device) for _ in range(self.world)])
        return lst[idx]


@pytest.mark.parametrize("world", [1, 2, 4])
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("shape,k,recompute", [((512, 512, 2048), 4, False), ((384, 1024, 4096), 8, True),
                                               ((300, 264, 520), 3, False)])
def test_mlp_slice_loop_over_emulated_ranks_matches_oracle(P, world, fused, shape, k, recompute):
    from paper_2209_13258_b200.zdp import ZdpSplitMLP
    M, H, F = shape
    if P.osdp_slice_range(F, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c = inputs.mlp_case(M, H, F, w_std=0.05, bias_std=0.1, layer=7)
    wf = to_dev(c["w_flat"])
    W1 = wf[c["off_w1"]:c["off_w1"] + F * H].view(F, H)
    W2 = wf[c["off_w2"]:c["off_w2"] + H * F].view(H, F)
    b1, b2 = to_dev(c["b1"]), to_dev(c["b2"])
    shared = {"param": [[None] * world, [None] * world], "grad": [[None] * world, [None] * world],
              "acc": [[None] * world, [None] * world], "peer_next": [0] * world}
    layers = []
    for r in range(world):
        layer = ZdpSplitMLP(H, F, k, comm=EmulatedComm(r, world, shared), fused_scatter=fused)
        layer.load_full_weights(W1, W2)
        for i in range(2):
            shared["param"][i][r] = layer.param_shard[i]
            shared["grad"][i][r] = layer.grad_shard[i]
            shared["acc"][i][r] = torch.zeros(layer.grad_shard[i].numel(), dtype=torch.float64, device="cuda")
        layers.append(layer)
    y = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    db1 = torch.zeros(F, dtype=torch.float64, device="cuda")
    db2 = torch.zeros(H, dtype=torch.float64, device="cuda")
    x_all, dy_all = to_dev(c["x"]), to_dev(c["dy"])
    for r, layer in enumerate(layers):
        rows = torch.arange(r, M, world, device="cuda")
        xr, dyr = x_all[rows].contiguous(), dy_all[rows].contiguous()
        z1 = None if recompute else torch.empty(rows.numel(), F, dtype=torch.bfloat16, device="cuda")
        yr = layer.forward(xr, b1, b2, z1_save=z1)
        d1 = torch.empty(F, dtype=torch.float32, device="cuda")
        d2 = torch.empty(H, dtype=torch.float32, device="cuda")
        dxr = layer.backward(dyr, xr, z1_saved=z1, b1=b1, db1=d1, db2=d2)
        torch.cuda.synchronize()
        rc, st = P.osdp_read_device_status(layer._ws)
        assert rc == 0 and st == 0
        y[rows], dx[rows] = yr, dxr
        db1 += d1.double()
        db2 += d2.double()
    full = []
    for i in range(2):
        lay = layers[0].layouts[i]
        shards = []
        for q, l in enumerate(layers):
            t = shared["acc"][i][q].clone()
            for s in range(k):
                if l._scatter_ok(s):      # scattered by the epilogue: complete in the rank's own shard
                    n, o = lay.slices[s][3], lay.slices[s][4]
                    t[o:o + n] = l.grad_shard[i][o:o + n].double()
            shards.append(t)
        full.append(lay.unshard(shards))
    _, yo = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
    dXo, dW1o, db1o, dW2o, db2o = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    assert_close(to_f64(y), yo, "Y")
    assert_close(to_f64(dx), dXo, "dX")
    assert_close(full[0].cpu().numpy(), dW1o, "dW1 (sum over ranks)")
    assert_close(full[1].cpu().numpy(), dW2o, "dW2 (sum over ranks)")
    assert_close(db1.cpu().numpy(), db1o, "db1 (sum over ranks)")
    assert_close(db2.cpu().numpy(), db2o, "db2 (sum over ranks)")
    st = layers[0].staging_bytes(M)
    if fused and all(layers[0]._scatter_ok(s) for s in range(k)):
        assert st["grad_staging"] == 0
    # gathered weights: two slices' worth of each matrix
    per = sum(max(sl[3] for sl in lay.slices) for lay in layers[0].layouts) * world * 2
    assert st["weight_staging"] == (2 if k > 1 else 1) * per


MIXED = [((512, 512, 2048), 4, [0, 1, 1, 0]), ((512, 512, 2048), 4, [1, 0, 0, 0]), ((300, 264, 520), 3, [0, 0, 1]),
         ((384, 1024, 4096), 8, [1, 0, 1, 1, 0, 0, 1, 0]), ((256, 512, 1024), 2, [0, 0])]


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("fused,recompute", [(False, False), (True, True)])
@pytest.mark.parametrize("shape,k,modes", MIXED)
def test_mlp_slices_in_mixed_dp_and_zdp_modes_match_oracle(P, world, fused, recompute, shape, k, modes):
    """Section 3.3, last paragraph, for the block: some slices (both their weights) replicated, the others sharded."""
    from paper_2209_13258_b200.zdp import ZdpSplitMLP
    M, H, F = shape
    c = inputs.mlp_case(M, H, F, w_std=0.05, bias_std=0.1, layer=9)
    wf = to_dev(c["w_flat"])
    W1 = wf[c["off_w1"]:c["off_w1"] + F * H].view(F, H)
    W2 = wf[c["off_w2"]:c["off_w2"] + H * F].view(H, F)
    b1, b2 = to_dev(c["b1"]), to_dev(c["b2"])
    shared = {"param": [[None] * world, [None] * world], "grad": [[None] * world, [None] * world],
              "acc": [[None] * world, [None] * world], "peer_next": [0] * world}
    layers = []
    for r in range(world):
        layer = ZdpSplitMLP(H, F, k, comm=EmulatedComm(r, world, shared), fused_scatter=fused, slice_modes=modes)
        layer.load_full_weights(W1, W2)
        for i in range(2):
            shared["param"][i][r] = layer.param_shard[i]
            shared["grad"][i][r] = layer.grad_shard[i]
            shared["acc"][i][r] = torch.zeros(layer.grad_shard[i].numel(), dtype=torch.float64, device="cuda")
        layers.append(layer)
    # checkpoint round trip: the full weights come back from the ranks' parts
    for i, W in enumerate((W1, W2)):
        assert torch.equal(layers[0].full_from_parts(i, [l.param_shard[i] for l in layers], layers[0].dp_weight[i]), W)
    y = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    db1 = torch.zeros(F, dtype=torch.float64, device="cuda")
    db2 = torch.zeros(H, dtype=torch.float64, device="cuda")
    x_all, dy_all = to_dev(c["x"]), to_dev(c["dy"])
    for r, layer in enumerate(layers):
        rows = torch.arange(r, M, world, device="cuda")
        xr, dyr = x_all[rows].contiguous(), dy_all[rows].contiguous()
        z1 = None if recompute else torch.empty(rows.numel(), F, dtype=torch.bfloat16, device="cuda")
        yr = layer.forward(xr, b1, b2, z1_save=z1)
        d1 = torch.empty(F, dtype=torch.float32, device="cuda")
        d2 = torch.empty(H, dtype=torch.float32, device="cuda")
        dxr = layer.backward(dyr, xr, z1_saved=z1, b1=b1, db1=d1, db2=d2)
        torch.cuda.synchronize()
        rc, st = P.osdp_read_device_status(layer._ws)
        assert rc == 0 and st == 0
        y[rows], dx[rows] = yr, dxr
        db1 += d1.double()
        db2 += d2.double()
    full = []
    for i in range(2):
        lay = layers[0].layouts[i]
        shards = []
        for q, l in enumerate(layers):
            t = shared["acc"][i][q].clone()
            for s in l.zdp_slices:
                if l._scatter_ok(s):      # scattered by the epilogue: complete in the rank's own shard
                    n, o = lay.slices[s][3], l._zoff[i][s]
                    t[o:o + n] = l.grad_shard[i][o:o + n].double()
            shards.append(t)
        dp_parts = {s: shared["dp_acc"][(i, s)] for s in range(k) if modes[s] == 0}
        full.append(layers[0].full_from_parts(i, shards, dp_parts))
    _, yo = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
    dXo, dW1o, db1o, dW2o, db2o = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    assert_close(to_f64(y), yo, "Y")
    assert_close(to_f64(dx), dXo, "dX")
    assert_close(full[0].cpu().numpy(), dW1o, "dW1 (sum over ranks)")
    assert_close(full[1].cpu().numpy(), dW2o, "dW2 (sum over ranks)")
    assert_close(db1.cpu().numpy(), db1o, "db1 (sum over ranks)")
    assert_close(db2.cpu().numpy(), db2o, "db2 (sum over ranks)")
    # resident weights: whole DP slices plus 1/world of the ZDP slices (up to the 8-element padding), both matrices
    want = 0
    for lay in layers[0].layouts:
        dp_elems = sum(lay.slices[s][2] for s in range(k) if modes[s] == 0)
        zdp_shard = sum(lay.slices[s][3] for s in range(k) if modes[s] == 1)
        want += 2 * (dp_elems + max(zdp_shard, 8))
    assert layers[0].state_bytes()["weights"] == want
    assert all(len(st) == min(2, modes.count(1)) for st in layers[0].w_stage)


def test_sharded_loop_replays_from_a_cuda_graph(P):
    """The whole loop (gathers on the communication stream, slice kernels, reduce-scatters or epilogue scatter)
    is plain stream work with fork / join events: captured once on a one-rank NCCL group, the replay gives the
    bits of the eager run."""
    import torch.distributed as dist
    from paper_2209_13258_b200.zdp import ZdpSplitMLP
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    M, H, F, k = 512, 512, 2048, 4
    try:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29761", rank=0, world_size=1)
    except Exception as e:   # no usable loopback / port on this machine: nothing of the library is at fault
        pytest.skip("cannot form a one-rank NCCL group here: %r" % (e,))
    try:
        c = inputs.mlp_case(M, H, F, w_std=0.05, bias_std=0.1, layer=9)
        wf = to_dev(c["w_flat"])
        x, dy, b1, b2 = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["b1"]), to_dev(c["b2"])
        out = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
        dx = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
        z1 = torch.empty(M, F, dtype=torch.bfloat16, device="cuda")
        for fused in (False, True):
            try:
                layer = ZdpSplitMLP(H, F, k, fused_scatter=fused)
            except Exception as e:   # symmetric memory not available
                print("skipping the fused form:", repr(e)[:200])
                continue
            layer.load_full_weights(wf[c["off_w1"]:c["off_w1"] + F * H].view(F, H),
                                    wf[c["off_w2"]:c["off_w2"] + H * F].view(H, F))

            def step():
                layer.zero_grad()
                layer.forward(x, b1, b2, out=out, z1_save=z1)
                layer.backward(dy, x, z1_saved=z1, dx=dx)
            step()
            torch.cuda.synchronize()
            ref = (out.clone(), dx.clone(), layer.grad_shard[0].clone(), layer.grad_shard[1].clone())
            g, s = torch.cuda.CUDAGraph(), torch.cuda.Stream()
            with torch.cuda.stream(s):
                with torch.cuda.graph(g, stream=s):
                    step()
            out.zero_(); dx.zero_()
            for _ in range(2):
                g.replay()
            torch.cuda.synchronize()
            for a, b in zip((out, dx, layer.grad_shard[0], layer.grad_shard[1]), ref):
                assert torch.equal(bits(a), bits(b))
            _, yo = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
            assert_close(to_f64(out), yo, "Y")
    finally:
        dist.destroy_process_group()
