"""GPU parity of the sharded slice loop (Section 3.3 combined with zero-redundancy data parallelism):
the per-slice entry points that read a gathered compact slice, and the loop around them with the
ranks of a data-parallel group emulated one after another in this process (no kernel waits on
another rank), checked against the fp64 oracle on the whole batch."""
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


SHAPES = [(256, 2048, 512, 4), (300, 520, 328, 3), (130, 392, 264, 5), (1024, 1024, 2048, 2)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("act", [0, 1])
def test_gathered_slice_entry_points_match_flat_buffer_ones_bit_for_bit(P, shape, split, act):
    from paper_2209_13258_b200.zdp import ShardLayout
    M, N, K, k = shape
    D = N if split == 0 else K
    if P.osdp_slice_range(D, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c = inputs.linear_case(M, N, K, w_std=0.05, bias_std=0.2, w_offset=64, flat_pad=8)
    x, dy, wf, b = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"]), to_dev(c["bias"])
    off = c["w_offset"]
    W = wf[off:off + N * K].view(N, K)
    lay = ShardLayout(N, K, k, split, 1)
    _, n1 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, act, P.OP_LINEAR_FWD, P.FLAG_SLICE_MAJOR)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, act, P.OP_LINEAR_BWD, P.FLAG_SLICE_MAJOR)
    res = {}
    for staged in (False, True):
        ws = P.new_workspace(max(n1, n2))
        out, z, dx = Guarded((M, N), torch.bfloat16), Guarded((M, N), torch.bfloat16), Guarded((M, K), torch.bfloat16)
        dwf = torch.zeros(wf.numel(), dtype=torch.float32, device="cuda")
        db = Guarded((N,), torch.float32)
        zs = z.t if act else None
        dw_full = torch.zeros(N, K, dtype=torch.float32, device="cuda")
        for s in range(k):
            if staged:
                wslice = Guarded((lay.slices[s][2],), torch.bfloat16)
                wslice.t.copy_(lay.slice_matrix(W, s).contiguous().reshape(-1))
                P.osdp_zdp_linear_fwd_slice(x, wslice.t, lay.slices[s][5], b, M, N, K, k, split, act, s, out.t, zs, ws,
                                            check=True)
                wslice.check()
            else:
                P.osdp_split_linear_fwd_slice(x, wf, off, b, M, N, K, k, split, act, s, out.t, zs, ws, check=True)
        for s in range(k):
            if staged:
                bq, e, elems, _, _, ld = lay.slices[s]
                wslice = lay.slice_matrix(W, s).contiguous()
                dws = Guarded((elems,), torch.float32)
                P.osdp_zdp_linear_bwd_slice(dy, x, wslice, ld, zs, M, N, K, k, split, act, s, dx.t, dws.t, ld,
                                            P.DTYPE_FP32, 0, db.t, ws, check=True)
                dws.check()
                assert not bool(torch.isnan(dws.t).any()), "slice gradient not fully written"
                lay.slice_matrix(dw_full, s).copy_(dws.t.view(-1, ld))
            else:
                P.osdp_split_linear_bwd_slice(dy, x, wf, off, zs, M, N, K, k, split, act, s, dx.t, dwf, off,
                                              P.DTYPE_FP32, 0, db.t, ws, check=True)
        if not staged:
            dw_full = dwf[off:off + N * K].view(N, K).clone()
        rc, st = P.osdp_read_device_status(ws)
        assert rc == 0 and st == 0
        for g in (out, dx, db) + ((z,) if act else ()):
            g.check()
        res[staged] = {"y": out.t.clone(), "dx": dx.t.clone(), "dw": dw_full, "db": db.t.clone()}
    for name in ("y", "dx", "dw", "db"):
        assert torch.equal(bits(res[True][name]), bits(res[False][name])), name


def test_gathered_slice_argument_errors(P):
    M, N, K, k = 128, 256, 128, 2
    x = torch.zeros(M, K, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(N // k, K, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    _, n = P.osdp_split_linear_workspace_bytes(M, N, K, k, 0, 0, P.OP_LINEAR_BWD, P.FLAG_SLICE_MAJOR)
    ws = P.new_workspace(n)
    f = P.osdp_zdp_linear_fwd_slice
    assert f(x, w, 0, None, M, N, K, k, 0, 0, 0, out, None, ws) == 2        # ld_w <= 0
    assert f(x, w, K - 8, None, M, N, K, k, 0, 0, 0, out, None, ws) == 2    # ld_w below the slice's row length
    assert f(x, w, K + 4, None, M, N, K, k, 0, 0, 0, out, None, ws) == 4    # ld_w not a multiple of 8
    assert f(x, w, K, None, M, N, K, k, 0, 0, 2, out, None, ws) == 3        # slice index out of range
    assert f(x, None, K, None, M, N, K, k, 0, 0, 0, out, None, ws) == 1
    g = P.osdp_zdp_linear_bwd_slice
    dw = torch.zeros(N // k, K, dtype=torch.float32, device="cuda")
    assert g(out, x, w, K, None, M, N, K, k, 0, 0, 0, None, dw, 0, P.DTYPE_FP32, 0, None, ws) == 2
    assert g(out, x, w, K, None, M, N, K, k, 0, 0, 0, None, dw, K - 8, P.DTYPE_FP32, 0, None, ws) == 2
    assert g(out, x, w, K, None, M, N, K, k, 0, 0, 0, None, dw, K, P.DTYPE_FP32, P.FLAG_PAIR_SLICES, None, ws) == 6
    assert g(out, x, w, K, None, M, N, K, k, 0, 0, 0, None, None, 0, P.DTYPE_FP32, 0, None, ws) == 0   # dW skipped


class EmulatedComm:
    """The loop's collectives for `world` ranks that run one after another in this process: all ranks'
    parameter shards are visible, and reduce-scatter / all-reduce add the caller's contribution to shared
    fp64 accumulators (the sum over ranks is complete once every rank has run)."""

    def __init__(self, rank, world, shared):
        self.rank, self.world, self.shared = rank, world, shared

    def all_gather_slice(self, dst, shard_buf, off, n):
        assert shard_buf.data_ptr() == self.shared["param"][self.rank].data_ptr()
        for q in range(self.world):
            dst[q * n:(q + 1) * n].copy_(self.shared["param"][q][off:off + n])

    def reduce_scatter_slice(self, shard_buf, off, n, src):
        for q in range(self.world):
            self.shared["grad_acc"][q][off:off + n] += src[q * n:(q + 1) * n].double()
        shard_buf[off:off + n].copy_(src[self.rank * n:(self.rank + 1) * n])   # this rank's own term only

    def all_reduce(self, t, tag=None):
        acc = self.shared["dp_acc"]
        acc[tag] = t.double().clone() if tag not in acc else acc[tag] + t.double()

    def barrier(self):
        pass

    def peer_buffers(self, numel, dtype, device):
        # "peer" memory of the emulated ranks: one buffer per rank on this GPU, the same list for every rank
        key = ("peer", numel, dtype)
        if key not in self.shared:
            self.shared[key] = [torch.zeros(numel, dtype=dtype, device=device) for _ in range(self.world)]
        return self.shared[key]


def run_emulated_ranks(P, world, M, N, K, k, split, act, modes, fused=False, dw_dtype=None):
    """Forward + backward of the slice loop for every emulated rank on its own token rows; returns the
    assembled Y, dX, sum over ranks of dW and db, and the first rank's layer."""
    from paper_2209_13258_b200.zdp import ZdpSplitLinear
    c = inputs.linear_case(M, N, K, w_std=0.05, bias_std=0.2)
    W = to_dev(c["w_flat"])[c["w_offset"]:c["w_offset"] + N * K].view(N, K)
    bias = to_dev(c["bias"])
    shared = {"param": [None] * world, "grad_acc": [None] * world, "dp_acc": {}}
    layers = []
    for r in range(world):
        layer = ZdpSplitLinear(N, K, k, split, act=act, comm=EmulatedComm(r, world, shared), slice_modes=modes,
                               fused_scatter=fused, dw_dtype=P.DTYPE_FP32 if dw_dtype is None else dw_dtype)
        layer.load_full_weight(W)
        shared["param"][r] = layer.param_shard
        shared["grad_acc"][r] = torch.zeros(layer.grad_shard.numel(), dtype=torch.float64, device="cuda")
        layers.append(layer)
    y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(M, K, dtype=torch.bfloat16, device="cuda")
    db = torch.zeros(N, dtype=torch.float64, device="cuda")
    x_all, dy_all = to_dev(c["x"]), to_dev(c["dy"])
    for r, layer in enumerate(layers):
        rows = torch.arange(r, M, world, device="cuda")               # this rank's tokens
        xr, dyr = x_all[rows].contiguous(), dy_all[rows].contiguous()
        zr = torch.empty(rows.numel(), N, dtype=torch.bfloat16, device="cuda") if act else None
        yr = layer.forward(xr, bias=bias, z_save=zr)
        dbr = torch.empty(N, dtype=torch.float32, device="cuda")
        dxr = layer.backward(dyr, xr, z_saved=zr, dbias=dbr)
        torch.cuda.synchronize()
        rc, st = P.osdp_read_device_status(layer._ws)
        assert rc == 0 and st == 0
        y[rows], dx[rows] = yr, dxr
        db += dbr.double()
    if fused:
        # slices scattered by the epilogue are complete in the ranks' own shards; the others came through the
        # emulated collective and are complete in the fp64 accumulators
        shards = []
        for q, l in enumerate(layers):
            t = shared["grad_acc"][q].clone()
            for s in range(k):
                if l._scatter_ok(s):
                    n, o = l.layout.slices[s][3], l._zoff[s]
                    t[o:o + n] = l.grad_shard[o:o + n].double()
            shards.append(t)
        dW = layers[0].full_from_parts(shards, shared["dp_acc"])
    else:
        dW = layers[0].full_from_parts(shared["grad_acc"], shared["dp_acc"])
    return c, y, dx, dW, db, layers[0]


def check_against_oracle(c, y, dx, dW, db, act, k, split):
    z, yo = oracle.linear_fwd(c["x"], c["w"], c["bias"], act, k, split)
    dXo, dWo, dbo = oracle.linear_bwd(c["dy"], c["x"], c["w"], z, act, k, split)
    assert_close(to_f64(y), yo, "Y")
    assert_close(to_f64(dx), dXo, "dX")
    assert_close(dW.cpu().numpy(), dWo, "dW (sum over ranks)")
    assert_close(db.cpu().numpy(), dbo, "db (sum over ranks)")


@pytest.mark.parametrize("world", [1, 2, 3])
@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("case", [(384, 520, 264, 3, 1), (512, 2048, 512, 4, 0), (300, 1024, 1024, 8, 1)])
def test_slice_loop_over_emulated_ranks_matches_oracle(P, world, split, case):
    M, N, K, k, act = case
    D = N if split == 0 else K
    if P.osdp_slice_range(D, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c, y, dx, dW, db, layer = run_emulated_ranks(P, world, M, N, K, k, split, act, None)
    check_against_oracle(c, y, dx, dW, db, act, k, split)
    # the gathered weights never take more than two slices' worth
    st = layer.staging_bytes(M)
    assert st["weight_staging"] == 2 * 2 * world * max(sl[3] for sl in layer.layout.slices)
    assert st["weight_staging"] <= 2 * 2 * (N * K // k + 8 * world + max(N, K) * 8)
    assert layer.state_bytes()["weights"] == 2 * layer.layout.shard_total


@pytest.mark.parametrize("world", [1, 2, 4])
@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("case,modes", [((512, 2048, 512, 4, 0), None), ((384, 1024, 1024, 8, 1), None),
                                        ((512, 2048, 512, 4, 0), [0, 1, 1, 0]), ((256, 1024, 512, 1, 0), None),
                                        ((300, 520, 264, 3, 1), None)])
def test_reduce_scatter_fused_into_the_gemm_epilogue(P, world, split, case, modes):
    """The backward GEMM's epilogue reduce-adds each slice's dW into the owning ranks' shards (peer buffers
    emulated by one buffer per rank on this GPU); slices whose rows do not divide fall back to the collective."""
    M, N, K, k, act = case
    D = N if split == 0 else K
    if P.osdp_slice_range(D, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c, y, dx, dW, db, layer = run_emulated_ranks(P, world, M, N, K, k, split, act, modes, fused=True)
    check_against_oracle(c, y, dx, dW, db, act, k, split)
    rows = [(layer.layout.slices[s][1] - layer.layout.slices[s][0]) if split == 0 else N for s in range(k)]
    expect = [layer.modes[s] == 1 and rows[s] % (32 * world) == 0 for s in range(k)]
    assert [layer._scatter_ok(s) for s in range(k)] == expect
    if (M, N, K) == (512, 2048, 512) and modes is None:
        assert all(expect)          # this case really runs the fused path on every slice


@pytest.mark.parametrize("world", [2, 4])
def test_fused_scatter_with_bf16_gradients(P, world):
    """bf16 gradient shards: the epilogue's reduce-add is a bf16 addition per rank's term."""
    M, N, K, k = 512, 2048, 512, 4
    c, y, dx, dW, db, layer = run_emulated_ranks(P, world, M, N, K, k, 0, 0, None, fused=True, dw_dtype=P.DTYPE_BF16)
    assert all(layer._scatter_ok(s) for s in range(k)) and layer.grad_shard.dtype == torch.bfloat16
    check_against_oracle(c, y, dx, dW, db, 0, k, 0)


def test_fused_scatter_equals_staged_reduce_scatter_for_one_rank(P):
    """world = 1: the epilogue's scatter into the rank's own shard gives the bits of the staged path."""
    M, N, K, k = 512, 2048, 512, 4
    for split in (0, 1):
        res = []
        for fused in (False, True):
            c, y, dx, dW, db, layer = run_emulated_ranks(P, 1, M, N, K, k, split, 0, None, fused=fused)
            res.append(dW)
        assert torch.equal(res[0], res[1])


def test_scatter_argument_errors(P):
    M, N, K, k = 128, 256, 128, 2
    x = torch.zeros(M, K, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(N // k, K, dtype=torch.bfloat16, device="cuda")
    dy = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    _, n = P.osdp_split_linear_workspace_bytes(M, N, K, k, 0, 0, P.OP_LINEAR_BWD, P.FLAG_SLICE_MAJOR)
    ws = P.new_workspace(n)
    g = P.osdp_zdp_linear_bwd_slice_scatter
    sh = [torch.zeros(N // k * K // 2, dtype=torch.float32, device="cuda") for _ in range(2)]
    assert g(dy, x, w, K, None, M, N, K, k, 0, 0, 0, None, sh, P.DTYPE_FP32, 0, None, ws) == 0
    assert g(dy, x, w, K, None, M, N, K, k, 0, 0, 0, None, sh, P.DTYPE_FP32, P.FLAG_ACCUMULATE_DW, None, ws) == 6
    sh3 = sh + [sh[0]]
    assert g(dy, x, w, K, None, M, N, K, k, 0, 0, 0, None, sh3, P.DTYPE_FP32, 0, None, ws) == 6     # 128 rows / 3 ranks
    sh8 = [sh[0]] * 8
    assert g(dy, x, w, K, None, M, N, K, k, 0, 0, 0, None, sh8, P.DTYPE_FP32, 0, None, ws) == 6     # 16 rows per rank
    assert g(dy, x, w, K, None, M, N, K, k, 0, 0, 0, None, [sh[0]] * 9, P.DTYPE_FP32, 0, None, ws) == 6
    assert g(dy, x, w, K, None, M, N, K, k, 0, 0, 0, None, [sh[0], 0], P.DTYPE_FP32, 0, None, ws) == 1


MIXED = [((512, 2048, 512, 4, 0), [0, 1, 1, 0]), ((512, 2048, 512, 4, 0), [1, 0, 0, 0]),
         ((384, 520, 264, 3, 1), [0, 0, 1]), ((300, 1024, 1024, 8, 1), [1, 0, 1, 1, 0, 0, 1, 0]),
         ((256, 512, 512, 2, 0), [0, 0])]


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("case,modes", MIXED)
def test_slices_in_mixed_dp_and_zdp_modes_match_oracle(P, world, split, case, modes):
    """Section 3.3, last paragraph: some slices of one operator replicated (DP), the others sharded (ZDP)."""
    M, N, K, k, act = case
    D = N if split == 0 else K
    if P.osdp_slice_range(D, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c, y, dx, dW, db, layer = run_emulated_ranks(P, world, M, N, K, k, split, act, modes)
    check_against_oracle(c, y, dx, dW, db, act, k, split)
    # resident weights: whole DP slices plus 1/world of the ZDP slices (up to the 8-element padding)
    dp_elems = sum(layer.layout.slices[s][2] for s in range(k) if modes[s] == 0)
    zdp_shard = sum(layer.layout.slices[s][3] for s in range(k) if modes[s] == 1)
    assert layer.state_bytes()["weights"] == 2 * (dp_elems + max(zdp_shard, 8))
    assert len(layer.w_stage) == min(2, modes.count(1))


def test_planned_granularity_and_modes_run_in_the_slice_loop(P):
    """The plan search's answer for one operator (granularity and how many slices stay replicated) drives the
    slice loop: states held are what the plan priced, results match the oracle."""
    from paper_2209_13258_b200.zdp import slice_modes_from_plan
    M, N, K, world = 256, 2048, 512, 2
    params = float(N * K)
    op = (2.0 * params, 2.0 * M * (N + K), 0.0, 2.0 * params, 1e-4)        # states = the bf16 weights alone
    # room for three quarters of the weights replicated: only a 4-way cut can use it
    limit = 2.0 * params * (0.75 + 0.25 / world) + op[1] + 1.0
    rc, ks, dps, b, t, _ = P.osdp_plan_search_granularity([op], [[(1, 0.0), (2, 0.0), (4, 0.0)]], world, 0.0, 1e-9,
                                                          limit, 1)
    assert (rc, ks, dps, b) == (0, [4], [3], 1)
    modes = slice_modes_from_plan(ks[0], dps[0])
    c, y, dx, dW, db, layer = run_emulated_ranks(P, world, M, N, K, ks[0], 0, 0, modes)
    check_against_oracle(c, y, dx, dW, db, 0, ks[0], 0)
    assert layer.state_bytes()["weights"] <= limit - op[1]


def test_slice_loop_on_a_one_rank_nccl_group(P):
    """The product's own communicator (torch.distributed, NCCL) with world size 1: every collective
    of the loop runs, on its own stream, and the result matches the oracle."""
    import torch.distributed as dist
    from paper_2209_13258_b200.zdp import ZdpSplitLinear
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    M, N, K, k = 512, 1024, 512, 4
    try:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29753", rank=0, world_size=1)
    except Exception as e:   # no usable loopback / port on this machine: nothing of the library is at fault
        pytest.skip("cannot form a one-rank NCCL group here: %r" % (e,))
    try:
        for split, modes in ((0, None), (1, None), (0, [0, 1, 1, 0]), (1, [1, 0, 0, 1])):
            c = inputs.linear_case(M, N, K, w_std=0.05, bias_std=0.2)
            W = to_dev(c["w_flat"])[c["w_offset"]:c["w_offset"] + N * K].view(N, K)
            layer = ZdpSplitLinear(N, K, k, split, act=1, slice_modes=modes)
            layer.load_full_weight(W)
            x, dy, bias = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["bias"])
            z = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
            db = torch.empty(N, dtype=torch.float32, device="cuda")
            for _ in range(2):   # twice: staging buffers and events are reused correctly
                y = layer.forward(x, bias=bias, z_save=z)
                dx = layer.backward(dy, x, z_saved=z, dbias=db)
            torch.cuda.synchronize()
            dW = layer.full_from_parts([layer.grad_shard], layer.dp_grad)
            zo, yo = oracle.linear_fwd(c["x"], c["w"], c["bias"], 1, k, split)
            dXo, dWo, dbo = oracle.linear_bwd(c["dy"], c["x"], c["w"], zo, 1, k, split)
            assert_close(to_f64(y), yo, "Y")
            assert_close(to_f64(dx), dXo, "dX")
            assert_close(to_f64(dW), dWo, "dW")
            assert_close(to_f64(db), dbo, "db")
            # accumulate=True adds a second identical gradient
            layer.backward(dy, x, z_saved=z, dbias=db, accumulate=True)
            torch.cuda.synchronize()
            assert_close(to_f64(layer.full_from_parts([layer.grad_shard], layer.dp_grad)), 2 * dWo, "dW accumulated")
        # the autograd wrapper over the same loop: parameters are the shard and the DP slices, their .grad the
        # summed gradients; a second backward accumulates like any torch parameter
        from paper_2209_13258_b200.nn import ZdpLinear
        for split, modes in ((0, None), (1, [1, 0, 0, 1])):
            c = inputs.linear_case(M, N, K, w_std=0.05, bias_std=0.2, layer=5)
            W = to_dev(c["w_flat"])[c["w_offset"]:c["w_offset"] + N * K].view(N, K)
            m = ZdpLinear(K, N, bias=True, k_split=k, split_dim=split, act=1, slice_modes=modes)
            m.load_full_weight(W)
            with torch.no_grad():
                m.bias.copy_(to_dev(c["bias"]))
            assert m.shard.data_ptr() == m.impl.param_shard.data_ptr()
            x = to_dev(c["x"]).view(4, M // 4, K).requires_grad_(True)
            for _ in range(2):
                y = m(x)
                y.backward(to_dev(c["dy"]).view(4, M // 4, N))
            torch.cuda.synchronize()
            zo, yo = oracle.linear_fwd(c["x"], c["w"], c["bias"], 1, k, split)
            dXo, dWo, dbo = oracle.linear_bwd(c["dy"], c["x"], c["w"], zo, 1, k, split)
            assert_close(to_f64(y).reshape(M, N), yo, "Y (module)")
            assert_close(to_f64(x.grad).reshape(M, K), 2 * dXo, "dX (module, two backward passes)")
            dp = {s: p.grad for s, p in zip(m._dp_order, m.dp_parts)}
            assert_close(to_f64(m.impl.full_from_parts([m.shard.grad], dp)), 2 * dWo, "dW (module)")
            assert_close(to_f64(m.bias.grad), 2 * dbo, "db (module)")
        # the epilogue's scatter into a shard allocated as symmetric memory (one rank: its own buffer)
        try:
            layer = ZdpSplitLinear(N, K, k, 0, act=0, fused_scatter=True)
        except Exception as e:   # symmetric memory not available in this build / on this machine
            print("symmetric memory unavailable:", repr(e)[:200])
            layer = None
        if layer is not None:
            c = inputs.linear_case(M, N, K, w_std=0.05)
            W = to_dev(c["w_flat"])[c["w_offset"]:c["w_offset"] + N * K].view(N, K)
            layer.load_full_weight(W)
            x, dy = to_dev(c["x"]), to_dev(c["dy"])
            assert all(layer._scatter_ok(s) for s in range(k))
            for _ in range(2):
                layer.zero_grad()
                y = layer.forward(x)
                dx = layer.backward(dy, x)
                layer.comm.barrier()
            torch.cuda.synchronize()
            zo, yo = oracle.linear_fwd(c["x"], c["w"], None, 0, k, 0)
            dXo, dWo, _ = oracle.linear_bwd(c["dy"], c["x"], c["w"], zo, 0, k, 0)
            assert_close(to_f64(y), yo, "Y")
            assert_close(to_f64(dx), dXo, "dX")
            assert_close(to_f64(layer.full_from_parts([layer.grad_shard], {})), dWo, "dW scattered by the epilogue")
    finally:
        dist.destroy_process_group()
