"""Host side of the sharded slice loop (Section 3.3 with zero-redundancy data parallelism), on CPU:
the shard layout the C ABI reports, and two gloo ranks that gather every weight slice and
reduce-scatter every slice's weight gradient.  The per-rank arithmetic is done here by the fp64
oracle (this file is a test; the product's arithmetic runs only in the CUDA kernels)."""
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def P():
    import paper_2209_13258_b200 as pkg
    pkg.lib()
    return pkg


CASES = [(2048, 512, 4, 0), (2048, 512, 4, 1), (264, 136, 3, 0), (264, 136, 3, 1), (40, 24, 3, 1), (8, 8, 1, 0),
         (1032, 72, 5, 0), (72, 1032, 8, 1)]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_layout_covers_every_slice_once(P, case, world):
    N, K, k, split = case
    D, other = (N, K) if split == 0 else (K, N)
    total = 0
    covered = 0
    for s in range(k):
        rc, elems, shard, off, ld = P.osdp_zdp_shard_layout(N, K, k, split, world, s)
        assert rc == 0
        rc, b, e = P.osdp_slice_range(D, k, s)
        assert rc == 0
        assert elems == (e - b) * other              # the slice's compact matrix
        assert ld == (K if split == 0 else e - b)
        assert shard % 8 == 0 and world * shard >= elems and world * (shard - 8) < elems   # minimal padding
        assert off == total                          # slices stored one after another
        total += shard
        covered += elems
    rc, elems, shard, off, _ = P.osdp_zdp_shard_layout(N, K, k, split, world, k)
    assert (rc, elems, shard, off) == (0, 0, 0, total)
    assert covered == N * K


def test_layout_argument_errors(P):
    assert P.osdp_zdp_shard_layout(0, 8, 1, 0, 1, 0)[0] == 2            # bad shape
    assert P.osdp_zdp_shard_layout(12, 8, 1, 0, 1, 0)[0] == 4           # N not a multiple of 8
    assert P.osdp_zdp_shard_layout(16, 8, 1, 2, 1, 0)[0] == 3           # bad split enum
    assert P.osdp_zdp_shard_layout(16, 8, 3, 0, 1, 0)[0] == 3           # k = 3 would leave an empty slice
    assert P.osdp_zdp_shard_layout(16, 8, 2, 0, 1, 3)[0] == 3           # slice index past k
    assert P.osdp_zdp_shard_layout(16, 8, 2, 0, 0, 0)[0] == 2           # world < 1
    assert P.lib().osdp_zdp_shard_layout(16, 8, 2, 0, 2, 1, None, None, None, None) == 0   # outputs optional


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("world", [1, 2, 3])
def test_shard_and_unshard_round_trip(P, case, world):
    from paper_2209_13258_b200.zdp import ShardLayout
    N, K, k, split = case
    lay = ShardLayout(N, K, k, split, world)
    full = torch.arange(N * K, dtype=torch.float32).reshape(N, K)
    shards = [lay.shard_of(full, r) for r in range(world)]
    assert all(sh.numel() == lay.shard_total for sh in shards)
    assert torch.equal(lay.unshard(shards), full)
    # every element of W is held by exactly one rank
    assert sum(int((sh != 0).sum()) for sh in shards) == N * K - 1      # element 0 is the only zero payload


def test_slice_modes_from_plan():
    from paper_2209_13258_b200.zdp import slice_modes_from_plan, DP, ZDP
    assert slice_modes_from_plan(4, 3) == [DP, DP, DP, ZDP]
    assert slice_modes_from_plan(1, 0) == [ZDP] and slice_modes_from_plan(2, 2) == [DP, DP]
    for bad in ((0, 0), (2, 3), (2, -1)):
        with pytest.raises(ValueError):
            slice_modes_from_plan(*bad)


def test_runtime_refuses_to_run_without_a_gpu(P):
    if torch.cuda.is_available():
        pytest.skip("CUDA device present")
    from paper_2209_13258_b200.zdp import ZdpSplitLinear

    class Fake:
        rank, world = 0, 1
    with pytest.raises(RuntimeError):
        ZdpSplitLinear(64, 64, 2, 0, comm=Fake())


WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    import oracle
    from paper_2209_13258_b200 import inputs
    from paper_2209_13258_b200.zdp import ShardLayout, DistComm
    dist.init_process_group("gloo")
    comm = DistComm()
    rank, world = comm.rank, comm.world
    worst = 0.0
    for (M, N, K, k, split) in [(96, 264, 136, 3, 0), (96, 264, 136, 3, 1), (64, 128, 64, 4, 0), (64, 64, 128, 4, 1)]:
        c = inputs.linear_case(M, N, K, w_std=0.1)
        W = torch.from_numpy(np.asarray(c["w"], dtype=np.float64))
        lay = ShardLayout(N, K, k, split, world)
        shard = lay.shard_of(W, rank)
        # this rank's tokens (rows rank::world of the batch), gradients by the oracle
        rows = np.arange(rank, M, world)
        z, _ = oracle.linear_fwd(c["x"][rows], c["w"], None, 0, k, split)
        _, dW_r, _ = oracle.linear_bwd(c["dy"][rows], c["x"][rows], c["w"], z, 0, k, split)
        dW_r = torch.from_numpy(np.ascontiguousarray(dW_r))
        stage = torch.zeros(lay.stage_elems, dtype=torch.float64)
        gstage = torch.zeros(lay.stage_elems, dtype=torch.float64)
        gshard = torch.zeros(lay.shard_total, dtype=torch.float64)
        for s, (b, e, elems, n, off, ld) in enumerate(lay.slices):
            comm.all_gather_slice(stage, shard, off, n)
            got = stage[:elems].reshape(-1, ld)
            assert torch.equal(got, lay.slice_matrix(W, s)), "gathered slice differs from W's slice"
            gstage.zero_()
            gstage[:elems] = lay.slice_matrix(dW_r, s).contiguous().reshape(-1)
            comm.reduce_scatter_slice(gshard, off, n, gstage)
        # data-parallel identity: the reduce-scattered sum is this rank's shard of the full-batch gradient
        z, _ = oracle.linear_fwd(c["x"], c["w"], None, 0, k, split)
        _, dW, _ = oracle.linear_bwd(c["dy"], c["x"], c["w"], z, 0, k, split)
        want = lay.shard_of(torch.from_numpy(np.ascontiguousarray(dW)), rank)
        err = float((gshard - want).abs().max() / want.abs().max())
        worst = max(worst, err)
    dist.barrier()
    print(json.dumps({"rank": rank, "world": world, "worst": worst}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_gather_and_reduce_scatter_by_slice():
    import json
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29741", OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-3000:]
    for o, _ in outs:
        line = json.loads(o.strip().splitlines()[-1])
        assert line["world"] == 2 and line["worst"] < 1e-12
