"""GPU parity of the fp8 (e4m3) operand variant: the split linear layer on tcgen05.mma.kind::f8f6f4 against
the fp64 oracle evaluated on the exactly widened e4m3 inputs and the per-tensor scales."""
import numpy as np
import pytest

import oracle
from paper_2209_13258_b200 import inputs
from util import Guarded, assert_close, to_f64

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2209_13258_b200 as pkg
    pkg.lib()
    return pkg


def dev8(bits):
    return torch.from_numpy(np.ascontiguousarray(bits)).cuda()


def bits(t):
    return t.view(torch.int32 if t.dtype == torch.float32 else torch.int16)


def run_f8(P, c, k, split, act=0, dw_fp32=True, flags=0):
    M, N, K, off = c["M"], c["N"], c["K"], c["w_offset"]
    x, dy, wf = dev8(c["x"]), dev8(c["dy"]), dev8(c["w_flat"])
    b = torch.from_numpy(c["bias"]).cuda()
    out, z, dx = Guarded((M, N), torch.bfloat16), Guarded((M, N), torch.bfloat16), Guarded((M, K), torch.bfloat16)
    dwf = Guarded((wf.numel(),), torch.float32 if dw_fp32 else torch.bfloat16)
    _, n1 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, act, P.OP_LINEAR_FWD, flags)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, 0, P.OP_LINEAR_BWD, flags)
    ws = P.new_workspace(max(n1, n2))
    zs = z.t if act else None
    P.osdp_split_linear_fwd_f8(x, wf, off, c["sx"] * c["sw"], b, M, N, K, k, split, act, out.t, zs, ws, check=True,
                               flags=flags)
    P.osdp_split_linear_bwd_f8(dy, x, wf, off, c["sdy"] * c["sw"], c["sdy"] * c["sx"], M, N, K, k, split, dx.t, dwf.t,
                               off, P.DTYPE_FP32 if dw_fp32 else P.DTYPE_BF16, flags, ws, check=True)
    rc, st = P.osdp_read_device_status(ws)
    assert rc == 0 and st == 0
    for g in (out, dx, dwf) + ((z,) if act else ()):
        g.check()
    dw = dwf.t[off:off + N * K].view(N, K)
    assert bool(torch.isnan(dwf.t[:off]).all()) and bool(torch.isnan(dwf.t[off + N * K:]).all())
    return {"y": out.t, "z": z.t if act else None, "dx": dx.t, "dw": dw}


def oracle_f8(c, act, k=1, split=None):
    X = oracle.e4m3_to_f64(c["x"]) * c["sx"]
    W = oracle.e4m3_to_f64(c["w"]) * c["sw"]
    DY = oracle.e4m3_to_f64(c["dy"]) * c["sdy"]
    z, y = oracle.linear_fwd(X, W, c["bias"], act, k, split)
    dX, dW, _ = oracle.linear_bwd(DY, X, W, None, 0, k, split)     # the fp8 backward has no activation
    return {"y": y, "z": z, "dx": dX, "dw": dW}


def compare(g, o, act):
    assert_close(to_f64(g["y"]), o["y"], "Y")
    if act:
        assert_close(to_f64(g["z"]), o["z"], "Z")
    assert_close(to_f64(g["dx"]), o["dx"], "dX")
    assert_close(to_f64(g["dw"]), o["dw"], "dW")


SHAPES = [(256, 2048, 512), (200, 272, 144), (300, 528, 336), (77, 1024, 80), (513, 16, 528), (1000, 1296, 2064)]


@pytest.mark.parametrize("shape", SHAPES)
def test_fp8_unsplit_matches_oracle(P, shape):
    M, N, K = shape
    c = inputs.linear_case_e4m3(M, N, K, w_std=0.05, bias_std=0.3, w_offset=48, flat_pad=16, layer=3)
    for act in (0, 1):
        compare(run_f8(P, c, 1, 0, act), oracle_f8(c, act), act)


@pytest.mark.parametrize("shape,k", [((256, 2048, 512), 4), ((300, 512, 256), 2), ((384, 1024, 1024), 8),
                                     ((200, 272, 144), 3), ((640, 2064, 1296), 3)])
@pytest.mark.parametrize("split", [0, 1])
def test_fp8_split_matches_oracle_and_unsplit_bits(P, shape, k, split):
    M, N, K = shape
    D = N if split == 0 else K
    rc, b, e = P.osdp_slice_range(D, k, 0)
    if rc != 0 or (e - b) % 16:
        # slice length not a multiple of 16: the call must say so rather than run
        c = inputs.linear_case_e4m3(M, N, K)
        x, wf = dev8(c["x"]), dev8(c["w_flat"])
        out = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        ws = P.new_workspace(1 << 24)
        assert P.osdp_split_linear_fwd_f8(x, wf, 0, 1.0, None, M, N, K, k, split, 0, out, None, ws) in (3, 4)
        return
    c = inputs.linear_case_e4m3(M, N, K, w_std=0.05, bias_std=0.3, w_offset=32, flat_pad=16, layer=4)
    g = run_f8(P, c, k, split, act=1)
    compare(g, oracle_f8(c, 1, k, split), 1)
    g1 = run_f8(P, c, 1, split, act=1)
    for name in (("y", "z", "dw") if split == 0 else ("dx", "dw")):     # concatenated outputs: same bits as k = 1
        assert torch.equal(bits(g[name]), bits(g1[name])), name


def test_fp8_benchmark_shape_sampled(P):
    """A tile-spanning shape through the 256-wide and 512-wide pair tiles, checked on sampled rows / columns."""
    M, N, K = 4096, 4096, 4096
    c = inputs.linear_case_e4m3(M, N, K, w_std=0.02, layer=5)
    g = run_f8(P, c, 4, 0, dw_fp32=False)
    rows = np.array([0, 1, 127, 128, 255, 256, 2047, 2048, 4095])
    X = oracle.e4m3_to_f64(c["x"]) * c["sx"]
    W = oracle.e4m3_to_f64(c["w"]) * c["sw"]
    DY = oracle.e4m3_to_f64(c["dy"]) * c["sdy"]
    assert_close(to_f64(g["y"][rows]), X[rows] @ W.T, "Y rows")
    assert_close(to_f64(g["dx"][rows]), DY[rows] @ W, "dX rows")
    assert_close(to_f64(g["dw"][rows]), DY[:, rows].T @ X, "dW rows")
    assert_close(to_f64(g["y"][:, rows]), X @ W[rows].T, "Y columns")


def test_fp8_argument_errors(P):
    M, N, K = 128, 256, 128
    x = torch.zeros(M, K, dtype=torch.uint8, device="cuda")
    w = torch.zeros(N * K + 64, dtype=torch.uint8, device="cuda")
    out = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    ws = P.new_workspace(1 << 22)
    f = P.osdp_split_linear_fwd_f8
    assert f(x, w, 8, 1.0, None, M, N, K, 1, 0, 0, out, None, ws) == 4              # offset not a multiple of 16
    assert f(x, w, 0, 1.0, None, M, N - 8, K, 1, 0, 0, out, None, ws) == 4          # N not a multiple of 16
    assert f(x, w, 0, float("inf"), None, M, N, K, 1, 0, 0, out, None, ws) == 6
    assert f(x, None, 0, 1.0, None, M, N, K, 1, 0, 0, out, None, ws) == 1
    assert f(x, w, 0, 1.0, None, M, N, K, 1, 0, 0, out, None, ws) == 0


@pytest.mark.parametrize("flags", [2, 8])
@pytest.mark.parametrize("split", [0, 1])
def test_fp8_summed_outputs_with_bf16_running_sum_and_paired_slices(P, flags, split):
    """The carry modes of the bf16 path apply unchanged to fp8 operands (flag 2: bf16 running sum, 8: pairs)."""
    M, N, K, k = 384, 1024, 1024, 4
    c = inputs.linear_case_e4m3(M, N, K, w_std=0.05, w_offset=16, flat_pad=16, layer=8)
    g = run_f8(P, c, k, split, act=0, flags=flags)
    o = oracle_f8(c, 0, k, split)
    tol = 3e-2 * (2 * k) ** 0.5 if flags == 2 else 3e-2     # the bf16 running sum rounds once more per slice
    assert_close(to_f64(g["y"]), o["y"], "Y", abs_tol=tol)
    assert_close(to_f64(g["dx"]), o["dx"], "dX", abs_tol=tol)
    assert_close(to_f64(g["dw"]), o["dw"], "dW")


@pytest.mark.parametrize("chunk", range(2))
def test_fp8_random_shapes_against_oracle(P, chunk):
    import random
    rng = random.Random(5000 + chunk)
    done = 0
    while done < 10:
        M = rng.choice([64, 130, 256, 300, 513, 1000])
        N, K = 16 * rng.randint(1, 110), 16 * rng.randint(1, 110)
        k, split = rng.choice([1, 2, 3, 4, 8]), rng.choice([0, 1])
        rc, b, e = P.osdp_slice_range(N if split == 0 else K, k, 0)
        if rc != 0 or (k > 1 and (e - b) % 16):
            continue
        act = rng.choice([0, 1])
        c = inputs.linear_case_e4m3(M, N, K, w_std=0.05, bias_std=0.2, w_offset=16 * rng.randint(0, 9), flat_pad=16,
                                    layer=70 + done)
        compare(run_f8(P, c, k, split, act), oracle_f8(c, act, k, split), act)
        done += 1
