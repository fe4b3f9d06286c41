"""Parity at the full sizes of the workload configurations, in the launch configuration bench.py times.

The fp64 oracle cannot compute a 16384 x 8192 x 8192 layer in seconds, so every output is checked
 (a) on sampled rows / columns that the oracle computes one by one (first and last, tile and slice
     boundaries, random ones), with the same slicing as the GPU call, and
 (b) through matrix-vector identities that involve every output element (Y r = X (W^T r), ...),
     evaluated in fp64 with a library mat-vec,
and every concatenated output additionally byte for byte against the GPU's own k = 1 result.
In the default order of an all-slices call even the summed output must have the k = 1 bits when the
slice length is a multiple of the 64-element k-block (all workload configurations).
"""
import functools

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2209_13258_b200 import inputs  # noqa: E402
from util import assert_close, to_dev, to_f64  # noqa: E402

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)


@pytest.fixture(scope="module")
def P():
    import paper_2209_13258_b200 as pkg
    pkg.lib()
    return pkg


def _bits(t):
    return t.contiguous().view(torch.int32 if t.dtype == torch.float32 else torch.int16)


@functools.lru_cache(maxsize=1)
def _case(M, N, K, w_std, layer):
    return inputs.linear_case(M, N, K, w_std=w_std, layer=layer)


def run(P, c, k, split, flags=0):
    """fwd + bwd (dX, bf16 dW, db) through the C ABI on NaN-prefilled outputs."""
    M, N, K = c["M"], c["N"], c["K"]
    x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
    nan = float("nan")
    out = torch.full((M, N), nan, dtype=torch.bfloat16, device="cuda")
    dx = torch.full((M, K), nan, dtype=torch.bfloat16, device="cuda")
    dw = torch.full((N * K,), nan, dtype=torch.bfloat16, device="cuda")
    db = torch.full((N,), nan, dtype=torch.float32, device="cuda")
    _, n1 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, 0, P.OP_LINEAR_FWD, flags)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, 0, P.OP_LINEAR_BWD, flags)
    ws = P.new_workspace(max(n1, n2))
    P.osdp_split_linear_fwd(x, wf, c["w_offset"], None, M, N, K, k, split, 0, out, None, ws, check=True, flags=flags)
    P.osdp_split_linear_bwd(dy, x, wf, c["w_offset"], None, M, N, K, k, split, 0, dx, dw, c["w_offset"], P.DTYPE_BF16,
                            flags, db, ws, check=True)
    assert P.osdp_read_device_status(ws) == (0, 0)
    return {"y": out, "dx": dx, "dw": dw.view(N, K), "db": db, "x": x, "dy": dy,
            "w": wf[c["w_offset"]:c["w_offset"] + N * K].view(N, K), "staging": max(n1, n2)}


def _sample(n, marks, rng, extra=4):
    idx = {0, n - 1}
    for b in marks:
        for d in (-1, 0):
            if 0 <= b + d < n:
                idx.add(b + d)
    idx.update(int(v) for v in rng.integers(0, n, extra))
    return np.array(sorted(idx))


def check_sampled(P, c, g, k, split, seed, outputs=("y", "dx", "dw", "db")):
    """Sampled token rows of Y / dX and sampled output features of dW / db against the oracle."""
    M, N, K = c["M"], c["N"], c["K"]
    rng = np.random.default_rng(seed)
    D = N if split == 0 else K
    L = P.osdp_slice_range(D, k, 0)[2]
    bounds = list(range(L, D, L))
    bounds = bounds[:2] + bounds[-1:]                      # a few slice boundaries, not all 31
    if "y" in outputs or "dx" in outputs:
        rows = _sample(M, [128, 256, M // 2], rng)
        xs, dys = c["x"][rows], c["dy"][rows]
        idx = torch.from_numpy(rows).cuda()
        if "y" in outputs:
            _, y = oracle.linear_fwd(xs, c["w"], None, 0, k, split)
            assert_close(to_f64(g["y"][idx]), y, "Y rows")
        if "dx" in outputs:
            dX, _, _ = oracle.linear_bwd(dys, xs, c["w"], None, 0, k, split)
            assert_close(to_f64(g["dx"][idx]), dX, "dX rows")
    if "dw" in outputs or "db" in outputs:
        ncols = _sample(N, bounds if split == 0 else [256, 512], rng, extra=3)
        dy_sub = np.ascontiguousarray(c["dy"][:, ncols])
        _, dW, db = oracle.linear_bwd(dy_sub, c["x"], np.ascontiguousarray(c["w"][ncols]), None, 0)
        nidx = torch.from_numpy(ncols).cuda()
        if "dw" in outputs:
            assert_close(to_f64(g["dw"][nidx]), dW, "dW rows")
        if "db" in outputs:
            assert_close(to_f64(g["db"][nidx]), db, "db")


def check_identities(g, seed, outputs=("y", "dx", "dw")):
    """Y r = X (W^T r), dX r = dY (W r), r^T dW = (dY r)^T X over every element, fp64 mat-vecs on the device.
    Each GPU element carries one bf16 rounding (2^-9 relative), so a random combination of n of them is
    off by about 2^-9 * rms * sqrt(n); eight times that is allowed."""
    gen = torch.Generator(device="cuda").manual_seed(seed)
    N, K = g["w"].shape
    rN = torch.randn(N, generator=gen, device="cuda", dtype=torch.float64)
    rK = torch.randn(K, generator=gen, device="cuda", dtype=torch.float64)
    W = g["w"].double()

    def close(a, b, out, n, name):
        rms = float(out.pow(2).mean().sqrt())
        err = float((a - b).abs().max())
        assert err <= 8 * 2.0 ** -9 * rms * n ** 0.5, "%s identity: %.3e" % (name, err)

    if "y" in outputs:
        Y = g["y"].double()
        assert bool(torch.isfinite(Y).all()), "Y has unwritten elements"
        close(Y @ rN, g["x"].double() @ (W.T @ rN), Y, N, "Y")
        del Y
    if "dx" in outputs:
        dX = g["dx"].double()
        assert bool(torch.isfinite(dX).all()), "dX has unwritten elements"
        close(dX @ rK, g["dy"].double() @ (W @ rK), dX, K, "dX")
        del dX
    if "dw" in outputs:
        dW = g["dw"].double()
        assert bool(torch.isfinite(dW).all()), "dW has unwritten elements"
        close(rN @ dW, (g["dy"].double() @ rN) @ g["x"].double(), dW, N, "dW")


def assert_same_bits(g, g1, names, what):
    for name in names:
        assert torch.equal(_bits(g[name]), _bits(g1[name])), "%s: %s differs from k = 1" % (what, name)


# ---------------------------------------------------------------------------------------------
# split sweep: M = 16384, N = K = 8192, k in {1, 2, 4, 8, 16, 32} x {output, reduction}

SWEEP = (16384, 8192, 8192, 0.02, 20)
_k1 = {}


def _unsplit(P, key):
    """The GPU's own k = 1 result for a shape, computed and checked once per module."""
    if key not in _k1:
        _k1.clear()                                # one full-size result resident at a time
        c = _case(*key)
        g = run(P, c, 1, 0)
        check_sampled(P, c, g, 1, 0, seed=key[4])
        check_identities(g, seed=key[4])
        _k1[key] = g
    return _k1[key]


def test_sweep_shape_unsplit(P):
    _unsplit(P, SWEEP)


@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("k", [2, 4, 8, 16, 32])
def test_sweep_shape_all_k_default_order(P, k, split):
    c = _case(*SWEEP)
    g1 = _unsplit(P, SWEEP)
    g = run(P, c, k, split)
    # every output, the summed one included, has the unsplit result's bits
    assert_same_bits(g, g1, ("y", "dx", "dw", "db"), "k=%d split=%d" % (k, split))
    # and the oracle with the same slicing agrees on the sampled rows of the summed output
    check_sampled(P, c, g, k, split, seed=100 + k, outputs=("dx",) if split == 0 else ("y",))
    assert g["staging"] == g1["staging"]           # no carry: the same scratch as the unsplit layer


@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("k", [2, 8, 16, 32])
def test_sweep_shape_slice_major_order(P, k, split):
    # the operator swept once per slice, fp32 carry through the workspace; k = 16 and 32 take the
    # one-launch-per-slice path of the summed GEMM (slices of 512 and 256)
    c = _case(*SWEEP)
    g1 = _unsplit(P, SWEEP)
    g = run(P, c, k, split, flags=P.FLAG_SLICE_MAJOR)
    concat = ("y", "dw", "db") if split == 0 else ("dx", "dw", "db")
    summed = "dx" if split == 0 else "y"
    assert_same_bits(g, g1, concat, "slice-major k=%d split=%d" % (k, split))
    check_sampled(P, c, g, k, split, seed=200 + k, outputs=(summed,))
    check_identities(g, seed=200 + k, outputs=(summed,))
    rows, cols = (c["M"], c["K"]) if split == 0 else (c["M"], c["N"])
    carry = rows * cols * 4                                     # the fp32 running sum, and nothing else, is added
    assert carry + 256 <= g["staging"] <= carry + g1["staging"]


# ---------------------------------------------------------------------------------------------
# wide-layer stress: hidden 8192, ffn 32768, 8192 tokens, k = 8: both linears along the output
# dimension and both along the reduction dimension

@pytest.mark.parametrize("NK", [(32768, 8192), (8192, 32768)])
def test_wide_layer_both_split_dims_k8(P, NK):
    N, K = NK
    key = (8192, N, K, 0.01, 40 + N // 32768)
    c = _case(*key)
    g1 = _unsplit(P, key)
    for split in (0, 1):
        g = run(P, c, 8, split)
        assert_same_bits(g, g1, ("y", "dx", "dw", "db"), "wide layer split=%d" % split)
        check_sampled(P, c, g, 8, split, seed=300 + split, outputs=("dx",) if split == 0 else ("y",))
        gs = run(P, c, 8, split, flags=P.FLAG_SLICE_MAJOR)
        summed = "dx" if split == 0 else "y"
        assert_same_bits(gs, g1, [n for n in ("y", "dx", "dw", "db") if n != summed], "wide layer slice-major")
        check_sampled(P, c, gs, 8, split, seed=310 + split, outputs=(summed,))
        check_identities(gs, seed=310 + split, outputs=(summed,))
        del g, gs


# ---------------------------------------------------------------------------------------------
# decoder-stack linears (hidden 2048, 8192 tokens), k = 4: the projection and the second MLP linear
# split along the reduction dimension (the others along the output dimension are covered elsewhere)

@pytest.mark.parametrize("NK", [(2048, 2048), (2048, 8192)])
def test_decoder_linears_reduction_split_k4(P, NK):
    N, K = NK
    key = (8192, N, K, 0.02, 50 + K // 8192)
    c = _case(*key)
    g1 = _unsplit(P, key)
    for flags in (0, P.FLAG_SLICE_MAJOR):
        g = run(P, c, 4, 1, flags=flags)
        assert_same_bits(g, g1, ("dx", "dw", "db") + (("y",) if flags == 0 else ()), "decoder linear RED")
        check_sampled(P, c, g, 4, 1, seed=400 + flags, outputs=("y",))
        check_identities(g, seed=400 + flags, outputs=("y",))


# ---------------------------------------------------------------------------------------------
# fp8 operands at the sweep size, k = 16 (slices of 512), both orders

def test_fp8_sweep_shape_k16(P):
    M, N, K, k = 16384, 8192, 8192, 16
    c = inputs.linear_case_e4m3(M, N, K, w_std=0.02, layer=60)

    def dev8(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    x, dy, wf = dev8(c["x"]), dev8(c["dy"]), dev8(c["w_flat"])
    off = c["w_offset"]
    rng = np.random.default_rng(60)
    rows = _sample(M, [128, 256, M // 2], rng)
    X = oracle.e4m3_to_f64(c["x"][rows]) * c["sx"]
    DY = oracle.e4m3_to_f64(c["dy"][rows]) * c["sdy"]
    W = oracle.e4m3_to_f64(c["w"]) * c["sw"]
    idx = torch.from_numpy(rows).cuda()
    res = {}
    for kk, split, flags in ((1, 0, 0), (k, 0, 0), (k, 1, 0), (k, 0, P.FLAG_SLICE_MAJOR), (k, 1, P.FLAG_SLICE_MAJOR)):
        out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        dx = torch.full((M, K), float("nan"), dtype=torch.bfloat16, device="cuda")
        dw = torch.full((wf.numel(),), float("nan"), dtype=torch.bfloat16, device="cuda")
        _, n1 = P.osdp_split_linear_workspace_bytes(M, N, K, kk, split, 0, P.OP_LINEAR_FWD, flags)
        _, n2 = P.osdp_split_linear_workspace_bytes(M, N, K, kk, split, 0, P.OP_LINEAR_BWD, flags)
        ws = P.new_workspace(max(n1, n2))
        P.osdp_split_linear_fwd_f8(x, wf, off, c["sx"] * c["sw"], None, M, N, K, kk, split, 0, out, None, ws,
                                   check=True, flags=flags)
        P.osdp_split_linear_bwd_f8(dy, x, wf, off, c["sdy"] * c["sw"], c["sdy"] * c["sx"], M, N, K, kk, split, dx, dw,
                                   off, P.DTYPE_BF16, flags, ws, check=True)
        assert P.osdp_read_device_status(ws) == (0, 0)
        g = {"y": out, "dx": dx, "dw": dw[off:off + N * K].view(N, K)}
        _, y = oracle.linear_fwd(X, W, None, 0, kk, split)
        dX, _, _ = oracle.linear_bwd(DY, X, W, None, 0, kk, split)
        assert_close(to_f64(out[idx]), y, "Y rows")
        assert_close(to_f64(dx[idx]), dX, "dX rows")
        assert bool(torch.isfinite(g["dw"].float()).all())
        if kk == 1:
            res = g
            ncols = _sample(N, [256, 512], rng, extra=2)
            DYc = oracle.e4m3_to_f64(np.ascontiguousarray(c["dy"][:, ncols])) * c["sdy"]
            Xall = oracle.e4m3_to_f64(c["x"]) * c["sx"]
            _, dW, _ = oracle.linear_bwd(DYc, Xall, np.ascontiguousarray(W[ncols]), None, 0)
            assert_close(to_f64(g["dw"][torch.from_numpy(ncols).cuda()]), dW, "dW rows")
        else:
            same = ("y", "dx", "dw") if flags == 0 else (("y", "dw") if split == 0 else ("dx", "dw"))
            assert_same_bits(g, res, same, "fp8 k=%d split=%d flags=%d" % (kk, split, flags))
