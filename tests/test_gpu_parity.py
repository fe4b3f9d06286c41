"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded bf16 inputs.  Tolerances: relative Frobenius <= 5e-3 and max abs <= 3e-2 (see util.py);
concatenated outputs of a split must be bit-identical to the GPU's own k = 1 result."""
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
    pkg.lib()   # fails loudly if the extension is missing: there is no fallback
    return pkg


def run_linear(P, c, k, split, act=0, dw_fp32=True, use_bias=True, accumulate=0, dw_init=None, per_slice=False,
               flags=0):
    """fwd + bwd through the C ABI; returns dict of cuda tensors."""
    M, N, K, off = c["M"], c["N"], c["K"], c["w_offset"]
    x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
    b = to_dev(c["bias"]) if use_bias else None
    out, z, dx = Guarded((M, N), torch.bfloat16), Guarded((M, N), torch.bfloat16), Guarded((M, K), torch.bfloat16)
    dwf = Guarded((wf.numel(),), torch.float32 if dw_fp32 else torch.bfloat16)
    if dw_init is not None:
        dwf.t.copy_(dw_init)
    db = Guarded((N,), torch.float32)
    qflags = flags | (P.FLAG_SLICE_MAJOR if per_slice else 0)     # one slice per call carries the sum in ws
    rc, n1 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, act, P.OP_LINEAR_FWD, qflags)
    rc2, n2 = P.osdp_split_linear_workspace_bytes(M, N, K, k, split, act, P.OP_LINEAR_BWD, qflags)
    assert rc == 0 and rc2 == 0
    ws = P.new_workspace(max(n1, n2))
    accumulate = accumulate | flags
    zs = z.t if act else None
    dt = P.DTYPE_FP32 if dw_fp32 else P.DTYPE_BF16
    if per_slice:
        for s in range(max(k, 1)):
            P.osdp_split_linear_fwd_slice(x, wf, off, b, M, N, K, k, split, act, s, out.t, zs, ws, check=True,
                                          flags=flags)
        for s in range(max(k, 1)):
            P.osdp_split_linear_bwd_slice(dy, x, wf, off, zs, M, N, K, k, split, act, s, dx.t, dwf.t, off, dt,
                                          accumulate, db.t, ws, check=True)
    else:
        P.osdp_split_linear_fwd(x, wf, off, b, M, N, K, k, split, act, out.t, zs, ws, check=True, flags=flags)
        P.osdp_split_linear_bwd(dy, x, wf, off, zs, M, N, K, k, split, act, dx.t, dwf.t, off, dt, accumulate, db.t,
                                ws, check=True)
    rc, st = P.osdp_read_device_status(ws)
    assert rc == 0 and st == 0
    for g in (out, dx, dwf, db) + ((z,) if act else ()):
        g.check()
    dw = dwf.t[off:off + N * K].view(N, K)
    # nothing outside W's window of the flat gradient buffer may be written
    if dw_init is None:
        assert bool(torch.isnan(dwf.t[:off]).all()) and bool(torch.isnan(dwf.t[off + N * K:]).all())
    return {"y": out.t, "z": z.t if act else None, "dx": dx.t, "dw": dw, "db": db.t}


def oracle_linear(c, act, k=1, split=None, use_bias=True):
    b = c["bias"] if use_bias else None
    z, y = oracle.linear_fwd(c["x"], c["w"], b, act, k, split)
    dX, dW, db = oracle.linear_bwd(c["dy"], c["x"], c["w"], z, act, k, split)
    return {"y": y, "z": z, "dx": dX, "dw": dW, "db": db}


def compare(g, o, act, dw_fp32=True, y_abs_tol=3e-2, dx_abs_tol=3e-2):
    assert_close(to_f64(g["y"]), o["y"], "Y", abs_tol=y_abs_tol)
    if act:
        assert_close(to_f64(g["z"]), o["z"], "Z")
    assert_close(to_f64(g["dx"]), o["dx"], "dX", abs_tol=dx_abs_tol)
    assert_close(to_f64(g["dw"]), o["dw"], "dW")
    assert_close(to_f64(g["db"]), o["db"], "db")


# ---------------------------------------------------------------------------------------------
# config 1: X [256,512], W [2048,512] ~N(0,0.02), bias zeros, k=4 along the output dim

def test_config1_exact_shapes(P):
    c = inputs.linear_case(256, 2048, 512)
    g = run_linear(P, c, 4, P.SPLIT_OUT)
    o = oracle_linear(c, 0, 4, oracle.SPLIT_OUT)
    compare(g, o, 0)
    # fp32 dW, fp32 db: the literal bounds hold with a wide margin
    relf, maxabs = assert_close(to_f64(g["dw"]), o["dw"], "dW fp32", relf_tol=1e-5)
    assert maxabs <= 3e-2
    # bit identity of the concatenated outputs with the GPU's own k = 1 result
    g1 = run_linear(P, c, 1, P.SPLIT_OUT)
    for name in ("y", "dw", "db"):
        assert torch.equal(g[name].view(torch.int32 if g[name].dtype == torch.float32 else torch.int16),
                           g1[name].view(torch.int32 if g1[name].dtype == torch.float32 else torch.int16)), name


def test_config1_with_bias_and_offset(P):
    c = inputs.linear_case(256, 2048, 512, bias_std=0.02, w_offset=4096 + 8, flat_pad=24)
    for split in (P.SPLIT_OUT, P.SPLIT_RED):
        g = run_linear(P, c, 4, split)
        compare(g, oracle_linear(c, 0, 4, split), 0)


# ---------------------------------------------------------------------------------------------
# ragged shapes spanning several tiles, every split / activation / dtype combination

RAGGED = [(200, 264, 136), (300, 520, 328), (77, 1032, 72), (513, 8, 520), (130, 392, 264)]


@pytest.mark.parametrize("shape", RAGGED)
@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("order", ["tile", "slice_major"])
def test_ragged_shapes_all_k(P, shape, split, order):
    # both orders of an all-slices call: slices inside a tile (sum kept in tensor memory) and
    # slice-major (sum carried through the workspace)
    M, N, K = shape
    c = inputs.linear_case(M, N, K, w_std=0.1, bias_std=0.3, w_offset=72, flat_pad=8, layer=2)
    D = N if split == 0 else K
    for k in (1, 2, 3, 5, 8, D // 8):
        if k < 1 or P.osdp_slice_range(D, k, 0)[0] != 0:
            continue
        g = run_linear(P, c, k, split, flags=P.FLAG_SLICE_MAJOR if order == "slice_major" else 0)
        compare(g, oracle_linear(c, 0, k, split), 0)


@pytest.mark.parametrize("act", [1, 2])
@pytest.mark.parametrize("split,k", [(0, 1), (0, 3), (1, 4), (0, 6)])
def test_activation_forward_backward(P, act, split, k):
    c = inputs.linear_case(260, 528, 200, w_std=0.08, bias_std=0.3, layer=4)
    g = run_linear(P, c, k, split, act=act)
    o = oracle_linear(c, act, k, split)
    compare(g, o, act)


def test_bf16_dw_and_accumulate(P):
    c = inputs.linear_case(384, 512, 256, w_std=0.1, layer=5)
    o = oracle_linear(c, 0)
    g = run_linear(P, c, 2, P.SPLIT_OUT, dw_fp32=False)
    assert g["dw"].dtype == torch.bfloat16
    assert_close(to_f64(g["dw"]), o["dw"], "dW bf16")
    # accumulate: dW += ..., starting from a known fp32 buffer
    init = torch.arange(c["w_flat"].size, dtype=torch.float32, device="cuda") * 1e-3
    for split in (0, 1):
        g = run_linear(P, c, 2, split, accumulate=1, dw_init=init)
        want = o["dw"] + to_f64(init)[c["w_offset"]:c["w_offset"] + 512 * 256].reshape(512, 256)
        assert_close(to_f64(g["dw"]), want, "dW accumulate", relf_tol=1e-5)


# ---------------------------------------------------------------------------------------------
# summed output kept in bf16 in the output buffer itself (no fp32 carry): one more rounding per slice

@pytest.mark.parametrize("shape", [(300, 520, 328), (1024, 2048, 1024)])
@pytest.mark.parametrize("split", [0, 1])
def test_bf16_running_sum(P, shape, split):
    M, N, K = shape
    c = inputs.linear_case(M, N, K, w_std=0.05, bias_std=0.3, layer=12)
    o = oracle_linear(c, 0)
    for k in (2, 3, 8):
        if P.osdp_slice_range(N if split == 0 else K, k, 0)[0] != 0:
            continue
        g = run_linear(P, c, k, split, flags=P.FLAG_CARRY_BF16)
        # The summed output is rounded to bf16 once per slice (partial and running sum): its worst-case
        # element error grows like sqrt(2k) roundings; the relative Frobenius bound 5e-3 still holds.
        loose = 3e-2 * (2 * k) ** 0.5
        compare(g, o, 0, y_abs_tol=loose if split == 1 else 3e-2, dx_abs_tol=loose if split == 0 else 3e-2)
        gs = run_linear(P, c, k, split, flags=P.FLAG_CARRY_BF16, per_slice=True)
        for name in ("y", "dx", "dw", "db"):
            assert torch.equal(_bits(g[name]), _bits(gs[name])), name
        # the concatenated outputs do not depend on how the summed one is carried
        g32 = run_linear(P, c, k, split)
        for name in (("y", "dw", "db") if split == 0 else ("dx", "dw", "db")):
            assert torch.equal(_bits(g[name]), _bits(g32[name])), name


# ---------------------------------------------------------------------------------------------
# adjacent slices accumulated in pairs (two slices live): exact fp32, half as many carried boundaries

@pytest.mark.parametrize("shape", [(300, 520, 328), (1024, 2048, 1024), (2100, 2560, 2304)])
@pytest.mark.parametrize("split", [0, 1])
def test_paired_slices(P, shape, split):
    M, N, K = shape
    c = inputs.linear_case(M, N, K, w_std=0.05, bias_std=0.3, layer=16)
    o = oracle_linear(c, 0)
    for k in (2, 3, 5, 8):
        if P.osdp_slice_range(N if split == 0 else K, k, 0)[0] != 0:
            continue
        g = run_linear(P, c, k, split, flags=P.FLAG_PAIR_SLICES)
        compare(g, o, 0)
        # concatenated outputs are untouched by the pairing
        plain = run_linear(P, c, k, split)
        for name in (("y", "dw", "db") if split == 0 else ("dx", "dw", "db")):
            assert torch.equal(_bits(g[name]), _bits(plain[name])), name
    # with an activation the forward's summed output still pairs (bias and activation after the last pair)
    if split == 1:
        ga = run_linear(P, c, 4, split, act=1, flags=0)
        oa = oracle_linear(c, 1, 4, split)
        compare(ga, oa, 1)


# ---------------------------------------------------------------------------------------------
# bit identity, per-slice calls, determinism

def _bits(t):
    return t.contiguous().view(torch.int32 if t.dtype == torch.float32 else torch.int16)


@pytest.mark.parametrize("shape", [(512, 2048, 1024), (300, 520, 328)])
def test_bit_identity_of_concatenated_outputs(P, shape):
    M, N, K = shape
    c = inputs.linear_case(M, N, K, bias_std=0.1, layer=6)
    g1 = run_linear(P, c, 1, 0, act=1)
    for k in (2, 4, 8):
        g = run_linear(P, c, k, P.SPLIT_OUT, act=1)
        for name in ("y", "z"):
            assert torch.equal(_bits(g[name]), _bits(g1[name])), (name, k)
    # without activation the backward's concatenated outputs are bit-identical too
    g1 = run_linear(P, c, 1, 0)
    for k in (2, 4, 8):
        g = run_linear(P, c, k, P.SPLIT_OUT)
        for name in ("y", "dw", "db"):
            assert torch.equal(_bits(g[name]), _bits(g1[name])), (name, k)
        if P.osdp_slice_range(K, k, 0)[0] != 0:
            continue
        g = run_linear(P, c, k, P.SPLIT_RED)
        for name in ("dx", "dw", "db"):
            assert torch.equal(_bits(g[name]), _bits(g1[name])), (name, k)


@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("act", [0, 1])
def test_per_slice_calls_equal_whole_call(P, split, act):
    # one call per slice == one slice-major call over all slices, bit for bit; the default order of an
    # all-slices call gives the same concatenated outputs and a summed output equal up to fp32 rounding order
    c = inputs.linear_case(300, 520, 328, w_std=0.1, bias_std=0.2, layer=7)
    a = run_linear(P, c, 3, split, act=act, flags=P.FLAG_SLICE_MAJOR)
    b = run_linear(P, c, 3, split, act=act, per_slice=True)
    for name in ("y", "dx", "dw", "db"):
        assert torch.equal(_bits(a[name]), _bits(b[name])), name
    d = run_linear(P, c, 3, split, act=act)
    summed = "dx" if split == 0 else "y"
    if split == 1 and act:
        # the saved pre-activation is itself the summed output here, so the whole backward sees other bits
        for name in ("y", "dx", "dw", "db"):
            assert_close(to_f64(d[name]), to_f64(a[name]), name + " tile order vs slice-major", relf_tol=3e-3)
        return
    for name in (("y", "dw", "db") if split == 0 else ("dx", "dw", "db")):
        assert torch.equal(_bits(a[name]), _bits(d[name])), name
    assert_close(to_f64(d[summed]), to_f64(a[summed]), summed + " tile order vs slice-major", relf_tol=3e-3)


@pytest.mark.parametrize("shape", [(512, 2048, 1024), (2048, 4096, 4096)])
def test_summed_output_in_tensor_memory_is_bit_identical_to_unsplit(P, shape):
    # default order, slice length a multiple of the 64-element k-block: a tile meets exactly the k-blocks
    # of the unsplit GEMM in the same order, so even the summed output has the unsplit result's bits
    M, N, K = shape
    c = inputs.linear_case(M, N, K, bias_std=0.1, layer=19)
    g1 = run_linear(P, c, 1, 0)
    for k in (2, 4, 8, 16):
        for split in (0, 1):
            g = run_linear(P, c, k, split)
            for name in ("y", "dx", "dw", "db"):
                assert torch.equal(_bits(g[name]), _bits(g1[name])), (name, k, split)
    # and the workspace of such a call holds no carry
    _, n = P.osdp_split_linear_workspace_bytes(M, N, K, 8, 1, 0, P.OP_LINEAR_FWD)
    assert n == 256


def test_repeated_runs_are_bitwise_equal(P):
    c = inputs.linear_case(1024, 1024, 512, layer=8)
    ref = run_linear(P, c, 4, P.SPLIT_RED)
    for _ in range(5):
        g = run_linear(P, c, 4, P.SPLIT_RED)
        for name in ("y", "dx", "dw", "db"):
            assert torch.equal(_bits(g[name]), _bits(ref[name])), name


def test_maximum_split_and_tiny_shapes(P):
    # slices of length 8 (the minimum), and a 1-token batch
    c = inputs.linear_case(1, 64, 64, w_std=0.2, layer=9)
    for split in (0, 1):
        g = run_linear(P, c, 8, split)
        compare(g, oracle_linear(c, 0, 8, split), 0)
    c = inputs.linear_case(8, 8, 8, w_std=0.5, layer=10)
    compare(run_linear(P, c, 1, 0), oracle_linear(c, 0), 0)


# ---------------------------------------------------------------------------------------------
# config 2: transformer MLP block, hidden 1024, ffn 4096, tokens 8 x 512, split along ffn

def run_mlp(P, c, k, act=1, dw_fp32=True, flags=0, recompute=False):
    M, H, F = c["M"], c["hidden"], c["ffn"]
    x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
    b1, b2 = to_dev(c["b1"]), to_dev(c["b2"])
    out, z1, dx = Guarded((M, H), torch.bfloat16), Guarded((M, F), torch.bfloat16), Guarded((M, H), torch.bfloat16)
    dwf = Guarded((wf.numel(),), torch.float32 if dw_fp32 else torch.bfloat16)
    db1, db2 = Guarded((F,), torch.float32), Guarded((H,), torch.float32)
    _, n1 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, act, P.OP_MLP_FWD, flags)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, act, P.OP_MLP_BWD, flags)
    ws = P.new_workspace(max(n1, n2))
    P.osdp_split_mlp_fwd(x, wf, c["off_w1"], b1, c["off_w2"], b2, M, H, F, k, act, out.t, z1.t, ws, check=True,
                         flags=flags)
    if recompute:
        # activation checkpointing: the backward gets no saved activation and recomputes it per slice
        _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, act, P.OP_MLP_BWD, flags | P.FLAG_RECOMPUTE)
        ws = P.new_workspace(max(n1, n2))
        P.osdp_split_mlp_bwd(dy, x, wf, c["off_w1"], c["off_w2"], None, M, H, F, k, act, dx.t, dwf.t, c["off_w1"],
                             c["off_w2"], P.DTYPE_FP32 if dw_fp32 else P.DTYPE_BF16, flags | P.FLAG_RECOMPUTE,
                             db1.t, db2.t, ws, check=True, b1=b1)
    else:
        P.osdp_split_mlp_bwd(dy, x, wf, c["off_w1"], c["off_w2"], z1.t, M, H, F, k, act, dx.t, dwf.t, c["off_w1"],
                             c["off_w2"], P.DTYPE_FP32 if dw_fp32 else P.DTYPE_BF16, flags, db1.t, db2.t, ws,
                             check=True)
    rc, st = P.osdp_read_device_status(ws)
    assert rc == 0 and st == 0
    for g in (out, z1, dx, dwf, db1, db2):
        g.check()
    return {"y": out.t, "dx": dx.t, "dw1": dwf.t[c["off_w1"]:c["off_w1"] + F * H].view(F, H),
            "dw2": dwf.t[c["off_w2"]:c["off_w2"] + H * F].view(H, F), "db1": db1.t, "db2": db2.t,
            "staging": (n1, n2)}


def compare_mlp(g, o, summed_abs_tol=3e-2):
    names = ("y", "dx", "dw1", "db1", "dw2", "db2")
    for name, ref in zip(names, o):
        assert_close(to_f64(g[name]), ref, name, abs_tol=summed_abs_tol if name in ("y", "dx") else 3e-2)


@pytest.mark.parametrize("flags", [0, 2])
@pytest.mark.parametrize("k", [1, 2, 3, 5])
def test_mlp_small_ragged(P, k, flags):
    c = inputs.mlp_case(200, 264, 520, w_std=0.08, layer=11)
    g = run_mlp(P, c, k, flags=flags)
    _, y = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
    grads = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    compare_mlp(g, (y,) + tuple(grads), summed_abs_tol=3e-2 * (2 * k) ** 0.5 if flags else 3e-2)


@pytest.mark.parametrize("k", [1, 3, 4])
def test_mlp_backward_with_recomputation(P, k):
    c = inputs.mlp_case(300, 264, 520, w_std=0.08, layer=15)
    saved = run_mlp(P, c, k)
    recomputed = run_mlp(P, c, k, recompute=True)
    _, y = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
    grads = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    compare_mlp(recomputed, (y,) + tuple(grads))
    # The recomputed pre-activation has the same bits as the saved one, so everything derived from
    # it is bit-identical.  dW2 = dY^T act(Z1) is not: the recomputation applies the activation to
    # the unrounded pre-activation, exactly as the forward did, the saved path to its bf16 rounding.
    for name in ("dx", "dw1", "db1", "db2"):
        assert torch.equal(_bits(saved[name]), _bits(recomputed[name])), name
    assert_close(to_f64(recomputed["dw2"]), to_f64(saved["dw2"]), "dW2 saved vs recomputed")
    assert recomputed["staging"][0] > 0


def test_config2_mlp_block_all_k(P):
    c = inputs.mlp_case(8 * 512, 1024, 4096)
    _, y = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, None)
    grads = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, None)
    staging = {}
    for k in (1, 2, 4, 8):
        g = run_mlp(P, c, k)
        compare_mlp(g, (y,) + tuple(grads))
        staging[k] = g["staging"]
    # the slice-sized intermediates shrink as 1/k (the fp32 carry of the summed output does not)
    M, H = 4096, 1024
    carry = M * H * 4
    for k in (2, 4, 8):
        slice_part_1 = staging[1][0] - 256
        slice_part_k = staging[k][0] - 256 - carry
        assert abs(slice_part_k - slice_part_1 / k) <= 1024, (k, staging)


# ---------------------------------------------------------------------------------------------
# full-size shapes: sampled rows/columns against the oracle + matrix-vector identities over
# every output element (launch configuration = the one bench.py times)

def _sample_idx(n, boundaries, rng, extra=6):
    idx = {0, n - 1}
    for b in boundaries:
        for d in (-1, 0):
            if 0 <= b + d < n:
                idx.add(b + d)
    idx.update(int(v) for v in rng.integers(0, n, extra))
    return np.array(sorted(idx))


def check_large_linear(P, M, N, K, k, split, w_std, layer):
    c = inputs.linear_case(M, N, K, w_std=w_std, layer=layer)
    g = run_linear(P, c, k, split, dw_fp32=False, use_bias=False)
    rng = np.random.default_rng(layer)
    D = N if split == 0 else K
    L = P.osdp_slice_range(D, k, 0)[2]
    bounds = list(range(L, D, L))
    rows = _sample_idx(M, [128, 256, M // 2], rng)
    # sampled rows of Y and dX: the oracle on the row subset (same slicing along N or K)
    sub = dict(c, x=c["x"][rows], dy=c["dy"][rows], M=len(rows))
    z, y = oracle.linear_fwd(sub["x"], c["w"], None, 0, k, split)
    dX, _, _ = oracle.linear_bwd(sub["dy"], sub["x"], c["w"], None, 0, k, split)
    idx = torch.from_numpy(rows).cuda()
    assert_close(to_f64(g["y"][idx]), y, "Y rows")
    assert_close(to_f64(g["dx"][idx]), dX, "dX rows")
    # sampled rows of dW (= columns of dY) and db: dW[n,:] = sum_m dY[m,n] X[m,:]
    ncols = _sample_idx(N, bounds if split == 0 else [256, 512], rng)
    dy_sub = np.ascontiguousarray(c["dy"][:, ncols])
    _, dW, db = oracle.linear_bwd(dy_sub, c["x"], np.ascontiguousarray(c["w"][ncols]), None, 0)
    nidx = torch.from_numpy(ncols).cuda()
    assert_close(to_f64(g["dw"][nidx]), dW, "dW rows")
    assert_close(to_f64(g["db"][nidx]), db, "db")
    # identities over every element: Y r = X (W^T r),  dX r = dY (W r),  r^T dW = (dY r)^T X
    Xf = inputs.bf16_bits_to_f32(c["x"]).astype(np.float64)
    Wf = inputs.bf16_bits_to_f32(c["w"]).astype(np.float64)
    Gf = inputs.bf16_bits_to_f32(c["dy"]).astype(np.float64)
    rN, rK = rng.standard_normal(N), rng.standard_normal(K)
    def close(a, b, scale, name):
        # every element of the GPU output carries one bf16 rounding (2^-9 relative): a random
        # combination of n of them has error ~ 2^-9 * rms * sqrt(n); allow 8x that
        err = np.abs(a - b).max()
        assert err <= 8 * scale, "%s identity: %.3e > %.3e" % (name, err, 8 * scale)
    Y = to_f64(g["y"]); dXg = to_f64(g["dx"]); dWg = to_f64(g["dw"])
    close(Y @ rN, Xf @ (Wf.T @ rN), 2.0 ** -9 * np.sqrt(np.mean(Y * Y)) * np.sqrt(N), "Y")
    close(dXg @ rK, Gf @ (Wf @ rK), 2.0 ** -9 * np.sqrt(np.mean(dXg * dXg)) * np.sqrt(K), "dX")
    close(rN @ dWg, (Gf @ rN) @ Xf, 2.0 ** -9 * np.sqrt(np.mean(dWg * dWg)) * np.sqrt(N), "dW")
    return g


def test_config5_split_sweep_shape_k8_out(P):
    check_large_linear(P, 16384, 8192, 8192, 8, 0, 0.02, 20)


def test_config5_split_sweep_shape_k8_red(P):
    check_large_linear(P, 16384, 8192, 8192, 8, 1, 0.02, 21)


@pytest.mark.parametrize("NK", [(6144, 2048), (2048, 2048), (8192, 2048), (2048, 8192)])
def test_config3_decoder_linears_k4(P, NK):
    N, K = NK
    check_large_linear(P, 8192, N, K, 4, 0, 0.02, 30 + N // 2048 + K // 8192)


def test_config4_wide_layer_k8(P):
    # hidden 8192, ffn 32768, tokens 4 x 2048: the first MLP linear, split along the output dim,
    # and the second, split along the reduction dim
    check_large_linear(P, 8192, 32768, 8192, 8, 0, 0.01, 40)
    check_large_linear(P, 8192, 8192, 32768, 8, 1, 0.01, 41)


# ---------------------------------------------------------------------------------------------
# failure detection without a fault: a wait that nothing satisfies ends with a status, not a hang

def test_bounded_wait_reports_timeout_and_context_stays_usable(P):
    import time
    ws = P.new_workspace(4096)
    assert P.osdp_read_device_status(ws) == (0, 0)
    t0 = time.perf_counter()
    P.osdp_debug_wait_probe(ws, 20000, check=True)        # 20 ms limit
    rc, st = P.osdp_read_device_status(ws)
    dt = time.perf_counter() - t0
    assert rc == 0 and st == 8                            # OSDP_ERR_DEVICE_TIMEOUT
    assert 0.015 < dt < 2.0
    assert P.osdp_read_device_status(ws) == (0, 0)        # the status word was cleared
    # the context is intact: a normal call still works and matches the oracle
    c = inputs.linear_case(128, 256, 64, layer=13)
    compare(run_linear(P, c, 2, P.SPLIT_OUT), oracle_linear(c, 0, 2, oracle.SPLIT_OUT), 0)
    assert P.osdp_debug_wait_probe(ws, 0) == 2 and P.osdp_debug_wait_probe(None, 10) == 1


# ---------------------------------------------------------------------------------------------
# config 4 as the chained MLP block (hidden 8192, ffn 32768, tokens 4 x 2048), k = 8 along ffn:
# sampled token rows (Y, dX) and sampled ffn units (dW1 rows, dW2 columns, db1) against the oracle

def test_config4_mlp_chain_k8_sampled(P):
    M, H, F, k = 8192, 8192, 32768, 8
    c = inputs.mlp_case(M, H, F, w_std=0.01, bias_std=0.01, layer=42)
    g = run_mlp(P, c, k, dw_fp32=False)
    rng = np.random.default_rng(42)
    L = F // k
    rows = _sample_idx(M, [128, 256, M // 2], rng, extra=4)
    _, y = oracle.mlp_fwd(c["x"][rows], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
    dX, _, _, _, _ = oracle.mlp_bwd(c["dy"][rows], c["x"][rows], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    idx = torch.from_numpy(rows).cuda()
    assert_close(to_f64(g["y"][idx]), y, "Y rows")
    assert_close(to_f64(g["dx"][idx]), dX, "dX rows")
    # gradients of the weights of sampled ffn units depend only on those units' rows of W1 / columns of W2
    fu = _sample_idx(F, list(range(L, F, L)), rng, extra=4)
    w1s = np.ascontiguousarray(c["w1"][fu]); w2s = np.ascontiguousarray(c["w2"][:, fu]); b1s = c["b1"][fu]
    _, dW1, db1, dW2, _ = oracle.mlp_bwd(c["dy"], c["x"], w1s, b1s, w2s, oracle.ACT_GELU_TANH, None)
    fidx = torch.from_numpy(fu).cuda()
    assert_close(to_f64(g["dw1"][fidx]), dW1, "dW1 rows")
    assert_close(to_f64(g["dw2"][:, fidx]), dW2, "dW2 columns")
    assert_close(to_f64(g["db1"][fidx]), db1, "db1")
    assert_close(to_f64(g["db2"]), inputs.bf16_bits_to_f32(c["dy"]).astype(np.float64).sum(axis=0), "db2",
                 relf_tol=1e-5)


# ---------------------------------------------------------------------------------------------
# the calls are plain asynchronous launches: a captured CUDA graph replays them bit for bit

def test_cuda_graph_replay_matches_eager(P):
    c = inputs.linear_case(512, 1024, 512, bias_std=0.1, layer=14)
    M, N, K = 512, 1024, 512
    x, dy, wf, b = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"]), to_dev(c["bias"])
    _, n1 = P.osdp_split_linear_workspace_bytes(M, N, K, 4, 1, 0, P.OP_LINEAR_FWD)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, N, K, 4, 1, 0, P.OP_LINEAR_BWD)
    ws = P.new_workspace(max(n1, n2))
    outs = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda"), torch.empty(M, K, dtype=torch.bfloat16, device="cuda"),
            torch.empty(N * K, dtype=torch.float32, device="cuda"), torch.empty(N, dtype=torch.float32, device="cuda")]

    def step():
        P.osdp_split_linear_fwd(x, wf, 0, b, M, N, K, 4, P.SPLIT_RED, 0, outs[0], None, ws, check=True)
        P.osdp_split_linear_bwd(dy, x, wf, 0, None, M, N, K, 4, P.SPLIT_RED, 0, outs[1], outs[2], 0, P.DTYPE_FP32, 0,
                                outs[3], ws, check=True)

    step()
    torch.cuda.synchronize()
    eager = [o.clone() for o in outs]
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            step()
    for o in outs:
        o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for e, o in zip(eager, outs):
        assert torch.equal(_bits(e), _bits(o))
    assert P.osdp_read_device_status(ws) == (0, 0)


@pytest.mark.parametrize("k", [2, 5])
def test_mlp_backward_with_subsets_of_outputs(P, k):
    """Every output of the MLP block's backward is optional; whatever is asked for has the same bits as in the call
    that asks for everything (k = 5: the slices are pipelined over two sets of slice buffers, with the weight
    gradients on the internal streams; without weight gradients nothing is forked)."""
    M, H, F = 300, 264, 520
    c = inputs.mlp_case(M, H, F, w_std=0.08, layer=29)
    x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
    b1, b2 = to_dev(c["b1"]), to_dev(c["b2"])
    _, n1 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_FWD)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_BWD)
    ws = P.new_workspace(max(n1, n2))
    y = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    z1 = torch.empty(M, F, dtype=torch.bfloat16, device="cuda")
    P.osdp_split_mlp_fwd(x, wf, c["off_w1"], b1, c["off_w2"], b2, M, H, F, k, 1, y, z1, ws, check=True)

    def bwd(want_dx, want_dw, want_db):
        dx = torch.full((M, H), 7.0, dtype=torch.bfloat16, device="cuda") if want_dx else None
        dwf = torch.full((2 * F * H,), 7.0, dtype=torch.float32, device="cuda") if want_dw else None
        db1 = torch.full((F,), 7.0, dtype=torch.float32, device="cuda") if want_db else None
        db2 = torch.full((H,), 7.0, dtype=torch.float32, device="cuda") if want_db else None
        P.osdp_split_mlp_bwd(dy, x, wf, c["off_w1"], c["off_w2"], z1, M, H, F, k, 1, dx, dwf, c["off_w1"], c["off_w2"],
                             P.DTYPE_FP32, 0, db1, db2, ws, check=True)
        torch.cuda.synchronize()
        return {"dx": dx, "dw": dwf, "db1": db1, "db2": db2}

    full = bwd(True, True, True)
    grads = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    assert_close(to_f64(full["dx"]), grads[0], "dx")
    assert_close(to_f64(full["db1"]), grads[2], "db1")
    for want in ((True, False, False), (False, True, False), (False, False, True), (True, False, True),
                 (False, True, True), (True, True, False)):
        part = bwd(*want)
        for name, t in part.items():
            if t is not None:
                assert torch.equal(_bits(t), _bits(full[name])), (want, name)
    assert P.osdp_read_device_status(ws) == (0, 0)


@pytest.mark.parametrize("k", [2, 5])
def test_mlp_cuda_graph_replay_matches_eager(P, k):
    """The MLP block's backward forks onto the library's internal streams (k = 5, small slices: pipelined over
    two sets of slice buffers; k = 2: one fork / join per slice); a capture follows them and replays the same bits."""
    M, H, F = 300, 264, 520
    c = inputs.mlp_case(M, H, F, w_std=0.08, layer=23)
    x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
    b1, b2 = to_dev(c["b1"]), to_dev(c["b2"])
    _, n1 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_FWD)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_BWD)
    ws = P.new_workspace(max(n1, n2))
    y = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    z1 = torch.empty(M, F, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    dwf = torch.empty(2 * F * H, dtype=torch.float32, device="cuda")
    db1 = torch.empty(F, dtype=torch.float32, device="cuda")
    db2 = torch.empty(H, dtype=torch.float32, device="cuda")
    outs = [y, z1, dx, dwf, db1, db2]

    def step():
        P.osdp_split_mlp_fwd(x, wf, c["off_w1"], b1, c["off_w2"], b2, M, H, F, k, 1, y, z1, ws, check=True)
        P.osdp_split_mlp_bwd(dy, x, wf, c["off_w1"], c["off_w2"], z1, M, H, F, k, 1, dx, dwf, c["off_w1"], c["off_w2"],
                             P.DTYPE_FP32, 0, db1, db2, ws, check=True)

    step()
    step()   # the second call reuses the events of the first
    torch.cuda.synchronize()
    eager = [o.clone() for o in outs]
    grads = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    assert_close(to_f64(dx), grads[0], "dx")
    assert_close(to_f64(dwf[c["off_w1"]:c["off_w1"] + F * H].view(F, H)), grads[1], "dw1")
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            step()
    for rep in range(2):
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for e, o in zip(eager, outs):
            assert torch.equal(_bits(e), _bits(o)), rep
    step()   # eager again after the capture ended: the internal streams are free again
    torch.cuda.synchronize()
    for e, o in zip(eager, outs):
        assert torch.equal(_bits(e), _bits(o))
    assert P.osdp_read_device_status(ws) == (0, 0)


# ---------------------------------------------------------------------------------------------
# seeded random shapes / splits / activations / flags: every tile-shape variant of the kernel
# (CTA pairs, single CTAs with 256-, 128- and 64-wide tiles), slices narrower than a tile, one-row
# batches, ragged everything

def _random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < n:
        big = rng.random() < 0.25
        M = int(rng.integers(1, 3000 if big else 600))
        N = 8 * int(rng.integers(1, 400 if big else 90))
        K = 8 * int(rng.integers(1, 300 if big else 90))
        split = int(rng.integers(0, 2))
        D = N if split == 0 else K
        k = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 12, 16, max(1, D // 8)]))
        act = int(rng.choice([0, 0, 1, 2]))
        flags = 2 if (act == 0 and 1 < k <= 8 and rng.random() < 0.3) else 0   # bf16 running sum: k <= 8 only
        if flags == 0 and rng.random() < 0.4:
            flags = 16                                                          # slice-major order, fp32 carry
        cases.append((M, N, K, k, split, act, flags))
    return cases


@pytest.mark.parametrize("chunk", range(4))
def test_random_shapes_against_oracle(P, chunk):
    for idx, (M, N, K, k, split, act, flags) in enumerate(_random_cases(40, 2209)[chunk * 10:(chunk + 1) * 10]):
        if P.osdp_slice_range(N if split == 0 else K, k, 0)[0] != 0:
            continue
        c = inputs.linear_case(M, N, K, w_std=0.05, bias_std=0.2, w_offset=8 * (idx % 5), flat_pad=8,
                               layer=100 + chunk * 10 + idx)
        g = run_linear(P, c, k, split, act=act, flags=flags, dw_fp32=bool(idx % 2))
        o = oracle_linear(c, act, k, split)
        loose = 3e-2 * (2 * k) ** 0.5 if flags == 2 else 3e-2
        try:
            compare(g, o, act, y_abs_tol=loose if split == 1 else 3e-2, dx_abs_tol=loose if split == 0 else 3e-2)
        except AssertionError as e:
            raise AssertionError("case M=%d N=%d K=%d k=%d split=%d act=%d flags=%d: %s" % (
                M, N, K, k, split, act, flags, e))


# ---------------------------------------------------------------------------------------------
# a shape for which the tile model picks the 256 x 512 tile (74 wide tiles = one round, reduction
# 8192) in a GEMM whose epilogue does more than store: bias + pre-activation save + GeLU (first layer
# forward, and its recomputation in the backward), next to 256-wide tiles in the same chain

def test_mlp_wide_tile_epilogues(P):
    M, H, F = 512, 8192, 18944
    c = inputs.mlp_case(M, H, F, w_std=0.01, bias_std=0.05, layer=17)
    _, y = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, None)
    grads = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, None)
    g = run_mlp(P, c, 1, dw_fp32=False)
    compare_mlp(g, (y,) + tuple(grads))
    g2 = run_mlp(P, c, 2, dw_fp32=False, recompute=True)
    compare_mlp(g2, (y,) + tuple(grads))


# ---------------------------------------------------------------------------------------------
# ragged extents on the 256 x 512 tile: 2000 x 4232 x 8200 makes the model pick it for the forward and
# for dX (72 and 136 wide tiles); with k = 3 the slices (length 1416) end inside a 512-wide tile

@pytest.mark.parametrize("k,split", [(1, 0), (3, 0), (3, 1)])
def test_ragged_extents_on_the_wide_tile(P, k, split):
    c = inputs.linear_case(2000, 4232, 8200, w_std=0.02, bias_std=0.1, w_offset=24, flat_pad=8, layer=18)
    g = run_linear(P, c, k, split, dw_fp32=False)
    compare(g, oracle_linear(c, 0), 0)
    if k > 1:
        g1 = run_linear(P, c, 1, split, dw_fp32=False)
        for name in (("y", "dw", "db") if split == 0 else ("dx", "dw", "db")):
            assert torch.equal(_bits(g[name]), _bits(g1[name])), name


# ---------------------------------------------------------------------------------------------
# seeded random MLP blocks: ragged extents, both GeLU forms, saved and recomputed pre-activation, both dW types

@pytest.mark.parametrize("chunk", range(2))
def test_random_mlp_blocks_against_oracle(P, chunk):
    import random
    rng = random.Random(4000 + chunk)
    done = 0
    while done < 8:
        M = rng.choice([64, 130, 256, 300, 513, 1000])
        H = 8 * rng.randint(1, 120)
        F = 8 * rng.randint(2, 300)
        k = rng.choice([1, 2, 3, 4, 5, 8])
        if P.osdp_slice_range(F, k, 0)[0] != 0:
            continue
        act = rng.choice([1, 2])
        c = inputs.mlp_case(M, H, F, w_std=0.05, bias_std=0.1, layer=30 + done)
        g = run_mlp(P, c, k, act=act, dw_fp32=rng.random() < 0.5, recompute=rng.random() < 0.4)
        _, y = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], act, k)
        grads = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], act, k)
        compare_mlp(g, (y,) + tuple(grads))
        done += 1


# ---------------------------------------------------------------------------------------------
# the calls allocate nothing: staging is exactly the caller's workspace

def test_calls_allocate_no_device_memory(P):
    M, N, K, k = 512, 2048, 1024, 4
    c = inputs.linear_case(M, N, K)
    x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
    out = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(M, K, dtype=torch.bfloat16, device="cuda")
    dw = torch.empty(N * K, dtype=torch.float32, device="cuda")
    db = torch.empty(N, dtype=torch.float32, device="cuda")
    _, n1 = P.osdp_split_linear_workspace_bytes(M, N, K, k, 1, 0, P.OP_LINEAR_FWD)
    _, n2 = P.osdp_split_linear_workspace_bytes(M, N, K, k, 0, 0, P.OP_LINEAR_BWD)
    ws = P.new_workspace(max(n1, n2))

    def step():
        P.osdp_split_linear_fwd(x, wf, 0, None, M, N, K, k, 1, 0, out, None, ws, check=True)
        P.osdp_split_linear_bwd(dy, x, wf, 0, None, M, N, K, k, 0, 0, dx, dw, 0, P.DTYPE_FP32, 0, db, ws, check=True)
    step()                                   # first use: kernel attributes, internal streams
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    before_alloc = torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.max_memory_allocated() == before_alloc       # nothing through torch's allocator
    assert free_after == free_before                                # and nothing behind its back
    # the reported staging is what the call needs: one byte less is refused, nothing is launched
    assert P.osdp_split_linear_bwd(dy, x, wf, 0, None, M, N, K, k, 0, 0, dx, dw, 0, P.DTYPE_FP32, 0, db,
                                   (ws.data_ptr(), n2 - 1)) == 5


# ---------------------------------------------------------------------------------------------
# two host threads, two streams, backward calls that fork onto the library's internal streams: the calls are
# serialised on the host while they enqueue, each is joined back into its own stream, results as when run alone

def test_two_threads_calling_backward_on_their_own_streams(P):
    import threading
    M, N, K, k = 1024, 1024, 512, 4
    jobs = []
    for t in range(2):
        c = inputs.linear_case(M, N, K, w_std=0.05, layer=22 + t)
        x, dy, wf = to_dev(c["x"]), to_dev(c["dy"]), to_dev(c["w_flat"])
        _, n = P.osdp_split_linear_workspace_bytes(M, N, K, k, 0, 0, P.OP_LINEAR_BWD)
        jobs.append({"x": x, "dy": dy, "wf": wf, "ws": P.new_workspace(n), "stream": torch.cuda.Stream(),
                     "dx": torch.empty(M, K, dtype=torch.bfloat16, device="cuda"),
                     "dw": torch.empty(N * K, dtype=torch.float32, device="cuda"),
                     "db": torch.empty(N, dtype=torch.float32, device="cuda")})

    def call(j, stream):
        P.osdp_split_linear_bwd(j["dy"], j["x"], j["wf"], 0, None, M, N, K, k, P.SPLIT_OUT, 0, j["dx"], j["dw"], 0,
                                P.DTYPE_FP32, 0, j["db"], j["ws"], stream=stream, check=True)

    want = []
    for j in jobs:                                   # alone, one after the other
        call(j, torch.cuda.current_stream())
        torch.cuda.synchronize()
        want.append([j[n].clone() for n in ("dx", "dw", "db")])
        for n in ("dx", "dw", "db"):
            j[n].fill_(float("nan"))
    errors = []

    def worker(j):
        try:
            torch.cuda.set_device(0)
            for _ in range(20):
                call(j, j["stream"])
            j["stream"].synchronize()
        except Exception as e:      # pragma: no cover
            errors.append(e)
    threads = [threading.Thread(target=worker, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    for j, w in zip(jobs, want):
        for n, ref in zip(("dx", "dw", "db"), w):
            assert torch.equal(_bits(j[n]), _bits(ref)), n
        assert P.osdp_read_device_status(j["ws"]) == (0, 0)
