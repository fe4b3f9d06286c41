"""Pins for the CPU oracle: each test checks it against something other than itself --
brute force, closed forms, finite differences, library routines, the split == unsplit
invariant -- so that a dropped term, a wrong sign or a transposed operand fails one of them."""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2209_13258_b200 import inputs

ACTS = [oracle.ACT_NONE, oracle.ACT_GELU_TANH, oracle.ACT_GELU_ERF]


def rnd(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


def relerr(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


# ------------------------------------------------------------------ bf16 helpers

def test_bf16_widen_exact_cases():
    bits = np.array([0x3F80, 0xBF80, 0x0000, 0x8000, 0x4000, 0x3F00, 0x7F80, 0xFF80, 0x0001], dtype=np.uint16)
    got = oracle.bf16_to_f64(bits)
    want = [1.0, -1.0, 0.0, -0.0, 2.0, 0.5, math.inf, -math.inf, 2.0 ** -133]
    assert np.array_equal(got, np.array(want))
    assert math.copysign(1.0, got[3]) == -1.0
    assert math.isnan(oracle.bf16_to_f64(np.array([0x7FC0], dtype=np.uint16))[0])


def test_bf16_round_nearest_even_cases():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20,
                  -1.0 - 2.0 ** -8, math.inf, -math.inf, 3.4028234663852886e38], dtype=np.float32)
    got = oracle.f32_to_bf16(x)
    # ties go to the even mantissa: 1+2^-8 -> 1.0 (0x3F80); 1+3*2^-8 -> 1+2^-6 (0x3F82)
    assert list(got[:7]) == [0x3F80, 0x3F80, 0x3F82, 0x3F81, 0xBF80, 0x7F80, 0xFF80]
    assert got[7] == 0x7F80  # the largest fp32 rounds up past the largest finite bf16 to +Inf
    nan = oracle.f32_to_bf16(np.array([math.nan], dtype=np.float32))[0]
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x007F) != 0


def test_bf16_round_matches_torch_and_generator():
    x = (rnd((1_000_000,), 3) * np.exp(rnd((1_000_000,), 4) * 8)).astype(np.float32)
    got = oracle.f32_to_bf16(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)
    assert np.array_equal(inputs.f32_to_bf16_bits(x), want)
    assert np.array_equal(oracle.bf16_to_f64(got), inputs.bf16_bits_to_f32(got).astype(np.float64))


# ------------------------------------------------------------------ GeLU closed forms and library

def test_gelu_closed_forms():
    for act in (oracle.ACT_GELU_TANH, oracle.ACT_GELU_ERF):
        assert oracle.gelu(0.0, act) == 0.0
        assert oracle.gelu_grad(0.0, act) == 0.5
        assert abs(oracle.gelu(40.0, act) - 40.0) < 1e-12
        assert abs(oracle.gelu(-40.0, act)) < 1e-12
        assert abs(oracle.gelu_grad(40.0, act) - 1.0) < 1e-12
        assert abs(oracle.gelu_grad(-40.0, act)) < 1e-12
    # gelu_erf(1) = Phi(1), the standard normal CDF at 1
    assert abs(oracle.gelu(1.0, oracle.ACT_GELU_ERF) - 0.8413447460685429) < 1e-15
    # gelu_erf(x) - gelu_erf(-x) = x for every x (Phi(x) + Phi(-x) = 1)
    for x in (0.3, 1.7, 4.2):
        assert abs(oracle.gelu(x, oracle.ACT_GELU_ERF) - oracle.gelu(-x, oracle.ACT_GELU_ERF) - x) < 1e-15
        assert abs(oracle.gelu(x, oracle.ACT_GELU_TANH) - oracle.gelu(-x, oracle.ACT_GELU_TANH) - x) < 1e-15
    assert oracle.gelu(1.25, oracle.ACT_NONE) == 1.25 and oracle.gelu_grad(1.25, oracle.ACT_NONE) == 1.0


def test_gelu_matches_torch_and_finite_differences():
    xs = np.linspace(-6, 6, 241)
    for act, approx in ((oracle.ACT_GELU_TANH, "tanh"), (oracle.ACT_GELU_ERF, "none")):
        t = torch.tensor(xs, dtype=torch.float64, requires_grad=True)
        y = torch.nn.functional.gelu(t, approximate=approx)
        y.sum().backward()
        got = np.array([oracle.gelu(v, act) for v in xs])
        gotg = np.array([oracle.gelu_grad(v, act) for v in xs])
        assert np.max(np.abs(got - y.detach().numpy())) < 1e-14
        assert np.max(np.abs(gotg - t.grad.numpy())) < 1e-13
        h = 1e-6
        fd = np.array([(oracle.gelu(v + h, act) - oracle.gelu(v - h, act)) / (2 * h) for v in xs])
        assert np.max(np.abs(fd - gotg)) < 1e-8


# ------------------------------------------------------------------ slice table

def test_slice_table_by_hand():
    # D=1024, k=4: L=256, even
    assert [oracle.slice_range(1024, 4, s) for s in range(4)] == [(0, 256), (256, 512), (512, 768), (768, 1024)]
    # D=1024, k=6: ceil=171 -> 176; 5 full slices + a tail of 144
    assert [oracle.slice_range(1024, 6, s) for s in range(6)] == [
        (0, 176), (176, 352), (352, 528), (528, 704), (704, 880), (880, 1024)]
    # k=0 means unsplit
    assert oracle.slice_range(40, 0, 0) == (0, 40)
    # D=40, k=5: L=8 exactly
    assert oracle.slice_range(40, 5, 4) == (32, 40)
    # D=40, k=6: L=8 would leave the 6th slice empty
    with pytest.raises(oracle.OracleError) as e:
        oracle.slice_range(40, 6, 0)
    assert e.value.code == oracle.BAD_SPLIT
    # slices tile the range without gaps for many (D,k)
    for D in (8, 24, 200, 1000, 4096):
        for k in range(1, 40):
            try:
                r = [oracle.slice_range(D, k, s) for s in range(k)]
            except oracle.OracleError:
                L = -(-(-(-D // k)) // 8) * 8
                assert (k - 1) * L >= D
                continue
            assert r[0][0] == 0 and r[-1][1] == D
            assert all(r[i][1] == r[i + 1][0] for i in range(k - 1))
            assert all(e > b for b, e in r)
            assert all((b % 8) == 0 for b, _ in r)


# ------------------------------------------------------------------ brute force on tiny shapes

def _exact(a):
    return [[Fraction(float(v)) for v in row] for row in a]


@pytest.mark.parametrize("split_dim", [None, oracle.SPLIT_OUT, oracle.SPLIT_RED])
def test_brute_force_exact_rational(split_dim):
    """No activation: every output is a finite sum of products, computed here exactly in
    rationals with plain index loops written from the definitions."""
    M, N, K = 5, 24, 40
    x = inputs.normal_bf16((M, K), 1.0, 101)
    w = inputs.normal_bf16((N, K), 0.5, 102)
    dy = inputs.normal_bf16((M, N), 1.0, 103)
    b = inputs.normal_f32((N,), 0.3, 104)
    X, W, DY = (_exact(inputs.bf16_bits_to_f32(t)) for t in (x, w, dy))
    B = [Fraction(float(v)) for v in b]
    Y = [[sum(X[m][j] * W[n][j] for j in range(K)) + B[n] for n in range(N)] for m in range(M)]
    dX = [[sum(DY[m][n] * W[n][j] for n in range(N)) for j in range(K)] for m in range(M)]
    dW = [[sum(DY[m][n] * X[m][j] for m in range(M)) for j in range(K)] for n in range(N)]
    db = [sum(DY[m][n] for m in range(M)) for n in range(N)]
    for k in ([1] if split_dim is None else [1, 2, 3]):
        z, y = oracle.linear_fwd(x, w, b, oracle.ACT_NONE, k, split_dim)
        gx, gw, gb = oracle.linear_bwd(dy, x, w, None, oracle.ACT_NONE, k, split_dim)
        for got, want in ((y, Y), (z, Y), (gx, dX), (gw, dW)):
            wantf = np.array([[float(v) for v in row] for row in want])
            assert np.max(np.abs(got - wantf)) <= 1e-13 * max(1.0, np.max(np.abs(wantf)))
        assert np.max(np.abs(gb - np.array([float(v) for v in db]))) <= 1e-13


# ------------------------------------------------------------------ closed forms

def test_identity_onehot_ones():
    n = 16
    X = rnd((7, n), 5)
    _, y = oracle.linear_fwd(X, np.eye(n), None)
    assert np.array_equal(y, X)                                   # W = I  =>  Y = X
    W = rnd((12, n), 6)
    onehot = np.zeros((n, n)); onehot[np.arange(n), (np.arange(n) * 5) % n] = 1.0
    _, y = oracle.linear_fwd(onehot, W, None)
    assert np.array_equal(y, W[:, (np.arange(n) * 5) % n].T)      # one-hot rows pick columns of W^T
    ones = np.ones((3, n))
    _, y = oracle.linear_fwd(ones, W, None, k=2, split_dim=oracle.SPLIT_RED)
    assert np.allclose(y, np.tile(W.sum(axis=1), (3, 1)), rtol=0, atol=1e-13)
    # backward with dY = ones: dX rows are column sums of W, dW rows are column sums of X, db = M
    dX, dW, db = oracle.linear_bwd(np.ones((7, 12)), X, W, k=2, split_dim=oracle.SPLIT_OUT)
    assert np.allclose(dX, np.tile(W.sum(axis=0), (7, 1)), atol=1e-13)
    assert np.allclose(dW, np.tile(X.sum(axis=0), (12, 1)), atol=1e-13)
    assert np.array_equal(db, np.full((12,), 7.0))
    # a transposed operand would break this asymmetric case: Y[m,n] = X[m,0] * W[n,0]
    X1 = np.zeros((4, 8)); X1[:, 0] = [1, 2, 3, 4]
    W1 = np.zeros((16, 8)); W1[:, 0] = np.arange(16)
    _, y = oracle.linear_fwd(X1, W1, None, k=2, split_dim=oracle.SPLIT_OUT)
    assert np.array_equal(y, np.outer([1, 2, 3, 4], np.arange(16)))


# ------------------------------------------------------------------ library routine (torch fp64 + autograd)

@pytest.mark.parametrize("act,approx", [(oracle.ACT_NONE, None), (oracle.ACT_GELU_TANH, "tanh"),
                                        (oracle.ACT_GELU_ERF, "none")])
@pytest.mark.parametrize("split", [(None, 1), (oracle.SPLIT_OUT, 3), (oracle.SPLIT_RED, 5), (oracle.SPLIT_OUT, 4)])
def test_linear_matches_torch_autograd(act, approx, split):
    split_dim, k = split
    M, N, K = 37, 88, 120
    x = inputs.normal_bf16((M, K), 1.0, 11); w = inputs.normal_bf16((N, K), 0.2, 12)
    dy = inputs.normal_bf16((M, N), 1.0, 13); b = inputs.normal_f32((N,), 0.5, 14)
    tx = torch.tensor(inputs.bf16_bits_to_f32(x), dtype=torch.float64, requires_grad=True)
    tw = torch.tensor(inputs.bf16_bits_to_f32(w), dtype=torch.float64, requires_grad=True)
    tb = torch.tensor(b, dtype=torch.float64, requires_grad=True)
    tz = tx @ tw.T + tb
    ty = tz if approx is None else torch.nn.functional.gelu(tz, approximate=approx)
    ty.backward(torch.tensor(inputs.bf16_bits_to_f32(dy), dtype=torch.float64))
    z, y = oracle.linear_fwd(x, w, b, act, k, split_dim)
    dX, dW, db = oracle.linear_bwd(dy, x, w, z, act, k, split_dim)
    assert relerr(z, tz.detach().numpy()) < 1e-13
    assert relerr(y, ty.detach().numpy()) < 1e-13
    assert relerr(dX, tx.grad.numpy()) < 1e-12
    assert relerr(dW, tw.grad.numpy()) < 1e-12
    assert relerr(db, tb.grad.numpy()) < 1e-12


@pytest.mark.parametrize("k", [None, 1, 2, 4, 7])
def test_mlp_matches_torch_autograd(k):
    M, H, F = 19, 48, 112
    c = inputs.mlp_case(M, H, F, w_std=0.3, layer=3)
    f = lambda a: torch.tensor(inputs.bf16_bits_to_f32(a), dtype=torch.float64, requires_grad=True)
    tx, tw1, tw2 = f(c["x"]), f(c["w1"]), f(c["w2"])
    tb1 = torch.tensor(c["b1"], dtype=torch.float64, requires_grad=True)
    tb2 = torch.tensor(c["b2"], dtype=torch.float64, requires_grad=True)
    ty = torch.nn.functional.gelu(tx @ tw1.T + tb1, approximate="tanh") @ tw2.T + tb2
    ty.backward(torch.tensor(inputs.bf16_bits_to_f32(c["dy"]), dtype=torch.float64))
    _, y = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
    dX, dW1, db1, dW2, db2 = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    assert relerr(y, ty.detach().numpy()) < 1e-13
    for got, want in ((dX, tx.grad), (dW1, tw1.grad), (db1, tb1.grad), (dW2, tw2.grad), (db2, tb2.grad)):
        assert relerr(got, want.numpy()) < 1e-12


# ------------------------------------------------------------------ invariant: slices reproduce the unsplit result

@pytest.mark.parametrize("act", ACTS)
def test_split_equals_unsplit(act):
    for (M, N, K) in ((9, 40, 64), (33, 72, 200), (4, 8, 8)):
        x = rnd((M, K), 21); w = rnd((N, K), 22, 0.3); dy = rnd((M, N), 23); b = rnd((N,), 24)
        z0, y0 = oracle.linear_fwd(x, w, b, act)
        g0 = oracle.linear_bwd(dy, x, w, z0, act)
        for split_dim, D in ((oracle.SPLIT_OUT, N), (oracle.SPLIT_RED, K)):
            for k in range(1, D // 8 + 1):
                try:
                    oracle.slice_range(D, k, 0)
                except oracle.OracleError:
                    continue
                z, y = oracle.linear_fwd(x, w, b, act, k, split_dim)
                g = oracle.linear_bwd(dy, x, w, z, act, k, split_dim)
                assert relerr(y, y0) < 1e-12 and relerr(z, z0) < 1e-12
                for a, a0 in zip(g, g0):
                    assert relerr(a, a0) < 1e-12


def test_split_rejects_empty_slice():
    x = rnd((4, 16), 1); w = rnd((16, 16), 2)
    with pytest.raises(oracle.OracleError):
        oracle.linear_fwd(x, w, None, oracle.ACT_NONE, 3, oracle.SPLIT_OUT)   # L=8 -> third slice empty


# ------------------------------------------------------------------ finite differences of L = sum(dY * Y)

@pytest.mark.parametrize("act", ACTS)
@pytest.mark.parametrize("split", [(None, 1), (oracle.SPLIT_OUT, 2), (oracle.SPLIT_RED, 3)])
def test_finite_difference_gradients(act, split):
    split_dim, k = split
    M, N, K = 3, 16, 24
    x = rnd((M, K), 31); w = rnd((N, K), 32, 0.4); b = rnd((N,), 33, 0.2); dy = rnd((M, N), 34)

    def loss(x_, w_, b_):
        return float(np.sum(dy * oracle.linear_fwd(x_, w_, b_, act, k, split_dim)[1]))

    z, _ = oracle.linear_fwd(x, w, b, act, k, split_dim)
    dX, dW, db = oracle.linear_bwd(dy, x, w, z, act, k, split_dim)
    h = 1e-6
    rng = np.random.default_rng(35)
    for arr, grad, which in ((x, dX, 0), (w, dW, 1), (b, db, 2)):
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h; am[idx] -= h
            args_p = [x, w, b]; args_m = [x, w, b]
            args_p[which] = ap; args_m[which] = am
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(grad[idx]))


def test_mlp_finite_difference():
    M, H, F = 3, 8, 24
    x = rnd((M, H), 41); w1 = rnd((F, H), 42, 0.5); b1 = rnd((F,), 43, 0.2)
    w2 = rnd((H, F), 44, 0.5); b2 = rnd((H,), 45, 0.2); dy = rnd((M, H), 46)
    for k in (None, 3):
        loss = lambda x_, w1_, w2_: float(np.sum(dy * oracle.mlp_fwd(x_, w1_, b1, w2_, b2, oracle.ACT_GELU_TANH, k)[1]))
        dX, dW1, db1, dW2, db2 = oracle.mlp_bwd(dy, x, w1, b1, w2, oracle.ACT_GELU_TANH, k)
        h = 1e-6
        for arr, grad, which in ((x, dX, 0), (w1, dW1, 1), (w2, dW2, 2)):
            for idx in ((0, 0), (2, 5), (1, 7)):
                ap, am = arr.copy(), arr.copy()
                ap[idx] += h; am[idx] -= h
                a_p = [x, w1, w2]; a_m = [x, w1, w2]
                a_p[which] = ap; a_m[which] = am
                fd = (loss(*a_p) - loss(*a_m)) / (2 * h)
                assert abs(fd - grad[idx]) <= 2e-6 * max(1.0, abs(grad[idx]))


# ------------------------------------------------------------------ the input generator

def test_generator_is_counter_based_and_normal():
    a = inputs.normal_f64(10_000, 7)
    assert np.array_equal(a[1234:1300], inputs.normal_f64(66, 7, start=1234))
    assert not np.array_equal(a[:100], inputs.normal_f64(100, 8))
    big = inputs.normal_f64(2_000_000, 9)
    assert abs(big.mean()) < 3e-3 and abs(big.std() - 1.0) < 3e-3
    assert abs(np.mean(big ** 3)) < 1e-2 and abs(np.mean(big ** 4) - 3.0) < 3e-2
    w = inputs.bf16_bits_to_f32(inputs.normal_bf16((512, 512), 0.02, 2))
    assert abs(w.std() - 0.02) < 2e-4
    c = inputs.linear_case(8, 16, 24, w_offset=40, flat_pad=8)
    assert np.array_equal(c["w_flat"][40:40 + 16 * 24].reshape(16, 24), c["w"])
    assert c["w_flat"].shape == (40 + 16 * 24 + 8,)


def test_slice_table_golden_file():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "slice_table.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        head, tail = line.split(":")
        D, k = (int(v) for v in head.split())
        want = [tuple(int(v) for v in pair.split(",")) for pair in tail.split()]
        assert [oracle.slice_range(D, k, s) for s in range(k)] == want
        n += 1
    assert n == 7


# ---------------------------------------------------------------------------------------------
# fp8 e4m3: the oracle's widening and the input generator's rounding, each against torch's own type

def test_e4m3_widening_matches_torch_on_all_codes():
    torch = pytest.importorskip("torch")
    codes = np.arange(256, dtype=np.uint8)
    mine = oracle.e4m3_to_f64(codes)
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).double().numpy()
    assert np.array_equal(np.isnan(mine), np.isnan(ref)) and int(np.isnan(mine).sum()) == 2
    ok = ~np.isnan(ref)
    assert np.array_equal(mine[ok], ref[ok])
    # landmarks of the format: largest value, smallest normal, smallest subnormal, signed zero
    assert mine[0x7E] == 448.0 and mine[0x08] == 2.0 ** -6 and mine[0x01] == 2.0 ** -9
    assert mine[0x80] == 0.0 and np.signbit(mine[0x80]) and mine[0x38] == 1.0


def test_e4m3_rounding_of_the_input_generator_matches_torch():
    torch = pytest.importorskip("torch")
    from paper_2209_13258_b200 import inputs
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.normal(0, 100, 200000), rng.normal(0, 1, 200000), rng.normal(0, 0.01, 200000),
                        oracle.e4m3_to_f64(np.arange(0x7F, dtype=np.uint8)),                       # exact values
                        (oracle.e4m3_to_f64(np.arange(0x7E, dtype=np.uint8)) +
                         oracle.e4m3_to_f64(np.arange(1, 0x7F, dtype=np.uint8))) / 2]).astype(np.float32)  # ties
    x = x[np.abs(x) <= 448.0]
    mine = inputs.f32_to_e4m3_bits(x)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    # -0 and +0 both stand for zero; everything else must be the same code
    zero = (mine & 0x7F) == 0
    assert np.array_equal(mine[~zero], ref[~zero]) and np.all((ref[zero] & 0x7F) == 0)
    assert inputs.f32_to_e4m3_bits(np.array([1e6, -1e6], np.float32)).tolist() == [0x7E, 0xFE]   # saturation
