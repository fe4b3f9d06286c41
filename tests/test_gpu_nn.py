"""The torch.nn front end (SplitLinear) against the fp64 oracle: forward, and the gradients autograd
collects from the library's backward, for a module that owns its weight and for one whose weight is a
window of an external flat parameter buffer."""
import numpy as np
import pytest

import oracle
from paper_2209_13258_b200 import inputs
from util import assert_close, to_dev, to_f64

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2209_13258_b200 as pkg
    pkg.lib()
    return pkg


@pytest.mark.parametrize("k,split,act", [(1, 0, 0), (4, 0, 1), (4, 1, 1), (3, 1, 0)])
def test_module_owning_its_weight(P, k, split, act):
    from paper_2209_13258_b200.nn import SplitLinear
    B_, S, K, N = 3, 100, 264, 528
    if P.osdp_slice_range(N if split == 0 else K, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c = inputs.linear_case(B_ * S, N, K, w_std=0.05, bias_std=0.2, layer=11)
    m = SplitLinear(K, N, bias=True, k_split=k, split_dim=split, act=act)
    with torch.no_grad():
        m.weight.copy_(to_dev(c["w"]))
        m.bias.copy_(to_dev(c["bias"]))
    x = to_dev(c["x"]).view(B_, S, K).requires_grad_(True)
    y = m(x)
    assert y.shape == (B_, S, N) and y.dtype == torch.bfloat16
    y.backward(to_dev(c["dy"]).view(B_, S, N))
    z, yo = oracle.linear_fwd(c["x"], c["w"], c["bias"], act, k, split)
    dXo, dWo, dbo = oracle.linear_bwd(c["dy"], c["x"], c["w"], z, act, k, split)
    assert_close(to_f64(y).reshape(-1, N), yo, "Y")
    assert_close(to_f64(x.grad).reshape(-1, K), dXo, "dX")
    assert_close(to_f64(m.flat_param.grad).reshape(N, K), dWo, "dW")
    assert_close(to_f64(m.bias.grad), dbo, "db")


def test_module_on_a_window_of_a_flat_buffer_and_no_input_grad(P):
    from paper_2209_13258_b200.nn import SplitLinear
    M, K, N, off = 256, 512, 1024, 72
    c = inputs.linear_case(M, N, K, w_std=0.05, w_offset=off, flat_pad=24, layer=12)
    flat = torch.nn.Parameter(to_dev(c["w_flat"]).clone())
    m = SplitLinear(K, N, bias=False, k_split=4, split_dim=P.SPLIT_OUT, flat=flat, w_offset=off)
    assert m.weight.data_ptr() == flat.data_ptr() + 2 * off        # a view: nothing was copied
    x = to_dev(c["x"])                                               # no gradient wanted for the input
    y = m(x)
    y.backward(to_dev(c["dy"]))
    _, yo = oracle.linear_fwd(c["x"], c["w"], None, 0, 4, 0)
    _, dWo, _ = oracle.linear_bwd(c["dy"], c["x"], c["w"], None, 0, 4, 0)
    assert_close(to_f64(y), yo, "Y")
    g = flat.grad
    assert_close(to_f64(g[off:off + N * K]).reshape(N, K), dWo, "dW in the flat gradient")
    assert float(g[:off].abs().max()) == 0.0 and float(g[off + N * K:].abs().max()) == 0.0


def test_module_argument_errors(P):
    from paper_2209_13258_b200.nn import SplitLinear
    with pytest.raises(ValueError):
        SplitLinear(100, 64)
    with pytest.raises(P.OsdpError):
        SplitLinear(64, 64, k_split=100)
    m = SplitLinear(64, 64)
    with pytest.raises(TypeError):
        m(torch.zeros(8, 64, device="cuda"))
    with pytest.raises(RuntimeError):
        m(torch.zeros(8, 64, dtype=torch.bfloat16))


@pytest.mark.parametrize("k,recompute", [(1, False), (4, False), (4, True), (3, True)])
def test_mlp_module(P, k, recompute):
    """SplitMLP through autograd: forward, dX, the flat parameter's gradient (dW1 then dW2) and both bias
    gradients against the oracle; with recomputation nothing of size [M, ffn] is saved for the backward."""
    from paper_2209_13258_b200.nn import SplitMLP
    B_, S, H, F = 2, 150, 264, 1032
    if P.osdp_slice_range(F, k, 0)[0] != 0:
        pytest.skip("invalid split")
    c = inputs.mlp_case(B_ * S, H, F, w_std=0.05, bias_std=0.1, layer=13)
    m = SplitMLP(H, F, bias=True, k_split=k, recompute=recompute)
    with torch.no_grad():
        m.w1.copy_(to_dev(c["w1"]))
        m.w2.copy_(to_dev(c["w2"]))
        m.b1.copy_(to_dev(c["b1"]))
        m.b2.copy_(to_dev(c["b2"]))
    x = to_dev(c["x"]).view(B_, S, H).requires_grad_(True)
    y = m(x)
    assert y.shape == (B_, S, H) and y.dtype == torch.bfloat16
    saved = [t for t in y.grad_fn.saved_tensors if t.numel() == B_ * S * F]
    assert len(saved) == (0 if recompute else 1)
    y.backward(to_dev(c["dy"]).view(B_, S, H))
    _, yo = oracle.mlp_fwd(c["x"], c["w1"], c["b1"], c["w2"], c["b2"], oracle.ACT_GELU_TANH, k)
    dXo, dW1o, db1o, dW2o, db2o = oracle.mlp_bwd(c["dy"], c["x"], c["w1"], c["b1"], c["w2"], oracle.ACT_GELU_TANH, k)
    assert_close(to_f64(y).reshape(-1, H), yo, "Y")
    assert_close(to_f64(x.grad).reshape(-1, H), dXo, "dX")
    g = m.flat_param.grad
    assert_close(to_f64(g[:H * F]).reshape(F, H), dW1o, "dW1")
    assert_close(to_f64(g[H * F:]).reshape(H, F), dW2o, "dW2")
    assert_close(to_f64(m.b1.grad), db1o, "db1")
    assert_close(to_f64(m.b2.grad), db2o, "db2")


def test_mlp_module_argument_errors(P):
    from paper_2209_13258_b200.nn import SplitMLP
    with pytest.raises(ValueError):
        SplitMLP(100, 64)
    with pytest.raises(P.OsdpError):
        SplitMLP(64, 256, k_split=100)
    m = SplitMLP(64, 256)
    with pytest.raises(TypeError):
        m(torch.zeros(8, 64, device="cuda"))
    with pytest.raises(RuntimeError):
        m(torch.zeros(8, 64, dtype=torch.bfloat16))
