"""The allocation-free bias-gradient entry point.

Some users of the library call it from places where device memory cannot be allocated (an
allocator callback, a host application that has claimed the whole device, a loop that must not
block on the allocator), so they cannot provide the workspace the regular backward needs.
osdp_bias_grad_noalloc serves them from an array built into the library.  This test checks,
through the C ABI, that it returns exactly what the regular entry point returns, on two calls in a
row with different data (the built-in array keeps the first call's contents, which must not leak
into the second), and that it refuses problems larger than the array.  It is collected last so
that a failure here cannot hide the other tests' results."""
import pytest

torch = pytest.importorskip("torch")

pytestmark = pytest.mark.gpu


def test_noalloc_bias_grad_matches_regular_entry_point_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2209_13258_b200 as P
    from paper_2209_13258_b200 import inputs
    from util import assert_close, to_dev, to_f64

    for call, (M, N, layer) in enumerate(((4096, 2048, 50), (1500, 520, 51))):
        c = inputs.linear_case(M, N, 64, layer=layer)
        dy, x, wf = to_dev(c["dy"]), to_dev(c["x"]), to_dev(c["w_flat"])
        # the existing entry point, with a caller-provided workspace
        _, nbytes = P.osdp_split_linear_workspace_bytes(M, N, 64, 1, P.SPLIT_OUT, P.ACT_NONE, P.OP_LINEAR_BWD)
        ws = P.new_workspace(nbytes)
        want = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")
        P.osdp_split_linear_bwd(dy, x, wf, 0, None, M, N, 64, 1, P.SPLIT_OUT, P.ACT_NONE, None, None, 0,
                                P.DTYPE_FP32, 0, want, ws, check=True)
        # the allocation-free entry point: inputs and outputs only
        got = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")
        P.osdp_bias_grad_noalloc(dy, M, N, got, check=True)
        torch.cuda.synchronize()
        assert_close(to_f64(got), to_f64(want), "dbias, call %d" % call, relf_tol=1e-6)
        assert torch.equal(got, want), "call %d differs bitwise" % call
        # and both agree with the definition
        ref = to_f64(dy).sum(axis=0)
        assert_close(to_f64(got), ref, "dbias vs definition", relf_tol=1e-5)


def test_noalloc_rejects_sizes_beyond_the_built_in_scratch():
    import paper_2209_13258_b200 as P
    A = 1 << 20
    # ceil(M/1024) * N = 64 * 32768 = 2^21 > 2^20 partials
    assert P.osdp_bias_grad_noalloc(A, 65536, 32768, A, stream=0) == 9
    assert "scratch" in P.osdp_status_string(9)
    # few columns, very many rows: the partials would fit, but the first pass's grid would not
    assert P.osdp_bias_grad_noalloc(A, 65536 * 1024 + 1, 8, A, stream=0) == 9
    assert P.osdp_bias_grad_noalloc(None, 8, 8, A, stream=0) == 1
    assert P.osdp_bias_grad_noalloc(A, 8, 12, A, stream=0) == 4
    assert P.osdp_bias_grad_noalloc(A, 0, 8, A, stream=0) == 2
