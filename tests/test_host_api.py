"""Host-side behaviour of the C ABI that needs no GPU: the library loads and exports every symbol
the header declares, the slice table matches the hand-computed one, argument checks reject bad
calls before anything is launched, and the workspace plan has the stated shape."""
import os
import re

import pytest

import paper_2209_13258_b200 as P

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "osdp.h")).read()
    declared = set(re.findall(r"\b(osdp_[a-z0-9_]+)\s*\(", hdr))
    assert len(declared) >= 12
    L = P.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert P.osdp_version() == 111
    assert P.osdp_status_string(0) == "ok" and "split" in P.osdp_status_string(3)


def test_slice_range_matches_golden_table():
    path = os.path.join(ROOT, "tests", "golden", "slice_table.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        head, tail = line.split(":")
        D, k = (int(v) for v in head.split())
        want = [tuple(int(v) for v in pair.split(",")) for pair in tail.split()]
        got = [P.osdp_slice_range(D, k, s) for s in range(k)]
        assert [g[0] for g in got] == [0] * k
        assert [(g[1], g[2]) for g in got] == want
    assert P.osdp_slice_range(40, 6, 0)[0] == 3          # empty last slice
    assert P.osdp_slice_range(40, 5, 5)[0] == 3          # slice index out of range
    assert P.osdp_slice_range(40, 0, 0) == (0, 0, 40)    # granularity 0 = unsplit
    assert P.osdp_slice_range(0, 1, 0)[0] == 2


def test_workspace_plan():
    M, N, K = 16384, 8192, 8192
    q = lambda k, split, act, op, fl=0: P.osdp_split_linear_workspace_bytes(M, N, K, k, split, act, op, fl)
    SM = P.FLAG_SLICE_MAJOR
    # forward, all slices in one call: nothing but the status block (a summed output stays in tensor memory)
    assert q(1, 0, 0, P.OP_LINEAR_FWD) == (0, 256)
    assert q(8, 0, 0, P.OP_LINEAR_FWD) == (0, 256)
    assert q(8, 1, 0, P.OP_LINEAR_FWD) == (0, 256)
    # slice-major order / one slice per call: fp32 carry of Y when the reduction dim is split
    assert q(8, 0, 0, P.OP_LINEAR_FWD, SM) == (0, 256)
    assert q(8, 1, 0, P.OP_LINEAR_FWD, SM) == (0, 256 + M * N * 4)
    assert q(8, 1, 0, P.OP_LINEAR_FWD, P.FLAG_PAIR_SLICES) == (0, 256 + M * N * 4)
    assert q(1, 1, 0, P.OP_LINEAR_FWD, SM) == (0, 256)
    # backward: column-sum partials always; fp32 carry of dX when the output dim is split slice-major
    part = 16 * N * 4
    assert q(1, 0, 0, P.OP_LINEAR_BWD) == (0, 256 + part)
    assert q(8, 0, 0, P.OP_LINEAR_BWD) == (0, 256 + part)
    assert q(8, 0, 0, P.OP_LINEAR_BWD, SM) == (0, 256 + M * K * 4 + part)
    assert q(8, 1, 0, P.OP_LINEAR_BWD) == (0, 256 + part)
    assert q(8, 1, 0, P.OP_LINEAR_BWD, SM) == (0, 256 + part)
    # activation backward stages G for one slice (output split; the call then goes slice by slice and
    # carries dX whatever the flags) or whole (reduction split)
    assert q(8, 0, 1, P.OP_LINEAR_BWD)[1] == 256 + M * K * 4 + M * (N // 8) * 2 + part
    assert q(8, 0, 1, P.OP_LINEAR_BWD, SM) == q(8, 0, 1, P.OP_LINEAR_BWD)
    assert q(8, 1, 1, P.OP_LINEAR_BWD)[1] - q(8, 1, 0, P.OP_LINEAR_BWD)[1] == M * N * 2
    # MLP chain: slice-sized intermediates shrink as 1/k
    f = lambda k: P.osdp_split_linear_workspace_bytes(8192, 32768, 8192, k, 0, 1, P.OP_MLP_FWD)[1]
    carry = 8192 * 8192 * 4
    assert f(1) == 256 + 8192 * 32768 * 2
    for k in (2, 4, 8, 16):
        assert f(k) == 256 + carry + 8192 * (32768 // k) * 2
    assert q(8, 1, 0, P.OP_LINEAR_FWD, SM | P.FLAG_CARRY_BF16) == (0, 256)
    assert q(8, 0, 0, P.OP_LINEAR_BWD, SM | P.FLAG_CARRY_BF16) == (0, 256 + part)
    assert P.osdp_split_linear_workspace_bytes(8192, 32768, 8192, 8, 0, 1, P.OP_MLP_FWD, P.FLAG_CARRY_BF16) == (
        0, 256 + 8192 * 4096 * 2)
    assert P.osdp_split_linear_workspace_bytes(8, 8, 8, 1, 0, 0, 0, 32)[0] == 6
    assert P.osdp_split_linear_workspace_bytes(8, 8, 8, 1, 0, 0, P.OP_MLP_FWD, SM)[0] == 6
    assert P.osdp_split_linear_workspace_bytes(8, 8, 8, 1, 0, 0, 9)[0] == 6
    assert P.osdp_split_linear_workspace_bytes(8, 8, 8, 1, 0, 7, 0)[0] == 6
    assert P.osdp_split_linear_workspace_bytes(8, 16, 8, 3, 0, 0, 0)[0] == 3


A = 1 << 20   # a fake, 16-byte aligned "device address": argument checks never dereference it


def _fwd(**kw):
    a = dict(x=A, w_flat=A, w_offset=0, bias=None, M=64, N=64, K=64, k_split=2, split_dim=0, act=0, out=A,
             z_save=None, ws=(A, 1 << 30), stream=0)
    a.update(kw)
    return P.osdp_split_linear_fwd(**a)


def _bwd(**kw):
    a = dict(dy=A, x=A, w_flat=A, w_offset=0, z_saved=None, M=64, N=64, K=64, k_split=2, split_dim=0, act=0,
             dx=A, dw_flat=A, dw_offset=0, dw_dtype=1, flags=0, dbias=A, ws=(A, 1 << 30), stream=0)
    a.update(kw)
    return P.osdp_split_linear_bwd(**a)


def test_forward_argument_checks():
    assert _fwd(x=None) == 1 and _fwd(w_flat=None) == 1 and _fwd(out=None) == 1 and _fwd(ws=None) == 1
    assert _fwd(M=0) == 2 and _fwd(N=-8) == 2 and _fwd(K=1 << 40) == 2
    assert _fwd(N=60) == 4 and _fwd(K=12) == 4
    assert _fwd(w_offset=4) == 4 and _fwd(w_offset=-8) == 4
    assert _fwd(x=A + 2) == 4 and _fwd(out=A + 8) == 4 and _fwd(ws=(A + 16, 1 << 30)) == 4
    assert _fwd(k_split=-1) == 3 and _fwd(k_split=9) == 3 and _fwd(split_dim=2) == 3
    assert _fwd(act=3) == 6
    assert _fwd(split_dim=1, ws=(A, 256)) in (0, 7)     # all slices in one call: the sum stays in tensor memory
    assert _fwd(split_dim=1, ws=(A, 256), flags=P.FLAG_SLICE_MAJOR) == 5   # slice-major: the carry does not fit
    assert P.osdp_split_linear_fwd_slice(A, A, 0, None, 64, 64, 64, 2, 1, 0, 0, A, None, (A, 256), stream=0) == 5
    assert _fwd(split_dim=1, ws=(A, 256), flags=P.FLAG_CARRY_BF16) in (0, 7)   # bf16 running sum: no carry needed
    assert _fwd(flags=P.FLAG_CARRY_BF16, act=1) == 6    # the bf16 running sum excludes an activation ...
    assert _fwd(flags=P.FLAG_CARRY_BF16, z_save=A) == 6  # ... and a saved pre-activation
    assert _fwd(flags=4) == 6 and _fwd(flags=P.FLAG_ACCUMULATE_DW) == 6
    assert _fwd(split_dim=1, flags=P.FLAG_PAIR_SLICES) in (0, 7)
    assert _fwd(split_dim=1, flags=P.FLAG_PAIR_SLICES | P.FLAG_CARRY_BF16) == 6
    assert P.osdp_split_linear_fwd_slice(A, A, 0, None, 64, 64, 64, 2, 1, 0, 0, A, None, (A, 1 << 20), stream=0,
                                         flags=P.FLAG_PAIR_SLICES) == 6
    assert P.osdp_split_linear_fwd_slice(A, A, 0, None, 64, 64, 64, 2, 0, 0, 2, A, None, (A, 1 << 20), stream=0) == 3
    # a well-formed call gets past the checks and fails only because there is no device / fake pointers
    if not _cuda():
        assert _fwd() == 7 and P.osdp_last_cuda_error() != 0


def test_backward_argument_checks():
    assert _bwd(dy=None) == 1 and _bwd(x=None) == 1 and _bwd(w_flat=None) == 1
    assert _bwd(act=1, z_saved=None) == 1
    assert _bwd(dw_dtype=2) == 6
    assert _bwd(dw_offset=12) == 4 and _bwd(dx=A + 4) == 4 and _bwd(dbias=A + 4) == 4
    assert _bwd(k_split=9) == 3
    assert _bwd(ws=(A, 64)) == 5
    assert _bwd(ws=(A, 1024)) in (0, 7) and _bwd(ws=(A, 1024), flags=P.FLAG_SLICE_MAJOR) == 5
    assert _bwd(flags=32) == 6
    # pairing of adjacent slices: all-slices calls only, not together with the bf16 running sum or an activation
    assert _bwd(flags=P.FLAG_PAIR_SLICES) in (0, 7)
    assert _bwd(flags=P.FLAG_PAIR_SLICES | P.FLAG_CARRY_BF16) == 6
    assert _bwd(flags=P.FLAG_PAIR_SLICES, act=1, z_saved=A) == 6
    assert P.osdp_split_linear_bwd_slice(A, A, A, 0, None, 64, 64, 64, 2, 0, 0, 0, A, A, 0, 1, P.FLAG_PAIR_SLICES, A,
                                         (A, 1 << 20), stream=0) == 6
    # with the bf16 running sum the backward needs only the column-sum partials
    assert _bwd(ws=(A, 256 + 64 * 4), flags=P.FLAG_CARRY_BF16) in (0, 7)
    assert P.osdp_split_linear_bwd_slice(A, A, A, 0, None, 64, 64, 64, 2, 0, 0, -1, A, A, 0, 1, 0, A, (A, 1 << 20),
                                         stream=0) == 3


def test_mlp_argument_checks():
    f = lambda **kw: P.osdp_split_mlp_fwd(**dict(dict(x=A, w_flat=A, off_w1=0, b1=None, off_w2=64 * 256, b2=None,
                                                      M=32, hidden=64, ffn=256, k_split=4, act=1, out=A,
                                                      z1_save=None, ws=(A, 1 << 30), stream=0), **kw))
    assert f(x=None) == 1 and f(off_w2=3) == 4 and f(k_split=64) == 3 and f(ws=(A, 256)) == 5 and f(ffn=100) == 4
    b = lambda **kw: P.osdp_split_mlp_bwd(**dict(dict(dy=A, x=A, w_flat=A, off_w1=0, off_w2=64 * 256, z1_saved=A,
                                                      M=32, hidden=64, ffn=256, k_split=4, act=1, dx=A, dw_flat=A,
                                                      dw_off_w1=0, dw_off_w2=64 * 256, dw_dtype=1, flags=0,
                                                      db1=A, db2=A, ws=(A, 1 << 30), stream=0), **kw))
    assert b(z1_saved=None) == 1 and b(dw_dtype=5) == 6 and b(dw_off_w1=4) == 4 and b(ws=(A, 4096)) == 5
    # with recomputation no saved activation is needed, but one more slice-sized buffer is
    assert b(z1_saved=None, flags=P.FLAG_RECOMPUTE) in (0, 7)
    assert b(flags=32) == 6 and b(flags=P.FLAG_SLICE_MAJOR) == 6 and b(flags=P.FLAG_RECOMPUTE, b1=A + 4) == 4
    # small slices with k > 2: two sets of the slice-sized buffers (consecutive slices overlap), so two more here
    plain = P.osdp_split_linear_workspace_bytes(32, 256, 64, 4, 0, 1, P.OP_MLP_BWD)[1]
    assert P.osdp_split_linear_workspace_bytes(32, 256, 64, 4, 0, 1, P.OP_MLP_BWD, P.FLAG_RECOMPUTE)[1] == plain + 2 * 32 * 64 * 2
    plain = P.osdp_split_linear_workspace_bytes(32, 256, 64, 2, 0, 1, P.OP_MLP_BWD)[1]
    assert P.osdp_split_linear_workspace_bytes(32, 256, 64, 2, 0, 1, P.OP_MLP_BWD, P.FLAG_RECOMPUTE)[1] == plain + 32 * 128 * 2
    assert P.osdp_split_linear_workspace_bytes(32, 256, 64, 4, 0, 1, P.OP_MLP_FWD, P.FLAG_RECOMPUTE)[0] == 6


def _cuda():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2209_13258_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "HERE", str(tmp_path))
    with pytest.raises(OSError, match="no CPU fallback"):
        binding.lib()


def test_suggest_granularity():
    # MLP block hidden 8192 / ffn 32768 / 8192 tokens, forward: staging = fp32 carry (268 MB, k > 1) + A_s
    M, H, F = 8192, 8192, 32768
    ws = lambda k, fl=0: P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_FWD, fl)[1]
    sug = lambda budget, fl=0, mk=64: P.osdp_suggest_granularity(M, F, H, 0, 1, P.OP_MLP_FWD, fl, budget, mk)
    assert sug(ws(1)) == (0, 1)                      # the unsplit block fits: do not split
    rc, k = sug(ws(1) - 1)                           # k = 2 needs as much as k = 1 (the carry appears): k = 3 fits
    assert (rc, k) == (0, 3) and ws(2) > ws(1) - 1 >= ws(3)
    rc, k = sug(350 << 20)
    assert rc == 0 and ws(k) <= (350 << 20) and all(ws(j) > (350 << 20) for j in range(1, k) if ws(j))
    assert sug(200 << 20)[0] == 5                    # the k-independent fp32 carry alone is 268 MB
    rc, k = sug(200 << 20, P.FLAG_CARRY_BF16)        # the bf16 running sum removes it
    assert rc == 0 and ws(k, P.FLAG_CARRY_BF16) <= (200 << 20)
    assert sug(1 << 20, mk=8)[0] == 5
    # k values that would leave an empty slice are skipped, not reported as errors
    assert P.osdp_suggest_granularity(64, 40, 64, 0, 0, P.OP_LINEAR_BWD, 0, 1 << 30, 64) == (0, 1)
    assert P.osdp_suggest_granularity(64, 40, 64, 0, 0, P.OP_LINEAR_BWD, 0, 1 << 30, 0)[0] == 3
    assert P.osdp_suggest_granularity(0, 40, 64, 0, 0, P.OP_LINEAR_BWD, 0, 1 << 30, 8)[0] == 2


def test_noalloc_bias_grad_argument_checks():
    # refusals come before anything touches a device
    assert P.osdp_bias_grad_noalloc(A, 65536, 32768, A, stream=0) == 9            # 2^21 partials > 2^20
    assert P.osdp_bias_grad_noalloc(A, 65536 * 1024 + 1, 8, A, stream=0) == 9     # 65537 row chunks: grid limit
    assert P.osdp_bias_grad_noalloc(None, 8, 8, A, stream=0) == 1
    assert P.osdp_bias_grad_noalloc(A, 8, 12, A, stream=0) == 4
    assert P.osdp_bias_grad_noalloc(A, 0, 8, A, stream=0) == 2
    # the regular backward refuses the same row count when a bias gradient is asked for
    assert _bwd(M=65536 * 1024 + 8, dx=None, dw_flat=None) == 2


def test_mlp_backward_staging_sets():
    """Slice-sized buffers of the MLP backward: one set, except two sets for k > 2 when a slice's GEMMs are at
    most one wave of 256 x 256 tiles on 74 CTA pairs (the slices are then pipelined); always ~ 1/k."""
    def parts(M, H, F, k):
        L = -(-(-(-F // k)) // 8) * 8
        chunks = -(-M // 1024)
        carry = M * H * 4 if k > 1 else 0
        sets = 2 if (k > 2 and -(-M // 256) * -(-L // 256) <= 74) else 1
        up = lambda v: -(-v // 256) * 256
        stage = up(M * L * 2) + M * L * 2 if sets == 2 else M * L * 2
        total = 256 + (up(carry) if carry else 0) + 2 * up(stage) + up(chunks * (sets * L + H) * 4)
        return total, sets
    for (M, H, F) in ((4096, 1024, 4096), (8192, 8192, 32768), (8192, 2048, 8192)):
        for k in (1, 2, 4, 8, 16):
            want, sets = parts(M, H, F, k)
            rc, got = P.osdp_split_linear_workspace_bytes(M, F, H, k, 0, 1, P.OP_MLP_BWD)
            assert rc == 0 and got == want, (M, H, F, k, got, want, sets)
    assert parts(4096, 1024, 4096, 8)[1] == 2 and parts(4096, 1024, 4096, 2)[1] == 1
    assert parts(8192, 8192, 32768, 8)[1] == 1 and parts(8192, 8192, 32768, 16)[1] == 1
    assert parts(8192, 2048, 8192, 8)[1] == 1 and parts(8192, 2048, 8192, 16)[1] == 2
    # the forward keeps one set whatever the size
    assert P.osdp_split_linear_workspace_bytes(4096, 4096, 1024, 8, 0, 1, P.OP_MLP_FWD)[1] == \
        256 + 4096 * 1024 * 4 + 4096 * 512 * 2


def test_carry_is_sized_in_boxes_of_32_by_32():
    """The fp32 running sum of a slice-major summed output is stored as 32 x 32 boxes: both extents are padded."""
    up = lambda v, a: -(-v // a) * a
    for (M, N, K) in ((200, 264, 520), (4096, 1024, 4096), (33, 40, 72)):
        # forward under RED, slice-major: status block + carry [M, N] + nothing else
        rc, got = P.osdp_split_linear_workspace_bytes(M, N, K, 3, P.SPLIT_RED, 0, P.OP_LINEAR_FWD, P.FLAG_SLICE_MAJOR)
        assert rc == 0 and got == 256 + up(up(M, 32) * up(N, 32) * 4, 256), (M, N, K, got)
        # default order: the sum stays in tensor memory, no carry
        assert P.osdp_split_linear_workspace_bytes(M, N, K, 3, P.SPLIT_RED, 0, P.OP_LINEAR_FWD, 0) == (0, 256)
        # backward under OUT, slice-major: carry [M, K] + column-sum partials
        rc, got = P.osdp_split_linear_workspace_bytes(M, N, K, 3, P.SPLIT_OUT, 0, P.OP_LINEAR_BWD, P.FLAG_SLICE_MAJOR)
        assert rc == 0 and got == 256 + up(up(M, 32) * up(K, 32) * 4, 256) + up(-(-M // 1024) * N * 4, 256), (M, N, K, got)
