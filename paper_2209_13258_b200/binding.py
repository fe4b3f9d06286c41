"""ctypes binding with the same names as the C ABI in include/osdp.h (argument marshalling only).

Tensor arguments may be torch CUDA tensors (their data pointer is passed) or integers
(raw device addresses) or None.  ``stream`` may be a torch.cuda.Stream, an integer handle or
None (torch's current stream).  Functions return the library's status code; ``check=True``
raises OsdpError on a non-zero status instead.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))

SPLIT_OUT, SPLIT_RED = 0, 1
ACT_NONE, ACT_GELU_TANH, ACT_GELU_ERF = 0, 1, 2
DTYPE_BF16, DTYPE_FP32 = 0, 1
OP_LINEAR_FWD, OP_LINEAR_BWD, OP_MLP_FWD, OP_MLP_BWD = 0, 1, 2, 3
FLAG_ACCUMULATE_DW, FLAG_CARRY_BF16, FLAG_RECOMPUTE, FLAG_PAIR_SLICES, FLAG_SLICE_MAJOR = 1, 2, 4, 8, 16

EXPORTS = [
    "osdp_version", "osdp_status_string", "osdp_last_cuda_error", "osdp_slice_range",
    "osdp_split_linear_workspace_bytes", "osdp_split_linear_fwd", "osdp_split_linear_fwd_slice",
    "osdp_split_linear_bwd", "osdp_split_linear_bwd_slice", "osdp_split_mlp_fwd", "osdp_split_mlp_bwd",
    "osdp_read_device_status", "osdp_bias_grad_noalloc", "osdp_debug_wait_probe", "osdp_suggest_granularity",
    "osdp_zdp_shard_layout", "osdp_zdp_linear_fwd_slice", "osdp_zdp_linear_bwd_slice",
    "osdp_plan_cost", "osdp_plan_search", "osdp_plan_expand_slices", "osdp_plan_search_granularity",
    "osdp_split_linear_fwd_f8", "osdp_split_linear_bwd_f8", "osdp_zdp_linear_bwd_slice_scatter",
    "osdp_zdp_mlp_fwd_slice", "osdp_zdp_mlp_bwd_slice",
]

_lib = None


class OsdpError(RuntimeError):
    def __init__(self, status, where=""):
        self.status = status
        msg = osdp_status_string(status)
        if status == 7:
            msg += " (cuda error %d)" % osdp_last_cuda_error()
        super().__init__("%s: %s" % (where, msg) if where else msg)


def lib_path() -> str:
    return os.path.join(HERE, "libosdp.so")


def lib():
    """Loads libosdp.so (built in-tree by paper_2209_13258_b200/build.py).  No fallback."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise OSError("%s is missing: run `python -m paper_2209_13258_b200.build` (needs nvcc); "
                          "there is no CPU fallback" % path)
        L = ctypes.CDLL(path)
        vp, i64, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
        L.osdp_version.restype = ci
        L.osdp_status_string.restype = ctypes.c_char_p
        L.osdp_status_string.argtypes = [ci]
        L.osdp_last_cuda_error.restype = ci
        L.osdp_slice_range.argtypes = [i64, ci, ci, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.osdp_split_linear_workspace_bytes.argtypes = [i64, i64, i64, ci, ci, ci, ci, ci, ctypes.POINTER(sz)]
        fwd = [vp, vp, i64, vp, i64, i64, i64, ci, ci, ci, ci]
        L.osdp_split_linear_fwd.argtypes = fwd + [vp, vp, vp, sz, vp]
        L.osdp_split_linear_fwd_slice.argtypes = fwd + [ci, vp, vp, vp, sz, vp]
        bwd = [vp, vp, vp, i64, vp, i64, i64, i64, ci, ci, ci]
        L.osdp_split_linear_bwd.argtypes = bwd + [vp, vp, i64, ci, ci, vp, vp, sz, vp]
        L.osdp_split_linear_bwd_slice.argtypes = bwd + [ci, vp, vp, i64, ci, ci, vp, vp, sz, vp]
        L.osdp_split_mlp_fwd.argtypes = [vp, vp, i64, vp, i64, vp, i64, i64, i64, ci, ci, ci, vp, vp, vp, sz, vp]
        L.osdp_split_mlp_bwd.argtypes = [vp, vp, vp, i64, vp, i64, vp, i64, i64, i64, ci, ci, vp, vp, i64, i64, ci,
                                         ci, vp, vp, vp, sz, vp]
        L.osdp_read_device_status.argtypes = [vp, ctypes.POINTER(ci), vp]
        L.osdp_bias_grad_noalloc.argtypes = [vp, i64, i64, vp, vp]
        L.osdp_debug_wait_probe.argtypes = [vp, i64, vp]
        L.osdp_suggest_granularity.argtypes = [i64, i64, i64, ci, ci, ci, ci, sz, ci, ctypes.POINTER(ci)]
        p64 = ctypes.POINTER(i64)
        L.osdp_zdp_shard_layout.argtypes = [i64, i64, ci, ci, ci, ci, p64, p64, p64, p64]
        L.osdp_zdp_linear_fwd_slice.argtypes = [vp, vp, i64, vp, i64, i64, i64, ci, ci, ci, ci, ci, vp, vp, vp, sz, vp]
        L.osdp_zdp_linear_bwd_slice.argtypes = [vp, vp, vp, i64, vp, i64, i64, i64, ci, ci, ci, ci, vp, vp, i64, ci,
                                                ci, vp, vp, sz, vp]
        pd, pu8, dbl = ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_uint8), ctypes.c_double
        L.osdp_plan_cost.argtypes = [pd, ci, ci, dbl, dbl, pu8, ci, pd, pd]
        L.osdp_plan_search.argtypes = [pd, ci, ci, dbl, dbl, dbl, ci, i64, pu8, ctypes.POINTER(ci), pd, p64]
        L.osdp_plan_expand_slices.argtypes = [pd, ci, dbl, pd]
        pci = ctypes.POINTER(ci)
        L.osdp_plan_search_granularity.argtypes = [pd, ci, pci, pci, pd, ci, dbl, dbl, dbl, dbl, ci, i64, pci, pci, pci, pd,
                                                   p64]
        f32 = ctypes.c_float
        pvp = ctypes.POINTER(vp)
        L.osdp_zdp_mlp_fwd_slice.argtypes = [vp, vp, vp, i64, vp, vp, i64, i64, i64, ci, ci, ci, ci, vp, vp, vp, sz, vp]
        L.osdp_zdp_mlp_bwd_slice.argtypes = [vp, vp, vp, vp, i64, vp, vp, i64, i64, i64, ci, ci, ci, vp, vp, vp, i64,
                                             pvp, pvp, ci, ci, ci, vp, vp, vp, sz, vp]
        L.osdp_zdp_linear_bwd_slice_scatter.argtypes = [vp, vp, vp, i64, vp, i64, i64, i64, ci, ci, ci, ci, vp,
                                                        ctypes.POINTER(vp), ci, ci, ci, vp, vp, sz, vp]
        L.osdp_split_linear_fwd_f8.argtypes = [vp, vp, i64, f32, vp, i64, i64, i64, ci, ci, ci, ci, vp, vp, vp, sz, vp]
        L.osdp_split_linear_bwd_f8.argtypes = [vp, vp, vp, i64, f32, f32, i64, i64, i64, ci, ci, vp, vp, i64, ci, ci,
                                               vp, sz, vp]
        for name in EXPORTS:
            getattr(L, name)
            if name not in ("osdp_status_string",):
                getattr(L, name).restype = ci
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    return ctypes.c_void_p(t.data_ptr())


def _stream(s):
    if s is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(s, int):
        return ctypes.c_void_p(s)
    return ctypes.c_void_p(s.cuda_stream)


def _ws(ws):
    if ws is None:
        return None, 0
    if isinstance(ws, tuple):
        return ctypes.c_void_p(ws[0]), int(ws[1])
    return ctypes.c_void_p(ws.data_ptr()), ws.numel() * ws.element_size()


def _ret(rc, check, where):
    if check and rc != 0:
        raise OsdpError(rc, where)
    return rc


def osdp_version() -> int:
    return lib().osdp_version()


def osdp_status_string(status: int) -> str:
    return lib().osdp_status_string(int(status)).decode()


def osdp_last_cuda_error() -> int:
    return lib().osdp_last_cuda_error()


def osdp_slice_range(D, k_split, slice_idx):
    """Returns (status, begin, end)."""
    b, e = ctypes.c_int64(), ctypes.c_int64()
    rc = lib().osdp_slice_range(int(D), int(k_split), int(slice_idx), ctypes.byref(b), ctypes.byref(e))
    return rc, b.value, e.value


def osdp_split_linear_workspace_bytes(M, N, K, k_split, split_dim, act, op, flags=0):
    """Returns (status, bytes)."""
    n = ctypes.c_size_t()
    rc = lib().osdp_split_linear_workspace_bytes(int(M), int(N), int(K), int(k_split), int(split_dim), int(act),
                                                 int(op), int(flags), ctypes.byref(n))
    return rc, n.value


def new_workspace(nbytes: int, device="cuda"):
    """A zeroed torch byte tensor usable as `ws` (torch allocations are 512-byte aligned)."""
    import torch
    return torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def osdp_split_linear_fwd(x, w_flat, w_offset, bias, M, N, K, k_split, split_dim, act, out, z_save, ws,
                          stream=None, check=False, flags=0):
    wp, wn = _ws(ws)
    rc = lib().osdp_split_linear_fwd(_ptr(x), _ptr(w_flat), int(w_offset), _ptr(bias), int(M), int(N), int(K),
                                     int(k_split), int(split_dim), int(act), int(flags), _ptr(out), _ptr(z_save),
                                     wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_split_linear_fwd")


def osdp_split_linear_fwd_slice(x, w_flat, w_offset, bias, M, N, K, k_split, split_dim, act, slice_idx, out,
                                z_save, ws, stream=None, check=False, flags=0):
    wp, wn = _ws(ws)
    rc = lib().osdp_split_linear_fwd_slice(_ptr(x), _ptr(w_flat), int(w_offset), _ptr(bias), int(M), int(N), int(K),
                                           int(k_split), int(split_dim), int(act), int(flags), int(slice_idx),
                                           _ptr(out), _ptr(z_save), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_split_linear_fwd_slice")


def osdp_split_linear_bwd(dy, x, w_flat, w_offset, z_saved, M, N, K, k_split, split_dim, act, dx, dw_flat,
                          dw_offset, dw_dtype, flags, dbias, ws, stream=None, check=False):
    wp, wn = _ws(ws)
    rc = lib().osdp_split_linear_bwd(_ptr(dy), _ptr(x), _ptr(w_flat), int(w_offset), _ptr(z_saved), int(M), int(N),
                                     int(K), int(k_split), int(split_dim), int(act), _ptr(dx), _ptr(dw_flat),
                                     int(dw_offset), int(dw_dtype), int(flags), _ptr(dbias), wp, wn,
                                     _stream(stream))
    return _ret(rc, check, "osdp_split_linear_bwd")


def osdp_split_linear_bwd_slice(dy, x, w_flat, w_offset, z_saved, M, N, K, k_split, split_dim, act, slice_idx, dx,
                                dw_flat, dw_offset, dw_dtype, flags, dbias, ws, stream=None, check=False):
    wp, wn = _ws(ws)
    rc = lib().osdp_split_linear_bwd_slice(_ptr(dy), _ptr(x), _ptr(w_flat), int(w_offset), _ptr(z_saved), int(M),
                                           int(N), int(K), int(k_split), int(split_dim), int(act), int(slice_idx),
                                           _ptr(dx), _ptr(dw_flat), int(dw_offset), int(dw_dtype), int(flags),
                                           _ptr(dbias), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_split_linear_bwd_slice")


def osdp_split_mlp_fwd(x, w_flat, off_w1, b1, off_w2, b2, M, hidden, ffn, k_split, act, out, z1_save, ws,
                       stream=None, check=False, flags=0):
    wp, wn = _ws(ws)
    rc = lib().osdp_split_mlp_fwd(_ptr(x), _ptr(w_flat), int(off_w1), _ptr(b1), int(off_w2), _ptr(b2), int(M),
                                  int(hidden), int(ffn), int(k_split), int(act), int(flags), _ptr(out),
                                  _ptr(z1_save), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_split_mlp_fwd")


def osdp_split_mlp_bwd(dy, x, w_flat, off_w1, off_w2, z1_saved, M, hidden, ffn, k_split, act, dx, dw_flat,
                       dw_off_w1, dw_off_w2, dw_dtype, flags, db1, db2, ws, stream=None, check=False, b1=None):
    """b1 is only read with FLAG_RECOMPUTE (z1_saved may then be None)."""
    wp, wn = _ws(ws)
    rc = lib().osdp_split_mlp_bwd(_ptr(dy), _ptr(x), _ptr(w_flat), int(off_w1), _ptr(b1), int(off_w2),
                                  _ptr(z1_saved), int(M),
                                  int(hidden), int(ffn), int(k_split), int(act), _ptr(dx), _ptr(dw_flat),
                                  int(dw_off_w1), int(dw_off_w2), int(dw_dtype), int(flags), _ptr(db1),
                                  _ptr(db2), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_split_mlp_bwd")


def osdp_read_device_status(ws, stream=None):
    """Returns (status of the call, device status)."""
    wp, _ = _ws(ws)
    st = ctypes.c_int(0)
    rc = lib().osdp_read_device_status(wp, ctypes.byref(st), _stream(stream))
    return rc, st.value


def osdp_bias_grad_noalloc(dy, M, N, dbias, stream=None, check=False):
    """dbias[n] = sum_m dy[m,n] using the library's built-in scratch: for callers that cannot
    allocate device memory (allocator callbacks, hosts that own all device memory, loops that must
    not touch the allocator).  Limit ceil(M/1024) * N <= 2**20; calls on one GPU must not overlap."""
    rc = lib().osdp_bias_grad_noalloc(_ptr(dy), int(M), int(N), _ptr(dbias), _stream(stream))
    return _ret(rc, check, "osdp_bias_grad_noalloc")


def osdp_debug_wait_probe(ws, limit_us, stream=None, check=False):
    """Launches the bounded-wait diagnostic: a wait that nothing satisfies ends after limit_us with the
    device status word set (read it with osdp_read_device_status)."""
    wp, _ = _ws(ws)
    rc = lib().osdp_debug_wait_probe(wp, int(limit_us), _stream(stream))
    return _ret(rc, check, "osdp_debug_wait_probe")


def osdp_suggest_granularity(M, N, K, split_dim, act, op, flags, budget_bytes, max_k=64):
    """Returns (status, k): the smallest valid k <= max_k whose workspace fits budget_bytes."""
    k = ctypes.c_int(0)
    rc = lib().osdp_suggest_granularity(int(M), int(N), int(K), int(split_dim), int(act), int(op), int(flags),
                                        int(budget_bytes), int(max_k), ctypes.byref(k))
    return rc, k.value


def osdp_zdp_shard_layout(N, K, k_split, split_dim, world, slice_idx):
    """Returns (status, slice_elems, shard_elems, shard_offset, ld) for one slice of a sharded operator."""
    a, b, c, d = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    rc = lib().osdp_zdp_shard_layout(int(N), int(K), int(k_split), int(split_dim), int(world), int(slice_idx),
                                     ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(d))
    return rc, a.value, b.value, c.value, d.value


def osdp_zdp_linear_fwd_slice(x, w_slice, ld_w, bias, M, N, K, k_split, split_dim, act, slice_idx, out, z_save, ws,
                              stream=None, check=False, flags=0):
    wp, wn = _ws(ws)
    rc = lib().osdp_zdp_linear_fwd_slice(_ptr(x), _ptr(w_slice), int(ld_w), _ptr(bias), int(M), int(N), int(K),
                                         int(k_split), int(split_dim), int(act), int(flags), int(slice_idx),
                                         _ptr(out), _ptr(z_save), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_zdp_linear_fwd_slice")


def osdp_zdp_linear_bwd_slice(dy, x, w_slice, ld_w, z_saved, M, N, K, k_split, split_dim, act, slice_idx, dx,
                              dw_slice, ld_dw, dw_dtype, flags, dbias, ws, stream=None, check=False):
    wp, wn = _ws(ws)
    rc = lib().osdp_zdp_linear_bwd_slice(_ptr(dy), _ptr(x), _ptr(w_slice), int(ld_w), _ptr(z_saved), int(M), int(N),
                                         int(K), int(k_split), int(split_dim), int(act), int(slice_idx), _ptr(dx),
                                         _ptr(dw_slice), int(ld_dw), int(dw_dtype), int(flags), _ptr(dbias), wp, wn,
                                         _stream(stream))
    return _ret(rc, check, "osdp_zdp_linear_bwd_slice")


def _ops_array(ops):
    flat = [float(v) for op in ops for v in op]
    if len(flat) != 5 * len(ops):
        raise ValueError("an operator is (model, act, extra, S, gamma)")
    return (ctypes.c_double * len(flat))(*flat)


def osdp_plan_cost(ops, world, alpha, beta, modes, batch):
    """Returns (status, memory, time) of one plan; ops = [(model, act, extra, S, gamma), ...], modes 0 DP / 1 ZDP."""
    m, t = ctypes.c_double(), ctypes.c_double()
    md = (ctypes.c_uint8 * len(ops))(*[int(v) for v in modes])
    rc = lib().osdp_plan_cost(_ops_array(ops), len(ops), int(world), float(alpha), float(beta), md, int(batch),
                              ctypes.byref(m), ctypes.byref(t))
    return rc, m.value, t.value


def osdp_plan_search(ops, world, alpha, beta, mem_limit, max_batch, max_nodes=0):
    """Returns (status, modes, batch, time_per_sample, nodes_visited)."""
    md = (ctypes.c_uint8 * len(ops))()
    b, t, nodes = ctypes.c_int(), ctypes.c_double(), ctypes.c_int64()
    rc = lib().osdp_plan_search(_ops_array(ops), len(ops), int(world), float(alpha), float(beta), float(mem_limit),
                                int(max_batch), int(max_nodes), md, ctypes.byref(b), ctypes.byref(t),
                                ctypes.byref(nodes))
    return rc, tuple(md), b.value, t.value, nodes.value


def osdp_plan_expand_slices(op, k, overhead=0.0):
    """Returns (status, [k slice operators])."""
    out = (ctypes.c_double * (5 * max(int(k), 1)))()
    rc = lib().osdp_plan_expand_slices((ctypes.c_double * 5)(*[float(v) for v in op]), int(k), float(overhead), out)
    return rc, [tuple(out[5 * s:5 * s + 5]) for s in range(max(int(k), 1))] if rc == 0 else []


def osdp_plan_search_granularity(ops, candidates, world, alpha, beta, mem_limit, max_batch, max_nodes=0,
                                 surge_factor=0.0):
    """candidates[i] = [(k, overhead), ...] allowed for operator i.  Returns (status, ks, dp_slices, batch,
    time_per_sample, nodes_visited): ks[i] slices for operator i, the first dp_slices[i] of them in DP.
    surge_factor * (largest gathered slice among operators with a ZDP slice) counts against mem_limit."""
    n = len(ops)
    if len(candidates) != n:
        raise ValueError("one candidate list per operator")
    begin, ks, ov = [0], [], []
    for c in candidates:
        for k, o in c:
            ks.append(int(k))
            ov.append(float(o))
        begin.append(len(ks))
    ci = ctypes.c_int
    k_out, dp = (ci * n)(), (ci * n)()
    b, t, nodes = ci(), ctypes.c_double(), ctypes.c_int64()
    rc = lib().osdp_plan_search_granularity(_ops_array(ops), n, (ci * len(begin))(*begin), (ci * max(len(ks), 1))(*ks),
                                            (ctypes.c_double * max(len(ov), 1))(*ov), int(world), float(alpha),
                                            float(beta), float(mem_limit), float(surge_factor), int(max_batch),
                                            int(max_nodes), k_out, dp,
                                            ctypes.byref(b), ctypes.byref(t), ctypes.byref(nodes))
    return rc, list(k_out), list(dp), b.value, t.value, nodes.value


def osdp_split_linear_fwd_f8(x8, w8_flat, w_offset, scale, bias, M, N, K, k_split, split_dim, act, out, z_save, ws,
                             stream=None, check=False, flags=0):
    wp, wn = _ws(ws)
    rc = lib().osdp_split_linear_fwd_f8(_ptr(x8), _ptr(w8_flat), int(w_offset), float(scale), _ptr(bias), int(M),
                                        int(N), int(K), int(k_split), int(split_dim), int(act), int(flags), _ptr(out),
                                        _ptr(z_save), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_split_linear_fwd_f8")


def osdp_split_linear_bwd_f8(dy8, x8, w8_flat, w_offset, scale_dx, scale_dw, M, N, K, k_split, split_dim, dx, dw_flat,
                             dw_offset, dw_dtype, flags, ws, stream=None, check=False):
    wp, wn = _ws(ws)
    rc = lib().osdp_split_linear_bwd_f8(_ptr(dy8), _ptr(x8), _ptr(w8_flat), int(w_offset), float(scale_dx),
                                        float(scale_dw), int(M), int(N), int(K), int(k_split), int(split_dim),
                                        _ptr(dx), _ptr(dw_flat), int(dw_offset), int(dw_dtype), int(flags), wp, wn,
                                        _stream(stream))
    return _ret(rc, check, "osdp_split_linear_bwd_f8")


def osdp_zdp_linear_bwd_slice_scatter(dy, x, w_slice, ld_w, z_saved, M, N, K, k_split, split_dim, act, slice_idx, dx,
                                      dw_peers, dw_dtype, flags, dbias, ws, stream=None, check=False):
    """dw_peers: one tensor (or raw device address) per rank: where that rank keeps its part of this slice."""
    wp, wn = _ws(ws)
    arr = (ctypes.c_void_p * len(dw_peers))(*[t if isinstance(t, int) else t.data_ptr() for t in dw_peers])
    rc = lib().osdp_zdp_linear_bwd_slice_scatter(_ptr(dy), _ptr(x), _ptr(w_slice), int(ld_w), _ptr(z_saved), int(M),
                                                 int(N), int(K), int(k_split), int(split_dim), int(act),
                                                 int(slice_idx), _ptr(dx), arr, len(dw_peers), int(dw_dtype),
                                                 int(flags), _ptr(dbias), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_zdp_linear_bwd_slice_scatter")


def _ptr_array(ts):
    if ts is None:
        return None
    return (ctypes.c_void_p * len(ts))(*[t if isinstance(t, int) else t.data_ptr() for t in ts])


def osdp_zdp_mlp_fwd_slice(x, w1_slice, w2_slice, ld_w2, b1, b2, M, hidden, ffn, k_split, act, slice_idx, out, z1_save,
                           ws, stream=None, check=False, flags=0):
    wp, wn = _ws(ws)
    rc = lib().osdp_zdp_mlp_fwd_slice(_ptr(x), _ptr(w1_slice), _ptr(w2_slice), int(ld_w2), _ptr(b1), _ptr(b2), int(M),
                                      int(hidden), int(ffn), int(k_split), int(act), int(flags), int(slice_idx),
                                      _ptr(out), _ptr(z1_save), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_zdp_mlp_fwd_slice")


def osdp_zdp_mlp_bwd_slice(dy, x, w1_slice, w2_slice, ld_w2, b1, z1_saved, M, hidden, ffn, k_split, act, slice_idx, dx,
                           dw1_slice, dw2_slice, ld_dw2, dw1_peers, dw2_peers, dw_dtype, flags, db1, db2, ws,
                           stream=None, check=False):
    """dw1_peers / dw2_peers: None, or one tensor (or device address) per rank for the epilogue's scatter."""
    wp, wn = _ws(ws)
    world = len(dw1_peers) if dw1_peers is not None else 0
    rc = lib().osdp_zdp_mlp_bwd_slice(_ptr(dy), _ptr(x), _ptr(w1_slice), _ptr(w2_slice), int(ld_w2), _ptr(b1),
                                      _ptr(z1_saved), int(M), int(hidden), int(ffn), int(k_split), int(act),
                                      int(slice_idx), _ptr(dx), _ptr(dw1_slice), _ptr(dw2_slice), int(ld_dw2),
                                      _ptr_array(dw1_peers), _ptr_array(dw2_peers), world, int(dw_dtype), int(flags),
                                      _ptr(db1), _ptr(db2), wp, wn, _stream(stream))
    return _ret(rc, check, "osdp_zdp_mlp_bwd_slice")
