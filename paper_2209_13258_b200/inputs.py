"""Seeded synthetic inputs shared by the CPU oracle tests and the CUDA parity tests.

This module holds none of the split-linear arithmetic: it only draws numbers and
rounds them to bfloat16 bit patterns, so that the oracle and the CUDA path can be
fed the very same bits.  The generator is counter based (element i of stream t
depends only on (seed, t, i)), so the order in which tensors are drawn, and the
chunking used to draw them, never changes a value.

Recipe: two 64-bit hashes per element -> two uniforms -> one Box-Muller normal
(fp64) -> mean + std * z -> fp32 (round to nearest even) -> bf16 (round to nearest
even).  "N(0, 0.02)" in the workload descriptions is read as a standard deviation.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 220913258

# stream ids: 16 * layer + one of these
STREAM_X, STREAM_W, STREAM_B, STREAM_DY, STREAM_W2, STREAM_B2 = 1, 2, 3, 4, 5, 6

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = np.uint64(0x9E3779B97F4A7C15)


def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix64(np.array([np.uint64(seed) * _GOLD + np.uint64(stream)], dtype=np.uint64))
    return k[0]


def normal_f64(n: int, stream: int, seed: int = BASE_SEED, start: int = 0) -> np.ndarray:
    """n standard normals (fp64), elements [start, start+n) of the given stream."""
    out = np.empty(n, dtype=np.float64)
    key = _key(seed, stream)
    chunk = 1 << 22
    with np.errstate(over="ignore"):
        for lo in range(0, n, chunk):
            hi = min(n, lo + chunk)
            i = np.arange(start + lo, start + hi, dtype=np.uint64)
            a = _mix64(key + np.uint64(2) * i)
            b = _mix64(key + np.uint64(2) * i + np.uint64(1))
            u1 = ((a >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
            u2 = (b >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
            out[lo:hi] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest even); returns the uint16 bit patterns."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = bits + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) exactly to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, std: float, stream: int, seed: int = BASE_SEED, mean: float = 0.0) -> np.ndarray:
    """bf16 bit patterns (uint16 array of the given shape) of mean + std * N(0,1)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    chunk = 1 << 22
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        z = normal_f64(hi - lo, stream, seed, start=lo)
        out[lo:hi] = f32_to_bf16_bits((mean + std * z).astype(np.float32))
    return out.reshape(shape)


def normal_f32(shape, std: float, stream: int, seed: int = BASE_SEED, mean: float = 0.0) -> np.ndarray:
    """fp32 values mean + std * N(0,1) (used for biases, which stay fp32)."""
    n = int(np.prod(shape))
    return (mean + std * normal_f64(n, stream, seed)).astype(np.float32).reshape(shape)


def _e4m3_table() -> np.ndarray:
    """Values of the 127 non-negative finite e4m3 codes 0x00..0x7E, ascending (code = index)."""
    codes = np.arange(127)
    e, m = codes >> 3, codes & 7
    return np.where(e == 0, m / 8.0 * 2.0 ** -6, (1.0 + m / 8.0) * 2.0 ** (e.astype(np.float64) - 7.0))


def f32_to_e4m3_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to fp8 e4m3 (nearest, ties to the even code, magnitudes above 448 saturate to 448);
    returns the uint8 bit patterns.  Table search: the nearest of the 127 finite magnitudes."""
    x = np.ascontiguousarray(x, dtype=np.float32).astype(np.float64)
    tab = _e4m3_table()
    a = np.minimum(np.abs(x), 448.0)
    lo = np.clip(np.searchsorted(tab, a, side="right") - 1, 0, 126)
    hi = np.minimum(lo + 1, 126)
    dlo, dhi = a - tab[lo], tab[hi] - a
    pick_hi = (dhi < dlo) | ((dhi == dlo) & (hi % 2 == 0) & (hi != lo))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return code | (np.signbit(x).astype(np.uint8) << np.uint8(7))


def normal_e4m3(shape, std: float, stream: int, seed: int = BASE_SEED):
    """fp8 e4m3 bit patterns (uint8) of std * N(0,1) / scale and the per-tensor fp32 scale = max|x| / 448, so
    that value = scale * e4m3(bits)."""
    n = int(np.prod(shape))
    z = (std * normal_f64(n, stream, seed)).astype(np.float32)
    scale = np.float32(max(float(np.max(np.abs(z))), 1e-30) / 448.0)
    return f32_to_e4m3_bits(z / scale).reshape(shape), float(scale)


def linear_case_e4m3(M: int, N: int, K: int, *, x_std=1.0, w_std=0.02, dy_std=1.0, bias_std=0.0,
                     layer: int = 0, seed: int = BASE_SEED, w_offset: int = 0, flat_pad: int = 0):
    """linear_case with fp8 e4m3 operands: x, dy, w, w_flat are uint8 bit patterns with per-tensor scales
    sx, sdy, sw (value = scale * e4m3(bits)); bias stays fp32."""
    x, sx = normal_e4m3((M, K), x_std, stream_id(layer, STREAM_X), seed)
    dy, sdy = normal_e4m3((M, N), dy_std, stream_id(layer, STREAM_DY), seed)
    w, sw = normal_e4m3((N, K), w_std, stream_id(layer, STREAM_W), seed)
    flat, _ = normal_e4m3((w_offset + N * K + flat_pad,), 1.0, stream_id(layer, 15), seed)
    flat[w_offset:w_offset + N * K] = w.reshape(-1)
    bias = normal_f32((N,), bias_std, stream_id(layer, STREAM_B), seed) if bias_std > 0.0 else np.zeros((N,), np.float32)
    return {"x": x, "dy": dy, "w": w, "w_flat": flat, "w_offset": w_offset, "bias": bias, "sx": sx, "sdy": sdy,
            "sw": sw, "M": M, "N": N, "K": K}


def stream_id(layer: int, which: int) -> int:
    return 16 * layer + which


def align_up(v: int, a: int) -> int:
    return (v + a - 1) // a * a


def linear_case(M: int, N: int, K: int, *, x_std=1.0, w_std=0.02, dy_std=1.0, bias_std=0.0,
                layer: int = 0, seed: int = BASE_SEED, w_offset: int = 0, flat_pad: int = 0):
    """One linear layer's tensors.

    Returns a dict with bf16 bit patterns: x [M,K], dy [M,N], w_flat (1-D flat parameter
    buffer of w_offset + N*K + flat_pad elements holding W [N,K] row-major at element
    offset w_offset; the elements outside W are filled from another stream so that a
    wrong offset shows), and bias [N] fp32.
    """
    x = normal_bf16((M, K), x_std, stream_id(layer, STREAM_X), seed)
    dy = normal_bf16((M, N), dy_std, stream_id(layer, STREAM_DY), seed)
    w = normal_bf16((N, K), w_std, stream_id(layer, STREAM_W), seed)
    flat = normal_bf16((w_offset + N * K + flat_pad,), 1.0, stream_id(layer, 15), seed)
    flat[w_offset:w_offset + N * K] = w.reshape(-1)
    if bias_std > 0.0:
        bias = normal_f32((N,), bias_std, stream_id(layer, STREAM_B), seed)
    else:
        bias = np.zeros((N,), dtype=np.float32)
    return {"x": x, "dy": dy, "w": w, "w_flat": flat, "w_offset": w_offset, "bias": bias,
            "M": M, "N": N, "K": K}


def mlp_case(M: int, hidden: int, ffn: int, *, x_std=1.0, w_std=0.02, dy_std=1.0, bias_std=0.02,
             layer: int = 0, seed: int = BASE_SEED):
    """Transformer MLP block tensors, weights packed in one flat bf16 buffer.

    Flat layout (element offsets, each 8-element = 16-byte aligned):
    [W1 ffn x hidden | W2 hidden x ffn].  Biases b1 [ffn], b2 [hidden] are fp32 arrays of
    their own (a bf16 flat buffer cannot hold fp32 values).
    """
    x = normal_bf16((M, hidden), x_std, stream_id(layer, STREAM_X), seed)
    dy = normal_bf16((M, hidden), dy_std, stream_id(layer, STREAM_DY), seed)
    w1 = normal_bf16((ffn, hidden), w_std, stream_id(layer, STREAM_W), seed)
    w2 = normal_bf16((hidden, ffn), w_std, stream_id(layer, STREAM_W2), seed)
    off_w1 = 0
    off_w2 = align_up(off_w1 + ffn * hidden, 8)
    total = align_up(off_w2 + hidden * ffn, 8)
    flat = np.zeros((total,), dtype=np.uint16)
    flat[off_w1:off_w1 + ffn * hidden] = w1.reshape(-1)
    flat[off_w2:off_w2 + hidden * ffn] = w2.reshape(-1)
    if bias_std > 0.0:
        b1 = normal_f32((ffn,), bias_std, stream_id(layer, STREAM_B), seed)
        b2 = normal_f32((hidden,), bias_std, stream_id(layer, STREAM_B2), seed)
    else:
        b1 = np.zeros((ffn,), dtype=np.float32)
        b2 = np.zeros((hidden,), dtype=np.float32)
    return {"x": x, "dy": dy, "w1": w1, "w2": w2, "w_flat": flat, "off_w1": off_w1, "off_w2": off_w2,
            "b1": b1, "b2": b2, "M": M, "hidden": hidden, "ffn": ffn}
