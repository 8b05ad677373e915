"""CPU oracle for the GPTQ int4 matmul - TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``gptq_oracle.c`` (plain C, OpenMP).  Only tests,
the smoke check and the CPU-baseline leg of the benchmark may import this
package; the CUDA product path never does, and this package never imports
the CUDA package.  See the header of ``gptq_oracle.c`` for what is computed
and which passage of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gptq_oracle.c")
_LIB = os.path.join(_HERE, "libgptq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_half_to_float.restype = ctypes.c_float
        lib.oracle_half_to_float.argtypes = [ctypes.c_uint16]
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_bfloat16_to_float.restype = ctypes.c_float
        lib.oracle_bfloat16_to_float.argtypes = [ctypes.c_uint16]
        for name in ("oracle_unpack_q", "oracle_unpack_z", "oracle_dequant_f32",
                     "oracle_gemm_f64", "oracle_gemm_f64_at", "oracle_dequant_f32_v1", "oracle_gemm_f64_v1", "oracle_silu_mul_f64",
                     "oracle_add_bias_residual_f64", "oracle_dequant_f32_bf16", "oracle_gemm_f64_bf16",
                     "oracle_gemm_f64_bf16_at", "oracle_unpack_q8", "oracle_unpack_z8", "oracle_dequant_f32_w8",
                     "oracle_gemm_f64_w8", "oracle_gemm_f64_w8_at", "oracle_unpack_qn", "oracle_unpack_zn",
                     "oracle_dequant_f32_wn", "oracle_gemm_f64_wn"):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a, shape=None):
    a = np.ascontiguousarray(a, dtype=np.int32)
    if shape is not None:
        assert a.shape == shape, (a.shape, shape)
    return a


def _f16(a, shape=None):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16, a.dtype
    if shape is not None:
        assert a.shape == shape, (a.shape, shape)
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def half_to_float(bits: int) -> float:
    return float(_load().oracle_half_to_float(ctypes.c_uint16(bits)))


def unpack_q(qweight: np.ndarray) -> np.ndarray:
    """int32[K/8, N] -> uint8[K, N]."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    out = np.empty((R * 8, N), dtype=np.uint8)
    _load().oracle_unpack_q(_p(qweight), ctypes.c_int(R * 8), ctypes.c_int(N), _p(out))
    return out


def unpack_z(qzeros: np.ndarray) -> np.ndarray:
    """int32[G, N/8] -> uint8[G, N]."""
    qzeros = _i32(qzeros)
    G, C = qzeros.shape
    out = np.empty((G, C * 8), dtype=np.uint8)
    _load().oracle_unpack_z(_p(qzeros), ctypes.c_int(G), ctypes.c_int(C * 8), _p(out))
    return out


def dequant_f32(qweight, qzeros, scales, g_idx, group_size: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp32[K, N] dequantised weights; ``g_idx`` None means no act-order.  With ``zeros_minus_one`` the stored
    zero-point nibble is z - 1 (older checkpoints) and a separate oracle function is called."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 8
    G = K // group_size
    qzeros = _i32(qzeros, (G, N // 8))
    scales = _f16(scales, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    out = np.empty((K, N), dtype=np.float32)
    fn = _load().oracle_dequant_f32_v1 if zeros_minus_one else _load().oracle_dequant_f32
    fn(_p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(K),
                               ctypes.c_int(N), ctypes.c_int(group_size), _p(out))
    return out


def gemm_f64(x, qweight, qzeros, scales, g_idx, group_size: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp64[M, N] = x[M, K] . dequant(W)[K, N], k ascending (``zeros_minus_one``: see dequant_f32)."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 8
    G = K // group_size
    x = _f16(x)
    M = x.shape[0]
    assert x.shape == (M, K)
    qzeros = _i32(qzeros, (G, N // 8))
    scales = _f16(scales, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    out = np.empty((M, N), dtype=np.float64)
    fn = _load().oracle_gemm_f64_v1 if zeros_minus_one else _load().oracle_gemm_f64
    fn(_p(x), _p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(M),
                            ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group_size), _p(out))
    return out


def gemm_f64_at(x, qweight, qzeros, scales, g_idx, group_size: int, rows, cols) -> np.ndarray:
    """The same sum as :func:`gemm_f64` for chosen (row, col) outputs only."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 8
    G = K // group_size
    x = _f16(x)
    M = x.shape[0]
    assert x.shape == (M, K)
    qzeros = _i32(qzeros, (G, N // 8))
    scales = _f16(scales, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    rows = _i32(rows)
    cols = _i32(cols)
    assert rows.shape == cols.shape and rows.ndim == 1
    assert rows.min(initial=0) >= 0 and rows.max(initial=0) < M
    assert cols.min(initial=0) >= 0 and cols.max(initial=0) < N
    out = np.empty(rows.shape[0], dtype=np.float64)
    _load().oracle_gemm_f64_at(_p(x), _p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(M),
                               ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group_size),
                               _p(rows), _p(cols), ctypes.c_int(rows.shape[0]), _p(out))
    return out


def silu_mul_f64(y: np.ndarray) -> np.ndarray:
    """out[M, I] = silu(y[:, :I]) * y[:, I:] in fp64 for the [gate | up] columns of a gate_up projection."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    M, N = y.shape
    assert N % 2 == 0
    out = np.empty((M, N // 2), dtype=np.float64)
    _load().oracle_silu_mul_f64(_p(y), ctypes.c_int(M), ctypes.c_int(N // 2), _p(out))
    return out


def add_bias_residual_f64(y: np.ndarray, bias: np.ndarray | None, residual: np.ndarray | None) -> np.ndarray:
    """out[M, N] = y + bias[n] + residual[m, n] in fp64 (bias fp16 [N], residual fp16 [M, N]; either may be None)."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    M, N = y.shape
    b = None if bias is None else _f16(bias, (N,))
    r = None if residual is None else _f16(residual, (M, N))
    out = np.empty((M, N), dtype=np.float64)
    _load().oracle_add_bias_residual_f64(_p(y), _p(b), _p(r), ctypes.c_int(M), ctypes.c_int(N), _p(out))
    return out


# ---- bfloat16 activations and scales: numpy has no such type, so they travel as uint16 bit patterns ----------------

def _bf16_bits(a, shape=None):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    if shape is not None:
        assert a.shape == shape, (a.shape, shape)
    return a


def bfloat16_to_float(bits: int) -> float:
    return float(_load().oracle_bfloat16_to_float(ctypes.c_uint16(bits)))


def dequant_f32_bf16(qweight, qzeros, scales_bits, g_idx, group_size: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp32[K, N] dequantised weights for bfloat16 scales given as uint16 bit patterns [G, N]."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 8
    G = K // group_size
    qzeros = _i32(qzeros, (G, N // 8))
    scales_bits = _bf16_bits(scales_bits, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    out = np.empty((K, N), dtype=np.float32)
    _load().oracle_dequant_f32_bf16(_p(qweight), _p(qzeros), _p(scales_bits), _p(g), ctypes.c_int(K), ctypes.c_int(N),
                                    ctypes.c_int(group_size), ctypes.c_int(1 if zeros_minus_one else 0), _p(out))
    return out


def gemm_f64_bf16(x_bits, qweight, qzeros, scales_bits, g_idx, group_size: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp64[M, N] = x . dequant(W) for bfloat16 x [M, K] and scales [G, N], both as uint16 bit patterns."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 8
    G = K // group_size
    x_bits = _bf16_bits(x_bits)
    M = x_bits.shape[0]
    assert x_bits.shape == (M, K)
    qzeros = _i32(qzeros, (G, N // 8))
    scales_bits = _bf16_bits(scales_bits, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    out = np.empty((M, N), dtype=np.float64)
    _load().oracle_gemm_f64_bf16(_p(x_bits), _p(qweight), _p(qzeros), _p(scales_bits), _p(g), ctypes.c_int(M),
                                 ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group_size),
                                 ctypes.c_int(1 if zeros_minus_one else 0), _p(out))
    return out


def gemm_f64_bf16_at(x_bits, qweight, qzeros, scales_bits, g_idx, group_size: int, rows, cols,
                     zeros_minus_one: bool = False) -> np.ndarray:
    """The same sum as :func:`gemm_f64_bf16` for chosen (row, col) outputs only."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 8
    G = K // group_size
    x_bits = _bf16_bits(x_bits)
    M = x_bits.shape[0]
    assert x_bits.shape == (M, K)
    qzeros = _i32(qzeros, (G, N // 8))
    scales_bits = _bf16_bits(scales_bits, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    rows = _i32(rows)
    cols = _i32(cols)
    assert rows.shape == cols.shape and rows.ndim == 1
    assert rows.min(initial=0) >= 0 and rows.max(initial=0) < M
    assert cols.min(initial=0) >= 0 and cols.max(initial=0) < N
    out = np.empty(rows.shape[0], dtype=np.float64)
    _load().oracle_gemm_f64_bf16_at(_p(x_bits), _p(qweight), _p(qzeros), _p(scales_bits), _p(g), ctypes.c_int(M),
                                    ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group_size),
                                    ctypes.c_int(1 if zeros_minus_one else 0),
                                    _p(rows), _p(cols), ctypes.c_int(rows.shape[0]), _p(out))
    return out


# ---- 8-bit weights: qweight int32[K/4, N], qzeros int32[G, N/4] ------------------------------------------------------

def unpack_q8(qweight: np.ndarray) -> np.ndarray:
    """int32[K/4, N] -> uint8[K, N]."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    out = np.empty((R * 4, N), dtype=np.uint8)
    _load().oracle_unpack_q8(_p(qweight), ctypes.c_int(R * 4), ctypes.c_int(N), _p(out))
    return out


def unpack_z8(qzeros: np.ndarray) -> np.ndarray:
    """int32[G, N/4] -> uint8[G, N]."""
    qzeros = _i32(qzeros)
    G, C = qzeros.shape
    out = np.empty((G, C * 4), dtype=np.uint8)
    _load().oracle_unpack_z8(_p(qzeros), ctypes.c_int(G), ctypes.c_int(C * 4), _p(out))
    return out


def _w8_args(qweight, qzeros, scales, g_idx, group_size):
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 4
    G = K // group_size
    qzeros = _i32(qzeros, (G, N // 4))
    scales = _f16(scales, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    return qweight, qzeros, scales, g, K, N


def dequant_f32_w8(qweight, qzeros, scales, g_idx, group_size: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp32[K, N] dequantised 8-bit weights."""
    qweight, qzeros, scales, g, K, N = _w8_args(qweight, qzeros, scales, g_idx, group_size)
    out = np.empty((K, N), dtype=np.float32)
    _load().oracle_dequant_f32_w8(_p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(K), ctypes.c_int(N),
                                  ctypes.c_int(group_size), ctypes.c_int(1 if zeros_minus_one else 0), _p(out))
    return out


def gemm_f64_w8(x, qweight, qzeros, scales, g_idx, group_size: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp64[M, N] = x[M, K] . dequant(W8)[K, N], k ascending."""
    qweight, qzeros, scales, g, K, N = _w8_args(qweight, qzeros, scales, g_idx, group_size)
    x = _f16(x)
    M = x.shape[0]
    assert x.shape == (M, K)
    out = np.empty((M, N), dtype=np.float64)
    _load().oracle_gemm_f64_w8(_p(x), _p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(M), ctypes.c_int(N),
                               ctypes.c_int(K), ctypes.c_int(group_size), ctypes.c_int(1 if zeros_minus_one else 0), _p(out))
    return out


def gemm_f64_w8_at(x, qweight, qzeros, scales, g_idx, group_size: int, rows, cols, zeros_minus_one: bool = False) -> np.ndarray:
    """The same sum as :func:`gemm_f64_w8` for chosen (row, col) outputs only."""
    qweight, qzeros, scales, g, K, N = _w8_args(qweight, qzeros, scales, g_idx, group_size)
    x = _f16(x)
    M = x.shape[0]
    assert x.shape == (M, K)
    rows = _i32(rows)
    cols = _i32(cols)
    assert rows.shape == cols.shape and rows.ndim == 1
    assert rows.min(initial=0) >= 0 and rows.max(initial=0) < M
    assert cols.min(initial=0) >= 0 and cols.max(initial=0) < N
    out = np.empty(rows.shape[0], dtype=np.float64)
    _load().oracle_gemm_f64_w8_at(_p(x), _p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(M), ctypes.c_int(N),
                                  ctypes.c_int(K), ctypes.c_int(group_size), ctypes.c_int(1 if zeros_minus_one else 0),
                                  _p(rows), _p(cols), ctypes.c_int(rows.shape[0]), _p(out))
    return out


# ---- 2- and 3-bit weights: qweight int32[K * bits / 32, N], qzeros int32[G, N * bits / 32] ---------------------------

def unpack_qn(qweight: np.ndarray, bits: int) -> np.ndarray:
    """int32[K * bits / 32, N] -> uint8[K, N]."""
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 32 // bits
    out = np.empty((K, N), dtype=np.uint8)
    _load().oracle_unpack_qn(_p(qweight), ctypes.c_int(K), ctypes.c_int(N), ctypes.c_int(bits), _p(out))
    return out


def unpack_zn(qzeros: np.ndarray, bits: int) -> np.ndarray:
    """int32[G, N * bits / 32] -> uint8[G, N]."""
    qzeros = _i32(qzeros)
    G, C = qzeros.shape
    N = C * 32 // bits
    out = np.empty((G, N), dtype=np.uint8)
    _load().oracle_unpack_zn(_p(qzeros), ctypes.c_int(G), ctypes.c_int(N), ctypes.c_int(bits), _p(out))
    return out


def _wn_args(qweight, qzeros, scales, g_idx, group_size, bits):
    assert bits in (2, 3)
    qweight = _i32(qweight)
    R, N = qweight.shape
    K = R * 32 // bits
    G = K // group_size
    qzeros = _i32(qzeros, (G, N * bits // 32))
    scales = _f16(scales, (G, N))
    g = None if g_idx is None else _i32(g_idx, (K,))
    return qweight, qzeros, scales, g, K, N


def dequant_f32_wn(qweight, qzeros, scales, g_idx, group_size: int, bits: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp32[K, N] dequantised 2- or 3-bit weights."""
    qweight, qzeros, scales, g, K, N = _wn_args(qweight, qzeros, scales, g_idx, group_size, bits)
    out = np.empty((K, N), dtype=np.float32)
    _load().oracle_dequant_f32_wn(_p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(K), ctypes.c_int(N),
                                  ctypes.c_int(group_size), ctypes.c_int(bits), ctypes.c_int(1 if zeros_minus_one else 0), _p(out))
    return out


def gemm_f64_wn(x, qweight, qzeros, scales, g_idx, group_size: int, bits: int, zeros_minus_one: bool = False) -> np.ndarray:
    """fp64[M, N] = x[M, K] . dequant(W)[K, N] for 2- or 3-bit weights, k ascending."""
    qweight, qzeros, scales, g, K, N = _wn_args(qweight, qzeros, scales, g_idx, group_size, bits)
    x = _f16(x)
    M = x.shape[0]
    assert x.shape == (M, K)
    out = np.empty((M, N), dtype=np.float64)
    _load().oracle_gemm_f64_wn(_p(x), _p(qweight), _p(qzeros), _p(scales), _p(g), ctypes.c_int(M), ctypes.c_int(N),
                               ctypes.c_int(K), ctypes.c_int(group_size), ctypes.c_int(bits),
                               ctypes.c_int(1 if zeros_minus_one else 0), _p(out))
    return out
