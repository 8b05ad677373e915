"""Thin ctypes binding over libgptq_b200.so - argument marshalling only.

Every function has the name and argument order of its C-ABI entry point
(``include/gptq_b200.h``).  Device buffers are passed as torch CUDA tensors
(or raw integer addresses); torch is used for device memory and streams only.
Nothing here computes: if the compiled library is missing the import of this
module fails, there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# GPTQ_B200_LIB names another build of the same library (the timeline tool loads its instrumented build this way)
LIB_PATH = os.environ.get("GPTQ_B200_LIB") or os.path.join(_HERE, "libgptq_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2511_19438_b200.build` "
        "(nvcc, sm_100a). There is no CPU or PyTorch fallback for the GPTQ matmul.")

_lib = ctypes.CDLL(LIB_PATH)

GPTQ_FORMAT_ZEROS_MINUS_ONE = 1
GPTQ_FORMAT_GATE_UP = 2
GPTQ_FORMAT_BF16 = 4
GPTQ_ACT_ORDER_PRESORTED = 2
GPTQ_OK = 0
GPTQ_ERR_NULL = -1
GPTQ_ERR_SHAPE = -2
GPTQ_ERR_ALIGN = -3
GPTQ_ERR_UNSUPPORTED = -4
GPTQ_ERR_LAYOUT = -5
GPTQ_ERR_GIDX = -6
GPTQ_ERR_WORKSPACE = -7
GPTQ_ERR_CUDA = -8
GPTQ_ERR_TIMEOUT = -9


class gptq_plan_t(ctypes.Structure):
    _fields_ = [
        ("kernel_name", ctypes.c_char * 48),
        ("kernel", ctypes.c_int), ("m_tile", ctypes.c_int), ("m_chunks", ctypes.c_int),
        ("stages", ctypes.c_int), ("ctas", ctypes.c_int), ("items", ctypes.c_int),
        ("split_panels", ctypes.c_int), ("smem_bytes", ctypes.c_int),
        ("workspace_bytes", ctypes.c_size_t), ("cluster_size", ctypes.c_int),
        ("tail_ctas", ctypes.c_int), ("tail_cluster_size", ctypes.c_int),
    ]


class gptq_host_problem_t(ctypes.Structure):
    _fields_ = [
        ("x_host", ctypes.c_void_p), ("qweight", ctypes.c_void_p), ("qzeros", ctypes.c_void_p),
        ("scales", ctypes.c_void_p), ("g_idx", ctypes.c_void_p), ("y_host", ctypes.c_void_p),
        ("x_stage", ctypes.c_void_p), ("y_stage", ctypes.c_void_p),
        ("M", ctypes.c_int), ("N", ctypes.c_int), ("K", ctypes.c_int), ("group_size", ctypes.c_int),
        ("act_order", ctypes.c_int),
    ]


_vp, _i, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
_SIGNATURES = {
    "gptq_status_string": (ctypes.c_char_p, [_i]),
    "gptq_last_cuda_error": (_i, []),
    "gptq_unpack_u8": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "gptq_dequant_f32": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]),
    "gptq_dequant_f32_format": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]),
    "gptq_repack_bytes": (_sz, [_i, _i, _i, _i, _i]),
    "gptq_repack_format": (_i, [_vp] * 8 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_repack": (_i, [_vp] * 8 + [_i, _i, _i, _i, _vp]),
    "gptq_workspace_bytes": (_sz, [_i, _i, _i, _i, _i]),
    "gptq_set_workspace": (_i, [_vp, _sz]),
    "gptq_gemm": (_i, [_vp] * 6 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_gemm_bf16": (_i, [_vp] * 6 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_repack_bits_scratch_bytes": (ctypes.c_size_t, [_i, _i, _i, _i]),
    "gptq_repack_bits": (_i, [_i] + [_vp] * 9 + [ctypes.c_size_t, _i, _i, _i, _i, _i, _vp]),
    "gptq_dequant_f32_bits": (_i, [_i] + [_vp] * 5 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_repack_w8_bytes": (ctypes.c_size_t, [_i, _i, _i, _i]),
    "gptq_repack_w8_scratch_bytes": (ctypes.c_size_t, [_i, _i, _i]),
    "gptq_repack_w8": (_i, [_vp] * 9 + [ctypes.c_size_t, _i, _i, _i, _i, _i, _vp]),
    "gptq_dequant_f32_w8": (_i, [_vp] * 5 + [_i, _i, _i, _i, _i, _i, _vp]),
    "gptq_gemm_w8": (_i, [_vp] * 6 + [_i, _i, _i, _i, _vp]),
    "gptq_gemm_silu_mul": (_i, [_vp] * 6 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_gemm_bias_residual": (_i, [_vp] * 8 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_gemm_silu_mul_scatter": (_i, [_vp] * 7 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_invert_perm": (_i, [_vp, _vp, _i, _vp]),
    "gptq_set_cta_pairs": (_i, [_i]),
    "gptq_gemm_host": (_i, [_vp] * 8 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_gemm_noalloc": (_i, [_vp] * 6 + [_i, _i, _i, _i, _i, _vp]),
    "gptq_noalloc_scratch_bytes": (_sz, []),
    "gptq_gemm_host_batch": (_i, [ctypes.POINTER(gptq_host_problem_t), _i, _vp, ctypes.POINTER(_i)]),
    "gptq_gemm_host_batch_bf16": (_i, [ctypes.POINTER(gptq_host_problem_t), _i, _vp, ctypes.POINTER(_i)]),
    "gptq_gemm_host_batch_w8": (_i, [ctypes.POINTER(gptq_host_problem_t), _i, _vp, ctypes.POINTER(_i)]),
    "gptq_check_status": (_i, [_vp]),
    "gptq_selftest_wait_timeout": (_i, [ctypes.c_uint, _vp]),
    "gptq_trace_reset": (_i, [_vp]),
    "gptq_trace_read": (_i, [_vp, _i, _vp]),
    "gptq_plan": (_i, [_i, _i, _i, _i, _i, _i, ctypes.POINTER(gptq_plan_t)]),
    "gptq_plan_noalloc": (_i, [_i, _i, _i, _i, _i, _i, ctypes.POINTER(gptq_plan_t)]),
    "gptq_plan_cta_range": (_i, [_i, _i, _i, ctypes.POINTER(_i), ctypes.POINTER(_i)]),
    "gptq_plan_panel_owners": (_i, [_i, _i, _i, _i, ctypes.POINTER(_i), ctypes.POINTER(_i)]),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args

EXPORTED = tuple(_SIGNATURES)


class GptqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {gptq_status_string(status)} (status {status})")


def _ptr(t):
    """Address of a torch tensor / numpy array / raw int (None -> NULL)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def check(status: int, where: str) -> None:
    if status != GPTQ_OK:
        raise GptqError(status, where)


def gptq_status_string(status: int) -> str:
    return _lib.gptq_status_string(status).decode()


def gptq_last_cuda_error() -> int:
    return _lib.gptq_last_cuda_error()


def gptq_unpack_u8(qweight, qzeros, q_out, z_out, N, K, group_size, stream=None) -> int:
    return _lib.gptq_unpack_u8(_ptr(qweight), _ptr(qzeros), _ptr(q_out), _ptr(z_out), N, K, group_size,
                               _stream(stream))


def gptq_dequant_f32(qweight, qzeros, scales, g_idx, w_out, N, K, group_size, act_order, repacked,
                     stream=None) -> int:
    return _lib.gptq_dequant_f32(_ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(w_out), N, K,
                                 group_size, int(act_order), int(repacked), _stream(stream))


def gptq_dequant_f32_format(qweight, qzeros, scales, g_idx, w_out, N, K, group_size, act_order, repacked, fmt,
                            stream=None) -> int:
    return _lib.gptq_dequant_f32_format(_ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(w_out), N, K,
                                        group_size, int(act_order), int(repacked), int(fmt), _stream(stream))


def gptq_repack_format(qweight, qzeros, scales, g_idx, qweight_out, qzeros_out, scales_out, perm_out, N, K,
                       group_size, act_order, fmt, stream=None) -> int:
    return _lib.gptq_repack_format(_ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(qweight_out),
                                   _ptr(qzeros_out), _ptr(scales_out), _ptr(perm_out), N, K, group_size,
                                   int(act_order), int(fmt), _stream(stream))


def gptq_repack_bytes(which, N, K, group_size, act_order) -> int:
    return _lib.gptq_repack_bytes(which, N, K, group_size, int(act_order))


def gptq_repack(qweight, qzeros, scales, g_idx, qweight_out, qzeros_out, scales_out, perm_out, N, K,
                group_size, act_order, stream=None) -> int:
    return _lib.gptq_repack(_ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(qweight_out),
                            _ptr(qzeros_out), _ptr(scales_out), _ptr(perm_out), N, K, group_size,
                            int(act_order), _stream(stream))


def gptq_workspace_bytes(M, N, K, group_size, act_order) -> int:
    return _lib.gptq_workspace_bytes(M, N, K, group_size, int(act_order))


def gptq_set_workspace(ptr, nbytes) -> int:
    return _lib.gptq_set_workspace(_ptr(ptr), nbytes)


def gptq_gemm(x, qweight, qzeros, scales, g_idx, y, M, N, K, group_size, act_order, stream=None) -> int:
    return _lib.gptq_gemm(_ptr(x), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(y), M, N, K,
                          group_size, int(act_order), _stream(stream))


def gptq_gemm_bf16(x, qweight, qzeros, scales, g_idx, y, M, N, K, group_size, act_order, stream=None) -> int:
    return _lib.gptq_gemm_bf16(_ptr(x), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(y), M, N, K,
                               group_size, act_order, _stream(stream))


def gptq_repack_bits_scratch_bytes(bits, N, K, group_size) -> int:
    return int(_lib.gptq_repack_bits_scratch_bytes(bits, N, K, group_size))


def gptq_repack_bits(bits, qweight, qzeros, scales, g_idx, qweight_out, qzeros_out, scales_out, perm_out, scratch,
                     scratch_bytes, N, K, group_size, act_order, fmt, stream=None) -> int:
    return _lib.gptq_repack_bits(bits, _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(qweight_out),
                                 _ptr(qzeros_out), _ptr(scales_out), _ptr(perm_out), _ptr(scratch), int(scratch_bytes), N, K,
                                 group_size, int(act_order), int(fmt), _stream(stream))


def gptq_dequant_f32_bits(bits, qweight, qzeros, scales, g_idx, w_out, N, K, group_size, act_order, fmt, stream=None) -> int:
    return _lib.gptq_dequant_f32_bits(bits, _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(w_out), N, K,
                                      group_size, int(act_order), int(fmt), _stream(stream))


def gptq_repack_w8_bytes(which, N, K, group_size) -> int:
    return int(_lib.gptq_repack_w8_bytes(which, N, K, group_size))


def gptq_repack_w8_scratch_bytes(N, K, group_size) -> int:
    return int(_lib.gptq_repack_w8_scratch_bytes(N, K, group_size))


def gptq_repack_w8(qweight, qzeros, scales, g_idx, qweight_out, qzeros_out, scales_out, perm_out, scratch, scratch_bytes,
                   N, K, group_size, act_order, fmt, stream=None) -> int:
    return _lib.gptq_repack_w8(_ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(qweight_out), _ptr(qzeros_out),
                               _ptr(scales_out), _ptr(perm_out), _ptr(scratch), int(scratch_bytes), N, K, group_size,
                               int(act_order), int(fmt), _stream(stream))


def gptq_dequant_f32_w8(qweight, qzeros, scales, g_idx, w_out, N, K, group_size, act_order, repacked, fmt, stream=None) -> int:
    return _lib.gptq_dequant_f32_w8(_ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(w_out), N, K, group_size,
                                    int(act_order), int(repacked), int(fmt), _stream(stream))


def gptq_gemm_w8(x, qweight, qzeros, scales, perm, y, M, N, K, group_size, stream=None) -> int:
    return _lib.gptq_gemm_w8(_ptr(x), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(perm), _ptr(y), M, N, K, group_size,
                             _stream(stream))


def gptq_set_cta_pairs(enable) -> int:
    return _lib.gptq_set_cta_pairs(int(bool(enable)))


def gptq_gemm_host(x_host, qweight, qzeros, scales, g_idx, y_host, x_stage, y_stage, M, N, K, group_size,
                   act_order, stream=None) -> int:
    return _lib.gptq_gemm_host(_ptr(x_host), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx),
                               _ptr(y_host), _ptr(x_stage), _ptr(y_stage), M, N, K, group_size,
                               int(act_order), _stream(stream))


def gptq_gemm_silu_mul(x, qweight, qzeros, scales, g_idx, out, M, N, K, group_size, act_order, stream=None) -> int:
    return _lib.gptq_gemm_silu_mul(_ptr(x), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(out), M, N,
                                   K, group_size, int(act_order), _stream(stream))


def gptq_gemm_silu_mul_scatter(x, qweight, qzeros, scales, g_idx, out_index, out, M, N, K, group_size, act_order,
                               stream=None) -> int:
    return _lib.gptq_gemm_silu_mul_scatter(_ptr(x), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(out_index),
                                           _ptr(out), M, N, K, group_size, int(act_order), _stream(stream))


def gptq_invert_perm(perm, inverse, K, stream=None) -> int:
    return _lib.gptq_invert_perm(_ptr(perm), _ptr(inverse), K, _stream(stream))


def gptq_gemm_bias_residual(x, qweight, qzeros, scales, g_idx, bias, residual, y, M, N, K, group_size, act_order,
                            stream=None) -> int:
    return _lib.gptq_gemm_bias_residual(_ptr(x), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(bias),
                                        _ptr(residual), _ptr(y), M, N, K, group_size, int(act_order), _stream(stream))


def gptq_gemm_noalloc(x, qweight, qzeros, scales, g_idx, y, M, N, K, group_size, act_order, stream=None) -> int:
    return _lib.gptq_gemm_noalloc(_ptr(x), _ptr(qweight), _ptr(qzeros), _ptr(scales), _ptr(g_idx), _ptr(y), M, N,
                                  K, group_size, int(act_order), _stream(stream))


def gptq_noalloc_scratch_bytes() -> int:
    return _lib.gptq_noalloc_scratch_bytes()


def make_host_problems(items):
    """Marshals a list of (x_host, qweight, qzeros, scales, g_idx, y_host, x_stage, y_stage, M, N, K, group_size,
    act_order) tuples into a C array for gptq_gemm_host_batch (build once, reuse every step)."""
    arr = (gptq_host_problem_t * len(items))()
    for i, it in enumerate(items):
        ptrs = [_ptr(v) for v in it[:8]]
        arr[i] = gptq_host_problem_t(*ptrs, int(it[8]), int(it[9]), int(it[10]), int(it[11]), int(bool(it[12])))
    return arr


def gptq_gemm_host_batch(problems, stream=None):
    """Returns (status, bad_index); `problems` comes from make_host_problems."""
    bad = ctypes.c_int(-1)
    st = _lib.gptq_gemm_host_batch(problems, len(problems), _stream(stream), ctypes.byref(bad))
    return st, bad.value


def gptq_gemm_host_batch_bf16(problems, stream=None):
    """gptq_gemm_host_batch for bfloat16 layers and activations."""
    bad = ctypes.c_int(-1)
    st = _lib.gptq_gemm_host_batch_bf16(problems, len(problems), _stream(stream), ctypes.byref(bad))
    return st, bad.value


def gptq_gemm_host_batch_w8(problems, stream=None):
    """gptq_gemm_host_batch for 8-bit layers (each problem's g_idx is the layer's perm_out)."""
    bad = ctypes.c_int(-1)
    st = _lib.gptq_gemm_host_batch_w8(problems, len(problems), _stream(stream), ctypes.byref(bad))
    return st, bad.value


def gptq_check_status(stream=None) -> int:
    return _lib.gptq_check_status(_stream(stream))


def gptq_selftest_wait_timeout(limit_us, stream=None) -> int:
    return _lib.gptq_selftest_wait_timeout(int(limit_us), _stream(stream))


def gptq_trace_reset(stream=None) -> int:
    return _lib.gptq_trace_reset(_stream(stream))


def gptq_trace_read(max_rows: int = 64, stream=None):
    """Returns (status or row count, rows) with rows a list of 8-tuples of ints (see the header)."""
    buf = (ctypes.c_ulonglong * (8 * max_rows))()
    n = _lib.gptq_trace_read(ctypes.cast(buf, ctypes.c_void_p), max_rows, _stream(stream))
    rows = [tuple(buf[8 * i + j] for j in range(8)) for i in range(max(n, 0))]
    return n, rows


def plan_kernel_name(plan) -> str:
    return plan.kernel_name.decode()


def gptq_plan(M, N, K, group_size, act_order, sm_count):
    """Returns (status, gptq_plan_t).  Host-only: makes no CUDA call."""
    out = gptq_plan_t()
    st = _lib.gptq_plan(M, N, K, group_size, int(act_order), sm_count, ctypes.byref(out))
    return st, out


def gptq_plan_noalloc(M, N, K, group_size, act_order, sm_count):
    """Returns (status, gptq_plan_t) for gptq_gemm_noalloc.  Host-only: makes no CUDA call."""
    out = gptq_plan_t()
    st = _lib.gptq_plan_noalloc(M, N, K, group_size, int(act_order), sm_count, ctypes.byref(out))
    return st, out


def gptq_plan_cta_range(items, ctas, cta):
    """Returns (status, first_item, end_item)."""
    a, b = ctypes.c_int(), ctypes.c_int()
    st = _lib.gptq_plan_cta_range(items, ctas, cta, ctypes.byref(a), ctypes.byref(b))
    return st, a.value, b.value


def gptq_plan_panel_owners(items, ctas, groups, panel):
    """Returns (status, first_cta, last_cta)."""
    a, b = ctypes.c_int(), ctypes.c_int()
    st = _lib.gptq_plan_panel_owners(items, ctas, groups, panel, ctypes.byref(a), ctypes.byref(b))
    return st, a.value, b.value
