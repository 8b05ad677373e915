"""Device-side plumbing for tests and the benchmark: uploads a synthetic layer,
runs the one-time repack through the C ABI, keeps the workspace registered.

torch is used only to own device memory and streams; every computation is a
call into libgptq_b200.so through ``binding``.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import binding as B
from .workloads import QuantLinear


@dataclass
class DeviceLinear:
    """A layer resident on the GPU: canonical buffers (optional) and the tiled ones."""
    K: int
    N: int
    group_size: int
    act_order: bool
    qweight_t: torch.Tensor      # tiled
    qzeros_t: torch.Tensor
    scales_t: torch.Tensor
    perm: torch.Tensor | None    # int32[K], original index of sorted row i
    canonical: tuple | None      # (qweight, qzeros, scales, g_idx) device tensors, if kept


def to_device(a: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def upload_and_repack(L: QuantLinear, keep_canonical: bool = False, device="cuda", gate_up: bool = False,
                      scales_bf16_bits: np.ndarray | None = None) -> DeviceLinear:
    """``scales_bf16_bits`` (uint16 [G, N]) replaces the layer's fp16 scales by bfloat16 ones and marks the tiled
    layer as a bfloat16 layer (to be used with :func:`gemm_bf16`)."""
    qw = to_device(L.qweight, device)
    qz = to_device(L.qzeros, device)
    if scales_bf16_bits is not None:
        assert scales_bf16_bits.dtype == np.uint16 and scales_bf16_bits.shape == (L.K // L.group_size, L.N)
        sc = to_device(scales_bf16_bits.view(np.int16), device).view(torch.bfloat16)
    else:
        sc = to_device(L.scales, device)
    gi = to_device(L.g_idx, device) if L.act_order else None
    qw_t = torch.empty(B.gptq_repack_bytes(0, L.N, L.K, L.group_size, L.act_order), dtype=torch.uint8, device=device)
    qz_t = torch.empty(B.gptq_repack_bytes(1, L.N, L.K, L.group_size, L.act_order), dtype=torch.uint8, device=device)
    sc_t = torch.empty(B.gptq_repack_bytes(2, L.N, L.K, L.group_size, L.act_order), dtype=torch.uint8, device=device)
    perm = torch.empty(L.K, dtype=torch.int32, device=device) if L.act_order else None
    fmt = (B.GPTQ_FORMAT_ZEROS_MINUS_ONE if L.zeros_minus_one else 0) | (B.GPTQ_FORMAT_GATE_UP if gate_up else 0)
    fmt |= B.GPTQ_FORMAT_BF16 if scales_bf16_bits is not None else 0
    B.check(B.gptq_repack_format(qw, qz, sc, gi, qw_t, qz_t, sc_t, perm, L.N, L.K, L.group_size, L.act_order, fmt),
            "gptq_repack_format")
    torch.cuda.current_stream().synchronize()
    canonical = (qw, qz, sc, gi) if keep_canonical else None
    return DeviceLinear(L.K, L.N, L.group_size, L.act_order, qw_t, qz_t, sc_t, perm, canonical)


class WorkspaceHolder:
    """Owns one device scratch buffer and keeps it registered with the library."""

    def __init__(self, device="cuda"):
        self.device = device
        self.buf = None

    def ensure(self, nbytes: int) -> None:
        if nbytes <= 0:
            return
        if self.buf is None or self.buf.numel() < nbytes:
            torch.cuda.synchronize()
            self.buf = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        # registering is idempotent and cheap (a host-side pointer swap)
        B.check(B.gptq_set_workspace(self.buf, self.buf.numel()), "gptq_set_workspace")

    def ensure_for(self, M: int, D: DeviceLinear) -> None:
        self.ensure(B.gptq_workspace_bytes(M, D.N, D.K, D.group_size, D.act_order))


def gemm(x: torch.Tensor, D: DeviceLinear, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """y = x . dequant(W) through gptq_gemm (x fp16 [M, K] on the device)."""
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, D.N), dtype=torch.float16, device=x.device)
    B.check(B.gptq_gemm(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, y, M, D.N, D.K, D.group_size,
                        D.act_order, stream), "gptq_gemm")
    return y


def bf16_from_bits(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bit patterns -> a bfloat16 tensor on the device (no conversion: the same 16 bits)."""
    return to_device(np.ascontiguousarray(bits).view(np.int16), device).view(torch.bfloat16)


def bits_of_bf16(t: torch.Tensor) -> np.ndarray:
    """A bfloat16 tensor -> its bit patterns as a numpy uint16 array."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def gemm_bf16(x: torch.Tensor, D: DeviceLinear, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """y = x . dequant(W) through gptq_gemm_bf16 (x bfloat16 [M, K] on the device, D repacked with bfloat16 scales)."""
    assert x.dtype == torch.bfloat16
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, D.N), dtype=torch.bfloat16, device=x.device)
    B.check(B.gptq_gemm_bf16(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, y, M, D.N, D.K, D.group_size,
                             D.act_order, stream), "gptq_gemm_bf16")
    return y


def gemm_silu_mul(x: torch.Tensor, D: DeviceLinear, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """out[M, N / 2] = silu(gate) * up through gptq_gemm_silu_mul (D repacked with gate_up=True)."""
    M = x.shape[0]
    if out is None:
        out = torch.empty((M, D.N // 2), dtype=torch.float16, device=x.device)
    B.check(B.gptq_gemm_silu_mul(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, out, M, D.N, D.K, D.group_size,
                                 D.act_order, stream), "gptq_gemm_silu_mul")
    return out


def gemm_bias_residual(x: torch.Tensor, D: DeviceLinear, bias: torch.Tensor | None, residual: torch.Tensor | None,
                       y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """y = x . dequant(W) + bias + residual through gptq_gemm_bias_residual (y may be the residual buffer)."""
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, D.N), dtype=torch.float16, device=x.device)
    B.check(B.gptq_gemm_bias_residual(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, bias, residual, y, M, D.N, D.K,
                                      D.group_size, D.act_order, stream), "gptq_gemm_bias_residual")
    return y


def invert_perm(perm: torch.Tensor) -> torch.Tensor:
    """inverse[perm[i]] = i through gptq_invert_perm."""
    inv = torch.empty_like(perm)
    B.check(B.gptq_invert_perm(perm, inv, perm.numel()), "gptq_invert_perm")
    return inv


def gemm_silu_mul_scatter(x: torch.Tensor, D: DeviceLinear, out_index: torch.Tensor, out: torch.Tensor | None = None,
                          stream=None) -> torch.Tensor:
    """gemm_silu_mul whose output column i lands at column out_index[i]."""
    M = x.shape[0]
    if out is None:
        out = torch.empty((M, D.N // 2), dtype=torch.float16, device=x.device)
    B.check(B.gptq_gemm_silu_mul_scatter(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, out_index, out, M, D.N, D.K,
                                         D.group_size, D.act_order, stream), "gptq_gemm_silu_mul_scatter")
    return out


def gemm_presorted(x_sorted: torch.Tensor, D: DeviceLinear, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """gptq_gemm of an act-order layer whose input already is in the layer's sorted row order (no gather)."""
    M = x_sorted.shape[0]
    if y is None:
        y = torch.empty((M, D.N), dtype=torch.float16, device=x_sorted.device)
    B.check(B.gptq_gemm(x_sorted, D.qweight_t, D.qzeros_t, D.scales_t, None, y, M, D.N, D.K, D.group_size,
                        B.GPTQ_ACT_ORDER_PRESORTED, stream), "gptq_gemm (pre-sorted)")
    return y


# ---- 8-bit layers (stored as two stacked 4-bit planes) ----------------------------------------------------------------

def upload_and_repack_w8(L: QuantLinear, keep_canonical: bool = False, device="cuda") -> DeviceLinear:
    """Uploads a canonical 8-bit layer (qweight int32[K/4, N], qzeros int32[G, N/4]) and repacks it with gptq_repack_w8.
    The returned DeviceLinear keeps the checkpoint's K and group size; ``perm`` is int32[2 K]."""
    qw, qz, sc = to_device(L.qweight, device), to_device(L.qzeros, device), to_device(L.scales, device)
    gi = to_device(L.g_idx, device) if L.act_order else None
    outs = [torch.empty(B.gptq_repack_w8_bytes(w, L.N, L.K, L.group_size), dtype=torch.uint8, device=device) for w in range(3)]
    perm = torch.empty(2 * L.K, dtype=torch.int32, device=device)
    nscratch = B.gptq_repack_w8_scratch_bytes(L.N, L.K, L.group_size)
    scratch = torch.empty(nscratch, dtype=torch.uint8, device=device)
    fmt = B.GPTQ_FORMAT_ZEROS_MINUS_ONE if L.zeros_minus_one else 0
    B.check(B.gptq_repack_w8(qw, qz, sc, gi, outs[0], outs[1], outs[2], perm, scratch, nscratch, L.N, L.K, L.group_size,
                             L.act_order, fmt), "gptq_repack_w8")
    torch.cuda.current_stream().synchronize()
    canonical = (qw, qz, sc, gi) if keep_canonical else None
    return DeviceLinear(L.K, L.N, L.group_size, L.act_order, outs[0], outs[1], outs[2], perm, canonical)


def gemm_w8(x: torch.Tensor, D: DeviceLinear, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """y = x . dequant(W8) through gptq_gemm_w8 (the workspace must hold the gathered activations, see ensure_for_w8)."""
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, D.N), dtype=torch.float16, device=x.device)
    B.check(B.gptq_gemm_w8(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, y, M, D.N, D.K, D.group_size, stream), "gptq_gemm_w8")
    return y


def ensure_for_w8(ws: "WorkspaceHolder", M: int, D: DeviceLinear) -> None:
    ws.ensure(B.gptq_workspace_bytes(M, D.N, 2 * D.K, D.group_size, 1))


# ---- 2- and 3-bit layers (widened to a 4-bit layer by the repack) -----------------------------------------------------

def upload_and_repack_bits(L: QuantLinear, bits: int, keep_canonical: bool = False, device="cuda") -> DeviceLinear:
    """Uploads a canonical 2- or 3-bit layer and repacks it with gptq_repack_bits; the result is an ordinary tiled 4-bit
    layer for :func:`gemm`."""
    qw, qz, sc = to_device(L.qweight, device), to_device(L.qzeros, device), to_device(L.scales, device)
    gi = to_device(L.g_idx, device) if L.act_order else None
    outs = [torch.empty(B.gptq_repack_bytes(w, L.N, L.K, L.group_size, L.act_order), dtype=torch.uint8, device=device)
            for w in range(3)]
    perm = torch.empty(L.K, dtype=torch.int32, device=device) if L.act_order else None
    nscratch = B.gptq_repack_bits_scratch_bytes(bits, L.N, L.K, L.group_size)
    scratch = torch.empty(nscratch, dtype=torch.uint8, device=device)
    fmt = B.GPTQ_FORMAT_ZEROS_MINUS_ONE if L.zeros_minus_one else 0
    B.check(B.gptq_repack_bits(bits, qw, qz, sc, gi, outs[0], outs[1], outs[2], perm, scratch, nscratch, L.N, L.K,
                               L.group_size, L.act_order, fmt), "gptq_repack_bits")
    torch.cuda.current_stream().synchronize()
    canonical = (qw, qz, sc, gi) if keep_canonical else None
    return DeviceLinear(L.K, L.N, L.group_size, L.act_order, outs[0], outs[1], outs[2], perm, canonical)
