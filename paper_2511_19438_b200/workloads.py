"""Seeded synthetic inputs for the GPTQ int4 matmul path.

This module only *draws and encodes* inputs (random nibbles, scales, zero
points, activations, act-order permutations) and names the workload shapes.
It holds none of the method's arithmetic: no unpacking, no dequantisation,
no matmul.  Both the CUDA path and the CPU oracle are fed from here, so the
two never share anything but their inputs.

Storage format produced (the GPTQ checkpoint convention the path consumes):

* ``qweight int32[K/8, N]`` - nibble ``i`` (bits ``4i..4i+3``, LSB first) of
  word ``(r, n)`` is ``q[8r+i, n]`` in ``0..15``.
* ``qzeros int32[G, N/8]``  - nibble ``j`` of word ``(g, c)`` is ``z[g, 8c+j]``.
* ``scales fp16[G, N]``, ``G = K / group_size``.
* ``g_idx int32[K]`` (act-order only) - row ``k`` uses scale/zero row
  ``g_idx[k]``; here ``g_idx[k] = perm[k] // group_size`` for a seeded
  uniform permutation, so every group has exactly ``group_size`` rows.

Value distributions: ``x ~ fp16(N(0,1))``, ``q, z ~ U{0..15}``,
``scales = fp16(0.002 + |N(0, sigma=0.01)|)``.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass

import numpy as np

GROUP_SIZE = 128
SCALE_FLOOR = 0.002
SCALE_SIGMA = 0.01

# (K, N) of the decoder linears.  Llama-2-7B: hidden 4096, ffn 11008.
SHAPES_7B = {
    "qkv": (4096, 12288),
    "o": (4096, 4096),
    "gate_up": (4096, 22016),
    "down": (11008, 4096),
}
# Llama-2-13B: hidden 5120, ffn 13824 (the act-order configuration).
SHAPES_13B = {
    "qkv": (5120, 15360),
    "gate_up": (5120, 27648),
    "down": (13824, 5120),
}
LAYERS_7B = 32
DECODE_M = (1, 4, 8, 16)
ACT_ORDER_M = (1, 8)
PREFILL_M = (512, 1024, 2048, 4096)
STEP_M = (1, 8, 32, 64)


def seed_for(*parts) -> int:
    """Stable 32-bit seed from a tuple of names/numbers (printed in logs)."""
    return zlib.crc32("/".join(str(p) for p in parts).encode()) & 0xFFFFFFFF


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def pack_along_k(q: np.ndarray) -> np.ndarray:
    """uint8[K, N] nibbles -> int32[K/8, N], nibble i of a word = row 8r+i."""
    K, N = q.shape
    assert K % 8 == 0
    q32 = q.astype(np.uint32).reshape(K // 8, 8, N)
    w = np.zeros((K // 8, N), dtype=np.uint32)
    for i in range(8):
        w |= q32[:, i, :] << np.uint32(4 * i)
    return w.view(np.int32)


def pack_along_n(z: np.ndarray) -> np.ndarray:
    """uint8[G, N] nibbles -> int32[G, N/8], nibble j of a word = column 8c+j."""
    G, N = z.shape
    assert N % 8 == 0
    z32 = z.astype(np.uint32).reshape(G, N // 8, 8)
    w = np.zeros((G, N // 8), dtype=np.uint32)
    for j in range(8):
        w |= z32[:, :, j] << np.uint32(4 * j)
    return w.view(np.int32)


@dataclass
class QuantLinear:
    """One GPTQ linear layer in checkpoint (canonical) layout, host arrays."""
    K: int
    N: int
    group_size: int
    qweight: np.ndarray          # int32[K/8, N]
    qzeros: np.ndarray           # int32[G, N/8]
    scales: np.ndarray           # float16[G, N]
    g_idx: np.ndarray | None     # int32[K] or None
    seed: int
    zeros_minus_one: bool = False   # the stored zero-point nibble is z - 1 (older checkpoints)

    @property
    def act_order(self) -> bool:
        return self.g_idx is not None

    @property
    def G(self) -> int:
        return self.K // self.group_size


def make_scales(G: int, N: int, seed: int) -> np.ndarray:
    r = _rng(seed)
    s = SCALE_FLOOR + np.abs(r.standard_normal((G, N), dtype=np.float32) * SCALE_SIGMA)
    return s.astype(np.float16)


def make_g_idx(K: int, group_size: int, seed: int) -> np.ndarray:
    perm = _rng(seed).permutation(K)
    return (perm // group_size).astype(np.int32)


def make_linear(K: int, N: int, seed: int, group_size: int = GROUP_SIZE,
                act_order: bool = False, zeros_minus_one: bool = False) -> QuantLinear:
    """Random GPTQ layer.  Packed words are drawn directly as uniform 32-bit
    integers, which makes every nibble uniform on 0..15 and independent.
    ``zeros_minus_one`` only labels the layer: the same stored nibbles are then
    to be read as zero point minus one."""
    assert K % 8 == 0 and N % 8 == 0 and K % group_size == 0
    G = K // group_size
    r = _rng(seed)
    qweight = r.integers(0, 1 << 32, size=(K // 8, N), dtype=np.uint32).view(np.int32)
    qzeros = r.integers(0, 1 << 32, size=(G, N // 8), dtype=np.uint32).view(np.int32)
    scales = make_scales(G, N, seed ^ 0x5CA1E5)
    g_idx = make_g_idx(K, group_size, seed ^ 0x61D7) if act_order else None
    return QuantLinear(K, N, group_size, qweight, qzeros, scales, g_idx, seed, zeros_minus_one)


def make_linear_from_values(q: np.ndarray, z: np.ndarray, scales: np.ndarray,
                            group_size: int, g_idx: np.ndarray | None = None) -> QuantLinear:
    """Encode caller-chosen nibbles (tests use this for hand-built cases)."""
    K, N = q.shape
    return QuantLinear(K, N, group_size, pack_along_k(q), pack_along_n(z),
                       np.ascontiguousarray(scales, dtype=np.float16),
                       None if g_idx is None else np.ascontiguousarray(g_idx, dtype=np.int32), 0)


def make_x(M: int, K: int, seed: int) -> np.ndarray:
    return _rng(seed).standard_normal((M, K), dtype=np.float32).astype(np.float16)


def pack8_along_k(q: np.ndarray) -> np.ndarray:
    """uint8[K, N] bytes -> int32[K/4, N], byte i of a word = row 4r+i (8-bit weights)."""
    K, N = q.shape
    assert K % 4 == 0
    q32 = q.astype(np.uint32).reshape(K // 4, 4, N)
    w = np.zeros((K // 4, N), dtype=np.uint32)
    for i in range(4):
        w |= q32[:, i, :] << np.uint32(8 * i)
    return w.view(np.int32)


def pack8_along_n(z: np.ndarray) -> np.ndarray:
    """uint8[G, N] bytes -> int32[G, N/4], byte j of a word = column 4c+j (8-bit zero points)."""
    G, N = z.shape
    assert N % 4 == 0
    z32 = z.astype(np.uint32).reshape(G, N // 4, 4)
    w = np.zeros((G, N // 4), dtype=np.uint32)
    for j in range(4):
        w |= z32[:, :, j] << np.uint32(8 * j)
    return w.view(np.int32)


def make_linear_w8(K: int, N: int, seed: int, group_size: int = GROUP_SIZE, act_order: bool = False,
                   zeros_minus_one: bool = False) -> QuantLinear:
    """Random 8-bit GPTQ layer: qweight int32[K/4, N] and qzeros int32[G, N/4] drawn as uniform 32-bit words (every
    byte uniform on 0..255), scales and g_idx as for the 4-bit layers.  With ``zeros_minus_one`` no stored zero point
    is 255 (its meaning, 256, has no place in the library's tiling and real checkpoints centre the zero point)."""
    assert K % 8 == 0 and N % 8 == 0 and K % group_size == 0
    G = K // group_size
    r = _rng(seed)
    qweight = r.integers(0, 1 << 32, size=(K // 4, N), dtype=np.uint32).view(np.int32)
    z = r.integers(0, 255 if zeros_minus_one else 256, size=(G, N), dtype=np.uint32).astype(np.uint8)
    scales = make_scales(G, N, seed ^ 0x5CA1E5)
    g_idx = make_g_idx(K, group_size, seed ^ 0x61D7) if act_order else None
    return QuantLinear(K, N, group_size, qweight, pack8_along_n(z), scales, g_idx, seed, zeros_minus_one)


def pack_bits_stream(v: np.ndarray, bits: int) -> np.ndarray:
    """uint8[R, L] values below 2^bits -> int32[R, L * bits / 32]: each row is one bit stream, value i in bits
    [bits * i, bits * i + bits) of the little-endian concatenation of the row's 32-bit words (2- and 3-bit layers)."""
    R, L = v.shape
    assert (L * bits) % 32 == 0 and int(v.max(initial=0)) < (1 << bits)
    bit = ((v[:, :, None].astype(np.uint8) >> np.arange(bits, dtype=np.uint8)) & 1).reshape(R, L * bits)      # LSB first
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (bit.reshape(R, L * bits // 32, 32).astype(np.uint64) * weights).sum(axis=2).astype(np.uint32).view(np.int32)


def make_linear_wn(K: int, N: int, seed: int, bits: int, group_size: int = GROUP_SIZE, act_order: bool = False,
                   zeros_minus_one: bool = False) -> QuantLinear:
    """Random 2- or 3-bit GPTQ layer: qweight int32[K * bits / 32, N] (a bit stream per column), qzeros
    int32[G, N * bits / 32] (a bit stream per group), uniform values; scales and g_idx as for the 4-bit layers."""
    assert bits in (2, 3) and K % 32 == 0 and N % 32 == 0 and K % group_size == 0
    G = K // group_size
    r = _rng(seed)
    q = r.integers(0, 1 << bits, size=(K, N), dtype=np.uint8)
    z = r.integers(0, 1 << bits, size=(G, N), dtype=np.uint8)
    qweight = np.ascontiguousarray(pack_bits_stream(np.ascontiguousarray(q.T), bits).T)
    scales = make_scales(G, N, seed ^ 0x5CA1E5)
    g_idx = make_g_idx(K, group_size, seed ^ 0x61D7) if act_order else None
    return QuantLinear(K, N, group_size, qweight, pack_bits_stream(z, bits), scales, g_idx, seed, zeros_minus_one)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Finite float values -> the bit patterns (uint16) of the nearest bfloat16, ties to even.  Inputs for the
    bfloat16 variant travel in this form because numpy has no bfloat16 type."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def make_x_bf16(M: int, K: int, seed: int) -> np.ndarray:
    """Standard-normal activations as bfloat16 bit patterns [M, K]."""
    return bf16_bits(_rng(seed).standard_normal((M, K), dtype=np.float32))


def make_scales_bf16(G: int, N: int, seed: int) -> np.ndarray:
    """The scale recipe of :func:`make_scales`, rounded to bfloat16 instead of fp16 (bit patterns [G, N])."""
    r = _rng(seed)
    return bf16_bits(SCALE_FLOOR + np.abs(r.standard_normal((G, N), dtype=np.float32) * SCALE_SIGMA))


def algorithmic_bytes(M: int, K: int, N: int, group_size: int = GROUP_SIZE,
                      act_order: bool = False, wbits: int = 4) -> int:
    """Bytes the matmul must move: packed weights, scales, packed zeros,
    x, y and (act-order) the row permutation."""
    G = K // group_size
    b = K * N * wbits // 8 + G * N * 2 + G * N * wbits // 8 + M * K * 2 + M * N * 2
    if act_order:
        b += 4 * K
    return b


def matmul_flops(M: int, K: int, N: int) -> int:
    return 2 * M * K * N
