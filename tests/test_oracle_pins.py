"""Pins for the CPU oracle (no GPU needed).

The oracle is what every CUDA result is compared with, so it is checked here
against things that are not itself: a hand-packed layer decoded by hand,
brute force with exact rational arithmetic, closed forms, and special cases
that reduce to textbook results.  The paper (Opt4GPTQ) prints no value for the
matmul, so none of these is a printed example; they pin the definition.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2511_19438_b200 import workloads as wl
from tests.golden.loader import hex_words, load_fixture, numbers


# --------------------------------------------------------------------------- helpers
def local_pack_words(nibbles_8):
    """Test-local packer, written independently of the generator module: builds the
    32-bit word digit by digit from Python ints (nibble 0 is the least significant)."""
    word = 0
    for i, v in enumerate(nibbles_8):
        assert 0 <= int(v) <= 15
        word += int(v) * (16 ** i)
    return word


def local_pack_k(q):
    K, N = q.shape
    out = np.zeros((K // 8, N), dtype=np.uint32)
    for r in range(K // 8):
        for n in range(N):
            out[r, n] = local_pack_words(q[8 * r:8 * r + 8, n])
    return out.view(np.int32)


def local_pack_n(z):
    G, N = z.shape
    out = np.zeros((G, N // 8), dtype=np.uint32)
    for g in range(G):
        for c in range(N // 8):
            out[g, c] = local_pack_words(z[g, 8 * c:8 * c + 8])
    return out.view(np.int32)


@pytest.fixture(scope="module")
def tiny():
    f = load_fixture("tiny_k16_n8.txt")
    return dict(
        K=f["K"], N=f["N"], gs=f["group_size"],
        qweight=hex_words(f["qweight"]), qzeros=hex_words(f["qzeros"]),
        q=numbers(f["q"], np.int64), z=numbers(f["z"], np.int64),
        scales=numbers(f["scales"], np.float16), g_idx=numbers(f["g_idx"], np.int32)[0],
        x=numbers(f["x"], np.float16),
    )


# --------------------------------------------------------------------------- fp16 decode
def test_half_to_float_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


# --------------------------------------------------------------------------- hand-packed layer
def test_fixture_shapes(tiny):
    assert tiny["qweight"].shape == (2, 8) and tiny["qzeros"].shape == (2, 1)
    assert tiny["q"].shape == (16, 8) and tiny["z"].shape == (2, 8)


def test_unpack_matches_hand_decoded_nibbles(tiny):
    assert np.array_equal(oracle.unpack_q(tiny["qweight"]), tiny["q"].astype(np.uint8))
    assert np.array_equal(oracle.unpack_z(tiny["qzeros"]), tiny["z"].astype(np.uint8))


def test_dequant_matches_hand_tables(tiny):
    q, z, s, gs = tiny["q"], tiny["z"], tiny["scales"].astype(np.float64), tiny["gs"]
    w = oracle.dequant_f32(tiny["qweight"], tiny["qzeros"], tiny["scales"], None, gs)
    for k in range(16):
        for n in range(8):
            assert float(w[k, n]) == float((q[k, n] - z[k // gs, n]) * s[k // gs, n]), (k, n)
    # a few entries written out literally: (q - z) * s
    assert w[0, 0] == -1.0          # (0 - 1) * 1
    assert w[7, 5] == 1.125         # (15 - 6) * 0.125
    assert w[15, 7] == -0.125       # (13 - 15) * 0.0625
    assert w[8, 3] == 4.0           # (15 - 13) * 2
    assert w[3, 6] == 8.0           # (9 - 7) * 4


def test_dequant_act_order_matches_hand_tables(tiny):
    q, z, s, g_idx = tiny["q"], tiny["z"], tiny["scales"].astype(np.float64), tiny["g_idx"]
    w = oracle.dequant_f32(tiny["qweight"], tiny["qzeros"], tiny["scales"], g_idx, tiny["gs"])
    for k in range(16):
        g = int(g_idx[k])
        for n in range(8):
            assert float(w[k, n]) == float((q[k, n] - z[g, n]) * s[g, n]), (k, n)
    assert w[1, 0] == -1.0          # row 1 is in group 1: (1 - 3) * 0.5
    assert w[9, 7] == 6.0           # row 9 is in group 0: (14 - 8) * 1


def brute_force_y(x, q, z, s, groups):
    """Exact rational y[m][n] from the hand tables."""
    M, K = x.shape
    N = q.shape[1]
    y = [[Fraction(0) for _ in range(N)] for _ in range(M)]
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                g = groups[k]
                acc += Fraction(float(x[m, k])) * (int(q[k, n]) - int(z[g, n])) * Fraction(float(s[g, n]))
            y[m][n] = acc
    return y


@pytest.mark.parametrize("act_order", [False, True])
def test_gemm_matches_rational_brute_force(tiny, act_order):
    g_idx = tiny["g_idx"] if act_order else None
    groups = [int(g) for g in tiny["g_idx"]] if act_order else [k // tiny["gs"] for k in range(16)]
    want = brute_force_y(tiny["x"], tiny["q"], tiny["z"], tiny["scales"], groups)
    got = oracle.gemm_f64(tiny["x"], tiny["qweight"], tiny["qzeros"], tiny["scales"], g_idx, tiny["gs"])
    for m in range(2):
        for n in range(8):
            assert Fraction(float(got[m, n])) == want[m][n], (m, n)
    if not act_order:
        # column 0, x = ones: group 0 gives (0+..+7 - 8*1)*1 = 20, group 1 gives (28 - 8*3)*0.5 = 2
        assert got[0, 0] == 22.0


# --------------------------------------------------------------------------- invariants
@pytest.mark.parametrize("K,N,gs,seed", [(32, 16, 8, 1), (256, 24, 128, 2), (384, 40, 128, 3)])
def test_dequant_of_pack_reproduces_q_minus_z_times_s(K, N, gs, seed):
    r = np.random.default_rng(seed)
    G = K // gs
    q = r.integers(0, 16, (K, N), dtype=np.uint8)
    z = r.integers(0, 16, (G, N), dtype=np.uint8)
    s = wl.make_scales(G, N, seed)
    qw, qz = local_pack_k(q), local_pack_n(z)
    # the generator's packer must agree with the digit-by-digit one
    assert np.array_equal(qw, wl.pack_along_k(q)) and np.array_equal(qz, wl.pack_along_n(z))
    assert np.array_equal(oracle.unpack_q(qw), q) and np.array_equal(oracle.unpack_z(qz), z)
    w = oracle.dequant_f32(qw, qz, s, None, gs)
    grp = np.arange(K) // gs
    want64 = (q.astype(np.int64) - z[grp].astype(np.int64)).astype(np.float64) * s[grp].astype(np.float64)
    # <= 4 significant bits times <= 11 significant bits: the fp32 product is the exact real product
    assert np.array_equal(w.astype(np.float64), want64)
    assert np.array_equal(w, want64.astype(np.float32))


def test_act_order_with_trivial_g_idx_is_bit_identical():
    L = wl.make_linear(512, 64, seed=11)
    g_idx = (np.arange(512) // 128).astype(np.int32)
    a = oracle.dequant_f32(L.qweight, L.qzeros, L.scales, None, 128)
    b = oracle.dequant_f32(L.qweight, L.qzeros, L.scales, g_idx, 128)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    x = wl.make_x(3, 512, 12)
    ya = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, None, 128)
    yb = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, g_idx, 128)
    assert np.array_equal(ya, yb)


def test_row_permutation_leaves_y_unchanged():
    """Permuting (rows of q, entries of g_idx, columns of x) by the same permutation
    is a reordering of the sum over k only."""
    K, N, gs = 512, 48, 128
    L = wl.make_linear(K, N, seed=21, act_order=True)
    x = wl.make_x(4, K, 22)
    y0 = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs)
    p = np.random.default_rng(23).permutation(K)
    q = oracle.unpack_q(L.qweight)
    qw_p = local_pack_k(q[p])
    y1 = oracle.gemm_f64(np.ascontiguousarray(x[:, p]), qw_p, L.qzeros, L.scales, L.g_idx[p], gs)
    assert np.allclose(y0, y1, rtol=1e-12, atol=1e-12)
    assert not np.allclose(y0, oracle.gemm_f64(x, qw_p, L.qzeros, L.scales, L.g_idx[p], gs), atol=1e-3)


# --------------------------------------------------------------------------- GEMM special cases
def test_one_hot_x_selects_a_row_of_w():
    L = wl.make_linear(256, 32, seed=31, act_order=True)
    w = oracle.dequant_f32(L.qweight, L.qzeros, L.scales, L.g_idx, 128)
    for k in (0, 7, 8, 129, 255):
        x = np.zeros((1, 256), dtype=np.float16)
        x[0, k] = 1.0
        y = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, 128)
        assert np.array_equal(y[0], w[k].astype(np.float64))


def test_all_ones_x_gives_column_sums():
    L = wl.make_linear(384, 24, seed=41)
    w = oracle.dequant_f32(L.qweight, L.qzeros, L.scales, None, 128).astype(np.float64)
    y = oracle.gemm_f64(np.ones((1, 384), dtype=np.float16), L.qweight, L.qzeros, L.scales, None, 128)
    for n in range(24):
        assert abs(y[0, n] - math.fsum(w[:, n])) <= 1e-12 * max(1.0, abs(y[0, n]))


def test_integer_case_is_an_exact_integer_matrix_product():
    """z = 8, s = 1, small-integer x: y is the integer product x . (q - 8), exact in fp64."""
    K, N, M, gs = 256, 40, 5, 128
    r = np.random.default_rng(51)
    q = r.integers(0, 16, (K, N), dtype=np.uint8)
    z = np.full((K // gs, N), 8, dtype=np.uint8)
    s = np.ones((K // gs, N), dtype=np.float16)
    xi = r.integers(-4, 5, (M, K))
    L = wl.make_linear_from_values(q, z, s, gs)
    y = oracle.gemm_f64(xi.astype(np.float16), L.qweight, L.qzeros, L.scales, None, gs)
    want = xi.astype(np.int64) @ (q.astype(np.int64) - 8)
    assert np.array_equal(y, want.astype(np.float64))


def test_transposed_or_swapped_operands_would_be_caught():
    """A non-square, non-symmetric case: the result has shape [M, N] and differs from
    what x^T or W^T conventions would give."""
    K, N, M, gs = 128, 8, 2, 128
    q = np.zeros((K, N), dtype=np.uint8)
    q[5, 3] = 9                       # the only non-zero weight after z = 0
    z = np.zeros((1, N), dtype=np.uint8)
    s = np.full((1, N), 0.5, dtype=np.float16)
    x = np.zeros((M, K), dtype=np.float16)
    x[1, 5] = 2.0
    L = wl.make_linear_from_values(q, z, s, gs)
    y = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, None, gs)
    want = np.zeros((M, N))
    want[1, 3] = 9.0                  # 2 * (9 - 0) * 0.5
    assert np.array_equal(y, want)


def numpy_unpack(qweight, qzeros):
    K8, N = qweight.shape
    sh = (4 * np.arange(8, dtype=np.uint32))
    q = ((qweight.view(np.uint32)[:, None, :] >> sh[None, :, None]) & 15).reshape(K8 * 8, N)
    z = ((qzeros.view(np.uint32)[:, :, None] >> sh[None, None, :]) & 15).reshape(qzeros.shape[0], N)
    return q.astype(np.int64), z.astype(np.int64)


@pytest.mark.parametrize("K,N,act", [(4096, 4096, False), (5120, 1024, True)])
def test_against_library_fp64_matmul(K, N, act):
    """Config-1 shape (and one act-order shape) against numpy's fp64 matmul over a
    vectorised unpack: a different summation routine over the same definition."""
    L = wl.make_linear(K, N, seed=wl.seed_for("pin", K, N, act), act_order=act)
    x = wl.make_x(2, K, wl.seed_for("pin-x", K))
    q, z = numpy_unpack(L.qweight, L.qzeros)
    grp = L.g_idx if act else np.arange(K) // 128
    w = (q - z[grp]).astype(np.float64) * L.scales[grp].astype(np.float64)
    want = x.astype(np.float64) @ w
    got = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, 128)
    assert np.allclose(got, want, rtol=1e-11, atol=1e-10)
    # closed-form spread: var(q - z) = 2 * (16^2 - 1) / 12 = 42.5, E[s^2] from the half-normal
    # scale recipe = 0.002^2 + 2*0.002*0.01*sqrt(2/pi) + 0.01^2, var(x) = 1
    es2 = wl.SCALE_FLOOR ** 2 + 2 * wl.SCALE_FLOOR * wl.SCALE_SIGMA * math.sqrt(2 / math.pi) + wl.SCALE_SIGMA ** 2
    std_want = math.sqrt(K * 42.5 * es2)
    assert abs(got.std() / std_want - 1) < 0.04


def test_sampled_outputs_equal_full_product():
    L = wl.make_linear(256, 64, seed=61, act_order=True)
    x = wl.make_x(6, 256, 62)
    full = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, 128)
    rows = np.array([0, 5, 3, 3, 1], dtype=np.int32)
    cols = np.array([63, 0, 17, 18, 40], dtype=np.int32)
    at = oracle.gemm_f64_at(x, L.qweight, L.qzeros, L.scales, L.g_idx, 128, rows, cols)
    assert np.array_equal(at, full[rows, cols])


def test_generator_distributions():
    L = wl.make_linear(1024, 512, seed=71, act_order=True)
    q = oracle.unpack_q(L.qweight)
    z = oracle.unpack_z(L.qzeros)
    assert abs(q.mean() - 7.5) < 0.05 and abs(z.mean() - 7.5) < 0.2
    assert np.bincount(q.ravel(), minlength=16).min() > 0.9 * q.size / 16
    assert np.array_equal(np.bincount(L.g_idx, minlength=8), np.full(8, 128))
    s = L.scales.astype(np.float64)
    assert s.min() >= 0.002 - 1e-5 and abs(s.mean() - (0.002 + 0.01 * math.sqrt(2 / math.pi))) < 2e-4


# --------------------------------------------------------------------------- zero points stored minus one
def test_v1_zeros_hand_values(tiny):
    """The hand-packed layer read with the older convention (stored nibble = z - 1): every zero point is one
    larger than the hand table, so every weight is one scale smaller; the stored 15 of group 1, column 7 means 16."""
    q, z, s, gs = tiny["q"], tiny["z"], tiny["scales"].astype(np.float64), tiny["gs"]
    w = oracle.dequant_f32(tiny["qweight"], tiny["qzeros"], tiny["scales"], None, gs, zeros_minus_one=True)
    for k in range(16):
        for n in range(8):
            assert float(w[k, n]) == float((q[k, n] - (z[k // gs, n] + 1)) * s[k // gs, n]), (k, n)
    assert w[0, 0] == -2.0          # (0 - (1 + 1)) * 1
    assert w[7, 5] == 1.0           # (15 - (6 + 1)) * 0.125
    assert w[15, 7] == -0.1875      # (13 - (15 + 1)) * 0.0625: the stored 15 is the zero point 16
    assert w[8, 3] == 2.0           # (15 - (13 + 1)) * 2


def test_v1_zeros_repacked_by_hand_equal_plain_reading(tiny):
    """Pack z - 1 digit by digit (test-local packer) where every z >= 1: the older reading of those words must give
    bit for bit what the plain reading gives on the original words."""
    z = tiny["z"].copy()
    z[z == 0] = 1                                   # the hand table has one zero point equal to 0
    qz_plain = local_pack_n(z)
    qz_minus_one = local_pack_n(z - 1)
    a = oracle.dequant_f32(tiny["qweight"], qz_plain, tiny["scales"], tiny["g_idx"], tiny["gs"])
    b = oracle.dequant_f32(tiny["qweight"], qz_minus_one, tiny["scales"], tiny["g_idx"], tiny["gs"], zeros_minus_one=True)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_v1_gemm_is_plain_gemm_minus_scaled_group_sums_of_x():
    """(q - z - 1) s = (q - z) s - s, so y_v1 = y_plain - sum_g s[g, n] * sum_{k in g} x[m, k]: an identity that ties the
    second matmul function to the first through a computation done here in numpy fp64."""
    K, N, M, gs = 256, 24, 3, 32
    L = wl.make_linear(K, N, seed=91, group_size=gs, act_order=True)
    x = wl.make_x(M, K, 92)
    y_plain = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs)
    y_v1 = oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs, zeros_minus_one=True)
    xs = np.zeros((M, K // gs))
    for k in range(K):
        xs[:, L.g_idx[k]] += x[:, k].astype(np.float64)
    corr = xs @ L.scales.astype(np.float64)
    assert np.allclose(y_v1, y_plain - corr, rtol=0, atol=1e-9 * np.abs(y_plain).max())
    # and it is the matmul of its own dequantised weights
    w = oracle.dequant_f32(L.qweight, L.qzeros, L.scales, L.g_idx, gs, zeros_minus_one=True).astype(np.float64)
    assert np.allclose(y_v1, x.astype(np.float64) @ w, rtol=1e-13, atol=1e-12)


# --------------------------------------------------------------------------- silu(gate) * up
def test_silu_mul_special_values():
    y = np.array([[0.0, 1.0, -1.0, 40.0, -40.0, 2.0,      # gate
                   3.0, 2.0, 2.0, 0.5, 7.0, -1.5]])       # up
    out = oracle.silu_mul_f64(y)[0]
    assert out[0] == 0.0                                   # silu(0) = 0
    assert abs(out[1] - 2 * 0.7310585786300049) < 1e-15    # silu(1) = 1 / (1 + e^-1)
    assert abs(out[2] - 2 * -0.2689414213699951) < 1e-15   # silu(-1) = -1 / (1 + e)
    assert abs(out[3] - 20.0) < 1e-12                      # silu(t) -> t for large t
    assert abs(out[4]) < 1e-14                             # silu(t) -> 0 for very negative t
    assert abs(out[5] - (-1.5) * 2 / (1 + math.exp(-2))) < 1e-15


def test_silu_mul_against_the_tanh_form_and_its_symmetry():
    r = np.random.default_rng(3)
    y = r.normal(0, 4, (5, 64))
    out = oracle.silu_mul_f64(y)
    g, u = y[:, :32], y[:, 32:]
    assert np.allclose(out, g * 0.5 * (1 + np.tanh(g / 2)) * u, rtol=1e-13, atol=1e-15)   # sigmoid(t) = (1 + tanh(t/2)) / 2
    neg = oracle.silu_mul_f64(np.concatenate([-g, u], axis=1))
    assert np.allclose(out - neg, g * u, rtol=1e-13, atol=1e-13)                           # silu(t) - silu(-t) = t
    # gate columns first, up columns second: swapping the halves is a different function
    assert not np.allclose(out, oracle.silu_mul_f64(np.concatenate([u, g], axis=1)))


# ------------------------------------------------------------------------------- bias and residual
def test_add_bias_residual_small_integers_are_exact_and_oriented():
    """Small integers are exact in fp16 and fp64, so the sum has one right answer; a non-square case with a bias that
    counts columns and a residual that counts rows shows which operand goes along which axis."""
    M, N = 3, 5
    y = np.arange(M * N, dtype=np.float64).reshape(M, N) * 0.25
    bias = np.arange(N).astype(np.float16)                                  # bias[n] = n
    resid = np.repeat(np.arange(M)[:, None] * 100, N, axis=1).astype(np.float16)   # residual[m, n] = 100 m
    out = oracle.add_bias_residual_f64(y, bias, resid)
    for m in range(M):
        for n in range(N):
            assert out[m, n] == 0.25 * (m * N + n) + n + 100 * m
    assert np.array_equal(oracle.add_bias_residual_f64(y, None, None), y)
    assert np.array_equal(oracle.add_bias_residual_f64(y, bias, None) - y, np.tile(np.arange(N, dtype=np.float64), (M, 1)))
    assert np.array_equal(oracle.add_bias_residual_f64(y, None, resid) - y, resid.astype(np.float64))


def test_add_bias_residual_reads_fp16_exactly_and_adds_in_double():
    """The operands are the fp16 values themselves (0.1 is not representable: its fp16 neighbour is what is added), and
    the sum keeps what a single-precision sum would lose."""
    y = np.array([[1e8, -3.0]])
    bias = np.array([0.1, 65504.0], np.float16)
    resid = np.array([[1.0, 2.0 ** -24]], np.float16)                       # the smallest fp16 subnormal
    out = oracle.add_bias_residual_f64(y, bias, resid)
    assert out[0, 0] == 1e8 + 0.0999755859375 + 1.0                         # fp16(0.1) = 0.0999755859375; exact in fp64
    assert out[0, 1] == -3.0 + 65504.0 + 2.0 ** -24
    assert np.float32(1e8) + np.float32(0.0999755859375) == np.float32(1e8)   # fp32 would have dropped the bias


# --------------------------------------------------------------------------- bfloat16 activations and scales
def torch_bf16_bits_to_f64(bits):
    """bfloat16 bit patterns -> float64 through torch's own bfloat16 type (a library routine, not the oracle's shift)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def test_bfloat16_to_float_all_bit_patterns_against_torch():
    bits = np.arange(65536, dtype=np.uint16)
    want = torch_bf16_bits_to_f64(bits).astype(np.float32)
    got = np.array([oracle.bfloat16_to_float(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))
    # literal values from the format: 1 sign, 8 exponent (bias 127), 7 fraction bits
    assert oracle.bfloat16_to_float(0x3FC0) == 1.5
    assert oracle.bfloat16_to_float(0x4049) == 3.140625
    assert oracle.bfloat16_to_float(0xC2F7) == -123.5
    assert oracle.bfloat16_to_float(0x3080) == 2.0 ** -30        # far below the smallest fp16 subnormal
    assert oracle.bfloat16_to_float(0x0001) == 2.0 ** -133       # the smallest subnormal


def test_bf16_generator_rounds_to_nearest_even_like_torch():
    import torch
    a = np.concatenate([np.random.default_rng(5).standard_normal(4096).astype(np.float32) * 3,
                        np.array([1.00390625, 1.01171875, 1.0, -0.0, 3.0e38, 1e-40, 0.002, 65504.0], dtype=np.float32)])
    want = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(wl.bf16_bits(a), want)
    assert wl.bf16_bits(np.array([1.00390625], np.float32))[0] == 0x3F80     # tie: down to the even 1.0
    assert wl.bf16_bits(np.array([1.01171875], np.float32))[0] == 0x3F82     # tie: up to the even 1.015625


def test_bf16_dequant_hand_values(tiny):
    """The hand-packed layer with bfloat16 scales typed as bit patterns, among them values fp16 cannot hold
    (2^-30, 2^100) and one with all seven fraction bits set: every weight is (q - z) s exactly."""
    q, z, gs = tiny["q"], tiny["z"], tiny["gs"]
    s_bits = np.array([[0x3F80, 0x3F00, 0x3080, 0x7180, 0x3FFF, 0xBE80, 0x4000, 0x3E00],
                       [0x3F00, 0x3F80, 0x4040, 0x3080, 0x3C00, 0x3FC0, 0xC000, 0x3D80]], dtype=np.uint16)
    s = [[1.0, 0.5, 2.0 ** -30, 2.0 ** 100, 1.9921875, -0.25, 2.0, 0.125],
         [0.5, 1.0, 3.0, 2.0 ** -30, 2.0 ** -7, 1.5, -2.0, 0.0625]]
    w = oracle.dequant_f32_bf16(tiny["qweight"], tiny["qzeros"], s_bits, None, gs)
    for k in range(16):
        for n in range(8):
            assert float(w[k, n]) == float(np.float32((int(q[k, n]) - int(z[k // gs, n])) * s[k // gs][n])), (k, n)
    assert w[0, 0] == -1.0                    # (0 - 1) * 1
    assert w[7, 4] == (int(q[7, 4]) - int(z[0, 4])) * 1.9921875
    # the older zero convention: every weight one scale smaller
    w1 = oracle.dequant_f32_bf16(tiny["qweight"], tiny["qzeros"], s_bits, None, gs, zeros_minus_one=True)
    for k in range(16):
        for n in range(8):
            assert float(w1[k, n]) == float(np.float32((int(q[k, n]) - int(z[k // gs, n]) - 1) * s[k // gs][n])), (k, n)
    # act-order: row k uses the scales and zeros of group g_idx[k]
    wa = oracle.dequant_f32_bf16(tiny["qweight"], tiny["qzeros"], s_bits, tiny["g_idx"], gs)
    for k in range(16):
        g = int(tiny["g_idx"][k])
        for n in range(8):
            assert float(wa[k, n]) == float(np.float32((int(q[k, n]) - int(z[g, n])) * s[g][n])), (k, n)


@pytest.mark.parametrize("act_order", [False, True])
def test_bf16_gemm_matches_rational_brute_force(tiny, act_order):
    """Exact rational arithmetic over the hand tables, with bfloat16 x and scales typed as bit patterns whose values
    are written out beside them (so a wrong bit-field reading, or a detour through fp16, fails)."""
    s_bits = np.array([[0x3F80, 0x3F00, 0x3080, 0x3FFF, 0x3E00, 0xBE80, 0x4000, 0x3E00],
                       [0x3F00, 0x3F80, 0x4040, 0x3080, 0x3C00, 0x3FC0, 0xC000, 0x3D80]], dtype=np.uint16)
    s = np.array([[1.0, 0.5, 2.0 ** -30, 1.9921875, 0.125, -0.25, 2.0, 0.125],
                  [0.5, 1.0, 3.0, 2.0 ** -30, 2.0 ** -7, 1.5, -2.0, 0.0625]])
    x_vals = np.array([[1.0] * 16,
                       [0.5, -2.0, 3.0, 2.0 ** -20, 1.5, -0.0078125, 96.0, 1.0078125,
                        -1.0, 0.25, 7.0, -3.0, 2.0 ** 20, 0.0, 1.25, -0.75]])
    x_bits = wl.bf16_bits(x_vals)
    assert np.array_equal(torch_bf16_bits_to_f64(x_bits), x_vals)          # all exactly representable
    g_idx = tiny["g_idx"] if act_order else None
    groups = [int(g) for g in tiny["g_idx"]] if act_order else [k // tiny["gs"] for k in range(16)]
    want = brute_force_y(x_vals, tiny["q"], tiny["z"], s, groups)
    got = oracle.gemm_f64_bf16(x_bits, tiny["qweight"], tiny["qzeros"], s_bits, g_idx, tiny["gs"])
    for m in range(2):
        for n in range(8):
            assert abs(Fraction(float(got[m, n])) - want[m][n]) <= abs(want[m][n]) * Fraction(1, 2 ** 48), (m, n)
    if not act_order:
        assert got[0, 0] == 22.0          # as in the fp16 case: column 0 has scales 1 and 0.5


@pytest.mark.parametrize("K,N,act,gs", [(4096, 4096, False, 128), (5120, 1024, True, 128), (512, 256, True, 32)])
def test_bf16_gemm_against_library_fp64_matmul(K, N, act, gs):
    """numpy's fp64 matmul over a vectorised unpack, with torch turning the bfloat16 bits into numbers."""
    L = wl.make_linear(K, N, seed=wl.seed_for("pin-bf16", K, N, act), group_size=gs, act_order=act)
    s_bits = wl.make_scales_bf16(K // gs, N, wl.seed_for("pin-bf16-s", K, N))
    x_bits = wl.make_x_bf16(3, K, wl.seed_for("pin-bf16-x", K))
    q, z = numpy_unpack(L.qweight, L.qzeros)
    grp = L.g_idx if act else np.arange(K) // gs
    s64 = torch_bf16_bits_to_f64(s_bits)
    w = (q - z[grp]).astype(np.float64) * s64[grp]
    want = torch_bf16_bits_to_f64(x_bits) @ w
    got = oracle.gemm_f64_bf16(x_bits, L.qweight, L.qzeros, s_bits, L.g_idx, gs)
    assert np.allclose(got, want, rtol=1e-11, atol=1e-10)
    assert np.array_equal(oracle.dequant_f32_bf16(L.qweight, L.qzeros, s_bits, L.g_idx, gs).astype(np.float64), w)
    # the older zero convention: y_v1 = y - sum_g s[g, n] * sum_{k in g} x[m, k]
    got1 = oracle.gemm_f64_bf16(x_bits, L.qweight, L.qzeros, s_bits, L.g_idx, gs, zeros_minus_one=True)
    xs = np.zeros((3, K // gs))
    np.add.at(xs.T, grp, torch_bf16_bits_to_f64(x_bits).T)
    assert np.allclose(got1, want - xs @ s64, rtol=0, atol=1e-9 * np.abs(want).max())


def test_bf16_sampled_outputs_equal_full_product():
    L = wl.make_linear(256, 64, seed=71, act_order=True)
    s_bits = wl.make_scales_bf16(2, 64, 72)
    x_bits = wl.make_x_bf16(6, 256, 73)
    for zm in (False, True):
        full = oracle.gemm_f64_bf16(x_bits, L.qweight, L.qzeros, s_bits, L.g_idx, 128, zeros_minus_one=zm)
        rows = np.array([0, 5, 3, 3, 1], dtype=np.int32)
        cols = np.array([0, 63, 17, 18, 40], dtype=np.int32)
        at = oracle.gemm_f64_bf16_at(x_bits, L.qweight, L.qzeros, s_bits, L.g_idx, 128, rows, cols, zeros_minus_one=zm)
        assert np.array_equal(at, full[rows, cols])


# --------------------------------------------------------------------------- groups coarser than 128 rows
@pytest.mark.parametrize("gs,act", [(256, False), (256, True), (512, False), (512, True)])
def test_coarse_groups_and_per_channel_against_library_matmul(gs, act):
    """group_size 256 and group_size = K (one scale and zero point per column): numpy's fp64 matmul over a vectorised
    unpack, and the hand check that with one group every row of a column uses the same scale and zero point."""
    K, N, M = 512, 64, 3
    L = wl.make_linear(K, N, seed=wl.seed_for("pin-coarse", gs, act), group_size=gs, act_order=act)
    assert L.scales.shape == (K // gs, N) and L.qzeros.shape == (K // gs, N // 8)
    x = wl.make_x(M, K, wl.seed_for("pin-coarse-x", gs))
    q, z = numpy_unpack(L.qweight, L.qzeros)
    grp = L.g_idx if act else np.arange(K) // gs
    w = (q - z[grp]).astype(np.float64) * L.scales[grp].astype(np.float64)
    got_w = oracle.dequant_f32(L.qweight, L.qzeros, L.scales, L.g_idx, gs)
    assert np.array_equal(got_w.astype(np.float64), w)
    assert np.allclose(oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs), x.astype(np.float64) @ w,
                       rtol=1e-12, atol=1e-12)
    if gs == K:
        assert np.array_equal(w, (q - z[0][None, :]) * L.scales[0].astype(np.float64)[None, :])


# --------------------------------------------------------------------------- 8-bit weights
def local_pack_bytes(vals_4):
    """Test-local packer for 8-bit fields: the 32-bit word digit by digit in base 256 (byte 0 least significant)."""
    word = 0
    for i, v in enumerate(vals_4):
        assert 0 <= int(v) <= 255
        word += int(v) * (256 ** i)
    return word


def local_pack8_k(q):
    K, N = q.shape
    out = np.zeros((K // 4, N), dtype=np.uint32)
    for r in range(K // 4):
        for n in range(N):
            out[r, n] = local_pack_bytes(q[4 * r:4 * r + 4, n])
    return out.view(np.int32)


def local_pack8_n(z):
    G, N = z.shape
    out = np.zeros((G, N // 4), dtype=np.uint32)
    for g in range(G):
        for c in range(N // 4):
            out[g, c] = local_pack_bytes(z[g, 4 * c:4 * c + 4])
    return out.view(np.int32)


def test_w8_unpack_hand_typed_words():
    """Words typed as hex and decoded by hand: 0x04030201 holds rows 1, 2, 3, 4 (least significant byte first), the
    sign bit is just the top bit of the fourth byte, and a zero-point word holds four neighbouring columns."""
    qweight = np.array([[0x04030201, 0xFF00807F], [0x80000000, 0x12345678]], dtype=np.uint32).view(np.int32)
    want_q = np.array([[1, 0x7F], [2, 0x80], [3, 0x00], [4, 0xFF],
                       [0, 0x78], [0, 0x56], [0, 0x34], [0x80, 0x12]], dtype=np.uint8)
    assert np.array_equal(oracle.unpack_q8(qweight), want_q)
    qzeros = np.array([[0xDEADBEEF, 0x00FF0102]], dtype=np.uint32).view(np.int32)
    assert np.array_equal(oracle.unpack_z8(qzeros), np.array([[0xEF, 0xBE, 0xAD, 0xDE, 0x02, 0x01, 0xFF, 0x00]], dtype=np.uint8))
    # the generator's packers agree with the digit-by-digit ones
    r = np.random.default_rng(3)
    q = r.integers(0, 256, (16, 8)).astype(np.uint8)
    z = r.integers(0, 256, (2, 8)).astype(np.uint8)
    assert np.array_equal(wl.pack8_along_k(q), local_pack8_k(q)) and np.array_equal(wl.pack8_along_n(z), local_pack8_n(z))
    assert np.array_equal(oracle.unpack_q8(local_pack8_k(q)), q) and np.array_equal(oracle.unpack_z8(local_pack8_n(z)), z)


@pytest.mark.parametrize("act_order", [False, True])
@pytest.mark.parametrize("zm1", [False, True])
def test_w8_dequant_and_gemm_match_rational_brute_force(act_order, zm1):
    K, N, M, gs = 16, 8, 2, 8
    r = np.random.default_rng(17)
    q = r.integers(0, 256, (K, N)).astype(np.uint8)
    z = r.integers(0, 256, (K // gs, N)).astype(np.uint8)
    s = np.array([[1.0, 0.5, 0.25, 2.0, 0.125, 3.0, 0.0625, 1.5], [0.5, 1.0, 2.0, 0.75, 1.0, 0.25, 4.0, 0.375]], dtype=np.float16)
    groups = [int(g) for g in r.permutation(K) // gs] if act_order else [k // gs for k in range(K)]
    q[0, 0], z[groups[0], 0] = 0, 255               # the extremes: -255 (or -256 with the older convention)
    q[1, 1], z[groups[1], 1] = 255, 0
    g_idx = np.array(groups, dtype=np.int32) if act_order else None
    x = np.array([[1.0] * K, [0.5, -2.0, 3.0, 0.25, 1.5, -1.0, 7.0, -0.125, 2.0, 0.0, -3.0, 1.0, 0.75, -4.0, 6.0, 1.25]], dtype=np.float16)
    qw, qz = local_pack8_k(q), local_pack8_n(z)
    w = oracle.dequant_f32_w8(qw, qz, s, g_idx, gs, zeros_minus_one=zm1)
    for k in range(K):
        for n in range(N):
            assert float(w[k, n]) == (int(q[k, n]) - int(z[groups[k], n]) - int(zm1)) * float(s[groups[k], n]), (k, n)
    assert w[0, 0] == (-256.0 if zm1 else -255.0) * float(s[groups[0], 0])
    want = brute_force_y(x, q.astype(np.int64), z.astype(np.int64) + int(zm1), s, groups)
    got = oracle.gemm_f64_w8(x, qw, qz, s, g_idx, gs, zeros_minus_one=zm1)
    for m in range(M):
        for n in range(N):
            assert Fraction(float(got[m, n])) == want[m][n], (m, n)


def test_w8_with_empty_high_nibbles_is_the_4bit_layer():
    """An 8-bit layer whose weights and zero points are all below 16 is the 4-bit layer with the same values: ties the
    8-bit functions to the 4-bit ones, which have their own pins."""
    K, N, M, gs = 256, 16, 3, 64
    r = np.random.default_rng(23)
    q = r.integers(0, 16, (K, N)).astype(np.uint8)
    z = r.integers(0, 16, (K // gs, N)).astype(np.uint8)
    s = wl.make_scales(K // gs, N, 5)
    g_idx = wl.make_g_idx(K, gs, 6)
    x = wl.make_x(M, K, 7)
    L4 = wl.make_linear_from_values(q, z, s, gs, g_idx)
    for zm1 in (False, True):
        a = oracle.gemm_f64_w8(x, wl.pack8_along_k(q), wl.pack8_along_n(z), s, g_idx, gs, zeros_minus_one=zm1)
        b = oracle.gemm_f64(x, L4.qweight, L4.qzeros, L4.scales, g_idx, gs, zeros_minus_one=zm1)
        assert np.array_equal(a, b)


@pytest.mark.parametrize("K,N,act,gs", [(4096, 1024, False, 128), (1024, 512, True, 128), (512, 256, True, 32)])
def test_w8_against_library_fp64_matmul(K, N, act, gs):
    L = wl.make_linear_w8(K, N, seed=wl.seed_for("pin-w8", K, N, act), group_size=gs, act_order=act)
    x = wl.make_x(3, K, wl.seed_for("pin-w8-x", K))
    sh = (8 * np.arange(4, dtype=np.uint32))
    q = ((L.qweight.view(np.uint32)[:, None, :] >> sh[None, :, None]) & 255).reshape(K, N).astype(np.int64)
    z = ((L.qzeros.view(np.uint32)[:, :, None] >> sh[None, None, :]) & 255).reshape(K // gs, N).astype(np.int64)
    grp = L.g_idx if act else np.arange(K) // gs
    w = (q - z[grp]).astype(np.float64) * L.scales[grp].astype(np.float64)
    got = oracle.gemm_f64_w8(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs)
    assert np.allclose(got, x.astype(np.float64) @ w, rtol=1e-11, atol=1e-9)
    assert np.array_equal(oracle.dequant_f32_w8(L.qweight, L.qzeros, L.scales, L.g_idx, gs).astype(np.float64), w)
    # closed-form spread: var(q - z) = 2 * (256^2 - 1) / 12
    es2 = wl.SCALE_FLOOR ** 2 + 2 * wl.SCALE_FLOOR * wl.SCALE_SIGMA * math.sqrt(2 / math.pi) + wl.SCALE_SIGMA ** 2
    assert abs(got.std() / math.sqrt(K * (2 * (256 ** 2 - 1) / 12) * es2) - 1) < 0.06
    rows = np.array([0, 2, 1, 1], dtype=np.int32)
    cols = np.array([0, N - 1, 17, 18], dtype=np.int32)
    assert np.array_equal(oracle.gemm_f64_w8_at(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs, rows, cols), got[rows, cols])


# --------------------------------------------------------------------------- 2- and 3-bit weights
def local_pack_stream(vals, bits):
    """Test-local packer: one big Python integer holds the bit stream (value i at bit bits * i), cut into 32-bit words."""
    big = 0
    for i, v in enumerate(vals):
        assert 0 <= int(v) < (1 << bits)
        big += int(v) << (bits * i)
    n_words = len(vals) * bits // 32
    return [(big >> (32 * w)) & 0xFFFFFFFF for w in range(n_words)]


def test_wn_unpack_hand_typed_words():
    """3 bits: the values 0..7 take 24 bits, 0xFAC688 (0 in bits 0-2, 1 in 3-5, ... 7 in 21-23); four times over they
    fill three words, cut from the 96-bit stream 0xFAC688FAC688FAC688FAC688 at 32-bit boundaries: 0x88FAC688, 0xC688FAC6,
    0xFAC688FA.  Value 10 (= 2) then has its low two bits at the top of word 0 and its high bit at the bottom of word 1,
    value 21 (= 5) its low bit at the top of word 1.  2 bits: 0xE4 repeated is the sequence 0, 1, 2, 3."""
    vals = [i % 8 for i in range(32)]
    typed = np.array([[0x88FAC688], [0xC688FAC6], [0xFAC688FA]], dtype=np.uint32)
    assert local_pack_stream(vals, 3) == [int(w) for w in typed[:, 0]]
    # decode the typed words by hand rule: bit b of the stream is bit b % 32 of word b // 32
    stream = "".join(format(int(w), "032b")[::-1] for w in typed[:, 0])
    by_hand = [int(stream[3 * i:3 * i + 3][::-1], 2) for i in range(32)]
    assert by_hand == vals
    assert np.array_equal(oracle.unpack_qn(typed.view(np.int32), 3)[:, 0], np.array(vals, dtype=np.uint8))
    assert np.array_equal(oracle.unpack_zn(typed.T.copy().view(np.int32), 3)[0], np.array(vals, dtype=np.uint8))
    two = np.array([[0xE4E4E4E4]], dtype=np.uint32).view(np.int32)
    assert np.array_equal(oracle.unpack_qn(two, 2)[:, 0], np.array([0, 1, 2, 3] * 4, dtype=np.uint8))
    assert np.array_equal(oracle.unpack_zn(two, 2)[0], np.array([0, 1, 2, 3] * 4, dtype=np.uint8))


@pytest.mark.parametrize("bits", [2, 3])
def test_wn_generator_packer_agrees_with_the_big_integer_packer(bits):
    r = np.random.default_rng(41 + bits)
    v = r.integers(0, 1 << bits, (5, 64)).astype(np.uint8)
    got = wl.pack_bits_stream(v, bits).view(np.uint32)
    for row in range(5):
        assert [int(w) for w in got[row]] == local_pack_stream(v[row], bits)
    assert np.array_equal(oracle.unpack_zn(got.view(np.int32), bits), v)


@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("act_order,zm1", [(False, False), (True, True)])
def test_wn_dequant_and_gemm_match_rational_brute_force(bits, act_order, zm1):
    K, N, M, gs = 32, 32, 2, 16
    r = np.random.default_rng(50 + bits)
    q = r.integers(0, 1 << bits, (K, N)).astype(np.uint8)
    z = r.integers(0, 1 << bits, (K // gs, N)).astype(np.uint8)
    s = (2.0 ** r.integers(-4, 3, (K // gs, N))).astype(np.float16) * np.where(r.random((K // gs, N)) < 0.3, 1.5, 1.0).astype(np.float16)
    groups = [int(g) for g in r.permutation(K) // gs] if act_order else [k // gs for k in range(K)]
    g_idx = np.array(groups, dtype=np.int32) if act_order else None
    x = r.integers(-8, 9, (M, K)).astype(np.float16) / np.float16(4)
    qw = np.array([local_pack_stream(q[:, n], bits) for n in range(N)], dtype=np.uint32).T.copy().view(np.int32)
    qz = np.array([local_pack_stream(z[g], bits) for g in range(K // gs)], dtype=np.uint32).view(np.int32)
    w = oracle.dequant_f32_wn(qw, qz, s, g_idx, gs, bits, zeros_minus_one=zm1)
    for k in range(K):
        for n in range(N):
            assert float(w[k, n]) == (int(q[k, n]) - int(z[groups[k], n]) - int(zm1)) * float(s[groups[k], n]), (k, n)
    want = brute_force_y(x, q.astype(np.int64), z.astype(np.int64) + int(zm1), s, groups)
    got = oracle.gemm_f64_wn(x, qw, qz, s, g_idx, gs, bits, zeros_minus_one=zm1)
    for m in range(M):
        for n in range(N):
            assert Fraction(float(got[m, n])) == want[m][n], (m, n)


@pytest.mark.parametrize("bits", [2, 3])
def test_wn_layer_equals_the_4bit_layer_with_the_same_values(bits):
    """The same small values packed as a 4-bit layer must give what the (separately pinned) 4-bit functions give; and
    numpy's fp64 matmul agrees at a larger size."""
    K, N, M, gs = 1024, 256, 3, 128
    L = wl.make_linear_wn(K, N, seed=wl.seed_for("pin-wn", bits), bits=bits, group_size=gs, act_order=True)
    x = wl.make_x(M, K, wl.seed_for("pin-wn-x", bits))
    q, z = oracle.unpack_qn(L.qweight, bits), oracle.unpack_zn(L.qzeros, bits)
    L4 = wl.make_linear_from_values(q, z, L.scales, gs, L.g_idx)
    for zm1 in (False, True):
        a = oracle.gemm_f64_wn(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs, bits, zeros_minus_one=zm1)
        b = oracle.gemm_f64(x, L4.qweight, L4.qzeros, L4.scales, L.g_idx, gs, zeros_minus_one=zm1)
        assert np.array_equal(a, b)
    w = (q.astype(np.int64) - z.astype(np.int64)[L.g_idx]).astype(np.float64) * L.scales[L.g_idx].astype(np.float64)
    assert np.allclose(oracle.gemm_f64_wn(x, L.qweight, L.qzeros, L.scales, L.g_idx, gs, bits), x.astype(np.float64) @ w,
                       rtol=1e-11, atol=1e-10)
