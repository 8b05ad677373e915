"""Host-side checks of the C-ABI library that need no GPU: the shared object loads, exports
every symbol the header declares, validates arguments before touching CUDA, and plans the
stream-K partition consistently (every item covered once; the contributors the reducing CTA
expects are exactly the CTAs that write a partial tile for that panel)."""
import os
import re

import pytest

from paper_2511_19438_b200 import build as libbuild

libbuild.build()
from paper_2511_19438_b200 import binding as B  # noqa: E402
from paper_2511_19438_b200 import workloads as wl  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "gptq_b200.h")
A16 = 0x1000  # a fake, 16-byte aligned "device address"; validation never dereferences it


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(gptq_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(B._lib, n), f"{n} declared in the header but not exported"
    assert set(names) == set(B.EXPORTED), set(names) ^ set(B.EXPORTED)


def test_status_strings():
    assert B.gptq_status_string(0) == "ok"
    for code in range(-9, 0):
        assert B.gptq_status_string(code) not in ("ok", "unknown status")
    assert B.gptq_status_string(-77) == "unknown status"


def test_gemm_validation_order_without_gpu():
    ok = dict(M=1, N=4096, K=4096, group_size=128, act_order=0)

    def call(x=A16, qw=A16, qz=A16, sc=A16, gi=None, y=A16, **kw):
        a = dict(ok, **kw)
        return B.gptq_gemm(x, qw, qz, sc, gi, y, a["M"], a["N"], a["K"], a["group_size"], a["act_order"], stream=0)

    assert call(x=None) == B.GPTQ_ERR_NULL
    assert call(y=None) == B.GPTQ_ERR_NULL
    assert call(act_order=1, gi=None) == B.GPTQ_ERR_NULL
    assert call(M=0) == B.GPTQ_ERR_SHAPE
    assert call(K=4100) == B.GPTQ_ERR_SHAPE          # K % 8
    assert call(N=4097) == B.GPTQ_ERR_SHAPE
    assert call(K=4096 + 64) == B.GPTQ_ERR_SHAPE     # K % group_size
    assert call(group_size=0) == B.GPTQ_ERR_SHAPE
    assert call(x=A16 + 8) == B.GPTQ_ERR_ALIGN
    assert call(qw=A16 + 4) == B.GPTQ_ERR_ALIGN
    assert call(act_order=1, gi=A16 + 4) == B.GPTQ_ERR_ALIGN   # perm_out is read 16 bytes at a time
    assert call(group_size=16) == B.GPTQ_ERR_UNSUPPORTED   # 128, 64 and 32 have a tiled layout
    assert call(group_size=8) == B.GPTQ_ERR_UNSUPPORTED
    assert call(N=4096 + 64) == B.GPTQ_ERR_UNSUPPORTED


def test_other_entry_points_validate_without_gpu():
    assert B.gptq_unpack_u8(None, None, None, None, 128, 128, 128, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_unpack_u8(A16, A16, A16, A16, 130, 128, 128, stream=0) == B.GPTQ_ERR_SHAPE
    assert B.gptq_dequant_f32(A16, A16, A16, None, None, 128, 128, 128, 0, 0, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_dequant_f32(A16, A16, A16, None, A16, 128, 128, 128, 0, 2, stream=0) == B.GPTQ_ERR_LAYOUT
    assert B.gptq_dequant_f32(A16, A16, A16, None, A16, 64, 128, 128, 0, 1, stream=0) == B.GPTQ_ERR_UNSUPPORTED
    assert B.gptq_repack(A16, A16, A16, None, A16 + 16, None, A16, None, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_repack(A16, A16, A16, None, A16, A16 + 16, A16 + 32, None, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_LAYOUT
    assert B.gptq_repack(A16, A16, A16, None, A16 + 16, A16 + 32, A16 + 48, None, 128, 128, 16, 0, stream=0) == B.GPTQ_ERR_UNSUPPORTED
    assert B.gptq_repack_format(A16, A16, A16, None, A16 + 16, A16 + 32, A16 + 48, None, 128, 128, 64, 0, 8, stream=0) == B.GPTQ_ERR_LAYOUT
    assert B.gptq_dequant_f32_format(A16, A16, A16, None, A16, 128, 128, 128, 0, 0, B.GPTQ_FORMAT_GATE_UP, stream=0) == B.GPTQ_ERR_LAYOUT
    assert B.gptq_gemm_silu_mul(A16, A16, A16, A16, None, None, 1, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_NULL
    # the 8-bit entry points: argument checks come before any CUDA call
    assert B.gptq_repack_w8_bytes(0, 256, 512, 128) == 512 * 256 and B.gptq_repack_w8_bytes(1, 256, 512, 128) == 2 * 4 * 128 + 16
    assert B.gptq_repack_w8_bytes(2, 256, 512, 128) == 2 * 4 * 256 * 2 and B.gptq_repack_w8_bytes(3, 256, 512, 128) == 2 * 512 * 4
    assert B.gptq_repack_w8_bytes(0, 256, 512, 16) == 0 and B.gptq_repack_w8_scratch_bytes(256, 512, 16) == 0
    assert B.gptq_repack_w8_scratch_bytes(256, 512, 128) >= 512 * 256 + 2 * 4 * (128 + 512) + 2 * 512 * 4
    assert B.gptq_repack_w8(A16, A16, A16, None, A16, A16, A16, None, A16, 1 << 30, 128, 128, 128, 0, 0, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_repack_w8(A16, A16, A16, None, A16, A16, A16, A16, A16, 1 << 30, 128, 128, 128, 1, 0, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_repack_w8(A16, A16, A16, None, A16, A16, A16, A16, A16, 1 << 30, 128, 128, 128, 0, 2, stream=0) == B.GPTQ_ERR_LAYOUT
    assert B.gptq_repack_w8(A16, A16, A16, None, A16, A16, A16, A16, A16 + 16, 1 << 30, 128, 128, 128, 0, 0, stream=0) == B.GPTQ_ERR_ALIGN
    assert B.gptq_repack_w8(A16, A16, A16, None, A16, A16, A16, A16, A16 - A16 % 256 + 256, 10, 128, 128, 128, 0, 0, stream=0) == B.GPTQ_ERR_WORKSPACE
    assert B.gptq_gemm_w8(A16, A16, A16, A16, None, A16, 1, 128, 128, 128, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_gemm_w8(A16, A16, A16, A16, A16 + 4, A16, 1, 128, 128, 128, stream=0) == B.GPTQ_ERR_ALIGN
    assert B.gptq_gemm_w8(A16, A16, A16, A16, A16, A16, 1, 128, 192, 64, stream=0) == B.GPTQ_ERR_UNSUPPORTED
    assert B.gptq_dequant_f32_w8(A16, A16, A16, None, A16, 128, 128, 128, 0, 1, 0, stream=0) == B.GPTQ_ERR_NULL   # tiled: perm needed
    assert B.gptq_dequant_f32_w8(A16, A16, A16, None, A16, 128, 128, 128, 0, 0, 4, stream=0) == B.GPTQ_ERR_LAYOUT
    # 2- and 3-bit repack: checks before any CUDA call
    assert B.gptq_repack_bits_scratch_bytes(3, 256, 512, 128) >= 512 * 256 // 2 and B.gptq_repack_bits_scratch_bytes(4, 256, 512, 128) == 0
    assert B.gptq_repack_bits(5, A16, A16, A16, None, A16, A16, A16, None, A16 - A16 % 256 + 256, 1 << 30, 128, 128, 128, 0, 0, stream=0) == B.GPTQ_ERR_UNSUPPORTED
    assert B.gptq_repack_bits(2, A16, A16, A16, None, A16, A16, A16, None, None, 1 << 30, 128, 128, 128, 0, 0, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_repack_bits(2, A16, A16, A16, None, A16, A16, A16, None, A16 - A16 % 256 + 256, 8, 128, 128, 128, 0, 0, stream=0) == B.GPTQ_ERR_WORKSPACE
    assert B.gptq_dequant_f32_bits(3, A16, A16, A16, None, A16, 128, 136, 8, 0, 0, stream=0) == B.GPTQ_ERR_SHAPE   # K % 32
    assert B.gptq_dequant_f32_bits(3, A16, A16, A16, None, A16, 128, 128, 128, 1, 0, stream=0) == B.GPTQ_ERR_NULL
    # the bfloat16 matmul validates like gptq_gemm
    assert B.gptq_gemm_bf16(A16, A16, A16, A16, None, None, 1, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_gemm_bf16(A16, A16, A16, A16, None, A16, 1, 128, 128, 128, 1, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_gemm_bf16(A16 + 2, A16, A16, A16, None, A16, 1, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_ALIGN
    assert B.gptq_gemm_bf16(A16, A16, A16, A16, None, A16, 1, 128, 128, 16, 0, stream=0) == B.GPTQ_ERR_UNSUPPORTED
    assert B.gptq_gemm_bf16(A16, A16, A16, A16, None, A16, 0, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_SHAPE
    assert B.gptq_gemm_silu_mul_scatter(A16, A16, A16, A16, None, A16 + 4, A16, 1, 256, 128, 128, 0, stream=0) == B.GPTQ_ERR_ALIGN
    assert B.gptq_invert_perm(None, A16, 8, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_invert_perm(A16, A16, 0, stream=0) == B.GPTQ_ERR_SHAPE
    assert B.gptq_gemm(A16, A16, A16, A16, None, A16, 1, 128, 128, 128, 5, stream=0) == B.GPTQ_ERR_LAYOUT
    assert B.gptq_gemm_bias_residual(A16, A16, A16, A16, None, A16, A16, None, 1, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_gemm_bias_residual(A16, A16, A16, A16, None, A16 + 2, None, A16, 1, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_ALIGN
    assert B.gptq_gemm_bias_residual(A16, A16, A16, A16, None, None, A16 + 8, A16, 1, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_ALIGN
    assert B.gptq_gemm_silu_mul(A16, A16, A16, A16, None, A16, 1, 192, 128, 128, 0, stream=0) == B.GPTQ_ERR_UNSUPPORTED
    assert B.gptq_repack_bytes(1, 256, 512, 32, 0) == (512 // 32) * 256 // 2 + 16    # zero points + format trailer
    assert B.gptq_plan_noalloc(4, 128, 512, 64, 0, 148)[0] == B.GPTQ_ERR_UNSUPPORTED
    # groups coarser than 128 rows (multiples of 128, up to one group per column) are tiled as repeated 128-row groups
    assert B.gptq_repack_bytes(1, 256, 512, 256, 0) == (512 // 128) * 256 // 2 + 16
    assert B.gptq_repack_bytes(2, 256, 512, 512, 0) == (512 // 128) * 256 * 2
    assert B.gptq_repack_bytes(0, 256, 512, 512, 0) == 512 * 256 // 2
    for gs in (256, 1024, 4096):
        st, pl = B.gptq_plan(8, 4096, 4096, gs, 0, 148)
        st128, pl128 = B.gptq_plan(8, 4096, 4096, 128, 0, 148)
        assert st == B.GPTQ_OK and B.plan_kernel_name(pl) == B.plan_kernel_name(pl128) and pl.ctas == pl128.ctas
    assert B.gptq_plan(8, 256, 768, 192, 0, 148)[0] == B.GPTQ_ERR_UNSUPPORTED      # divides K, but no multiple of 128
    assert B.gptq_plan(8, 256, 768, 384, 0, 148)[0] == B.GPTQ_OK
    assert B.gptq_plan_noalloc(4, 128, 512, 512, 0, 148)[0] == B.GPTQ_OK
    assert B.gptq_workspace_bytes(4, 256, 512, 512, 1) == B.gptq_workspace_bytes(4, 256, 512, 128, 1) > 0
    assert B.gptq_repack(A16, A16, A16, A16, A16 + 16, A16 + 32, A16 + 48, None, 128, 128, 128, 1, stream=0) == B.GPTQ_ERR_NULL
    assert B.gptq_gemm_host(None, A16, A16, A16, None, A16, A16, A16, 1, 128, 128, 128, 0, stream=0) == B.GPTQ_ERR_NULL


def test_host_batch_validates_every_problem_before_running():
    good = (A16, A16, A16, A16, None, A16, A16, A16, 1, 128, 128, 128, 0)
    bad_shape = good[:9] + (130,) + good[10:]
    arr = B.make_host_problems([good, good, bad_shape])
    st, bad = B._lib.gptq_gemm_host_batch(arr, 3, 0, None), None
    assert st == B.GPTQ_ERR_SHAPE
    import ctypes
    idx = ctypes.c_int(-1)
    assert B._lib.gptq_gemm_host_batch(arr, 3, 0, ctypes.byref(idx)) == B.GPTQ_ERR_SHAPE and idx.value == 2
    missing = (None,) + good[1:]
    arr = B.make_host_problems([missing])
    assert B._lib.gptq_gemm_host_batch(arr, 1, 0, ctypes.byref(idx)) == B.GPTQ_ERR_NULL and idx.value == 0
    assert B._lib.gptq_gemm_host_batch(None, 1, 0, None) == B.GPTQ_ERR_NULL
    assert B._lib.gptq_gemm_host_batch(arr, 0, 0, None) == B.GPTQ_OK      # an empty step is fine


def test_repack_bytes_equal_canonical_sizes_plus_trailer():
    for (K, N) in list(wl.SHAPES_7B.values()) + list(wl.SHAPES_13B.values()):
        G = K // 128
        assert B.gptq_repack_bytes(0, N, K, 128, 0) == K * N // 2
        assert B.gptq_repack_bytes(1, N, K, 128, 0) == G * N // 2 + 16     # + the 16-byte format trailer
        assert B.gptq_repack_bytes(2, N, K, 128, 0) == G * N * 2
        assert B.gptq_repack_bytes(3, N, K, 128, 0) == 0
        assert B.gptq_repack_bytes(3, N, K, 128, 1) == 4 * K
    assert B.gptq_repack_bytes(7, 128, 128, 128, 0) == 0
    assert B.gptq_repack_bytes(0, 129, 128, 128, 0) == 0


SHAPES = list(wl.SHAPES_7B.values()) + list(wl.SHAPES_13B.values()) + [(128, 128), (256, 384), (1024, 128)]


@pytest.mark.parametrize("K,N", SHAPES)
@pytest.mark.parametrize("M", [1, 8, 9, 16, 33, 64, 200, 1000])
@pytest.mark.parametrize("sms", [148, 132, 7])
def test_cluster_plan_is_consistent(K, N, M, sms):
    st, pl = B.gptq_plan(M, N, K, 128, 0, sms)
    assert st == B.GPTQ_OK
    G, panels = K // 128, N // 128
    assert pl.items == G * panels and pl.workspace_bytes == 0
    if pl.kernel == 2:                        # tcgen05 kernel: one launch, 16- to 128-token tiles
        tok = 16 if M <= 16 else 32 if M <= 32 else 64 if M <= 64 else 128 if M <= 128 else 256
        assert pl.m_tile == tok and pl.m_chunks == 1
        assert pl.cluster_size in (1, 2, 4, 8) and pl.cluster_size <= G
        tiles = panels * -(-M // tok)
        cps_max = 1 if tok > 128 else 3 if tok <= 32 else 2
        if pl.tail_ctas:                      # the partly filled last wave goes to a K-split second launch
            tail_tiles = tiles % (sms * cps_max)
            assert pl.cluster_size == 1 and tiles > sms * cps_max and tail_tiles > 0
            assert pl.tail_cluster_size in (2, 4, 8) and pl.tail_cluster_size <= G
            assert pl.tail_ctas == tail_tiles * pl.tail_cluster_size <= sms * cps_max
            assert pl.ctas == tiles - tail_tiles
        else:
            assert pl.tail_cluster_size == 1
            assert pl.ctas == tiles * pl.cluster_size
        assert pl.split_panels == (panels if pl.cluster_size > 1 else 0)
        per_sm = min(-(-tiles * pl.cluster_size // sms), cps_max)
        assert per_sm * (pl.smem_bytes + 1024) <= 227 * 1024
        # ring slots hold one K group (one K64 block for 128-token tiles): never more than the CTA has, unless the
        # ring must also hold the fp32 partial tile of the split-K exchange
        assert 1 <= pl.stages <= 8
        if pl.cluster_size == 1:
            assert pl.stages <= (2 * G if tok == 128 else G)
        assert (per_sm + 1) * (pl.smem_bytes + 1024) > 227 * 1024
        if pl.cluster_size > 1:               # the ring doubles as the fp32 partial tile
            assert pl.smem_bytes - 2048 >= tok * 128 * 4
        return
    assert M <= 16
    assert pl.kernel == 1
    wide = pl.m_tile == 8                     # 8 token rows, group 128: 56 registers, four CTAs fit an SM, S = 3 and 6 allowed
    assert pl.cluster_size in ((1, 2, 3, 4, 6, 8) if wide else (1, 2, 4, 8)) and pl.cluster_size <= G
    assert pl.ctas == panels * pl.cluster_size
    assert pl.split_panels == (panels if pl.cluster_size > 1 else 0)
    assert pl.m_tile in (8, 16, 32, 64) and pl.m_tile >= min(M, 64)
    assert pl.m_chunks == (M + 63) // 64
    assert 1 <= pl.stages <= 8
    per_sm = min(-(-pl.ctas // sms), 4 if wide else 3 if pl.m_tile <= 16 else 1)
    assert per_sm * (pl.smem_bytes + 1024) <= 227 * 1024          # that many CTAs fit on an SM ...
    assert (per_sm + 1) * (pl.smem_bytes + 1024) > 227 * 1024     # ... and no more (even spreading)
    # the ring doubles as the fp32 partial tile of the cluster reduction
    assert pl.smem_bytes - 2048 >= pl.m_tile * 128 * 4
    assert pl.workspace_bytes == 0          # the partial sums stay on chip


@pytest.mark.parametrize("K,N", SHAPES)
@pytest.mark.parametrize("M", [1, 8, 9, 16, 33, 64, 200])
@pytest.mark.parametrize("sms", [148, 132, 7])
def test_streamk_plan_is_consistent(K, N, M, sms):
    st, pl = B.gptq_plan_noalloc(M, N, K, 128, 0, sms)
    assert st == B.GPTQ_OK
    G, panels = K // 128, N // 128
    assert pl.items == G * panels
    assert 1 <= pl.ctas <= min(pl.items, 2 * sms)
    assert pl.m_tile in (8, 16, 32, 64) and pl.m_tile >= min(M, 64)
    assert pl.m_chunks == (M + 63) // 64
    assert 2 <= pl.stages <= 8
    assert pl.smem_bytes <= 227 * 1024
    # every item is covered exactly once, ranges are contiguous and balanced within one item
    end_prev, sizes = 0, []
    for c in range(pl.ctas):
        st, a, b = B.gptq_plan_cta_range(pl.items, pl.ctas, c)
        assert st == B.GPTQ_OK and a == end_prev and b > a
        sizes.append(b - a)
        end_prev = b
    assert end_prev == pl.items and max(sizes) - min(sizes) <= 1
    # contributors per panel: the reducing CTA's view must match who actually writes partials
    writers = {}
    for c in range(pl.ctas):
        _, a, b = B.gptq_plan_cta_range(pl.items, pl.ctas, c)
        first_panel = a // G
        for p in range(a // G, (b - 1) // G + 1):
            lo, hi = max(a, p * G), min(b, (p + 1) * G)
            if not (lo == p * G and hi == (p + 1) * G):     # partial segment -> slot 0 or 1
                writers.setdefault(p, []).append((c, 0 if p == first_panel else 1))
    split = 0
    for p in range(panels):
        st, cf, cl = B.gptq_plan_panel_owners(pl.items, pl.ctas, G, p)
        assert st == B.GPTQ_OK
        if cf == cl:
            assert p not in writers
            continue
        split += 1
        expect = []
        for cc in range(cf, cl + 1):
            _, a, _b = B.gptq_plan_cta_range(pl.items, pl.ctas, cc)
            expect.append((cc, 0 if a // G == p else 1))
        assert writers[p] == expect
    assert split == pl.split_panels
    # slots are never reused by two panels of one CTA
    used = [w for ws in writers.values() for w in ws]
    assert len(used) == len(set(used))
    if split:
        rows = min(M, 64)
        assert pl.workspace_bytes >= 16384 + pl.ctas * 2 * rows * 128 * 4
    else:
        assert pl.workspace_bytes == 0


def test_plan_act_order_adds_gathered_x():
    for plan in (B.gptq_plan, B.gptq_plan_noalloc):
        st, a = plan(8, 5120, 13824, 128, 0, 148)
        st2, b = plan(8, 5120, 13824, 128, 1, 148)
        assert st == st2 == B.GPTQ_OK
        assert b.workspace_bytes - a.workspace_bytes >= 8 * 13824 * 2
    assert B.gptq_plan(8, 5120, 13824, 128, 0, 148)[1].workspace_bytes == 0


def test_plan_rejects_bad_arguments():
    assert B.gptq_plan(1, 4096, 4096, 128, 0, 0)[0] == B.GPTQ_ERR_SHAPE
    assert B.gptq_plan(1, 4096, 4096, 16, 0, 148)[0] == B.GPTQ_ERR_UNSUPPORTED
    assert B.gptq_plan(1, 4096, 4096, 32, 0, 148)[0] == B.GPTQ_OK
    assert B.gptq_plan_cta_range(10, 11, 0)[0] == B.GPTQ_ERR_SHAPE
    assert B.gptq_plan_panel_owners(10, 5, 3, 0)[0] == B.GPTQ_ERR_SHAPE


def test_plan_names_the_kernel():
    """The planner names the kernel instantiation a profiler would print; bench.py attributes time by it."""
    for M, want in ((1, "splitk_kernel<1,1>"), (8, "splitk_kernel<1,1>"), (16, "splitk_kernel<2,1>"),
                    (17, "umma_kernel<32,3,1,2,1>"), (64, "umma_kernel<64,4,1,2,1>"), (128, "umma_kernel<128,4,1,2,1>"),
                    (2048, "umma_kernel<256,4,1,2,1>")):
        st, pl = B.gptq_plan(M, 4096, 4096, 128, 0, 148)
        assert st == B.GPTQ_OK and B.plan_kernel_name(pl) == want
    assert B.plan_kernel_name(B.gptq_plan(4, 4096, 4096, 32, 0, 148)[1]) == "splitk_kernel<1,4>"     # four groups per item
    assert B.plan_kernel_name(B.gptq_plan(512, 4096, 4096, 64, 0, 148)[1]) == "umma_kernel<256,4,1,2,2>"
    for M, want in ((1, "streamk_kernel<1>"), (16, "streamk_kernel<2>"), (32, "streamk_kernel<4>"), (100, "streamk_kernel<8>")):
        st, pl = B.gptq_plan_noalloc(M, 1024, 1024, 128, 0, 148)
        assert st == B.GPTQ_OK and B.plan_kernel_name(pl) == want
