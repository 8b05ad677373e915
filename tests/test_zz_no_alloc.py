"""gptq_gemm_noalloc: the matmul for callers that cannot allocate device memory.

Some users of this library run inside a serving process that carved up the GPU's memory when it
started and must not call cudaMalloc afterwards (it is forbidden by the host program, or it would
stall the device in the middle of a latency-bound decode loop), so they cannot give gptq_gemm a
workspace.  gptq_gemm_noalloc keeps its split-K scratch in an array inside the library instead.
These tests call it through the C ABI twice in a row (the array keeps the first call's contents)
and require agreement with gptq_gemm (a different kernel, so a different summation order) and
with the CPU oracle, both within the tolerance the parity tests state.  The file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_19438_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2511_19438_b200 import build as libbuild
    libbuild.build()
    from paper_2511_19438_b200 import binding as B
    from paper_2511_19438_b200 import harness as H


def within_stated_tolerance(y, y64, K):
    err = np.abs(y.astype(np.float64) - y64)
    return np.all(err <= 1e-2 * math.sqrt(K / 4096) + 1e-2 * np.abs(y64))


def noalloc_scratch_need(M, N, K, act):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    st, pl = B.gptq_plan_noalloc(M, N, K, 128, act, sms)
    assert st == B.GPTQ_OK
    return pl.workspace_bytes


# M = 1 .. 8 run streamk_kernel<1>, 9 .. 16 <2>, 17 .. 32 <4>, 33 .. 64 <8>; above 64 rows the call loops over chunks
# of 64 that reuse the tickets and partial tiles
@pytest.mark.parametrize("K,N,M,act", [(4096, 4096, 1, False), (4096, 4096, 8, False), (2560, 1280, 5, True),
                                        (4096, 4096, 16, False), (1024, 512, 12, True), (1024, 512, 24, False),
                                        (1024, 512, 40, True), (2048, 768, 64, False), (1024, 512, 100, False),
                                        (1024, 512, 130, True)])
def test_noalloc_matches_gemm_on_two_calls_in_a_row(K, N, M, act):
    L = wl.make_linear(K, N, seed=wl.seed_for("noalloc", K, N, act), act_order=act)
    D = H.upload_and_repack(L)
    assert 0 < noalloc_scratch_need(M, N, K, act) <= B.gptq_noalloc_scratch_bytes()   # the scratch is used
    ws = H.WorkspaceHolder()
    ws.ensure_for(M, D)
    outs = []
    for call in range(2):                                   # second call meets a used scratch array
        x_np = wl.make_x(M, K, wl.seed_for("noalloc-x", K, M, call))
        x = H.to_device(x_np)
        want = H.gemm(x, D)                                 # existing entry point, caller's workspace
        y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.check(B.gptq_gemm_noalloc(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, y, M, N, K, 128, act),
                "gptq_gemm_noalloc")
        assert B.gptq_check_status() == B.GPTQ_OK
        if call == 1:                                       # (the first call on a device may load the kernel image)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
        assert within_stated_tolerance(y.cpu().numpy(), want.cpu().numpy().astype(np.float64), K), \
            f"call {call}: differs from gptq_gemm"
        y64 = oracle.gemm_f64(x_np, L.qweight, L.qzeros, L.scales, L.g_idx, 128)
        assert within_stated_tolerance(y.cpu().numpy(), y64, K)
        outs.append(y)
    assert not torch.equal(outs[0], outs[1])                # the two calls really had different inputs


def test_noalloc_needs_no_registered_workspace():
    K, N, M = 2048, 512, 4                                  # act-order: gptq_gemm needs a workspace here
    L = wl.make_linear(K, N, seed=wl.seed_for("noalloc-unreg"), act_order=True)
    D = H.upload_and_repack(L)
    x_np = wl.make_x(M, K, 7)
    x = H.to_device(x_np)
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    B.check(B.gptq_set_workspace(None, 0), "unregister")
    assert B.gptq_gemm(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, y, M, N, K, 128, 1) == B.GPTQ_ERR_WORKSPACE
    B.check(B.gptq_gemm_noalloc(x, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, y, M, N, K, 128, 1), "noalloc")
    assert B.gptq_check_status() == B.GPTQ_OK
    y64 = oracle.gemm_f64(x_np, L.qweight, L.qzeros, L.scales, L.g_idx, 128)
    assert within_stated_tolerance(y.cpu().numpy(), y64, K)


def test_noalloc_refuses_problems_beyond_its_scratch():
    K, N, M = 4096, 22016, 64                               # needs ~19 MB of partial tiles
    assert noalloc_scratch_need(M, N, K, 0) > B.gptq_noalloc_scratch_bytes()
    L = wl.make_linear(K, N, seed=wl.seed_for("noalloc-big"))
    D = H.upload_and_repack(L)
    x = H.to_device(wl.make_x(M, K, 9))
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    st = B.gptq_gemm_noalloc(x, D.qweight_t, D.qzeros_t, D.scales_t, None, y, M, N, K, 128, 0)
    assert st == B.GPTQ_ERR_WORKSPACE
    assert "workspace" in B.gptq_status_string(st)
    torch.cuda.synchronize()
    assert torch.count_nonzero(y) == 0                      # nothing was launched
