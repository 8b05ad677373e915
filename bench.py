#!/usr/bin/env python
"""Benchmark of the GPTQ int4 matmul path on B200.

A STEP is one pass of the whole path (stage x, stream packed weights, unpack, dequantise,
multiply-accumulate, reduce, store fp16 y) over every matmul of the workload:

  decode7b  (default)  the four Llama-2-7B decoder linears (qkv, o, gate_up, down), group 128,
                       at M = 1, 4, 8, 16, over `--layers` distinct seeded copies of the layer so
                       that each launch streams weights last touched ~0.8 GB ago (HBM-cold)
  step32               32 layers x 4 linears at M = 1, 8, 32, 64 (a full decode step's linears)
  actorder13b          Llama-2-13B shapes with act-order g_idx at M = 1, 8
  prefill7b            the 7B shapes at M = 512 .. 4096 (metric becomes TFLOP/s)

Every matmul is a gptq_gemm call through the C ABI.  The device-timed number replays CUDA graphs
of those calls (one graph per M) with CUDA events around them; the end-to-end number calls
gptq_gemm_host_batch (one call per step) with pinned host activations and outputs, copies inside
the timed region.  The default run (decode7b) also measures a short pass of prefill7b and reports it
as the `prefill` object of the same line, so both halves of the metric are in one record.
One JSON line is printed by rank 0.  With --impl reference the CPU oracle is timed instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_19438_b200 import workloads as wl  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
NOMINAL_FP16_TFLOPS = 2250.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_TFLOPS = 1590.0

# DRAM traffic of the dominant kernels from ncu captures (profiles/), as measured bytes over
# algorithmic bytes of the captured launches, with the digest of the kernel sources they were taken
# on (`--print-digest`); `traffic` is that ratio times the timed launches' algorithmic bytes, and
# null once the sources have changed since the capture.
NCU_TRAFFIC = {
    "splitk_kernel<1,1>": {"digest": "cafbf47bd6e61035", "ratio": 0.998, "Ms": (1, 4, 8),
                         "source": "ncu capture profiles/splitk_kernel_decode7b.md (108 launches: M = 1, 4, 8 on the four "
                                   "7B shapes): dram bytes / algorithmic bytes x algorithmic bytes per timed launch"},
    "umma_kernel<256,4,1,2,1>": {"digest": "36c16532a4b1d9c3", "ratio": 0.934, "Ms": (512, 1024, 2048, 4096),
                               "source": "ncu capture profiles/umma_kernel_prefill7b.md (161 launches: M = 512..4096 on "
                                         "the four 7B shapes, main + tail launches; y partly still in L2): ratio x "
                                         "algorithmic bytes per timed launch"},
}

WORKLOADS = {
    "decode7b": dict(shapes=wl.SHAPES_7B, Ms=wl.DECODE_M, act_order=False, layers=8, kind="decode",
                     describes="configs[1]: Llama-2-7B decoder linears, group 128, M in {1,4,8,16}"),
    "step32": dict(shapes=wl.SHAPES_7B, Ms=wl.STEP_M, act_order=False, layers=32, kind="decode",
                   describes="configs[4]: 32-layer Llama-2-7B decode step linears, M in {1,8,32,64}"),
    "actorder13b": dict(shapes=wl.SHAPES_13B, Ms=wl.ACT_ORDER_M, act_order=True, layers=4, kind="decode",
                        describes="configs[2]: Llama-2-13B shapes with act-order g_idx, M in {1,8}"),
    "prefill7b": dict(shapes=wl.SHAPES_7B, Ms=wl.PREFILL_M, act_order=False, layers=2, kind="prefill",
                      describes="configs[3]: Llama-2-7B shapes, M in {512,1024,2048,4096}"),
}


# the header files each captured kernel is built from (its own file and what that includes)
KERNEL_SOURCES = {
    "splitk_kernel<1,1>": ("gptq_common.cuh", "gptq_tma.cuh", "gptq_streamk.cuh", "gptq_splitk.cuh"),
    "umma_kernel<256,4,1,2,1>": ("gptq_common.cuh", "gptq_tma.cuh", "gptq_streamk.cuh", "gptq_splitk.cuh", "gptq_umma.cuh"),
}


def kernel_source_digest(kernel: str | None = None) -> str:
    """sha256 over the header files a kernel is built from (all kernel headers when the kernel is not listed)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2511_19438_b200", "csrc")
    names = KERNEL_SOURCES.get(kernel) or sorted(n for n in os.listdir(csrc) if n.endswith(".cuh"))
    for name in names:                        # the kernels; the .cu holds dispatch only
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), tflops_burst=float(p["bf16_tflops"]),
                    tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, tflops_burst=FALLBACK_TFLOPS, tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) in a thread."""

    REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
        0x80: "hw_power_brake_slowdown",
    }

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples = []
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self.max_mhz = None
        self.error = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                tok = ids[index] if index < len(ids) else ids[0]
                self.h = (pynvml.nvmlDeviceGetHandleByUUID(tok) if tok.startswith("GPU-")
                          else pynvml.nvmlDeviceGetHandleByIndex(int(tok)))
            else:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # no NVML: the clocks object says so
            self.nv = None
            self.error = repr(e)

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception as e:
                self.error = repr(e)
                return
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self, t0: float, t1: float, note: str = ""):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": len(inside)}
        if inside:
            out["sm_mhz"] = statistics.median(s[1] for s in inside)
            mask = 0
            for s in inside:
                mask |= s[2]
            out["reasons"] = sorted(name for bit, name in self.REASONS.items() if mask & bit)
        if note:
            out["note"] = note
        if self.error:
            out["error"] = self.error
        return out


# ------------------------------------------------------------------------------------ workload
def bf16_scales(L, layer, name):
    """The bfloat16 scales of the bfloat16 variant of a bench layer (bit patterns [G, N])."""
    return wl.make_scales_bf16(L.K // L.group_size, L.N, wl.seed_for("bench-bf16-scales", layer, name))


def make_layer(spec, K, N, seed):
    """One seeded layer of the workload: 4-bit, or 8-bit with --wbits 8."""
    if spec.get("w8", False):
        return wl.make_linear_w8(K, N, seed=seed, act_order=spec["act_order"])
    return wl.make_linear(K, N, seed=seed, act_order=spec["act_order"])


def build_problems(spec, layers, H, torch, device):
    """Uploads `layers` distinct seeded copies of every shape (repacked through the C ABI) and the
    activations; returns {M: [(D, x, y, name), ...]} in launch order (layer-major)."""
    Ms = spec["Ms"]
    per_m = {M: [] for M in Ms}
    host = {}
    for layer in range(layers):
        for name, (K, N) in spec["shapes"].items():
            L = make_layer(spec, K, N, wl.seed_for("bench", layer, name))
            bf16 = spec.get("bf16", False)
            if spec.get("w8", False):
                D = H.upload_and_repack_w8(L)
            else:
                D = H.upload_and_repack(L, scales_bf16_bits=bf16_scales(L, layer, name) if bf16 else None)
            if layer == 0:
                host[name] = L
            for M in Ms:
                if layer == 0 and bf16:
                    x = H.bf16_from_bits(wl.make_x_bf16(M, K, wl.seed_for("bench-x", name, M)), device)
                elif layer == 0:
                    x = H.to_device(wl.make_x(M, K, wl.seed_for("bench-x", name, M)), device)
                else:   # activations are tiny next to the weights: reuse layer 0's
                    x = per_m[M][list(spec["shapes"]).index(name)][1]
                if spec["kind"] == "prefill" and layer > 0:
                    y = per_m[M][list(spec["shapes"]).index(name)][2]
                else:
                    y = torch.empty((M, N), dtype=torch.bfloat16 if bf16 else torch.float16, device=device)
                per_m[M].append((D, x, y, name))
    return per_m, host


def step_bytes_flops(spec, layers):
    b = {M: 0 for M in spec["Ms"]}
    f = {M: 0 for M in spec["Ms"]}
    for M in spec["Ms"]:
        for (K, N) in spec["shapes"].values():
            b[M] += layers * wl.algorithmic_bytes(M, K, N, act_order=spec["act_order"], wbits=8 if spec.get("w8", False) else 4)
            f[M] += layers * wl.matmul_flops(M, K, N)
    return b, f


def launches_per_gemm(spec, M, name, sm_count):
    """Kernels one gptq_gemm call launches: the matmul (two launches when the tcgen05 kernel's last wave is split
    along K), plus the x gather with act-order."""
    from paper_2511_19438_b200 import binding as B
    K, N = spec["shapes"][name]
    if spec.get("w8", False):       # the 4-bit kernels on the stacked planes (2 K rows), always behind the x gather
        st, pl = B.gptq_plan(M, N, 2 * K, wl.GROUP_SIZE, 0, sm_count)
        assert st == B.GPTQ_OK
        return 2 + (1 if pl.tail_ctas > 0 else 0)
    st, pl = B.gptq_plan(M, N, K, wl.GROUP_SIZE, 1 if spec["act_order"] else 0, sm_count)
    assert st == B.GPTQ_OK
    return 1 + (1 if pl.tail_ctas > 0 else 0) + (1 if spec["act_order"] else 0)


def kernel_of(spec, M, sm_count):
    """The kernel instantiation gptq_gemm launches for M token rows, as the library's own planner names it
    (the widest shape of the workload decides when shapes differ)."""
    from paper_2511_19438_b200 import binding as B
    names = {}
    for (K, N) in spec["shapes"].values():
        if spec.get("w8", False):
            K = 2 * K
        st, pl = B.gptq_plan(M, N, K, wl.GROUP_SIZE, 1 if spec["act_order"] else 0, sm_count)
        assert st == B.GPTQ_OK
        names[B.plan_kernel_name(pl)] = names.get(B.plan_kernel_name(pl), 0) + K * N
    return max(names, key=names.get)


# ------------------------------------------------------------------------------------ reference arm
def oracle_sample(spec, budget_s):
    """The bounded sample of the workload the CPU oracle is timed on: layer 0 of the workload, the
    largest of a fixed ladder of (shapes, M) subsets whose estimated time fits `budget_s` (the
    estimate comes from a probe of the smallest shape at the smallest M)."""
    import oracle
    shapes = spec["shapes"]
    small = min(shapes, key=lambda n: shapes[n][0] * shapes[n][1])
    Ms = [M for M in spec["Ms"] if M <= 16] or [16]
    ladder = [([small], Ms[:1]), (list(shapes), Ms[:1]), (list(shapes), Ms[:2]), (list(shapes), Ms)]
    layer = {n: make_layer(spec, K, N, wl.seed_for("bench", 0, n)) for n, (K, N) in shapes.items()}
    Lp = layer[small]
    bf16 = spec.get("bf16", False)
    make_x = wl.make_x_bf16 if bf16 else wl.make_x
    xp = make_x(Ms[0], Lp.K, wl.seed_for("bench-x", small, Ms[0]))
    run_oracle_once([(Lp, xp, Ms[0], small)], spec)   # first touch
    t0 = time.perf_counter()
    run_oracle_once([(Lp, xp, Ms[0], small)], spec)
    rate = Ms[0] * Lp.K * Lp.N / (time.perf_counter() - t0)
    pick = ladder[0]
    for names, ms in ladder:
        macs = sum(M * shapes[n][0] * shapes[n][1] for n in names for M in ms)
        if macs / rate <= budget_s:
            pick = (names, ms)
    names, ms = pick
    items = [(layer[n], make_x(M, layer[n].K, wl.seed_for("bench-x", n, M)), M, n) for n in names for M in ms]
    text = f"layer 0 of the workload, shapes {names}, M in {list(ms)}, full outputs"
    return items, text


def run_oracle_once(items, spec):
    import oracle
    scales = {n: bf16_scales(L, 0, n) for (L, x, M, n) in items} if spec.get("bf16", False) else None
    t0 = time.perf_counter()
    for (L, x, M, n) in items:
        if scales is not None:
            oracle.gemm_f64_bf16(x, L.qweight, L.qzeros, scales[n], L.g_idx, L.group_size)
        elif spec.get("w8", False):
            oracle.gemm_f64_w8(x, L.qweight, L.qzeros, L.scales, L.g_idx, L.group_size)
        else:
            oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, L.group_size)
    dt = time.perf_counter() - t0
    nbytes = sum(wl.algorithmic_bytes(M, L.K, L.N, act_order=L.act_order, wbits=8 if spec.get("w8", False) else 4)
                 for (L, x, M, n) in items)
    flops = sum(wl.matmul_flops(M, L.K, L.N) for (L, x, M, n) in items)
    return dt, nbytes, flops


def metric_of(spec):
    if spec["kind"] == "prefill":
        return "GPTQ int4 matmul: prefill TFLOPS (% fp16 peak)", "TFLOP/s"
    return "GPTQ int4 matmul: decode HBM GB/s (% of 8 TB/s)", "GB/s"


def to_metric(spec, nbytes, flops, seconds):
    return (flops / seconds / 1e12) if spec["kind"] == "prefill" else (nbytes / seconds / 1e9)


def cpu_baseline(spec):
    import oracle
    oracle.build()
    items, text = oracle_sample(spec, budget_s=12.0)
    dt, nbytes, flops = run_oracle_once(items, spec)
    return {"value": to_metric(spec, nbytes, flops, dt), "unit": metric_of(spec)[1], "cores": oracle.num_threads(),
            "kind": "oracle", "sample": text, "seconds": round(dt, 3)}


def run_reference(args, spec):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    items, text = oracle_sample(spec, budget_s=min(12.0, args.ref_budget / max(args.steps + min(args.warmup, 1), 1)))
    for _ in range(min(args.warmup, 1)):
        run_oracle_once(items, spec)
    total = 0.0
    for _ in range(args.steps):
        dt, nbytes, flops = run_oracle_once(items, spec)
        total += dt
    value = to_metric(spec, nbytes * args.steps, flops * args.steps, total)
    metric, unit = metric_of(spec)
    line = {
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "describes": spec["describes"], "sample": text},
        "cpu_baseline": {"value": value, "unit": unit, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": text},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ replicas
def max_over_ranks(values, world, device="cpu"):
    """Element-wise maximum over all ranks of a list of per-rank times (a collective when world > 1)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(spec, world, step_bytes, step_flops, steps, slowest_ms):
    """Replicas only: every rank runs the same workload on its own GPU, so the job processed
    world x the units of one rank in the time of the slowest rank."""
    return world * to_metric(spec, step_bytes * steps, step_flops * steps, slowest_ms / 1e3)


# ------------------------------------------------------------------------------------ product arm
def measure_workload(name, spec, layers, steps, warmup, e2e_steps, env):
    """Builds one workload on the device, times `steps` graph-replayed steps and `e2e_steps` host-resident steps
    (max over ranks), and returns the raw numbers report_line() turns into the JSON fields."""
    torch, dist, B, H = env["torch"], env["dist"], env["B"], env["H"]
    device, world, local_rank = env["device"], env["world"], env["local_rank"]
    per_m, _host = build_problems(spec, layers, H, torch, device)
    ws = H.WorkspaceHolder(device)
    need = 0
    for M, probs in per_m.items():
        for (D, x, y, _n) in probs:
            if spec.get("w8", False):
                need = max(need, B.gptq_workspace_bytes(M, D.N, 2 * D.K, D.group_size, 1))
            need = max(need, B.gptq_workspace_bytes(M, D.N, D.K, D.group_size, D.act_order))
    ws.ensure(need)
    bytes_m, flops_m = step_bytes_flops(spec, layers)

    bf16 = spec.get("bf16", False)
    w8 = spec.get("w8", False)
    gemm = H.gemm_bf16 if bf16 else H.gemm_w8 if w8 else H.gemm

    def run_m(M):
        for (D, x, y, _n) in per_m[M]:
            gemm(x, D, y)

    # eager warm-up (configures the kernels), then one CUDA graph per M
    stream = torch.cuda.Stream(device)
    graphs = {}
    with torch.cuda.stream(stream):
        for M in spec["Ms"]:
            run_m(M)
        stream.synchronize()
        B.check(B.gptq_check_status(), "warm-up")
        for M in spec["Ms"]:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run_m(M)
            graphs[M] = g
    torch.cuda.synchronize()

    Ms = list(spec["Ms"])
    sampler = ClockSampler(local_rank)
    sampler.start()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            for M in Ms:
                graphs[M].replay()
        barrier()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(Ms) + 1)] for _ in range(steps)]
        t_host0 = time.perf_counter()
        for k in range(steps):
            ev[k][0].record(stream)
            for i, M in enumerate(Ms):
                graphs[M].replay()
                ev[k][i + 1].record(stream)
        barrier()
        t_host1 = time.perf_counter()
    total_ms = ev[0][0].elapsed_time(ev[-1][-1])
    seg_ms = {M: sum(ev[k][i].elapsed_time(ev[k][i + 1]) for k in range(steps)) for i, M in enumerate(Ms)}
    clocks = sampler.summary(t_host0, t_host1)
    if clocks["samples"] < 3:
        # the timed region was too short to catch a sample: keep replaying the same step, untimed
        t2 = time.perf_counter()
        with torch.cuda.stream(stream):
            while time.perf_counter() - t2 < 1.0:
                for M in Ms:
                    graphs[M].replay()
                stream.synchronize()
        clocks = sampler.summary(t2, time.perf_counter(),
                                 note="timed region shorter than the sampling period; sampled over 1 s of the same steps right after it")
    B.check(B.gptq_check_status(), "timed region")

    # ---- end to end: host activations in, host outputs back, every call through gptq_gemm_host
    host_io = {}
    h2d = d2h = 0
    for M in Ms:
        for (D, x, y, name) in per_m[M][:len(spec["shapes"])]:
            xh = x.cpu().pin_memory()
            yh = torch.empty((M, D.N), dtype=torch.bfloat16 if bf16 else torch.float16).pin_memory()
            host_io[(M, name)] = (xh, yh)
    for M in Ms:
        for (D, x, y, name) in per_m[M]:
            h2d += M * D.K * 2
            d2h += M * D.N * 2

    # device staging: one pair of buffers per matmul while that stays small (the pipeline then runs long chunks), else
    # the buffers of the device-timed run, which are shared between layers
    own_staging = (h2d + d2h) <= (4 << 30)
    step_items, staging = [], []
    for M in Ms:
        for (D, x, y, name) in per_m[M]:
            xh, yh = host_io[(M, name)]
            xs, ys = (torch.empty_like(x), torch.empty_like(y)) if own_staging else (x, y)
            staging.append((xs, ys))
            step_items.append((xh, D.qweight_t, D.qzeros_t, D.scales_t, D.perm, yh, xs, ys, M, D.N, D.K, D.group_size,
                               D.act_order))
    step_problems = B.make_host_problems(step_items)

    def e2e_step():
        st, bad = (B.gptq_gemm_host_batch_bf16 if bf16 else B.gptq_gemm_host_batch_w8 if w8 else B.gptq_gemm_host_batch)(step_problems)
        B.check(st, f"gptq_gemm_host_batch (problem {bad})")
        stream.synchronize()   # the step's results are on the host

    with torch.cuda.stream(stream):
        for _ in range(3):
            e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(stream)
        barrier()
    e2e_ms = e0.elapsed_time(e1)
    # the same step captured once into a CUDA graph (the call is stream-ordered: its copy streams fork from and join
    # the caller's stream) and replayed: every replay still copies x up, multiplies and copies y back
    batch_call = B.gptq_gemm_host_batch_bf16 if bf16 else B.gptq_gemm_host_batch_w8 if w8 else B.gptq_gemm_host_batch
    with torch.cuda.stream(stream):
        e2e_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(e2e_graph, stream=stream):
            st, bad = batch_call(step_problems)
            B.check(st, f"gptq_gemm_host_batch under capture (problem {bad})")
        for _ in range(3):
            e2e_graph.replay()
            stream.synchronize()
        barrier()
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_graph.replay()
            stream.synchronize()
        e1.record(stream)
        barrier()
    e2e_graph_ms = e0.elapsed_time(e1)
    B.check(B.gptq_check_status(), "end-to-end steps")
    del e2e_graph
    sampler.stop()

    # ---- reduce over ranks (max time), aggregate over replicas
    times = max_over_ranks([total_ms, e2e_ms, e2e_graph_ms] + [seg_ms[M] for M in Ms], world, device)
    total_ms, e2e_ms, e2e_graph_ms = times[0], times[1], times[2]
    seg_ms = {M: times[3 + i] for i, M in enumerate(Ms)}

    sms = torch.cuda.get_device_properties(device).multi_processor_count
    launches_step = sum(launches_per_gemm(spec, M, nm, sms) for M in Ms for (_D, _x, _y, nm) in per_m[M])
    kernels = {M: kernel_of(spec, M, sms) + (" bf16" if bf16 else " on 8-bit planes" if w8 else "") for M in Ms}
    out = dict(total_ms=total_ms, e2e_ms=e2e_ms, e2e_graph_ms=e2e_graph_ms, e2e_steps=e2e_steps, seg_ms=seg_ms, clocks=clocks, bytes_m=bytes_m,
               flops_m=flops_m, h2d=h2d, d2h=d2h, launches_step=launches_step, kernels=kernels,
               matmuls={M: len(per_m[M]) for M in Ms}, Ms=Ms)
    del per_m, graphs, step_problems, step_items, host_io, staging
    torch.cuda.empty_cache()
    return out


def per_shape_m1(spec, env, reps=20):
    """Each shape on its own at M = 1: a CUDA graph over enough distinct copies of the layer (600 MB) that every launch
    streams HBM-cold weights, CUDA events around its replays.  The first entry of the 7B shapes' `o` is configs[0]."""
    torch, B, H, device = env["torch"], env["B"], env["H"], env["device"]
    import math
    out = {}
    stream = torch.cuda.Stream(device=device)
    ws = H.WorkspaceHolder(device=device)
    for name, (K, N) in spec["shapes"].items():
        copies = max(2, math.ceil(600e6 / (K * N // 2)))
        w8 = spec.get("w8", False)
        if w8:
            copies = max(2, copies // 2)
        L = make_layer(spec, K, N, wl.seed_for("per-shape", name))
        bf16 = spec.get("bf16", False)
        gemm = H.gemm_bf16 if bf16 else H.gemm_w8 if w8 else H.gemm
        if w8:
            Ds = [H.upload_and_repack_w8(L, device=device) for _ in range(copies)]
        else:
            Ds = [H.upload_and_repack(L, device=device, scales_bf16_bits=bf16_scales(L, 0, name) if bf16 else None)
                  for _ in range(copies)]
        if bf16:
            x = H.bf16_from_bits(wl.make_x_bf16(1, K, wl.seed_for("per-shape-x", name)), device)
        else:
            x = H.to_device(wl.make_x(1, K, wl.seed_for("per-shape-x", name)), device)
        y = torch.empty((1, N), dtype=torch.bfloat16 if bf16 else torch.float16, device=device)
        ws.ensure_for(1, Ds[0])
        if w8:
            H.ensure_for_w8(ws, 1, Ds[0])
        with torch.cuda.stream(stream):
            for D in Ds:
                gemm(x, D, y, stream=stream)
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for D in Ds:
                    gemm(x, D, y, stream=stream)
            for _ in range(3):
                g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                g.replay()
            e1.record(stream)
            stream.synchronize()
        us = 1e3 * e0.elapsed_time(e1) / reps / copies
        gbs = wl.algorithmic_bytes(1, K, N, wbits=8 if w8 else 4) / us / 1e3
        out[name] = {"K": K, "N": N, "us": round(us, 3), "GB/s": round(gbs, 1),
                     "pct_of_nominal": round(100 * gbs / NOMINAL_HBM_GBS, 2), "copies": copies}
        del Ds, g
        torch.cuda.empty_cache()
    B.check(B.gptq_check_status(), "per-shape pass")
    return out


def report_line(name, spec, layers, steps, warmup, r, world):
    """The JSON fields of one measured workload."""
    total_ms, e2e_ms, e2e_steps, seg_ms, clocks = r["total_ms"], r["e2e_ms"], r["e2e_steps"], r["seg_ms"], r["clocks"]
    bytes_m, flops_m, h2d, d2h, launches_step, Ms = r["bytes_m"], r["flops_m"], r["h2d"], r["d2h"], r["launches_step"], r["Ms"]
    n_matmuls = r["matmuls"]
    peaks = measured_peaks()
    metric, unit = metric_of(spec)
    step_bytes, step_flops = sum(bytes_m.values()), sum(flops_m.values())
    value = whole_job_value(spec, world, step_bytes, step_flops, steps, total_ms)
    e2e_value = whole_job_value(spec, world, step_bytes, step_flops, e2e_steps, e2e_ms)
    e2e_graph_value = whole_job_value(spec, world, step_bytes, step_flops, e2e_steps, r["e2e_graph_ms"])
    per_m_report = {}
    for M in Ms:
        s = seg_ms[M] / 1e3
        per_m_report[str(M)] = {
            "GB/s": round(bytes_m[M] * steps / s / 1e9, 1),
            "TFLOP/s": round(flops_m[M] * steps / s / 1e12, 2),
            "us_per_matmul": round(1e6 * s / steps / n_matmuls[M], 3),
            "kernel": r["kernels"][M],
        }
    # dominant kernel: the kernel instantiation that took most of the timed region
    groups = {}
    for M in Ms:
        groups.setdefault(r["kernels"][M], []).append(M)
    kname = max(groups, key=lambda k: sum(seg_ms[M] for M in groups[k]))
    dom_Ms = groups[kname]
    dom_s = sum(seg_ms[M] for M in dom_Ms) / 1e3
    dom_launches = sum(n_matmuls[M] for M in dom_Ms) * steps
    if spec["kind"] == "prefill":
        achieved = sum(flops_m[M] for M in dom_Ms) * steps / dom_s / 1e12
        # a timed region of under a second runs at burst clocks: it is held against the burst cuBLAS figure,
        # a longer one (the power cap has pulled the clocks down) against the sustained one
        sustained = total_ms >= 1000.0
        peak, bound, runit = peaks["tflops_sustained" if sustained else "tflops_burst"], "tensor", "TFLOP/s"
    else:
        achieved = sum(bytes_m[M] for M in dom_Ms) * steps / dom_s / 1e9
        peak, bound, runit = peaks["hbm_gbs"], "hbm", "GB/s"
    digest = kernel_source_digest(kname)
    # DRAM bytes per launch come from an ncu capture of this kernel (never from this run): the capture's ratio of
    # measured to algorithmic bytes, scaled by the units a timed launch processes; null when the kernel sources
    # changed since, or when the timed launches cover token counts the capture did not
    traffic, traffic_source = None, None
    t = NCU_TRAFFIC.get(kname)
    if t and t.get("digest") == digest and set(dom_Ms) <= set(t["Ms"]):
        traffic = round(t["ratio"] * sum(bytes_m[M] for M in dom_Ms) * steps / dom_launches)
        traffic_source = t["source"]
    roofline = {
        "bound": bound, "achieved": round(achieved, 2), "peak": peak, "unit": runit,
        "frac": round(achieved / peak, 4), "traffic": traffic, "traffic_source": traffic_source, "kernel": kname,
        "peak_source": peaks["source"],
        "avg_launch_us": round(1e6 * dom_s / dom_launches, 3),
        "alg_bytes_per_launch": round(sum(bytes_m[M] for M in dom_Ms) * steps / dom_launches),
        "launches_timed": dom_launches, "M_covered": dom_Ms,
        "frac_of_nominal": round(achieved / (NOMINAL_FP16_TFLOPS if spec["kind"] == "prefill" else NOMINAL_HBM_GBS), 4),
    }
    line = {
        "metric": metric, "value": round(value, 2), "unit": unit, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": round(total_ms / steps, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if spec.get("bf16", False) else "f16", "data": "synthetic",
        "config": {"workload": name, "describes": spec["describes"], "layers": layers,
                   "matmuls_per_step": sum(n_matmuls[M] for M in Ms), "group_size": 128,
                   "act_order": spec["act_order"], "parallelism": f"{world} independent replica(s)",
                   "l2": f"inputs larger than L2: each M pass streams {round(bytes_m[Ms[0]] / 1e6)} MB of distinct weights",
                   "timing": "CUDA events around CUDA-graph replays of the " + ("gptq_gemm_bf16" if spec.get("bf16", False) else "gptq_gemm_w8" if spec.get("w8", False) else "gptq_gemm") +
                             " calls, one graph per M"},
        "clocks": clocks,
        "e2e": {"value": round(e2e_value, 2), "unit": unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": round(e2e_ms / e2e_steps, 4),
                "api": ("one gptq_gemm_host_batch_bf16" if spec.get("bf16", False) else "one gptq_gemm_host_batch_w8" if spec.get("w8", False) else "one gptq_gemm_host_batch") +
                       " call per step (x from pinned host memory, y back to it, per matmul)",
                "graph_replay": {"value": round(e2e_graph_value, 2), "ms_per_step": round(r["e2e_graph_ms"] / e2e_steps, 4),
                                 "what": "the same call captured once into a CUDA graph and replayed per step: the copies and "
                                         "the matmuls still run every step, the host only launches the graph"}},
        "gpu_launches": launches_step * steps,
        "per_M": per_m_report,
        "roofline": roofline,
        "pct_of_nominal": round(100 * value / world / (NOMINAL_FP16_TFLOPS if spec["kind"] == "prefill" else NOMINAL_HBM_GBS), 2),
    }
    if spec["kind"] == "prefill":
        roofline["peak_kind"] = "sustained" if sustained else "burst"
        roofline["frac_of_burst_peak"] = round(achieved / peaks["tflops_burst"], 4)
        roofline["frac_of_sustained_peak"] = round(achieved / peaks["tflops_sustained"], 4)
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="decode7b", choices=list(WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="distinct weight copies per shape (0 = workload default)")
    ap.add_argument("--e2e-steps", type=int, default=0, help="end-to-end steps (0 = min(steps, 20))")
    ap.add_argument("--ms", default="", help="comma-separated subset of the workload's token counts (profiling small cases)")
    ap.add_argument("--cta-pairs", action="store_true", help="prefill on CTA pairs (tcgen05 cta_group::2), off by default")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--wbits", type=int, default=4, choices=[4, 8],
                    help="8: the same workload with 8-bit GPTQ weights (gptq_repack_w8 / gptq_gemm_w8)")
    ap.add_argument("--dtype", default="f16", choices=["f16", "bf16"],
                    help="bf16: the same workload with bfloat16 activations and scales (gptq_gemm_bf16)")
    ap.add_argument("--prefill-steps", type=int, default=10,
                    help="decode7b only: steps of the prefill7b workload measured after it and reported as `prefill` (0 = skip)")
    ap.add_argument("--ref-budget", type=float, default=150.0,
                    help="--impl reference: seconds of CPU time the whole run should take (sizes the per-step sample)")
    ap.add_argument("--print-digest", action="store_true", help="print the kernel-source digest and exit")
    args = ap.parse_args()
    if args.print_digest:
        for k in KERNEL_SOURCES:
            print(k, kernel_source_digest(k))
        return
    spec = dict(WORKLOADS[args.workload])
    if args.ms:
        spec["Ms"] = tuple(int(m) for m in args.ms.split(","))
    if args.dtype == "bf16":
        spec["bf16"] = True
    if args.wbits == 8:
        if args.dtype == "bf16":
            raise SystemExit("--wbits 8 runs with fp16 activations only")
        spec["w8"] = True
        spec["describes"] += " - with 8-bit weights (gptq_gemm_w8: two stacked 4-bit planes)"
    layers = args.layers or spec["layers"]
    if args.impl == "reference":
        run_reference(args, spec)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the GPTQ matmul has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)

    from paper_2511_19438_b200 import build as libbuild
    if local_rank == 0:
        libbuild.build()
    if world > 1:
        dist.barrier()
    from paper_2511_19438_b200 import binding as B
    from paper_2511_19438_b200 import harness as H

    if args.cta_pairs:
        B.check(B.gptq_set_cta_pairs(1), "gptq_set_cta_pairs")
    env = dict(torch=torch, dist=dist, B=B, H=H, device=device, world=world, rank=rank, local_rank=local_rank)
    res = measure_workload(args.workload, spec, layers, args.steps, args.warmup, args.e2e_steps or min(args.steps, 20), env)
    # The metric has a second half (prefill TFLOP/s): the default run measures it too, as a short pass of the
    # prefill workload after the decode one, and reports it as a sub-object of the same line.
    prefill = None
    if args.workload == "decode7b" and not args.ms and args.prefill_steps > 0:
        pspec = dict(WORKLOADS["prefill7b"], bf16=spec.get("bf16", False), w8=spec.get("w8", False))
        prefill = measure_workload("prefill7b", pspec, pspec["layers"], args.prefill_steps, 3, min(args.prefill_steps, 5), env)
    shapes_m1 = None
    if args.workload == "decode7b" and not args.ms and world == 1:
        shapes_m1 = per_shape_m1(spec, env)
    if rank == 0:
        line = report_line(args.workload, spec, layers, args.steps, args.warmup, res, world)
        if shapes_m1 is not None:
            # configs[0] is the 4096 x 4096 layer at M = 1; the two performance targets, stated with what was measured
            line["per_shape_M1"] = shapes_m1
            m1 = line["per_M"].get("1", {})
            line["targets"] = {
                "decode_M1_pct_of_8TBs": round(100 * m1.get("GB/s", 0.0) / NOMINAL_HBM_GBS, 2), "decode_target_pct": 70,
                "decode_met": bool(m1.get("GB/s", 0.0) >= 0.7 * NOMINAL_HBM_GBS),
                "config1_o_4096x4096_M1_pct_of_8TBs": shapes_m1.get("o", {}).get("pct_of_nominal"),
            }
        if prefill is not None:
            pl = report_line("prefill7b", pspec, pspec["layers"], args.prefill_steps, 3, prefill, world)
            line["prefill"] = {k: pl[k] for k in ("metric", "value", "unit", "steps", "warmup", "ms_per_step", "config",
                                                  "clocks", "e2e", "gpu_launches", "per_M", "roofline", "pct_of_nominal")}
            if "targets" in line:
                worst = min(v["TFLOP/s"] for m, v in pl["per_M"].items() if int(m) >= 1024)
                line["targets"].update({"prefill_min_TFLOPs_M_ge_1024": worst, "prefill_target_TFLOPs": 0.5 * NOMINAL_FP16_TFLOPS,
                                           "prefill_met": bool(worst >= 0.5 * NOMINAL_FP16_TFLOPS)})
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(spec)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
