"""Launch timeline of a chain of decode matmuls: do consecutive launches overlap?

    python -m paper_2511_19438_b200.timeline [--shapes 7b|13b] [--only gate_up,down] [--m 1] [--rounds 3] [--act-order]

Builds the library with the launch timeline compiled in (as libgptq_b200_timeline.so, next to the normal build),
captures the layer's matmuls - each on distinct weights, so that every launch streams from HBM - in a CUDA graph,
replays it and prints, per launch, %globaltimer times relative to the moment the previous launch's last CTA was
done: first and last CTA started, first weight copy issued, griddepcontrol.wait first / last returned, first activation tile
landed, last CTA done.  A negative "started" or "weights" column is the overlap that programmatic dependent launch buys.
"""
from __future__ import annotations

import argparse
import os


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shapes", default="7b", choices=["7b", "13b"])
    ap.add_argument("--m", type=int, default=1)
    ap.add_argument("--rounds", type=int, default=3, help="times the layer's matmuls are chained (distinct weights each)")
    ap.add_argument("--act-order", action="store_true")
    ap.add_argument("--only", default="", help="comma-separated shape names: chain only these (e.g. gate_up)")
    args = ap.parse_args()

    from . import build as libbuild
    os.environ["GPTQ_B200_LIB"] = libbuild.build_timeline()
    import torch
    from . import binding as B, harness as H, workloads as wl

    shapes = wl.SHAPES_7B if args.shapes == "7b" else wl.SHAPES_13B
    if args.only:
        shapes = {k: v for k, v in shapes.items() if k in args.only.split(",")}
        assert shapes, "no such shape"
    M = args.m
    ws = H.WorkspaceHolder()
    chain = []
    for r in range(args.rounds):
        for name, (K, N) in shapes.items():
            L = wl.make_linear(K, N, seed=wl.seed_for("timeline", name, r), act_order=args.act_order)
            D = H.upload_and_repack(L)
            ws.ensure_for(M, D)
            x = H.to_device(wl.make_x(M, K, wl.seed_for("timeline-x", name)))
            y = torch.empty((M, N), dtype=torch.float16, device="cuda")
            chain.append((name, D, x, y))
    assert len(chain) <= 64, "the timeline holds 64 launches"
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _, D, x, y in chain:
            H.gemm(x, D, y, stream=stream)
        stream.synchronize()
        # launches take timeline rows round robin: find out which row the captured launches start at
        B.check(B.gptq_trace_reset(stream), "gptq_trace_reset")
        H.gemm(chain[0][2], chain[0][1], chain[0][3], stream=stream)
        n, rows = B.gptq_trace_read(64, stream)
        first_row = (next(i for i, r in enumerate(rows) if r[6] != 0) + 1) % 64
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _, D, x, y in chain:
                H.gemm(x, D, y, stream=stream)
        for _ in range(3):
            g.replay()
        stream.synchronize()
        B.check(B.gptq_trace_reset(stream), "gptq_trace_reset")
        g.replay()
        stream.synchronize()
        n, rows = B.gptq_trace_read(64, stream)
    assert B.gptq_check_status() == B.GPTQ_OK
    launches = [rows[(first_row + i) % 64] for i in range(len(rows))]
    launches = [r for r in launches if r[6] != 0]
    print(f"M = {M}, {len(chain)} matmuls ({'act-order: a gather launch precedes each, not traced' if args.act_order else 'no act-order'}); "
          f"{len(launches)} traced launches; microseconds relative to the previous launch's last CTA being done")
    print(f"{'launch':>6} {'shape':>8} {'kernel':>8} {'CTAs':>5} | {'started':>8} {'last CTA':>8} {'weights':>8} {'wait first':>10} {'wait last':>9} "
          f"{'x landed':>8} {'done':>7} | {'own duration':>12}")
    prev_exit = None
    names = [c[0] for c in chain]
    for i, r in enumerate(launches):
        entry, wissue, wait0, wait1, data, last, kc, last_entry = r
        kid, ctas = kc >> 32, kc & 0xffffffff
        ref = prev_exit if prev_exit is not None else entry
        f = lambda v: f"{(v - ref) / 1e3:8.2f}" if v not in (0, 2 ** 64 - 1) else "       -"
        name = names[i] if len(launches) == len(chain) else "?"
        print(f"{i:6d} {name:>8} {'mma.sync' if kid == 1 else 'tcgen05':>8} {ctas:5d} | {f(entry)} {f(last_entry)} {f(wissue)} {f(wait0):>10} {f(wait1):>9} "
              f"{f(data)} {f(last):>7} | {(last - entry) / 1e3:12.2f}")
        prev_exit = last


if __name__ == "__main__":
    main()
