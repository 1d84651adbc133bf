"""Runs a few aggregations of one workload at a chosen dimension: the command
line that profiler captures (ncu) and quick timings are taken on.

    python -m paper_1905_04374_b200.profile_case --config 3 --d 2000000 --rule multi_bulyan --reps 3
"""
from __future__ import annotations

import argparse

import torch

import paper_1905_04374_b200 as pkg


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--d", type=int, default=None)
    ap.add_argument("--rule", default="multi_bulyan")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--stages", action="store_true", help="time the three kernels separately")
    args = ap.parse_args()
    wl = pkg.workloads.WORKLOADS[args.config]
    G, _ = pkg.workloads.make_gradients(args.config, d=args.d, device="cuda:0")
    n, d = G.shape
    out = torch.empty(d, dtype=torch.float32, device="cuda:0")
    for _ in range(2):
        pkg.gar_aggregate(args.rule, G, wl.f, out=out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        pkg.gar_aggregate(args.rule, G, wl.f, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.reps
    theta = pkg.gar_theta(args.rule, n, wl.f)
    print(f"{args.rule} n={n} f={wl.f} d={d} theta={theta}: {ms:.4f} ms per aggregation")
    if args.stages:
        dist = torch.empty(n, n, dtype=torch.float64, device="cuda:0")
        sel = pkg.new_selection("cuda:0")

        def timed(fn):
            fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(args.reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.reps

        preagg = int(args.rule in ("multi_bulyan", "multi_krum", "average"))
        t1 = timed(lambda: pkg.gar_pairwise_distances(G, dist=dist))
        t2 = timed(lambda: pkg.gar_select(args.rule, dist, n, wl.f, sel=sel))
        t3 = timed(lambda: pkg.gar_coordinate_phase(G, sel, theta, preagg, out=out))
        s = pkg.read_selection(sel)
        rows = s.nu
        print(f"  distances {t1:.4f} ms ({4e-6 * n * d / t1:.0f} GB/s of n*d*4)   select {t2:.4f} ms   "
              f"coordinate {t3:.4f} ms ({4e-6 * (rows + 1) * d / t3:.0f} GB/s of (rows+1)*d*4, rows={rows}, plan adds={s.total_adds})")


if __name__ == "__main__":
    main()
