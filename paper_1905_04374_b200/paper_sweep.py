"""The timing grid of Section 5.1 on this library: n in {7, 9, .., 39}, f = floor((n - 3) / 4),
d in {1e5, 1e6, 1e7}, n gradients drawn i.i.d. from U(0, 1)^d, and the section's protocol:
synchronise, start a wall-clock timer, aggregate on the GPU, synchronise, stop; seven runs, the
two farthest from the median dropped, mean and standard deviation of the other five.

    python -m paper_1905_04374_b200.paper_sweep [--rules multi_bulyan,multi_krum,median] [--markdown] [--linearity]

Prints one line per (rule, d, n): mean and standard deviation in milliseconds.  `--linearity`
adds the check behind Theorem 2 (ii) (O(d) computation): at fixed n the times at d = 1e7, 2e7,
4e7, 8e7 must lie within 25 % of one straight line a + b d (a: launches and the selection).
"""
from __future__ import annotations

import argparse
import statistics
import time

def robust_mean_std(times, keep: int = 5):
    """Section 5.1's statistic: of the measured runs drop the ones farthest from the median until
    `keep` are left (seven runs, two dropped), then mean and (population) standard deviation."""
    times = list(times)
    med = statistics.median(times)
    kept = sorted(times, key=lambda t: abs(t - med))[:keep]
    return statistics.mean(kept), statistics.pstdev(kept)


def time_rule(rule: str, G, f: int, out, runs: int = 7, keep: int = 5):
    import torch
    import paper_1905_04374_b200 as pkg
    pkg.gar_aggregate(rule, G, f, out=out)          # first call: module load, cached workspace
    times = []
    for _ in range(runs):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        pkg.gar_aggregate(rule, G, f, out=out)
        torch.cuda.synchronize()
        times.append((time.perf_counter() - t0) * 1e3)
    return robust_mean_std(times, keep)


def linearity(rule: str = "multi_bulyan", ns=(15, 39), dims=(10_000_000, 20_000_000, 40_000_000, 80_000_000)):
    """Times at fixed n over growing d against their least-squares line a + b d (Theorem 2 (ii):
    the computation is O(d))."""
    import torch
    import paper_1905_04374_b200 as pkg
    ok = True
    for n in ns:
        f = (n - 3) // 4
        ts = []
        for d in dims:
            G = pkg.workloads.make_uniform(n, d, device="cuda:0", seed=1905 + n)
            out = torch.empty(d, dtype=torch.float32, device="cuda:0")
            ts.append(time_rule(rule, G, f, out)[0])
            del G, out
        mx, my = sum(dims) / len(dims), sum(ts) / len(ts)
        b = sum((x - mx) * (y - my) for x, y in zip(dims, ts)) / sum((x - mx) ** 2 for x in dims)
        a = my - b * mx
        worst = max(abs(y - (a + b * x)) / y for x, y in zip(dims, ts))
        ok &= worst <= 0.25
        print(f"linearity {rule} n={n}: ms at d={list(dims)}: " + ", ".join(f"{t:.3f}" for t in ts) +
              f"; line {a:.3f} ms + {b * 1e6:.4f} ns/coordinate; largest residual {100 * worst:.1f} % "
              f"({'ok' if worst <= 0.25 else 'NOT linear'})")
    return ok


def main():
    import torch
    import paper_1905_04374_b200 as pkg
    ap = argparse.ArgumentParser()
    ap.add_argument("--rules", default="multi_bulyan,bulyan,multi_krum,median,average")
    ap.add_argument("--dims", default="100000,1000000,10000000")
    ap.add_argument("--markdown", action="store_true", help="one table per rule, n down, d across")
    ap.add_argument("--linearity", action="store_true", help="only the O(d) check of Theorem 2 (ii)")
    args = ap.parse_args()
    if args.linearity:
        raise SystemExit(0 if linearity() else 1)
    rules = args.rules.split(",")
    dims = [int(x) for x in args.dims.split(",")]
    ns = list(range(7, 40, 2))
    res = {}
    for d in dims:
        for n in ns:
            f = (n - 3) // 4
            G = pkg.workloads.make_uniform(n, d, device="cuda:0", seed=1905 + n)
            out = torch.empty(d, dtype=torch.float32, device="cuda:0")
            for rule in rules:
                res[(rule, d, n)] = time_rule(rule, G, f, out)
                if not args.markdown:
                    m, s = res[(rule, d, n)]
                    print(f"{rule:13s} d={d:<9d} n={n:<3d} f={f:<2d} {m:9.4f} ms +- {s:.4f}")
            del G, out
    if args.markdown:
        for rule in rules:
            print(f"\n### {rule}\n")
            print("| n | f | " + " | ".join(f"d = {d:.0e}" for d in dims) + " |")
            print("|---|---|" + "---|" * len(dims))
            for n in ns:
                cells = " | ".join("%.3f ± %.3f" % res[(rule, d, n)] for d in dims)
                print(f"| {n} | {(n - 3) // 4} | {cells} |")


if __name__ == "__main__":
    main()
