"""Last calibration step of the latency model: one scale factor per variant group.

    python bench.py --validate-model 400 --validate-roof-us 0.3 --dump-candidates cand.csv     (on a B200)
    python -m paper_2608_10803_b200.calibrate cand.csv                                          (anywhere)

Reads the CSV of timed configurations (every legal configuration of the sampled shapes with the
model's prediction and the measured time) and prints, per variant group, the geometric mean of
measured / predicted time and the number of configurations behind it, then the initializer for
``Calib::group_bias`` in ``csrc/adapt_internal.h``.  The predictions in the CSV already carry the
factors the library was built with, so the printed table is the product of old and new factors
when the old ones are passed with ``--current``.  Groups mirror ``calib_group`` in
``csrc/adapt_select.cpp``.
"""
from __future__ import annotations

import argparse
import csv
import math

GROUPS = 40
NAMES = {0: "plain P_k=1", 1: "plain P_k=1 + prologue", 2: "plain split-K", 3: "plain split-K + prologue", 4: "plain fused split-K",
         5: "plain stream-K", 6: "row classes P_k=1", 7: "row classes split-K", 8: "row classes fused", 9: "halo class tiles",
         10: "k-class accumulators", 11: "k classes as splits", 12: "k classes fused", 13: "warp-level P_k=1", 14: "warp-level split-K",
         15: "CUDA-core P_k=1", 16: "CUDA-core split-K", 17: "one-launch cluster of 1", 18: "one-launch cluster > 1"}


def group_of(row) -> int:
    fam, bn, pk = row["family"], int(row["BN"]), int(row["P_k"])
    src_a, src_b = int(row["srcA"]), int(row["srcB"])
    fused, sk, cluster = int(row["fused"]), int(row["streamk"]), int(row["cluster"])
    if fam == "skinny":
        return 13 if pk == 1 else 14
    if fam == "simt":
        return 15 if pk == 1 else 16
    if fam == "cluster":
        return 17 if cluster == 1 else 18
    pro = src_a == 1 or src_b == 1
    if src_b == 3:
        g = 10 if bn == 64 else (12 if fused else 11)
    elif src_a == 3:
        g = 9 if bn % 64 else (8 if fused else (6 if pk == 1 else 7))
    elif fused:
        g = 4
    elif sk:
        g = 5
    else:
        g = (0 if pk == 1 else 2) + (1 if pro else 0)
    return g + (20 if fam == "umma_2cta" else 0)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("csv", nargs="+")
    ap.add_argument("--current", default="", help="comma-separated factors the library was built with (default: all 1)")
    ap.add_argument("--near-best", type=float, default=3.0, help="only configurations within this factor of their shape's best time count")
    args = ap.parse_args()
    current = [1.0] * GROUPS
    if args.current:
        vals = [float(x) for x in args.current.split(",")]
        current[:len(vals)] = vals
    rows = []
    for path in args.csv:
        with open(path, newline="") as f:
            rows += list(csv.DictReader(f))
    best = {}
    for r in rows:
        key = (r["M"], r["N"], r["K"], r["dtype"])
        best[key] = min(best.get(key, float("inf")), float(r["time_us"]))
    sums, counts = [0.0] * GROUPS, [0] * GROUPS
    for r in rows:
        t, pred = float(r["time_us"]), float(r["pred_us"])
        # configurations far from the best of their shape never decide a selection: leave them out of the fit
        if t <= 0 or pred <= 0 or t > args.near_best * best[(r["M"], r["N"], r["K"], r["dtype"])]:
            continue
        g = group_of(r)
        sums[g] += math.log(t / pred)
        counts[g] += 1
    out = []
    for g in range(GROUPS):
        f = math.exp(sums[g] / counts[g]) if counts[g] >= 20 else 1.0
        out.append(current[g] * f)
        if counts[g]:
            name = NAMES.get(g % 20, "?") + (" (pair tiles)" if g >= 20 else "")
            print(f"group {g:2d} {name:32s} n={counts[g]:6d} measured/predicted {f:.3f} -> factor {out[-1]:.3f}")
    print("group_bias = {" + ", ".join(f"{x:.3f}" for x in out) + "};")


if __name__ == "__main__":
    main()
