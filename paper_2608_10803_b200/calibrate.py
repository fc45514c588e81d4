"""Calibration of the latency model from timed configurations.

Two tools over the same input, the CSV that ``bench.py --validate-model N --dump-candidates cand.csv`` writes on
a B200 (every legal configuration of the sampled shapes, with the model's prediction and the measured time):

``python -m paper_2608_10803_b200.calibrate fit train.csv [more.csv] [--check other_seed.csv]`` moves the model's
constants (``adapt_get_calibration`` / ``adapt_set_calibration``) by coordinate descent so that the configuration
the model picks is, on average, as close as possible to the fastest timed one (mean regret), and prints the
constants that changed; ``--check`` reports the same figures on a shape set the fit has not seen.  It needs no GPU:
the model runs on the host.

``python -m paper_2608_10803_b200.calibrate cand.csv`` (no sub-command) is the older per-group report:

Last calibration step of the latency model: one scale factor per variant group.

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


FAMILY_ID = {"umma_1cta": 0, "umma_2cta": 1, "skinny": 2, "simt": 3, "cluster": 4}


class TimedSet:
    """Timed configurations of a set of shapes, keyed the way the model's candidates are."""

    def __init__(self, paths):
        self.shapes = {}
        for path in paths:
            with open(path, newline="") as f:
                for r in csv.DictReader(f):
                    shape = (int(r["M"]), int(r["N"]), int(r["K"]), int(r["dtype"]))
                    cfg = (FAMILY_ID[r["family"]], int(r["BN"]), int(r["stages"]), int(r["P_k"]), int(r["cluster"]), int(r["fused"]),
                           int(r["streamk"]), int(r["srcA"]), int(r["srcB"]))
                    t = float(r["time_us"])
                    d = self.shapes.setdefault(shape, {})
                    d[cfg] = min(d.get(cfg, float("inf")), t)

    def metrics(self, ab):
        """Regret of the model's pick among the timed configurations of every shape, with the constants now set."""
        regrets, picked, best_sum, sq, n_near = [], 0.0, 0.0, 0.0, 0
        for (M, N, K, dt), timed in self.shapes.items():
            best = min(timed.values())
            pick_pred, pick_t = float("inf"), None
            for c in ab.adapt_plan_candidates(M, N, K, dt):
                t = timed.get((c.family, c.BN, c.stages, c.P_k, c.cluster, c.fused, c.streamk, c.srcA, c.srcB))
                if t is None:
                    continue
                if c.predicted_us < pick_pred:
                    pick_pred, pick_t = c.predicted_us, t
                if t <= 1.5 * best:
                    sq += math.log(c.predicted_us / t) ** 2
                    n_near += 1
            if pick_t is None:
                continue
            regrets.append(pick_t / best)
            picked += pick_t
            best_sum += best
        regrets.sort()
        n = len(regrets)
        return {"shapes": n, "mean": sum(regrets) / n, "p95": regrets[min(n - 1, int(0.95 * n))], "max": regrets[-1],
                "exact": sum(1 for r in regrets if r <= 1.0001) / n, "within_2pct": sum(1 for r in regrets if r <= 1.02) / n,
                "time_weighted": picked / best_sum, "rms_log_error_near_best": math.sqrt(sq / max(1, n_near))}


def fit(argv):
    ap = argparse.ArgumentParser(prog="calibrate fit")
    ap.add_argument("csv", nargs="+", help="timed configurations to fit on")
    ap.add_argument("--check", nargs="*", default=[], help="timed configurations of shapes the fit does not see")
    ap.add_argument("--rounds", type=int, default=1)
    ap.add_argument("--steps", default="0.8,0.9,1.1,1.25", help="factors tried on each constant")
    ap.add_argument("--only", default="", help="comma-separated names of the constants to move (default: all)")
    args = ap.parse_args(argv)
    from . import binding as ab
    train = TimedSet(args.csv)
    check = TimedSet(args.check) if args.check else None
    names = [x for x in args.only.split(",") if x] or ab.adapt_calibration_names()
    steps = [float(x) for x in args.steps.split(",")]
    start = {k: ab.adapt_get_calibration(k) for k in names}

    def objective(m):      # the regret decides; the prediction error only breaks ties between equal selections
        return m["mean"] + 0.5 * (m["time_weighted"] - 1.0) + 0.05 * m["rms_log_error_near_best"]

    def show(tag, m):
        print(tag, " ".join(f"{k}={v:.4f}" if isinstance(v, float) else f"{k}={v}" for k, v in m.items()), flush=True)

    m0 = train.metrics(ab)
    show("fit set, before:  ", m0)
    if check:
        show("check set, before:", check.metrics(ab))
    best = objective(m0)
    for rnd in range(args.rounds):
        moved = False
        for k in names:
            x0 = ab.adapt_get_calibration(k)
            for f in steps:
                ab.adapt_set_calibration(k, x0 * f)
                m = train.metrics(ab)
                if objective(m) < best - 2e-4:
                    best, moved = objective(m), True
                    print(f"round {rnd}: {k} {x0:g} -> {x0 * f:g}  mean regret {m['mean']:.4f}", flush=True)
                    x0 = x0 * f
                else:
                    ab.adapt_set_calibration(k, x0)
        if not moved:
            break
    show("fit set, after:   ", train.metrics(ab))
    if check:
        show("check set, after: ", check.metrics(ab))
    for k in names:
        v = ab.adapt_get_calibration(k)
        if v != start[k]:
            print(f"    double {k} = {v:.4g};    // was {start[k]:g}")


def main():
    import sys
    if len(sys.argv) > 1 and sys.argv[1] == "fit":
        return fit(sys.argv[2:])
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
