#!/usr/bin/env python
"""Benchmark of the adaptive GEMM library on the 2,000-shape dynamic sweep (one B200 per rank).

    python bench.py --gpus 1 --steps 5 --warmup 3
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference ...        # the CPU oracle on a bounded sample (context only)

A "step" is one pass of the whole hot path (plan lookup -> launch, every kernel family the
selector chose) over all 2,000 shapes of the sweep, inputs resident in HBM.  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

NOMINAL_FLOPS = 2.25e15      # dense fp16/bf16, the roofline the target is stated against
NOMINAL_HBM = 8.0e12
L2_BYTES = 126e6
METRIC = "TFLOP/s and roofline fraction per shape (geomean over sweep) on 1 B200"
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) over algorithmic bytes, from the ncu
# captures summarised in profiles/kernels_ncu_full.md (small cases of the same kernels: traffic
# grows with the bytes a launch moves, so the ratio is applied to the launch's algorithmic bytes).
# Keyed by kernel variant (family / tiling mode).
NCU_TRAFFIC_RATIO = {
    "umma_1cta/halo_class_tiles": 0.93,      # 20000 x 20001 x 12: 746.9 / 801.0 MB (part of C still in L2 at kernel end)
    "umma_1cta/row_class_tiles": 1.02,       # 20000 x 8 x 60001: 2445.2 / 2401.3 MB
    "umma_1cta/k_classes_as_splits": 1.04,   # 8 x 30001 x 8000: 497.6 / 480.6 MB
    "umma_1cta/k_classes_as_splits+fused_reduce": 1.04,
    "umma_1cta/row_class_tiles+fused_reduce": 1.02,
    "umma_1cta/plain_tiles+fused_reduce": 1.01,
    "umma_2cta/k_classes_as_splits": 1.04,
    "umma_1cta/plain_tiles": 1.01,           # 16 x 65536 x 4096: 546.8 / 539.1 MB
    "umma_2cta/plain_tiles": 0.87,           # 4096^3: 87.9 / 100.7 MB
    "umma_2cta/plain_tiles+stream_k": 0.87,
    "umma_1cta/plain_tiles+stream_k": 1.01,
}


def kernel_variant(ab, info):
    """Kernel variant of a plan: family / tiling mode (the template instantiations that share an access pattern)."""
    fam = ab.FAMILY_NAMES[info.family]
    if not fam.startswith("umma"):
        return fam
    if info.srcB == 3:
        mode = "k_class_accumulators" if info.BN == 64 else "k_classes_as_splits"
    elif info.srcA == 3:
        mode = "halo_class_tiles" if info.BN % 64 else "row_class_tiles"
    else:
        mode = "plain_tiles"
    return f"{fam}/{mode}" + ("+fused_reduce" if info.fused else "") + ("+stream_k" if info.streamk else "")


def max_over_ranks(x, dist, device):
    """The slowest rank's value: a multi-GPU number is timed on the device as the maximum over ranks."""
    if dist is None:
        return x
    import torch
    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replicas_value(units_per_rank, world, seconds):
    """Whole-job throughput of `world` independent replicas (weak scaling, no data-path collective)."""
    return units_per_rank * world / seconds


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm": d["hbm_gbs"] * 1e9, "tensor_burst": d["bf16_tflops"] * 1e12,
                "tensor_sustained": d["bf16_tflops_sustained"] * 1e12, "source": "measured"}
    return {"hbm": 6.65e12, "tensor_burst": 1.59e15, "tensor_sustained": 1.4e15, "source": "fallback"}


def t_roof_nominal(case):
    return max(case.flops / NOMINAL_FLOPS, case.bytes / NOMINAL_HBM)


def geomean(xs):
    xs = [x for x in xs if x > 0]
    return math.exp(sum(math.log(x) for x in xs) / len(xs)) if xs else 0.0


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            with open(self.path) as f:
                for line in f:
                    p = [x.strip() for x in line.split(",")]
                    if len(p) < 7:
                        continue
                    try:
                        sm.append(float(p[0]))
                        mx.append(float(p[1]))
                    except ValueError:
                        continue
                    for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                        if v.lower().startswith("active"):
                            reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ---------------------------------------------------------------------------------------------
# the CPU oracle on a bounded sample (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------
def oracle_sample(cases, mac_budget):
    """Seeded sample of the sweep for the CPU oracle: shapes of the oracle subset whose operands
    are small enough to draw on the host, complete rows up to a per-shape MAC cap."""
    import numpy as np
    from paper_2608_10803_b200 import synth
    picked, total = [], 0.0
    for idx in synth.sweep_oracle_subset():
        c = cases[idx]
        if c.M * c.K + c.K * c.N > 48e6:
            continue
        rows = int(max(1, min(c.M, 1.5e9 // max(1, c.N * c.K))))
        macs = float(rows) * c.N * c.K
        if macs < 1e6:
            continue
        picked.append((c, rows))
        total += macs
        if total >= mac_budget:
            break
    return picked, total


def run_oracle_sample(sample):
    import numpy as np
    from oracle import gemm as og
    from paper_2608_10803_b200 import synth
    data = []
    for c, rows in sample:
        A, B = synth.draw_case(c, "cpu")
        data.append((c, synth.bits(A).reshape(-1), synth.bits(B).reshape(-1), np.arange(rows, dtype=np.int64)))
    og.gemm_rows(data[0][1], data[0][2], data[0][0].M, data[0][0].N, data[0][0].K, data[0][0].dtype, rows=data[0][3][:1])

    def one_pass():
        t0 = time.perf_counter()
        for c, a, b, r in data:
            og.gemm_rows(a, b, c.M, c.N, c.K, c.dtype, rows=r, want16=True)
        return time.perf_counter() - t0
    return one_pass, og.max_threads()


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2608_10803_b200 import synth
    cases = synth.config_sweep()
    sample, macs = oracle_sample(cases, args.ref_macs)
    one_pass, threads = run_oracle_sample(sample)
    for _ in range(args.warmup):
        one_pass()
    times = [one_pass() for _ in range(args.steps)]
    total = sum(times)
    value = 2.0 * macs * args.steps / total / 1e12
    desc = f"{len(sample)} shapes of the sweep's oracle subset, {macs:.3g} MACs per step (complete leading rows, <=1.5e9 MACs per shape)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "dynamic-shape sweep (2,000 seeded shapes), bounded sample for the CPU oracle", "sample": desc},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------
class Ring:
    def __init__(self, base_ptr, nbytes):
        self.base, self.size, self.off = base_ptr, nbytes, 0

    def take(self, nbytes):
        nbytes = (nbytes + 255) & ~255
        if nbytes > self.size:
            raise RuntimeError("pool smaller than one operand")
        if self.off + nbytes > self.size:
            self.off = 0
        p = self.base + self.off
        self.last_off = self.off
        self.off += nbytes
        return p


def ours(args):
    import torch
    from paper_2608_10803_b200 import binding as ab
    from paper_2608_10803_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    ab.adapt_init(local)
    if args.batch_streams:
        ab.adapt_set_option("batch_streams", args.batch_streams)
    stream = torch.cuda.current_stream().cuda_stream
    peaks = measured_peaks()

    if args.workload == "sweep":
        cases = synth.config_sweep()
        workload = "dynamic-shape sweep: 2,000 seeded shapes, M,N,K log-uniform in [1,1e5], M*N*K<=2^38, fp16/bf16 alternating"
    else:
        cases = synth.config_reco() + synth.config_llm() + synth.config_large() + synth.config_context()
        workload = "named configs: recommendation, LLM-layer, large/tall-K and paper-named shapes"
    if args.limit:
        cases = cases[:args.limit]

    # ---- resident operands: one input pool per dtype, one output pool; shapes take ring slots ----
    gib = 1 << 30
    in_bytes = int(args.pool_gb * gib)
    out_bytes = int(max(14.0, args.pool_gb * 0.6) * gib)
    pools = {}
    for dt in (0, 1):
        if any(c.dtype == dt for c in cases):
            pools[dt] = synth.draw_operand(1, in_bytes // 2, synth.U11, 1234 + dt, dt, "cuda").view(-1)
    out_pool = torch.empty(out_bytes, dtype=torch.uint8, device="cuda")
    rings = {dt: Ring(t.data_ptr(), t.numel() * 2) for dt, t in pools.items()}
    out_ring = Ring(out_pool.data_ptr(), out_bytes)

    plans, infos, slots = [], [], []
    t_plan0 = time.perf_counter()
    for c in cases:
        plans.append(ab.adapt_matmul_plan(c.M, c.N, c.K, c.dtype))
    plan_ms = (time.perf_counter() - t_plan0) * 1e3
    for c, h in zip(cases, plans):
        infos.append(ab.adapt_plan_info(h))
        nb = int(min(8, max(1, math.ceil(2 * L2_BYTES / c.bytes))))
        s = []
        for _ in range(nb):
            a = rings[c.dtype].take(2 * c.M * c.K)
            oa = rings[c.dtype].last_off
            b = rings[c.dtype].take(2 * c.K * c.N)
            ob = rings[c.dtype].last_off
            cc = out_ring.take(2 * c.M * c.N)
            oc = out_ring.last_off
            s.append((a, b, cc, oa, ob, oc))
        slots.append(s)

    lib = ab.load()
    # Pointer policy, the same in the headline pass and in the per-shape pass: every shape owns up to eight
    # operand sets (enough to exceed L2 twice over) and consecutive calls of a shape rotate through them.  The
    # library keeps the tensor-map encodings of the eight most recent pointer sets per plan, so after the
    # warm-up passes no call encodes a map (checked below through adapt_map_encode_count); what a call with
    # never-seen pointers pays is measured separately (dispatch_cost: host_us_call_map_miss).
    n_rot = max(len(s) for s in slots)
    plan_arr = ab.pointer_array(plans)
    rot = []
    for r in range(n_rot):
        rot.append(tuple(ab.pointer_array([s[r % len(s)][j] for s in slots]) for j in range(3)))
    pass_no = [0]

    def one_pass():
        a, b, c_ = rot[pass_no[0] % n_rot]
        pass_no[0] += 1
        st = lib.adapt_matmul_batch(len(plans), plan_arr, a, b, c_, stream)
        if st != 0:
            raise RuntimeError(f"adapt_matmul failed: {lib.adapt_last_error_message().decode()}")

    def barrier():
        if dist is not None:
            dist.barrier()

    for _ in range(max(3, args.warmup, n_rot)):
        one_pass()
    torch.cuda.synchronize()
    ab.adapt_poll_device_status(stream)
    encodes0 = ab.adapt_map_encode_count()

    sampler = ClockSampler(local)
    sampler.start()
    launches0 = ab.adapt_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    ev0.record()
    for _ in range(args.steps):
        one_pass()
    ev1.record()
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = ab.adapt_launch_count() - launches0
    clocks = sampler.stop()
    ms_total = max_over_ranks(ms_total, dist, "cuda")
    ms_step = ms_total / args.steps
    flops_pass = sum(c.flops for c in cases)
    value = replicas_value(flops_pass, world, ms_step * 1e-3) / 1e12

    # ---- per-shape timing: R back-to-back calls between two events, rotating buffer sets ----
    per_shape = None
    if args.shape_passes > 0:
        reps = []
        for info, c in zip(infos, cases):
            reps.append(int(min(20, max(1, 60.0 / max(info.predicted_us, 1.0)))))
        passes = []
        sets = [tuple(ab.pointer_array([x[j] for x in s]) for j in range(3)) for s in slots]
        for _ in range(args.shape_passes):
            evs = []
            for h, s, st3, r in zip(plans, slots, sets, reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                lib.adapt_matmul_repeat(h, len(s), st3[0], st3[1], st3[2], r, stream)
                e1.record()
                evs.append((e0, e1))
            torch.cuda.synchronize()
            passes.append([e0.elapsed_time(e1) * 1e-3 / r for (e0, e1), r in zip(evs, reps)])
        per_shape = [statistics.median(p[i] for p in passes) for i in range(len(cases))]
    ab.adapt_poll_device_status(stream)
    map_encodes_timed = ab.adapt_map_encode_count() - encodes0

    # ---- the launch floor and the host cost of the online call (timed inside the library, in C) ----
    floor = None
    dispatch = None
    if rank == 0 and not args.no_dispatch:
        h_pdl, d_pdl = ab.adapt_measure_empty_launch(20000, True, stream)
        h_np, d_np = ab.adapt_measure_empty_launch(20000, False, stream)
        floor = {"empty_kernel_us_pdl": d_pdl, "empty_kernel_us_no_pdl": d_np, "host_us_per_launch_pdl": h_pdl,
                 "host_us_per_launch_no_pdl": h_np,
                 "how": "20,000 empty kernels back to back on the stream in batches of 128, CUDA events around each batch (device) and steady_clock around the launches (host)"}
        dispatch = {}
        seen_kinds = {}
        for i, (c, info) in enumerate(zip(cases, infos)):
            kind = kernel_variant(ab, info) + ("+reduce" if info.P_k > 1 and info.family != ab.FAM_CLUSTER and not info.fused else "")
            if kind in seen_kinds or c.bytes > 64e6:
                continue
            seen_kinds[kind] = i
        want = ["umma_1cta/plain_tiles", "umma_1cta/halo_class_tiles", "umma_1cta/row_class_tiles", "cluster", "simt",
                "umma_1cta/plain_tiles+reduce", "umma_1cta/k_classes_as_splits+reduce", "umma_1cta/plain_tiles+fused_reduce",
                "umma_1cta/k_classes_as_splits+fused_reduce", "umma_1cta/row_class_tiles+fused_reduce"]
        for kind in want:
            if kind not in seen_kinds:
                continue
            i = seen_kinds[kind]
            a, b, c_ = slots[i][0][:3]
            dc = ab.adapt_measure_dispatch(plans[i], a, b, c_, stream, 20000 if cases[i].bytes < 4e6 else 2000)
            dispatch[kind] = dict(dc.as_dict(), shape=[cases[i].M, cases[i].N, cases[i].K])

    # ---- vendor-library reference (context, not the product): torch.matmul on the same buffers ----
    vendor = None
    if args.vendor and per_shape is not None:
        def views(c, slot):
            _, _, _, oa, ob, oc = slot
            pool = pools[c.dtype]
            A_ = pool[oa // 2: oa // 2 + c.M * c.K].view(c.M, c.K)
            B_ = pool[ob // 2: ob // 2 + c.K * c.N].view(c.K, c.N)
            C_ = out_pool[oc: oc + 2 * c.M * c.N].view(pool.dtype).view(c.M, c.N)
            return A_, B_, C_
        vendor = []
        reps_v = [int(min(20, max(1, 60.0 / max(t * 1e6, 1.0)))) for t in per_shape]
        evs = []
        for c, s, r in zip(cases, slots, reps_v):
            vs = [views(c, sl) for sl in s]
            torch.matmul(vs[0][0], vs[0][1], out=vs[0][2])
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for j in range(r):
                A_, B_, C_ = vs[j % len(vs)]
                torch.matmul(A_, B_, out=C_)
            e1.record()
            evs.append((e0, e1, r))
        torch.cuda.synchronize()
        vendor = [e0.elapsed_time(e1) * 1e-3 / r for e0, e1, r in evs]

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16/fp16 inputs, fp32 accumulate", "data": "synthetic",
        "config": {"workload": workload, "shapes": len(cases), "parallelism": f"replicas x{world} (no collective)",
                   "l2": "ring of resident operands (2 x %.0f GiB in, %.0f GiB out), far larger than L2, no reuse between consecutive calls"
                         % (args.pool_gb, out_bytes / gib),
                   "timing": "CUDA events on the launching stream around K passes; per-shape: events around R back-to-back calls with rotated buffers, median of passes",
                   "batch": "each pass is one adapt_matmul_batch call; the library spreads its calls over %s internal stream(s) between a fork from and a join to the launching stream and orders calls whose buffers overlap" % (args.batch_streams or 4)},
        "clocks": clocks, "gpu_launches": int(launches), "host_wall_ms_per_step": wall / args.steps * 1e3,
        "plan_ms_cold_total": plan_ms,
        "pointer_policy": {"operand_sets_per_shape_max": n_rot, "map_cache_slots_per_plan": 8,
                           "tensor_maps_encoded_in_timed_regions": int(map_encodes_timed),
                           "note": "headline pass p uses set p mod n of every shape, the per-shape pass rotates the same sets; all sets fit the per-plan tensor-map cache, so no timed call encodes a map; the cost of a miss is in dispatch_cost"},
    }
    if floor is not None:
        line["launch_floor"] = floor
        line["dispatch_cost"] = dispatch

    if rank == 0 and per_shape is not None:
        fr_nom, fr_meas, tf = [], [], []
        fam_time = {}
        var_time, var_bytes, var_flops, var_n = {}, {}, {}, {}
        big = []
        for c, info, t in zip(cases, infos, per_shape):
            tr = t_roof_nominal(c)
            fr_nom.append(tr / t)
            fr_meas.append(max(c.flops / peaks["tensor_burst"], c.bytes / peaks["hbm"]) / t)
            tf.append(c.flops / t / 1e12)
            if tr >= 20e-6:
                big.append(tr / t)
            key = ab.FAMILY_NAMES[info.family]
            fam_time[key] = fam_time.get(key, 0.0) + t
            k2 = kernel_variant(ab, info)
            var_time[k2] = var_time.get(k2, 0.0) + t
            var_bytes[k2] = var_bytes.get(k2, 0.0) + c.bytes
            var_flops[k2] = var_flops.get(k2, 0.0) + c.flops
            var_n[k2] = var_n.get(k2, 0) + 1
        total_t = sum(per_shape)
        if vendor is not None:
            sp = [v / t for v, t in zip(vendor, per_shape)]
            bigsp = [v / t for v, t, c in zip(vendor, per_shape, cases) if t_roof_nominal(c) >= 20e-6]
            line["vendor_reference"] = {"library": "cuBLAS via torch.matmul (context, not the product)",
                                        "geomean_time_ratio_vendor_over_ours": geomean(sp),
                                        "geomean_time_ratio_troof_ge_20us": geomean(bigsp),
                                        "sum_vendor_time_ms": sum(vendor) * 1e3, "sum_our_time_ms": sum(per_shape) * 1e3}
        # the same fractions against roofline time + the launch floor (what a perfect kernel behind one launch
        # would reach), and by bucket of nominal roofline time
        floor_us = floor["empty_kernel_us_pdl"] if floor else None
        buckets = []
        edges = [0.0, 0.1e-6, 1e-6, 5e-6, 20e-6, 100e-6, float("inf")]
        for lo, hi in zip(edges[:-1], edges[1:]):
            idx = [i for i, c in enumerate(cases) if lo <= t_roof_nominal(c) < hi]
            if not idx:
                continue
            b = {"t_roof_us": [lo * 1e6, hi * 1e6 if hi != float("inf") else None], "shapes": len(idx),
                 "median_call_us": statistics.median(per_shape[i] for i in idx) * 1e6,
                 "geomean_frac_nominal": geomean([fr_nom[i] for i in idx]),
                 "sum_call_ms": sum(per_shape[i] for i in idx) * 1e3}
            if floor_us is not None:
                b["geomean_frac_vs_troof_plus_launch"] = geomean([(t_roof_nominal(cases[i]) + floor_us * 1e-6) / per_shape[i] for i in idx])
            if vendor is not None:
                b["geomean_time_ratio_vendor_over_ours"] = geomean([vendor[i] / per_shape[i] for i in idx])
            buckets.append(b)
        line["sweep"] = {
            "roofline_frac_geomean_vs_troof_plus_launch":
                geomean([(t_roof_nominal(c) + floor_us * 1e-6) / t for c, t in zip(cases, per_shape)]) if floor_us is not None else None,
            "roofline_frac_geomean_if_every_call_took_troof_plus_launch":
                geomean([t_roof_nominal(c) / (t_roof_nominal(c) + floor_us * 1e-6) for c in cases]) if floor_us is not None else None,
            "by_t_roof_bucket": buckets,
            "roofline_frac_geomean_nominal": geomean(fr_nom),
            "roofline_frac_geomean_measured_peaks": geomean(fr_meas),
            "roofline_frac_geomean_troof_ge_20us": geomean(big), "shapes_troof_ge_20us": len(big),
            "tflops_geomean": geomean(tf), "sum_shape_time_ms": total_t * 1e3,
            "sum_t_roof_nominal_ms": sum(t_roof_nominal(c) for c in cases) * 1e3,
            "time_share_by_family": {k: v / total_t for k, v in fam_time.items()},
            "time_share_by_kernel_variant": {k: v / total_t for k, v in sorted(var_time.items(), key=lambda kv: -kv[1])},
        }
        # Roofline of the dominant kernel: the kernel variant (family / tiling mode) with the largest share of
        # the pass.  achieved = sum of algorithmic bytes (or flops) of its calls / sum of their CUDA-event
        # times; a call's time includes the small prologue (re-pitch of the small operand) or reduce launch
        # where the variant has one, so the figure is a lower bound for the kernel itself.
        dom = max(var_time, key=lambda k: var_time[k])
        ratio = NCU_TRAFFIC_RATIO.get(dom)
        mem_t = var_bytes[dom] / peaks["hbm"]
        ten_t = var_flops[dom] / peaks["tensor_sustained"]
        common = {"kernel": dom, "share_of_pass": var_time[dom] / total_t,
                  "traffic": ratio * var_bytes[dom] / var_n[dom] if ratio else None,
                  "peak_source": peaks["source"], "launches": var_n[dom],
                  "avg_launch_us": var_time[dom] / var_n[dom] * 1e6}
        if mem_t >= ten_t:
            ach = var_bytes[dom] / var_time[dom] / 1e9
            line["roofline"] = dict(common, bound="hbm", achieved=ach, peak=peaks["hbm"] / 1e9, unit="GB/s",
                                    frac=ach / (peaks["hbm"] / 1e9), algorithmic_bytes_per_launch=var_bytes[dom] / var_n[dom])
        else:
            ach = var_flops[dom] / var_time[dom] / 1e12
            line["roofline"] = dict(common, bound="tensor", achieved=ach, peak=peaks["tensor_sustained"] / 1e12, unit="TFLOP/s",
                                    frac=ach / (peaks["tensor_sustained"] / 1e12),
                                    algorithmic_flops_per_launch=var_flops[dom] / var_n[dom])
        if args.dump:
            os.makedirs(os.path.dirname(os.path.abspath(args.dump)), exist_ok=True)
            with open(args.dump, "w") as f:
                f.write("index,M,N,K,dtype,family,class,BM,BN,stages,P_k,fused,streamk,srcA,srcB,pred_us,time_us,tflops,frac_nominal,t_roof_us,vendor_us\n")
                for i, (c, info, t) in enumerate(zip(cases, infos, per_shape)):
                    vu = f"{vendor[i] * 1e6:.3f}" if vendor is not None else ""
                    f.write(f"{i},{c.M},{c.N},{c.K},{c.dtype},{ab.FAMILY_NAMES[info.family]},{info.taxonomy_class},{info.BM},{info.BN},"
                            f"{info.stages},{info.P_k},{info.fused},{info.streamk},{info.srcA},{info.srcB},{info.predicted_us:.3f},{t * 1e6:.3f},"
                            f"{c.flops / t / 1e12:.4f},{t_roof_nominal(c) / t:.5f},{t_roof_nominal(c) * 1e6:.4f},{vu}\n")

    # ---- dispatch overhead of a cached plan (host clock, C call through ctypes) ----
    if rank == 0:
        f = lib.adapt_matmul_plan
        n = 0
        t0 = time.perf_counter()
        for _ in range(20):
            for c in cases[:500]:
                f(c.M, c.N, c.K, c.dtype, 0, 0)
                n += 1
        line["dispatch_us_cached_plan_via_ctypes"] = (time.perf_counter() - t0) / n * 1e6

    # ---- end to end: host buffers, copies inside the timed region, through adapt_matmul_host ----
    if not args.no_e2e:
        try:
            line["e2e"] = e2e(args, cases, plans, pools, stream, world, dist)
        except Exception as e:      # report, never fake
            line["e2e"] = {"value": None, "unit": "TFLOP/s", "error": repr(e)[:200]}

    # ---- the CPU oracle beside it (rank 0, N = 1 only) ----
    if rank == 0 and world == 1 and not args.no_cpu:
        sample, macs = oracle_sample(synth.config_sweep(), 1.5e11)
        one_pass_cpu, threads = run_oracle_sample(sample)
        dt = one_pass_cpu()
        line["cpu_baseline"] = {"value": 2.0 * macs / dt / 1e12, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                                "sample": f"{len(sample)} shapes of the sweep's oracle subset, {macs:.3g} MACs, {dt:.1f} s"}

    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def e2e(args, cases, plans, pools, stream, world, dist):
    import torch
    from paper_2608_10803_b200 import binding as ab
    avail = 64e9
    try:
        with open("/proc/meminfo") as f:
            for ln in f:
                if ln.startswith("MemAvailable"):
                    avail = float(ln.split()[1]) * 1024
    except Exception:
        pass
    # pinned host buffers: one for A, one for B, one for C, shared by every shape (each operand of a
    # kept shape must fit; shapes with a larger operand are left out and counted)
    cap_op = min(14e9, avail / (10.0 * max(1, world)))
    keep = [i for i, c in enumerate(cases) if 2.0 * max(c.M * c.K, c.K * c.N, c.M * c.N) <= cap_op]
    max_a = max(2 * cases[i].M * cases[i].K for i in keep)
    max_b = max(2 * cases[i].K * cases[i].N for i in keep)
    max_c = max(2 * cases[i].M * cases[i].N for i in keep)
    hA = torch.empty(max_a, dtype=torch.uint8).pin_memory()
    hB = torch.empty(max_b, dtype=torch.uint8).pin_memory()
    hC = torch.empty(max_c, dtype=torch.uint8).pin_memory()
    src = next(iter(pools.values())).view(torch.uint8)      # seeded fp16/bf16 bits already on the device
    hA.copy_(src[:max_a])
    hB.copy_(src[-max_b:])
    lib = ab.load()
    mh = lib.adapt_matmul_host
    order = sorted(keep, key=lambda i: -cases[i].bytes)

    def one_pass(idx):
        for i in idx:
            c = cases[i]
            st = mh(plans[i], hA.data_ptr(), hB.data_ptr(), hC.data_ptr(), stream)
            if st != 0:
                raise RuntimeError(lib.adapt_last_error_message().decode())
    one_pass(order[:6])            # grows the staging slots to their final sizes
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.e2e_steps):
        one_pass(order)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    ms = max_over_ranks(ms, dist, "cuda")
    fl = sum(cases[i].flops for i in keep)
    return {"value": replicas_value(fl * args.e2e_steps, world, ms * 1e-3) / 1e12, "unit": "TFLOP/s",
            "h2d_bytes_per_step": int(sum(2 * (cases[i].M * cases[i].K + cases[i].K * cases[i].N) for i in keep)),
            "d2h_bytes_per_step": int(sum(2 * cases[i].M * cases[i].N for i in keep)),
            "shapes": len(keep), "shapes_left_out": len(cases) - len(keep), "steps": args.e2e_steps, "ms_per_step": ms / args.e2e_steps,
            "api": "adapt_matmul_host (pinned host operands; H2D of A and B, kernels, D2H of C inside the timed region; calls issued largest shape first, the library pipelines copy-in, kernels and copy-out of consecutive calls)"}


def one_shape(args):
    """Time a single GEMM shape (used for profiler captures and quick checks): prints one line."""
    import torch
    from paper_2608_10803_b200 import binding as ab
    from paper_2608_10803_b200 import synth
    M, N, K, dt = (int(x) for x in args.shape.split(","))
    ab.adapt_init(0)
    A = synth.draw_operand(M, K, synth.U11, 1, dt, "cuda")
    B = synth.draw_operand(K, N, synth.U11, 2, dt, "cuda")
    C = torch.empty((M, N), dtype=A.dtype, device="cuda")
    if args.family >= 0:
        cands = [c for c in ab.adapt_plan_candidates(M, N, K, dt) if c.family == args.family]
        if args.bn:
            cands = [c for c in cands if c.BN == args.bn]
        if args.pk:
            cands = [c for c in cands if c.P_k == args.pk]
        if args.stages:
            cands = [c for c in cands if c.stages == args.stages]
        if args.src:
            cands = [c for c in cands if f"{c.srcA}{c.srcB}" == args.src]
        if args.fused >= 0:
            cands = [c for c in cands if c.fused == args.fused]
        if args.streamk >= 0:
            cands = [c for c in cands if c.streamk == args.streamk]
        plan = ab.adapt_matmul_plan_forced(M, N, K, dt, 0, 0, cands[0].tiling_key)
    else:
        plan = ab.adapt_matmul_plan(M, N, K, dt)
    info = ab.adapt_plan_info(plan)
    st = torch.cuda.current_stream().cuda_stream
    ab.adapt_matmul(plan, A.data_ptr(), B.data_ptr(), C.data_ptr(), st)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        ab.adapt_matmul(plan, A.data_ptr(), B.data_ptr(), C.data_ptr(), st)
    e1.record()
    torch.cuda.synchronize()
    ab.adapt_poll_device_status(st)
    t = e0.elapsed_time(e1) / args.reps * 1e-3
    byts = 2.0 * (M * K + K * N + M * N)
    line = (f"{M}x{N}x{K} dt{dt} {ab.FAMILY_NAMES[info.family]} {info.BM}x{info.BN} st{info.stages} P_k{info.P_k} "
            f"src{info.srcA}{info.srcB}{' fused' if info.fused else ''}{' stream-K' if info.streamk else ''}: {t * 1e6:.1f} us  {2.0 * M * N * K / t / 1e12:.1f} TFLOP/s  {byts / t / 1e9:.0f} GB/s  "
            f"predicted {info.predicted_us:.1f} us")
    if args.cublas:
        torch.matmul(A, B, out=C)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.reps):
            torch.matmul(A, B, out=C)
        e1.record()
        torch.cuda.synchronize()
        tc = e0.elapsed_time(e1) / args.reps * 1e-3
        line += f"  | torch.matmul (cuBLAS, vendor reference) {tc * 1e6:.1f} us {2.0 * M * N * K / tc / 1e12:.1f} TFLOP/s"
    print(line)
    return 0


def store_ceiling(args):
    """Write-only ceiling of the GEMM's store path: the epilogue's store pattern with nothing in front of it
    (TMA box stores, 3-d TMA stores, plain 32-byte stores), on a 0.8 GB and a 13 GB output."""
    import torch
    from paper_2608_10803_b200 import binding as ab
    ab.adapt_init(0)
    st = torch.cuda.current_stream().cuda_stream
    out = {"store_ceiling": []}
    for rows, cols in ((20000, 20032), (94851, 69952)):
        buf = torch.empty(rows * cols, dtype=torch.float16, device="cuda")
        gb = rows * cols * 2 / 1e9
        for mode, name in ((0, "tma_box_32x64"), (1, "tma_3d_32xtile"), (2, "st_global_v8")):
            for tile_cols in (192, 256):
                for order in (0, 1):
                    for hint in (False, True):
                        if mode == 2 and hint:
                            continue
                        us = ab.adapt_measure_store_rate(buf.data_ptr(), rows, cols, mode, tile_cols, order, hint, 3, st)
                        out["store_ceiling"].append({"rows": rows, "cols": cols, "GB": round(gb, 2), "mode": name, "tile_cols": tile_cols,
                                                     "order": "gemm_raster" if order == 0 else "row_block_major",
                                                     "evict_first": hint, "us": round(us, 1), "TBps": round(gb / us * 1e3, 3)})
        # context: the same bytes through cudaMemset-like torch fill
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        buf.fill_(1.0)
        e0.record()
        for _ in range(3):
            buf.fill_(1.0)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / 3 * 1e3
        out["store_ceiling"].append({"rows": rows, "cols": cols, "GB": round(gb, 2), "mode": "torch.fill_ (context)", "us": round(us, 1),
                                     "TBps": round(gb / us * 1e3, 3)})
        del buf
    print(json.dumps(out))
    return 0


def validate_model(args):
    """The paper's model check (Section 6.6): time every legal configuration of a shape, call the
    fastest the oracle configuration, and count how often the analytical model picked it."""
    import numpy as np
    import torch
    from paper_2608_10803_b200 import binding as ab
    from paper_2608_10803_b200 import synth
    ab.adapt_init(0)
    st = torch.cuda.current_stream().cuda_stream
    if args.validate_heldout:
        # a second shape set drawn with the sweep's recipe from another seed: no model constant was fitted on it
        cases = synth.sweep_like(args.validate_heldout, 4 * args.validate_model + 200)
        order = list(range(len(cases)))
    else:
        cases = synth.config_sweep()
        rng = np.random.default_rng(7)
        order = [int(i) for i in rng.permutation(len(cases))]
    picked = [i for i in order if args.validate_roof_us * 1e-6 <= t_roof_nominal(cases[i]) and cases[i].bytes < 3e9][: args.validate_model]
    cand_rows = []
    hits, exact, cut, regrets, rows = 0, 0, 0, [], []
    for i in picked:
        c = cases[i]
        A, B = synth.draw_case(c, "cuda")
        # the bench's pointer policy: up to eight operand sets (twice L2 in total), consecutive calls rotate through them,
        # so that a small problem is timed with its operands coming from HBM, as in the sweep pass
        n_sets = int(min(8, max(1, math.ceil(2 * L2_BYTES / c.bytes))))
        As, Bs = [A] + [A.clone() for _ in range(n_sets - 1)], [B] + [B.clone() for _ in range(n_sets - 1)]
        Cs = [torch.empty((c.M, c.N), dtype=A.dtype, device="cuda") for _ in range(n_sets)]
        pa, pb, pc = (ab.pointer_array([t.data_ptr() for t in ts]) for ts in (As, Bs, Cs))
        all_cands = ab.adapt_plan_candidates(c.M, c.N, c.K, c.dtype)
        cands = all_cands[:args.validate_cap]
        cut += int(len(all_cands) > len(cands))
        times = []
        for cand in cands:
            plan = ab.adapt_matmul_plan_forced(c.M, c.N, c.K, c.dtype, 0, 0, cand.tiling_key)
            ab.adapt_matmul_repeat(plan, pa, pb, pc, n_sets, st)        # every set once: its tensor maps are cached
            torch.cuda.synchronize()
            reps = int(min(16, max(2, 200.0 / max(cand.predicted_us, 1.0))))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ab.adapt_matmul_repeat(plan, pa, pb, pc, reps, st)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) / reps * 1e3)
        for cand, t in zip(cands, times):
            cand_rows.append((c.M, c.N, c.K, c.dtype, ab.FAMILY_NAMES[cand.family], cand.BN, cand.stages, cand.P_k, cand.cluster, cand.fused,
                              cand.streamk, cand.srcA, cand.srcB, cand.predicted_us, cand.t_pro_us, cand.t_main_us, cand.t_epi_us, t))
        best = int(np.argmin(times))
        hits += int(best == 0 or times[0] <= 1.02 * times[best])
        exact += int(best == 0)
        regrets.append(times[0] / times[best])
        rows.append((c.M, c.N, c.K, len(cands), times[0], times[best], cands[0].predicted_us))
        del A, B, As, Bs, Cs
    out = {"model_validation": {"shapes": len(picked), "set": f"held-out, seed {args.validate_heldout}" if args.validate_heldout else "sweep (the set the constants were fitted on)",
                                "min_t_roof_us": args.validate_roof_us,
                                "exact_hit_rate": exact / max(1, len(picked)),
                                "top1_hit_rate_within_2pct": hits / max(1, len(picked)),
                                "mean_regret": float(np.mean(regrets)), "p95_regret": float(np.percentile(regrets, 95)),
                                "max_regret": float(np.max(regrets)),
                                "geomean_regret": geomean(regrets),
                                "candidates_timed_per_shape_cap": args.validate_cap, "shapes_with_more_candidates_than_cap": cut,
                                "operands": "up to eight rotating operand sets per shape (twice L2 in total), as in the sweep pass",
                                "note": "regret = time of the model's pick / time of the fastest legal configuration; the paper reports 63.86 % exact hits on its own hardware"}}
    print(json.dumps(out))
    if args.dump_candidates:
        with open(args.dump_candidates, "w") as f:
            f.write("M,N,K,dtype,family,BN,stages,P_k,cluster,fused,streamk,srcA,srcB,pred_us,t_pro,t_main,t_epi,time_us\n")
            for r in cand_rows:
                f.write(",".join(f"{x:.3f}" if isinstance(x, float) else str(x) for x in r) + "\n")
    if args.dump:
        with open(args.dump, "w") as f:
            f.write("M,N,K,candidates,picked_us,best_us,predicted_us\n")
            for r in rows:
                f.write(",".join(f"{x:.3f}" if isinstance(x, float) else str(x) for x in r) + "\n")
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="sweep", choices=["sweep", "configs"])
    ap.add_argument("--pool-gb", type=float, default=24.0, help="input pool per dtype, GiB")
    ap.add_argument("--shape-passes", type=int, default=3)
    ap.add_argument("--batch-streams", type=int, default=0, help="1: the batch entry runs its calls one after the other (library default: four internal streams)")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--limit", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-dispatch", action="store_true", help="skip the launch-floor and dispatch-cost measurements")
    ap.add_argument("--dump", default="", help="write the per-shape table to this CSV")
    ap.add_argument("--vendor", action="store_true", help="also time torch.matmul (cuBLAS) per shape as a vendor reference")
    ap.add_argument("--validate-model", type=int, default=0,
                    help="time every legal configuration of this many seeded sweep shapes and report how often the model's pick is the fastest")
    ap.add_argument("--validate-heldout", type=int, default=0, help="with --validate-model: draw the shapes with the sweep's recipe from this seed instead of from the sweep")
    ap.add_argument("--validate-cap", type=int, default=128, help="with --validate-model: time at most this many candidates per shape (best predicted first)")
    ap.add_argument("--validate-roof-us", type=float, default=5.0, help="with --validate-model: only shapes whose nominal roofline time is at least this")
    ap.add_argument("--dump-candidates", default="", help="with --validate-model: write every timed configuration (prediction and time) to this CSV")
    ap.add_argument("--ref-macs", type=float, default=5e10, help="with --impl reference: multiply-accumulates of the oracle's bounded sample per step")
    ap.add_argument("--shape", default="", help="M,N,K,dtype: time this one shape only (dtype 0 = fp16, 1 = bf16)")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--family", type=int, default=-1, help="with --shape: force a kernel family (0 umma_1cta, 1 umma_2cta, 2 skinny, 3 simt, 4 cluster)")
    ap.add_argument("--bn", type=int, default=0)
    ap.add_argument("--pk", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--src", type=str, default="", help="with --family: operand sources as two digits, e.g. 13 = A copied, B through k-class views")
    ap.add_argument("--streamk", type=int, default=-1, help="with --family: 1 = only stream-K configurations, 0 = none of them")
    ap.add_argument("--fused", type=int, default=-1, help="with --family: 1 = only fused split-K configurations, 0 = only unfused")
    ap.add_argument("--store-ceiling", action="store_true", help="measure the write-only ceiling of the store path (0.8 GB and 13 GB outputs)")
    ap.add_argument("--cublas", action="store_true", help="with --shape: also time torch.matmul as the vendor reference")
    args = ap.parse_args()
    if args.shape:
        return one_shape(args)
    if args.store_ceiling:
        return store_ceiling(args)
    if args.validate_model:
        return validate_model(args)
    if args.impl == "reference":
        return reference_arm(args)
    return ours(args)


if __name__ == "__main__":
    sys.exit(main())
