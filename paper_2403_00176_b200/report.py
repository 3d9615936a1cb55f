"""Per-config measurement report (all five workloads): latency, per-group roofline fractions, planning
overhead, arena size, and the oracle timed on the host cores.  Prints one JSON object per config and a
markdown table.  Measurement only: every device number comes from CUDA events.

    python -m paper_2403_00176_b200.report [--configs 1,2,3,4,5] [--reps 30] [--oracle-budget 10]
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return d["hbm_gbs"], d["bf16_tflops_sustained"], "measured"
    return 6650.0, 1400.0, "fallback"


def _units(cfg, reqs):
    if cfg == 1:
        return sum(2 * r.syms["N"] for r in reqs), "rows"
    if cfg == 2:
        return sum(r.syms["L"] for r in reqs), "tokens"
    if cfg == 3:
        return sum(r.syms["N0"] for r in reqs), "input tokens"
    if cfg == 4:
        return sum(r.syms["H"] * r.syms["W"] for r in reqs), "pixels"
    return reqs[0].inputs["x"].shape[0], "images"


def measure(cfg: int, reps: int, oracle_budget: float):
    import torch
    from oracle import interp as O
    from paper_2403_00176_b200 import profile as PF
    from paper_2403_00176_b200 import workloads as WL
    from paper_2403_00176_b200.session import Session

    hbm, tf, src = _peaks()
    wl = {1: WL.cfg1, 2: WL.cfg2, 3: WL.cfg3, 4: WL.cfg4, 5: WL.cfg5}[cfg]()
    sess = Session(wl)
    n_batches = 3 if cfg in (4, 5) else 5
    preps = [sess.prepare(wl.batch(j)) for j in range(n_batches)]
    dev = sess.dev
    stream = torch.cuda.current_stream(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for p in preps:
        p.run()
    torch.cuda.synchronize(dev)
    preps[0].check_device_status()
    times = []
    for i in range(reps):
        flush.fill_(i & 0xFF)
        p = preps[i % len(preps)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        p.run()
        e1.record(stream)
        torch.cuda.synchronize(dev)
        times.append(e0.elapsed_time(e1))
    # the same batches, each replayed as one CUDA graph (captured beforehand)
    for p in preps:
        p.run_graph()
    torch.cuda.synchronize(dev)
    gtimes = []
    for i in range(reps):
        flush.fill_(i & 0xFF)
        p = preps[i % len(preps)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        p.run_graph()
        e1.record(stream)
        torch.cuda.synchronize(dev)
        gtimes.append(e0.elapsed_time(e1))
    extra = {}
    if cfg == 1:
        # launch-bound: one request per inference (its own plan, one launch), against a kernel that does nothing
        from paper_2403_00176_b200 import binding as B

        def timed(fn, n):
            ts = []
            for i in range(n):
                flush.fill_(i & 0xFF)      # also keeps the GPU busy while the host enqueues: device time, not enqueue time
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn()
                e1.record(stream)
                torch.cuda.synchronize(dev)
                ts.append(e0.elapsed_time(e1))
            return float(np.median(ts))

        singles = [sess.prepare([r]) for r in wl.batch(0)]
        for p1 in singles:
            p1.run()
        B.sod2_launch_empty(sess.stream)
        torch.cuda.synchronize(dev)
        single_ms = float(np.median([timed(p1.run, 10) for p1 in singles]))
        empty_ms = timed(lambda: B.sod2_launch_empty(sess.stream), 50)
        extra = {"ms_one_request_per_inference": single_ms, "ms_empty_kernel": empty_ms, "ratio_to_empty_kernel": single_ms / empty_ms}
    # per-group roofline on the first batch
    rep = PF.group_report(preps[0], hbm, tf, reps=5)
    kinds = PF.kind_summary(rep)
    sum_ms = sum(r["ms"] for r in rep)
    sum_roof = sum(r["t_roof_ms"] for r in rep)
    # worst group among those that matter (at least 1 % of the time of all groups)
    worst = min((r for r in rep if r["t_roof_ms"] > 0 and r["ms"] >= 0.01 * sum_ms), key=lambda r: r["frac"])
    # planning overhead
    plan_us = []
    for i in range(5):
        reqs = preps[i % len(preps)].reqs
        t0 = time.perf_counter()
        b = sess.graph.bind_dims(wl.sym_names, [[r.syms[s] for s in wl.sym_names] for r in reqs])
        pl = b.plan()
        plan_us.append((time.perf_counter() - t0) * 1e6)
        del pl, b
    # the same through the plan cache, every bound symbol tuple seen before
    sess.graph.set_plan_cache(len(preps) + 1)
    hit_us = []
    for i in range(2 * len(preps) + 3):
        reqs = preps[i % len(preps)].reqs
        t0 = time.perf_counter()
        _, _, hit = sess.graph.plan_cached(wl.sym_names, [[r.syms[s] for s in wl.sym_names] for r in reqs])
        if hit:
            hit_us.append((time.perf_counter() - t0) * 1e6)
    sess.graph.set_plan_cache(0)
    mem = preps[0].plan.memory()
    # oracle on a bounded sample
    t0 = time.perf_counter()
    done = 0
    reqs0 = preps[0].reqs
    if cfg == 5:
        small = WL.cfg5(B=2)
        O.run(small.ir, small.consts, small.batch(0)[0].inputs)
        dt = time.perf_counter() - t0
        oracle_ms = dt * 1e3 * (32 / 2)
        sample = "2 of 32 images, scaled by images"
    else:
        order = sorted(range(len(reqs0)), key=lambda i: _units(cfg, [reqs0[i]])[0])
        for i in order:
            O.run(wl.ir, wl.consts, reqs0[i].inputs)
            done += _units(cfg, [reqs0[i]])[0]
            if time.perf_counter() - t0 > oracle_budget:
                break
        dt = time.perf_counter() - t0
        total = _units(cfg, reqs0)[0]
        oracle_ms = dt * 1e3 * total / done
        sample = f"{done} of {total} {_units(cfg, reqs0)[1]} of batch 0, scaled"
    units, uname = _units(cfg, reqs0)
    n_req = len(reqs0) if cfg != 5 else reqs0[0].inputs["x"].shape[0]
    return {
        "cfg": cfg, "workload": wl.name, "ms_median": float(np.median(times)), "ms_min": float(np.min(times)),
        "ms_graph_median": float(np.median(gtimes)), "ms_graph_min": float(np.min(gtimes)),
        "ms_per_request": float(np.median(times)) / n_req, "units_batch0": units, "unit": uname,
        "sum_t_roof_over_sum_t_groups": sum_roof / sum_ms, "sum_t_roof_over_t_step": sum_roof / float(np.median(times)),
        "worst_group": {"kind": worst["kind"], "frac": worst["frac"], "bound": worst["bound"], "ms": worst["ms"]},
        "kinds": {k: {"ms": round(v["ms"], 4), "frac": round(v["frac"], 3), "tflops": round(v["tflops"], 1), "gbs": round(v["gbs"], 1)} for k, v in kinds.items()},
        "plan_us_median": float(np.median(plan_us)), "plan_us_cache_hit": float(np.median(hit_us)) if hit_us else None, "arena_bytes": mem["arena_bytes"], "peak_live_bytes": mem["peak_live_bytes"],
        "sum_tensor_bytes": mem["sum_bytes"], "n_groups": sess.graph.num_groups(), "n_ops": sess.graph.num_ops(),
        "gpu_launches": preps[0].plan.run_timed and None,
        "oracle_ms": oracle_ms, "oracle_cores": os.cpu_count(), "oracle_sample": sample, "peaks": src,
        **extra,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4,5")
    ap.add_argument("--reps", type=int, default=30)
    ap.add_argument("--oracle-budget", type=float, default=10.0)
    a = ap.parse_args()
    rows = []
    for c in [int(x) for x in a.configs.split(",")]:
        r = measure(c, a.reps, a.oracle_budget)
        r.pop("gpu_launches", None)
        print(json.dumps(r), flush=True)
        rows.append(r)
    print("\n| cfg | ms per inference (median, min) | as one CUDA graph (median, min) | ms per request | sum t_roof / t_step | worst group: fraction, bound | bind+plan us (cache hit) | arena / peak-live MB | oracle ms (cores) |")
    print("|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['cfg']} | {r['ms_median']:.3f}, {r['ms_min']:.3f} | {r['ms_graph_median']:.3f}, {r['ms_graph_min']:.3f} | {r['ms_per_request']:.4f} | {r['sum_t_roof_over_t_step']:.3f} | "
              f"{r['worst_group']['kind']}: {r['worst_group']['frac']:.3f}, {r['worst_group']['bound']} | {r['plan_us_median']:.0f} ({r['plan_us_cache_hit'] or 0:.0f}) | "
              f"{r['arena_bytes'] / 1e6:.1f} / {r['peak_live_bytes'] / 1e6:.1f} | {r['oracle_ms']:.0f} ({r['oracle_cores']}) |")
    for r in rows:
        if "ratio_to_empty_kernel" in r:
            print(f"\ncfg {r['cfg']} is launch-bound: one request per inference {r['ms_one_request_per_inference'] * 1e3:.2f} us, "
                  f"a kernel that does nothing {r['ms_empty_kernel'] * 1e3:.2f} us (ratio {r['ratio_to_empty_kernel']:.2f}); "
                  f"the {r['units_batch0']} rows of all requests as one packed launch {r['ms_median'] * 1e3:.2f} us. "
                  "A roofline fraction says nothing at this size.")


if __name__ == "__main__":
    main()
