"""Per-config measurement (all five workloads): latency, per-group roofline fractions, planning
overhead and arena size.  Prints one JSON object per config and a markdown table.  Measurement only:
every device number comes from CUDA events, and nothing here touches the CPU oracle (bench.py times
that, in its cpu_baseline leg).  bench.py calls measure() for the per-config records of its line.

    python report.py [--configs 1,2,3,4,5] [--reps 30]
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time
from typing import Dict, List

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def group_times(prep, reps: int = 5, repeat: int = 1) -> List[float]:
    """Median device time (ms) of every fused group over `reps` timed inferences.  repeat > 1: every launch issued
    `repeat` times back to back between its events (duration inside a busy stream, see sod2_run_timed_repeat)."""
    ins = [t.data_ptr() for t in prep.in_dev]
    outs = [t.data_ptr() for t in prep.out_dev]
    runs = [prep.plan.run_timed(ins, outs, prep.arena.data_ptr(), prep.arena.numel(), prep.s.stream, repeat) for _ in range(reps)]
    return [float(np.median([r[g] for r in runs])) for g in range(len(runs[0]))]


def group_report(prep, hbm_gbs: float, tensor_tflops: float, reps: int = 5, repeat: int = 1) -> List[Dict]:
    """Per group: kind, ms, algorithmic flops / bytes, roofline time and fraction."""
    g = prep.s.graph
    ms = group_times(prep, reps, repeat)
    out = []
    for gi in range(g.num_groups()):
        info = g.group_info(gi)
        flops, nbytes = prep.plan.group_cost(gi)
        t_hbm = nbytes / (hbm_gbs * 1e9) * 1e3
        t_tc = flops / (tensor_tflops * 1e12) * 1e3
        t_roof = max(t_hbm, t_tc)
        out.append({"group": gi, "kind": info["kind"], "n_ops": info["n_ops"], "ms": ms[gi], "flops": flops, "bytes": nbytes,
                    "bound": "tensor" if t_tc >= t_hbm else "hbm", "t_roof_ms": t_roof, "frac": t_roof / ms[gi] if ms[gi] > 0 else 0.0})
    return out


def kind_summary(report: List[Dict]) -> Dict[str, Dict]:
    agg: Dict[str, Dict] = {}
    for r in report:
        a = agg.setdefault(r["kind"], {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "t_roof_ms": 0.0, "launch_groups": 0})
        for k in ("ms", "flops", "bytes", "t_roof_ms"):
            a[k] += r[k]
        a["launch_groups"] += 1
    for a in agg.values():
        a["tflops"] = a["flops"] / (a["ms"] * 1e-3) / 1e12 if a["ms"] > 0 else 0.0
        a["gbs"] = a["bytes"] / (a["ms"] * 1e-3) / 1e9 if a["ms"] > 0 else 0.0
        a["frac"] = a["t_roof_ms"] / a["ms"] if a["ms"] > 0 else 0.0
    return agg


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


def measure(cfg: int, reps: int, device: str = "cuda:0", opt_flags: int = 0):
    import torch
    from paper_2403_00176_b200 import workloads as WL
    from paper_2403_00176_b200.session import Session

    hbm, tf, src = _peaks()
    wl = {1: WL.cfg1, 2: WL.cfg2, 3: WL.cfg3, 4: WL.cfg4, 5: WL.cfg5}[cfg]()
    sess = Session(wl, device=device, opt_flags=opt_flags)
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
    if cfg == 5:
        # execution-determined extents handled exactly (counts read back, the rest planned again at the true sizes)
        # beside the default bounded form: wall time of the call (it synchronises the stream at every stage)
        for p in preps:
            p.run_exact()
        torch.cuda.synchronize(dev)
        ex = []
        for i in range(max(5, reps // 2)):
            flush.fill_(i & 0xFF)
            torch.cuda.synchronize(dev)
            p = preps[i % len(preps)]
            t0 = time.perf_counter()
            info = p.run_exact()
            torch.cuda.synchronize(dev)
            ex.append(((time.perf_counter() - t0) * 1e3, info.reserved[2], info.reserved[3], info.reserved[4] / 1e6))
        extra = {"exact_edo": {"ms_wall": float(np.median([e[0] for e in ex])), "stages": int(ex[0][1]),
                               "arena_bytes": int(np.median([e[2] for e in ex])), "bind_plan_ms": float(np.median([e[3] for e in ex])),
                               "bounded_arena_bytes": int(preps[0].plan.arena_bytes)}}
    # per-group roofline on the first batch
    rep = group_report(preps[0], hbm, tf, reps=5)
    kinds = kind_summary(rep)
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
    # end to end through the public API with host buffers: H2D (pinned) + bind + plan + run + D2H (pinned)
    pin_in = [[torch.from_numpy(h).pin_memory() for h in p.in_host] for p in preps]
    pin_out = [[torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in p.out_dev] for p in preps]
    e2e = []
    for i in range(2 * len(preps) + 1):
        k = i % len(preps)
        pr = preps[k]
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        for dst, src_ in zip(pr.in_dev, pin_in[k]):
            dst.copy_(src_, non_blocking=True)
        b = sess.graph.bind_dims(wl.sym_names, [[r.syms[s] for s in wl.sym_names] for r in pr.reqs])
        pl = b.plan()
        pl.run([t.data_ptr() for t in pr.in_dev], [t.data_ptr() for t in pr.out_dev], pr.arena.data_ptr(), pr.arena.numel(), sess.stream)
        for dst, src_ in zip(pin_out[k], pr.out_dev):
            dst.copy_(src_, non_blocking=True)
        torch.cuda.synchronize(dev)
        if i > 0:
            e2e.append((time.perf_counter() - t0) * 1e3)
        del pl, b
    mem = preps[0].plan.memory()
    reqs0 = preps[0].reqs
    units, uname = _units(cfg, reqs0)
    n_req = len(reqs0) if cfg != 5 else reqs0[0].inputs["x"].shape[0]
    return {
        "cfg": cfg, "workload": wl.name, "ms_median": float(np.median(times)), "ms_min": float(np.min(times)),
        "ms_graph_median": float(np.median(gtimes)), "ms_graph_min": float(np.min(gtimes)),
        "e2e_ms": float(np.median(e2e)), "h2d_bytes": int(sum(t.numel() for t in pin_in[0])), "d2h_bytes": int(sum(t.numel() for t in pin_out[0])),
        "ms_per_request": float(np.median(times)) / n_req, "units_batch0": units, "unit": uname,
        "sum_t_roof_over_sum_t_groups": sum_roof / sum_ms, "sum_t_roof_over_t_step": sum_roof / float(np.median(times)),
        "worst_group": {"kind": worst["kind"], "frac": worst["frac"], "bound": worst["bound"], "ms": worst["ms"]},
        "kinds": {k: {"ms": round(v["ms"], 4), "frac": round(v["frac"], 3), "tflops": round(v["tflops"], 1), "gbs": round(v["gbs"], 1)} for k, v in kinds.items()},
        "plan_us_median": float(np.median(plan_us)), "plan_us_cache_hit": float(np.median(hit_us)) if hit_us else None, "arena_bytes": mem["arena_bytes"], "peak_live_bytes": mem["peak_live_bytes"],
        "sum_tensor_bytes": mem["sum_bytes"], "n_groups": sess.graph.num_groups(), "n_ops": sess.graph.num_ops(),
        "gpu_launches": int(preps[0].run().gpu_launches), "peaks": src,
        "group_times": "CUDA events around every launch (no overlap between dependent kernels, no graph): the groups sum to more than ms_median",
        **extra,
    }


def chain_case(spec: str, reps: int = 20, device: str = "cuda:0"):
    """The paper's fusion example (Fig. 4: Sigmoid(A[I,1,1]) + B[I,J,K], one fused group) at a given size:
    spec = "I,J,K,dtype,n_requests".  Device time of the whole inference (one launch) against the HBM roofline of its
    algorithmic bytes (B in, C out; A is I values)."""
    import torch
    from paper_2403_00176_b200 import workloads as WL
    from paper_2403_00176_b200.session import Session
    from paper_2403_00176_b200.workloads import Request, bf16_round
    i, j, k, dt, n = spec.split(",")
    i, j, k, n = int(i), int(j), int(k), int(n)
    hbm, _, src = _peaks()
    wl = WL.fig4_chain(dt)
    rng = np.random.default_rng(0)
    rnd = (lambda a: bf16_round(a.astype(np.float32))) if dt == "bf16" else (lambda a: a.astype(np.float32))
    reqs = [Request({"I": i, "J": j, "K": k}, {"A": rnd(rng.standard_normal((i, 1, 1))), "B": rnd(rng.standard_normal((i, j, k)))}) for _ in range(n)]
    sess = Session(wl, device=device)
    p = sess.prepare(reqs)
    p.run()
    torch.cuda.synchronize(sess.dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=sess.dev)
    stream = torch.cuda.current_stream(sess.dev)
    lone = []
    for it in range(reps):
        flush.fill_(it & 0xFF)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        p.run()
        e1.record(stream)
        torch.cuda.synchronize(sess.dev)
        lone.append(e0.elapsed_time(e1))
    b2b = group_times(p, reps=5, repeat=20)[0]
    _, nbytes = p.plan.group_cost(0)
    ms = float(np.median(lone))
    return {"case": spec, "launches": int(p.run().gpu_launches), "bytes": nbytes, "ms_lone_launch": ms, "gbs_lone_launch": nbytes / ms / 1e6,
            "ms_back_to_back": b2b, "gbs_back_to_back": nbytes / b2b / 1e6, "frac_of_hbm_back_to_back": nbytes / b2b / 1e6 / hbm, "peaks": src}


def gemm_sweep(spec: str, device: str = "cuda:0"):
    """Kernel time of one bias GEMM against K: spec = "M,N,K1:K2:...".  For the single-CTA kernel and for the CTA-pair
    kernel (SOD2_OPT_GEMM_PAIR, forced wherever it is eligible): device time of one launch with 20 launches back to back
    between the events.  The slope over K is the main loop's time per 64-wide k-stage; what is left at K -> 0 is the
    fixed part of the kernel (fill, epilogue, launch)."""
    import torch
    from paper_2403_00176_b200 import binding as B
    from paper_2403_00176_b200 import workloads as WL
    from paper_2403_00176_b200.session import Session
    from paper_2403_00176_b200.workloads import Request, bf16_round
    os.environ["SOD2_GEMM_PAIR_FORCE"] = "1"      # read once by the library, only under the flag
    m, n, ks = spec.split(",")
    m, n, ks = int(m), int(n), [int(x) for x in ks.split(":")]
    rng = np.random.default_rng(0)
    rows = []
    for name, flags in (("one CTA per tile", 0), ("CTA pair per tile", B.OPT_GEMM_PAIR)):
        us = []
        for k in ks:
            ir = (f"sym M 1 16384\ninput x bf16 [1,M,{k}]\nconst w bf16 [{k},{n}]\nconst b bf16 [{n}]\n"
                  "node MatMul x w -> y0\nnode Add y0 b -> y\noutput y\n")
            consts = {"w": bf16_round((rng.standard_normal((k, n)) * 0.02).astype(np.float32)), "b": bf16_round((rng.standard_normal(n) * 0.02).astype(np.float32))}
            req = Request({"M": m}, {"x": bf16_round(rng.standard_normal((1, m, k)).astype(np.float32))})
            wl = WL.Workload(f"gemm_{m}x{n}x{k}", "bf16", ir, consts, ["M"], ["y"], {"batch_fn": lambda j: [req]})
            sess = Session(wl, device=device, opt_flags=flags)
            p = sess.prepare([req])
            p.run()
            torch.cuda.synchronize(sess.dev)
            us.append(group_times(p, reps=7, repeat=20)[0] * 1e3)
        slope = (us[-1] - us[-2]) / ((ks[-1] - ks[-2]) / 64) if len(ks) > 1 else None
        rows.append({"kernel": name, "M": m, "N": n, "K": ks, "us": us, "us_per_k_stage_at_the_large_end": slope})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gemm-sweep", default=None, help="M,N,K1:K2:...: kernel time of one bias GEMM against K, single-CTA and CTA-pair kernel")
    ap.add_argument("--chain-case", default=None, help="I,J,K,dtype,n_requests: time the Fig. 4 fused chain at this size instead of the configs")
    ap.add_argument("--configs", default="1,2,3,4,5")
    ap.add_argument("--reps", type=int, default=30)
    ap.add_argument("--opt-flags", type=int, default=0, help="SOD2_OPT_* bits for sod2_graph_create (A/B measurements)")
    a = ap.parse_args()
    if a.chain_case:
        print(json.dumps(chain_case(a.chain_case)))
        return
    if a.gemm_sweep:
        for r in gemm_sweep(a.gemm_sweep):
            print(json.dumps(r))
        return
    rows = []
    for c in [int(x) for x in a.configs.split(",")]:
        r = measure(c, a.reps, opt_flags=a.opt_flags)
        print(json.dumps(r), flush=True)
        rows.append(r)
    print("\n| cfg | ms per inference (median, min) | as one CUDA graph (median, min) | ms per request | sum t_roof / t_step | worst group: fraction, bound | bind+plan us (cache hit) | arena / peak-live MB |")
    print("|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['cfg']} | {r['ms_median']:.3f}, {r['ms_min']:.3f} | {r['ms_graph_median']:.3f}, {r['ms_graph_min']:.3f} | {r['ms_per_request']:.4f} | {r['sum_t_roof_over_t_step']:.3f} | "
              f"{r['worst_group']['kind']}: {r['worst_group']['frac']:.3f}, {r['worst_group']['bound']} | {r['plan_us_median']:.0f} ({r['plan_us_cache_hit'] or 0:.0f}) | "
              f"{r['arena_bytes'] / 1e6:.1f} / {r['peak_live_bytes'] / 1e6:.1f} |")
    for r in rows:
        if "ratio_to_empty_kernel" in r:
            print(f"\ncfg {r['cfg']} is launch-bound: one request per inference {r['ms_one_request_per_inference'] * 1e3:.2f} us, "
                  f"a kernel that does nothing {r['ms_empty_kernel'] * 1e3:.2f} us (ratio {r['ratio_to_empty_kernel']:.2f}); "
                  f"the {r['units_batch0']} rows of all requests as one packed launch {r['ms_median'] * 1e3:.2f} us. "
                  "A roofline fraction says nothing at this size.")


if __name__ == "__main__":
    main()
