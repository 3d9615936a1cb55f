"""Per-group device timing against the algorithmic roofline of a planned batch (measurement only;
every number here comes from CUDA events recorded by the library on the caller's stream)."""
from __future__ import annotations

from typing import Dict, List

import numpy as np


def group_times(prep, reps: int = 5) -> List[float]:
    """Median device time (ms) of every fused group over `reps` timed inferences."""
    ins = [t.data_ptr() for t in prep.in_dev]
    outs = [t.data_ptr() for t in prep.out_dev]
    runs = [prep.plan.run_timed(ins, outs, prep.arena.data_ptr(), prep.arena.numel(), prep.s.stream) for _ in range(reps)]
    return [float(np.median([r[g] for r in runs])) for g in range(len(runs[0]))]


def group_report(prep, hbm_gbs: float, tensor_tflops: float, reps: int = 5) -> List[Dict]:
    """Per group: kind, ms, algorithmic flops / bytes, roofline time and fraction."""
    g = prep.s.graph
    ms = group_times(prep, reps)
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
