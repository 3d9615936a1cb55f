"""Shared helpers for the GPU parity tests: run a workload batch through the C ABI and compare
with the oracle, free-running (end to end) and in lock-step (every materialised tensor, with the
oracle fed the GPU's own inputs to that operator)."""
from __future__ import annotations

import numpy as np

from oracle import interp as O
from paper_2403_00176_b200 import binding as B
from paper_2403_00176_b200.session import Session

BAND = 2.0 ** -40


def run_batch(wl, reqs, opt_flags=0):
    s = Session(wl, opt_flags=opt_flags)
    p = s.prepare(reqs)
    p.run()
    p.check_device_status()
    return s, p, p.outputs()


def materialised(sess, prep, graph):
    names = []
    for nd in graph.nodes:
        for o in nd.outs:
            try:
                prep.plan.slot(o)
            except B.Sod2Error:
                continue
            if 4 in sess.graph.tensor_info(o)[1]:
                continue        # execution-determined extent: the arena slot is sized for the upper bound
            names.append(o)
    return names


def lockstep(wl, sess, prep, outs, r, float_tol, index_names=()):
    """Returns (max per-tensor error, per-tensor dict). Index tensors must match bit-exactly unless
    the deciding scores are within the 2^-40 band."""
    g = O.parse(wl.ir)
    names = materialised(sess, prep, g)
    over = {n: prep.read_arena_tensor(n, r).astype(np.float64) for n in names}
    for n, v in outs[r].items():
        over[n] = v.astype(np.float64) if v.dtype != np.int64 else v
    computed = {}
    O.run(wl.ir, wl.consts, prep.reqs[r].inputs, overrides=over, g=g, computed=computed)
    errs = {}
    for n, ref in computed.items():
        got = over[n]
        assert got.shape == np.shape(ref), (n, got.shape, np.shape(ref))
        if n in index_names or np.asarray(ref).dtype == np.int64:
            if not np.array_equal(got, ref):
                errs[n] = ("index", got, ref)
            continue
        errs[n] = O.rel_err(got, ref)
    return errs
