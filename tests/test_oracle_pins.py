"""Pins for the CPU oracle: every operator definition is checked against something other
than itself (hand loops, scipy, closed forms, invariants), so that a dropped term, a wrong
sign or index or a transposed operand fails here."""
import math

import numpy as np
import pytest
import scipy.signal

from oracle import interp as O
from paper_2403_00176_b200 import workloads as WL

rng = np.random.default_rng(7)


def test_matmul_vs_loops():
    a = rng.standard_normal((2, 3, 5))
    b = rng.standard_normal((5, 4))
    ref = np.zeros((2, 3, 4))
    for i in range(2):
        for m in range(3):
            for n in range(4):
                ref[i, m, n] = sum(a[i, m, k] * b[k, n] for k in range(5))
    assert np.allclose(O.op_matmul(a, b), ref, rtol=0, atol=1e-13)


def test_conv_vs_scipy_correlate():
    x = rng.standard_normal((1, 3, 7, 6))
    w = rng.standard_normal((4, 3, 3, 3))
    b = rng.standard_normal(4)
    got = O.op_conv(x, w, b, 1, 1)
    assert got.shape == (1, 4, 7, 6)
    for o in range(4):
        ref = sum(scipy.signal.correlate2d(np.pad(x[0, c], 1), w[o, c], mode="valid") for c in range(3)) + b[o]
        assert np.allclose(got[0, o], ref, atol=1e-12)


def test_conv_stride2_pad3_shape_and_values():
    x = rng.standard_normal((2, 2, 9, 11))
    w = rng.standard_normal((3, 2, 7, 7))
    got = O.op_conv(x, w, None, 2, 3)
    assert got.shape == (2, 3, (9 + 6 - 7) // 2 + 1, (11 + 6 - 7) // 2 + 1)
    for n in range(2):
        for o in range(3):
            full = sum(scipy.signal.correlate2d(np.pad(x[n, c], 3), w[o, c], mode="valid") for c in range(2))
            assert np.allclose(got[n, o], full[::2, ::2], atol=1e-12)


def test_conv_1x1_is_matmul_and_delta_is_shift():
    x = rng.standard_normal((1, 5, 4, 4))
    w = rng.standard_normal((6, 5, 1, 1))
    got = O.op_conv(x, w, None, 1, 0)
    ref = np.einsum("oc,chw->ohw", w[:, :, 0, 0], x[0])
    assert np.allclose(got[0], ref, atol=1e-13)
    d = np.zeros((5, 5, 3, 3))
    for c in range(5):
        d[c, c, 1, 2] = 1.0          # tap one to the right of the centre
    sh = O.op_conv(x, d, None, 1, 1)
    assert np.array_equal(sh[0, :, :, :-1], x[0, :, :, 1:]) and np.all(sh[0, :, :, -1] == 0)
    d = np.zeros((5, 5, 3, 3))
    for c in range(5):
        d[c, c, 1, 1] = 1.0
    assert np.array_equal(O.op_conv(x, d, None, 1, 1), x)


def test_gelu_values_and_identities():
    xs = np.array([-3.0, -1.0, -0.25, 0.0, 0.5, 1.0, 2.5])
    ref = np.array([0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in xs])
    assert np.allclose(O.op_gelu(xs), ref, atol=1e-15)
    assert O.op_gelu(np.array([0.0]))[0] == 0.0
    assert np.allclose(O.op_gelu(xs) - O.op_gelu(-xs), xs, atol=1e-15)
    # Gelu(1) = Phi(1) = 0.8413447460685429...
    assert abs(O.op_gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15


def test_layernorm_invariants():
    x = rng.standard_normal((3, 5, 64)) * 3 + 1.5
    y = O.op_layernorm(x, np.ones(64), np.zeros(64), -1, 1e-5)
    assert np.max(np.abs(y.mean(-1))) < 1e-12
    var = x.var(-1)
    assert np.allclose((y * y).mean(-1), var / (var + 1e-5), atol=1e-12)
    c = O.op_layernorm(np.full((2, 8), 3.25), np.ones(8), np.zeros(8), -1, 1e-5)
    assert np.all(c == 0)
    g, b = rng.standard_normal(64), rng.standard_normal(64)
    assert np.allclose(O.op_layernorm(x, g, b, -1, 1e-5), y * g + b, atol=1e-12)


def test_softmax_invariants():
    x = rng.standard_normal((4, 9)) * 5
    p = O.op_softmax(x, -1)
    assert np.all(p >= 0) and np.allclose(p.sum(-1), 1, atol=1e-14)
    assert np.allclose(O.op_softmax(x + 100.0, -1), p, atol=1e-13)
    assert np.allclose(p[:, 1] / p[:, 0], np.exp(x[:, 1] - x[:, 0]), rtol=1e-12)
    assert O.op_softmax(np.array([[2.0]]), -1)[0, 0] == 1.0


def test_sigmoid():
    assert O.op_sigmoid(np.array([0.0]))[0] == 0.5
    x = rng.standard_normal(10)
    assert np.allclose(O.op_sigmoid(x) + O.op_sigmoid(-x), 1.0, atol=1e-15)


def test_topk_keep_vs_stable_argsort():
    for n, k in [(10, 7), (5, 5), (33, 1), (20, 14)]:
        s = rng.integers(0, 6, size=(2, n)).astype(np.float64)   # many exact ties
        vals, idx = O.op_topk(s, k, -1, True, "index")
        for r in range(2):
            ref = np.sort(np.argsort(-s[r], kind="stable")[:k])
            assert np.array_equal(idx[r], ref)
            assert np.array_equal(vals[r], s[r][ref])
        _, idv = O.op_topk(s, k, -1, True, "value")
        for r in range(2):
            assert np.array_equal(idv[r], np.argsort(-s[r], kind="stable")[:k])
    s = np.full((1, 9), 2.0)
    assert np.array_equal(O.op_topk(s, 4, -1, True, "index")[1][0], np.arange(4))
    assert np.array_equal(O.op_topk(rng.standard_normal((1, 6)), 6, -1, True, "index")[1][0], np.arange(6))


def test_keep_count_formula_is_ceil():
    # K = (7N+9)//10 must equal ceil(0.7 N) for every N the workloads can reach
    for n in range(1, 2049):
        assert (7 * n + 9) // 10 == math.ceil(7 * n / 10) == -((-7 * n) // 10)


def test_nonzero_vs_numpy():
    x = rng.standard_normal((3, 4, 5))
    x[rng.uniform(size=x.shape) < 0.5] = 0
    assert np.array_equal(O.op_nonzero(x), np.array(np.nonzero(x)))
    assert O.op_nonzero(np.zeros((2, 3))).shape == (2, 0)
    assert O.op_nonzero(np.ones((2, 3))).shape == (2, 6)


def test_switch_combine_equals_masked_execute_all():
    # regrouped execution must equal "execute all paths, strip out invalid results"
    x = rng.standard_normal((6, 3, 4, 4))
    gate = np.array([1, 0, 0, 1, 1, 0]).reshape(6, 1)
    f = lambda t: np.maximum(t * 2.0 - 0.1, 0)
    xe, xs = O.op_switch(x, gate)
    assert xe.shape[0] == 3 and xs.shape[0] == 3
    y = O.op_combine(f(xe), xs, gate)
    ref = np.where(gate.reshape(6, 1, 1, 1).astype(bool), f(x), x)
    assert np.array_equal(y, ref)
    for gv in (np.zeros((6, 1)), np.ones((6, 1))):
        xe, xs = O.op_switch(x, gv)
        assert np.array_equal(O.op_combine(f(xe), xs, gv), f(x) if gv[0, 0] else x)


def test_fig4_chain_vs_loops():
    wl = WL.fig4_chain()
    req = wl.batch(0)[0]
    out = O.run(wl.ir, wl.consts, req.inputs)["C"]
    a, b = req.inputs["A"].astype(np.float64), req.inputs["B"].astype(np.float64)
    I, J, K = b.shape
    for i in range(I):
        for j in range(0, J, 3):
            for k in range(0, K, 5):
                assert abs(out[i, j, k] - (1 / (1 + math.exp(-a[i, 0, 0])) + b[i, j, k])) < 1e-15


def test_cfg1_graph_fused_formula():
    # the whole group written as one formula per row, in plain loops
    wl = WL.cfg1()
    req = wl.batch(0)[0]
    y = O.run(wl.ir, wl.consts, req.inputs)["Y"]
    x = req.inputs["X"].astype(np.float64)
    W, b = wl.consts["W"].astype(np.float64), wl.consts["bias"].astype(np.float64)
    assert y.shape == x.shape
    for bi in range(2):
        for n in range(0, x.shape[1], 7):
            t = [sum(x[bi, n, k] * W[k, j] for k in range(64)) + b[j] for j in range(64)]
            t = [0.5 * v * (1 + math.erf(v / math.sqrt(2))) + x[bi, n, j] for j, v in enumerate(t)]
            mu = sum(t) / 64
            var = sum((v - mu) ** 2 for v in t) / 64
            ref = [(v - mu) / math.sqrt(var + 1e-5) for v in t]
            assert np.allclose(y[bi, n], ref, atol=1e-12)


def test_tiny_encoder_attention_vs_loops():
    # attention through Slice/Reshape/Transpose equals per-head softmax(q k^T / sqrt(dh)) v
    wl = WL.cfg2(layers=1, D=16, H=2, F=32, n_requests=2, lmin=3, lmax=9)
    req = wl.batch(0)[0]
    env = O.run(wl.ir, wl.consts, req.inputs)
    L = req.syms["L"]
    x = req.inputs["x"].astype(np.float64)[0]
    qkv = x @ wl.consts["l0.Wqkv"].astype(np.float64) + wl.consts["l0.bqkv"].astype(np.float64)
    ctx = np.zeros((L, 16))
    for h in range(2):
        q = qkv[:, h * 8:(h + 1) * 8]
        k = qkv[:, 16 + h * 8:16 + (h + 1) * 8]
        v = qkv[:, 32 + h * 8:32 + (h + 1) * 8]
        for i in range(L):
            s = np.array([np.dot(q[i], k[j]) / math.sqrt(8) for j in range(L)])
            p = np.exp(s - s.max())
            p /= p.sum()
            ctx[i, h * 8:(h + 1) * 8] = sum(p[j] * v[j] for j in range(L))
    name = [n.outs[0] for n in O.parse(wl.ir).nodes if n.outs[0].startswith("ctx")][0]
    assert env[name].shape == (1, L, 16)
    assert np.allclose(env[name][0], ctx, atol=1e-13)
    assert env["y"].shape == (1, L, 16)


def test_tiny_pruning_shapes_and_indices():
    wl = WL.cfg3(layers=3, D=16, H=2, F=32, n_requests=2, nmin=5, nmax=20)
    req = wl.batch(1)[0]
    env = O.run(wl.ir, wl.consts, req.inputs)
    n = req.syms["N0"]
    for l in range(3):
        k = -((-7 * n) // 10)
        y = env[f"y{l}"][0]
        ref = np.sort(np.argsort(-(y * y).sum(-1), kind="stable")[:k])
        assert np.array_equal(env[f"idx{l}"][0], ref)
        assert np.array_equal(env[f"keep{l}"][0], y[ref])
        n = k


def test_tiny_gated_network_runs():
    wl = WL.cfg5(B=4, side=16, widths=(4, 8), per_stage=2)
    req = wl.batch(0)[0]
    env = O.run(wl.ir, wl.consts, req.inputs)
    assert env["gap"].shape == (4, 8, 1, 1)
    assert env["stem"].shape == (4, 4, 8, 8)
    # masked execute-all for block 0 equals the regrouped result
    x = env["stem"]
    g = env["gate0"].reshape(-1)
    w1, b1, w2, b2 = (wl.consts[f"b0.{k}"].astype(np.float64) for k in ("w1", "b1", "w2", "b2"))
    full = np.maximum(x + O.op_conv(np.maximum(O.op_conv(x, w1, b1, 1, 1), 0), w2, b2, 1, 1), 0)
    ref = np.where(g.reshape(-1, 1, 1, 1), full, x)
    assert np.allclose(env["blk0"], ref, atol=1e-12)


def test_rel_err_metric():
    a = np.array([1.0, -2.0, 0.0])
    assert O.rel_err(a, a) == 0
    assert O.rel_err(np.array([]), np.array([])) == 0
