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


# --------------------------------------------------------------------------- pins through tiny graphs
# Each test below writes a few lines of graph text, runs the interpreter and compares with literal
# arrays or explicit loops, so that every operator branch of the interpreter meets something that is
# not the interpreter (a wrong axis, sign, comparison direction or off-by-one fails here).
def _run(ir, inputs=None, consts=None):
    return O.run(ir, consts or {}, inputs or {})


def test_global_average_pool_vs_loops_non_square():
    x = rng.standard_normal((2, 3, 4, 7))          # H != W, N != C: a wrong axis pair changes shape or values
    env = _run("input x f32 [2,3,4,7]\nnode GlobalAveragePool x -> p\noutput p\n", {"x": x})
    assert env["p"].shape == (2, 3, 1, 1)
    for n in range(2):
        for c in range(3):
            s = 0.0
            for h in range(4):
                for w in range(7):
                    s += x[n, c, h, w]
            assert abs(env["p"][n, c, 0, 0] - s / 28.0) < 1e-14


def test_greater_is_strict_and_directed():
    a = np.array([[-1.0], [0.0], [0.5], [2.0]])
    env = _run("input a f32 [4,1]\nfconst z f32 [] = 0.0\nfconst one f32 [] = 1.0\n"
               "node Greater a z -> g0\nnode Greater z a -> g1\nnode Greater a one -> g2\n", {"a": a})
    assert env["g0"].reshape(-1).tolist() == [False, False, True, True]      # 0 > 0 is false
    assert env["g1"].reshape(-1).tolist() == [True, False, False, False]     # operands are not swapped
    assert env["g2"].reshape(-1).tolist() == [False, False, False, True]


def test_gate_chain_of_gated_block_vs_loops_with_exact_zero_logit():
    # the gate of a block: z_b = sum_c w_c * mean_hw x[b,c] + b0, gate_b = z_b > 0 (true = execute);
    # sample 1 is built so that z is exactly 0 and must be skipped
    wl = WL.cfg5(B=4, side=16, widths=(4, 8), per_stage=2, calibrated=False)
    g = O.parse(wl.ir)
    x = np.zeros((4, 4, 8, 8))
    x[0] = rng.integers(-4, 5, size=(4, 8, 8)) / 4.0
    x[1] = 0.0                                     # pooled features 0 -> z = bias
    x[2] = rng.integers(-4, 5, size=(4, 8, 8)) / 4.0 + 1.0
    x[3] = -x[2]
    gw = np.array([[0.5], [-1.0], [2.0], [0.25]])
    consts = dict(wl.consts)
    consts["b0.gw"] = gw
    consts["b0.gb"] = np.array([0.0])              # exact zero logit for sample 1
    env = O.run(wl.ir, consts, wl.batch(0)[0].inputs, overrides={"stem": x}, g=g)
    z = []
    for b in range(4):
        acc = 0.0
        for c in range(4):
            m = 0.0
            for h in range(8):
                for w in range(8):
                    m += x[b, c, h, w]
            acc += gw[c, 0] * (m / 64.0)
        z.append(acc + 0.0)
    assert z[1] == 0.0
    want = [bool(v > 0) for v in z]
    assert want[1] is False and any(want) and not all(want)
    assert env["gate0"].reshape(-1).astype(bool).tolist() == want
    assert np.allclose(env["logit0"].reshape(-1), z, atol=1e-14)
    # and the block output follows the decision sample by sample: skipped samples pass through unchanged
    for b in range(4):
        if not want[b]:
            assert np.array_equal(env["blk0"][b], x[b])
        else:
            assert not np.array_equal(env["blk0"][b], x[b])


def test_range_constant_of_shape_cast_literals():
    env = _run("iconst s i64 [] = 2\niconst e i64 [] = 11\niconst d i64 [] = 3\niconst dn i64 [] = -4\niconst shp i64 [2] = 2 3\n"
               "input f f32 [4]\n"
               "node Range s e d -> r\nnode Range e s dn -> rn\nnode ConstantOfShape shp -> c {value=1.5}\n"
               "node Cast f -> fi {to=i64}\nnode Cast r -> rf {to=f32}\n",
               {"f": np.array([1.9, -1.9, 0.0, 7.2])})
    assert env["r"].tolist() == [2, 5, 8] and env["r"].dtype == np.int64           # end is exclusive
    assert env["rn"].tolist() == [11, 7, 3]                                        # negative step counts down
    assert env["c"].shape == (2, 3) and np.all(env["c"] == 1.5)
    assert env["fi"].tolist() == [1, -1, 0, 7] and env["fi"].dtype == np.int64     # truncation toward zero
    assert env["rf"].dtype == np.float64 and env["rf"].tolist() == [2.0, 5.0, 8.0]


def test_float_div_sub_and_integer_div_literals():
    a = np.array([[6.0, -3.0], [1.0, 0.5]])
    b = np.array([4.0, 2.0])                      # broadcast over rows
    env = _run("input a f32 [2,2]\ninput b f32 [2]\niconst i i64 [3] = 7 -7 9\niconst j i64 [] = 2\n"
               "node Div a b -> q\nnode Sub a b -> d\nnode Sub b a -> e\nnode Div i j -> iq\nnode Mul a b -> m\nnode Add a b -> s\n",
               {"a": a, "b": b})
    assert env["q"].tolist() == [[1.5, -1.5], [0.25, 0.25]]
    assert env["d"].tolist() == [[2.0, -5.0], [-3.0, -1.5]]
    assert env["e"].tolist() == [[-2.0, 5.0], [3.0, 1.5]]                          # Sub is not commutative: operand order
    assert env["iq"].tolist() == [3, -4, 4] and env["iq"].dtype == np.int64        # integer Div floors
    assert env["m"].tolist() == [[24.0, -6.0], [4.0, 1.0]]
    assert env["s"].tolist() == [[10.0, -1.0], [5.0, 2.5]]


def test_reshape_zero_and_minus_one_rules():
    x = np.arange(24.0).reshape(2, 3, 4)
    env = _run("input x f32 [2,3,4]\niconst a i64 [3] = 0 -1 2\niconst b i64 [2] = -1 0\niconst c i64 [3] = 0 0 4\n"
               "node Reshape x a -> ra\nnode Reshape x b -> rb\nnode Reshape x c -> rc\n", {"x": x})
    assert env["ra"].shape == (2, 6, 2)            # 0 copies input dim 0, -1 takes the rest
    assert env["rb"].shape == (8, 3)               # 0 at position 1 copies input dim 1 (= 3)
    assert env["rc"].shape == (2, 3, 4)
    assert env["ra"].reshape(-1).tolist() == list(range(24))     # row-major order is kept
    assert env["ra"][1, 2, 1] == 17.0 and env["rb"][5, 1] == 16.0


def test_reduce_sum_square_relu_shape_transpose_concat_gather_slice_literals():
    x = np.array([[1.0, -2.0, 3.0], [0.5, 0.0, -1.0]])
    env = _run("input x f32 [2,3]\niconst ix i64 [2] = 2 0\niconst i0 i64 [1] = 1\n"
               "iconst st i64 [1] = 1\niconst en i64 [1] = 3\niconst ax i64 [1] = 1\n"
               "node ReduceSumSquare x -> q {axis=-1 keepdims=0}\nnode ReduceSumSquare x -> qk {axis=-1 keepdims=1}\n"
               "node Relu x -> r\nnode Shape x -> s\nnode Transpose x -> t {perm=1,0}\nnode Concat x x -> c {axis=0}\n"
               "node Concat x x -> c1 {axis=1}\nnode Gather x ix -> g {axis=1}\nnode Gather x i0 -> g0 {axis=0}\n"
               "node Slice x st en ax -> sl\n",
               {"x": x})
    assert env["q"].tolist() == [14.0, 1.25] and env["qk"].shape == (2, 1)         # squares, no square root
    assert env["r"].tolist() == [[1.0, 0.0, 3.0], [0.5, 0.0, 0.0]]
    assert env["s"].tolist() == [2, 3]
    assert env["t"].tolist() == [[1.0, 0.5], [-2.0, 0.0], [3.0, -1.0]]
    assert env["c"].shape == (4, 3) and env["c1"].shape == (2, 6) and env["c1"][1].tolist() == [0.5, 0.0, -1.0, 0.5, 0.0, -1.0]
    assert env["g"].tolist() == [[3.0, 1.0], [-1.0, 0.5]]                          # columns 2 and 0, in that order
    assert env["g0"].tolist() == [[0.5, 0.0, -1.0]]
    assert env["sl"].tolist() == [[-2.0, 3.0], [0.0, -1.0]]                        # columns 1..2


def test_sigmoid_values_and_softmax_axis():
    v = O.op_sigmoid(np.array([1.0, -2.0]))
    assert abs(v[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16 and abs(v[1] - 1.0 / (1.0 + math.exp(2.0))) < 1e-16
    x = rng.standard_normal((3, 4))
    env = _run("input x f32 [3,4]\nnode Softmax x -> p {axis=-1}\nnode Softmax x -> p0 {axis=0}\n", {"x": x})
    for i in range(3):
        den = sum(math.exp(x[i, j]) for j in range(4))
        for j in range(4):
            assert abs(env["p"][i, j] - math.exp(x[i, j]) / den) < 1e-14
    assert np.allclose(env["p0"].sum(0), 1.0, atol=1e-14) and not np.allclose(env["p0"].sum(1), 1.0)


def test_layernorm_values_vs_loops():
    x = rng.standard_normal((2, 5)) * 2 + 0.7
    g, b = rng.standard_normal(5), rng.standard_normal(5)
    y = O.op_layernorm(x, g, b, -1, 1e-3)
    for i in range(2):
        mu = sum(x[i]) / 5
        var = sum((v - mu) ** 2 for v in x[i]) / 5
        for j in range(5):
            assert abs(y[i, j] - ((x[i, j] - mu) / math.sqrt(var + 1e-3) * g[j] + b[j])) < 1e-13


def test_expand_literals():
    x = np.array([[1.0], [2.0], [3.0]])                       # [3,1]
    env = _run("input x f32 [3,1]\niconst s1 i64 [2] = 3 4\niconst s2 i64 [3] = 2 1 4\nnode Expand x s1 -> a\nnode Expand x s2 -> b\n", {"x": x})
    assert env["a"].tolist() == [[1.0] * 4, [2.0] * 4, [3.0] * 4]
    assert env["b"].shape == (2, 3, 4) and env["b"][1].tolist() == [[1.0] * 4, [2.0] * 4, [3.0] * 4]   # the 1 in the target keeps x's 3


def test_resize_nearest_vs_repeat_literal_and_torch():
    import torch
    import torch.nn.functional as F
    x = rng.standard_normal((2, 3, 4, 5))
    env = _run("input x f32 [2,3,4,5]\niconst sz i64 [4] = 2 3 6 3\nnode Resize x -> a {scales=1,1,2,3}\nnode Upsample x -> b {scales=1,2,1,1}\n"
               "node Resize x sz -> c\n", {"x": x})
    # integer scales repeat every element: numpy.repeat along each axis is the definition
    assert np.array_equal(env["a"], np.repeat(np.repeat(x, 2, axis=2), 3, axis=3))
    assert np.array_equal(env["b"], np.repeat(x, 2, axis=1))
    # fractional ratio 4 -> 6 rows and 5 -> 3 columns: source indices floor(o * in / out) written out by hand
    rows, cols = [0, 0, 1, 2, 2, 3], [0, 1, 3]
    for i, r_ in enumerate(rows):
        for j, c_ in enumerate(cols):
            assert np.array_equal(env["c"][:, :, i, j], x[:, :, r_, c_])
    # the library's nearest mode uses the same rule (source = floor(o * in / out))
    t = torch.from_numpy(x)
    assert np.array_equal(env["a"], F.interpolate(t, scale_factor=(2, 3), mode="nearest").numpy())
    assert np.array_equal(env["c"], F.interpolate(t, size=(6, 3), mode="nearest").numpy())
    # a 1-D literal
    e2 = _run("input v f32 [3]\nnode Resize v -> w {scales=2}\n", {"v": np.array([1.0, 2.0, 3.0])})
    assert e2["w"].tolist() == [1.0, 1.0, 2.0, 2.0, 3.0, 3.0]
