"""CPU oracle: a plain op-by-op interpreter of the operator semantics.  TEST INFRASTRUCTURE ONLY.

The method under test (rank-and-dimension propagation, fusion, planning) is a set of
optimisations that must reach exactly the result of naive unfused execution (the paper,
Section 4: all optimisations keep a deterministic sequence and a consistent output).  So
the oracle is that naive execution written out: one request at a time, one operator at a
time, every intermediate materialised as its own array with its concrete shape, no
fusion, no packing, no masks, no arena.  Floats are float64 throughout; integer tensors are
int64.  Shapes are whatever the arrays turn out to be ("brute-force shape inference"):
Section 3's OS <- F(IS...) for the shape-determined classes, and SHAPE_OF(OV) after
running the operator for the execution-determined class.

It shares no code with the CUDA path or its host library; it has its own reader for the
graph text.  Only tests, the smoke check and the bench's CPU-baseline leg may import it.

Pins (tests/test_oracle_pins.py): MatMul and Conv against hand loops and scipy's
correlate2d, 1x1 conv == MatMul, delta-kernel conv == shift; Gelu against math.erf and
the identity Gelu(x)-Gelu(-x)=x; LayerNorm and Softmax invariants; top-k keep against a
stable argsort; NonZero against numpy.nonzero; Switch/Combine against masked
execute-all; the Fig. 4 chain against explicit loops; GlobalAveragePool, the gate chain
(pool -> linear -> Greater, with a logit of exactly zero), LayerNorm and Softmax values against
loops; Greater, Range, ConstantOfShape, Cast, Div, Sub, Reshape's 0 / -1 rules, ReduceSumSquare,
Relu, Shape, Transpose, Concat, Gather, Slice and Expand against literal arrays; Resize / Upsample (nearest)
against numpy.repeat for integer scales, a literal array for a fractional ratio and
torch.nn.functional.interpolate.  Nothing here is
"parity unpinned" except the reading of tolerances and decision bands, which is a convention,
not a value.
"""
from __future__ import annotations

import math
import re
from typing import Dict, List, Optional

import numpy as np


# --------------------------------------------------------------------------- graph text reader
class Node:
    __slots__ = ("op", "ins", "outs", "attrs")

    def __init__(self, op, ins, outs, attrs):
        self.op, self.ins, self.outs, self.attrs = op, ins, outs, attrs


class Graph:
    def __init__(self):
        self.syms: List[str] = []
        self.inputs: Dict[str, tuple] = {}   # name -> (dtype, dims as str/int)
        self.consts: Dict[str, tuple] = {}
        self.inline: Dict[str, np.ndarray] = {}
        self.nodes: List[Node] = []
        self.outputs: List[str] = []


def _dims(txt: str):
    txt = txt.strip()[1:-1].strip()
    if not txt:
        return []
    out = []
    for d in txt.split(","):
        d = d.strip()
        out.append(int(d) if re.fullmatch(r"-?\d+", d) else d)
    return out


def parse(text: str) -> Graph:
    g = Graph()
    for raw in text.splitlines():
        line = raw.split("#")[0].strip()
        if not line:
            continue
        kw, rest = line.split(None, 1)
        if kw == "sym":
            g.syms.append(rest.split()[0])
        elif kw in ("input", "const"):
            m = re.fullmatch(r"(\S+)\s+(\S+)\s+(\[.*\])", rest)
            (g.inputs if kw == "input" else g.consts)[m.group(1)] = (m.group(2), _dims(m.group(3)))
        elif kw in ("iconst", "fconst"):
            m = re.fullmatch(r"(\S+)\s+(\S+)\s+(\[.*?\])\s*=\s*(.*)", rest)
            dims = _dims(m.group(3))
            vals = m.group(4).split()
            if kw == "iconst":
                a = np.array([int(v) for v in vals], dtype=np.int64)
            else:
                a = np.array([float(v) for v in vals], dtype=np.float64)
            g.inline[m.group(1)] = a.reshape(dims)
        elif kw == "node":
            attrs = {}
            m = re.search(r"\{(.*)\}", rest)
            if m:
                for kv in m.group(1).split():
                    k, v = kv.split("=", 1)
                    attrs[k] = v
                rest = rest[: m.start()].strip()
            lhs, rhs = rest.split("->")
            toks = lhs.split()
            g.nodes.append(Node(toks[0], toks[1:], rhs.split(), attrs))
        elif kw == "output":
            g.outputs.append(rest.strip())
        else:
            raise ValueError(f"bad statement: {raw}")
    return g


# --------------------------------------------------------------------------- operator definitions
def op_matmul(a, b):
    """Y[..,m,n] = sum_k A[..,m,k] * B[..,k,n], batch dims broadcast."""
    return np.matmul(a, b)


def op_gelu(x):
    """Gelu(x) = 0.5 x (1 + erf(x / sqrt 2))."""
    erf = np.vectorize(math.erf, otypes=[np.float64])
    return 0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))


def op_sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def op_softmax(x, axis):
    m = np.max(x, axis=axis, keepdims=True)
    e = np.exp(x - m)
    return e / np.sum(e, axis=axis, keepdims=True)


def op_layernorm(x, gamma, beta, axis, eps):
    """mu = mean, var = mean((x-mu)^2) (biased), y = (x-mu)/sqrt(var+eps)*gamma+beta over the last axes."""
    ax = tuple(range(axis % x.ndim, x.ndim))
    mu = np.mean(x, axis=ax, keepdims=True)
    var = np.mean((x - mu) ** 2, axis=ax, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * gamma + beta


def op_conv(x, w, b, stride, pad):
    """2-D cross-correlation, NCHW x OIHW, zero padding, out = floor((in + 2p - k)/s) + 1."""
    n, c, h, wd = x.shape
    o, ci, kh, kw = w.shape
    assert ci == c
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (wd + 2 * pad - kw) // stride + 1
    xp = np.zeros((n, c, h + 2 * pad, wd + 2 * pad), dtype=np.float64)
    xp[:, :, pad:pad + h, pad:pad + wd] = x
    y = np.zeros((n, o, ho, wo), dtype=np.float64)
    for ky in range(kh):
        for kx in range(kw):
            win = xp[:, :, ky:ky + stride * (ho - 1) + 1:stride, kx:kx + stride * (wo - 1) + 1:stride]
            # y[n,o,h,w] += sum_c w[o,c,ky,kx] * win[n,c,h,w]   (one matrix product per tap)
            y += np.moveaxis(np.tensordot(w[:, :, ky, kx], win, axes=(1, 1)), 0, 1)
    if b is not None:
        y += b.reshape(1, o, 1, 1)
    return y


def op_topk(score, k, axis, largest, order):
    """rank_i = #{j : s_j better than s_i} + #{j < i : s_j == s_i}; keep rank_i < k.
    order=index: kept positions ascending; order=value: by rank."""
    s = np.moveaxis(score, axis, -1)
    lead = s.shape[:-1]
    s2 = s.reshape(-1, s.shape[-1])
    n = s2.shape[1]
    vals = np.zeros((s2.shape[0], k), dtype=np.float64)
    idxs = np.zeros((s2.shape[0], k), dtype=np.int64)
    for r in range(s2.shape[0]):
        row = s2[r]
        better = (row[None, :] > row[:, None]) if largest else (row[None, :] < row[:, None])
        tie = (row[None, :] == row[:, None]) & (np.arange(n)[None, :] < np.arange(n)[:, None])
        rank = better.sum(axis=1) + tie.sum(axis=1)
        if order == "index":
            keep = [i for i in range(n) if rank[i] < k]
        else:
            keep = [0] * k
            for i in range(n):
                if rank[i] < k:
                    keep[rank[i]] = i
        idxs[r] = keep
        vals[r] = row[keep]
    shp = lead + (k,)
    return np.moveaxis(vals.reshape(shp), -1, axis), np.moveaxis(idxs.reshape(shp), -1, axis)


def op_nonzero(x):
    """int64 [rank, nnz]: coordinates of non-zero elements in row-major order."""
    coords = []
    for lin in range(x.size):
        c = np.unravel_index(lin, x.shape) if x.ndim else ()
        if x[c] != 0:
            coords.append(c)
    out = np.zeros((x.ndim, len(coords)), dtype=np.int64)
    for j, c in enumerate(coords):
        out[:, j] = c
    return out


def op_reshape(x, shape):
    shape = [int(v) for v in shape]
    for i, v in enumerate(shape):
        if v == 0:
            shape[i] = x.shape[i]
    return x.reshape(shape)


def op_slice(x, starts, ends, axes, steps):
    sl = [slice(None)] * x.ndim
    for i, ax in enumerate(axes):
        ax = int(ax) % x.ndim
        st = int(steps[i]) if steps is not None else 1
        sl[ax] = slice(int(starts[i]), int(ends[i]), st)
    return x[tuple(sl)]


def op_switch(x, gate):
    """Regroup samples by the gate: (samples with gate true, samples with gate false), each in sample order."""
    g = gate.reshape(-1).astype(bool)
    return x[g], x[~g]


def op_combine(y_true, y_false, gate):
    """Merge the two branches back into original sample order."""
    g = gate.reshape(-1).astype(bool)
    shape = (g.shape[0],) + (y_true.shape[1:] if y_true.shape[0] else y_false.shape[1:])
    y = np.zeros(shape, dtype=np.float64)
    y[g] = y_true
    y[~g] = y_false
    return y


def _is_int(a):
    return np.issubdtype(np.asarray(a).dtype, np.integer)


# --------------------------------------------------------------------------- interpreter
def run(text: str, consts: Dict[str, np.ndarray], inputs: Dict[str, np.ndarray],
        overrides: Optional[Dict[str, np.ndarray]] = None, g: Optional[Graph] = None,
        computed: Optional[Dict[str, np.ndarray]] = None, storage_round=None) -> Dict[str, np.ndarray]:
    """Execute the graph on one request.  Returns every tensor by name.

    overrides: tensors whose value is replaced right after they are produced (used to keep
    the oracle in lock-step with another implementation's data-dependent decisions).
    computed: if given, receives for every overridden tensor the value the oracle itself computed
    from its (possibly overridden) inputs, i.e. the per-operator lock-step reference.
    storage_round: optional function applied to every float operator output ("faithful" variant:
    what unfused execution with a narrow storage type would produce; used only to measure the
    rounding noise inherent to that storage type, never as the parity reference)."""
    g = g or parse(text)
    env: Dict[str, np.ndarray] = {}
    for name in g.inputs:
        env[name] = np.asarray(inputs[name], dtype=np.float64)
    for name in g.consts:
        env[name] = np.asarray(consts[name], dtype=np.float64)
    env.update(g.inline)
    overrides = overrides or {}
    for nd in g.nodes:
        x = [env[i] for i in nd.ins]
        a = nd.attrs
        op = nd.op
        if op == "MatMul":
            out = op_matmul(x[0], x[1])
        elif op in ("Add", "Sub", "Mul"):
            out = {"Add": np.add, "Sub": np.subtract, "Mul": np.multiply}[op](x[0], x[1])
        elif op == "Div":
            out = np.floor_divide(x[0], x[1]) if (_is_int(x[0]) and _is_int(x[1])) else x[0] / x[1]
        elif op == "Gelu":
            out = op_gelu(x[0])
        elif op == "Relu":
            out = np.maximum(x[0], 0.0)
        elif op == "Sigmoid":
            out = op_sigmoid(x[0])
        elif op == "Softmax":
            out = op_softmax(x[0], int(a.get("axis", -1)))
        elif op == "LayerNormalization":
            out = op_layernorm(x[0], x[1], x[2], int(a.get("axis", -1)), float(a.get("epsilon", 1e-5)))
        elif op == "Conv":
            out = op_conv(x[0], x[1], x[2] if len(x) > 2 else None, int(a.get("stride", 1)), int(a.get("pad", 0)))
        elif op == "GlobalAveragePool":
            out = np.mean(x[0], axis=(2, 3), keepdims=True)
        elif op == "ReduceSumSquare":
            out = np.sum(x[0] * x[0], axis=int(a.get("axis", -1)), keepdims=bool(int(a.get("keepdims", 1))))
        elif op == "TopK":
            out = op_topk(x[0], int(np.asarray(x[1]).reshape(-1)[0]), int(a.get("axis", -1)),
                          bool(int(a.get("largest", 1))), a.get("order", "value"))
        elif op == "NonZero":
            out = op_nonzero(x[0])
        elif op == "Gather":
            out = np.take(x[0], np.asarray(x[1], dtype=np.int64), axis=int(a.get("axis", 0)))
        elif op == "Shape":
            out = np.array(x[0].shape, dtype=np.int64)
        elif op == "Reshape":
            out = op_reshape(x[0], x[1])
        elif op == "Transpose":
            out = np.transpose(x[0], [int(v) for v in a["perm"].split(",")])
        elif op == "Concat":
            out = np.concatenate(x, axis=int(a.get("axis", 0)))
        elif op == "Slice":
            out = op_slice(x[0], x[1], x[2], x[3] if len(x) > 3 else np.arange(len(x[1])), x[4] if len(x) > 4 else None)
        elif op == "Cast":
            out = x[0].astype(np.int64) if a.get("to") == "i64" else x[0].astype(np.float64)
        elif op == "Range":
            out = np.arange(int(x[0]), int(x[1]), int(x[2]), dtype=np.int64)
        elif op == "ConstantOfShape":
            out = np.full([int(v) for v in x[0]], float(a.get("value", 0.0)))
        elif op == "Expand":
            # broadcast x against the VALUE of the shape operand (multidirectional: either side may be 1)
            out = np.array(x[0] * np.ones([int(v) for v in x[1]], dtype=x[0].dtype))
        elif op in ("Resize", "Upsample"):
            # nearest neighbour (Table 2 lists Resize / Upsample as input shape & value determined): the output extents
            # are the VALUE of the sizes operand, or extent * integer scale; output index o along an axis reads source
            # index floor(o * in / out)
            src = x[0]
            if len(x) > 1:
                sizes = [int(v) for v in np.asarray(x[1]).reshape(-1)]
            else:
                sizes = [d * int(v) for d, v in zip(src.shape, a["scales"].split(","))]
            out = src
            for ax, (n_in, n_out) in enumerate(zip(src.shape, sizes)):
                pick = [min(n_in - 1, (o * n_in) // n_out) for o in range(n_out)]
                out = np.take(out, pick, axis=ax)
        elif op == "Greater":
            out = (x[0] > x[1])
        elif op == "Switch":
            out = op_switch(x[0], x[1])
        elif op == "Combine":
            out = op_combine(x[0], x[1], x[2])
        else:
            raise NotImplementedError(op)
        outs = out if isinstance(out, tuple) else (out,)
        for name, val in zip(nd.outs, outs):
            if storage_round is not None and np.asarray(val).dtype == np.float64:
                val = storage_round(val)
            if name in overrides:
                if computed is not None:
                    computed[name] = val
                env[name] = np.asarray(overrides[name]).reshape(np.shape(val))
            else:
                env[name] = val
    return env


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i |g_i - o_i| / (|o_i| + rms(o)): relative error that stays defined at zero crossings."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    ref = np.asarray(ref, dtype=np.float64).reshape(-1)
    if ref.size == 0:
        return 0.0
    rms = math.sqrt(float(np.mean(ref * ref)))
    return float(np.max(np.abs(got - ref) / (np.abs(ref) + rms + 1e-300)))
