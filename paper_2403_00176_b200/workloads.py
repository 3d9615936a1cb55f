"""Seeded synthetic workloads: graph IR text, constants, per-request dims and inputs.

This module is the one piece shared by the CUDA path's tests/bench and by the CPU
oracle.  It holds no arithmetic of the method: it only draws random numbers, rounds
them to the storage type and writes the graph of each workload in the line-oriented
IR that both sides parse on their own.

IR grammar (one statement per line, '#' starts a comment):
    sym    NAME [min max]
    input  NAME DTYPE [d0,d1,...]            dims are integers or symbol names
    const  NAME DTYPE [d0,...]               float constant, data supplied separately
    iconst NAME i64 [n] = v0 v1 ...          small inline integer constant ([] = scalar)
    fconst NAME f32 [] = 0.125               inline float scalar
    node   OP in0 in1 ... -> out0 ... {k=v k=v}
    output NAME
Operator names follow the ONNX operator set the paper classifies (Table 2) plus the
<Switch, Combine> pair, Gelu and LayerNormalization.

Workloads stand in for the paper's evaluation models (whose weights and datasets are
not available): shapes, ranges and structure follow the paper's description of its
dynamic models (sequence lengths 32-512, image sides 224-640 in multiples of 32,
top-k token pruning, per-sample skip gates); values are synthetic.
"""
from __future__ import annotations

import dataclasses
import os
from typing import Dict, List

import numpy as np

SEED0 = 240300176


# --------------------------------------------------------------------------- storage rounding
def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return (u.astype(np.uint32) << 16).view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array holding bf16-representable values -> uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).reshape(bits.shape)


@dataclasses.dataclass
class Request:
    syms: Dict[str, int]
    inputs: Dict[str, np.ndarray]  # float32 (bf16-exact when the graph dtype is bf16)


@dataclasses.dataclass
class Workload:
    name: str
    dtype: str  # "f32" | "bf16"
    ir: str
    consts: Dict[str, np.ndarray]  # float32
    sym_names: List[str]
    outputs: List[str]
    meta: dict

    def batch(self, j: int) -> List[Request]:
        return self.meta["batch_fn"](j)


def _rng(cfg: int, j: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(SEED0 + 1000 * cfg + j))


class _IR:
    def __init__(self):
        self.lines: List[str] = []
        self._n = 0

    def add(self, s: str):
        self.lines.append(s)

    def tmp(self, p="t"):
        self._n += 1
        return f"{p}{self._n}"

    def node(self, op, ins, outs, **attrs):
        a = ""
        if attrs:
            a = " {" + " ".join(f"{k}={v}" for k, v in attrs.items()) + "}"
        if isinstance(outs, str):
            outs = [outs]
        self.add(f"node {op} {' '.join(ins)} -> {' '.join(outs)}{a}")
        return outs[0] if len(outs) == 1 else outs

    def text(self):
        return "\n".join(self.lines) + "\n"


# --------------------------------------------------------------------------- cfg 1
def cfg1(D: int = 64, n_max: int = 64, n_requests: int = 32) -> Workload:
    """One fused group in fp32: MatMul -> +bias -> GELU -> +X -> LayerNorm over D."""
    ir = _IR()
    ir.add(f"sym N 1 {n_max}")
    ir.add(f"input X f32 [2,N,{D}]")
    ir.add(f"const W f32 [{D},{D}]")
    ir.add(f"const bias f32 [{D}]")
    ir.add(f"const gamma f32 [{D}]")
    ir.add(f"const beta f32 [{D}]")
    ir.node("MatMul", ["X", "W"], "t0")
    ir.node("Add", ["t0", "bias"], "t1")
    ir.node("Gelu", ["t1"], "t2")
    ir.node("Add", ["t2", "X"], "t3")
    ir.node("LayerNormalization", ["t3", "gamma", "beta"], "Y", axis=-1, epsilon=1e-5)
    ir.add("output Y")
    rw = _rng(1, 999)
    s = 1.0 / np.sqrt(D)
    consts = {
        "W": (rw.standard_normal((D, D)) * s).astype(np.float32),
        "bias": (rw.standard_normal(D) * s).astype(np.float32),
        "gamma": np.ones(D, np.float32),
        "beta": np.zeros(D, np.float32),
    }

    def batch_fn(j: int) -> List[Request]:
        r = _rng(1, j)
        out = []
        for _ in range(n_requests):
            n = int(r.integers(1, n_max + 1))
            x = (r.standard_normal((2, n, D)) * s).astype(np.float32)
            out.append(Request({"N": n}, {"X": x}))
        return out

    return Workload("cfg1_fused_group_f32", "f32", ir.text(), consts, ["N"], ["Y"],
                    {"batch_fn": batch_fn, "D": D, "cfg": 1})


# --------------------------------------------------------------------------- transformer pieces
def _attention(ir: _IR, x: str, pre: str, D: int, H: int, consts_decl: dict, dt: str, sym: str):
    """Multi-head self-attention on x:[1,sym,D]; returns the context tensor [1,sym,D]."""
    dh = D // H
    consts_decl[f"{pre}Wqkv"] = (D, 3 * D)
    consts_decl[f"{pre}bqkv"] = (3 * D,)
    a0 = ir.node("MatMul", [x, f"{pre}Wqkv"], ir.tmp())
    qkv = ir.node("Add", [a0, f"{pre}bqkv"], ir.tmp("qkv"))
    # shape tensors are computed in-graph from Shape(x): value propagation makes the
    # Reshape below (shape & value determined) behave as shape determined.
    xs = ir.node("Shape", [x], ir.tmp("shp"))
    bl = ir.node("Gather", [xs, "i_01"], ir.tmp("shp"), axis=0)
    shp4 = ir.node("Concat", [bl, "i_heads"], ir.tmp("shp"), axis=0)
    shp3 = ir.node("Concat", [bl, "i_D"], ir.tmp("shp"), axis=0)
    parts = []
    for i, nm in enumerate("qkv"):
        sl = ir.node("Slice", [qkv, f"i_st{i}", f"i_en{i}", "i_ax2"], ir.tmp(nm))
        r4 = ir.node("Reshape", [sl, shp4], ir.tmp(nm))
        perm = "0,2,3,1" if nm == "k" else "0,2,1,3"
        parts.append(ir.node("Transpose", [r4], ir.tmp(nm), perm=perm))
    q, kT, v = parts
    s0 = ir.node("MatMul", [q, kT], ir.tmp("s"))
    s1 = ir.node("Mul", [s0, "f_scale"], ir.tmp("s"))
    p = ir.node("Softmax", [s1], ir.tmp("p"), axis=-1)
    o = ir.node("MatMul", [p, v], ir.tmp("o"))
    oT = ir.node("Transpose", [o], ir.tmp("o"), perm="0,2,1,3")
    return ir.node("Reshape", [oT, shp3], ir.tmp("ctx"))


def _attn_iconsts(ir: _IR, D: int, H: int):
    dh = D // H
    ir.add("iconst i_01 i64 [2] = 0 1")
    ir.add(f"iconst i_heads i64 [2] = {H} {dh}")
    ir.add(f"iconst i_D i64 [1] = {D}")
    ir.add("iconst i_ax2 i64 [1] = 2")
    for i in range(3):
        ir.add(f"iconst i_st{i} i64 [1] = {i * D}")
        ir.add(f"iconst i_en{i} i64 [1] = {(i + 1) * D}")
    ir.add(f"fconst f_scale f32 [] = {float(1.0 / np.sqrt(dh))!r}")


def _ffn(ir: _IR, x: str, pre: str, D: int, F: int, decl: dict):
    decl[f"{pre}W1"] = (D, F)
    decl[f"{pre}b1"] = (F,)
    decl[f"{pre}W2"] = (F, D)
    decl[f"{pre}b2"] = (D,)
    f0 = ir.node("MatMul", [x, f"{pre}W1"], ir.tmp())
    f1 = ir.node("Add", [f0, f"{pre}b1"], ir.tmp())
    f2 = ir.node("Gelu", [f1], ir.tmp())
    f3 = ir.node("MatMul", [f2, f"{pre}W2"], ir.tmp())
    return ir.node("Add", [f3, f"{pre}b2"], ir.tmp())


def _draw_consts(decl: dict, rng: np.random.Generator, std: float, dtype: str):
    consts = {}
    for name, shape in decl.items():
        base = name.split(".")[-1]
        if base.startswith("g_"):
            a = np.ones(shape, np.float32)
        elif base.startswith("be_"):
            a = np.zeros(shape, np.float32)
        else:
            a = (rng.standard_normal(shape) * std).astype(np.float32)
        consts[name] = bf16_round(a) if dtype == "bf16" else a
    return consts


# --------------------------------------------------------------------------- cfg 2
def cfg2(layers: int = 6, D: int = 768, H: int = 12, F: int = 3072, n_requests: int = 8,
         lmin: int = 16, lmax: int = 512) -> Workload:
    """Post-LN transformer encoder on one request x:[1,L,D]; a batch is n_requests requests."""
    ir = _IR()
    ir.add(f"sym L {1} {max(lmax, 1)}")
    ir.add(f"input x bf16 [1,L,{D}]")
    _attn_iconsts(ir, D, H)
    decl: dict = {}
    x = "x"
    for l in range(layers):
        pre = f"l{l}."
        ctx = _attention(ir, x, pre, D, H, decl, "bf16", "L")
        decl[f"{pre}Wo"] = (D, D)
        decl[f"{pre}bo"] = (D,)
        decl[f"{pre}g_1"] = (D,)
        decl[f"{pre}be_1"] = (D,)
        decl[f"{pre}g_2"] = (D,)
        decl[f"{pre}be_2"] = (D,)
        a1 = ir.node("MatMul", [ctx, f"{pre}Wo"], ir.tmp())
        a2 = ir.node("Add", [a1, f"{pre}bo"], ir.tmp())
        a3 = ir.node("Add", [a2, x], ir.tmp())
        x1 = ir.node("LayerNormalization", [a3, f"{pre}g_1", f"{pre}be_1"], ir.tmp("x"), axis=-1, epsilon=1e-5)
        f4 = _ffn(ir, x1, pre, D, F, decl)
        f5 = ir.node("Add", [f4, x1], ir.tmp())
        out = f"y" if l == layers - 1 else ir.tmp("x")
        x = ir.node("LayerNormalization", [f5, f"{pre}g_2", f"{pre}be_2"], out, axis=-1, epsilon=1e-5)
    ir.add("output y")
    head = [ln for ln in ir.lines if not ln.startswith("node") and not ln.startswith("output")]
    body = [ln for ln in ir.lines if ln.startswith("node") or ln.startswith("output")]
    cl = [f"const {n} bf16 [{','.join(map(str, s))}]" for n, s in decl.items()]
    text = "\n".join(head + cl + body) + "\n"
    consts = _draw_consts(decl, _rng(2, 999), 0.02, "bf16")

    def batch_fn(j: int) -> List[Request]:
        r = _rng(2, j)
        out = []
        for _ in range(n_requests):
            L = int(r.integers(lmin, lmax + 1))
            xx = bf16_round(r.standard_normal((1, L, D)).astype(np.float32))
            out.append(Request({"L": L}, {"x": xx}))
        return out

    return Workload("cfg2_dynamic_seq_encoder_bf16", "bf16", text, consts, ["L"], ["y"],
                    {"batch_fn": batch_fn, "D": D, "H": H, "F": F, "layers": layers, "cfg": 2})


# --------------------------------------------------------------------------- cfg 3
def cfg3(layers: int = 12, D: int = 384, H: int = 6, F: int = 1536, n_requests: int = 16,
         nmin: int = 196, nmax: int = 784) -> Workload:
    """Pre-LN ViT-style stack with top-k token keeping after every layer."""
    ir = _IR()
    ir.add(f"sym N0 1 {nmax}")
    ir.add(f"input x bf16 [1,N0,{D}]")
    _attn_iconsts(ir, D, H)
    ir.add("iconst i_1 i64 [] = 1")
    ir.add("iconst i_7 i64 [] = 7")
    ir.add("iconst i_9 i64 [] = 9")
    ir.add("iconst i_10 i64 [] = 10")
    ir.add("iconst i_m1 i64 [1] = -1")
    ir.add("iconst i_0v i64 [1] = 0")
    decl: dict = {}
    x = "x"
    outs = []
    for l in range(layers):
        pre = f"l{l}."
        for nm in ("g_1", "be_1", "g_2", "be_2"):
            decl[f"{pre}{nm}"] = (D,)
        decl[f"{pre}Wo"] = (D, D)
        decl[f"{pre}bo"] = (D,)
        h1 = ir.node("LayerNormalization", [x, f"{pre}g_1", f"{pre}be_1"], ir.tmp("h"), axis=-1, epsilon=1e-5)
        ctx = _attention(ir, h1, pre, D, H, decl, "bf16", "N")
        a1 = ir.node("MatMul", [ctx, f"{pre}Wo"], ir.tmp())
        a2 = ir.node("Add", [a1, f"{pre}bo"], ir.tmp())
        x1 = ir.node("Add", [a2, x], ir.tmp("x"))
        h2 = ir.node("LayerNormalization", [x1, f"{pre}g_2", f"{pre}be_2"], ir.tmp("h"), axis=-1, epsilon=1e-5)
        f4 = _ffn(ir, h2, pre, D, F, decl)
        yl = ir.node("Add", [f4, x1], f"y{l}")
        # K = ceil(0.7 * N) written on integers: (7*N + 9) / 10, with N taken from Shape.
        ys = ir.node("Shape", [yl], ir.tmp("shp"))
        n = ir.node("Gather", [ys, "i_1"], ir.tmp("n"), axis=0)
        n7 = ir.node("Mul", [n, "i_7"], ir.tmp("n"))
        n79 = ir.node("Add", [n7, "i_9"], ir.tmp("n"))
        kk = ir.node("Div", [n79, "i_10"], ir.tmp("k"))
        k1 = ir.node("Reshape", [kk, "i_m1"], ir.tmp("k"))
        sc = ir.node("ReduceSumSquare", [yl], f"score{l}", axis=-1, keepdims=0)
        vals, idx = ir.node("TopK", [sc, k1], [ir.tmp("tv"), f"idx{l}"], axis=-1, largest=1, order="index")
        idx1 = ir.node("Reshape", [idx, "i_m1"], ir.tmp("ix"))
        x = ir.node("Gather", [yl, idx1], f"keep{l}", axis=1)
        outs += [f"idx{l}"]
    ir.add(f"output {x}")
    for o in outs:
        ir.add(f"output {o}")
    head = [ln for ln in ir.lines if not ln.startswith("node") and not ln.startswith("output")]
    body = [ln for ln in ir.lines if ln.startswith("node") or ln.startswith("output")]
    cl = [f"const {n} bf16 [{','.join(map(str, s))}]" for n, s in decl.items()]
    text = "\n".join(head + cl + body) + "\n"
    consts = _draw_consts(decl, _rng(3, 999), 0.02, "bf16")

    def batch_fn(j: int) -> List[Request]:
        r = _rng(3, j)
        out = []
        for _ in range(n_requests):
            n0 = int(r.integers(nmin, nmax + 1))
            xx = bf16_round(r.standard_normal((1, n0, D)).astype(np.float32))
            out.append(Request({"N0": n0}, {"x": xx}))
        return out

    return Workload("cfg3_token_pruning_vit_bf16", "bf16", text, consts, ["N0"], [x] + outs,
                    {"batch_fn": batch_fn, "D": D, "H": H, "F": F, "layers": layers, "cfg": 3})


# --------------------------------------------------------------------------- cfg 4
def cfg4(blocks: int = 8, C: int = 64, n_requests: int = 4, side_lo: int = 224, side_step: int = 32,
         side_n: int = 14) -> Workload:
    """Dynamic-resolution conv stage: blocks of y = x + ReLU(conv3x3(x) + b), then global average pool.
    Batch norm is folded into (w, b) here, by the generator."""
    ir = _IR()
    ir.add("sym H 1 4096")
    ir.add("sym W 1 4096")
    ir.add(f"input x bf16 [1,{C},H,W]")
    decl = {}
    x = "x"
    for b in range(blocks):
        decl[f"b{b}.w"] = (C, C, 3, 3)
        decl[f"b{b}.b"] = (C,)
        c = ir.node("Conv", [x, f"b{b}.w", f"b{b}.b"], ir.tmp("c"), kernel=3, stride=1, pad=1)
        r = ir.node("Relu", [c], ir.tmp("r"))
        x = ir.node("Add", [x, r], f"blk{b}")
    ir.node("GlobalAveragePool", [x], "gap")
    ir.add("output gap")
    ir.add(f"output {x}")
    head = [ln for ln in ir.lines if not ln.startswith("node") and not ln.startswith("output")]
    body = [ln for ln in ir.lines if ln.startswith("node") or ln.startswith("output")]
    cl = [f"const {n} bf16 [{','.join(map(str, s))}]" for n, s in decl.items()]
    text = "\n".join(head + cl + body) + "\n"
    rw = _rng(4, 999)
    consts = {}
    for b in range(blocks):
        w = rw.standard_normal((C, C, 3, 3)) * np.sqrt(2.0 / (C * 9))
        g = rw.uniform(0.5, 1.5, C)
        beta = rw.standard_normal(C) * 0.1
        mu = rw.standard_normal(C) * 0.1
        var = rw.uniform(0.5, 1.5, C)
        s = g / np.sqrt(var + 1e-5)
        consts[f"b{b}.w"] = bf16_round((w * s[:, None, None, None]).astype(np.float32))
        consts[f"b{b}.b"] = bf16_round((beta - mu * s).astype(np.float32))

    def batch_fn(j: int) -> List[Request]:
        r = _rng(4, j)
        out = []
        for _ in range(n_requests):
            h = side_lo + side_step * int(r.integers(0, side_n))
            w = side_lo + side_step * int(r.integers(0, side_n))
            xx = bf16_round(r.uniform(-1, 1, (1, C, h, w)).astype(np.float32))
            out.append(Request({"H": h, "W": w}, {"x": xx}))
        return out

    return Workload("cfg4_dynamic_resolution_conv_bf16", "bf16", text, consts, ["H", "W"], ["gap", x],
                    {"batch_fn": batch_fn, "C": C, "blocks": blocks, "cfg": 4})


# --------------------------------------------------------------------------- cfg 5
def cfg5(B: int = 32, side: int = 224, widths=(64, 128, 256, 512), per_stage: int = 4, cin: int = 3,
         calibrated: bool = True) -> Workload:
    """Gated skip network.  Stem conv7x7/2, then residual blocks; each block has a per-sample
    gate (linear on the global average pool, compared with 0).  Samples are regrouped by
    the gate (Switch), only the gated subset runs the block, Combine restores sample order."""
    ir = _IR()
    ir.add(f"input x bf16 [{B},{cin},{side},{side}]")
    ir.add("fconst f_zero f32 [] = 0.0")
    decl = {"stem.w": (widths[0], cin, 7, 7), "stem.b": (widths[0],)}
    c = ir.node("Conv", ["x", "stem.w", "stem.b"], ir.tmp("c"), kernel=7, stride=2, pad=3)
    x = ir.node("Relu", [c], "stem")
    cprev = widths[0]
    gates = []
    bi = 0
    for si, wdt in enumerate(widths):
        for k in range(per_stage):
            pre = f"b{bi}."
            down = (k == 0 and si > 0)
            ir.add(f"iconst {pre}pshape i64 [2] = {B} {cprev}")
            decl[f"{pre}gw"] = (cprev, 1)
            decl[f"{pre}gb"] = (1,)
            p = ir.node("GlobalAveragePool", [x], ir.tmp("p"))
            p2 = ir.node("Reshape", [p, f"{pre}pshape"], ir.tmp("p"))
            z = ir.node("MatMul", [p2, f"{pre}gw"], ir.tmp("z"))
            z2 = ir.node("Add", [z, f"{pre}gb"], f"logit{bi}")
            g = ir.node("Greater", [z2, "f_zero"], f"gate{bi}")
            xe, xs = ir.node("Switch", [x, g], [ir.tmp("xe"), ir.tmp("xs")])
            decl[f"{pre}w1"] = (wdt, cprev, 3, 3)
            decl[f"{pre}b1"] = (wdt,)
            decl[f"{pre}w2"] = (wdt, wdt, 3, 3)
            decl[f"{pre}b2"] = (wdt,)
            stride = 2 if down else 1
            c1 = ir.node("Conv", [xe, f"{pre}w1", f"{pre}b1"], ir.tmp("c"), kernel=3, stride=stride, pad=1)
            r1 = ir.node("Relu", [c1], ir.tmp("r"))
            c2 = ir.node("Conv", [r1, f"{pre}w2", f"{pre}b2"], ir.tmp("c"), kernel=3, stride=1, pad=1)
            if down:
                decl[f"{pre}ws"] = (wdt, cprev, 1, 1)
                decl[f"{pre}bs"] = (wdt,)
                sce = ir.node("Conv", [xe, f"{pre}ws", f"{pre}bs"], ir.tmp("sc"), kernel=1, stride=2, pad=0)
                scs = ir.node("Conv", [xs, f"{pre}ws", f"{pre}bs"], ir.tmp("sc"), kernel=1, stride=2, pad=0)
            else:
                sce, scs = xe, xs
            a = ir.node("Add", [sce, c2], ir.tmp("a"))
            ye = ir.node("Relu", [a], ir.tmp("ye"))
            x = ir.node("Combine", [ye, scs, g], f"blk{bi}")
            gates.append(f"gate{bi}")
            cprev = wdt
            bi += 1
    ir.node("GlobalAveragePool", [x], "gap")
    ir.add("output gap")
    for g in gates:
        ir.add(f"output {g}")
    head = [ln for ln in ir.lines if not ln.startswith("node") and not ln.startswith("output")]
    body = [ln for ln in ir.lines if ln.startswith("node") or ln.startswith("output")]
    cl = [f"const {n} bf16 [{','.join(map(str, s))}]" for n, s in decl.items()]
    text = "\n".join(head + cl + body) + "\n"
    rw = _rng(5, 999)
    consts = {}
    for name, shape in decl.items():
        base = name.split(".")[-1]
        if base in ("w1", "w2", "ws", "w"):
            fan_in = shape[1] * shape[2] * shape[3]
            a = rw.standard_normal(shape) * np.sqrt(2.0 / fan_in)
        elif base == "gw":
            a = rw.standard_normal(shape) * np.sqrt(1.0 / shape[0]) * 8.0
        elif base == "gb":
            a = rw.uniform(-0.3, 0.1, shape)
        else:
            a = rw.standard_normal(shape) * 0.05
        consts[name] = bf16_round(a.astype(np.float32))
    # gate biases calibrated (by a script that runs only the oracle) so that about 40-70 % of a
    # calibration batch skips each block; they apply to the default network only
    cal = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg5_gate_bias.txt")
    if calibrated and os.path.exists(cal) and (side, tuple(widths), per_stage, cin) == (224, (64, 128, 256, 512), 4, 3):
        vals = [float(ln) for ln in open(cal) if ln.strip() and not ln.startswith("#")]
        for i, v in enumerate(vals):
            if f"b{i}.gb" in consts:
                consts[f"b{i}.gb"] = bf16_round(np.array([v], np.float32))

    def batch_fn(j: int) -> List[Request]:
        r = _rng(5, j)
        # per-sample contrast and offset so that pooled features, and hence gates, differ by sample
        gain = r.uniform(0.5, 1.5, (B, 1, 1, 1))
        off = r.standard_normal((B, cin, 1, 1)) * 0.5
        xx = bf16_round((r.standard_normal((B, cin, side, side)) * gain + off).astype(np.float32))
        return [Request({}, {"x": xx})]

    return Workload("cfg5_gated_skip_network_bf16", "bf16", text, consts, [], ["gap"] + gates,
                    {"batch_fn": batch_fn, "B": B, "widths": widths, "cfg": 5})


# --------------------------------------------------------------------------- small graphs used by tests
def fig4_chain(dtype: str = "f32") -> Workload:
    """The paper's fusion example: Sigmoid(A[I',J',K']) + B[I,J,K] with A resolved to [I,1,1]."""
    ir = _IR()
    for s in ("I", "J", "K"):
        ir.add(f"sym {s} 1 4096")
    ir.add(f"input A {dtype} [I,1,1]")
    ir.add(f"input B {dtype} [I,J,K]")
    s = ir.node("Sigmoid", ["A"], "s")
    ir.node("Add", [s, "B"], "C")
    ir.add("output C")

    def batch_fn(j: int) -> List[Request]:
        r = _rng(6, j)
        out = []
        for _ in range(4):
            i, jj, k = (int(v) for v in r.integers(1, 40, 3))
            a = r.standard_normal((i, 1, 1)).astype(np.float32)
            b = r.standard_normal((i, jj, k)).astype(np.float32)
            if dtype == "bf16":
                a, b = bf16_round(a), bf16_round(b)
            out.append(Request({"I": i, "J": jj, "K": k}, {"A": a, "B": b}))
        return out

    return Workload("fig4_sigmoid_add", dtype, ir.text(), {}, ["I", "J", "K"], ["C"], {"batch_fn": batch_fn, "cfg": 6})


def nonzero_graph() -> Workload:
    """Execution-determined output: NonZero of a [R,C] tensor."""
    ir = _IR()
    ir.add("sym R 1 4096")
    ir.add("sym C 1 4096")
    ir.add("input x f32 [R,C]")
    ir.node("NonZero", ["x"], "nz")
    ir.add("output nz")

    def batch_fn(j: int) -> List[Request]:
        r = _rng(7, j)
        out = []
        for _ in range(4):
            rr, cc = (int(v) for v in r.integers(1, 70, 2))
            x = r.standard_normal((rr, cc)).astype(np.float32)
            x[r.uniform(size=x.shape) < 0.6] = 0.0
            out.append(Request({"R": rr, "C": cc}, {"x": x}))
        return out

    return Workload("nonzero", "f32", ir.text(), {}, ["R", "C"], ["nz"], {"batch_fn": batch_fn, "cfg": 7})
