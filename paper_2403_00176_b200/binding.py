"""ctypes binding of libsod2.so: argument marshalling only, same names as include/sod2.h.

PyTorch is used by callers for device memory and streams; this module never computes.
The library is built in-tree (paper_2403_00176_b200/build.py); importing fails loudly if it is
missing, and there is no CPU fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsod2.so")

STATUS = ["SOD2_OK", "SOD2_E_INVALID_ARG", "SOD2_E_PARSE", "SOD2_E_UNSUPPORTED_OP", "SOD2_E_RANK_MISMATCH",
          "SOD2_E_NOT_CONVERGED", "SOD2_E_UNBOUND_SYMBOL", "SOD2_E_BAD_DIM", "SOD2_E_SHAPE_CONFLICT",
          "SOD2_E_ARENA_TOO_SMALL", "SOD2_E_MISALIGNED", "SOD2_E_CUDA", "SOD2_E_TIMEOUT", "SOD2_E_INTERNAL"]
OPT_NO_FUSION = 1
OPT_NO_REUSE = 2
OPT_SPLITK_LN = 4
OPT_LEGACY_ATTENTION = 8
OPT_COPY_REGROUP = 16
OPT_NO_SEP = 32
OPT_MULTI_VERSION = 64
OPT_LN_FOLD = 128
OPT_GEMM_CHAIN = 256
OPT_GUARD_BANDS = 512
OPT_GEMM_PAIR = 1024
DYN_CLASS = ["ISDO", "ISDOS", "ISVDOS", "EDO"]


class Sod2Error(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS[status] if 0 <= status < len(STATUS) else status}: {msg}")
        self.status = status
        self.status_name = STATUS[status] if 0 <= status < len(STATUS) else str(status)


class RunInfo(C.Structure):
    _fields_ = [("host_enqueue_ns", C.c_int64), ("gpu_launches", C.c_int64), ("reserved", C.c_int64 * 6)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2403_00176_b200.build` (needs nvcc). "
                          "There is no fallback path.")
    lib = C.CDLL(LIB_PATH)
    vp, cp, sz, i32, i64 = C.c_void_p, C.c_char_p, C.c_size_t, C.c_int, C.c_int64
    P = C.POINTER
    sig = {
        "sod2_graph_create": [cp, sz, C.c_uint32, P(vp)],
        "sod2_graph_set_const": [vp, cp, vp, sz],
        "sod2_graph_prepack_bytes": [vp, P(sz)],
        "sod2_graph_prepack": [vp, vp, sz, vp],
        "sod2_bind_dims": [vp, i32, i32, P(cp), P(i64), P(vp)],
        "sod2_plan": [vp, vp, P(vp), P(sz)],
        "sod2_graph_set_plan_cache": [vp, i32],
        "sod2_plan_cached": [vp, i32, i32, P(cp), P(i64), P(vp), P(vp), P(sz), P(i32)],
        "sod2_run": [vp, P(vp), P(vp), vp, sz, vp, P(RunInfo)],
        "sod2_run_graph": [vp, P(vp), P(vp), vp, sz, vp, P(RunInfo)],
        "sod2_run_exact": [vp, P(vp), P(vp), vp, sz, vp, P(RunInfo)],
        "sod2_run_timed": [vp, P(vp), P(vp), vp, sz, vp, P(C.c_float), i32],
        "sod2_run_timed_repeat": [vp, P(vp), P(vp), vp, sz, vp, i32, P(C.c_float), i32],
        "sod2_plan_device_status": [vp, vp, vp],
        "sod2_plan_poison_arena": [vp, vp, sz, vp],
        "sod2_plan_check_guards": [vp, vp, vp, P(i32), cp, sz],
        "sod2_graph_tensor_info": [vp, cp, P(i32), P(i32), cp, sz],
        "sod2_graph_tensor_value": [vp, cp, cp, sz],
        "sod2_graph_tensor_dtype": [vp, cp, P(i32)],
        "sod2_graph_op_info": [vp, i32, cp, sz, P(i32), P(i32), P(i32), P(i32)],
        "sod2_graph_group_info": [vp, i32, cp, sz, P(i32), P(i32), P(i32)],
        "sod2_classify": [cp, P(i32)],
        "sod2_graph_reanalyse": [vp, P(i32), i32],
        "sod2_graph_order_info": [vp, P(i64)],
        "sod2_binding_shape": [vp, i32, cp, P(i64), P(i32)],
        "sod2_plan_slot": [vp, cp, P(sz), P(sz), P(i32), P(i32)],
        "sod2_plan_instance_offset": [vp, cp, i32, P(sz)],
        "sod2_plan_memory": [vp, P(sz), P(sz), P(sz)],
        "sod2_plan_group_cost": [vp, i32, P(C.c_double), P(C.c_double)],
        "sod2_plan_group_on_side_stream": [vp, i32, P(C.c_int)],
        "sod2_plan_tensor_strides": [vp, cp, i32, P(i64), P(i32)],
        "sod2_run_output_shape": [vp, vp, vp, i32, i32, P(i64), P(i32)],
        "sod2_nonzero_static": [vp, i32, i32, P(i64), vp, vp, vp],
        "sod2_launch_empty": [vp],
        "sod2_selftest_bounded_wait": [vp, vp],
        "sod2_selftest_mma_rate": [i32, i32, i32, i32, i32, i32, vp, P(C.c_double)],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = i32
    for name in ("sod2_graph_num_ops", "sod2_graph_num_groups", "sod2_graph_num_subgraphs", "sod2_graph_rdp_sweeps"):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = i32
    for name in ("sod2_graph_destroy", "sod2_binding_destroy", "sod2_plan_destroy"):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = None
    lib.sod2_last_error.argtypes = [vp]
    lib.sod2_last_error.restype = cp
    return lib


lib = _load()
EXPORTS = ["sod2_graph_create", "sod2_graph_destroy", "sod2_graph_set_const", "sod2_graph_prepack_bytes",
           "sod2_graph_prepack", "sod2_bind_dims", "sod2_binding_destroy", "sod2_plan", "sod2_plan_destroy", "sod2_graph_set_plan_cache", "sod2_plan_cached",
           "sod2_run", "sod2_run_graph", "sod2_run_exact", "sod2_run_timed", "sod2_run_timed_repeat", "sod2_plan_device_status", "sod2_plan_poison_arena", "sod2_plan_check_guards", "sod2_graph_tensor_info", "sod2_graph_tensor_value", "sod2_graph_tensor_dtype",
           "sod2_graph_num_ops", "sod2_graph_op_info", "sod2_graph_num_groups", "sod2_graph_group_info",
           "sod2_graph_num_subgraphs", "sod2_graph_rdp_sweeps", "sod2_classify", "sod2_graph_reanalyse", "sod2_graph_order_info",
           "sod2_binding_shape", "sod2_plan_slot", "sod2_plan_instance_offset", "sod2_plan_memory", "sod2_plan_group_cost", "sod2_plan_group_on_side_stream", "sod2_plan_tensor_strides",
           "sod2_run_output_shape", "sod2_nonzero_static", "sod2_launch_empty", "sod2_selftest_bounded_wait", "sod2_selftest_mma_rate", "sod2_last_error"]


def _check(status: int, handle=None):
    if status != 0:
        msg = lib.sod2_last_error(handle).decode() if handle is not None else lib.sod2_last_error(None).decode()
        raise Sod2Error(status, msg)


def sod2_classify(op: str) -> str:
    c = C.c_int()
    _check(lib.sod2_classify(op.encode(), C.byref(c)))
    return DYN_CLASS[c.value]


NONZERO_STATIC_MAX_ELEMS = 16777216


def sod2_launch_empty(stream: int) -> None:
    """One kernel that does nothing, on `stream`: the yardstick for launch-bound groups."""
    _check(lib.sod2_launch_empty(C.c_void_p(stream)))


def sod2_selftest_bounded_wait(dev_status_word: int, stream: int) -> None:
    """Launches the kernel whose bounded wait runs out: it sets the device status word and returns by itself."""
    _check(lib.sod2_selftest_bounded_wait(C.c_void_p(dev_status_word), C.c_void_p(stream)))


def sod2_selftest_mma_rate(pair: bool, n_cols: int, per_stage: int, handshake: int, stream: int, iters: int = 4096, clusters: int = 74) -> float:
    """SM cycles per tcgen05.mma (128 x n_cols x 16 on one CTA, 256 x n_cols x 16 on a CTA pair) issued in stages of
    `per_stage`; handshake 0 = MMAs only, 1 = commit per stage, 2 = full / empty barrier handshake per stage."""
    out = C.c_double()
    _check(lib.sod2_selftest_mma_rate(int(bool(pair)), n_cols, per_stage, handshake, iters, clusters, C.c_void_p(stream), C.byref(out)))
    return out.value


def sod2_nonzero_static(dev_x: int, dtype: int, dims: Sequence[int], dev_out: int, dev_count: int, stream: int) -> None:
    """NonZero for callers that cannot allocate device memory (no arena, no cudaMalloc): the scratch
    is a fixed array inside the library.  See include/sod2.h for the limits (input size, shared
    scratch, first call outside stream capture)."""
    d = (C.c_int64 * max(len(dims), 1))(*[int(v) for v in dims])
    _check(lib.sod2_nonzero_static(C.c_void_p(dev_x), dtype, len(dims), d, C.c_void_p(dev_out), C.c_void_p(dev_count),
                                   C.c_void_p(stream)))


class Graph:
    """sod2_graph handle."""

    def __init__(self, ir_text: str, opt_flags: int = 0):
        raw = ir_text.encode()
        h = C.c_void_p()
        _check(lib.sod2_graph_create(raw, len(raw), opt_flags, C.byref(h)))
        self.h = h
        self._keep = []

    def __del__(self):
        if getattr(self, "h", None) and lib is not None:   # lib is None while the interpreter shuts down
            lib.sod2_graph_destroy(self.h)
            self.h = None

    def set_const(self, name: str, dev_ptr: int, nbytes: int, keep=None):
        _check(lib.sod2_graph_set_const(self.h, name.encode(), C.c_void_p(dev_ptr), nbytes), self.h)
        if keep is not None:
            self._keep.append(keep)

    def prepack_bytes(self) -> int:
        n = C.c_size_t()
        _check(lib.sod2_graph_prepack_bytes(self.h, C.byref(n)), self.h)
        return n.value

    def prepack(self, dev_ws: int, nbytes: int, stream: int, keep=None):
        _check(lib.sod2_graph_prepack(self.h, C.c_void_p(dev_ws), nbytes, C.c_void_p(stream)), self.h)
        if keep is not None:
            self._keep.append(keep)

    def set_plan_cache(self, capacity: int):
        _check(lib.sod2_graph_set_plan_cache(self.h, capacity), self.h)

    def plan_cached(self, sym_names: Sequence[str], values: Sequence[Sequence[int]]):
        """bind_dims + plan through the graph's plan cache: (Binding, Plan, hit).  The handles are borrowed
        from the graph (valid until evicted); the wrappers keep the graph alive and never destroy them."""
        n_req, n_sym = len(values), len(sym_names)
        names = (C.c_char_p * max(n_sym, 1))(*[s.encode() for s in sym_names])
        flat = [int(v) for row in values for v in row]
        vals = (C.c_int64 * max(len(flat), 1))(*flat)
        hb, hp, ab, hit = C.c_void_p(), C.c_void_p(), C.c_size_t(), C.c_int()
        _check(lib.sod2_plan_cached(self.h, n_req, n_sym, names, vals, C.byref(hb), C.byref(hp), C.byref(ab), C.byref(hit)), self.h)
        b = Binding.__new__(Binding)
        b.graph, b.h, b.n_req, b.borrowed = self, hb, n_req, True
        p = Plan.__new__(Plan)
        p.binding, p.graph, p.h, p.arena_bytes, p.borrowed = b, self, hp, ab.value, True
        return b, p, bool(hit.value)

    def bind_dims(self, sym_names: Sequence[str], values: Sequence[Sequence[int]]) -> "Binding":
        return Binding(self, sym_names, values)

    def tensor_info(self, name: str) -> Tuple[int, List[int], str]:
        rank = C.c_int()
        kinds = (C.c_int * 16)()
        buf = C.create_string_buffer(1024)
        _check(lib.sod2_graph_tensor_info(self.h, name.encode(), C.byref(rank), kinds, buf, 1024), self.h)
        return rank.value, list(kinds[: max(rank.value, 0)]), buf.value.decode()

    def tensor_dtype(self, name: str) -> str:
        d = C.c_int()
        _check(lib.sod2_graph_tensor_dtype(self.h, name.encode(), C.byref(d)), self.h)
        return ["f32", "bf16", "i64", "bool"][d.value]

    def tensor_value(self, name: str) -> str:
        buf = C.create_string_buffer(1024)
        _check(lib.sod2_graph_tensor_value(self.h, name.encode(), buf, 1024), self.h)
        return buf.value.decode()

    def num_ops(self) -> int:
        return lib.sod2_graph_num_ops(self.h)

    def op_info(self, i: int) -> dict:
        t = C.create_string_buffer(64)
        a, b, g, s = C.c_int(), C.c_int(), C.c_int(), C.c_int()
        _check(lib.sod2_graph_op_info(self.h, i, t, 64, C.byref(a), C.byref(b), C.byref(g), C.byref(s)), self.h)
        return {"op": t.value.decode(), "cls": DYN_CLASS[a.value], "eff_cls": DYN_CLASS[b.value], "group": g.value,
                "subgraph": s.value}

    def num_groups(self) -> int:
        return lib.sod2_graph_num_groups(self.h)

    def group_info(self, i: int) -> dict:
        t = C.create_string_buffer(64)
        n, v, s = C.c_int(), C.c_int(), C.c_int()
        _check(lib.sod2_graph_group_info(self.h, i, t, 64, C.byref(n), C.byref(v), C.byref(s)), self.h)
        return {"kind": t.value.decode(), "n_ops": n.value, "versions": v.value, "subgraph": s.value}

    def num_subgraphs(self) -> int:
        return lib.sod2_graph_num_subgraphs(self.h)

    def rdp_sweeps(self) -> int:
        return lib.sod2_graph_rdp_sweeps(self.h)

    def order_info(self) -> dict:
        """Static execution planning (Section 4.3): peaks of the default and planned group order."""
        out = (C.c_int64 * 9)()
        _check(lib.sod2_graph_order_info(self.h, out), self.h)
        keys = ("default_peak_hi", "default_peak_lo", "planned_peak_hi", "planned_peak_lo", "states",
                "searched_subgraphs", "reordered_subgraphs", "abandoned_subgraphs", "unbounded")
        return dict(zip(keys, [int(v) for v in out]))

    def reanalyse(self, order: Sequence[int]):
        arr = (C.c_int * len(order))(*order)
        _check(lib.sod2_graph_reanalyse(self.h, arr, len(order)), self.h)


class Binding:
    """sod2_binding handle (per-request symbol values)."""

    def __init__(self, graph: Graph, sym_names: Sequence[str], values: Sequence[Sequence[int]]):
        self.graph = graph
        n_req, n_sym = len(values), len(sym_names)
        names = (C.c_char_p * max(n_sym, 1))(*[s.encode() for s in sym_names])
        flat = [int(v) for row in values for v in row]
        vals = (C.c_int64 * max(len(flat), 1))(*flat)
        h = C.c_void_p()
        _check(lib.sod2_bind_dims(graph.h, n_req, n_sym, names, vals, C.byref(h)), graph.h)
        self.h = h
        self.n_req = n_req

    def __del__(self):
        if getattr(self, "h", None) and lib is not None and not getattr(self, "borrowed", False):   # lib is None at shutdown
            lib.sod2_binding_destroy(self.h)
            self.h = None

    def shape(self, request: int, tensor: str) -> List[int]:
        dims = (C.c_int64 * 16)()
        rank = C.c_int()
        _check(lib.sod2_binding_shape(self.h, request, tensor.encode(), dims, C.byref(rank)), self.graph.h)
        return list(dims[: rank.value])

    def plan(self) -> "Plan":
        return Plan(self)


class Plan:
    """sod2_plan_t handle (arena plan + launch plan)."""

    def __init__(self, binding: Binding):
        self.binding = binding
        self.graph = binding.graph
        h = C.c_void_p()
        ab = C.c_size_t()
        _check(lib.sod2_plan(self.graph.h, binding.h, C.byref(h), C.byref(ab)), self.graph.h)
        self.h = h
        self.arena_bytes = ab.value

    def __del__(self):
        if getattr(self, "h", None) and lib is not None and not getattr(self, "borrowed", False):   # lib is None at shutdown
            lib.sod2_plan_destroy(self.h)
            self.h = None

    def run(self, inputs: Sequence[int], outputs: Sequence[int], arena: int, arena_bytes: int, stream: int) -> RunInfo:
        ins = (C.c_void_p * max(len(inputs), 1))(*inputs)
        outs = (C.c_void_p * max(len(outputs), 1))(*outputs)
        info = RunInfo()
        _check(lib.sod2_run(self.h, ins, outs, C.c_void_p(arena), arena_bytes, C.c_void_p(stream), C.byref(info)), self.h)
        return info

    def run_graph(self, inputs: Sequence[int], outputs: Sequence[int], arena: int, arena_bytes: int, stream: int) -> RunInfo:
        """The same inference as one CUDA graph (captured on first use and when a buffer pointer changes)."""
        ins = (C.c_void_p * max(len(inputs), 1))(*inputs)
        outs = (C.c_void_p * max(len(outputs), 1))(*outputs)
        info = RunInfo()
        _check(lib.sod2_run_graph(self.h, ins, outs, C.c_void_p(arena), arena_bytes, C.c_void_p(stream), C.byref(info)), self.h)
        return info

    def run_exact(self, inputs: Sequence[int], outputs: Sequence[int], arena: int, arena_bytes: int, stream: int) -> RunInfo:
        """The inference with exact handling of execution-determined extents: counts read back after every Switch /
        NonZero, the remaining sub-graphs planned again at their true sizes (synchronises the stream at each)."""
        ins = (C.c_void_p * max(len(inputs), 1))(*inputs)
        outs = (C.c_void_p * max(len(outputs), 1))(*outputs)
        info = RunInfo()
        _check(lib.sod2_run_exact(self.h, ins, outs, C.c_void_p(arena), arena_bytes, C.c_void_p(stream), C.byref(info)), self.h)
        return info

    def run_timed(self, inputs: Sequence[int], outputs: Sequence[int], arena: int, arena_bytes: int, stream: int, reps: int = 1) -> List[float]:
        """Device time per fused group (ms).  reps > 1: every launch repeated back to back, time divided by reps."""
        ins = (C.c_void_p * max(len(inputs), 1))(*inputs)
        outs = (C.c_void_p * max(len(outputs), 1))(*outputs)
        n = self.graph.num_groups()
        ms = (C.c_float * max(n, 1))()
        if reps > 1:
            _check(lib.sod2_run_timed_repeat(self.h, ins, outs, C.c_void_p(arena), arena_bytes, C.c_void_p(stream), reps, ms, n), self.h)
        else:
            _check(lib.sod2_run_timed(self.h, ins, outs, C.c_void_p(arena), arena_bytes, C.c_void_p(stream), ms, n), self.h)
        return list(ms[:n])

    def poison_arena(self, arena: int, arena_bytes: int, stream: int):
        """Fill the arena behind its header with 0xFF bytes (graphs created with OPT_GUARD_BANDS)."""
        _check(lib.sod2_plan_poison_arena(self.h, C.c_void_p(arena), arena_bytes, C.c_void_p(stream)), self.h)

    def check_guards(self, arena: int, stream: int):
        """(damaged bands, name of the tensor behind which the lowest damaged band lies)."""
        n = C.c_int()
        buf = C.create_string_buffer(256)
        _check(lib.sod2_plan_check_guards(self.h, C.c_void_p(arena), C.c_void_p(stream), C.byref(n), buf, 256), self.h)
        return n.value, buf.value.decode()

    def device_status(self, arena: int, stream: int):
        _check(lib.sod2_plan_device_status(self.h, C.c_void_p(arena), C.c_void_p(stream)), self.h)

    def slot(self, tensor: str) -> dict:
        off, nb = C.c_size_t(), C.c_size_t()
        d, l = C.c_int(), C.c_int()
        _check(lib.sod2_plan_slot(self.h, tensor.encode(), C.byref(off), C.byref(nb), C.byref(d), C.byref(l)), self.h)
        return {"offset": off.value, "bytes": nb.value, "def_step": d.value, "last_use_step": l.value}

    def instance_offset(self, tensor: str, request: int) -> int:
        off = C.c_size_t()
        _check(lib.sod2_plan_instance_offset(self.h, tensor.encode(), request, C.byref(off)), self.h)
        return off.value

    def memory(self) -> dict:
        a, p, s = C.c_size_t(), C.c_size_t(), C.c_size_t()
        _check(lib.sod2_plan_memory(self.h, C.byref(a), C.byref(p), C.byref(s)), self.h)
        return {"arena_bytes": a.value, "peak_live_bytes": p.value, "sum_bytes": s.value}

    def tensor_strides(self, tensor: str, request: int) -> List[int]:
        st = (C.c_int64 * 16)()
        rank = C.c_int()
        _check(lib.sod2_plan_tensor_strides(self.h, tensor.encode(), request, st, C.byref(rank)), self.h)
        return list(st[: rank.value])

    def group_cost(self, group: int):
        f, b = C.c_double(), C.c_double()
        _check(lib.sod2_plan_group_cost(self.h, group, C.byref(f), C.byref(b)), self.h)
        return f.value, b.value

    def group_on_side_stream(self, group: int) -> bool:
        v = C.c_int()
        _check(lib.sod2_plan_group_on_side_stream(self.h, group, C.byref(v)), self.h)
        return bool(v.value)

    def output_shape(self, arena: int, stream: int, request: int, output: int) -> List[int]:
        dims = (C.c_int64 * 16)()
        rank = C.c_int()
        _check(lib.sod2_run_output_shape(self.h, C.c_void_p(arena), C.c_void_p(stream), request, output, dims,
                                         C.byref(rank)), self.h)
        return list(dims[: rank.value])
