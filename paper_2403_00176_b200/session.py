"""Convenience driver around the C ABI: device buffers (torch), packing of per-request tensors,
constant upload and prepack.  Marshalling only; every computation runs in libsod2.so's kernels."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from .workloads import Request, Workload, bf16_bits, bits_to_f32

_NP = {"f32": np.float32, "bf16": np.uint16, "i64": np.int64, "bool": np.uint8}
_ESZ = {"f32": 4, "bf16": 2, "i64": 8, "bool": 1}


def _to_storage(a: np.ndarray, dt: str) -> np.ndarray:
    if dt == "bf16":
        return bf16_bits(np.asarray(a, np.float32))
    return np.ascontiguousarray(a, dtype=_NP[dt])


def _from_storage(a: np.ndarray, dt: str) -> np.ndarray:
    if dt == "bf16":
        return bits_to_f32(a)
    return a


class Session:
    """One graph on one GPU: constants resident in HBM, weights prepacked once."""

    def __init__(self, wl: Workload, device: str = "cuda:0", opt_flags: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: the library has no CPU path")
        self.wl = wl
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.graph = B.Graph(wl.ir, opt_flags)
        self.stream = torch.cuda.current_stream(self.dev).cuda_stream
        self._consts = {}
        for name, arr in wl.consts.items():
            dt = self.graph.tensor_dtype(name)
            host = _to_storage(arr, dt)
            t = torch.from_numpy(host.view(np.uint8).reshape(-1).copy()).to(self.dev)
            self._consts[name] = t
            self.graph.set_const(name, t.data_ptr(), t.numel())
        nb = self.graph.prepack_bytes()
        self._ws = torch.empty(max(nb, 256), dtype=torch.uint8, device=self.dev)
        self.graph.prepack(self._ws.data_ptr(), self._ws.numel(), self.stream)
        torch.cuda.synchronize(self.dev)
        self.in_names = [ln.split()[1] for ln in wl.ir.splitlines() if ln.startswith("input ")]
        self.out_names = [ln.split()[1] for ln in wl.ir.splitlines() if ln.startswith("output ")]

    # ---- planning
    def prepare(self, reqs: Sequence[Request]) -> "Prepared":
        return Prepared(self, reqs)


class Prepared:
    """A bound + planned batch with its device buffers."""

    def __init__(self, s: Session, reqs: Sequence[Request]):
        self.s = s
        self.reqs = list(reqs)
        names = s.wl.sym_names
        self.binding = s.graph.bind_dims(names, [[r.syms[n] for n in names] for r in reqs])
        self.plan = self.binding.plan()
        self.n = len(reqs)
        g = s.graph
        self.in_dt = [g.tensor_dtype(n) for n in s.in_names]
        self.out_dt = [g.tensor_dtype(n) for n in s.out_names]
        self.in_host = [self._pack_input(n, dt) for n, dt in zip(s.in_names, self.in_dt)]
        self.in_dev = [torch.from_numpy(h).to(s.dev) for h in self.in_host]
        self.out_bytes = [self._packed_bytes(n, dt) for n, dt in zip(s.out_names, self.out_dt)]
        self.out_dev = [torch.zeros(max(nb, 16), dtype=torch.uint8, device=s.dev) for nb in self.out_bytes]
        self.arena = torch.empty(max(self.plan.arena_bytes, 256), dtype=torch.uint8, device=s.dev)

    def _inst_bytes(self, name: str, dt: str, r: int) -> int:
        shp = self.binding.shape(r, name)
        return int(np.prod(shp, dtype=np.int64)) * _ESZ[dt] if shp else _ESZ[dt]

    def _packed_bytes(self, name: str, dt: str) -> int:
        last = self.n - 1
        return self.plan.instance_offset(name, last) + ((self._inst_bytes(name, dt, last) + 15) & ~15)

    def _pack_input(self, name: str, dt: str) -> np.ndarray:
        buf = np.zeros(max(self._packed_bytes(name, dt), 16), dtype=np.uint8)
        for r, req in enumerate(self.reqs):
            raw = _to_storage(req.inputs[name], dt).view(np.uint8).reshape(-1)
            off = self.plan.instance_offset(name, r)
            buf[off:off + raw.size] = raw
        return buf

    def run(self) -> B.RunInfo:
        return self.plan.run([t.data_ptr() for t in self.in_dev], [t.data_ptr() for t in self.out_dev],
                             self.arena.data_ptr(), self.arena.numel(), self.s.stream)

    def run_graph(self) -> B.RunInfo:
        """The inference as one CUDA graph over this batch's own buffers (captured by the first call)."""
        return self.plan.run_graph([t.data_ptr() for t in self.in_dev], [t.data_ptr() for t in self.out_dev],
                                   self.arena.data_ptr(), self.arena.numel(), self.s.stream)

    def run_exact(self) -> B.RunInfo:
        """The inference with counts read back and the remaining sub-graphs planned again at their true sizes."""
        return self.plan.run_exact([t.data_ptr() for t in self.in_dev], [t.data_ptr() for t in self.out_dev],
                                   self.arena.data_ptr(), self.arena.numel(), self.s.stream)

    def check_device_status(self):
        self.plan.device_status(self.arena.data_ptr(), self.s.stream)

    def outputs(self) -> List[Dict[str, np.ndarray]]:
        """Per request: output name -> array (float32 for float tensors), with the true shape."""
        torch.cuda.synchronize(self.s.dev)
        res = []
        host = [t.cpu().numpy() for t in self.out_dev]
        for r in range(self.n):
            d = {}
            for j, (name, dt) in enumerate(zip(self.s.out_names, self.out_dt)):
                shp = self.plan.output_shape(self.arena.data_ptr(), self.s.stream, r, j)
                cnt = int(np.prod(shp, dtype=np.int64)) if shp else 1
                off = self.plan.instance_offset(name, r)
                raw = host[j][off:off + cnt * _ESZ[dt]].view(_NP[dt])
                d[name] = _from_storage(raw, dt).reshape(shp)
            res.append(d)
        return res

    def read_arena_tensor(self, name: str, r: int) -> np.ndarray:
        """An inter-group tensor of request r straight from the arena (meaningful with OPT_NO_REUSE)."""
        torch.cuda.synchronize(self.s.dev)
        dt = self.s.graph.tensor_dtype(name)
        shp = self.binding.shape(r, name)
        slot = self.plan.slot(name)
        off = slot["offset"] + self.plan.instance_offset(name, r)
        cnt = int(np.prod(shp, dtype=np.int64))
        raw = self.arena[off:off + cnt * _ESZ[dt]].cpu().numpy().view(_NP[dt])
        flat = _from_storage(raw, dt)
        strides = self.plan.tensor_strides(name, r)
        if cnt == 0:
            return flat.reshape(shp)
        # storage order may differ from the logical dim order (channels-last): gather through the strides
        return np.lib.stride_tricks.as_strided(flat, shape=shp, strides=[s * flat.itemsize for s in strides]).copy()
