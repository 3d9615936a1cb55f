"""The allocation-free NonZero entry point against the regular (arena-based) path.

sod2_nonzero_static exists for callers that may not allocate device memory: they pass only the
input and output buffers, and the compaction's counters live in a fixed array inside the library.
The test calls it through the C ABI twice in a row (the second call on a smaller input, so stale
counters from the first call would show) and requires bit-identical coordinates and counts to the
regular path, which takes its scratch from the caller's arena.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2403_00176_b200 import binding as B
from paper_2403_00176_b200 import workloads as WL
from paper_2403_00176_b200.workloads import Request
from tests.gpu_harness import run_batch

pytestmark = pytest.mark.gpu


def _static_nonzero(x: np.ndarray):
    dev = torch.device("cuda:0")
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(dev)
    out = torch.full((x.ndim * max(x.size, 1),), -1, dtype=torch.int64, device=dev)
    cnt = torch.full((1,), -1, dtype=torch.int64, device=dev)
    B.sod2_nonzero_static(xd.data_ptr(), 0, list(x.shape), out.data_ptr(), cnt.data_ptr(),
                          torch.cuda.current_stream(dev).cuda_stream)
    torch.cuda.synchronize(dev)
    n = int(cnt.item())
    return out[: x.ndim * n].cpu().numpy().reshape(x.ndim, n), n


def test_static_scratch_nonzero_matches_arena_path_twice():
    rng = np.random.default_rng(21)
    big = rng.standard_normal((900, 1100)).astype(np.float32)
    big[rng.uniform(size=big.shape) < 0.8] = 0
    small = rng.standard_normal((37, 53)).astype(np.float32)
    small[rng.uniform(size=small.shape) < 0.5] = 0
    wl = WL.nonzero_graph()
    reqs = [Request({"R": a.shape[0], "C": a.shape[1]}, {"x": a}) for a in (big, small)]
    _, _, ref = run_batch(wl, reqs)
    for a, want in ((big, ref[0]["nz"]), (small, ref[1]["nz"])):      # two calls in a row
        got, n = _static_nonzero(a)
        assert n == want.shape[1]
        assert np.array_equal(got, want)


def test_static_scratch_nonzero_edges_and_limit():
    got, n = _static_nonzero(np.zeros((5, 7), np.float32))
    assert n == 0 and got.shape == (2, 0)
    got, n = _static_nonzero(np.ones((3, 4, 5), np.float32))
    assert n == 60 and np.array_equal(got, np.array(np.nonzero(np.ones((3, 4, 5)))))
    dev = torch.device("cuda:0")
    buf = torch.zeros(16, dtype=torch.int64, device=dev)
    with pytest.raises(B.Sod2Error) as e:     # rejected on the host, before any launch
        B.sod2_nonzero_static(buf.data_ptr(), 0, [B.NONZERO_STATIC_MAX_ELEMS + 1], buf.data_ptr(), buf.data_ptr(), 0)
    assert e.value.status_name == "SOD2_E_BAD_DIM" and "limit" in str(e.value)
    # extents whose product wraps around the 64-bit range must be rejected, not taken for a small or empty input
    for dims in ([1 << 24, 1 << 40], [2, 1 << 62, 4], [1 << 32, 1 << 32], [0, 1 << 40]):
        with pytest.raises(B.Sod2Error) as e:
            B.sod2_nonzero_static(buf.data_ptr(), 0, dims, buf.data_ptr(), buf.data_ptr(), 0)
        assert e.value.status_name == "SOD2_E_BAD_DIM", dims
