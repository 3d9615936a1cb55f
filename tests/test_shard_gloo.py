"""N>1 path on CPU: requests / batches are independent units, sharded across ranks with no data-path
collective; only the timing (max over ranks) and the unit count (sum) are reduced."""
import os
import subprocess
import sys
import textwrap

from paper_2403_00176_b200.shard import assign_batches, assign_requests


def test_assign_batches_partitions():
    for world in (1, 2, 3, 8):
        seen = []
        for r in range(world):
            seen += assign_batches(20, r, world)
        assert sorted(seen) == list(range(20))
    assert assign_batches(2, 5, 8) == [5 % 2]          # more ranks than batches: every rank still works


def test_assign_requests_longest_first_balances():
    costs = [512, 16, 300, 299, 64, 64, 450, 17]
    parts = assign_requests(costs, 2)
    assert sorted(parts[0] + parts[1]) == list(range(len(costs)))
    loads = [sum(costs[i] for i in p) for p in parts]
    assert abs(loads[0] - loads[1]) <= max(costs) // 4


def test_world_size_2_gloo_reduction(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(textwrap.dedent("""
        import os, sys, json
        sys.path.insert(0, %r)
        import torch, torch.distributed as dist
        from paper_2403_00176_b200.shard import assign_batches
        from paper_2403_00176_b200 import workloads as WL, binding as B
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        mine = assign_batches(6, rank, world)
        wl = WL.cfg2(layers=1, D=128, H=2, F=256)
        g = B.Graph(wl.ir)
        tokens = 0
        for j in mine:                      # each rank binds and plans only its own batches
            reqs = wl.batch(j)
            p = g.bind_dims(wl.sym_names, [[r.syms[s] for s in wl.sym_names] for r in reqs]).plan()
            assert p.arena_bytes > 0
            tokens += sum(r.syms["L"] for r in reqs)
        t = torch.tensor([float(rank + 1)])             # stand-in for this rank's elapsed time
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        n = torch.tensor([float(tokens)])
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
        ids = [None] * world
        dist.all_gather_object(ids, mine)
        if rank == 0:
            print(json.dumps({"max_t": t.item(), "tokens": n.item(), "ids": ids}))
        dist.destroy_process_group()
    """ % os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1]
    d = json.loads(line)
    assert d["max_t"] == 2.0
    assert sorted(d["ids"][0] + d["ids"][1]) == list(range(6))
    from paper_2403_00176_b200 import workloads as WL
    wl = WL.cfg2(layers=1, D=128, H=2, F=256)
    assert d["tokens"] == sum(r.syms["L"] for j in range(6) for r in wl.batch(j))
