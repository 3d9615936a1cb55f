"""Host-side method on CPU: operator classification (Table 2), RDP (Algorithm 1), fusion groups,
partition at execution-determined operators, binding.  RDP-inferred shapes must equal the shapes
produced by brute-force unfused execution (the oracle) on tiny inputs."""
import os
import random

import numpy as np
import pytest

from oracle import interp as O
from paper_2403_00176_b200 import binding as B
from paper_2403_00176_b200 import workloads as WL
from paper_2403_00176_b200.workloads import Request

GOLD = os.path.join(os.path.dirname(__file__), "golden", "table2_classes.txt")


def test_table2_classification():
    rows = [ln.split() for ln in open(GOLD) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 30
    for op, cls in rows:
        assert B.sod2_classify(op) == cls, op
    with pytest.raises(B.Sod2Error):
        B.sod2_classify("NoSuchOp")


def _tiny_workloads():
    return [
        WL.cfg1(),
        WL.cfg2(layers=2, D=16, H=2, F=32, n_requests=3, lmin=1, lmax=12),
        WL.cfg3(layers=3, D=16, H=2, F=32, n_requests=3, nmin=4, nmax=30),
        WL.cfg4(blocks=2, C=4, n_requests=2, side_lo=5, side_step=3, side_n=4),
        WL.cfg5(B=4, side=16, widths=(4, 8), per_stage=2),
        WL.fig4_chain(),
        WL.nonzero_graph(),
    ]


@pytest.mark.parametrize("wl", _tiny_workloads(), ids=lambda w: w.name)
def test_rdp_shapes_equal_bruteforce_execution(wl):
    """evaluate(RDP expression) == shape of the array the oracle produced, for every tensor whose
    shape RDP calls known; tensors RDP calls execution-determined must descend from an EDO operator
    and their evaluated upper bound must dominate the true extent."""
    g = B.Graph(wl.ir)
    og = O.parse(wl.ir)
    edo_descendants = set()
    for nd in og.nodes:
        if nd.op in ("NonZero", "Switch", "Combine") or any(i in edo_descendants for i in nd.ins):
            edo_descendants.update(nd.outs)
    checked = 0
    for j in range(3):
        reqs = wl.batch(j)[:3]
        bind = g.bind_dims(wl.sym_names, [[r.syms[s] for s in wl.sym_names] for r in reqs])
        for r, req in enumerate(reqs):
            env = O.run(wl.ir, wl.consts, req.inputs, g=og)
            for nd in og.nodes:
                for name in nd.outs:
                    rank, kinds, txt = g.tensor_info(name)
                    true = list(np.shape(env[name]))
                    assert rank == len(true), (name, txt, true)
                    got = bind.shape(r, name)
                    if 4 in kinds:
                        assert name in edo_descendants, (name, txt)
                        assert all(a >= b for a, b in zip(got, true)), (name, got, true)
                    else:
                        assert 0 not in kinds, (name, txt)
                        assert got == true, (name, txt, got, true)
                    checked += 1
    assert checked > 0


def test_expected_smaps_per_config():
    g = B.Graph(WL.cfg1().ir)
    for t in ("t0", "t1", "t2", "t3", "Y"):
        assert g.tensor_info(t)[2] == "[2,N,64]"
    assert g.num_groups() == 1 and g.group_info(0) == {"kind": "gemm", "n_ops": 5, "versions": 1, "subgraph": 0}
    assert all(g.op_info(i)["cls"] == "ISDOS" for i in range(g.num_ops()))

    wl = WL.cfg2(layers=1)
    g = B.Graph(wl.ir)
    og = O.parse(wl.ir)
    shapes = {o: g.tensor_info(o)[2] for nd in og.nodes for o in nd.outs}
    assert "[1,12,L,64]" in shapes.values() and "[1,12,64,L]" in shapes.values() and "[1,12,L,L]" in shapes.values()
    assert "[1,L,2304]" in shapes.values() and "[1,L,3072]" in shapes.values() and shapes["y"] == "[1,L,768]"
    kinds = [g.group_info(i)["kind"] for i in range(g.num_groups())]
    assert kinds == ["gemm", "attention", "gemm", "layernorm", "gemm", "gemm", "layernorm"]
    # opt-in: the LayerNorm between the attention projection and the FFN is folded into the GEMMs around it (the
    # last one produces the graph output and stays); every operator still belongs to some group
    gf = B.Graph(wl.ir, B.OPT_LN_FOLD)
    assert [gf.group_info(i)["kind"] for i in range(gf.num_groups())] == ["gemm", "attention", "gemm", "gemm", "gemm", "layernorm"]
    assert sum(gf.group_info(i)["n_ops"] for i in range(6)) == sum(g.group_info(i)["n_ops"] for i in range(7))
    # opt-in: the two residual GEMMs of a post-LN layer absorb their LayerNorm (split-K GEMM + finishing kernel)
    g2 = B.Graph(wl.ir, B.OPT_SPLITK_LN)
    kinds2 = [g2.group_info(i)["kind"] for i in range(g2.num_groups())]
    assert kinds2 == ["gemm", "attention", "gemm", "gemm", "gemm"]
    assert g.num_subgraphs() == 1
    # the Reshape's shape tensor is computed in-graph from Shape(x): its value map is known
    rs = [nd for nd in og.nodes if nd.op == "Reshape"][0]
    assert g.tensor_value(rs.ins[1]) == "[1,L,12,64]"

    g = B.Graph(WL.cfg3(layers=3).ir)
    assert g.tensor_info("idx0")[2] == "[1,floordiv(7*N0+9,10)]"
    assert g.tensor_info("keep1")[2] == "[1,floordiv(7*floordiv(7*N0+9,10)+9,10),384]"
    assert 4 not in g.tensor_info("keep2")[1]          # no nac: K is derived from shapes only
    assert g.num_subgraphs() == 1

    g = B.Graph(WL.cfg4(blocks=2).ir)
    assert g.tensor_info("blk1")[2] == "[1,64,H,W]"    # conv k=3,p=1,s=1 simplifies to exactly H, W
    assert g.tensor_info("gap")[2] == "[1,64,1,1]"

    g = B.Graph(WL.cfg5().ir)
    assert g.tensor_info("stem")[2] == "[32,64,112,112]"
    assert g.tensor_info("blk15")[2] == "[32,512,14,14]"   # Combine restores the batch extent
    assert g.num_subgraphs() == 1 + 2 * 16
    n_switch = sum(1 for i in range(g.num_ops()) if g.op_info(i)["op"] == "Switch")
    assert n_switch == 16


def test_value_propagation_and_reclassification():
    """An ISVDOS operator whose shape-determining inputs are known constants behaves as ISDOS
    (Section 3): TopK with K computed from Shape, Reshape with an in-graph shape tensor, Slice
    with constant bounds."""
    wl = WL.cfg3(layers=1)
    g = B.Graph(wl.ir)
    seen = set()
    for i in range(g.num_ops()):
        info = g.op_info(i)
        if info["op"] in ("TopK", "Reshape", "Slice"):
            assert info["cls"] == "ISVDOS" and info["eff_cls"] == "ISDOS", info
            seen.add(info["op"])
        if info["op"] == "Shape":
            assert info["cls"] == "ISDO"
    assert seen == {"TopK", "Reshape", "Slice"}
    og = O.parse(wl.ir)
    tk = [nd for nd in og.nodes if nd.op == "TopK"][0]
    assert g.tensor_value(tk.ins[1]) == "[floordiv(7*N0+9,10)]"


def test_topk_with_runtime_k_is_nac():
    ir = """
sym N 1 100
input x f32 [1,N]
input kk i64 [1]
node TopK x kk -> v i {axis=-1 largest=1 order=index}
output v
"""
    g = B.Graph(ir)
    rank, kinds, txt = g.tensor_info("v")
    assert rank == 2 and txt == "[1,nac]" and kinds == [1, 4]
    assert g.op_info(0)["eff_cls"] == "ISVDOS"


def test_fixpoint_independent_of_visiting_order():
    for wl in (WL.cfg2(layers=1, D=16, H=2, F=32), WL.cfg3(layers=2, D=16, H=2, F=32), WL.cfg5(B=4, side=16, widths=(4, 8), per_stage=1)):
        g = B.Graph(wl.ir)
        og = O.parse(wl.ir)
        names = [o for nd in og.nodes for o in nd.outs]
        ref = {n: (g.tensor_info(n), g.tensor_value(n)) for n in names}
        ref_groups = [g.group_info(i) for i in range(g.num_groups())]
        rnd = random.Random(1)
        for _ in range(3):
            order = list(range(g.num_ops()))
            rnd.shuffle(order)
            g.reanalyse(order)
            assert {n: (g.tensor_info(n), g.tensor_value(n)) for n in names} == ref
            assert [g.group_info(i) for i in range(g.num_groups())] == ref_groups
        g.reanalyse(list(reversed(range(g.num_ops()))))
        assert {n: (g.tensor_info(n), g.tensor_value(n)) for n in names} == ref
        assert g.rdp_sweeps() >= 2


def test_fig4_versions():
    """Fig. 4: with A resolved to [I,1,1] one fused version suffices; with three unrelated extents
    fusion would need 2^3 = 8 versions and the operators stay unfused."""
    g = B.Graph(WL.fig4_chain().ir)
    assert g.num_groups() == 1 and g.group_info(0)["versions"] == 1 and g.group_info(0)["n_ops"] == 2
    ir = """
sym I 1 64
sym J 1 64
sym K 1 64
sym Ip 1 64
sym Jp 1 64
sym Kp 1 64
input A f32 [Ip,Jp,Kp]
input B f32 [I,J,K]
node Sigmoid A -> s
node Add s B -> C
output C
"""
    g = B.Graph(ir)
    assert g.num_groups() == 2
    assert max(g.group_info(i)["versions"] for i in range(2)) == 8
    # binding that violates "1 or same" is caught by the recorded assertion-free max() rule:
    b = g.bind_dims(["I", "J", "K", "Ip", "Jp", "Kp"], [[4, 5, 6, 4, 1, 1]])
    assert b.shape(0, "C") == [4, 5, 6]
    # an extent pair that is neither equal nor 1 is rejected when the symbols are bound
    with pytest.raises(B.Sod2Error) as e:
        g.bind_dims(["I", "J", "K", "Ip", "Jp", "Kp"], [[4, 5, 6, 3, 1, 1]])
    assert "SHAPE_CONFLICT" in str(e.value) and "broadcast" in str(e.value)
    # multi-version fusion: the chain is fused across the three unresolved pairs, 2^3 versions, the version
    # (which extents broadcast) being chosen when the symbols are bound
    g2 = B.Graph(ir, B.OPT_MULTI_VERSION)
    assert g2.num_groups() == 1 and g2.group_info(0)["versions"] == 8 and g2.group_info(0)["n_ops"] == 2
    for vals, shape in [([4, 5, 6, 4, 1, 1], [4, 5, 6]), ([4, 5, 6, 1, 5, 1], [4, 5, 6]), ([4, 1, 6, 4, 5, 6], [4, 5, 6]), ([1, 1, 1, 2, 3, 4], [2, 3, 4])]:
        b2 = g2.bind_dims(["I", "J", "K", "Ip", "Jp", "Kp"], [vals])
        assert b2.shape(0, "C") == shape
        b2.plan()
    with pytest.raises(B.Sod2Error):
        g2.bind_dims(["I", "J", "K", "Ip", "Jp", "Kp"], [[4, 5, 6, 4, 2, 1]])


def test_backward_transfer():
    ir = """
input x f32 [?,?]
const W f32 [64,32]
node Relu x -> y
node MatMul y W -> z
output z
"""
    g = B.Graph(ir)
    # the contracted extent flows backwards MatMul -> y -> (Relu) -> x; the row count gets a fresh symbol
    assert g.tensor_info("y")[2].endswith(",64]")
    assert g.tensor_info("x")[2].endswith(",64]")
    assert g.tensor_info("z")[2].endswith(",32]")
    ir2 = """
input x f32 [?,?,?]
node Transpose x -> t {perm=2,0,1}
node Shape t -> s
output s
"""
    g = B.Graph(ir2)
    assert g.tensor_info("s")[2] == "[3]"
    # Shape's symbolic value names the unknown extents (Algorithm 1, step 3)
    assert g.tensor_value("s").count("d") == 3


def test_backward_transfer_more_operator_classes():
    # broadcast operands: where the partner's extent is the constant 1 and the output's is not, the operand must carry
    # the output's extent (an extent the partner shares stays undetermined: {1, d})
    g = B.Graph("""
input a f32 [?,?,?]
input b f32 [1,6,1]
input c f32 [?,?,?]
input d f32 [4,6,8]
const W f32 [8,16]
node Add a b -> t
node Relu t -> u
node MatMul u W -> z
node Add c d -> q
node Relu q -> v
node MatMul v W -> z2
output z
output z2
""")
    # MatMul fixes u's last extent (8), Relu hands it to t, and since b's last extent is 1 it must come from a
    assert g.tensor_info("t")[2].endswith(",8]") and g.tensor_info("a")[2].endswith(",8]")
    # c + d: d's extents are 4, 6, 8 (none is 1), so c's stay undetermined by this operator ({1, d} each): they are
    # named by fresh symbols, not copied from d
    assert g.tensor_info("q")[2].endswith(",8]") and g.tensor_info("c")[2] != "[4,6,8]"
    # Shape: the VALUE of its output is the shape of its input (backward, shape-determined-output class)
    g = B.Graph("""
sym N 1 64
input x f32 [?,?]
input y f32 [N,32]
node Shape y -> sy
node Reshape x sy -> r
node Shape r -> sr
output sr
""")
    assert g.tensor_value("sr") == "[N,32]"
    # Reshape: one unknown input extent from the element count of the known output
    g = B.Graph("""
sym N 1 64
input x f32 [?,16]
input y f32 [N,4,4]
node Shape y -> sy
node Reshape x sy -> r
output r
""")
    assert g.tensor_info("r")[2] == "[N,4,4]" and g.tensor_info("x")[2] == "[N,16]"
    # Concat: the operand left unknown on the axis takes what the others leave; off the axis it copies the output
    g = B.Graph("""
sym N 1 64
input a f32 [N,5]
input b f32 [?,?]
const W f32 [12,3]
node Concat a b -> t {axis=1}
node MatMul t W -> z
output z
""")
    assert g.tensor_info("t")[2] == "[N,12]" and g.tensor_info("b")[2] == "[N,7]"


def test_nac_partition_and_runtime_symbol():
    g = B.Graph(WL.nonzero_graph().ir)
    rank, kinds, txt = g.tensor_info("nz")
    assert rank == 2 and kinds == [1, 4] and txt == "[2,nnz(x)]"
    assert g.op_info(0)["cls"] == "EDO"
    b = g.bind_dims(["R", "C"], [[3, 5]])
    assert b.shape(0, "nz") == [2, 15]   # static upper bound numel(x)


def test_error_paths_return_codes():
    def fails(ir, code):
        with pytest.raises(B.Sod2Error) as e:
            B.Graph(ir)
        assert e.value.status_name == code, e.value

    fails("input x f32 [2,3]\nnode Bogus x -> y\noutput y\n", "SOD2_E_UNSUPPORTED_OP")
    fails("input x f32 [2,3\noutput x\n", "SOD2_E_PARSE")
    fails("input x f32 [N]\noutput x\n", "SOD2_E_PARSE")                 # undeclared symbol
    fails("input x f32 [2,3]\n", "SOD2_E_PARSE")                         # no output
    fails("input x f32 [2,3]\ninput y f32 [2,4]\nnode Add x y -> z\noutput z\n", "SOD2_E_SHAPE_CONFLICT")
    fails("input x f32 [2,3]\nnode Transpose x -> z {perm=0,1,2}\noutput z\n", "SOD2_E_RANK_MISMATCH")
    g = B.Graph(WL.cfg1().ir)
    with pytest.raises(B.Sod2Error) as e:
        g.bind_dims([], [[]])
    assert e.value.status_name == "SOD2_E_UNBOUND_SYMBOL"
    with pytest.raises(B.Sod2Error) as e:
        g.bind_dims(["N"], [[0]])
    assert e.value.status_name == "SOD2_E_BAD_DIM"
    with pytest.raises(B.Sod2Error) as e:
        g.bind_dims(["M"], [[3]])
    assert e.value.status_name == "SOD2_E_INVALID_ARG"
    # conflicting dims caught at bind time by an assertion RDP recorded
    ir = """
sym A 1 100
sym Bn 1 100
input x f32 [A,8]
input y f32 [Bn,8]
node Add x y -> z
output z
"""
    g2 = B.Graph(ir)
    b = g2.bind_dims(["A", "Bn"], [[5, 5]])
    assert b.shape(0, "z") == [5, 8]


def test_run_rejects_bad_arena_before_touching_the_device():
    wl = WL.cfg2(layers=1, D=128, H=2, F=256)
    g = B.Graph(wl.ir)
    b = g.bind_dims(["L"], [[17], [40]])
    p = b.plan()
    assert p.arena_bytes > 256
    fake = 0x10000
    with pytest.raises(B.Sod2Error) as e:
        p.run([fake], [fake], fake, 16, 0)
    assert e.value.status_name == "SOD2_E_ARENA_TOO_SMALL"
    with pytest.raises(B.Sod2Error) as e:
        p.run([fake], [fake], fake + 8, p.arena_bytes, 0)
    assert e.value.status_name == "SOD2_E_MISALIGNED"
    with pytest.raises(B.Sod2Error) as e:
        p.run([0], [fake], fake, p.arena_bytes, 0)
    assert e.value.status_name == "SOD2_E_INVALID_ARG"


def test_side_stream_only_for_a_pooling_group_that_reads_the_layout_groups_own_input():
    # A pooling group runs beside the preceding layout change only when both read the SAME tensor: the memory plan
    # knows liveness by step, so with different inputs the pooled output could be given the slot of a tensor the
    # layout kernel still reads.  Case 1: the output's layout change and the pooling both read the last block (the
    # documented case).  Case 2: the layout change reads X, the pooling reads Y and writes an arena tensor.
    C = 64
    ir1 = (f"sym H 8 64\nsym W 8 64\ninput x bf16 [1,{C},H,W]\nconst w bf16 [{C},{C},1,1]\n"
           "node Conv x w -> y {stride=1 pad=0}\nnode GlobalAveragePool y -> gp\noutput gp\noutput y\n")
    g1 = B.Graph(ir1, 0)
    p1 = g1.bind_dims(["H", "W"], [[16, 24]]).plan()
    kinds1 = [g1.group_info(i)["kind"] for i in range(g1.num_groups())]
    gi = kinds1.index("gap")
    assert kinds1[gi - 1] == "layout" and p1.group_on_side_stream(gi)
    ir2 = (f"sym H 8 64\nsym W 8 64\ninput x bf16 [1,{C},H,W]\ninput z bf16 [1,{C},H,W]\nconst w bf16 [{C},{C},1,1]\nconst v bf16 [{C},{C},1,1]\n"
           "node Conv x w -> y {stride=1 pad=0}\nnode GlobalAveragePool z -> gp\nnode Conv z v -> u {stride=1 pad=0}\nnode Sigmoid gp -> sg\n"
           "output sg\noutput y\noutput u\n")
    g2 = B.Graph(ir2, 0)
    p2 = g2.bind_dims(["H", "W"], [[16, 24]]).plan()
    kinds2 = [g2.group_info(i)["kind"] for i in range(g2.num_groups())]
    gi2 = kinds2.index("gap")
    # the group before the pooling is the layout change of the convolution output u; the pooling reads z and writes an
    # arena tensor (the Sigmoid's input): different tensors, so it stays on the main stream
    assert kinds2[gi2 - 1] == "layout" and kinds2[gi2 - 2] == "conv", kinds2
    assert not any(p2.group_on_side_stream(i) for i in range(len(kinds2))), kinds2
    assert p2.slot("gp")["bytes"] > 0
