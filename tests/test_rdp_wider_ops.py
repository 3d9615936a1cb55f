"""Forward transfer functions of the remaining Table 2 operators (shape analysis only: these operators have
no executor).  The symbolic shapes are checked as text; bound to concrete values they are checked against
the shapes numpy / PyTorch produce for the same operator."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_2403_00176_b200 import binding as B


def _g(ir):
    return B.Graph(ir)


def test_pooling_shapes_follow_the_window_rule():
    ir = """
sym H 8 640
sym W 8 640
input x f32 [2,16,H,W]
node MaxPool x -> a {kernel=3 stride=2 pad=1}
node AveragePool a -> b {kernel=2}
node MaxUnpool b b -> c {kernel=2}
output c
"""
    g = _g(ir)
    assert g.tensor_info("a")[2] == "[2,16,floordiv(H+1,2),floordiv(W+1,2)]"   # floor((H + 2 - 3) / 2) + 1, canonical form
    assert [g.op_info(i)["cls"] for i in range(3)] == ["ISDOS", "ISDOS", "ISVDOS"]
    for h, w in [(8, 8), (9, 15), (224, 640), (33, 50)]:
        b = g.bind_dims(["H", "W"], [[h, w]])
        x = torch.zeros(2, 16, h, w)
        a = F.max_pool2d(x, 3, 2, 1)
        bb = F.avg_pool2d(a, 2)
        c = F.max_unpool2d(bb, torch.zeros_like(bb, dtype=torch.int64), 2)
        assert b.shape(0, "a") == list(a.shape) and b.shape(0, "b") == list(bb.shape) and b.shape(0, "c") == list(c.shape)


def test_expand_broadcasts_against_the_value_of_its_shape_input():
    ir = """
sym N 1 64
sym M 1 64
input x f32 [N,1,8]
input y f32 [3,M,8]
node Shape y -> sy
node Expand x sy -> e
iconst tgt i64 [4] = 2 1 5 8
node Expand x tgt -> f
output e
output f
"""
    g = _g(ir)
    # [N,1,8] against [3,M,8]: M resolves against 1, N against 3 does not (one unresolved pair, checked at bind time)
    assert g.tensor_info("e")[2] == "[max(3,N),M,8]"
    assert g.tensor_info("f")[2] == "[2,N,5,8]"
    assert g.op_info(1)["cls"] == "ISVDOS" and g.op_info(1)["eff_cls"] == "ISDOS"   # the shape value is known to RDP
    for n, m in [(3, 7), (1, 1), (1, 9)]:
        b = g.bind_dims(["N", "M"], [[n, m]])
        assert b.shape(0, "e") == list(np.broadcast_shapes((n, 1, 8), (3, m, 8)))
        assert b.shape(0, "f") == list(np.broadcast_shapes((n, 1, 8), (2, 1, 5, 8)))
    with pytest.raises(B.Sod2Error):
        g.bind_dims(["N", "M"], [[2, 4]])      # 2 against 3


def test_resize_upsample_onehot_eyelike_groupnorm():
    ir = """
sym H 4 256
sym W 4 256
sym T 1 128
input x f32 [1,8,H,W]
input idx i64 [T]
iconst depth i64 [1] = 10
iconst sizes i64 [4] = 1 8 64 96
const gs f32 [8]
const gb f32 [8]
node Resize x -> r {scales=1,1,2,2}
node Upsample r -> u {scales=1,1,1,3}
node Resize x sizes -> rs
node GroupNormalization u gs gb -> gn
node OneHot idx depth -> oh
node EyeLike gn -> ey
output ey
output rs
output oh
"""
    g = _g(ir)
    assert g.tensor_info("r")[2] == "[1,8,2*H,2*W]"
    assert g.tensor_info("u")[2] == "[1,8,2*H,6*W]"
    assert g.tensor_info("rs")[2] == "[1,8,64,96]"
    assert g.tensor_info("gn")[2] == g.tensor_info("u")[2] == g.tensor_info("ey")[2]
    assert g.tensor_info("oh")[2] == "[T,10]"
    b = g.bind_dims(["H", "W", "T"], [[5, 7, 3]])
    x = torch.zeros(1, 8, 5, 7)
    u = F.interpolate(F.interpolate(x, scale_factor=(2, 2)), scale_factor=(1, 3))
    assert b.shape(0, "u") == list(u.shape)
    assert b.shape(0, "oh") == list(F.one_hot(torch.zeros(3, dtype=torch.int64), 10).shape)


def test_non_max_suppression_is_execution_determined():
    ir = """
sym Nb 1 4096
input boxes f32 [1,Nb,4]
input scores f32 [1,3,Nb]
node NonMaxSuppression boxes scores -> sel
output sel
"""
    g = _g(ir)
    rank, kinds, txt = g.tensor_info("sel")
    assert rank == 2 and kinds == [4, 1]           # [execution determined, 3]
    assert g.op_info(0)["cls"] == "EDO"
    assert g.tensor_value("sel") == "nac"
    b = g.bind_dims(["Nb"], [[100]])
    assert b.shape(0, "sel") == [300, 3]           # planned at the static upper bound: every (class, box) pair
