"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element."""
import math

import numpy as np
import pytest
import torch

from oracle import interp as O
from paper_2403_00176_b200 import binding as B
from paper_2403_00176_b200 import workloads as WL
from paper_2403_00176_b200.workloads import Request, bf16_round
from tests.gpu_harness import lockstep, run_batch
from paper_2403_00176_b200.session import Session

pytestmark = pytest.mark.gpu

F32_TOL = 1e-5     # the benchmark spec: 1e-5 relative for fp32
BF16_TOL = 2e-2    # 2e-2 max relative error for bf16 tensor-core paths


def _oracle_out(wl, req, name):
    return O.run(wl.ir, wl.consts, req.inputs)[name]


def test_cfg1_fused_group_fp32_all_requests():
    wl = WL.cfg1()
    reqs = wl.batch(0)
    # add the edge sizes: N = 1 (two rows) and N = 64
    rng = np.random.default_rng(3)
    for n in (1, 64, 33):
        reqs.append(Request({"N": n}, {"X": (rng.standard_normal((2, n, 64)) / 8).astype(np.float32)}))
    s, p, outs = run_batch(wl, reqs)
    assert s.graph.num_groups() == 1 and s.graph.group_info(0)["n_ops"] == 5
    worst = 0.0
    for r, req in enumerate(reqs):
        ref = _oracle_out(wl, req, "Y")
        assert outs[r]["Y"].shape == ref.shape == (2, req.syms["N"], 64)
        worst = max(worst, O.rel_err(outs[r]["Y"], ref))
    assert worst <= F32_TOL, worst
    # determinism: a second run is bit-identical
    p.run()
    outs2 = p.outputs()
    for a, b in zip(outs, outs2):
        assert np.array_equal(a["Y"], b["Y"])


def test_fig4_chain_one_fused_version():
    for dt, tol in (("f32", F32_TOL), ("bf16", BF16_TOL)):
        wl = WL.fig4_chain(dt)
        reqs = wl.batch(0)
        s, p, outs = run_batch(wl, reqs)
        assert s.graph.num_groups() == 1 and s.graph.group_info(0)["versions"] == 1
        for r, req in enumerate(reqs):
            assert O.rel_err(outs[r]["C"], _oracle_out(wl, req, "C")) <= tol


def test_standalone_softmax_and_layernorm_over_a_runtime_length_dim():
    # Softmax over a run-time length (the row-reduction chain kernel), alone and behind an elementwise chain, and
    # LayerNormalization forms that the packed-row LayerNorm kernel does not take (fp32 rows; a width that is not
    # a multiple of 8)
    rng = np.random.default_rng(13)
    for dt, tol in (("f32", F32_TOL), ("bf16", BF16_TOL)):
        ir = (f"sym L 1 4096\ninput x {dt} [3,5,L]\ninput m {dt} [1,5,1]\nfconst s f32 [] = 0.25\n"
              "node Softmax x -> p {axis=-1}\nnode Mul x s -> t1\nnode Add t1 m -> t2\nnode Softmax t2 -> q {axis=-1}\n"
              "output p\noutput q\n")
        rnd = (lambda a: bf16_round(a.astype(np.float32))) if dt == "bf16" else (lambda a: a.astype(np.float32))
        reqs = [Request({"L": L}, {"x": rnd(rng.standard_normal((3, 5, L)) * 3), "m": rnd(rng.standard_normal((1, 5, 1)))}) for L in (1, 17, 343, 784)]
        wl = WL.Workload("softmax_rows", dt, ir, {}, ["L"], ["p", "q"], {"batch_fn": lambda j: reqs})
        s, p, outs = run_batch(wl, reqs)
        kinds = [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())]
        assert kinds == ["chain", "chain"] and s.graph.group_info(1)["n_ops"] == 3
        for r, req in enumerate(reqs):
            env = O.run(ir, {}, req.inputs)
            for name in ("p", "q"):
                assert outs[r][name].shape == env[name].shape
                assert O.rel_err(outs[r][name], env[name]) <= tol, (dt, req.syms, name)
                assert np.allclose(outs[r][name].astype(np.float64).sum(-1), 1.0, atol=3e-2 if dt == "bf16" else 1e-5)
    for dt, D, tol in (("f32", 96, F32_TOL), ("bf16", 100, BF16_TOL), ("bf16", 2048, BF16_TOL)):
        ir = (f"sym L 1 4096\ninput x {dt} [1,L,{D}]\ninput r {dt} [1,L,{D}]\nconst g {dt} [{D}]\nconst b {dt} [{D}]\n"
              "node Add x r -> t\nnode LayerNormalization t g b -> y {axis=-1 epsilon=1e-5}\noutput y\n")
        rnd = (lambda a: bf16_round(a.astype(np.float32))) if dt == "bf16" else (lambda a: a.astype(np.float32))
        consts = {"g": rnd(rng.uniform(0.5, 1.5, D)), "b": rnd(rng.normal(0, 0.2, D))}
        reqs = [Request({"L": L}, {"x": rnd(rng.standard_normal((1, L, D)) + 0.5), "r": rnd(rng.standard_normal((1, L, D)))}) for L in (1, 9, 130)]
        wl = WL.Workload("ln_rows", dt, ir, consts, ["L"], ["y"], {"batch_fn": lambda j: reqs})
        s, p, outs = run_batch(wl, reqs)
        assert [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())] == ["chain"]
        for r, req in enumerate(reqs):
            assert O.rel_err(outs[r]["y"], O.run(ir, consts, req.inputs)["y"]) <= tol, (dt, D, req.syms)


def test_cfg1_unfused_execution_equals_fused_and_oracle():
    # fusion must equal unfused execution: the five operators of the fp32 group one kernel each (SOD2_OPT_NO_FUSION)
    wl = WL.cfg1()
    reqs = wl.batch(0)[:8] + [Request({"N": 1}, {"X": (np.random.default_rng(2).standard_normal((2, 1, 64)) / 8).astype(np.float32)})]
    s0, p0, o0 = run_batch(wl, reqs)
    s1, p1, o1 = run_batch(wl, reqs, opt_flags=B.OPT_NO_FUSION)
    assert s0.graph.num_groups() == 1 and s1.graph.num_groups() == 5
    for r, req in enumerate(reqs):
        ref = _oracle_out(wl, req, "Y")
        assert O.rel_err(o1[r]["Y"], ref) <= F32_TOL and O.rel_err(o0[r]["Y"], ref) <= F32_TOL
        assert O.rel_err(o1[r]["Y"], o0[r]["Y"]) <= F32_TOL


def test_unfused_execution_of_the_encoder_and_the_pruning_stack():
    # SOD2_OPT_NO_FUSION: one kernel per operator, every intermediate materialised in the graph's storage type
    # (attention as MatMul, Mul, Softmax, MatMul; pruning as ReduceSumSquare, TopK, Gather).  Every operator output
    # in lock-step with the oracle; the encoder's final output against the fused run.
    wl, reqs = _encoder_edge()
    reqs = [reqs[i] for i in (0, 3, 7, 10)]
    s0, p0, o0 = run_batch(wl, reqs)
    s1, p1, o1 = run_batch(wl, reqs, opt_flags=B.OPT_NO_FUSION | B.OPT_NO_REUSE)
    kinds = [s1.graph.group_info(i)["kind"] for i in range(s1.graph.num_groups())]
    assert "attention" not in kinds and kinds.count("bmm") == 4 and s1.graph.num_groups() > 2 * s0.graph.num_groups()
    for r, req in enumerate(reqs):
        errs = lockstep(wl, s1, p1, o1, r, BF16_TOL)
        assert len(errs) >= 30
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert not bad, (req.syms, bad)
        # about twice as many storage roundings as the fused run: compare with the noise of unfused bf16 storage
        ref = _oracle_out(wl, req, "y")
        noisy = O.run(wl.ir, wl.consts, req.inputs, storage_round=lambda a: bf16_round(a.astype(np.float32)).astype(np.float64))["y"]
        assert O.rel_err(o1[r]["y"], ref) <= max(BF16_TOL, 2 * O.rel_err(noisy, ref)), req.syms
    wl3 = WL.cfg3(layers=2, D=128, H=2, F=256, n_requests=1, nmin=4, nmax=800)
    rng = np.random.default_rng(17)
    reqs3 = [Request({"N0": n}, {"x": bf16_round(rng.standard_normal((1, n, 128)).astype(np.float32))}) for n in (4, 65, 300)]
    s3, p3, o3 = run_batch(wl3, reqs3, opt_flags=B.OPT_NO_FUSION | B.OPT_NO_REUSE)
    kinds3 = [s3.graph.group_info(i)["kind"] for i in range(s3.graph.num_groups())]
    assert kinds3.count("sumsq") == 2 and kinds3.count("topk") == 2 and kinds3.count("gather") == 2 and "topk_keep" not in kinds3
    for r, req in enumerate(reqs3):
        # the kept indices are decided on the stored (bf16) scores: bit-exact against the oracle's TopK of those scores
        errs = lockstep(wl3, s3, p3, o3, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert errs and not bad, (req.syms, bad)
        n = req.syms["N0"]
        for l in range(2):
            n = (7 * n + 9) // 10
            assert o3[r][f"idx{l}"].shape == (1, n) and np.all(np.diff(o3[r][f"idx{l}"][0]) > 0)


def test_guard_bands_and_poisoned_arena():
    # SOD2_OPT_GUARD_BANDS: 256 bytes behind every arena tensor and scratch region.  With the arena filled with NaN
    # bytes before the run, results must not change (nothing reads memory that nothing wrote) and every band must
    # survive (no kernel stores past the end of its tensor), on every kind of workload; a band damaged from the host
    # is found and named.
    cases = [(_encoder_edge()[0], _encoder_edge()[1][:6]), (WL.cfg3(layers=2, D=128, H=2, F=256), None), (WL.cfg4(blocks=2), None),
             (WL.cfg5(B=6, side=32, widths=(64, 128), per_stage=2), None)]
    for wl, reqs in cases:
        reqs = reqs if reqs is not None else wl.batch(0)
        if wl.meta.get("cfg") == 4:
            reqs = _conv_requests(wl, [(17, 33), (8, 200), (40, 96)])
        _, _, ref = run_batch(wl, reqs)
        s = Session(wl, opt_flags=B.OPT_GUARD_BANDS)
        p = s.prepare(reqs)
        assert p.plan.arena_bytes > 0
        p.plan.poison_arena(p.arena.data_ptr(), p.arena.numel(), s.stream)
        p.run()
        p.check_device_status()
        n_bad, name = p.plan.check_guards(p.arena.data_ptr(), s.stream)
        assert n_bad == 0, (wl.name, n_bad, name)
        got = p.outputs()
        for r in range(len(reqs)):
            for nm in ref[r]:
                assert np.array_equal(ref[r][nm], got[r][nm]), (wl.name, nm)
    # damage the band behind one tensor from the host: reported with the tensor's name
    name = "stem"
    slot = p.plan.slot(name)
    band = slot["offset"] + (slot["bytes"] + 255) // 256 * 256
    p.arena[band + 100: band + 104] = 0
    n_bad, first = p.plan.check_guards(p.arena.data_ptr(), s.stream)
    assert n_bad == 1 and first == name, (n_bad, first)


def test_expand_range_constant_of_shape_executors():
    # shape-and-value determined operators whose extents are expressions of the bound symbols: Expand against
    # Shape(y) (a copy with broadcast strides), Range(0, N, 1) and ConstantOfShape([2, N]) filled on the device
    ir = ("sym N 1 4096\ninput x bf16 [1,N,1]\ninput y bf16 [2,N,8]\niconst i0 i64 [] = 0\niconst i1 i64 [] = 1\niconst ix1 i64 [1] = 1\n"
          "iconst two i64 [1] = 2\nnode Shape y -> sy\nnode Expand x sy -> e\nnode Add e y -> z\nnode Gather sy ix1 -> nvec {axis=0}\n"
          "iconst shp0 i64 [0] =\nnode Reshape nvec shp0 -> n\nnode Range i0 n i1 -> r\nnode Concat two nvec -> cs {axis=0}\n"
          "node ConstantOfShape cs -> c {value=1.5}\noutput z\noutput e\noutput r\noutput c\n")
    rng = np.random.default_rng(4)
    reqs = [Request({"N": n}, {"x": bf16_round(rng.standard_normal((1, n, 1)).astype(np.float32)), "y": bf16_round(rng.standard_normal((2, n, 8)).astype(np.float32))})
            for n in (1, 7, 300)]
    wl = WL.Workload("expand_range", "bf16", ir, {}, ["N"], ["z", "e", "r", "c"], {"batch_fn": lambda j: reqs})
    s, p, outs = run_batch(wl, reqs)
    kinds = [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())]
    assert kinds.count("fill") == 2 and kinds.count("chain") == 2, kinds
    for r, req in enumerate(reqs):
        env = O.run(ir, {}, req.inputs)
        n = req.syms["N"]
        assert np.array_equal(outs[r]["r"], np.arange(n)) and np.array_equal(outs[r]["r"], env["r"])
        assert outs[r]["c"].shape == (2, n) and np.all(outs[r]["c"] == 1.5)
        assert outs[r]["e"].shape == (2, n, 8) and np.array_equal(outs[r]["e"].astype(np.float64), env["e"])
        assert O.rel_err(outs[r]["z"], env["z"]) <= BF16_TOL


def test_resize_upsample_nearest_executor():
    # Resize / Upsample (nearest): integer scales, and a sizes operand computed from the Shape of another runtime-sized
    # tensor (the output extents are expressions of the bound symbols); fp32 packed, bf16 behind a convolution
    # (channels-last storage), fractional ratios both up and down.  A copy: the values must be bit-exact.
    ir = ("sym H 1 512\nsym W 1 512\nsym P 1 512\nsym Q 1 512\ninput x f32 [2,3,H,W]\ninput t f32 [2,3,P,Q]\n"
          "node Resize x -> a {scales=1,1,2,3}\nnode Shape t -> st\nnode Resize x st -> b\nnode Upsample a -> c {scales=1,2,1,1}\n"
          "output a\noutput b\noutput c\n")
    rng = np.random.default_rng(12)
    reqs = [Request({"H": h, "W": w, "P": pp, "Q": q}, {"x": rng.standard_normal((2, 3, h, w)).astype(np.float32), "t": np.zeros((2, 3, pp, q), np.float32)})
            for h, w, pp, q in ((1, 1, 5, 4), (4, 5, 6, 3), (37, 29, 100, 11), (64, 96, 33, 200))]
    wl = WL.Workload("resize_f32", "f32", ir, {}, ["H", "W", "P", "Q"], ["a", "b", "c"], {"batch_fn": lambda j: reqs})
    s, p, outs = run_batch(wl, reqs)
    kinds = [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())]
    assert kinds.count("resize") == 3, kinds
    for r, req in enumerate(reqs):
        env = O.run(ir, {}, req.inputs)
        for name in ("a", "b", "c"):
            assert outs[r][name].shape == env[name].shape, (name, outs[r][name].shape, env[name].shape)
            assert np.array_equal(outs[r][name].astype(np.float64), env[name]), (r, name)
    # bf16, channels-last: 1x1 convolution -> Upsample x2 -> 1x1 convolution (the feature-pyramid pattern)
    C = 64
    ir2 = (f"sym H 1 512\nsym W 1 512\ninput x bf16 [1,{C},H,W]\nconst w1 bf16 [{C},{C},1,1]\nconst w2 bf16 [{C},{C},1,1]\n"
           "node Conv x w1 -> y {stride=1 pad=0}\nnode Resize y -> u {scales=1,1,2,2}\nnode Conv u w2 -> z {stride=1 pad=0}\noutput z\noutput u\n")
    consts = {"w1": bf16_round((rng.standard_normal((C, C, 1, 1)) / 8).astype(np.float32)), "w2": bf16_round((rng.standard_normal((C, C, 1, 1)) / 8).astype(np.float32))}
    reqs2 = [Request({"H": h, "W": w}, {"x": bf16_round(rng.standard_normal((1, C, h, w)).astype(np.float32))}) for h, w in ((8, 8), (13, 21))]
    wl2 = WL.Workload("resize_bf16", "bf16", ir2, consts, ["H", "W"], ["z", "u"], {"batch_fn": lambda j: reqs2})
    for req in reqs2:
        s2, p2, outs2 = run_batch(wl2, [req])
        env = O.run(ir2, consts, req.inputs)
        u = outs2[0]["u"].astype(np.float64)
        assert u.shape == env["u"].shape
        # the upsampled map repeats the convolution output exactly
        assert np.array_equal(u[:, :, ::2, ::2], u[:, :, 1::2, 1::2]) and np.array_equal(u[:, :, ::2, ::2], u[:, :, ::2, 1::2])
        assert O.rel_err(u, env["u"]) <= BF16_TOL and O.rel_err(outs2[0]["z"], env["z"]) <= BF16_TOL


def test_mma_issue_rate_one_cta_and_cta_pair():
    # The machine facts the GEMM versions are built on, pinned: a tcgen05.mma of 128 x 256 x 16 occupies the pipe for
    # 128 cycles and the 256 x 256 x 16 form of a CTA pair for the same 128 (both SMs at full rate); narrower
    # instructions do not get cheaper than ~74 cycles; the issuing thread's own work between stages (wait, fence,
    # commit) is not overlapped by the pipe, for either form.  Printed with -s.
    st = torch.cuda.current_stream().cuda_stream
    rows = []
    for pair in (False, True):
        for n, per_stage in ((256, 4), (128, 8), (64, 8)):
            r = [B.sod2_selftest_mma_rate(pair, n, per_stage, hs, st) for hs in (0, 1, 2)]
            rows.append((pair, n, per_stage, r))
            print(f"{'pair 256' if pair else 'one CTA 128'}x{n}x16, {per_stage} per stage: MMAs only {r[0]:.1f}, + commit {r[1]:.1f}, "
                  f"+ full/empty handshake {r[2]:.1f} cycles per MMA")
    rate = {(pair, n): r for pair, n, _, r in rows}
    for pair in (False, True):
        assert 126.0 <= rate[(pair, 256)][0] <= 132.0          # 8192 flop / clk / SM
        assert 126.0 <= rate[(pair, 256)][1] <= 134.0          # a commit per stage is free
        assert 70.0 <= rate[(pair, 128)][0] <= 80.0 and 70.0 <= rate[(pair, 64)][0] <= 80.0
        assert rate[(pair, 256)][2] >= rate[(pair, 256)][0] + 15.0    # the handshake is exposed
    # the pair is neither slower nor faster per instruction than one CTA
    for n in (256, 128, 64):
        for hs in range(3):
            assert abs(rate[(True, n)][hs] - rate[(False, n)][hs]) <= 0.05 * rate[(False, n)][hs] + 2.0
    with pytest.raises(B.Sod2Error):
        B.sod2_selftest_mma_rate(False, 96, 4, 0, st)


def test_topk_keep_with_nan_rows_keeps_exactly_k():
    # a row of NaN (an overflow upstream) has a NaN score, which compares false with everything: it must rank last, not
    # be kept by every chunk, so that exactly k rows are kept (in ascending order) and nothing is written past them
    ir = ("sym N 1 4096\ninput y bf16 [1,N,64]\niconst k i64 [1] = 5\niconst i_m1 i64 [1] = -1\n"
          "node ReduceSumSquare y -> sc {axis=-1 keepdims=0}\nnode TopK sc k -> tv idx {axis=-1 largest=1 order=index}\n"
          "node Reshape idx i_m1 -> ix\nnode Gather y ix -> keep {axis=1}\noutput keep\noutput idx\n")
    rng = np.random.default_rng(8)
    reqs = []
    for n, bad in ((12, [0, 3, 4, 5, 6, 7, 9]), (200, list(range(60, 140)))):
        y = bf16_round(rng.standard_normal((1, n, 64)).astype(np.float32))
        y[0, bad, 3] = np.nan
        reqs.append(Request({"N": n}, {"y": y}))
    wl = WL.Workload("topk_nan", "bf16", ir, {}, ["N"], ["keep", "idx"], {"batch_fn": lambda j: reqs})
    s, p, outs = run_batch(wl, reqs)
    assert [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())] == ["topk_keep"]
    for r, req in enumerate(reqs):
        y = req.inputs["y"][0].astype(np.float64)
        idx = outs[r]["idx"][0]
        assert idx.shape == (5,) and np.all(np.diff(idx) > 0)
        sc = (y * y).sum(-1)
        finite = np.flatnonzero(np.isfinite(sc))
        want = np.sort(finite[np.argsort(-sc[finite], kind="stable")[:5]])
        assert np.array_equal(idx, want), (idx, want)          # the NaN rows rank behind every finite one
        assert np.array_equal(outs[r]["keep"][0], req.inputs["y"][0][idx])


def test_bounded_wait_runs_out_and_is_reported():
    # Every device-side wait gives up after a bounded number of polls, raises the status word and returns.  The
    # self-test kernel waits on a barrier that nothing ever arrives on, with a limit of a few thousand polls: it must
    # come back by itself, and the status call must then report the timeout; the next run clears the word.
    wl, reqs = _encoder_edge(layers=1)
    s, p, outs = run_batch(wl, reqs[:3])
    p.check_device_status()
    B.sod2_selftest_bounded_wait(p.arena.data_ptr(), s.stream)
    with pytest.raises(B.Sod2Error) as e:
        p.check_device_status()
    assert e.value.status_name == "SOD2_E_TIMEOUT"
    p.run()
    p.check_device_status()
    for a, b in zip(outs, p.outputs()):
        assert np.array_equal(a["y"], b["y"])


EDGE_L = [1, 15, 16, 17, 63, 64, 65, 127, 128, 129, 200, 257, 512]


def test_multi_version_chain_version_chosen_at_bind_time():
    # extent pairs that RDP cannot resolve (three at the Add; three more at the Mul, whose left extents are
    # max(I, Ip) etc.): with multi-version fusion the three operators are one group with 2^6 versions;
    # every request of the batch binds another version (which operand broadcasts where)
    ir = """
sym I 1 64
sym J 1 64
sym K 1 640
sym Ip 1 64
sym Jp 1 64
sym Kp 1 640
input A f32 [Ip,Jp,Kp]
input B f32 [I,J,K]
node Sigmoid A -> s
node Add s B -> t
node Mul t B -> C
output C
"""
    rng = np.random.default_rng(5)
    combos = [(4, 5, 6, 4, 1, 1), (4, 5, 6, 1, 5, 1), (4, 5, 6, 1, 1, 6), (4, 5, 6, 4, 5, 6), (1, 5, 6, 4, 5, 6), (7, 1, 300, 7, 9, 1),
              (1, 1, 1, 3, 2, 5), (5, 1, 1, 1, 4, 1)]
    reqs = []
    for i_, j_, k_, ip, jp, kp in combos:
        reqs.append(Request({"I": i_, "J": j_, "K": k_, "Ip": ip, "Jp": jp, "Kp": kp},
                            {"A": rng.standard_normal((ip, jp, kp)).astype(np.float32), "B": rng.standard_normal((i_, j_, k_)).astype(np.float32)}))
    wl = WL.Workload("multi_version", "f32", ir, {}, ["I", "J", "K", "Ip", "Jp", "Kp"], ["C"], {"batch_fn": lambda j: reqs})
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_MULTI_VERSION)
    assert s.graph.num_groups() == 1 and s.graph.group_info(0)["versions"] == 64
    s0, p0, outs0 = run_batch(wl, reqs)                       # unfused: the default
    assert s0.graph.num_groups() >= 2
    for r, req in enumerate(reqs):
        ref = O.run(ir, {}, req.inputs)["C"]
        assert outs[r]["C"].shape == ref.shape, (req.syms, outs[r]["C"].shape)
        assert O.rel_err(outs[r]["C"], ref) <= F32_TOL, req.syms
        assert np.array_equal(outs[r]["C"], outs0[r]["C"])


def _encoder_edge(layers=2, F=256):
    wl = WL.cfg2(layers=layers, D=128, H=2, F=F, n_requests=1, lmin=1, lmax=512)
    rng = np.random.default_rng(11)
    reqs = [Request({"L": L}, {"x": bf16_round(rng.standard_normal((1, L, 128)).astype(np.float32))}) for L in EDGE_L]
    return wl, reqs


def test_cfg2_small_encoder_edge_lengths_lockstep():
    wl, reqs = _encoder_edge()
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    for r, req in enumerate(reqs):
        ref = _oracle_out(wl, req, "y")
        assert outs[r]["y"].shape == ref.shape
        assert O.rel_err(outs[r]["y"], ref) <= BF16_TOL
        errs = lockstep(wl, s, p, outs, r, BF16_TOL)
        assert errs, "no materialised tensor was compared"
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert not bad, (req.syms, bad)


def test_cfg2_small_encoder_layernorm_fold_against_unfolded():
    # Opt-in: a LayerNorm between two GEMMs is folded into them (the producer writes row statistics, the
    # consumers normalise in their epilogues, the normalised tensor is never stored).  Without the flag the
    # LayerNorm kernel runs: both forms meet the oracle group by group, and each other end to end.
    wl, reqs = _encoder_edge()
    s0, p0, o0 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    s1, p1, o1 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_LN_FOLD)
    k0 = [s0.graph.group_info(i)["kind"] for i in range(s0.graph.num_groups())]
    k1 = [s1.graph.group_info(i)["kind"] for i in range(s1.graph.num_groups())]
    assert k0.count("layernorm") == 4 and k1.count("layernorm") == 1
    for r, req in enumerate(reqs):
        errs = lockstep(wl, s1, p1, o1, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert errs and not bad, (req.syms, bad)
        assert O.rel_err(o1[r]["y"], o0[r]["y"]) <= BF16_TOL, req.syms
    # deterministic: the folded form gives the same bits when run again
    _, _, o2 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_LN_FOLD)
    for a, b in zip(o1, o2):
        assert np.array_equal(a["y"], b["y"])


def test_layernorm_fold_with_affine_parameters_and_offset_rows():
    # gamma, beta away from (1, 0) and rows whose mean is several standard deviations from zero: the folded
    # form subtracts mean * column-sum from the product of the raw rows, so this is where it would lose bits
    wl = WL.cfg2(layers=2, D=128, H=2, F=256, n_requests=1, lmin=1, lmax=512)
    rng = np.random.default_rng(23)
    consts = dict(wl.consts)
    n_affine = 0
    for name in list(consts):
        base = name.split(".")[-1]
        if base.startswith("g_"):
            consts[name] = bf16_round(rng.uniform(0.5, 1.5, consts[name].shape).astype(np.float32))
            n_affine += 1
        if base.startswith("be_"):
            consts[name] = bf16_round(rng.normal(0, 0.3, consts[name].shape).astype(np.float32))
    assert n_affine == 4
    wl2 = WL.Workload(wl.name, wl.dtype, wl.ir, consts, wl.sym_names, wl.outputs, wl.meta)
    reqs = [Request({"L": L}, {"x": bf16_round((rng.standard_normal((1, L, 128)) + 3.0).astype(np.float32))}) for L in (1, 77, 130, 300)]
    s, p, outs = run_batch(wl2, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_LN_FOLD)
    assert [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())].count("layernorm") == 1
    for r, req in enumerate(reqs):
        # end to end the bound is the storage noise of the two layers (as in the full-size test below); the
        # per-group bound, in lock-step, is the strict one
        ref = O.run(wl2.ir, wl2.consts, req.inputs)["y"]
        noisy = O.run(wl2.ir, wl2.consts, req.inputs, storage_round=lambda a: bf16_round(a.astype(np.float32)).astype(np.float64))["y"]
        assert O.rel_err(outs[r]["y"], ref) <= max(BF16_TOL, 2 * O.rel_err(noisy, ref))
        errs = lockstep(wl2, s, p, outs, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert errs and not bad, (req.syms, bad)


def test_gemm_chain_kernel_against_one_launch_per_gemm():
    # Opt-in: consecutive dependent GEMM groups (projection -> FFN1 -> FFN2 -> next layer's QKV, LayerNorm folded)
    # run as one persistent kernel with row-block dependency counters.  Against one launch per GEMM: fewer
    # launches, the same results within the tolerance, each form in lock-step with the oracle; run twice for
    # determinism (the counters are cleared by every run).
    wl, reqs = _encoder_edge(layers=3)
    s0, p0, o0 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    s1, p1, o1 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_LN_FOLD | B.OPT_GEMM_CHAIN)
    assert p1.run().gpu_launches < p0.run().gpu_launches
    p1.check_device_status()
    o1b = p1.outputs()
    for r, req in enumerate(reqs):
        assert np.array_equal(o1[r]["y"], o1b[r]["y"])
        assert O.rel_err(o1[r]["y"], o0[r]["y"]) <= BF16_TOL, req.syms
        for s_, p_, o_ in ((s0, p0, o0), (s1, p1, o1)):
            errs = lockstep(wl, s_, p_, o_, r, BF16_TOL)
            bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
            assert errs and not bad, (req.syms, bad)
    # a batch of several requests (several row blocks, ragged last block), with arena reuse on
    wl2 = WL.cfg2(layers=2, D=128, H=2, F=256, n_requests=6, lmin=1, lmax=300)
    reqs2 = wl2.batch(3)
    _, _, a = run_batch(wl2, reqs2)
    _, _, b = run_batch(wl2, reqs2, opt_flags=B.OPT_LN_FOLD | B.OPT_GEMM_CHAIN)
    # without the fold only FFN1 -> FFN2 chain (a LayerNorm kernel sits between the others)
    _, pc, cc = run_batch(wl2, reqs2, opt_flags=B.OPT_GEMM_CHAIN)
    for r in range(len(reqs2)):
        assert O.rel_err(cc[r]["y"], a[r]["y"]) <= BF16_TOL
    for r, req in enumerate(reqs2):
        ref = _oracle_out(wl2, req, "y")
        assert O.rel_err(b[r]["y"], ref) <= BF16_TOL and O.rel_err(a[r]["y"], ref) <= BF16_TOL


def test_cfg2_small_encoder_splitk_layernorm_groups_lockstep():
    # opt-in form of the residual GEMM + LayerNorm pair: split-K GEMM into fp32 slabs + finishing kernel
    # (F = 1024 gives the second GEMM 16 pipeline stages, i.e. several K ranges per tile)
    wl, reqs = _encoder_edge(F=1024)
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_SPLITK_LN)
    kinds = [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())]
    assert "layernorm" not in kinds
    for r, req in enumerate(reqs):
        ref = _oracle_out(wl, req, "y")
        assert O.rel_err(outs[r]["y"], ref) <= BF16_TOL
        errs = lockstep(wl, s, p, outs, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert errs and not bad, (req.syms, bad)
    # deterministic: a second run gives the same bits
    _, _, outs2 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_SPLITK_LN)
    for a, b in zip(outs, outs2):
        assert np.array_equal(a["y"], b["y"])


def test_cfg2_small_encoder_legacy_attention_kernel_lockstep():
    # the mma.sync attention kernel is the fallback for operand layouts the tensor maps cannot express
    wl, reqs = _encoder_edge()
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_LEGACY_ATTENTION)
    for r, req in enumerate(reqs):
        errs = lockstep(wl, s, p, outs, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert errs and not bad, (req.syms, bad)


def test_cfg2_small_encoder_arena_reuse_matches_no_reuse():
    wl, reqs = _encoder_edge()
    _, p1, o1 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    _, p2, o2 = run_batch(wl, reqs)
    assert p2.plan.arena_bytes < p1.plan.arena_bytes
    for a, b in zip(o1, o2):
        assert np.array_equal(a["y"], b["y"])


def test_cfg2_plan_cache_reuses_a_plan_with_other_buffers():
    # a cached plan run with fresh inputs, outputs and arena gives the bits of a freshly made plan
    wl, reqs = _encoder_edge()
    s1, p1, o1 = run_batch(wl, reqs)
    s = Session(wl)
    s.graph.set_plan_cache(2)
    names = wl.sym_names
    vals = [[r.syms[n] for n in names] for r in reqs]
    for rep in range(2):
        b, pl, hit = s.graph.plan_cached(names, vals)
        assert hit == (rep == 1)
        pr = s.prepare(reqs)                      # its own buffers and arena
        assert pr.arena.numel() >= pl.arena_bytes
        pl.run([t.data_ptr() for t in pr.in_dev], [t.data_ptr() for t in pr.out_dev], pr.arena.data_ptr(), pr.arena.numel(), s.stream)
        pl.device_status(pr.arena.data_ptr(), s.stream)
        outs = pr.outputs()
        for r in range(len(reqs)):
            assert np.array_equal(outs[r]["y"], o1[r]["y"])


def test_cuda_graph_replay_matches_stream_launches():
    # the whole launch sequence as one CUDA graph: captured by the first call, replayed by the next,
    # captured again for other buffers; bit-identical to the stream launches.  All kernel kinds: encoder
    # (GEMM, attention, LayerNorm), token pruning (scores, top-k), gated convolutions (device-side counts).
    cases = [(WL.cfg2(layers=2, D=128, H=2, F=256), "y"), (WL.cfg3(layers=2, D=128, H=2, F=256), None),
             (WL.cfg5(B=6, side=32, widths=(64, 128), per_stage=2), None)]
    for wl, _ in cases:
        reqs = wl.batch(0)
        s = Session(wl)
        a, b = s.prepare(reqs), s.prepare(reqs)          # two sets of buffers, one plan each
        a.run()
        a.check_device_status()
        ref = a.outputs()
        i1 = a.run_graph(); a.check_device_status(); o1 = a.outputs()
        i2 = a.run_graph(); a.check_device_status(); o2 = a.outputs()
        assert i1.reserved[1] == 1 and i2.reserved[1] == 0 and i1.gpu_launches == i2.gpu_launches > 0
        # the same plan with the other buffers: a new capture
        i3 = a.plan.run_graph([t.data_ptr() for t in b.in_dev], [t.data_ptr() for t in b.out_dev], b.arena.data_ptr(), b.arena.numel(), s.stream)
        assert i3.reserved[1] == 1
        o3 = b.outputs()
        for r in range(len(reqs)):
            for name in ref[r]:
                assert np.array_equal(ref[r][name], o1[r][name]) and np.array_equal(ref[r][name], o2[r][name]), (wl.name, name)
                assert np.array_equal(ref[r][name], o3[r][name]), (wl.name, name)


def test_cfg2_full_config_batch0():
    wl = WL.cfg2()
    reqs = wl.batch(0)
    s, p, outs = run_batch(wl, reqs)
    order = np.argsort([r.syms["L"] for r in reqs])
    for r in (order[0], order[len(order) // 2], order[-1]):    # shortest, median, longest request
        ref = _oracle_out(wl, reqs[r], "y")
        got = outs[r]["y"].astype(np.float64)
        # After 6 layers (about 50 roundings to bf16 storage on any implementation) the MAX error is
        # dominated by that storage noise, so end to end we bound (a) the rms error by the tolerance
        # and (b) the max error by the tolerance or twice the noise of unfused bf16-storage
        # execution of the same graph, whichever is larger.  The per-group bound is test-ed in
        # lock-step (next test), where it is well posed.
        rms = math.sqrt(np.mean((got - ref) ** 2) / np.mean(ref ** 2))
        assert rms <= BF16_TOL, rms
        noisy = O.run(wl.ir, wl.consts, reqs[r].inputs, storage_round=lambda a: bf16_round(a.astype(np.float32)).astype(np.float64))["y"]
        noise = O.rel_err(noisy, ref)
        assert O.rel_err(got, ref) <= max(BF16_TOL, 2 * noise), (O.rel_err(got, ref), noise)
        big = np.abs(ref) >= 0.25          # plain max |g - o| / |o| over elements well away from zero
        print(f"cfg2 batch 0 request {r} (L = {reqs[r].syms['L']}): end-to-end rel_err {O.rel_err(got, ref):.4f}, rms {rms:.4f}, "
              f"max |g-o|/|o| over |o| >= 0.25: {np.max(np.abs(got - ref)[big] / np.abs(ref)[big]):.4f}, "
              f"bf16-storage noise of the oracle {noise:.4f}")
    # properties that hold at any size: LayerNorm output rows have mean ~0 and unit mean-square
    for r in range(len(reqs)):
        y = outs[r]["y"][0].astype(np.float64)
        assert np.all(np.isfinite(y))
        assert np.max(np.abs(y.mean(-1))) < 2e-2
        assert np.max(np.abs((y * y).mean(-1) - 1.0)) < 5e-2
    # the launch configuration the benchmark times: the same plan replayed as one CUDA graph, same bits
    p.run_graph()
    p.run_graph()
    p.check_device_status()
    outs_graph = p.outputs()
    for r in range(len(reqs)):
        assert np.array_equal(outs[r]["y"], outs_graph[r]["y"])


def test_cfg2_full_config_lockstep_per_group():
    wl = WL.cfg2()
    reqs = wl.batch(1)
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    order = np.argsort([r.syms["L"] for r in reqs])
    for r in (order[0], order[-1]):
        errs = lockstep(wl, s, p, outs, r, BF16_TOL)
        assert len(errs) >= 6 * 7
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert not bad, bad


def _check_topk_lockstep(wl, reqs, layers):
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    banded = 0
    for r, req in enumerate(reqs):
        errs = lockstep(wl, s, p, outs, r, BF16_TOL)
        for name, v in errs.items():
            if isinstance(v, tuple):     # index mismatch: only acceptable inside the score band
                _, got, ref = v
                l = int(name[3:])
                y = p.read_arena_tensor(f"y{l}", r).astype(np.float64)[0]
                sc = np.sort((y * y).sum(-1))[::-1]
                k = ref.shape[-1]
                assert k < sc.size and abs(sc[k - 1] - sc[k]) <= 2.0 ** -40 * sc[k - 1], (req.syms, name)
                banded += 1
            else:
                assert v <= BF16_TOL, (req.syms, name, v)
        n = req.syms["N0"]
        for l in range(layers):
            n = (7 * n + 9) // 10
            assert outs[r][f"idx{l}"].shape == (1, n)
            idx = outs[r][f"idx{l}"][0]
            assert np.all(np.diff(idx) > 0)          # stable index order, no duplicates
    # the fp64 scores of bf16 squares do not depend on the summation order beyond 2^-53: the band is never needed
    assert banded == 0
    return s, p, outs


def test_cfg3_small_pruning_lockstep_and_ties():
    wl = WL.cfg3(layers=3, D=128, H=2, F=256, n_requests=1, nmin=4, nmax=800)
    rng = np.random.default_rng(5)
    reqs = []
    for n0 in (4, 5, 10, 63, 64, 65, 196, 343, 784):
        x = bf16_round(rng.standard_normal((1, n0, 128)).astype(np.float32))
        reqs.append(Request({"N0": n0}, {"x": x}))
    # exact ties: duplicated token rows must keep the lower index
    x = bf16_round(rng.standard_normal((1, 40, 128)).astype(np.float32))
    x[0, 20:40] = x[0, 0:20]
    reqs.append(Request({"N0": 40}, {"x": x}))
    # a request of several 64-token chunks with ties across the chunk boundaries
    x = bf16_round(rng.standard_normal((1, 300, 128)).astype(np.float32))
    x[0, 120:140] = x[0, 100:120]
    x[0, 250:270] = x[0, 100:120]
    reqs.append(Request({"N0": 300}, {"x": x}))
    _check_topk_lockstep(wl, reqs, 3)


def test_more_requests_than_one_attention_or_pruning_launch_holds():
    # attention and the pruning step take up to 32 requests per launch: 40 requests make them launch twice
    rng = np.random.default_rng(31)
    wl2 = WL.cfg2(layers=1, D=128, H=2, F=256, n_requests=1, lmin=1, lmax=512)
    reqs2 = [Request({"L": int(L)}, {"x": bf16_round(rng.standard_normal((1, int(L), 128)).astype(np.float32))}) for L in rng.integers(1, 90, 40)]
    s, p, outs = run_batch(wl2, reqs2)
    for r in (0, 17, 31, 32, 39):
        assert O.rel_err(outs[r]["y"], _oracle_out(wl2, reqs2[r], "y")) <= BF16_TOL, reqs2[r].syms
    wl3 = WL.cfg3(layers=2, D=128, H=2, F=256, n_requests=1, nmin=4, nmax=800)
    reqs3 = [Request({"N0": int(n)}, {"x": bf16_round(rng.standard_normal((1, int(n), 128)).astype(np.float32))}) for n in rng.integers(4, 150, 40)]
    _check_topk_lockstep(wl3, reqs3, 2)


def test_cfg3_full_config_batch0_lockstep():
    # the whole 16-request batch (about 8000 tokens in layer 0: the tile versions and the two-launch request
    # tables the bench times), every request in lock-step with the oracle through all 12 layers
    wl = WL.cfg3()
    reqs = wl.batch(0)
    assert len(reqs) == 16
    _check_topk_lockstep(wl, reqs, 12)


def test_nonzero_compaction():
    wl = WL.nonzero_graph()
    reqs = wl.batch(0)
    rng = np.random.default_rng(9)
    reqs.append(Request({"R": 3, "C": 5}, {"x": np.zeros((3, 5), np.float32)}))          # all zero
    reqs.append(Request({"R": 7, "C": 300}, {"x": np.ones((7, 300), np.float32)}))       # all non-zero
    big = rng.standard_normal((700, 900)).astype(np.float32)
    big[rng.uniform(size=big.shape) < 0.7] = 0
    reqs.append(Request({"R": 700, "C": 900}, {"x": big}))
    s, p, outs = run_batch(wl, reqs)
    for r, req in enumerate(reqs):
        ref = O.run(wl.ir, wl.consts, req.inputs)["nz"] if req.inputs["x"].size < 5000 else np.array(np.nonzero(req.inputs["x"]))
        assert outs[r]["nz"].shape == ref.shape
        assert np.array_equal(outs[r]["nz"], ref)


# ------------------------------------------------------------------------------------------------ cfg 4
def _conv_requests(wl, shapes, seed=17):
    rng = np.random.default_rng(seed)
    return [Request({"H": h, "W": w}, {"x": bf16_round(rng.uniform(-1, 1, (1, 64, h, w)).astype(np.float32))}) for h, w in shapes]


def test_cfg4_small_conv_stage_edge_shapes_lockstep():
    wl = WL.cfg4(blocks=3)
    shapes = [(1, 1), (3, 5), (8, 16), (16, 8), (17, 33), (4, 130), (33, 40), (64, 64)]
    reqs = _conv_requests(wl, shapes)
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    kinds = [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())]
    assert kinds == ["layout", "conv", "conv", "conv", "layout", "gap"]
    for r, req in enumerate(reqs):
        env = O.run(wl.ir, wl.consts, req.inputs)
        for name in ("blk2", "gap"):
            assert outs[r][name].shape == env[name].shape
            assert O.rel_err(outs[r][name], env[name]) <= BF16_TOL, (req.syms, name)
        errs = lockstep(wl, s, p, outs, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert not bad, (req.syms, bad)
    # determinism
    p.run()
    outs2 = p.outputs()
    for a, b in zip(outs, outs2):
        assert np.array_equal(a["blk2"], b["blk2"]) and np.array_equal(a["gap"], b["gap"])


def test_cfg4_more_requests_than_one_launch_holds():
    # layout changes, row-halo convolutions and pooling take up to eight requests per launch: nineteen requests
    # (wide rows for the row-halo kernel, narrow ones for the general kernel, mixed) make every group flush twice
    wl = WL.cfg4(blocks=2)
    rng = np.random.default_rng(23)
    shapes = [(int(rng.integers(1, 12)), int(rng.choice([5, 40, 96, 128, 130, 200]))) for _ in range(19)]
    reqs = _conv_requests(wl, shapes, seed=29)
    s, p, outs = run_batch(wl, reqs)
    for r, req in enumerate(reqs):
        env = O.run(wl.ir, wl.consts, req.inputs)
        for name in ("blk1", "gap"):
            assert outs[r][name].shape == env[name].shape
            assert O.rel_err(outs[r][name], env[name]) <= BF16_TOL, (req.syms, name)


def test_cfg4_rows_of_640_pixels_meet_the_oracle():
    # the widest row of the workload (five 128-pixel tiles per row in the row-halo kernel) on a few rows, beside
    # a width that is not a multiple of the tile
    wl = WL.cfg4(blocks=3)
    reqs = _conv_requests(wl, [(8, 640), (5, 608), (3, 130)], seed=41)
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    for r, req in enumerate(reqs):
        env = O.run(wl.ir, wl.consts, req.inputs)
        for name in ("blk2", "gap"):
            assert O.rel_err(outs[r][name], env[name]) <= BF16_TOL, (req.syms, name)
        errs = lockstep(wl, s, p, outs, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert errs and not bad, (req.syms, bad)


def test_cfg4_full_config_smallest_and_largest_request_and_properties():
    wl = WL.cfg4()
    reqs = wl.batch(0)
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    order = np.argsort([r.syms["H"] * r.syms["W"] for r in reqs])
    last = [n for n in outs[0] if n.startswith("blk")][0]
    r = int(order[0])
    env = O.run(wl.ir, wl.consts, reqs[r].inputs)
    assert O.rel_err(outs[r][last], env[last]) <= BF16_TOL
    assert O.rel_err(outs[r]["gap"], env["gap"]) <= BF16_TOL
    # the largest image of the batch, block by block in lock-step (every block output from the GPU's own block input)
    r = int(order[-1])
    errs = lockstep(wl, s, p, outs, r, BF16_TOL)
    assert sum(k.startswith("blk") for k in errs) >= 7, sorted(errs)
    bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
    assert not bad, (reqs[r].syms, bad)
    # the default plan (arena reuse on) gives the same bits
    _, _, outs_reuse = run_batch(wl, reqs)
    for r in range(len(reqs)):
        assert np.array_equal(outs[r][last], outs_reuse[r][last]) and np.array_equal(outs[r]["gap"], outs_reuse[r]["gap"])
    for r in range(len(reqs)):   # properties at any size: shapes, finiteness, gap == mean of the returned map
        y = outs[r][last].astype(np.float64)
        assert y.shape == (1, 64, reqs[r].syms["H"], reqs[r].syms["W"]) and np.all(np.isfinite(y))
        assert np.allclose(outs[r]["gap"].reshape(-1), y.mean(axis=(2, 3)).reshape(-1), rtol=1e-2, atol=1e-2)


@pytest.mark.parametrize("C", [64, 1088])
def test_global_average_pool_sums_are_exact_over_a_wide_range(C):
    """The pooling kernel adds groups of eight inputs in fp32 where that is provably exact and in fp64
    where it is not.  Inputs 26 binades apart that cancel across the image: any fp32 shortcut taken
    where it is not exact loses the small terms, and the mean with them."""
    H, W = 48, 40
    ir = (f"input x bf16 [1,{C},{H},{W}]\nconst w bf16 [{C},{C},1,1]\nconst b bf16 [{C}]\n"
          "node Conv x w b -> c1 {kernel=1 stride=1 pad=0}\nnode Relu c1 -> r2\nnode Add x r2 -> y\n"
          "node GlobalAveragePool y -> gap\noutput gap\noutput y\n")
    consts = {"w": np.zeros((C, C, 1, 1), np.float32), "b": np.zeros((C,), np.float32)}   # y == x
    rng = np.random.default_rng(C)
    x = np.full((1, C, H, W), 2.0 ** -6, np.float32)
    x[0, 1::4] = bf16_round(rng.uniform(-2, 2, (len(range(1, C, 4)), H, W)).astype(np.float32))   # ordinary channels
    x[0, 2::4] = 0.0
    x[0, 2::4, ::3, ::5] = -0.0
    big = 2.0 ** 20
    x[0, 0::4, 0, 0] = big
    x[0, 0::4, H - 1, W - 1] = -big
    x[0, 3::4, H // 2, 3] = big
    x[0, 3::4, 1, W - 2] = -big
    wl = WL.Workload("gap_exact", "bf16", ir, consts, [], ["gap", "y"], {})
    s, p, outs = run_batch(wl, [Request({}, {"x": x})])
    assert np.array_equal(outs[0]["y"].astype(np.float32), x)
    exact = bf16_round(x.astype(np.float64).mean(axis=(2, 3)).astype(np.float32)).reshape(-1)
    got = outs[0]["gap"].astype(np.float32).reshape(-1)
    assert exact[0] == bf16_round(np.float32((H * W - 2) * 2.0 ** -6 / (H * W)))   # the small terms ARE the mean
    assert np.array_equal(got, exact), np.flatnonzero(got != exact)[:8]


def _gemm_graph(K, N, act, residual):
    lines = ["sym M 1 4096", f"input x bf16 [1,M,{K}]"]
    if residual:
        lines.append(f"input r bf16 [1,M,{N}]")
    lines += [f"const W bf16 [{K},{N}]", f"const b bf16 [{N}]", "node MatMul x W -> t0", "node Add t0 b -> t1"]
    cur = "t1"
    if act:
        lines.append(f"node {act} {cur} -> t2"); cur = "t2"
    if residual:
        lines.append(f"node Add {cur} r -> t3"); cur = "t3"
    lines.append(f"node Relu {cur} -> y" if residual and not act else f"node Add {cur} b -> y")
    lines.append("output y")
    return "\n".join(lines) + "\n"


def test_gemm_epilogue_forms_ragged_shapes():
    # the tcgen05 GEMM group over row counts around the 128-row tile, column counts that are not
    # multiples of the 64-column pass (8-column granularity) and K of one to several 64-chunks, in every
    # epilogue form: bias, bias+ReLU, bias+GELU, bias+residual(+ReLU)
    rng = np.random.default_rng(7)
    cases = [(64, 8, None, False), (64, 72, "Relu", False), (192, 136, "Gelu", False), (128, 264, None, True),
             (320, 520, "Gelu", False), (64, 768, None, True)]
    for K, N, act, residual in cases:
        ir = _gemm_graph(K, N, act, residual)
        consts = {"W": bf16_round((rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32)),
                  "b": bf16_round(rng.standard_normal(N).astype(np.float32))}
        reqs = []
        for M in (1, 127, 128, 129, 300):
            ins = {"x": bf16_round(rng.standard_normal((1, M, K)).astype(np.float32))}
            if residual:
                ins["r"] = bf16_round(rng.standard_normal((1, M, N)).astype(np.float32))
            reqs.append(Request({"M": M}, ins))
        wl = WL.Workload("gemm_case", "bf16", ir, consts, ["M"], ["y"], {"batch_fn": lambda j: reqs})
        s, p, outs = run_batch(wl, reqs)
        kinds = [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())]
        assert kinds[0] == "gemm", kinds
        for r, req in enumerate(reqs):
            ref = O.run(ir, consts, req.inputs)["y"]
            assert outs[r]["y"].shape == ref.shape
            assert O.rel_err(outs[r]["y"], ref) <= BF16_TOL, (K, N, act, residual, req.syms)


def test_gemm_on_cta_pairs_matches_the_single_cta_kernel_and_the_oracle():
    # SOD2_OPT_GEMM_PAIR: two CTAs of a cluster share a 256-row tile (tcgen05.mma.cta_group::2), each loading its own
    # rows and half of the weight tile.  Row counts around the 256-row pair tile (an odd number of 128-row tiles leaves
    # the second CTA of the last pair without rows), both tile widths, every epilogue form; against the oracle and
    # against the single-CTA kernel.  SOD2_GEMM_PAIR_FORCE makes the planner take the pair kernel wherever it can.
    import os
    os.environ["SOD2_GEMM_PAIR_FORCE"] = "1"
    try:
        rng = np.random.default_rng(19)
        # (the last two shapes are wide enough for the planner to take the 256-wide pair tile at 1929 rows)
        cases = [(64, 256, None, False), (128, 136, "Relu", False), (192, 768, "Gelu", False), (768, 768, None, True), (320, 520, "Gelu", False),
                 (128, 2304, None, False), (64, 2048, "Gelu", True)]
        for K, N, act, residual in cases:
            ir = _gemm_graph(K, N, act, residual)
            consts = {"W": bf16_round((rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32)),
                      "b": bf16_round(rng.standard_normal(N).astype(np.float32))}
            reqs = []
            for M in (129, 256, 257, 385, 902):
                ins = {"x": bf16_round(rng.standard_normal((1, M, K)).astype(np.float32))}
                if residual:
                    ins["r"] = bf16_round(rng.standard_normal((1, M, N)).astype(np.float32))
                reqs.append(Request({"M": M}, ins))
            wl = WL.Workload("gemm_pair_case", "bf16", ir, consts, ["M"], ["y"], {"batch_fn": lambda j: reqs})
            # one request per plan (each its own row count), then all of them packed into one launch (1929 rows)
            for group in ([[r] for r in reqs] + [reqs]):
                s1, p1, o1 = run_batch(wl, group, opt_flags=B.OPT_GEMM_PAIR)
                s0, p0, o0 = run_batch(wl, group)
                for r, req in enumerate(group):
                    ref = O.run(ir, consts, req.inputs)["y"]
                    assert O.rel_err(o1[r]["y"], ref) <= BF16_TOL, (K, N, act, residual, req.syms)
                    assert O.rel_err(o1[r]["y"], o0[r]["y"]) <= 1e-2, (K, N, act, residual, req.syms)
                p1.run()
                for a, b_ in zip(o1, p1.outputs()):
                    assert np.array_equal(a["y"], b_["y"])
        # the encoder with every eligible GEMM on pairs
        wl, reqs = _encoder_edge()
        s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | B.OPT_GEMM_PAIR)
        for r, req in enumerate(reqs):
            errs = lockstep(wl, s, p, outs, r, BF16_TOL)
            bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
            assert errs and not bad, (req.syms, bad)
    finally:
        del os.environ["SOD2_GEMM_PAIR_FORCE"]


def test_branched_graph_planned_order_matches_default_order_and_oracle():
    # static execution planning reorders the groups of a branched graph (smaller live peak); the result
    # is bit-identical to the default order's and agrees with the oracle
    from tests.test_execution_order import _branched_graph
    import random
    rnd = random.Random(21)
    ir = _branched_graph(rnd, 4)
    g = O.parse(ir)
    rng = np.random.default_rng(3)
    consts = {}
    for ln in ir.splitlines():
        if ln.startswith("const"):
            _, name, _, shp = ln.split()
            k, n = [int(v) for v in shp.strip("[]").split(",")]
            consts[name] = bf16_round((rng.standard_normal((k, n)) / np.sqrt(k)).astype(np.float32))
    reqs = [Request({"N": n}, {"x": bf16_round(rng.standard_normal((1, n, 64)).astype(np.float32))}) for n in (2, 130, 515)]
    out_name = [ln.split()[1] for ln in ir.splitlines() if ln.startswith("output")][0]
    wl = WL.Workload("branched", "bf16", ir, consts, ["N"], [out_name], {"batch_fn": lambda j: reqs})
    s1, p1, o1 = run_batch(wl, reqs)
    s2, p2, o2 = run_batch(wl, reqs, opt_flags=B.OPT_NO_SEP)
    info = s1.graph.order_info()
    assert info["reordered_subgraphs"] == 1 and info["planned_peak_hi"] < info["default_peak_hi"]
    assert p1.plan.memory()["peak_live_bytes"] < p2.plan.memory()["peak_live_bytes"]
    assert p1.plan.memory()["arena_bytes"] < p2.plan.memory()["arena_bytes"]
    s3, p3, o3 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)   # planned order, every intermediate kept
    for r, req in enumerate(reqs):
        assert np.array_equal(o1[r][out_name], o2[r][out_name]) and np.array_equal(o1[r][out_name], o3[r][out_name])
        assert O.rel_err(o1[r][out_name], _oracle_out(wl, req, out_name)) <= BF16_TOL
        errs = lockstep(wl, s3, p3, o3, r, BF16_TOL)
        bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
        assert errs and not bad, (req.syms, bad)


def test_rgb_stem_convolution_fused_kernel_shapes():
    # the fused 7x7 / stride 2 / 3 -> 64 stem: image widths that are (not) multiples of 8 (16-byte and
    # element-wise patch copies), odd heights, one to three 128-pixel segments per output row, several
    # images per request and requests of different sizes in one batch; with and without the ReLU
    rng = np.random.default_rng(23)
    for relu in (True, False):
        lines = ["sym H 8 1024", "sym W 8 1024", "input x bf16 [2,3,H,W]", "const w bf16 [64,3,7,7]", "const b bf16 [64]",
                 "node Conv x w b -> c {kernel=7 stride=2 pad=3}" if relu else "node Conv x w b -> y {kernel=7 stride=2 pad=3}"]
        if relu:
            lines.append("node Relu c -> y")
        lines.append("output y")
        ir = "\n".join(lines) + "\n"
        consts = {"w": bf16_round((rng.standard_normal((64, 3, 7, 7)) / np.sqrt(147)).astype(np.float32)),
                  "b": bf16_round((rng.standard_normal(64) * 0.1).astype(np.float32))}
        shapes = [(32, 32), (30, 36), (17, 8), (224, 224), (70, 520)] if relu else [(33, 72), (64, 260)]
        reqs = [Request({"H": h, "W": w}, {"x": bf16_round(rng.uniform(-1, 1, (2, 3, h, w)).astype(np.float32))}) for h, w in shapes]
        wl = WL.Workload("stem", "bf16", ir, consts, ["H", "W"], ["y"], {"batch_fn": lambda j: reqs})
        s, p, outs = run_batch(wl, reqs)
        kinds = [s.graph.group_info(i)["kind"] for i in range(s.graph.num_groups())]
        assert "conv" in kinds, kinds
        assert p.plan.memory()["arena_bytes"] < 8 << 20       # the conv outputs (5.7 MB), no patch matrix (9.6 MB more)
        for r, req in enumerate(reqs):
            ref = O.run(ir, consts, req.inputs)["y"]
            assert outs[r]["y"].shape == ref.shape, (req.syms, outs[r]["y"].shape, ref.shape)
            assert O.rel_err(outs[r]["y"], ref) <= BF16_TOL, (req.syms, O.rel_err(outs[r]["y"], ref))


# ------------------------------------------------------------------------------------------------ cfg 5
def _check_gated(wl, reqs, n_blocks, extra_flags=0):
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE | extra_flags)
    req = reqs[0]
    env = O.run(wl.ir, wl.consts, req.inputs)
    # lock-step: every full-batch tensor (stem, block outputs, gates) from the GPU's own inputs
    errs = lockstep(wl, s, p, outs, 0, BF16_TOL)
    assert any(k.startswith("blk") for k in errs)
    bad = {k: v for k, v in errs.items() if not (isinstance(v, float) and v <= BF16_TOL)}
    assert not bad, bad
    gates = np.stack([outs[0][f"gate{i}"].reshape(-1) for i in range(n_blocks)])
    # gate decisions recomputed by the oracle from the GPU's own block inputs must match bit-exactly
    g = O.parse(wl.ir)
    over = {n: p.read_arena_tensor(n, 0).astype(np.float64) for n in ["stem"] + [f"blk{i}" for i in range(n_blocks - 1)]}
    comp = {}
    env2 = O.run(wl.ir, wl.consts, req.inputs, overrides=over, g=g, computed=comp)
    for i in range(n_blocks):
        assert np.array_equal(outs[0][f"gate{i}"].reshape(-1).astype(bool), env2[f"gate{i}"].reshape(-1)), i
    assert O.rel_err(outs[0]["gap"], env2["gap"]) <= BF16_TOL
    # free-running agreement (information + sanity): same decisions unless a logit is within rounding noise
    free = np.stack([env[f"gate{i}"].reshape(-1) for i in range(n_blocks)])
    assert (gates.astype(bool) == free).mean() >= 0.9
    return gates


def test_cfg5_small_gated_network_lockstep():
    wl = WL.cfg5(B=6, side=32, widths=(64, 128), per_stage=2)
    gates = _check_gated(wl, wl.batch(0), 4)
    assert gates.shape == (4, 6)


def test_cfg5_more_samples_than_a_warp_of_gate_lanes():
    # 45 samples: the one-CTA gate kernel walks its 32 warps over the images twice and partitions two chunks of ids
    wl = WL.cfg5(B=45, side=32, widths=(64,), per_stage=2, calibrated=False)
    gates = _check_gated(wl, wl.batch(0), 2)
    assert gates.shape == (2, 45) and 0 < gates.sum() < gates.size


def test_cfg5_small_gated_network_copy_regroup_lockstep():
    # Switch / Combine as whole-sample copies (the form used where the index-indirect pattern does not apply)
    wl = WL.cfg5(B=6, side=32, widths=(64, 128), per_stage=2)
    gates = _check_gated(wl, wl.batch(0), 4, extra_flags=B.OPT_COPY_REGROUP)
    assert gates.shape == (4, 6)
    # the default form plans no storage for the regrouped copies
    g0, g1 = B.Graph(wl.ir), B.Graph(wl.ir, B.OPT_COPY_REGROUP)
    m0 = g0.bind_dims(wl.sym_names, [[]]).plan().memory()
    m1 = g1.bind_dims(wl.sym_names, [[]]).plan().memory()
    assert m0["sum_bytes"] < m1["sum_bytes"]


def test_cfg5_small_in_place_blocks_match_the_no_reuse_run():
    # default flags: identity-shortcut blocks run in place (the Combine output takes over the Switch
    # input's storage); OPT_NO_REUSE keeps every intermediate in its own buffer.  Same bits either way.
    wl = WL.cfg5(B=6, side=32, widths=(64, 128), per_stage=3)
    reqs = wl.batch(0)
    s0, p0, o0 = run_batch(wl, reqs)
    s1, p1, o1 = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    assert p0.plan.memory()["sum_bytes"] < p1.plan.memory()["sum_bytes"]
    for name in o0[0]:
        assert np.array_equal(o0[0][name], o1[0][name]), name
    env = O.run(wl.ir, wl.consts, reqs[0].inputs)
    assert O.rel_err(o0[0]["gap"], env["gap"]) <= BF16_TOL


def test_cfg5_all_skip_and_all_execute():
    # degenerate gate batches: nothing executes (Bx = 0 launches no tile) / everything executes
    for bias_val in (-50.0, 50.0):
        wl = WL.cfg5(B=4, side=32, widths=(64, 128), per_stage=2)
        for k in list(wl.consts):
            if k.endswith(".gb"):
                wl.consts[k] = np.full_like(wl.consts[k], bias_val)
        gates = _check_gated(wl, wl.batch(1), 4)
        assert np.all(gates == (1 if bias_val > 0 else 0))


def test_cfg5_exact_staging_matches_the_bounded_run():
    # Execution-determined extents handled exactly (counts read back after every Switch, the remaining sub-graphs
    # planned again at their true sizes around the tensors in place) against the default bounded form (counts stay on
    # the device, memory planned at the upper bound): same kernels, same bits, one stage per Switch, no larger arena
    cases = [(WL.cfg5(B=6, side=32, widths=(64, 128), per_stage=2), 4, 0), (WL.cfg5(B=6, side=32, widths=(64, 128), per_stage=3), 6, B.OPT_COPY_REGROUP),
             (WL.cfg5(B=45, side=32, widths=(64,), per_stage=2, calibrated=False), 2, 0)]
    for bias_val in (-50.0, 50.0):                       # nothing executes (empty sub-batches) / everything executes
        wl = WL.cfg5(B=4, side=32, widths=(64, 128), per_stage=2)
        for k in list(wl.consts):
            if k.endswith(".gb"):
                wl.consts[k] = np.full_like(wl.consts[k], bias_val)
        cases.append((wl, 4, 0))
    for wl, n_blocks, flags in cases:
        reqs = wl.batch(0)
        s, p, ref = run_batch(wl, reqs, opt_flags=flags)
        info = p.run_exact()
        p.check_device_status()
        got = p.outputs()
        assert info.reserved[2] == n_blocks + 1, info.reserved[2]          # the first stage + one per Switch
        assert 0 < info.reserved[3] <= p.plan.arena_bytes
        for name in ref[0]:
            assert np.array_equal(ref[0][name], got[0][name]), (wl.name, name)
        # and again (the stages leave nothing behind), then the bounded form on the same buffers
        p.run_exact()
        again = p.outputs()
        p.run()
        bounded = p.outputs()
        for name in ref[0]:
            assert np.array_equal(ref[0][name], again[0][name]) and np.array_equal(ref[0][name], bounded[0][name])
    # a graph without execution-determined operators is one stage
    wl2, reqs2 = _encoder_edge(layers=1)
    s2, p2, o2 = run_batch(wl2, reqs2[:4])
    i2 = p2.run_exact()
    assert i2.reserved[2] == 1
    for a, b_ in zip(o2, p2.outputs()):
        assert np.array_equal(a["y"], b_["y"])


def test_cfg5_full_depth_reduced_batch_lockstep():
    # all 16 blocks and widths 64..512 at 224x224, 4 images (the oracle needs ~100 GFLOP in fp64)
    wl = WL.cfg5(B=4)
    gates = _check_gated(wl, wl.batch(0), 16)
    assert gates.shape == (16, 4)


def _gate_subgraph(full, i):
    """The operators between a block's input tensor and its gate (pool -> reshape -> linear -> compare) as a graph of
    their own for the oracle: input = the block input, output = gate i."""
    prod = {o: nd for nd in full.nodes for o in nd.outs}
    chain, t = [], f"gate{i}"
    while prod[t].op != "GlobalAveragePool":
        chain.append(prod[t])
        t = prod[t].ins[0]
    chain.append(prod[t])
    g = O.Graph()
    g.inputs = {chain[-1].ins[0]: ("bf16", [])}
    g.consts = {n: full.consts[n] for nd in chain for n in nd.ins if n in full.consts}
    g.inline = full.inline
    g.nodes = chain[::-1]
    return g, chain[-1].ins[0]


def test_cfg5_full_config_gate_bits_of_all_blocks_from_the_gpu_block_inputs():
    # B = 32 at full depth: the oracle cannot afford the convolutions, but it can recompute every decision.  For each of
    # the 16 blocks the gate chain runs in the oracle on the GPU's own block input (all 32 samples): bits must match
    wl = WL.cfg5()
    reqs = wl.batch(0)
    s, p, outs = run_batch(wl, reqs, opt_flags=B.OPT_NO_REUSE)
    full = O.parse(wl.ir)
    n_exec = 0
    for i in range(16):
        g, src = _gate_subgraph(full, i)
        x = p.read_arena_tensor(src, 0).astype(np.float64)
        assert x.shape[0] == 32
        env = O.run("", {n: wl.consts[n] for n in g.consts}, {src: x}, g=g)
        want = env[f"gate{i}"].reshape(-1).astype(bool)
        got = outs[0][f"gate{i}"].reshape(-1).astype(bool)
        assert np.array_equal(got, want), (i, np.flatnonzero(got != want), env[f"logit{i}"].reshape(-1)[got != want])
        n_exec += int(got.sum())
    assert 0 < n_exec < 16 * 32
    # and the default plan (in-place blocks, arena reuse) takes the same decisions and returns the same pooled output
    _, _, o2 = run_batch(wl, reqs)
    for i in range(16):
        assert np.array_equal(outs[0][f"gate{i}"], o2[0][f"gate{i}"])
    assert np.array_equal(outs[0]["gap"], o2[0]["gap"])


def test_cfg5_full_config_properties():
    wl = WL.cfg5()
    reqs = wl.batch(0)
    s, p, outs = run_batch(wl, reqs)
    assert s.graph.num_subgraphs() == 33
    gates = np.stack([outs[0][f"gate{i}"].reshape(-1) for i in range(16)])
    assert gates.shape == (16, 32) and set(np.unique(gates)) <= {0, 1}
    assert np.all(np.isfinite(outs[0]["gap"])) and outs[0]["gap"].shape == (32, 512, 1, 1)
    assert 0.05 < gates.mean() < 0.95          # both branches are exercised
    p.run()
    outs2 = p.outputs()
    assert np.array_equal(outs[0]["gap"], outs2[0]["gap"])
    for i in range(16):
        assert np.array_equal(outs[0][f"gate{i}"], outs2[0][f"gate{i}"])
    print("skip fraction per block:", 1 - gates.mean(axis=1))
