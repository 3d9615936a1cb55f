"""Plan cache: bind + plan once per bound symbol tuple, least recently used first out."""
import pytest

from paper_2403_00176_b200 import binding as B
from paper_2403_00176_b200 import workloads as WL


def _vals(wl, j):
    return [[r.syms[s] for s in wl.sym_names] for r in wl.batch(j)]


def test_cache_disabled_by_default():
    wl = WL.cfg2(layers=2)
    g = B.Graph(wl.ir)
    with pytest.raises(B.Sod2Error) as e:
        g.plan_cached(wl.sym_names, _vals(wl, 0))
    assert "disabled" in str(e.value)


def test_hits_misses_and_lru_eviction():
    wl = WL.cfg2(layers=2)
    g = B.Graph(wl.ir)
    g.set_plan_cache(2)
    b0, p0, hit = g.plan_cached(wl.sym_names, _vals(wl, 0))
    assert not hit
    b0b, p0b, hit = g.plan_cached(wl.sym_names, _vals(wl, 0))
    assert hit and p0b.h.value == p0.h.value and b0b.h.value == b0.h.value
    _, p1, hit = g.plan_cached(wl.sym_names, _vals(wl, 1))
    assert not hit and p1.h.value != p0.h.value
    _, _, hit = g.plan_cached(wl.sym_names, _vals(wl, 0))      # batch 0 is now the most recently used
    assert hit
    _, _, hit = g.plan_cached(wl.sym_names, _vals(wl, 2))      # evicts batch 1
    assert not hit
    _, _, hit = g.plan_cached(wl.sym_names, _vals(wl, 0))
    assert hit
    _, _, hit = g.plan_cached(wl.sym_names, _vals(wl, 1))      # was evicted
    assert not hit
    # a different number of requests with the same leading values is a different key
    _, _, hit = g.plan_cached(wl.sym_names, _vals(wl, 1)[:3])
    assert not hit
    g.set_plan_cache(0)
    with pytest.raises(B.Sod2Error):
        g.plan_cached(wl.sym_names, _vals(wl, 0))


def test_cached_plan_equals_a_fresh_plan_and_survives_destroy_calls():
    wl = WL.cfg3(layers=3)
    g = B.Graph(wl.ir)
    g.set_plan_cache(4)
    vals = _vals(wl, 0)
    bc, pc, _ = g.plan_cached(wl.sym_names, vals)
    pf = g.bind_dims(wl.sym_names, vals).plan()
    assert pc.arena_bytes == pf.arena_bytes and pc.memory() == pf.memory()
    for name in ("x", wl.out_names[0] if hasattr(wl, "out_names") else "x"):
        assert bc.shape(0, name) == pf.binding.shape(0, name)
    # the library ignores destroy calls on borrowed handles
    B.lib.sod2_plan_destroy(pc.h)
    B.lib.sod2_binding_destroy(bc.h)
    _, pc2, hit = g.plan_cached(wl.sym_names, vals)
    assert hit and pc2.h.value == pc.h.value and pc2.memory() == pf.memory()


def test_bad_symbols_are_reported_and_not_cached():
    wl = WL.cfg2(layers=2)
    g = B.Graph(wl.ir)
    g.set_plan_cache(2)
    vals = _vals(wl, 0)
    vals[0][0] = 10 ** 9                                        # outside the declared range
    with pytest.raises(B.Sod2Error):
        g.plan_cached(wl.sym_names, vals)
    with pytest.raises(B.Sod2Error):
        g.plan_cached(wl.sym_names, vals)
