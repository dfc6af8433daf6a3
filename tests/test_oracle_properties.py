"""Randomised invariants of the oracle's selection (hypothesis): sizes, disjoint stages, order, budgets."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import criticalkv_oracle as oc


@settings(max_examples=60, deadline=None)
@given(seed=st.integers(0, 10 ** 6), Hkv=st.integers(1, 4), G=st.integers(1, 3), n=st.integers(4, 90),
       frac=st.floats(0.0, 1.0), alpha=st.sampled_from([0.0, 0.25, 0.5, 0.75, 1.0]), quant=st.booleans(),
       mode=st.sampled_from(["uniform", "adaptive"]), floor=st.sampled_from([0.0, 0.5]))
def test_selection_invariants(seed, Hkv, G, n, frac, alpha, quant, mode, floor):
    r = np.random.default_rng(seed)
    P = r.random((Hkv * G, n)) ** 4
    nu = np.exp(r.standard_normal((Hkv * G, n)))
    if quant:
        P, nu = np.round(P * 5) / 5, np.round(nu)
    budget = int(frac * n) if mode == "uniform" else int(frac * n * Hkv)
    out = oc.select(P, nu, G=G, budget_mode=mode, budget=budget, alpha=alpha, adaptive_floor=floor)
    off = out["offsets"]
    assert off[0] == 0 and np.all(np.diff(off) >= 0)
    if mode == "uniform":
        assert np.all(np.diff(off) == budget)
    else:
        assert off[-1] <= budget and np.all(np.diff(off) <= n)
        if floor == 0.0:
            assert off[-1] == budget
    for g in range(Hkv):
        seg, stg = out["idx"][off[g]:off[g + 1]], out["stage"][off[g]:off[g + 1]]
        assert np.all(np.diff(seg) > 0) and (seg.size == 0 or (seg[0] >= 0 and seg[-1] < n))
        b1, b2 = oc.split_budget(seg.size, alpha)
        assert (stg == 1).sum() == b1 and (stg == 2).sum() == b2
        a, c = out["a"][g], out["c"][g]
        s1, s2 = seg[stg == 1], seg[stg == 2]
        rest = np.setdiff1d(np.arange(n), s1)
        if s1.size and rest.size:
            assert a[s1].min() >= a[rest].max()                       # stage 1 holds the largest attention scores
        out2 = np.setdiff1d(rest, s2)
        if s2.size and out2.size:
            assert c[s2].min() >= c[out2].max()                       # stage 2 the largest products among the rest
