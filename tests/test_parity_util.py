"""The comparison harness itself, on the CPU: it accepts the oracle's own output and rejects planted mistakes."""
import numpy as np
import pytest

from gen import make_layer, small_workload
from oracle import criticalkv_oracle as oc

import parity_util as pu


def _case(mode="uniform", budget=30):
    wl = small_workload(cfg_id=70, n=200, w=8, kp=5, budget_mode=mode, budget=budget)
    L = make_layer(wl)
    P, nu, sel = pu.oracle_layer(L, wl)
    Ko, Vo = oc.compact(L.K_store, L.V_store, sel["idx"], sel["offsets"])
    out = dict(attn=P.astype(np.float32), vnorm=nu.astype(np.float32), idx=sel["idx"].copy(),
               offsets=sel["offsets"].copy(), stage=sel["stage"].copy(), K_out=Ko, V_out=Vo)
    return wl, L, sel, out


@pytest.mark.parametrize("mode,budget", [("uniform", 30), ("adaptive", 70)])
def test_accepts_oracle_output(mode, budget):
    wl, L, sel, out = _case(mode, budget)
    rep = pu.check_layer_against_oracle(L, wl, out)
    assert rep["exact_heads"] == wl.Hkv and rep["differing_entries"] == 0


def test_rejects_wrong_score():
    wl, L, sel, out = _case()
    out["vnorm"][1, 17] *= 1.01
    with pytest.raises(AssertionError):
        pu.check_layer_against_oracle(L, wl, out)


def test_rejects_wrong_index_outside_tie_band():
    wl, L, sel, out = _case()
    seg = set(out["idx"][:30].tolist())
    worst = int(np.argmin(np.where(np.isin(np.arange(wl.n), list(seg)), np.inf, sel["c"][0] + sel["a"][0])))
    idx = out["idx"].copy()
    idx[0:30] = np.sort(np.array(sorted(seg - {int(out["idx"][3])}) + [worst]))
    out["idx"] = idx
    out["K_out"], out["V_out"] = oc.compact(L.K_store, L.V_store, idx, out["offsets"])
    with pytest.raises(AssertionError):
        pu.check_layer_against_oracle(L, wl, out)


def test_rejects_corrupted_gather():
    wl, L, sel, out = _case()
    out["K_out"] = out["K_out"].copy()
    out["K_out"][5, 3] += 1
    with pytest.raises(AssertionError):
        pu.check_layer_against_oracle(L, wl, out)


def test_accepts_swap_inside_tie_band():
    # two candidates for the last stage-2 slot whose scores differ by 1e-6 relative: either choice is valid
    wl, L, sel, out = _case()
    g = 0
    seg = out["idx"][:30]
    st = out["stage"][:30]
    c = sel["c"][g]
    s2 = seg[st == 2]
    last = s2[np.argmin(c[s2])]
    outside = np.setdiff1d(np.arange(wl.n), seg)
    runner = outside[np.argmax(c[outside])]
    sel2 = dict(sel)
    c2 = sel["c"].copy()
    c2[g, runner] = c2[g, last] * np.float32(1 - 1e-6)
    sel2["c"] = c2
    new_seg = np.sort(np.concatenate([np.setdiff1d(seg, [last]), [runner]]))
    idx = out["idx"].copy()
    idx[:30] = new_seg
    stage = out["stage"].copy()
    stage[:30] = np.where(np.isin(new_seg, seg[st == 1]), 1, 2)
    rep = pu.compare_selection(sel2, idx, out["offsets"], stage, n=wl.n, alpha=wl.alpha, budget_mode="uniform",
                               budget=30)
    assert rep["differing_entries"] == 2
