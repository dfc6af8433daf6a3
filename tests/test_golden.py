"""Stored oracle output on configuration 0 (written by tests/golden/make_golden.py from the oracle alone)."""
import json
import os

import numpy as np
import pytest

from gen import config, make_layer
from oracle import criticalkv_oracle as oc

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "cfg0_oracle.json")


def _golden():
    with open(GOLDEN) as f:
        return json.load(f)


def test_oracle_reproduces_its_stored_output():
    g = _golden()
    wl = config(0)
    L = make_layer(wl, 0)
    out = oc.compress_layer(L.Qw, L.K, L.V, L.WO, kp=wl.kp, budget_mode=wl.budget_mode, budget=wl.budget,
                            alpha=wl.alpha, eps=wl.eps, scale=wl.scale)
    assert out["offsets"].tolist() == g["offsets"]
    assert out["idx"].tolist() == g["idx"] and out["stage"].tolist() == g["stage"]
    for h, i, v in g["attn_probe"]:
        assert abs(out["P"][h, i] - v) <= 1e-12 * max(abs(v), 1e-300) + 1e-300
    for h, i, v in g["vnorm_probe"]:
        assert abs(out["nu"][h, i] - v) <= 1e-12 * abs(v)


@pytest.mark.gpu
def test_gpu_selection_matches_stored_oracle_selection():
    import parity_util as pu
    from gpu_util import run_layers
    g = _golden()
    wl = config(0)
    L = make_layer(wl, 0)
    outs, _ = run_layers([L], wl)
    out = outs[0]
    assert out["offsets"].tolist() == g["offsets"]
    assert out["idx"].tolist() == g["idx"] and out["stage"].tolist() == g["stage"]
    for h, i, v in g["attn_probe"]:
        assert abs(out["attn"][h, i] - v) <= pu.SCORE_RTOL * abs(v)
    for h, i, v in g["vnorm_probe"]:
        assert abs(out["vnorm"][h, i] - v) <= pu.SCORE_RTOL * abs(v)
