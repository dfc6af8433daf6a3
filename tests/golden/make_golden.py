"""Writes the stored expected values under tests/golden/ by running the CPU oracle only.

    python tests/golden/make_golden.py

The paper prints no worked numeric example of the compression step, so nothing here is a paper value: the files pin
the oracle's own output on the seeded tiny configuration (so that an accidental change of the oracle or of the
generators is noticed) and give the GPU tests an expected selection that does not come from the CUDA path.
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from gen import config, make_layer  # noqa: E402
from oracle import criticalkv_oracle as oc  # noqa: E402


def main():
    wl = config(0)
    L = make_layer(wl, 0)
    out = oc.compress_layer(L.Qw, L.K, L.V, L.WO, kp=wl.kp, budget_mode=wl.budget_mode, budget=wl.budget,
                            alpha=wl.alpha, eps=wl.eps, scale=wl.scale, K_store=L.K_store, V_store=L.V_store)
    doc = {
        "what": "oracle output on configuration 0 (tiny float32 layer, seed 0): Algorithm 2 window attention, "
                "Algorithm 1 projection norm and two-stage selection, uniform budget 128 per KV head, alpha 0.5",
        "source": "oracle/criticalkv_oracle.py via tests/golden/make_golden.py (not from the paper, not from the GPU)",
        "offsets": out["offsets"].tolist(),
        "idx": out["idx"].tolist(),
        "stage": out["stage"].tolist(),
        "attn_sum_per_head": [float(x) for x in out["P"].sum(axis=1)],
        "vnorm_sum_per_head": [float(x) for x in out["nu"].sum(axis=1)],
        "attn_probe": [[h, i, float(out["P"][h, i])] for h in range(wl.Hq) for i in (0, 100, 300, 495, 511)],
        "vnorm_probe": [[h, i, float(out["nu"][h, i])] for h in range(wl.Hq) for i in (0, 100, 300, 495, 511)],
    }
    with open(os.path.join(HERE, "cfg0_oracle.json"), "w") as f:
        json.dump(doc, f, indent=1)
    print("wrote cfg0_oracle.json")


if __name__ == "__main__":
    main()
