"""Perturbation quantities of Section 3 on a synthetic workload, for the two-stage rule against attention-only selection.

    python -m paper_2502_03805_b200.diagnostics_report [--cfg 1] [--layers 2] [--fractions 0.2 0.4]

For every budget fraction and stage split alpha in {1.0 (attention only, Algorithm 2's regular selection), 0.75, 0.5
(the paper's setting), 0.25} the GPU path compresses the generated layers and
criticalkv_diagnose evaluates, per query head and window row, sigma (Assumption 3.4), the output perturbation
L = ||(A - A') V W^O||_1 (Definition 3.1) and the bounds theta (Theorem 3.3), theta_hat (Theorem 3.5) and theta_relax
(relaxed bound of the appendix).  The table reports their means: the analogue, on synthetic inputs, of the paper's
bound-tightness table.  Everything is computed by the CUDA kernels; inputs come from gen.workloads.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    import numpy as np
    import torch
    from gen import config, make_layer
    from . import binding as B
    from .session import session_for, to_device

    p = argparse.ArgumentParser()
    p.add_argument("--cfg", type=int, default=1)
    p.add_argument("--layers", type=int, default=2)
    p.add_argument("--fractions", type=float, nargs="+", default=[0.2, 0.4])
    p.add_argument("--json", action="store_true")
    args = p.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    base = config(args.cfg)
    if base.w > 64:
        raise SystemExit("criticalkv_diagnose supports windows of at most 64 rows")
    rows = []
    for frac in args.fractions:
        budget = int(frac * base.n) if base.budget_mode == "uniform" else int(frac * base.n * base.Hkv)
        for alpha in (1.0, 0.75, 0.5, 0.25):
            wl = base.with_(budget=budget, alpha=alpha)
            acc = {k: [] for k in B.DIAG_FIELDS}
            for layer in range(args.layers):
                L = make_layer(wl, layer)
                s = session_for(wl, nb=1)
                Q, K, V, WO = (to_device(getattr(L, k)[None], wl.dtype) for k in
                               ("Qw_store", "K_store", "V_store", "WO_store"))
                s.compress(Q, K, V, WO)
                diag = torch.zeros((1, wl.Hq, wl.w, len(B.DIAG_FIELDS)), dtype=torch.float32, device="cuda")
                ws = torch.empty(B.criticalkv_diagnose_workspace_bytes(s.desc), dtype=torch.uint8, device="cuda")
                B.criticalkv_diagnose(s.handle, s.desc, Q, K, V, WO, s.vnorm, s.idx, s.offsets, s.stage, diag, ws)
                torch.cuda.synchronize()
                if s.device_status() != 0:
                    raise SystemExit("device status word set")
                d = diag[0].cpu().numpy().astype(np.float64)
                for i, k in enumerate(B.DIAG_FIELDS):
                    acc[k].append(d[..., i].reshape(-1))
            m = {k: float(np.concatenate(v).mean()) for k, v in acc.items()}
            sig = np.concatenate(acc["sigma"])
            rows.append(dict(fraction=frac, alpha=alpha, budget=budget, sigma_mean=m["sigma"],
                             sigma_above_half=float((sig > 0.5).mean()),
                             mass_kept=m["mass_kept"], L=m["L"], theta=m["theta"], theta_hat=m["theta_hat"],
                             theta_relax=m["theta_relax"], C=m["C"]))
    if args.json:
        print(json.dumps(dict(workload=base.name, layers=args.layers, rows=rows)))
        return
    print(f"workload {base.name}: {args.layers} layers, n = {base.n}, window {base.w}, {base.budget_mode} budgets")
    print("| kept | alpha | retained attention mass | L (measured) | theta (Thm 3.3) | theta_hat (Thm 3.5) | theta_relax |"
          " sigma > 0.5 |")
    print("|---|---|---|---|---|---|---|---|")
    for r in rows:
        sa = "-" if r["sigma_above_half"] is None else f"{100 * r['sigma_above_half']:.1f} %"
        print(f"| {100 * r['fraction']:.0f} % | {r['alpha']:.1f} | {r['mass_kept']:.4f} | {r['L']:.4f} | "
              f"{r['theta']:.4f} | {r['theta_hat']:.4f} | {r['theta_relax']:.4f} | {sa} |")


if __name__ == "__main__":
    main()
