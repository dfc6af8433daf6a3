"""Comparison of the CUDA path with the CPU oracle (used by the GPU tests and by the smoke check).

Tolerances (written here once, used everywhere):
  * scores (attn, vnorm): 2e-3 relative, denominator floored at 1e-30 * max |ref|
  * selection: index sets identical outside the ambiguity band = entries whose oracle score lies within 1e-4
    relative of the stage's k-th score (widened by as many ranks as earlier ambiguous decisions can shift it);
    with an empty band the index arrays, stage bytes and compacted K/V are bit-identical
  * post-eviction window output: 1e-3 relative L2
"""
from __future__ import annotations

import numpy as np

from oracle import criticalkv_oracle as oc

SCORE_RTOL = 2e-3
TIE_BAND = 1e-4
OUTPUT_RTOL = 1e-3


def record_report(name, report):
    """Appends one JSON line with the parity report of a full-size test to parity_reports.jsonl in the run's output
    folder (CRITICALKV_REPORT_DIR, or the scratch output folder at the repository root), so that how exact the large
    comparisons were rests on a record and not on a printed line."""
    import json
    import os
    out_dir = os.environ.get("CRITICALKV_REPORT_DIR") or os.path.join(
        os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "gpurun_out")
    os.makedirs(out_dir, exist_ok=True)
    clean = {k: (v.item() if hasattr(v, "item") else v) for k, v in report.items()}
    with open(os.path.join(out_dir, "parity_reports.jsonl"), "a") as f:
        f.write(json.dumps({"test": name, **clean}) + "\n")


def rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.maximum(np.abs(ref), 1e-30 * max(float(np.abs(ref).max()), 1e-300))
    return np.abs(got - ref) / den


def assert_scores_close(got, ref, what, rtol=SCORE_RTOL):
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    err = rel_err(got, ref)
    worst = float(err.max())
    assert worst <= rtol, f"{what}: max relative error {worst:.3e} > {rtol} at {np.unravel_index(err.argmax(), err.shape)}"
    return worst


def _band(values, k, shift):
    """Indices whose value lies within TIE_BAND (relative) of the values ranked k-shift .. k+1+shift (1-based)."""
    n = values.size
    if k <= 0 or k >= n:
        return np.zeros(n, bool) if shift == 0 else np.ones(n, bool)
    srt = np.sort(values.astype(np.float64))[::-1]
    hi = srt[max(k - 1 - shift, 0)]
    lo = srt[min(k + shift, n - 1)]
    return (values >= lo * (1 - TIE_BAND) - 1e-300) & (values <= hi * (1 + TIE_BAND) + 1e-300)


def compare_selection(ref, gpu_idx, gpu_offsets, gpu_stage, *, n, alpha, budget_mode, budget):
    """ref: output of oracle.select (a, c, budgets, idx, offsets, stage).  Returns a report dict; raises on a
    difference outside the ambiguity band."""
    a, c = ref["a"], ref["c"]
    Hkv = a.shape[0]
    gpu_offsets = np.asarray(gpu_offsets)
    report = dict(heads=Hkv, exact_heads=0, ambiguous_entries=0, differing_entries=0)
    gpu_budgets = np.diff(gpu_offsets)
    assert gpu_offsets[0] == 0 and np.all(gpu_budgets >= 0)
    flat_shift = 0
    if budget_mode == "adaptive":
        assert gpu_offsets[-1] == budget, "adaptive budgets must sum to B_total"
        flat = a.reshape(-1)
        fb = _band(flat, int(budget), 0)
        srt = np.sort(flat.astype(np.float64))[::-1]
        kth = srt[budget - 1] if 0 < budget <= flat.size else None
        flat_shift = int(fb.sum()) if kth is not None else 0
        diff = np.abs(gpu_budgets - ref["budgets"])
        assert np.all(diff <= flat_shift), f"adaptive budgets differ beyond the tie band: {gpu_budgets} vs {ref['budgets']}"
    else:
        np.testing.assert_array_equal(gpu_budgets, ref["budgets"])
    for g in range(Hkv):
        seg = np.asarray(gpu_idx[gpu_offsets[g]:gpu_offsets[g + 1]])
        st = np.asarray(gpu_stage[gpu_offsets[g]:gpu_offsets[g + 1]]) if gpu_stage is not None else None
        assert np.all(np.diff(seg) > 0), f"head {g}: indices not strictly ascending"
        assert seg.size == 0 or (seg.min() >= 0 and seg.max() < n)
        rs = ref["idx"][ref["offsets"][g]:ref["offsets"][g + 1]]
        rst = ref["stage"][ref["offsets"][g]:ref["offsets"][g + 1]]
        if seg.size == rs.size and np.array_equal(seg, rs) and (st is None or np.array_equal(st, rst)):
            report["exact_heads"] += 1
            continue
        b = int(ref["budgets"][g])
        b1, b2 = oc.split_budget(b, alpha)
        shift1 = flat_shift
        band1 = _band(a[g], b1, shift1)
        in_s1 = np.zeros(n, bool)
        in_s1[rs[rst == 1]] = True
        cand = ~in_s1 | band1
        cvals = np.where(cand, c[g], -np.inf)
        shift2 = int(band1.sum()) + flat_shift
        band2 = _band(cvals, b2, shift2) & cand
        amb = band1 | band2
        sym = np.setxor1d(seg, rs)
        bad = [int(i) for i in sym if not amb[i]]
        assert not bad, (f"head {g}: {len(bad)} selected entries differ outside the tie band, e.g. {bad[:5]} "
                         f"(a={a[g][bad[:5]]}, c={c[g][bad[:5]]})")
        if st is not None:
            # stage labels may only differ on ambiguous entries
            common = np.intersect1d(seg, rs)
            s_gpu = st[np.searchsorted(seg, common)]
            s_ref = rst[np.searchsorted(rs, common)]
            badst = [int(i) for i in common[s_gpu != s_ref] if not amb[i]]
            assert not badst, f"head {g}: stage labels differ outside the tie band: {badst[:5]}"
        report["ambiguous_entries"] += int(amb.sum())
        report["differing_entries"] += int(sym.size)
    return report


def assert_compaction_exact(K_store, V_store, gpu_idx, gpu_offsets, K_out, V_out):
    """K_out / V_out must be the bit-exact row gather of the stored inputs at the GPU's own indices."""
    Ko, Vo = oc.compact(K_store, V_store, np.asarray(gpu_idx), np.asarray(gpu_offsets))
    tot = int(gpu_offsets[-1])
    np.testing.assert_array_equal(np.asarray(K_out)[:tot], Ko[:tot])
    np.testing.assert_array_equal(np.asarray(V_out)[:tot], Vo[:tot])


def assert_post_eviction_output(L, wl, ref_sel, gpu_idx, gpu_offsets, heads=None):
    """Window-query attention output on the retained cache: GPU selection vs oracle selection (1e-3 rel. L2)."""
    worst = 0.0
    heads = range(wl.Hq) if heads is None else heads
    for h in heads:
        g = h // wl.G
        s_gpu = np.asarray(gpu_idx[gpu_offsets[g]:gpu_offsets[g + 1]])
        s_ref = ref_sel["idx"][ref_sel["offsets"][g]:ref_sel["offsets"][g + 1]]
        if np.array_equal(s_gpu, s_ref):
            continue
        o_ref = oc.post_eviction_output(L.Qw[h], L.K[g], L.V[g], s_ref, wl.scale)
        o_gpu = oc.post_eviction_output(L.Qw[h], L.K[g], L.V[g], s_gpu, wl.scale)
        err = float(np.linalg.norm(o_gpu - o_ref) / max(np.linalg.norm(o_ref), 1e-300))
        worst = max(worst, err)
        assert err <= OUTPUT_RTOL, f"head {h}: post-eviction output differs by {err:.3e}"
    return worst


def oracle_layer(L, wl, *, nu=None, P=None, group_sum=False, norm="l1"):
    """Oracle scores and selection of one generated layer."""
    if P is None:
        P = oc.pooled_window_attention(L.Qw, L.K, wl.kp, wl.scale)
    if nu is None:
        nu = (oc.projection_norm_group_sum(L.V, L.WO, wl.G, wl.dtype, norm=norm) if group_sum
              else oc.projection_norm(L.V, L.WO, norm=norm))
    sel = oc.select(P, nu, G=wl.G, budget_mode=wl.budget_mode, budget=wl.budget, alpha=wl.alpha, eps=wl.eps,
                    group_sum=group_sum)
    return P, nu, sel


def check_layer_against_oracle(L, wl, out, *, full_output_check=True, group_sum=False, norm="l1"):
    """out: dict of host arrays attn, vnorm [Hq,n] ([Hkv,n] for the group-summed variant); idx, stage [Btot];
    offsets [Hkv+1]; K_out, V_out [Btot, dh].  Returns a report with the worst errors."""
    P, nu, sel = oracle_layer(L, wl, group_sum=group_sum, norm=norm)
    rep = dict(attn_err=assert_scores_close(out["attn"], P, "attn"),
               vnorm_err=assert_scores_close(out["vnorm"], nu, "vnorm"))
    rep.update(compare_selection(sel, out["idx"], out["offsets"], out.get("stage"), n=wl.n, alpha=wl.alpha,
                                 budget_mode=wl.budget_mode, budget=wl.budget))
    assert_compaction_exact(L.K_store, L.V_store, out["idx"], out["offsets"], out["K_out"], out["V_out"])
    if rep["differing_entries"] == 0:
        np.testing.assert_array_equal(out["idx"][: sel["idx"].size], sel["idx"])
        Ko, Vo = oc.compact(L.K_store, L.V_store, sel["idx"], sel["offsets"])
        np.testing.assert_array_equal(out["K_out"][: Ko.shape[0]], Ko)
        np.testing.assert_array_equal(out["V_out"][: Vo.shape[0]], Vo)
        rep["output_err"] = 0.0
    elif full_output_check:
        rep["output_err"] = assert_post_eviction_output(L, wl, sel, out["idx"], out["offsets"])
    return rep
