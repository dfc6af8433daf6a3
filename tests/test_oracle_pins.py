"""Pins for the CPU oracle: what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each checks an oracle function
against something other than itself: a library routine (scipy softmax, scipy
sliding maximum), a closed form, a pure-Python loop on a tiny case, or an
exhaustive enumeration backing one of the paper's theorems.
"""
import math
from itertools import combinations

import numpy as np
import pytest
from scipy.ndimage import maximum_filter1d
from scipy.special import softmax as scipy_softmax

from oracle import criticalkv_oracle as oc

RNG = np.random.default_rng


# ----------------------------------------------------------------------------- step 1
def test_softmax_rows_sum_to_one_and_mask_is_causal():
    r = RNG(1)
    n, w, dh = 50, 7, 16
    Q = r.standard_normal((w, dh))
    K = r.standard_normal((n, dh))
    A = oc.window_softmax(Q, K, 1 / math.sqrt(dh))
    assert A.shape == (w, n)
    np.testing.assert_allclose(A.sum(axis=1), 1.0, rtol=0, atol=1e-14)
    for j in range(w):
        last = n - w + j
        assert np.all(A[j, last + 1:] == 0.0)
        assert np.all(A[j, : last + 1] > 0.0)
    # window mean of distributions is a distribution (Algorithm 2, mean over the window)
    assert abs(oc.window_mean(A).sum() - 1.0) < 1e-14


def test_single_query_reduces_to_library_softmax():
    # w = 1, kp = 1: the textbook single-query softmax of Eq. 2
    r = RNG(2)
    n, dh = 33, 8
    Q = r.standard_normal((1, 1, dh))
    K = r.standard_normal((1, n, dh))
    P = oc.pooled_window_attention(Q, K, kp=1)
    ref = scipy_softmax((Q[0, 0] @ K[0].T) / math.sqrt(dh))
    np.testing.assert_allclose(P[0], ref, rtol=1e-13, atol=0)


def test_explicit_scale_argument():
    r = RNG(21)
    n, dh = 20, 4
    Q = r.standard_normal((1, 1, dh))
    K = r.standard_normal((1, n, dh))
    P = oc.pooled_window_attention(Q, K, kp=1, scale=0.37)
    np.testing.assert_allclose(P[0], scipy_softmax(0.37 * (Q[0, 0] @ K[0].T)), rtol=1e-13)


def test_window_attention_python_loop():
    # brute force with math.exp, including the causal mask and the mean over w rows
    r = RNG(3)
    n, w, dh, kp = 12, 4, 5, 3
    Q = r.standard_normal((1, w, dh))
    K = r.standard_normal((1, n, dh))
    scale = 1 / math.sqrt(dh)
    abar = [0.0] * n
    for j in range(w):
        last = n - w + j
        lg = [scale * sum(Q[0, j, t] * K[0, i, t] for t in range(dh)) for i in range(last + 1)]
        den = sum(math.exp(x) for x in lg)
        for i in range(last + 1):
            abar[i] += math.exp(lg[i]) / den / w
    pooled = [max(abar[max(0, i - 1): min(n, i + 2)]) for i in range(n)]
    P = oc.pooled_window_attention(Q, K, kp=kp)
    np.testing.assert_allclose(P[0], pooled, rtol=1e-12)


def test_gqa_query_head_reads_its_kv_head():
    # KV head g has one key aligned with a probe direction at position p_g
    n, dh, Hkv, G, w = 40, 8, 3, 2, 1
    K = np.zeros((Hkv, n, dh))
    peaks = [5, 17, 29]
    for g in range(Hkv):
        K[g, peaks[g], 0] = 50.0
    Q = np.zeros((Hkv * G, w, dh))
    Q[:, :, 0] = 1.0
    P = oc.pooled_window_attention(Q, K, kp=1)
    for h in range(Hkv * G):
        assert int(np.argmax(P[h])) == peaks[h // G]


@pytest.mark.parametrize("kp", [1, 3, 5, 7, 9])
def test_max_pool_against_library_and_loop(kp):
    r = RNG(4)
    x = r.random((3, 37))
    got = oc.max_pool(x, kp)
    ref = maximum_filter1d(x, size=kp, axis=-1, mode="constant", cval=-np.inf)
    np.testing.assert_array_equal(got, ref)
    rad = (kp - 1) // 2
    for i in range(x.shape[1]):
        assert got[1, i] == max(x[1, max(0, i - rad): i + rad + 1])
    if kp == 1:
        np.testing.assert_array_equal(got, x)
    assert np.all(got >= x) and got.max() == x.max()


def test_max_pool_rejects_even_kernel():
    with pytest.raises(ValueError):
        oc.max_pool(np.zeros(4), 2)


def test_max_pool_shorter_than_kernel():
    x = np.array([1.0, 3.0, 2.0])
    np.testing.assert_array_equal(oc.max_pool(x, 7), [3.0, 3.0, 3.0])


# ----------------------------------------------------------------------------- step 2
def test_projection_norm_identity_gives_row_l1():
    r = RNG(5)
    Hkv, G, n, dh, dm = 2, 2, 9, 4, 6
    V = r.standard_normal((Hkv, n, dh))
    WO = np.zeros((Hkv * G, dh, dm))
    WO[:, np.arange(dh), np.arange(dh)] = 1.0          # [I | 0]
    nu = oc.projection_norm(V, WO)
    for h in range(Hkv * G):
        np.testing.assert_allclose(nu[h], np.abs(V[h // G]).sum(axis=1), rtol=1e-14)


def test_projection_norm_one_hot_column_and_row_scaling():
    r = RNG(6)
    n, dh, dm = 7, 5, 3
    V = r.standard_normal((1, n, dh))
    WO = np.zeros((1, dh, dm))
    WO[0, 2, 1] = -3.0                                  # only V[:, 2] reaches the output, times -3
    nu = oc.projection_norm(V, WO)
    np.testing.assert_allclose(nu[0], 3.0 * np.abs(V[0, :, 2]), rtol=1e-14)
    WO = r.standard_normal((1, dh, dm))
    base = oc.projection_norm(V, WO)
    V2 = V.copy()
    V2[0, 3] *= -2.5
    scaled = oc.projection_norm(V2, WO)
    np.testing.assert_allclose(scaled[0, 3], 2.5 * base[0, 3], rtol=1e-13)
    np.testing.assert_allclose(np.delete(scaled[0], 3), np.delete(base[0], 3), rtol=1e-14)


def test_projection_norm_triple_loop_and_head_slices():
    r = RNG(7)
    Hkv, G, n, dh, dm = 2, 3, 5, 3, 4                   # dh != dm catches a transposed operand
    V = r.standard_normal((Hkv, n, dh))
    WO = r.standard_normal((Hkv * G, dh, dm))
    nu = oc.projection_norm(V, WO, chunk=2)
    for h in range(Hkv * G):
        for i in range(n):
            tot = 0.0
            for c in range(dm):
                tot += abs(sum(V[h // G, i, t] * WO[h, t, c] for t in range(dh)))
            assert abs(nu[h, i] - tot) < 1e-12
    # rows subset
    np.testing.assert_allclose(oc.projection_norm(V, WO, rows=[4, 1])[:, 0], nu[:, 4])
    # zeroing every head's slice but one silences the others
    WO2 = np.zeros_like(WO)
    WO2[4] = WO[4]
    nu2 = oc.projection_norm(V, WO2)
    assert np.all(nu2[[0, 1, 2, 3, 5]] == 0) and np.all(nu2[4] > 0)


def test_projection_norm_l2_variant():
    r = RNG(8)
    V = r.standard_normal((1, 6, 4))
    WO = r.standard_normal((1, 4, 5))
    nu = oc.projection_norm(V, WO, norm="l2")
    gram = WO[0] @ WO[0].T                              # ||vW||_2^2 = v (W W^T) v^T
    ref = np.sqrt(np.einsum("it,ts,is->i", V[0], gram, V[0]))
    np.testing.assert_allclose(nu[0], ref, rtol=1e-12)


def test_group_sum_projection_special_cases():
    r = RNG(80)
    Hkv, G, n, dh, dm = 2, 3, 6, 4, 5
    V = r.standard_normal((Hkv, n, dh))
    WO = r.standard_normal((Hkv * G, dh, dm)).astype(np.float32)
    # a group of one head is the per-head norm
    np.testing.assert_allclose(oc.projection_norm_group_sum(V, WO[:2], 1), oc.projection_norm(V, WO[:2]), rtol=1e-12)
    # only one head of each group non-zero: that head's norm
    W1 = np.zeros_like(WO)
    W1[1], W1[5] = WO[1], WO[5]
    nu = oc.projection_norm_group_sum(V, W1, G)
    np.testing.assert_allclose(nu, oc.projection_norm(V, W1)[[1, 5]], rtol=1e-12)
    # opposite slices cancel before the norm is taken (a sum of per-head norms would not)
    W2 = np.zeros_like(WO)
    W2[0], W2[1] = WO[0], -WO[0]
    assert np.all(oc.projection_norm_group_sum(V, W2, G)[0] == 0)
    # scaled identities: nu = |sum of scales| * ||v||_1
    W3 = np.zeros((G, dh, dm), np.float32)
    for h, sc in enumerate((0.5, -2.0, 4.0)):
        W3[h, np.arange(dh), np.arange(dh)] = sc
    np.testing.assert_allclose(oc.projection_norm_group_sum(V[:1], W3, G)[0], 2.5 * np.abs(V[0]).sum(axis=1), rtol=1e-12)
    # triple loop
    nu = oc.projection_norm_group_sum(V, WO, G)
    for g in range(Hkv):
        for i in range(n):
            tot = 0.0
            for c in range(dm):
                tot += abs(sum(V[g, i, t] * sum(float(WO[g * G + q, t, c]) for q in range(G)) for t in range(dh)))
            assert abs(nu[g, i] - tot) < 1e-5 * tot          # float32 sums of the slices


def test_group_sum_projection_rounds_once_to_bf16():
    import torch
    r = RNG(81)
    WO = torch.from_numpy(r.standard_normal((4, 3, 8)).astype(np.float32)).to(torch.bfloat16).to(torch.float32).numpy()
    Wt = oc.group_summed_projection(WO, 4, "bf16")
    exact = WO.astype(np.float64).sum(axis=0)
    assert np.all(np.abs(Wt[0] - exact) <= 2.0 ** -8 * np.abs(exact) + 1e-30)                  # one bf16 rounding
    assert np.array_equal(Wt, torch.from_numpy(Wt).to(torch.bfloat16).to(torch.float32).numpy())  # representable


def test_group_sum_scores():
    r = RNG(82)
    P = r.random((6, 20)).astype(np.float32)
    nu = (r.random((2, 20)) * 9).astype(np.float32)
    a, c = oc.group_scores_group_sum(P, nu, 3, 1e-4)
    a_ref, _ = oc.group_scores(P, np.ones_like(P), 3)
    np.testing.assert_array_equal(a, a_ref)
    np.testing.assert_allclose(c, (P.reshape(2, 3, -1).mean(axis=1) + 1e-4) * nu, rtol=1e-6)
    out = oc.select(P, nu, G=3, budget_mode="uniform", budget=5, group_sum=True)
    assert out["idx"].size == 10


# ----------------------------------------------------------------------------- step 3
def test_group_scores_special_cases():
    r = RNG(9)
    n = 11
    P = r.random((4, n)).astype(np.float32)
    nu = (r.random((4, n)) * 10).astype(np.float32)
    a, c = oc.group_scores(P, nu, G=1, eps=0.0)
    np.testing.assert_array_equal(a, P)
    np.testing.assert_array_equal(c, P * nu)
    # identical heads inside a group: the mean equals each member (power-of-two G is exact)
    P2 = np.repeat(P[:2], 2, axis=0)
    nu2 = np.repeat(nu[:2], 2, axis=0)
    a2, c2 = oc.group_scores(P2, nu2, G=2, eps=1e-4)
    np.testing.assert_array_equal(a2, P[:2])
    np.testing.assert_array_equal(c2, ((P[:2] + np.float32(1e-4)) * nu[:2]).astype(np.float32))
    # eps enters before the multiplication (Algorithm 1: (A + eps) * norm)
    z = np.zeros((1, n), dtype=np.float32)
    _, c3 = oc.group_scores(z, nu[:1], G=1, eps=1e-4)
    np.testing.assert_allclose(c3, np.float32(1e-4) * nu[:1], rtol=1e-7)
    assert a.dtype == np.float32 and c.dtype == np.float32


def test_group_scores_close_to_float64_mean():
    r = RNG(10)
    P = r.random((6, 50))
    nu = r.random((6, 50)) * 100
    a, c = oc.group_scores(P, nu, G=3, eps=1e-4)
    np.testing.assert_allclose(a, P.reshape(2, 3, -1).mean(axis=1), rtol=1e-6)
    np.testing.assert_allclose(c, ((P + 1e-4) * nu).reshape(2, 3, -1).mean(axis=1), rtol=1e-6)


@pytest.mark.parametrize("b,alpha,exp", [(128, 0.5, (64, 64)), (819, 0.5, (409, 410)), (13107, 0.5, (6553, 6554)),
                                         (10, 0.25, (2, 8)), (7, 1.0, (7, 0)), (7, 0.0, (0, 7)), (0, 0.5, (0, 0)),
                                         (1, 0.5, (0, 1))])
def test_split_budget(b, alpha, exp):
    assert oc.split_budget(b, alpha) == exp


def test_stable_topk_ties_go_to_lower_index():
    x = np.array([1.0, 5.0, 5.0, 3.0, 5.0, 0.0], dtype=np.float32)
    assert list(oc.stable_topk(x, 2)) == [1, 2]
    assert list(oc.stable_topk(x, 4)) == [1, 2, 4, 3]
    assert list(oc.stable_topk(x, 0)) == []
    # brute force on random tied data
    r = RNG(11)
    for _ in range(20):
        y = r.integers(0, 4, size=15).astype(np.float32)
        k = int(r.integers(0, 16))
        ref = sorted(range(15), key=lambda i: (-y[i], i))[:k]
        assert list(oc.stable_topk(y, k)) == ref


def test_adaptive_budgets():
    r = RNG(12)
    Hkv, n, B = 4, 30, 37
    a = r.random((Hkv, n)).astype(np.float32)
    a[2] *= 5                                            # one head holds most of the mass
    counts = oc.allocate_budgets(a, "adaptive", B)
    assert counts.sum() == B and counts[2] == max(counts) and np.all(counts <= n)
    thr = np.sort(a.reshape(-1))[::-1][B - 1]
    np.testing.assert_array_equal(counts, (a >= thr).sum(axis=1))      # no ties here
    # all-equal scores: flattened order fills head 0 first
    flat = oc.allocate_budgets(np.ones((3, 10), np.float32), "adaptive", 14)
    assert list(flat) == [10, 4, 0]
    assert list(oc.allocate_budgets(a, "uniform", 9)) == [9] * Hkv


def test_adaptive_floor():
    r = RNG(83)
    Hkv, n, B = 4, 50, 80
    a = r.random((Hkv, n)).astype(np.float32)
    a[0] *= 10                                            # head 0 would take almost everything
    plain = oc.allocate_budgets(a, "adaptive", B)
    assert plain.sum() == B and plain[0] >= 40 and plain[1:].min() < 15
    half = oc.allocate_budgets(a, "adaptive", B, floor=0.5)
    assert half.min() >= 10                               # floor(0.5 * 80 / 4) guaranteed per head
    rest = oc.allocate_budgets(a, "adaptive", B - 4 * 10)
    np.testing.assert_array_equal(half, np.minimum(rest + 10, n))
    full = oc.allocate_budgets(a, "adaptive", B, floor=1.0)
    assert list(full) == [20, 20, 20, 20]                 # floor 1 is the uniform split
    np.testing.assert_array_equal(oc.allocate_budgets(a, "adaptive", B, floor=0.0), plain)


def test_protect_window_keeps_the_last_w_entries():
    r = RNG(84)
    Hq, G, n, w = 4, 2, 40, 6
    P = r.random((Hq, n))
    P[:, n - w:] = 0.0                                    # the window would otherwise be dropped
    nu = np.exp(r.standard_normal((Hq, n)))
    for mode, budget in (("uniform", 10), ("adaptive", 24)):
        out = oc.select(P, nu, G=G, budget_mode=mode, budget=budget, protect_w=w)
        base = oc.select(P, nu, G=G, budget_mode=mode, budget=budget)
        for g in range(2):
            seg = out["idx"][out["offsets"][g]:out["offsets"][g + 1]]
            assert set(range(n - w, n)) <= set(seg.tolist())
            assert not set(range(n - w, n)) & set(base["idx"][base["offsets"][g]:base["offsets"][g + 1]].tolist())
    # a budget smaller than the window keeps its first entries (lowest index first)
    tiny = oc.select(P, nu, G=G, budget_mode="uniform", budget=4, protect_w=w)
    assert tiny["idx"][:4].tolist() == [n - w, n - w + 1, n - w + 2, n - w + 3]


# ----------------------------------------------------------------------------- step 4
def _scores(seed, n=40, dup=False):
    r = RNG(seed)
    a = r.random(n).astype(np.float32)
    if dup:
        a = np.round(a * 6).astype(np.float32) / 6       # many exact ties (as max-pooling produces)
    nu = np.exp(r.standard_normal(n)).astype(np.float32)
    c = ((a + np.float32(1e-4)) * nu).astype(np.float32)
    return a, c


@pytest.mark.parametrize("dup", [False, True])
def test_two_stage_invariants_and_definition(dup):
    for seed in range(10):
        a, c = _scores(100 + seed, dup=dup)
        n = a.size
        for b, alpha in [(10, 0.5), (11, 0.5), (1, 0.5), (40, 0.5), (0, 0.5), (13, 0.3)]:
            S1, S2 = oc.two_stage_select(a, c, b, alpha)
            b1, b2 = oc.split_budget(b, alpha)
            assert S1.size == b1 and S2.size == b2
            assert not set(S1) & set(S2)
            assert np.all(np.diff(S1) > 0) and np.all(np.diff(S2) > 0)
            # definition by explicit sorting with (score desc, index asc)
            ref1 = sorted(range(n), key=lambda i: (-a[i], i))[:b1]
            rest = [i for i in range(n) if i not in set(ref1)]
            ref2 = sorted(rest, key=lambda i: (-c[i], i))[:b2]
            assert sorted(ref1) == list(S1) and sorted(ref2) == list(S2)


def test_alpha_one_is_plain_attention_topk_and_alpha_zero_is_score_topk():
    # Algorithm 2, "regular selection": Top_k(A_bar, b)
    a, c = _scores(7)
    S1, S2 = oc.two_stage_select(a, c, 12, 1.0)
    assert S2.size == 0 and sorted(np.argsort(-a, kind="stable")[:12]) == list(S1)
    S1, S2 = oc.two_stage_select(a, c, 12, 0.0)
    assert S1.size == 0 and sorted(np.argsort(-c, kind="stable")[:12]) == list(S2)


def test_constant_norm_reduces_to_attention_only():
    # relaxed-bound theorem: with all row norms equal the two rules coincide (eps = 0, distinct a)
    r = RNG(13)
    a = r.permutation(60).astype(np.float32) / 60
    c = (a * np.float32(3.0)).astype(np.float32)
    for alpha in (0.0, 0.25, 0.5, 0.75, 1.0):
        S1, S2 = oc.two_stage_select(a, c, 20, alpha)
        assert sorted(np.concatenate([S1, S2])) == sorted(np.argsort(-a, kind="stable")[:20])


def test_select_layout_and_stage_bytes():
    r = RNG(14)
    Hq, G, n = 4, 2, 25
    P = r.random((Hq, n))
    nu = np.exp(r.standard_normal((Hq, n)))
    out = oc.select(P, nu, G=G, budget_mode="uniform", budget=8, alpha=0.5)
    assert list(out["offsets"]) == [0, 8, 16]
    for g in range(2):
        seg = out["idx"][8 * g: 8 * g + 8]
        assert np.all(np.diff(seg) > 0) and seg.min() >= 0 and seg.max() < n
        S1, S2 = oc.two_stage_select(out["a"][g], out["c"][g], 8, 0.5)
        st = out["stage"][8 * g: 8 * g + 8]
        assert set(seg[st == 1]) == set(S1) and set(seg[st == 2]) == set(S2)
    ada = oc.select(P, nu, G=G, budget_mode="adaptive", budget=15, alpha=0.5)
    assert ada["offsets"][-1] == 15 and ada["budgets"].sum() == 15
    giv = oc.select(P, nu, G=G, budget_mode="given", budget=0, budgets_in=[3, 11])
    assert list(giv["offsets"]) == [0, 3, 14]


def test_compact_is_a_row_gather():
    r = RNG(15)
    K = r.integers(0, 2 ** 16, size=(2, 9, 4)).astype(np.uint16)
    V = r.integers(0, 2 ** 16, size=(2, 9, 4)).astype(np.uint16)
    idx = np.array([0, 3, 8, 1, 2], dtype=np.int32)
    off = np.array([0, 3, 5], dtype=np.int32)
    Ko, Vo = oc.compact(K, V, idx, off)
    np.testing.assert_array_equal(Ko, np.concatenate([K[0][[0, 3, 8]], K[1][[1, 2]]]))
    np.testing.assert_array_equal(Vo, np.concatenate([V[0][[0, 3, 8]], V[1][[1, 2]]]))


# ----------------------------------------------------------------------------- theory (Section 3)
def _tiny_head(seed, n=12, dh=4, dm=6, peaked=True):
    r = RNG(seed)
    q = r.standard_normal(dh)
    K = r.standard_normal((n, dh))
    if peaked:
        K[r.choice(n, 3, replace=False)] += 3.0 * q / np.linalg.norm(q)
    V = r.standard_normal((n, dh)) * np.exp(r.standard_normal((n, 1)))
    W = r.standard_normal((dh, dm))
    logits = q @ K.T / math.sqrt(dh)
    A = scipy_softmax(logits)
    Vp = V @ W
    nu = np.abs(Vp).sum(axis=1)
    return logits, A, Vp, nu


def test_theorem_3_2_mask_rewrite_identity():
    for seed in range(5):
        logits, A, _, _ = _tiny_head(seed)
        r = RNG(50 + seed)
        keep = np.zeros(A.size, bool)
        keep[r.choice(A.size, 5, replace=False)] = True
        lhs = oc.masked_softmax(logits, keep)
        rhs = keep * A / (keep * A).sum()
        np.testing.assert_allclose(lhs, rhs, rtol=1e-12, atol=1e-300)
        assert abs(lhs.sum() - 1) < 1e-14 and np.all(lhs[~keep] == 0)


@pytest.mark.parametrize("n,b", [(8, 3), (10, 5), (12, 4), (12, 6), (14, 7)])
def test_theorem_3_3_bound_holds_for_every_subset(n, b):
    for seed in range(3):
        logits, A, Vp, nu = _tiny_head(200 + seed, n=n, peaked=(seed != 2))
        worst = -np.inf
        for keep in oc.all_subsets(n, b):
            L = oc.perturbation(A, oc.masked_softmax(logits, keep), Vp)
            th = oc.theta_bound(A, nu, keep)
            assert L <= th * (1 + 1e-12) + 1e-12
            worst = max(worst, L / th)
        assert 0 < worst <= 1 + 1e-9


def test_theta_matches_its_unsimplified_form():
    # theta = sum_i |A_i - N_i A_i / sum(N A)| * nu_i  (proof of Theorem 3.3)
    logits, A, Vp, nu = _tiny_head(31)
    keep = np.zeros(A.size, bool)
    keep[[0, 2, 5, 7]] = True
    Ap = keep * A / A[keep].sum()
    direct = float((np.abs(A - Ap) * nu).sum())
    # valid when the retained mass is below one (always) and each kept weight grows
    assert abs(oc.theta_bound(A, nu, keep) - direct) < 1e-12


@pytest.mark.parametrize("n,b", [(10, 4), (12, 6), (13, 6), (16, 8)])
def test_theorem_3_5_stage_two_minimises_theta_hat(n, b):
    checked = 0
    for seed in range(6):
        logits, A, Vp, nu = _tiny_head(300 + seed, n=n)
        a32 = A.astype(np.float32)
        c32 = (a32 * nu.astype(np.float32)).astype(np.float32)          # eps = 0
        S1, S2 = oc.two_stage_select(a32, c32, b, 0.5)
        k1 = np.zeros(n, bool)
        k1[S1] = True
        sigma = A[k1].sum()
        if sigma <= 0.5:                                                  # Assumption 3.4 must hold
            continue
        checked += 1
        rest = [i for i in range(n) if not k1[i]]
        best, best_set = np.inf, None
        for comb in combinations(rest, S2.size):
            k2 = np.zeros(n, bool)
            k2[list(comb)] = True
            th_hat = oc.theta_hat_bound(A, nu, k1, k2)
            th = oc.theta_bound(A, nu, k1 | k2)
            L = oc.perturbation(A, oc.masked_softmax(logits, k1 | k2), Vp)
            assert L <= th * (1 + 1e-12) + 1e-12 and th <= th_hat + 1e-12
            assert th_hat <= oc.theta_relax_bound(A, nu, k1, k2) + 1e-12
            if th_hat < best:
                best, best_set = th_hat, set(comb)
        assert best_set == set(S2.tolist())
        assert abs(oc.stage1_mass(a32, b, 0.5) - sigma) < 1e-6
    assert checked >= 3


def test_attention_only_selection_minimises_relaxed_bound():
    logits, A, Vp, nu = _tiny_head(77, n=12)
    a32 = A.astype(np.float32)
    S1, S2 = oc.two_stage_select(a32, a32, 6, 0.5)                       # stage 2 by attention alone
    k1 = np.zeros(12, bool)
    k1[S1] = True
    assert A[k1].sum() > 0.5
    rest = [i for i in range(12) if not k1[i]]
    vals = {}
    for comb in combinations(rest, 3):
        k2 = np.zeros(12, bool)
        k2[list(comb)] = True
        vals[comb] = oc.theta_relax_bound(A, nu, k1, k2)
    assert set(min(vals, key=vals.get)) == set(S2.tolist())


def test_row_diagnostics_agree_with_the_single_row_functions():
    # the batched diagnostics restate theta / theta_hat / theta_relax / L: check them against the per-row functions
    # that the brute-force theorem pins already cover, and against the masked softmax of Section 3.3
    r = RNG(90)
    n, w, dh, dm = 30, 4, 6, 9
    Q, K = r.standard_normal((w, dh)), r.standard_normal((n, dh))
    K[[3, 11, 20]] += 2.5 * Q[-1] / np.linalg.norm(Q[-1])
    V, W = r.standard_normal((n, dh)) * np.exp(r.standard_normal((n, 1))), r.standard_normal((dh, dm))
    sc = 1 / math.sqrt(dh)
    S1, S2 = np.array([3, 11, 20, 25]), np.array([0, 7, 18])
    D = oc.row_diagnostics(Q, K, V, W, S1, S2, sc)
    A = oc.window_softmax(Q, K, sc)
    Vp = V @ W
    nu = np.abs(Vp).sum(axis=1)
    k1 = np.isin(np.arange(n), S1)
    k2 = np.isin(np.arange(n), S2)
    for j in range(w):
        vis = np.arange(n) <= n - w + j
        logits = (Q[j] @ K.T) * sc
        A_kept = oc.masked_softmax(np.where(vis, logits, -1e300), (k1 | k2) & vis)
        f = dict(zip(oc.DIAG_FIELDS, D[j]))
        assert abs(f["L"] - oc.perturbation(A[j], A_kept, Vp)) < 1e-10
        assert abs(f["theta"] - oc.theta_bound(A[j], nu, k1 | k2)) < 1e-10
        assert abs(f["theta_hat"] - oc.theta_hat_bound(A[j], nu, k1, k2)) < 1e-10
        assert abs(f["theta_relax"] - oc.theta_relax_bound(A[j], nu, k1, k2)) < 1e-10
        assert abs(f["sigma"] - A[j][k1].sum()) < 1e-14 and abs(f["nu_min"] - nu.min()) < 1e-14
        assert f["L"] <= f["theta"] + 1e-12
        if f["sigma"] > 0.5:
            assert f["theta"] <= f["theta_hat"] + 1e-12 <= f["theta_relax"] + 2e-12


def test_post_eviction_output_full_cache_is_plain_attention():
    r = RNG(16)
    n, w, dh = 20, 3, 4
    Q, K, V = r.standard_normal((w, dh)), r.standard_normal((n, dh)), r.standard_normal((n, dh))
    sc = 1 / math.sqrt(dh)
    full = oc.post_eviction_output(Q, K, V, None, sc)
    np.testing.assert_allclose(full, oc.window_softmax(Q, K, sc) @ V, rtol=1e-12)
    kept = np.arange(n)
    np.testing.assert_allclose(oc.post_eviction_output(Q, K, V, kept, sc), full, rtol=1e-12)
    # keeping one visible entry returns that value row
    one = oc.post_eviction_output(Q, K, V, np.array([4]), sc)
    np.testing.assert_allclose(one, np.repeat(V[4:5], w, axis=0), rtol=1e-12)


def test_chunked_compress_single_chunk_and_positions():
    from gen import make_layer, small_workload
    wl = small_workload(n=120, w=8, kp=5, budget=30, cfg_id=71)
    L = make_layer(wl)
    # one chunk = plain compression; positions are the selected indices
    K1, V1, pos, hist = oc.chunked_compress([(L.Qw, L.K, L.V)], L.WO, kp=wl.kp, w=wl.w, budgets=[30])
    ref = oc.compress_layer(L.Qw, L.K, L.V, L.WO, kp=wl.kp, budget_mode="uniform", budget=30)
    np.testing.assert_array_equal(pos.reshape(-1), ref["idx"])
    np.testing.assert_array_equal(K1.reshape(-1, wl.dh), ref["K_hat"])
    # two chunks: the second step sees [30 retained ; 60 new] and positions stay original, ascending, in range
    L2 = make_layer(wl.with_(n=60), 1)
    K2, V2, pos2, hist2 = oc.chunked_compress([(L.Qw, L.K, L.V), (L2.Qw, L2.K, L2.V)], L.WO, kp=wl.kp, w=wl.w,
                                              budgets=[30, 40])
    assert pos2.shape == (wl.Hkv, 40) and np.all(np.diff(pos2, axis=1) > 0) and pos2.max() < 180
    for g in range(wl.Hkv):
        old = pos2[g][pos2[g] < 120]
        assert set(old.tolist()) <= set(pos[g].tolist())          # nothing evicted in step 1 comes back
        for p, krow in zip(pos2[g], K2[g]):
            src = L.K[g][p] if p < 120 else L2.K[g][p - 120]
            np.testing.assert_array_equal(krow, src)


def _ragged_case(cut=(0, 37), **kw):
    from gen import make_layer, small_workload
    wl = small_workload(n=160, w=8, kp=5, cfg_id=72, **kw)
    L = make_layer(wl)
    K_list = [L.K[g][cut[g]:] for g in range(wl.Hkv)]
    V_list = [L.V[g][cut[g]:] for g in range(wl.Hkv)]
    return wl, L, K_list, V_list


@pytest.mark.parametrize("mode,budget", [("uniform", 31), ("adaptive", 70)])
def test_ragged_compress_with_equal_lengths_is_the_plain_path(mode, budget):
    wl, L, K_list, V_list = _ragged_case(cut=(0, 0))
    rag = oc.compress_layer_ragged(L.Qw, K_list, V_list, L.WO, kp=wl.kp, budget_mode=mode, budget=budget)
    ref = oc.compress_layer(L.Qw, L.K, L.V, L.WO, kp=wl.kp, budget_mode=mode, budget=budget)
    np.testing.assert_array_equal(rag["idx"], ref["idx"])
    np.testing.assert_array_equal(rag["offsets"], ref["offsets"])
    np.testing.assert_array_equal(rag["stage"], ref["stage"])
    np.testing.assert_array_equal(np.stack(rag["P"]), ref["P"])


def test_ragged_compress_treats_every_head_as_its_own_sequence():
    # a head's scores depend only on its own list: they equal the plain path run on that head alone, and the
    # adaptive allocation equals a brute-force ranking of all (score, head, entry) triples
    wl, L, K_list, V_list = _ragged_case(cut=(0, 37))
    B = 90
    rag = oc.compress_layer_ragged(L.Qw, K_list, V_list, L.WO, kp=wl.kp, budget_mode="adaptive", budget=B)
    G = wl.G
    for g in range(wl.Hkv):
        alone = oc.compress_layer(L.Qw[g * G:(g + 1) * G], K_list[g][None], V_list[g][None], L.WO[g * G:(g + 1) * G],
                                  kp=wl.kp, budget_mode="uniform", budget=int(rag["budgets"][g]))
        np.testing.assert_array_equal(alone["a"][0], rag["a"][g])
        np.testing.assert_array_equal(alone["c"][0], rag["c"][g])
        np.testing.assert_array_equal(alone["idx"], rag["idx"][rag["offsets"][g]:rag["offsets"][g + 1]])
    triples = sorted(((-float(v), g, i) for g in range(wl.Hkv) for i, v in enumerate(rag["a"][g])))[:B]
    counts = np.bincount([t[1] for t in triples], minlength=wl.Hkv)
    np.testing.assert_array_equal(counts, rag["budgets"])
    assert rag["budgets"].sum() == B and np.all(rag["budgets"] <= [k.shape[0] for k in K_list])


def test_ragged_compress_equals_left_padded_selection_with_excluded_padding():
    # the layout the CUDA path uses: heads right-aligned in a common length, padding scored below every real entry
    wl, L, K_list, V_list = _ragged_case(cut=(0, 37))
    cut = (0, 37)
    rag = oc.compress_layer_ragged(L.Qw, K_list, V_list, L.WO, kp=wl.kp, budget_mode="adaptive", budget=90)
    n = wl.n
    a = np.full((wl.Hkv, n), -1.0, np.float32)
    c = np.full((wl.Hkv, n), -1.0, np.float32)
    for g in range(wl.Hkv):
        a[g, cut[g]:], c[g, cut[g]:] = rag["a"][g], rag["c"][g]
    budgets = oc.allocate_budgets(a, "adaptive", 90)
    np.testing.assert_array_equal(budgets, rag["budgets"])
    for g in range(wl.Hkv):
        S1, S2 = oc.two_stage_select(a[g], c[g], int(budgets[g]), 0.5)
        got = np.sort(np.concatenate([S1, S2])) - cut[g]
        np.testing.assert_array_equal(got, rag["idx"][rag["offsets"][g]:rag["offsets"][g + 1]])


def test_chunked_compress_adaptive_budgets_leave_a_ragged_cache():
    from gen import make_layer, small_workload
    wl = small_workload(n=120, w=8, kp=5, budget=30, cfg_id=73)
    L = make_layer(wl)
    L2 = make_layer(wl.with_(n=60), 1)
    chunks = [(L.Qw, L.K, L.V), (L2.Qw, L2.K, L2.V)]
    K1, V1, pos1, hist1 = oc.chunked_compress(chunks[:1], L.WO, kp=wl.kp, w=wl.w, budgets=[70], budget_mode="adaptive")
    ref = oc.compress_layer(L.Qw, L.K, L.V, L.WO, kp=wl.kp, budget_mode="adaptive", budget=70)
    for g in range(wl.Hkv):
        np.testing.assert_array_equal(pos1[g], ref["idx"][ref["offsets"][g]:ref["offsets"][g + 1]])
    K2, V2, pos2, hist2 = oc.chunked_compress(chunks, L.WO, kp=wl.kp, w=wl.w, budgets=[70, 90],
                                              budget_mode="adaptive")
    assert sum(p.size for p in pos2) == 90
    for g in range(wl.Hkv):
        assert np.all(np.diff(pos2[g]) > 0) and pos2[g].max() < 180
        assert set(pos2[g][pos2[g] < 120].tolist()) <= set(pos1[g].tolist())
        for p, krow, vrow in zip(pos2[g], K2[g], V2[g]):
            np.testing.assert_array_equal(krow, L.K[g][p] if p < 120 else L2.K[g][p - 120])
            np.testing.assert_array_equal(vrow, L.V[g][p] if p < 120 else L2.V[g][p - 120])


def test_compress_layer_end_to_end_small():
    from gen import make_layer, small_workload
    wl = small_workload(n=96, w=8, kp=5, budget=20)
    L = make_layer(wl)
    out = oc.compress_layer(L.Qw, L.K, L.V, L.WO, kp=wl.kp, budget_mode="uniform", budget=wl.budget,
                            K_store=L.K_store, V_store=L.V_store)
    assert out["idx"].size == wl.Hkv * wl.budget
    for g in range(wl.Hkv):
        seg = out["idx"][g * wl.budget:(g + 1) * wl.budget]
        np.testing.assert_array_equal(out["K_hat"][g * wl.budget:(g + 1) * wl.budget], L.K_store[g][seg])
        np.testing.assert_array_equal(out["V_hat"][g * wl.budget:(g + 1) * wl.budget], L.V_store[g][seg])


# ----------------------------------------------------------------------------- equalities between the bounds
def test_bounds_coincide_where_the_theorems_say_so():
    r = RNG(77)
    for trial in range(20):
        n = int(r.integers(4, 12))
        A = r.random(n) ** 3
        A /= A.sum()
        nu = np.exp(r.standard_normal(n))
        order = np.argsort(-A)
        k1 = np.zeros(n, bool)
        k1[order[: int(r.integers(1, n - 1))]] = True
        rest = np.flatnonzero(~k1)
        k2 = np.zeros(n, bool)
        k2[r.choice(rest, size=int(r.integers(1, rest.size + 1)), replace=False)] = True
        none = np.zeros(n, bool)
        # Theorem 3.5 with an empty second stage is Theorem 3.3 for the stage-1 set (sigma is then the kept mass)
        assert abs(oc.theta_hat_bound(A, nu, k1, none) - oc.theta_bound(A, nu, k1)) < 1e-12
        # the relaxed bound replaces nu_i of the stage-2 entries by M = min nu: equal when nu is constant
        flat = np.full(n, float(nu[0]))
        assert abs(oc.theta_hat_bound(A, flat, k1, k2) - oc.theta_relax_bound(A, flat, k1, k2)) < 1e-12
        # keeping every entry leaves nothing to perturb
        assert abs(oc.theta_bound(A, nu, np.ones(n, bool))) < 1e-12


def test_bounds_on_a_case_worked_by_hand():
    # A = (0.5, 0.3, 0.2), nu = (2, 1, 4): C = 1.0 + 0.3 + 0.8 = 2.1.  Stage 1 keeps entries 0 and 1:
    # sigma = 0.8, 2 - 1/sigma = 0.75, sum of A nu over stage 1 = 1.3.  Stage 2 keeps entry 2 (A nu = 0.8, A = 0.2).
    A, nu = np.array([0.5, 0.3, 0.2]), np.array([2.0, 1.0, 4.0])
    k1, k2 = np.array([True, True, False]), np.array([False, False, True])
    assert abs(oc.theta_hat_bound(A, nu, k1, k2) - (2.1 - 0.75 * 1.3 - 0.75 * 0.8)) < 1e-12       # 0.525
    assert abs(oc.theta_relax_bound(A, nu, k1, k2) - (2.1 - 0.75 * 1.3 - 1.0 * 0.75 * 0.2)) < 1e-12  # 0.975
    assert abs(oc.theta_bound(A, nu, k1) - (2.1 - 0.75 * 1.3)) < 1e-12                             # 1.125
