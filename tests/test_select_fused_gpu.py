"""Steps 3-4 on the GPU: the single-kernel selection, the multi-kernel selection with a cluster of CTAs per head and the
multi-kernel selection with one CTA per head against the oracle on identical float32 scores, where every integer
decision must agree bit for bit (Algorithm 1, stage 1 / stage 2; Algorithm 2, budget allocation)."""
import numpy as np
import pytest
import torch

from gen import small_workload
from oracle import criticalkv_oracle as oc

pytestmark = pytest.mark.gpu

FUSED_BIT = 32
CLUSTER_BIT = 64


def _paths():
    """(flags, single kernel ran, cluster kernel ran) of the three implementations of steps 3-4 for a call with few
    heads; without flags such a call takes the cluster path."""
    from paper_2502_03805_b200 import binding as B
    return [(B.CKV_FLAG_SELECT_SINGLE_KERNEL, True, False), (0, False, True),
            (B.CKV_FLAG_SELECT_MULTIPASS, False, True),
            (B.CKV_FLAG_SELECT_MULTIPASS | B.CKV_FLAG_SELECT_NO_CLUSTER, False, False)]


def _select(P, nu, wl, *, flags=0, budgets_in=None, nb=1, adaptive_floor=0.0):
    """P, nu: [nb, Hq, n] float32 scores fed to criticalkv_select unchanged."""
    from paper_2502_03805_b200 import session_for
    s = session_for(wl, nb=nb, flags=flags, adaptive_floor=adaptive_floor)
    attn = torch.from_numpy(np.ascontiguousarray(P, dtype=np.float32)).cuda()
    vnorm = torch.from_numpy(np.ascontiguousarray(nu, dtype=np.float32)).cuda()
    bi = None if budgets_in is None else torch.tensor(budgets_in, dtype=torch.int32, device="cuda")
    s.select(attn, vnorm, budgets_in=bi)
    torch.cuda.synchronize()
    assert s.device_status() == 0
    return s.idx.cpu().numpy(), s.offsets.cpu().numpy(), s.stage.cpu().numpy(), s.last_path


def _check_against_oracle(P, nu, wl, G, *, flags=0, expect_fused=None, expect_cluster=None, budgets_in=None,
                          adaptive_floor=0.0, **okw):
    nb = P.shape[0]
    idx, off, st, path = _select(P, nu, wl, flags=flags, budgets_in=budgets_in, nb=nb, adaptive_floor=adaptive_floor)
    if expect_fused is not None:
        assert bool(path & FUSED_BIT) == expect_fused, path
    if expect_cluster is not None:
        assert bool(path & CLUSTER_BIT) == expect_cluster, path
    for b in range(nb):
        ref = oc.select(P[b], nu[b], G=G, budget_mode=wl.budget_mode, budget=wl.budget, alpha=wl.alpha, eps=wl.eps,
                        budgets_in=None if budgets_in is None else budgets_in[b], adaptive_floor=adaptive_floor, **okw)
        np.testing.assert_array_equal(off[b], ref["offsets"])
        tot = ref["offsets"][-1]
        np.testing.assert_array_equal(idx[b][:tot], ref["idx"])
        np.testing.assert_array_equal(st[b][:tot], ref["stage"])
    return idx, off, st


def _scores(seed, nb, Hq, n, ties=False, pooled=False):
    r = np.random.default_rng(seed)
    P = r.random((nb, Hq, n)).astype(np.float32) ** 8
    nu = np.exp(r.standard_normal((nb, Hq, n))).astype(np.float32)
    if pooled:   # runs of equal neighbours, as the max-pool of Algorithm 2 leaves them
        from scipy.ndimage import maximum_filter1d
        P = maximum_filter1d(P, size=7, axis=-1, mode="nearest").astype(np.float32)
    if ties:
        P = (np.round(P * 8) / 8).astype(np.float32)
        nu = np.round(nu).astype(np.float32)
    return P, nu


SHAPES = [
    # Hq, Hkv, n, mode, budget, alpha
    (12, 4, 1237, "uniform", 97, 0.5),       # n neither a multiple of 4 nor of 32
    (12, 4, 1236, "adaptive", 500, 0.5),     # multiple of 4 only
    (8, 8, 4096, "adaptive", 6553, 0.5),
    (32, 8, 4096, "uniform", 819, 0.5),
    (10, 2, 2048, "adaptive", 1000, 0.25),
    (5, 1, 999, "adaptive", 333, 0.5),       # cluster of one CTA
    (6, 6, 640, "uniform", 640, 0.5),        # everything kept
    (6, 6, 640, "uniform", 0, 0.5),          # nothing kept
    (4, 4, 515, "uniform", 1, 0.5),          # b' = 0
    (4, 4, 515, "uniform", 100, 1.0),        # attention only
    (4, 4, 515, "uniform", 100, 0.0),        # perturbation-aware score only
    (16, 8, 32768, "adaptive", 52428, 0.5),  # one layer of the headline shape
]


@pytest.mark.parametrize("case", range(len(SHAPES)))
@pytest.mark.parametrize("kind", ["plain", "pooled", "ties"])
def test_all_selection_paths_match_the_oracle(case, kind):
    Hq, Hkv, n, mode, budget, alpha = SHAPES[case]
    if n > 8192 and kind == "ties":
        pytest.skip("the large shape is run on the two realistic score kinds")
    from paper_2502_03805_b200 import binding as B
    nb = 1 if n > 8192 else 2
    P, nu = _scores(100 + case, nb, Hq, n, ties=kind == "ties", pooled=kind == "pooled")
    wl = small_workload(cfg_id=150 + case, Hq=Hq, Hkv=Hkv, n=n, budget_mode=mode, budget=budget, alpha=alpha)
    outs = [_check_against_oracle(P, nu, wl, Hq // Hkv, flags=f, expect_fused=fu, expect_cluster=cl)
            for f, fu, cl in _paths()]
    for other in outs[1:]:
        for x, y in zip(outs[0], other):
            np.testing.assert_array_equal(x, y)


def test_threshold_bin_larger_than_the_candidate_list_takes_the_full_walk():
    # stage 2 scores with three distinct values over 20000 entries: the bin of the threshold holds far more entries
    # than the candidate list, and the ties inside it are resolved by index
    r = np.random.default_rng(7)
    Hq, Hkv, n = 4, 2, 20000
    P = (r.random((1, Hq, n)).astype(np.float32) ** 4)
    nu = r.integers(1, 3, size=(1, Hq, n)).astype(np.float32)
    P[:] = np.float32(0.25)        # equal attention: c = (0.25 + eps) * nu takes three values per head pair
    for f, fu, cl in _paths():
        wl = small_workload(cfg_id=170, Hq=Hq, Hkv=Hkv, n=n, budget_mode="uniform", budget=9000)
        _check_against_oracle(P, nu, wl, 2, flags=f, expect_fused=fu, expect_cluster=cl)
        wl = small_workload(cfg_id=171, Hq=Hq, Hkv=Hkv, n=n, budget_mode="adaptive", budget=17001)
        _check_against_oracle(P, nu, wl, 2, flags=f, expect_fused=fu, expect_cluster=cl)


def test_ties_at_the_stage_two_threshold_go_to_the_lower_index():
    # few distinct c values inside one threshold bin, list not exceeded: the index rounds decide
    r = np.random.default_rng(8)
    Hq, Hkv, n = 2, 2, 3000
    P = np.full((1, Hq, n), 0.5, np.float32)
    P[..., ::7] = 0.75
    nu = r.integers(1, 3, size=(1, Hq, n)).astype(np.float32)
    for budget in (700, 1501, 2999):
        wl = small_workload(cfg_id=172, Hq=Hq, Hkv=Hkv, n=n, budget_mode="uniform", budget=budget)
        for f, fu, cl in _paths():
            _check_against_oracle(P, nu, wl, 1, flags=f, expect_fused=fu, expect_cluster=cl)


def test_long_heads_and_heads_beyond_the_single_kernel_limit():
    # several words per thread in every walk
    P, nu = _scores(9, 1, 4, 70001)
    wl = small_workload(cfg_id=173, Hq=4, Hkv=2, n=70001, budget_mode="adaptive", budget=14000)
    for f, fu, cl in _paths():
        _check_against_oracle(P, nu, wl, 2, flags=f, expect_fused=fu, expect_cluster=cl)
    # more than 4096 words per head: beyond the single kernel, which hands the call to the separate kernels
    P, nu = _scores(10, 1, 2, 140003)
    wl = small_workload(cfg_id=177, Hq=2, Hkv=2, n=140003, budget_mode="adaptive", budget=28000)
    for f, fu, cl in _paths():
        _check_against_oracle(P, nu, wl, 1, flags=f, expect_fused=False, expect_cluster=cl or fu)


@pytest.mark.parametrize("floor", [0.0, 0.3, 1.0])
@pytest.mark.parametrize("protect", [False, True])
def test_floor_protected_window_and_given_budgets_on_both_paths(floor, protect):
    from paper_2502_03805_b200 import binding as B
    r = np.random.default_rng(11)
    Hq, Hkv, n, w, budget = 8, 4, 900, 8, 700
    P = r.random((1, Hq, n)).astype(np.float32) ** 6
    P[:, :4] *= 20
    P[..., n - w:] *= 1e-3
    nu = np.exp(r.standard_normal((1, Hq, n))).astype(np.float32)
    wl = small_workload(cfg_id=174, Hq=Hq, Hkv=Hkv, n=n, w=w, budget_mode="adaptive", budget=budget)
    pf = B.CKV_FLAG_PROTECT_WINDOW if protect else 0
    for f, fused, cl in _paths():
        _check_against_oracle(P, nu, wl, 2, flags=pf | f, expect_fused=fused, expect_cluster=cl, adaptive_floor=floor,
                              protect_w=w if protect else 0)
    wl = small_workload(cfg_id=175, Hq=Hq, Hkv=Hkv, n=n, w=w, budget_mode="given", budget=1200)
    budgets = [[0, 900, 17, 100]]
    for f, fused, cl in _paths():
        _check_against_oracle(P, nu, wl, 2, flags=pf | f, expect_fused=fused, expect_cluster=cl, budgets_in=budgets,
                              protect_w=w if protect else 0)


def test_group_summed_scores_on_both_paths():
    from paper_2502_03805_b200 import binding as B
    r = np.random.default_rng(12)
    Hq, Hkv, n = 8, 2, 2052
    P = r.random((2, Hq, n)).astype(np.float32) ** 5
    nu = np.exp(r.standard_normal((2, Hkv, n))).astype(np.float32)     # one norm per KV head
    wl = small_workload(cfg_id=176, Hq=Hq, Hkv=Hkv, n=n, budget_mode="adaptive", budget=800)
    for f, fused, cl in _paths():
        _check_against_oracle(P, nu, wl, 4, flags=B.CKV_FLAG_WO_GROUP_SUM | f, expect_fused=fused, expect_cluster=cl,
                              group_sum=True)


@pytest.mark.parametrize("nb,Hkv,G,mode,budget", [(48, 8, 2, "adaptive", 900), (60, 6, 1, "adaptive", 777),
                                                  (70, 5, 3, "uniform", 101)])
def test_more_heads_than_resident_ctas(nb, Hkv, G, mode, budget):
    # more (slice, KV head) items than the GPU holds CTAs of the single kernel: every CTA works on several items, and
    # the heads of a slice still meet at their barriers (the grid is a multiple of Hkv)
    n = 700
    P, nu = _scores(40 + Hkv, nb, Hkv * G, n, pooled=True)
    wl = small_workload(cfg_id=180 + Hkv, Hq=Hkv * G, Hkv=Hkv, n=n, budget_mode=mode, budget=budget)
    _check_against_oracle(P, nu, wl, G, expect_fused=True, expect_cluster=False)


@pytest.mark.parametrize("nb,Hkv", [(3, 8), (5, 4), (9, 8), (37, 2)])
def test_cluster_sizes_eight_four_and_two(nb, Hkv):
    # the number of CTAs per head shrinks as the call has more heads (8 up to 13 heads, 4 up to 27, 2 up to 74)
    n, G = 5000, 2
    P, nu = _scores(60 + nb, nb, Hkv * G, n, pooled=True)
    for mode, budget in (("uniform", 611), ("adaptive", 611 * Hkv)):
        wl = small_workload(cfg_id=190 + Hkv, Hq=Hkv * G, Hkv=Hkv, n=n, budget_mode=mode, budget=budget)
        _check_against_oracle(P, nu, wl, G, expect_fused=False, expect_cluster=True)
