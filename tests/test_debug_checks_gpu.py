"""Debug checks and guard zones: the substitute for a memory checker.  Every buffer the library is given sits between
guard zones that must be intact after each call on the shapes most likely to run past an edge (n = w, n = w + 1, n off
every tile size, budgets 0 / 1 / n, ragged heads), with CKV_FLAG_DEBUG_CHECKS set; and indices, offsets or budgets
that point outside a buffer are skipped and reported in the status word instead of being used."""
import numpy as np
import pytest
import torch

from canary_util import Guarded, GuardedSession
from gen import make_layer, small_workload
from gpu_util import upload_layers
from paper_2502_03805_b200 import binding as B

pytestmark = pytest.mark.gpu

EDGE_SHAPES = [
    # dtype, Hq, Hkv, dh, dm, n, w, kp, mode, budget
    ("f32", 4, 2, 64, 128, 16, 16, 5, "uniform", 16),       # n = w, everything kept
    ("f32", 4, 2, 64, 128, 17, 16, 5, "uniform", 0),        # n = w + 1, nothing kept
    ("f32", 4, 2, 64, 128, 17, 16, 5, "uniform", 1),
    ("bf16", 8, 2, 128, 256, 33, 32, 7, "uniform", 33),     # tensor-core window, one key more than the window
    ("bf16", 8, 2, 128, 256, 32, 32, 7, "adaptive", 64),    # n = w, B_total = all entries
    ("bf16", 8, 2, 128, 256, 1237, 32, 7, "adaptive", 600), # n off every tile size
    ("bf16", 8, 4, 64, 136, 259, 16, 3, "uniform", 100),    # d_model not a multiple of a tile
    ("f32", 6, 3, 64, 128, 301, 8, 1, "adaptive", 1),
    ("bf16", 8, 2, 128, 256, 4097, 64, 9, "adaptive", 2 * 4097),   # one past a power of two, everything kept
]


@pytest.mark.parametrize("case", range(len(EDGE_SHAPES)))
@pytest.mark.parametrize("multipass", [False, True])
def test_guard_zones_survive_the_edge_shapes(case, multipass):
    dtype, Hq, Hkv, dh, dm, n, w, kp, mode, budget = EDGE_SHAPES[case]
    wl = small_workload(cfg_id=300 + case, dtype=dtype, Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, n=n, w=w, kp=kp,
                        budget_mode=mode, budget=budget)
    L = make_layer(wl, 0)
    Qw, K, V, WO = upload_layers([L, L], wl)
    flags = B.CKV_FLAG_DEBUG_CHECKS | (B.CKV_FLAG_SELECT_MULTIPASS if multipass else 0)
    s = GuardedSession(nb=2, Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, n=n, w=w, pool_k=kp, dtype=dtype, budget_mode=mode,
                       budget=budget, flags=flags)
    assert s.run(Qw, K, V, WO) == 0
    assert s.damaged() == []
    off = s.offsets.cpu().numpy()
    assert (off[:, 0] == 0).all() and (np.diff(off, axis=1) >= 0).all() and (off[:, -1] == s.btot).all()
    idx = s.idx.cpu().numpy()
    for b in range(2):
        for g in range(Hkv):
            seg = idx[b, off[b, g]:off[b, g + 1]]
            assert ((seg >= 0) & (seg < n)).all() and (np.diff(seg) > 0).all()
    s.close()


@pytest.mark.parametrize("dtype,w", [("bf16", 32), ("f32", 8)])
def test_guard_zones_survive_ragged_heads(dtype, w):
    Hq, Hkv, dh, dm, n = 8, 4, 64 if dtype == "f32" else 128, 128, 777
    wl = small_workload(cfg_id=320, dtype=dtype, Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, n=n, w=w, kp=7,
                        budget_mode="adaptive", budget=500)
    L = make_layer(wl, 0)
    Qw, K, V, WO = upload_layers([L], wl)
    vf = torch.tensor([[0, 5, n - w, 300]], dtype=torch.int32, device="cuda")
    s = GuardedSession(nb=1, Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, n=n, w=w, pool_k=7, dtype=dtype, budget_mode="adaptive",
                       budget=500, flags=B.CKV_FLAG_DEBUG_CHECKS, valid_from=vf)
    assert s.run(Qw, K, V, WO) == 0
    assert s.damaged() == []
    off = s.offsets.cpu().numpy()[0]
    idx = s.idx.cpu().numpy()[0]
    for g in range(Hkv):
        assert (idx[off[g]:off[g + 1]] >= int(vf[0, g])).all()     # padding is never selected while budget allows
    s.close()


def _compact_fixture(flags):
    wl = small_workload(cfg_id=330, dtype="bf16", Hq=4, Hkv=2, dh=128, dm=128, n=200, w=16, kp=5,
                        budget_mode="uniform", budget=10)
    L = make_layer(wl, 0)
    _, K, V, _ = upload_layers([L], wl)
    s = GuardedSession(nb=1, Hq=4, Hkv=2, dh=128, dm=128, n=200, w=16, pool_k=5, dtype="bf16", budget_mode="uniform",
                       budget=10, flags=flags)
    return s, K, V


@pytest.mark.parametrize("checks", [True, False])
def test_indices_outside_the_cache_are_skipped_and_reported(checks):
    s, K, V = _compact_fixture(B.CKV_FLAG_DEBUG_CHECKS if checks else 0)
    idx = torch.arange(20, dtype=torch.int32, device="cuda").reshape(1, 20) * 3
    idx[0, 4] = -5          # before the cache
    idx[0, 13] = 200        # one past the last entry
    s.idx.copy_(idx)
    s.offsets.copy_(torch.tensor([[0, 10, 20]], dtype=torch.int32, device="cuda"))
    B.criticalkv_compact(s.handle, s.desc, K, V, s.idx, s.offsets, s.K_out, s.V_out)
    pos_in = torch.arange(2 * 200, dtype=torch.int32, device="cuda").reshape(1, 2, 200)
    pos_out = Guarded((1, 20), torch.int32, fill=-7)
    B.criticalkv_gather_positions(s.handle, s.desc, pos_in, s.idx, s.offsets, pos_out.t)
    torch.cuda.synchronize()
    assert B.criticalkv_device_status(s.handle) == (B.CKV_EBOUNDS if checks else 0)
    assert s.damaged() == [] and pos_out.intact()
    Ko, K16 = s.K_out.view(torch.int16)[0], K.view(torch.int16)[0]
    for r in range(20):
        g, src = r // 10, int(idx[0, r])
        if 0 <= src < 200:
            assert torch.equal(Ko[r], K16[g, src]) and int(pos_out.t[0, r]) == g * 200 + src
        else:
            assert int(Ko[r].abs().sum()) == 0 and int(pos_out.t[0, r]) == -7     # left as they were
    s.close()


def test_offsets_that_decrease_or_exceed_the_capacity_are_reported():
    s, K, V = _compact_fixture(B.CKV_FLAG_DEBUG_CHECKS)
    s.idx.copy_(torch.arange(20, dtype=torch.int32, device="cuda").reshape(1, 20))
    for bad in ([0, 12, 8], [0, 10, 25], [3, 10, 20]):
        s.offsets.copy_(torch.tensor([bad], dtype=torch.int32, device="cuda"))
        B.criticalkv_compact(s.handle, s.desc, K, V, s.idx, s.offsets, s.K_out, s.V_out)
        torch.cuda.synchronize()
        assert B.criticalkv_device_status(s.handle) == B.CKV_EBOUNDS, bad
        assert s.damaged() == []
    s.offsets.copy_(torch.tensor([[0, 10, 20]], dtype=torch.int32, device="cuda"))
    B.criticalkv_compact(s.handle, s.desc, K, V, s.idx, s.offsets, s.K_out, s.V_out)
    torch.cuda.synchronize()
    assert B.criticalkv_device_status(s.handle) == 0
    s.close()


@pytest.mark.parametrize("multipass", [False, True])
def test_given_budgets_beyond_the_capacity_never_write_past_idx(multipass):
    r = np.random.default_rng(3)
    Hq, Hkv, n = 4, 4, 640
    flags = B.CKV_FLAG_DEBUG_CHECKS | (B.CKV_FLAG_SELECT_MULTIPASS if multipass else 0)
    s = GuardedSession(nb=1, Hq=Hq, Hkv=Hkv, dh=64, dm=128, n=n, w=8, pool_k=5, dtype="f32", budget_mode="given",
                       budget=800, flags=flags)
    s.attn.copy_(torch.from_numpy(r.random((1, Hq, n)).astype(np.float32)))
    s.vnorm.copy_(torch.from_numpy(r.random((1, Hq, n)).astype(np.float32)))
    for budgets in ([640, 640, 0, 0], [-3, 900, 100, 100], [0, 0, 0, 801]):
        bi = torch.tensor([budgets], dtype=torch.int32, device="cuda")
        B.criticalkv_select(s.handle, s.desc, s.attn, s.vnorm, bi, s.idx, s.offsets, s.stage, s.ws_select,
                            ws_bytes=s.select_bytes)
        torch.cuda.synchronize()
        assert B.criticalkv_device_status(s.handle) != 0       # clipped budgets are reported
        assert s.damaged() == []
        assert int(s.offsets[0, -1]) <= 800
    s.close()


def test_tensor_cores_can_be_required():
    wl = small_workload(cfg_id=340, dtype="bf16", Hq=4, Hkv=2, dh=128, dm=128, n=300, w=8, kp=5,
                        budget_mode="uniform", budget=30)     # w = 8 is not a tensor-core window
    L = make_layer(wl, 0)
    Qw, K, V, WO = upload_layers([L], wl)
    s = GuardedSession(nb=1, Hq=4, Hkv=2, dh=128, dm=128, n=300, w=8, pool_k=5, dtype="bf16", budget_mode="uniform",
                       budget=30, flags=B.CKV_FLAG_REQUIRE_TENSOR_CORES)
    rc = B.criticalkv_score(s.handle, s.desc, Qw, K, V, WO, s.attn, s.vnorm, s.ws_score, ws_bytes=s.score_bytes,
                            check=False)
    assert rc == B.CKV_ENOTSUP
    s.close()
    wl = wl.with_(w=32)
    L = make_layer(wl, 0)
    Qw, K, V, WO = upload_layers([L], wl)
    s = GuardedSession(nb=1, Hq=4, Hkv=2, dh=128, dm=128, n=300, w=32, pool_k=5, dtype="bf16", budget_mode="uniform",
                       budget=30, flags=B.CKV_FLAG_REQUIRE_TENSOR_CORES)
    assert s.run(Qw, K, V, WO) == 0 and (B.criticalkv_last_path(s.handle) & 3) == 3
    assert s.damaged() == []
    s.close()


def test_self_test_refuses_long_waits():
    h = B.criticalkv_create(0)
    obs = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert B.criticalkv_selftest_bounded_wait(h, B.CKV_SELFTEST_MAX_WAIT_NS + 1, obs, check=False) == B.CKV_EINVAL
    assert B.criticalkv_selftest_bounded_wait(h, 2_000_000, obs, check=False) == B.CKV_OK
    torch.cuda.synchronize()
    assert B.criticalkv_device_status(h) == B.CKV_ETIMEOUT and int(obs[0]) == 0
    B.criticalkv_destroy(h)
