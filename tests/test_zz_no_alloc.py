"""criticalkv_select_static: the selection step for callers that cannot allocate device memory.

A server that gave all of HBM to its own pools, or a loop that must avoid the device-wide synchronisation of
cudaMalloc / cudaFree, cannot hand the library a workspace.  The static variant keeps its scratch in a fixed array
inside the library instead.  It must give exactly the indices, offsets and stage bytes of criticalkv_select (integer
outputs: compared bit for bit), also on a second call that finds the previous call's data in the shared array, and it
must refuse shapes that do not fit the array.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2502_03805_b200 import binding as B
from paper_2502_03805_b200 import session_for
from gen import small_workload

pytestmark = pytest.mark.gpu


def _scores(seed, Hq, n):
    r = np.random.default_rng(seed)
    P = (r.random((1, Hq, n)).astype(np.float32) ** 6)
    P = np.maximum(P, np.roll(P, 1, axis=-1))                 # runs of equal neighbours, like pooled attention
    nu = np.exp(r.standard_normal((1, Hq, n))).astype(np.float32)
    return torch.from_numpy(P).cuda(), torch.from_numpy(nu).cuda()


@pytest.mark.parametrize("mode,budget", [("uniform", 300), ("adaptive", 1500)])
def test_static_select_matches_select_on_two_calls_in_a_row(mode, budget):
    Hq, Hkv, n = 8, 4, 3001
    wl = small_workload(cfg_id=160, Hq=Hq, Hkv=Hkv, n=n, budget_mode=mode, budget=budget)
    ref, sta = session_for(wl), session_for(wl)
    for call, seed in enumerate((11, 12)):                    # second call: new data over the first call's leftovers
        attn, vnorm = _scores(seed, Hq, n)
        ref.select(attn, vnorm)
        B.criticalkv_select_static(sta.handle, sta.desc, attn, vnorm, None, sta.idx, sta.offsets, sta.stage)
        torch.cuda.synchronize()
        assert sta.device_status() == 0
        np.testing.assert_array_equal(sta.offsets.cpu().numpy(), ref.offsets.cpu().numpy())
        tot = int(ref.offsets[0, -1])
        assert tot == wl.btot
        np.testing.assert_array_equal(sta.idx.cpu().numpy()[:, :tot], ref.idx.cpu().numpy()[:, :tot])
        np.testing.assert_array_equal(sta.stage.cpu().numpy()[:, :tot], ref.stage.cpu().numpy()[:, :tot])


def test_static_select_refuses_shapes_beyond_its_scratch():
    Hq, Hkv, n = 8, 8, 131072 + 8192                         # 6% more scored entries than the array holds
    desc = B.make_desc(nb=1, Hq=Hq, Hkv=Hkv, dh=64, dm=128, n=n, w=8, pool_k=5, dtype="f32",
                       budget_mode="uniform", budget=10)
    assert B.criticalkv_workspace_bytes(desc)[1] > B.CKV_STATIC_SCRATCH_BYTES
    h = B.criticalkv_create(0)
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")
    rc = B.criticalkv_select_static(h, desc, dummy, dummy, None, dummy, dummy, None, check=False)
    assert rc == B.CKV_EWORKSPACE
    assert b"holds" in B.load().criticalkv_last_cuda_error(h)
    B.criticalkv_destroy(h)
