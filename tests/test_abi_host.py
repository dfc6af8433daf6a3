"""Host-side checks of the C ABI that need no GPU: the library loads, exports what the header declares, and rejects
bad descriptors before any CUDA call."""
import os
import re

import pytest

from paper_2502_03805_b200 import binding as B
from paper_2502_03805_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.load()


def _desc(**kw):
    base = dict(nb=1, Hq=4, Hkv=2, dh=64, dm=256, n=512, w=16, pool_k=5, dtype="f32", budget_mode="uniform",
                budget=128)
    base.update(kw)
    return B.make_desc(**base)


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "criticalkv.h")).read()
    declared = re.findall(r"CKV_API\s+[\w\s\*]+?\b(criticalkv_\w+)\s*\(", header)
    assert len(declared) >= 12 and set(declared) == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert B.status_string(B.CKV_OK) == "ok"
    assert "aligned" in B.status_string(B.CKV_EALIGN)
    assert "unknown" in B.status_string(-99)


def test_workspace_bytes_are_sane(lib):
    sb, tb = B.criticalkv_workspace_bytes(_desc())
    assert sb % 256 == 0 and tb % 256 == 0
    assert sb >= 4 * 512 * 4 and tb >= 2 * 2 * 512 * 4
    sb2, tb2 = B.criticalkv_workspace_bytes(_desc(nb=3))
    assert sb2 > sb and tb2 > tb
    # every documented flag is accepted, alone and together with the others of its group
    for flags in (B.CKV_FLAG_SELECT_MULTIPASS, B.CKV_FLAG_SELECT_SINGLE_KERNEL, B.CKV_FLAG_SELECT_NO_CLUSTER,
                  B.CKV_FLAG_SELECT_MULTIPASS | B.CKV_FLAG_SELECT_NO_CLUSTER, B.CKV_FLAG_DEBUG_CHECKS,
                  B.CKV_FLAG_REQUIRE_TENSOR_CORES, B.CKV_FLAG_PROTECT_WINDOW, B.CKV_FLAG_WO_SHARED):
        assert B.criticalkv_workspace_bytes(_desc(flags=flags)) == (sb, tb) or flags == B.CKV_FLAG_WO_SHARED


@pytest.mark.parametrize("kw,status", [
    (dict(nb=0), B.CKV_EINVAL), (dict(Hq=5), B.CKV_EINVAL), (dict(dh=96), B.CKV_ENOTSUP),
    (dict(dm=250), B.CKV_EINVAL), (dict(n=8), B.CKV_EINVAL), (dict(w=0), B.CKV_EINVAL), (dict(w=257, n=512), B.CKV_ENOTSUP),
    (dict(pool_k=4), B.CKV_EINVAL), (dict(pool_k=65), B.CKV_ENOTSUP), (dict(dtype=7), B.CKV_EINVAL),
    (dict(alpha=1.5), B.CKV_EINVAL), (dict(alpha=-0.1), B.CKV_EINVAL), (dict(eps=-1.0), B.CKV_EINVAL),
    (dict(budget=513), B.CKV_EINVAL), (dict(budget=-1), B.CKV_EINVAL),
    (dict(budget_mode="adaptive", budget=2 * 512 + 1), B.CKV_EINVAL), (dict(budget_mode=9), B.CKV_EINVAL),
    (dict(norm=3), B.CKV_EINVAL), (dict(adaptive_floor=1.5), B.CKV_EINVAL), (dict(adaptive_floor=-0.1), B.CKV_EINVAL), (dict(flags=1 << 9), B.CKV_EINVAL), (dict(flags=1 << 31), B.CKV_EINVAL),
    (dict(k_stride=(0, 0, 63)), B.CKV_EALIGN), (dict(k_stride=(0, 0, 32)), B.CKV_EINVAL),
    (dict(Hq=65, Hkv=65), B.CKV_ENOTSUP),      # more KV heads per slice than the selection kernels handle
])
def test_bad_descriptors_are_rejected_on_the_host(lib, kw, status):
    assert B.criticalkv_workspace_bytes(_desc(**kw), check=False) == status


def test_null_handle_and_null_pointers(lib):
    d = _desc()
    assert B.criticalkv_score(None, d, 16, 16, 16, 16, 16, 16, 256, ws_bytes=1 << 20, check=False) == B.CKV_EINVAL
    assert B.criticalkv_select(None, d, 16, 16, None, 16, 16, None, 256, ws_bytes=1 << 20, check=False) == B.CKV_EINVAL
    assert B.criticalkv_compact(None, d, 16, 16, 16, 16, 16, 16, check=False) == B.CKV_EINVAL
    assert B.criticalkv_launch_count(None) == 0 and B.criticalkv_last_path(None) == 0


def test_create_without_a_gpu_reports_an_error_instead_of_crashing(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(B.CriticalKVError):
        B.criticalkv_create(0)
