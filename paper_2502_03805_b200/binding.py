"""ctypes binding of libcriticalkv: argument marshalling only.

Every function has the name and argument order of its C entry point (include/criticalkv.h) and forwards device
pointers of torch tensors (or raw integer addresses).  No arithmetic happens here.  If the shared library has not
been built, loading raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

# CRITICALKV_LIB may point at another build of the same library (e.g. one compiled with different tile shapes)
_LIB_PATH = os.environ.get("CRITICALKV_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)),
                                                             "libcriticalkv.so")
_lib = None

CKV_OK, CKV_EINVAL, CKV_ENOTSUP, CKV_EALIGN, CKV_EWORKSPACE, CKV_ECUDA, CKV_ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
CKV_F32, CKV_BF16 = 0, 1
CKV_BUDGET_UNIFORM, CKV_BUDGET_FLAT_ADAPTIVE, CKV_BUDGET_GIVEN = 0, 1, 2
CKV_NORM_L1, CKV_NORM_L2 = 0, 1
CKV_FLAG_WO_SHARED, CKV_FLAG_FORCE_SIMT, CKV_FLAG_WO_GROUP_SUM, CKV_FLAG_PROTECT_WINDOW = 1, 2, 4, 8
CKV_FLAG_SELECT_MULTIPASS = 32
CKV_FLAG_SELECT_SINGLE_KERNEL = 16
CKV_FLAG_SELECT_NO_CLUSTER = 256
CKV_FLAG_DEBUG_CHECKS = 64
CKV_FLAG_REQUIRE_TENSOR_CORES = 128
CKV_EBOUNDS = -7
CKV_SELFTEST_MAX_WAIT_NS = 100_000_000
CKV_STATIC_SCRATCH_BYTES = (8 << 20) + (64 << 10)

EXPORTS = ("criticalkv_create", "criticalkv_destroy", "criticalkv_workspace_bytes", "criticalkv_score",
           "criticalkv_select", "criticalkv_group_scores", "criticalkv_allocate_budgets",
           "criticalkv_select_static", "criticalkv_compact", "criticalkv_gather_positions", "criticalkv_compress",
           "criticalkv_host_staging_bytes", "criticalkv_compress_host", "criticalkv_selftest_bounded_wait",
           "criticalkv_diagnose_workspace_bytes", "criticalkv_diagnose", "criticalkv_device_status",
           "criticalkv_status_string", "criticalkv_last_cuda_error", "criticalkv_last_path",
           "criticalkv_launch_count")


class criticalkv_desc(C.Structure):
    _fields_ = [("nb", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("dh", C.c_int32), ("dm", C.c_int32),
                ("n", C.c_int32), ("w", C.c_int32), ("pool_k", C.c_int32), ("dtype", C.c_int32),
                ("scale", C.c_float), ("alpha", C.c_float), ("eps", C.c_float),
                ("budget_mode", C.c_int32), ("norm", C.c_int32), ("budget", C.c_int64),
                ("flags", C.c_uint32), ("reserved", C.c_uint32),
                ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 3), ("v_stride", C.c_int64 * 3),
                ("adaptive_floor", C.c_float), ("reserved2", C.c_uint32), ("valid_from", C.c_void_p)]


class CriticalKVError(RuntimeError):
    def __init__(self, status, where, detail=""):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status}) {detail}".strip())


def library_path() -> str:
    return _LIB_PATH


def load():
    """Load libcriticalkv.so (once).  Raises if it is missing: build it with paper_2502_03805_b200.build."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2502_03805_b200.build` (needs nvcc); "
                           "there is no CPU fallback")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    dp = C.POINTER(criticalkv_desc)
    lib.criticalkv_create.argtypes = [C.POINTER(vp), i32]
    lib.criticalkv_destroy.argtypes = [vp]
    lib.criticalkv_workspace_bytes.argtypes = [dp, C.POINTER(sz), C.POINTER(sz)]
    lib.criticalkv_score.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.criticalkv_select.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.criticalkv_group_scores.argtypes = [vp, dp, vp, vp, vp, vp, vp]
    lib.criticalkv_allocate_budgets.argtypes = [vp, dp, vp, vp, vp]
    lib.criticalkv_select_static.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp]
    lib.criticalkv_compact.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp]
    lib.criticalkv_gather_positions.argtypes = [vp, dp, vp, vp, vp, vp, vp]
    lib.criticalkv_compress.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.criticalkv_host_staging_bytes.argtypes = [dp, C.POINTER(sz)]
    lib.criticalkv_compress_host.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.criticalkv_diagnose_workspace_bytes.argtypes = [dp, C.POINTER(sz)]
    lib.criticalkv_diagnose.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.criticalkv_selftest_bounded_wait.argtypes = [vp, C.c_uint64, vp, vp]
    lib.criticalkv_device_status.argtypes = [vp, vp, C.POINTER(i32)]
    lib.criticalkv_status_string.argtypes = [i32]
    lib.criticalkv_status_string.restype = C.c_char_p
    lib.criticalkv_last_cuda_error.argtypes = [vp]
    lib.criticalkv_last_cuda_error.restype = C.c_char_p
    lib.criticalkv_last_path.argtypes = [vp]
    lib.criticalkv_launch_count.argtypes = [vp]
    lib.criticalkv_launch_count.restype = C.c_int64
    _lib = lib
    return lib


def _ptr(x):
    """Device (or host) address of a tensor / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return C.c_void_p(x)
    return C.c_void_p(x.data_ptr())


def _stream(stream):
    if stream is None:
        return None
    if isinstance(stream, int):
        return C.c_void_p(stream)
    return C.c_void_p(stream.cuda_stream)


def _nbytes(ws, ws_bytes):
    if ws_bytes is not None:
        return ws_bytes
    return 0 if ws is None or isinstance(ws, int) else ws.numel() * ws.element_size()


def status_string(status: int) -> str:
    return load().criticalkv_status_string(int(status)).decode()


def make_desc(*, nb, Hq, Hkv, dh, dm, n, w, pool_k, dtype, budget_mode, budget, alpha=0.5, eps=1e-4, scale=0.0,
              flags=0, norm=CKV_NORM_L1, q_stride=(0, 0, 0), k_stride=(0, 0, 0), v_stride=(0, 0, 0),
              adaptive_floor=0.0, valid_from=None):
    """valid_from: device int32 tensor [nb, Hkv] (or an address) for right-aligned ragged heads; the caller keeps it
    alive while the descriptor is in use."""
    d = criticalkv_desc()
    d.nb, d.Hq, d.Hkv, d.dh, d.dm, d.n, d.w, d.pool_k = nb, Hq, Hkv, dh, dm, n, w, pool_k
    d.dtype = {"f32": CKV_F32, "bf16": CKV_BF16}.get(dtype, dtype)
    d.scale, d.alpha, d.eps = scale, alpha, eps
    d.budget_mode = {"uniform": CKV_BUDGET_UNIFORM, "adaptive": CKV_BUDGET_FLAT_ADAPTIVE,
                     "given": CKV_BUDGET_GIVEN}.get(budget_mode, budget_mode)
    d.norm, d.budget, d.flags, d.reserved = norm, budget, flags, 0
    d.q_stride[:] = q_stride
    d.k_stride[:] = k_stride
    d.v_stride[:] = v_stride
    d.adaptive_floor, d.reserved2 = adaptive_floor, 0
    d.valid_from = None if valid_from is None else (valid_from if isinstance(valid_from, int)
                                                    else valid_from.data_ptr())
    return d


def criticalkv_create(device: int = 0):
    h = C.c_void_p()
    rc = load().criticalkv_create(C.byref(h), int(device))
    if rc != CKV_OK:
        raise CriticalKVError(rc, "criticalkv_create")
    return h


def criticalkv_destroy(handle):
    return load().criticalkv_destroy(handle)


def criticalkv_workspace_bytes(desc, check=True):
    a, b = C.c_size_t(), C.c_size_t()
    rc = load().criticalkv_workspace_bytes(C.byref(desc), C.byref(a), C.byref(b))
    if rc != CKV_OK:
        if check:
            raise CriticalKVError(rc, "criticalkv_workspace_bytes")
        return rc
    return a.value, b.value


def _check(handle, rc, where, check):
    if check and rc != CKV_OK:
        detail = load().criticalkv_last_cuda_error(handle).decode() if rc == CKV_ECUDA else ""
        raise CriticalKVError(rc, where, detail)
    return rc


def criticalkv_score(handle, desc, Qw, K, V, WO, attn, vnorm, ws, ws_bytes=None, stream=None, check=True):
    rc = load().criticalkv_score(handle, C.byref(desc), _ptr(Qw), _ptr(K), _ptr(V), _ptr(WO), _ptr(attn),
                                 _ptr(vnorm), _ptr(ws), _nbytes(ws, ws_bytes), _stream(stream))
    return _check(handle, rc, "criticalkv_score", check)


def criticalkv_select(handle, desc, attn, vnorm, budgets_in, idx, offsets, stage, ws, ws_bytes=None, stream=None,
                      check=True):
    rc = load().criticalkv_select(handle, C.byref(desc), _ptr(attn), _ptr(vnorm), _ptr(budgets_in), _ptr(idx),
                                  _ptr(offsets), _ptr(stage), _ptr(ws), _nbytes(ws, ws_bytes), _stream(stream))
    return _check(handle, rc, "criticalkv_select", check)


def criticalkv_group_scores(handle, desc, attn, vnorm, a_out, c_out=None, stream=None, check=True):
    rc = load().criticalkv_group_scores(handle, C.byref(desc), _ptr(attn), _ptr(vnorm), _ptr(a_out), _ptr(c_out),
                                        _stream(stream))
    return _check(handle, rc, "criticalkv_group_scores", check)


def criticalkv_allocate_budgets(handle, desc, a, budgets_out, stream=None, check=True):
    rc = load().criticalkv_allocate_budgets(handle, C.byref(desc), _ptr(a), _ptr(budgets_out), _stream(stream))
    return _check(handle, rc, "criticalkv_allocate_budgets", check)


def criticalkv_select_static(handle, desc, attn, vnorm, budgets_in, idx, offsets, stage, stream=None, check=True):
    """criticalkv_select without a workspace argument: the scratch is a fixed array inside the library, for callers
    that cannot allocate device memory when they compress (memory fully handed to their own pools, or a loop that
    must not hit the synchronisation an allocation implies).  Shapes whose select workspace exceeds
    CKV_STATIC_SCRATCH_BYTES are refused with CKV_EWORKSPACE; calls share the array, so do not let two overlap."""
    rc = load().criticalkv_select_static(handle, C.byref(desc), _ptr(attn), _ptr(vnorm), _ptr(budgets_in), _ptr(idx),
                                         _ptr(offsets), _ptr(stage), _stream(stream))
    return _check(handle, rc, "criticalkv_select_static", check)


def criticalkv_compact(handle, desc, K, V, idx, offsets, K_out, V_out, stream=None, check=True):
    rc = load().criticalkv_compact(handle, C.byref(desc), _ptr(K), _ptr(V), _ptr(idx), _ptr(offsets), _ptr(K_out),
                                   _ptr(V_out), _stream(stream))
    return _check(handle, rc, "criticalkv_compact", check)


def criticalkv_gather_positions(handle, desc, pos_in, idx, offsets, pos_out, stream=None, check=True):
    rc = load().criticalkv_gather_positions(handle, C.byref(desc), _ptr(pos_in), _ptr(idx), _ptr(offsets),
                                            _ptr(pos_out), _stream(stream))
    return _check(handle, rc, "criticalkv_gather_positions", check)


def criticalkv_compress(handle, desc, Qw, K, V, WO, budgets_in, attn, vnorm, idx, offsets, stage, K_out, V_out, ws,
                        ws_bytes=None, stream=None, check=True):
    rc = load().criticalkv_compress(handle, C.byref(desc), _ptr(Qw), _ptr(K), _ptr(V), _ptr(WO), _ptr(budgets_in),
                                    _ptr(attn), _ptr(vnorm), _ptr(idx), _ptr(offsets), _ptr(stage), _ptr(K_out),
                                    _ptr(V_out), _ptr(ws), _nbytes(ws, ws_bytes), _stream(stream))
    return _check(handle, rc, "criticalkv_compress", check)


def criticalkv_host_staging_bytes(desc):
    out = C.c_size_t()
    rc = load().criticalkv_host_staging_bytes(C.byref(desc), C.byref(out))
    if rc != CKV_OK:
        raise CriticalKVError(rc, "criticalkv_host_staging_bytes")
    return out.value


def criticalkv_compress_host(handle, desc, Qw, K, V, WO, budgets_in, idx, offsets, K_out, V_out, staging,
                             staging_bytes=None, stream=None, check=True):
    """Host tensors in (Qw, K, V, WO[, budgets_in]) and out (idx, offsets, K_out, V_out); `staging` is device memory."""
    rc = load().criticalkv_compress_host(handle, C.byref(desc), _ptr(Qw), _ptr(K), _ptr(V), _ptr(WO),
                                         _ptr(budgets_in), _ptr(idx), _ptr(offsets), _ptr(K_out), _ptr(V_out),
                                         _ptr(staging), _nbytes(staging, staging_bytes), _stream(stream))
    return _check(handle, rc, "criticalkv_compress_host", check)


DIAG_FIELDS = ("sigma", "mass_kept", "C", "C_stage1", "C_stage2", "nu_min", "L", "theta", "theta_hat", "theta_relax")


def criticalkv_diagnose_workspace_bytes(desc):
    out = C.c_size_t()
    rc = load().criticalkv_diagnose_workspace_bytes(C.byref(desc), C.byref(out))
    if rc != CKV_OK:
        raise CriticalKVError(rc, "criticalkv_diagnose_workspace_bytes")
    return out.value


def criticalkv_diagnose(handle, desc, Qw, K, V, WO, vnorm, idx, offsets, stage, diag, ws, ws_bytes=None, stream=None,
                        check=True):
    rc = load().criticalkv_diagnose(handle, C.byref(desc), _ptr(Qw), _ptr(K), _ptr(V), _ptr(WO), _ptr(vnorm),
                                    _ptr(idx), _ptr(offsets), _ptr(stage), _ptr(diag), _ptr(ws),
                                    _nbytes(ws, ws_bytes), _stream(stream))
    return _check(handle, rc, "criticalkv_diagnose", check)


def criticalkv_selftest_bounded_wait(handle, limit_ns, observed, stream=None, check=True):
    rc = load().criticalkv_selftest_bounded_wait(handle, int(limit_ns), _ptr(observed), _stream(stream))
    return _check(handle, rc, "criticalkv_selftest_bounded_wait", check)


def criticalkv_device_status(handle, stream=None):
    out = C.c_int(0)
    rc = load().criticalkv_device_status(handle, _stream(stream), C.byref(out))
    if rc != CKV_OK:
        raise CriticalKVError(rc, "criticalkv_device_status")
    return out.value


def criticalkv_last_path(handle) -> int:
    return load().criticalkv_last_path(handle)


def criticalkv_launch_count(handle) -> int:
    return load().criticalkv_launch_count(handle)
