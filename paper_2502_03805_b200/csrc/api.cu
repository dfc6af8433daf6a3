// C ABI of libcriticalkv: argument validation, workspace carving and kernel dispatch.
// All checks run on the host before the first launch; nothing here synchronises except criticalkv_device_status.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <new>

#include "ckv_internal.h"

struct criticalkv_handle_s {
  int device;
  int sm_count;
  int cc_major, cc_minor;
  int* status_word;  // device
  int smem_optin;
  int last_path;
  int last_select_fused;
  long long launches;
  char cuda_error[256];
  // host-staged path: two copy/compute streams and the events that tie them to the caller's stream
  bool host_ready;
  cudaStream_t host_stream[2];
  cudaEvent_t host_event[3];
};

namespace {

using ckv::Dims;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int record_cuda(criticalkv_handle h, cudaError_t e) {
  if (e == cudaSuccess) return CKV_OK;
  if (h) snprintf(h->cuda_error, sizeof(h->cuda_error), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
  return CKV_ECUDA;
}

// Validates the descriptor and resolves defaults.  Returns CKV_OK or the status to hand back.
int resolve(const criticalkv_desc* d, Dims* o) {
  if (!d || !o) return CKV_EINVAL;
  if (d->nb < 1 || d->Hq < 1 || d->Hkv < 1 || d->Hq % d->Hkv != 0) return CKV_EINVAL;
  if (d->Hkv > 64) return CKV_ENOTSUP;
  if (d->dh != 64 && d->dh != 128) return CKV_ENOTSUP;
  if (d->dm < 8 || d->dm % 8 != 0) return CKV_EINVAL;
  if (d->w < 1) return CKV_EINVAL;
  if (d->w > 256) return CKV_ENOTSUP;
  if (d->n < d->w) return CKV_EINVAL;
  if (d->pool_k < 1 || d->pool_k % 2 == 0) return CKV_EINVAL;
  if (d->pool_k > 63) return CKV_ENOTSUP;
  if (d->dtype != CKV_F32 && d->dtype != CKV_BF16) return CKV_EINVAL;
  if (!(d->alpha >= 0.f && d->alpha <= 1.f)) return CKV_EINVAL;
  if (!(d->eps >= 0.f) || !isfinite(d->eps)) return CKV_EINVAL;
  if (d->norm != CKV_NORM_L1 && d->norm != CKV_NORM_L2) return CKV_EINVAL;
  if (d->reserved != 0 || d->reserved2 != 0) return CKV_EINVAL;
  if (!(d->adaptive_floor >= 0.f && d->adaptive_floor <= 1.f)) return CKV_EINVAL;
  if (d->flags & ~(uint32_t)(CKV_FLAG_WO_SHARED | CKV_FLAG_FORCE_SIMT | CKV_FLAG_WO_GROUP_SUM |
                             CKV_FLAG_PROTECT_WINDOW | CKV_FLAG_SELECT_MULTIPASS | CKV_FLAG_SELECT_SINGLE_KERNEL |
                             CKV_FLAG_SELECT_NO_CLUSTER |
                             CKV_FLAG_DEBUG_CHECKS | CKV_FLAG_REQUIRE_TENSOR_CORES))
    return CKV_EINVAL;
  if (d->budget < 0) return CKV_EINVAL;
  if ((long long)d->n * d->Hkv > 0x7fffffffLL) return CKV_ENOTSUP;
  o->nb = d->nb; o->Hq = d->Hq; o->Hkv = d->Hkv; o->G = d->Hq / d->Hkv;
  o->dh = d->dh; o->dm = d->dm; o->n = d->n; o->w = d->w; o->kp = d->pool_k; o->dtype = d->dtype;
  o->scale = d->scale > 0.f ? d->scale : (float)(1.0 / sqrt((double)d->dh));
  o->alpha = d->alpha; o->eps = d->eps;
  o->budget_mode = d->budget_mode; o->budget = d->budget;
  switch (d->budget_mode) {
    case CKV_BUDGET_UNIFORM:
      if (d->budget > d->n) return CKV_EINVAL;
      o->btot = (long long)d->budget * d->Hkv;
      break;
    case CKV_BUDGET_FLAT_ADAPTIVE:
    case CKV_BUDGET_GIVEN:
      if (d->budget > (long long)d->n * d->Hkv) return CKV_EINVAL;
      o->btot = d->budget;
      break;
    default:
      return CKV_EINVAL;
  }
  if (o->btot > 0x7fffffffLL) return CKV_ENOTSUP;
  o->wo_shared = (d->flags & CKV_FLAG_WO_SHARED) ? 1 : 0;
  o->group_sum = (d->flags & CKV_FLAG_WO_GROUP_SUM) ? 1 : 0;
  o->protect_window = (d->flags & CKV_FLAG_PROTECT_WINDOW) ? 1 : 0;
  o->norm = d->norm;
  o->debug_checks = (d->flags & CKV_FLAG_DEBUG_CHECKS) ? 1 : 0;
  o->floor_b = 0;
  if (d->budget_mode == CKV_BUDGET_FLAT_ADAPTIVE) {
    long long fb = (long long)floor((double)d->adaptive_floor * (double)d->budget / (double)d->Hkv);
    const long long cap = d->budget / d->Hkv;
    o->floor_b = fb < 0 ? 0 : (fb > cap ? cap : fb);
  }
  const long long dq[3] = {(long long)d->Hq * d->w * d->dh, (long long)d->w * d->dh, d->dh};
  const long long dk[3] = {(long long)d->Hkv * d->n * d->dh, (long long)d->n * d->dh, d->dh};
  const int vec = d->dtype == CKV_F32 ? 4 : 8;  // elements per 16 bytes
  for (int i = 0; i < 3; ++i) {
    o->qs[i] = d->q_stride[i] ? d->q_stride[i] : dq[i];
    o->ks[i] = d->k_stride[i] ? d->k_stride[i] : dk[i];
    o->vs[i] = d->v_stride[i] ? d->v_stride[i] : dk[i];
    if (o->qs[i] < 0 || o->ks[i] < 0 || o->vs[i] < 0) return CKV_EINVAL;
    if (o->qs[i] % vec || o->ks[i] % vec || o->vs[i] % vec) return CKV_EALIGN;
  }
  if (o->qs[2] < d->dh || o->ks[2] < d->dh || o->vs[2] < d->dh) return CKV_EINVAL;
  if (reinterpret_cast<uintptr_t>(d->valid_from) & 3u) return CKV_EALIGN;
  o->valid_from = d->valid_from;
  return CKV_OK;
}

struct ScoreLayout {
  size_t part_m, part_l, rowstat, abar, wsum, gram, total;
};
ScoreLayout score_layout(const Dims& d) {
  ScoreLayout L;
  const size_t rows = (size_t)d.nb * d.Hq * d.w;
  // one partial per 256 keys on the CUDA-core path; the tensor-core path writes two per work item of at least
  // four 128-key tiles, the last item of a head possibly shorter: never more than ceil(n / 256) + 2
  const size_t nchunks = (d.n + ckv::kAttnChunk - 1) / ckv::kAttnChunk + 2;
  size_t off = 0;
  L.part_m = off; off = align_up(off + rows * nchunks * sizeof(float), 256);
  L.part_l = off; off = align_up(off + rows * nchunks * sizeof(float), 256);
  L.rowstat = off; off = align_up(off + rows * 2 * sizeof(float), 256);
  L.abar = off; off = align_up(off + (size_t)d.nb * d.Hq * d.n * sizeof(float), 256);
  L.wsum = off;
  if (d.group_sum)
    off = align_up(off + (size_t)(d.wo_shared ? 1 : d.nb) * d.Hkv * d.dh * d.dm * (d.dtype == CKV_F32 ? 4 : 2), 256);
  L.gram = off;
  if (d.norm == CKV_NORM_L2) off = align_up(off + ckv::vnorm_l2_workspace_bytes(d), 1024);
  L.total = off;
  return L;
}
struct SelectLayout {
  size_t a, c, budgets, sync, sync_bytes, total;
};
// with_sync: room for the per-slice block the single-kernel selection needs for adaptive budgets
SelectLayout select_layout(const Dims& d, bool with_sync = true) {
  SelectLayout L;
  const size_t per = (size_t)d.nb * d.Hkv * ckv::select_head_stride(d.n) * sizeof(float);
  size_t off = 0;
  L.a = off; off = align_up(off + per, 256);
  L.c = off; off = align_up(off + per, 256);
  L.budgets = off; off = align_up(off + (size_t)d.nb * d.Hkv * sizeof(int32_t), 256);
  L.sync = off;
  L.sync_bytes = with_sync ? ckv::select_sync_bytes(d) : 0;
  off = align_up(off + L.sync_bytes, 256);
  L.total = off;
  return L;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (prev == dev) prev = -1;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" {

int criticalkv_create(criticalkv_handle* out, int device) {
  if (!out) return CKV_EINVAL;
  *out = nullptr;
  int count = 0;
  cudaError_t e = cudaGetDeviceCount(&count);
  if (e != cudaSuccess) return CKV_ECUDA;
  if (device < 0 || device >= count) return CKV_EINVAL;
  criticalkv_handle h = new (std::nothrow) criticalkv_handle_s();
  if (!h) return CKV_EINVAL;
  memset(h, 0, sizeof(*h));
  h->device = device;
  DeviceGuard guard(device);
  cudaDeviceProp prop;
  if (!guard.ok || (e = cudaGetDeviceProperties(&prop, device)) != cudaSuccess ||
      (e = cudaMalloc(&h->status_word, sizeof(int))) != cudaSuccess ||
      (e = cudaMemset(h->status_word, 0, sizeof(int))) != cudaSuccess) {
    delete h;
    return CKV_ECUDA;
  }
  h->sm_count = prop.multiProcessorCount;
  h->cc_major = prop.major;
  h->cc_minor = prop.minor;
  h->smem_optin = (int)prop.sharedMemPerBlockOptin;
  *out = h;
  return CKV_OK;
}

int criticalkv_destroy(criticalkv_handle h) {
  if (!h) return CKV_EINVAL;
  DeviceGuard guard(h->device);
  if (h->host_ready) {
    for (int i = 0; i < 2; ++i) cudaStreamDestroy(h->host_stream[i]);
    for (int i = 0; i < 3; ++i) cudaEventDestroy(h->host_event[i]);
  }
  if (h->status_word) cudaFree(h->status_word);
  delete h;
  return CKV_OK;
}

int criticalkv_workspace_bytes(const criticalkv_desc* d, size_t* score_bytes, size_t* select_bytes) {
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (score_bytes) *score_bytes = score_layout(dd).total;
  if (select_bytes) *select_bytes = select_layout(dd).total;
  return CKV_OK;
}

int criticalkv_score(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K, const void* V,
                     const void* WO, float* attn, float* vnorm, void* ws, size_t ws_bytes, void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (!attn && !vnorm) return CKV_EINVAL;
  if (attn && (!Qw || !K)) return CKV_EINVAL;
  if (vnorm && (!V || !WO)) return CKV_EINVAL;
  if (!ws) return CKV_EINVAL;
  if (!aligned16(Qw) || !aligned16(K) || !aligned16(V) || !aligned16(WO) || !aligned16(attn) || !aligned16(vnorm) ||
      (reinterpret_cast<uintptr_t>(ws) & 255u))
    return CKV_EALIGN;
  const ScoreLayout L = score_layout(dd);
  if (ws_bytes < L.total) return CKV_EWORKSPACE;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  cudaStream_t st = (cudaStream_t)stream;
  char* base = (char*)ws;
  ckv::ScoreWorkspace sw{(float*)(base + L.part_m), (float*)(base + L.part_l), (float*)(base + L.rowstat),
                         (float*)(base + L.abar), (void*)(base + L.wsum), (void*)(base + L.gram)};
  int launches = 0, path = 0;
  cudaError_t e = cudaSuccess;
  if ((d->flags & CKV_FLAG_REQUIRE_TENSOR_CORES) && dd.dtype == CKV_BF16 &&
      ((d->flags & CKV_FLAG_FORCE_SIMT) || h->cc_major != 10 ||
       (vnorm && dd.norm == CKV_NORM_L1 && !ckv::vnorm_umma_supported(dd))))
    return CKV_ENOTSUP;   // nothing has been launched
  if (attn) {
    bool done = false;
    if (dd.dtype == CKV_BF16 && !(d->flags & CKV_FLAG_FORCE_SIMT) && h->cc_major == 10) {
      e = ckv::launch_window_attn_umma(dd, Qw, K, attn, sw, h->sm_count, h->status_word, st, &launches);
      if (e == cudaSuccess) {
        done = true;
        path |= 1;
      } else if (e == cudaErrorNotSupported) {
        e = cudaSuccess;
      }
    }
    if (!done && e == cudaSuccess) {
      if (dd.dtype == CKV_BF16 && (d->flags & CKV_FLAG_REQUIRE_TENSOR_CORES)) return CKV_ENOTSUP;
      e = ckv::launch_window_attn_simt(dd, Qw, K, attn, sw, st, &launches);
      path |= 4;
    }
  }
  if (e == cudaSuccess && vnorm && dd.group_sum) {
    // one projection per KV head through the group's summed W^O slice: same kernels, seen as Hkv heads of group size 1
    e = ckv::launch_wo_group_sum(dd, WO, sw.wsum, st, &launches);
    WO = sw.wsum;
    dd.Hq = dd.Hkv;
    dd.G = 1;
  }
  if (e == cudaSuccess && vnorm && dd.norm == CKV_NORM_L2) {
    int tc = 0;
    e = ckv::launch_vnorm_l2(dd, V, WO, vnorm, sw.gram, h->sm_count, h->cc_major,
                             (d->flags & CKV_FLAG_FORCE_SIMT) != 0, h->status_word, st, &launches, &tc);
    path |= tc ? 2 : 8;
  } else if (e == cudaSuccess && vnorm) {
    bool done = false;
    if (dd.dtype == CKV_BF16 && !(d->flags & CKV_FLAG_FORCE_SIMT) && h->cc_major == 10) {
      e = ckv::launch_vnorm_umma(dd, V, WO, vnorm, h->sm_count, h->status_word, st, &launches);
      if (e == cudaSuccess) {
        done = true;
        path |= 2;
      } else if (e == cudaErrorNotSupported) {
        e = cudaSuccess;
      }
    }
    if (!done && e == cudaSuccess) {
      if (dd.dtype == CKV_BF16 && (d->flags & CKV_FLAG_REQUIRE_TENSOR_CORES)) {
        h->launches += launches;
        h->last_path = path;
        return CKV_ENOTSUP;
      }
      e = ckv::launch_vnorm_simt(dd, V, WO, vnorm, st, &launches);
      path |= 8;
    }
  }
  h->launches += launches;
  h->last_path = path;
  return record_cuda(h, e);
}

int criticalkv_select(criticalkv_handle h, const criticalkv_desc* d, const float* attn, const float* vnorm,
                      const int32_t* budgets_in, int32_t* idx, int32_t* offsets, uint8_t* stage, void* ws,
                      size_t ws_bytes, void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (!attn || !vnorm || !idx || !offsets || !ws) return CKV_EINVAL;
  if (dd.budget_mode == CKV_BUDGET_GIVEN && !budgets_in) return CKV_EINVAL;
  if (!aligned16(attn) || !aligned16(vnorm) || (reinterpret_cast<uintptr_t>(idx) & 3u) ||
      (reinterpret_cast<uintptr_t>(offsets) & 3u) || (reinterpret_cast<uintptr_t>(budgets_in) & 3u) ||
      (reinterpret_cast<uintptr_t>(ws) & 255u))
    return CKV_EALIGN;
  const SelectLayout L = select_layout(dd);
  if (ws_bytes < L.total) return CKV_EWORKSPACE;
  // heads too long for the single kernel go through the multi-kernel path, whose bit masks live in shared memory
  if (ckv::two_stage_smem_bytes(dd.n) > (size_t)h->smem_optin) return CKV_ENOTSUP;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  char* base = (char*)ws;
  ckv::SelectWorkspace sw{(float*)(base + L.a), (float*)(base + L.c), (int32_t*)(base + L.budgets),
                          L.sync_bytes ? (void*)(base + L.sync) : nullptr};
  int launches = 0;
  const ckv::SelectDevice sd{h->sm_count, h->smem_optin, (d->flags & CKV_FLAG_SELECT_MULTIPASS) ? 0 : 1,
                             (d->flags & CKV_FLAG_SELECT_SINGLE_KERNEL) ? 1 : 0,
                             (d->flags & CKV_FLAG_SELECT_NO_CLUSTER) ? 0 : 1};
  cudaError_t e = ckv::launch_select(dd, attn, vnorm, budgets_in, idx, offsets, stage, sw, sd, (cudaStream_t)stream,
                                     &launches, h->status_word, &h->last_select_fused);
  h->launches += launches;
  return record_cuda(h, e);
}

int criticalkv_compact(criticalkv_handle h, const criticalkv_desc* d, const void* K, const void* V,
                       const int32_t* idx, const int32_t* offsets, void* K_out, void* V_out, void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (!K || !V || !idx || !offsets || !K_out || !V_out) return CKV_EINVAL;
  if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out) ||
      (reinterpret_cast<uintptr_t>(idx) & 3u) || (reinterpret_cast<uintptr_t>(offsets) & 3u))
    return CKV_EALIGN;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  if (dd.btot == 0) return CKV_OK;
  int launches = 0;
  cudaError_t e = ckv::launch_compact(dd, K, V, idx, offsets, K_out, V_out, h->sm_count, h->status_word,
                                      (cudaStream_t)stream, &launches);
  h->launches += launches;
  return record_cuda(h, e);
}

int criticalkv_group_scores(criticalkv_handle h, const criticalkv_desc* d, const float* attn, const float* vnorm,
                            float* a_out, float* c_out, void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (!attn || !vnorm || !a_out) return CKV_EINVAL;
  if (!aligned16(attn) || !aligned16(vnorm) || !aligned16(a_out) || !aligned16(c_out)) return CKV_EALIGN;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  int launches = 0;
  cudaError_t e = ckv::launch_group_scores(dd, attn, vnorm, a_out, c_out, (cudaStream_t)stream, &launches);
  h->launches += launches;
  return record_cuda(h, e);
}

int criticalkv_allocate_budgets(criticalkv_handle h, const criticalkv_desc* d, const float* a, int32_t* budgets_out,
                                void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (dd.budget_mode != CKV_BUDGET_FLAT_ADAPTIVE) return CKV_EINVAL;
  if (!a || !budgets_out) return CKV_EINVAL;
  if (!aligned16(a) || (reinterpret_cast<uintptr_t>(budgets_out) & 3u)) return CKV_EALIGN;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  int launches = 0;
  cudaError_t e = ckv::launch_allocate_budgets(dd, a, budgets_out, h->smem_optin, (cudaStream_t)stream, &launches);
  h->launches += launches;
  return record_cuda(h, e);
}

int criticalkv_gather_positions(criticalkv_handle h, const criticalkv_desc* d, const int32_t* pos_in,
                                const int32_t* idx, const int32_t* offsets, int32_t* pos_out, void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (!pos_in || !idx || !offsets || !pos_out) return CKV_EINVAL;
  if ((reinterpret_cast<uintptr_t>(pos_in) | reinterpret_cast<uintptr_t>(idx) | reinterpret_cast<uintptr_t>(offsets) |
       reinterpret_cast<uintptr_t>(pos_out)) & 3u)
    return CKV_EALIGN;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  if (dd.btot == 0) return CKV_OK;
  int launches = 0;
  cudaError_t e = ckv::launch_gather_positions(dd, pos_in, idx, offsets, pos_out, h->sm_count, h->status_word,
                                               (cudaStream_t)stream, &launches);
  h->launches += launches;
  return record_cuda(h, e);
}

int criticalkv_compress(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K, const void* V,
                        const void* WO, const int32_t* budgets_in, float* attn, float* vnorm, int32_t* idx,
                        int32_t* offsets, uint8_t* stage, void* K_out, void* V_out, void* ws, size_t ws_bytes,
                        void* stream) {
  if (!attn || !vnorm) return CKV_EINVAL;
  int rc = criticalkv_score(h, d, Qw, K, V, WO, attn, vnorm, ws, ws_bytes, stream);
  if (rc != CKV_OK) return rc;
  rc = criticalkv_select(h, d, attn, vnorm, budgets_in, idx, offsets, stage, ws, ws_bytes, stream);
  if (rc != CKV_OK) return rc;
  return criticalkv_compact(h, d, K, V, idx, offsets, K_out, V_out, stream);
}

// ---- host-staged compression ------------------------------------------------------------------------------------
}  // extern "C"
namespace {
struct HostStaging {   // byte offsets inside one of the two device staging buffers
  size_t Qw, K, V, WO, attn, vnorm, budgets, idx, offsets, K_out, V_out, ws, ws_bytes, total;
  size_t nQw, nK, nV, nWO, nidx, noffsets, nout;   // bytes per nb slice
};
HostStaging host_staging_layout(const Dims& one) {
  HostStaging L;
  const size_t es = one.dtype == CKV_F32 ? 4 : 2;
  L.nQw = (size_t)one.Hq * one.w * one.dh * es;
  L.nK = L.nV = (size_t)one.Hkv * one.n * one.dh * es;
  L.nWO = (size_t)one.Hq * one.dh * one.dm * es;
  L.nidx = (size_t)one.btot * sizeof(int32_t);
  L.noffsets = (size_t)(one.Hkv + 1) * sizeof(int32_t);
  L.nout = (size_t)one.btot * one.dh * es;
  const size_t nscore = (size_t)one.Hq * one.n * sizeof(float);
  const size_t sb = score_layout(one).total, tb = select_layout(one).total;
  L.ws_bytes = sb > tb ? sb : tb;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + (bytes ? bytes : 16), 256); return o; };
  L.Qw = take(L.nQw); L.K = take(L.nK); L.V = take(L.nV); L.WO = take(L.nWO);
  L.attn = take(nscore); L.vnorm = take(nscore);
  L.budgets = take((size_t)one.Hkv * sizeof(int32_t));
  L.idx = take(L.nidx); L.offsets = take(L.noffsets); L.K_out = take(L.nout); L.V_out = take(L.nout);
  L.ws = take(L.ws_bytes);
  L.total = off;
  return L;
}
// Descriptor of a single dense nb slice of the caller's problem.
criticalkv_desc single_slice_desc(const criticalkv_desc& d) {
  criticalkv_desc o = d;
  o.nb = 1;
  for (int i = 0; i < 3; ++i) o.q_stride[i] = o.k_stride[i] = o.v_stride[i] = 0;
  o.flags &= ~(uint32_t)CKV_FLAG_WO_SHARED;
  return o;
}
}  // namespace
extern "C" {

int criticalkv_host_staging_bytes(const criticalkv_desc* d, size_t* bytes) {
  if (!d || !bytes) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  criticalkv_desc one = single_slice_desc(*d);
  Dims d1;
  if ((rc = resolve(&one, &d1)) != CKV_OK) return rc;
  *bytes = 2 * host_staging_layout(d1).total;
  return CKV_OK;
}

int criticalkv_compress_host(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K,
                             const void* V, const void* WO, const int32_t* budgets_in, int32_t* idx,
                             int32_t* offsets, void* K_out, void* V_out, void* staging, size_t staging_bytes,
                             void* stream) {
  if (!h || !d) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (!Qw || !K || !V || !WO || !idx || !offsets || !K_out || !V_out || !staging) return CKV_EINVAL;
  if (dd.budget_mode == CKV_BUDGET_GIVEN && !budgets_in) return CKV_EINVAL;
  if (d->valid_from) return CKV_ENOTSUP;   // the per-head offsets would have to be host memory here
  for (int i = 0; i < 3; ++i)
    if (d->q_stride[i] || d->k_stride[i] || d->v_stride[i]) return CKV_ENOTSUP;  // host arrays must be dense
  if (reinterpret_cast<uintptr_t>(staging) & 255u) return CKV_EALIGN;
  criticalkv_desc one = single_slice_desc(*d);
  Dims d1;
  if ((rc = resolve(&one, &d1)) != CKV_OK) return rc;
  const HostStaging L = host_staging_layout(d1);
  if (staging_bytes < 2 * L.total) return CKV_EWORKSPACE;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  cudaError_t e = cudaSuccess;
  if (!h->host_ready) {
    for (int i = 0; i < 2 && e == cudaSuccess; ++i)
      e = cudaStreamCreateWithFlags(&h->host_stream[i], cudaStreamNonBlocking);
    for (int i = 0; i < 3 && e == cudaSuccess; ++i)
      e = cudaEventCreateWithFlags(&h->host_event[i], cudaEventDisableTiming);
    if (e != cudaSuccess) return record_cuda(h, e);
    h->host_ready = true;
  }
  cudaStream_t user = (cudaStream_t)stream;
  // the staging streams start after whatever the caller has queued on its stream
  if ((e = cudaEventRecord(h->host_event[2], user)) != cudaSuccess) return record_cuda(h, e);
  for (int i = 0; i < 2; ++i)
    if ((e = cudaStreamWaitEvent(h->host_stream[i], h->host_event[2], 0)) != cudaSuccess) return record_cuda(h, e);

  const bool wo_shared = dd.wo_shared != 0;
  const char* hq = (const char*)Qw; const char* hk = (const char*)K; const char* hv = (const char*)V;
  const char* hw = (const char*)WO;
  for (int b = 0; b < dd.nb && rc == CKV_OK; ++b) {
    const int p = b & 1;
    cudaStream_t st = h->host_stream[p];
    char* base = (char*)staging + (size_t)p * L.total;
    // a shared W^O is uploaded once per staging buffer (slices 0 and 1)
    const bool copy_wo = !wo_shared || b < 2;
    if ((e = cudaMemcpyAsync(base + L.Qw, hq + (size_t)b * L.nQw, L.nQw, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(base + L.K, hk + (size_t)b * L.nK, L.nK, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(base + L.V, hv + (size_t)b * L.nV, L.nV, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (copy_wo && (e = cudaMemcpyAsync(base + L.WO, hw + (wo_shared ? 0 : (size_t)b * L.nWO), L.nWO,
                                         cudaMemcpyHostToDevice, st)) != cudaSuccess))
      break;   // the common tail below joins the staging streams before the error is returned
    const int32_t* bud = nullptr;
    if (dd.budget_mode == CKV_BUDGET_GIVEN) {
      if ((e = cudaMemcpyAsync(base + L.budgets, budgets_in + (size_t)b * dd.Hkv, (size_t)dd.Hkv * sizeof(int32_t),
                               cudaMemcpyHostToDevice, st)) != cudaSuccess)
        break;
      bud = (const int32_t*)(base + L.budgets);
    }
    rc = criticalkv_score(h, &one, base + L.Qw, base + L.K, base + L.V, base + L.WO, (float*)(base + L.attn),
                          (float*)(base + L.vnorm), base + L.ws, L.ws_bytes, st);
    if (rc != CKV_OK) break;
    rc = criticalkv_select(h, &one, (const float*)(base + L.attn), (const float*)(base + L.vnorm), bud,
                           (int32_t*)(base + L.idx), (int32_t*)(base + L.offsets), nullptr, base + L.ws,
                           L.ws_bytes, st);
    if (rc != CKV_OK) break;
    rc = criticalkv_compact(h, &one, base + L.K, base + L.V, (const int32_t*)(base + L.idx),
                            (const int32_t*)(base + L.offsets), base + L.K_out, base + L.V_out, st);
    if (rc != CKV_OK) break;
    if ((L.nidx && (e = cudaMemcpyAsync((char*)idx + (size_t)b * L.nidx, base + L.idx, L.nidx,
                                        cudaMemcpyDeviceToHost, st)) != cudaSuccess) ||
        (e = cudaMemcpyAsync((char*)offsets + (size_t)b * L.noffsets, base + L.offsets, L.noffsets,
                             cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
        (L.nout && ((e = cudaMemcpyAsync((char*)K_out + (size_t)b * L.nout, base + L.K_out, L.nout,
                                         cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
                    (e = cudaMemcpyAsync((char*)V_out + (size_t)b * L.nout, base + L.V_out, L.nout,
                                         cudaMemcpyDeviceToHost, st)) != cudaSuccess)))
      break;
  }
  // join (also after an error: slices already queued keep writing into the caller's host arrays until they finish):
  // the caller's stream continues after both staging streams, and the call returns with the results on the host
  for (int i = 0; i < 2; ++i) {
    cudaError_t e2 = cudaEventRecord(h->host_event[i], h->host_stream[i]);
    if (e2 == cudaSuccess) e2 = cudaStreamWaitEvent(user, h->host_event[i], 0);
    if (e == cudaSuccess) e = e2;
  }
  cudaError_t e3 = cudaStreamSynchronize(user);
  if (e == cudaSuccess) e = e3;
  if (rc != CKV_OK) return rc;
  return record_cuda(h, e);
}

int criticalkv_diagnose_workspace_bytes(const criticalkv_desc* d, size_t* bytes) {
  if (!bytes) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  *bytes = score_layout(dd).total + align_up((size_t)dd.nb * dd.Hkv * dd.n, 256);
  return CKV_OK;
}

int criticalkv_diagnose(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K, const void* V,
                        const void* WO, const float* vnorm, const int32_t* idx, const int32_t* offsets,
                        const uint8_t* stage, float* diag, void* ws, size_t ws_bytes, void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (dd.group_sum) return CKV_ENOTSUP;  // the bounds are stated with per-head norms
  if (dd.valid_from) return CKV_ENOTSUP;
  if (dd.w > 64) return CKV_ENOTSUP;     // the diagnostics kernel keeps a window's rows in registers
  if (!Qw || !K || !V || !WO || !vnorm || !idx || !offsets || !stage || !diag || !ws) return CKV_EINVAL;
  if (!aligned16(Qw) || !aligned16(K) || !aligned16(V) || !aligned16(WO) || !aligned16(vnorm) || !aligned16(diag) ||
      (reinterpret_cast<uintptr_t>(idx) & 3u) || (reinterpret_cast<uintptr_t>(offsets) & 3u) ||
      (reinterpret_cast<uintptr_t>(ws) & 255u))
    return CKV_EALIGN;
  const ScoreLayout L = score_layout(dd);
  if (ws_bytes < L.total + align_up((size_t)dd.nb * dd.Hkv * dd.n, 256)) return CKV_EWORKSPACE;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  char* base = (char*)ws;
  ckv::ScoreWorkspace sw{(float*)(base + L.part_m), (float*)(base + L.part_l), (float*)(base + L.rowstat),
                         (float*)(base + L.abar), (void*)(base + L.wsum), (void*)(base + L.gram)};
  int launches = 0;
  cudaError_t e = ckv::launch_diagnostics(dd, Qw, K, V, WO, vnorm, idx, offsets, stage, diag, sw,
                                          (uint8_t*)(base + L.total), (cudaStream_t)stream, &launches);
  h->launches += launches;
  return record_cuda(h, e);
}

int criticalkv_selftest_bounded_wait(criticalkv_handle h, uint64_t limit_ns, int* observed_device, void* stream) {
  if (!h || !observed_device) return CKV_EINVAL;
  if (limit_ns > CKV_SELFTEST_MAX_WAIT_NS) return CKV_EINVAL;   // no wait of the library may hold an SM for long
  if (h->cc_major < 9) return CKV_ENOTSUP;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  cudaError_t e = ckv::launch_bounded_wait_selftest(h->status_word, limit_ns, observed_device, (cudaStream_t)stream);
  h->launches += 1;
  return record_cuda(h, e);
}

int criticalkv_device_status(criticalkv_handle h, void* stream, int* out) {
  if (!h || !out) return CKV_EINVAL;
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  cudaStream_t st = (cudaStream_t)stream;
  int v = 0;
  cudaError_t e = cudaMemcpyAsync(&v, h->status_word, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->status_word, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  *out = v;
  return record_cuda(h, e);
}

// ---- allocation-free select ------------------------------------------------------------------------------------
// Scratch for criticalkv_select_static.  The symbol below is only a stand-in on the host: kernels must be given the
// device address that cudaGetSymbolAddress returns for the current device, never the name itself.
}  // extern "C"
static __device__ __align__(256) unsigned char g_select_static_scratch[CKV_STATIC_SCRATCH_BYTES];
namespace {
constexpr int kMaxStaticDevices = 64;
std::mutex g_static_mutex;
void* g_static_scratch_addr[kMaxStaticDevices];  // per device ordinal, resolved on first use

// Device address of the scratch array on `device` (which must be current).  Looked up once per device.
cudaError_t static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxStaticDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_scratch_addr[device]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_select_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_scratch_addr[device] = p;
  }
  *out = g_static_scratch_addr[device];
  return cudaSuccess;
}
}  // namespace
extern "C" {

int criticalkv_select_static(criticalkv_handle h, const criticalkv_desc* d, const float* attn, const float* vnorm,
                             const int32_t* budgets_in, int32_t* idx, int32_t* offsets, uint8_t* stage,
                             void* stream) {
  if (!h) return CKV_EINVAL;
  Dims dd;
  int rc = resolve(d, &dd);
  if (rc != CKV_OK) return rc;
  if (!attn || !vnorm || !idx || !offsets) return CKV_EINVAL;
  if (dd.budget_mode == CKV_BUDGET_GIVEN && !budgets_in) return CKV_EINVAL;
  if (!aligned16(attn) || !aligned16(vnorm) || (reinterpret_cast<uintptr_t>(idx) & 3u) ||
      (reinterpret_cast<uintptr_t>(offsets) & 3u) || (reinterpret_cast<uintptr_t>(budgets_in) & 3u))
    return CKV_EALIGN;
  if (ckv::two_stage_smem_bytes(dd.n) > (size_t)h->smem_optin) return CKV_ENOTSUP;
  const SelectLayout L = select_layout(dd, false);
  if (L.total > CKV_STATIC_SCRATCH_BYTES) {
    snprintf(h->cuda_error, sizeof(h->cuda_error),
             "criticalkv_select_static: this shape needs %zu bytes of scratch, the built-in array holds %zu",
             L.total, (size_t)CKV_STATIC_SCRATCH_BYTES);
    return CKV_EWORKSPACE;
  }
  DeviceGuard guard(h->device);
  if (!guard.ok) return CKV_ECUDA;
  void* scratch = nullptr;
  cudaError_t e = static_scratch_address(h->device, &scratch);
  if (e != cudaSuccess) return record_cuda(h, e);
  char* base = (char*)scratch;
  ckv::SelectWorkspace sw{(float*)(base + L.a), (float*)(base + L.c), (int32_t*)(base + L.budgets),
                          L.sync_bytes ? (void*)(base + L.sync) : nullptr};
  int launches = 0;
  const ckv::SelectDevice sd{h->sm_count, h->smem_optin, (d->flags & CKV_FLAG_SELECT_MULTIPASS) ? 0 : 1,
                             (d->flags & CKV_FLAG_SELECT_SINGLE_KERNEL) ? 1 : 0,
                             (d->flags & CKV_FLAG_SELECT_NO_CLUSTER) ? 0 : 1};
  e = ckv::launch_select(dd, attn, vnorm, budgets_in, idx, offsets, stage, sw, sd, (cudaStream_t)stream, &launches,
                         h->status_word, &h->last_select_fused);
  h->launches += launches;
  return record_cuda(h, e);
}

const char* criticalkv_status_string(int s) {
  switch (s) {
    case CKV_OK: return "ok";
    case CKV_EINVAL: return "invalid argument";
    case CKV_ENOTSUP: return "not supported";
    case CKV_EALIGN: return "pointer or stride not 16-byte aligned";
    case CKV_EWORKSPACE: return "workspace too small";
    case CKV_ECUDA: return "CUDA call failed";
    case CKV_ETIMEOUT: return "device-side wait timed out";
    case CKV_EBOUNDS: return "debug check: index, offset or count outside its buffer";
    default: return "unknown status";
  }
}

const char* criticalkv_last_cuda_error(criticalkv_handle h) { return h ? h->cuda_error : ""; }
int criticalkv_last_path(criticalkv_handle h) { return h ? (h->last_path | (h->last_select_fused == 1 ? 32 : 0) | (h->last_select_fused == 2 ? 64 : 0)) : 0;
}
int64_t criticalkv_launch_count(criticalkv_handle h) { return h ? h->launches : 0; }

}  // extern "C"
