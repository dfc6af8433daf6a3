// Internal declarations shared by the translation units of libcriticalkv (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "criticalkv.h"

namespace ckv {

// Resolved problem description handed to the launchers (host side).
struct Dims {
  int nb, Hq, Hkv, G, dh, dm, n, w, kp;
  int dtype;
  float scale, alpha, eps;
  int budget_mode;
  long long budget;   // as in criticalkv_desc
  long long btot;     // capacity of idx per nb slice
  int wo_shared;
  int group_sum;      // CKV_FLAG_WO_GROUP_SUM
  int protect_window; // CKV_FLAG_PROTECT_WINDOW
  int norm;           // criticalkv_norm
  int debug_checks;   // CKV_FLAG_DEBUG_CHECKS
  long long floor_b;  // guaranteed entries per KV head (adaptive budgets)
  long long qs[3], ks[3], vs[3];  // element strides: nb, head, row
  const int32_t* valid_from;      // device [nb, Hkv] or null: first real row of every KV head (rows before it are padding)
};

// Keys of the window-attention kernels are processed in chunks of this many tokens (one CTA each).
constexpr int kAttnChunk = 256;

struct ScoreWorkspace {   // carved out of the caller's workspace by the API layer
  float* part_m;    // [nb*Hq*w, nchunks]   partial row maxima
  float* part_l;    // [nb*Hq*w, nchunks]   partial row sums of exp
  float* rowstat;   // [nb*Hq*w, 2]         final (max, 1/(w*sum))
  float* abar;      // [nb*Hq, n]           window-mean attention before pooling
  void* wsum;       // [nbw, Hkv, dh, dm]   group-summed W^O (CKV_FLAG_WO_GROUP_SUM only)
  void* gram;       // [nbw, Hq, dh, dh]    W^O_h W^O_h^T (CKV_NORM_L2 only): float32, or bf16 hi and lo parts
};

struct SelectWorkspace {
  float* a;         // [nb, Hkv, n]  (single-kernel path: integer keys, [nb*Hkv][32][words], see select_fused.cu)
  float* c;         // [nb, Hkv, n]  (same)
  int32_t* budgets; // [nb, Hkv]
  void* sync;       // select_sync_bytes(): per-slice histograms and barrier counters of the single-kernel path, or null
};
// Floats per head in each of the regions a and c: n rounded up to a whole, even number of 32-entry words.
inline size_t select_head_stride(int n) { return (size_t)32 * ((((size_t)n + 31) / 32 + 1) & ~(size_t)1); }
size_t select_sync_bytes(const Dims& d);

// ---- launchers (each returns the first CUDA error of its launches) ----
cudaError_t launch_window_attn_simt(const Dims& d, const void* Qw, const void* K, float* attn,
                                    const ScoreWorkspace& ws, cudaStream_t st, int* launches);
cudaError_t launch_vnorm_simt(const Dims& d, const void* V, const void* WO, float* vnorm, cudaStream_t st,
                              int* launches);
// Pieces of the window-attention path shared by the CUDA-core and tensor-core front ends.
cudaError_t launch_attn_combine(const float* part_m, const float* part_l, float* rowstat, int rows, int nchunks,
                                int w, cudaStream_t st);
cudaError_t launch_maxpool(const float* abar, float* attn, int n, int kp, int nrows, cudaStream_t st);
cudaError_t launch_window_stats_simt(const Dims& d, const void* Qw, const void* K, const ScoreWorkspace& ws,
                                     cudaStream_t st, int* launches);
cudaError_t launch_diagnostics(const Dims& d, const void* Qw, const void* K, const void* V, const void* WO,
                               const float* vnorm, const int32_t* idx, const int32_t* offsets, const uint8_t* stage,
                               float* diag, const ScoreWorkspace& ws, uint8_t* stage_of, cudaStream_t st,
                               int* launches);
// Tensor-core window attention (bf16).  cudaErrorNotSupported = shape or layout outside what it handles.
cudaError_t launch_window_attn_umma(const Dims& d, const void* Qw, const void* K, float* attn,
                                    const ScoreWorkspace& ws, int sm_count, int* status_word, cudaStream_t st,
                                    int* launches);
// Tensor-core projection norm (bf16).  cudaErrorNotSupported = this layout cannot be expressed as a tensor map;
// the caller then uses the CUDA-core kernel.
bool vnorm_umma_supported(const Dims& d);
cudaError_t launch_vnorm_umma(const Dims& d, const void* V, const void* WO, float* vnorm, int sm_count,
                              int* status_word, cudaStream_t st, int* launches);
cudaError_t launch_bounded_wait_selftest(int* status_word, unsigned long long limit_ns, int* observed,
                                         cudaStream_t st);
// W_tilde[bw, g] = round(sum_h WO[bw, g*G + h]) for the group-summed projection variant.
cudaError_t launch_wo_group_sum(const Dims& d, const void* WO, void* wsum, cudaStream_t st, int* launches);
// L2 variant of step 2 through the Gram matrix.
size_t vnorm_l2_workspace_bytes(const Dims& d);
cudaError_t launch_vnorm_l2(const Dims& d, const void* V, const void* WO, float* vnorm, void* gram, int sm_count,
                            int cc_major, bool force_simt, int* status_word, cudaStream_t st, int* launches,
                            int* used_tensor_cores);
// The two front steps of launch_select on their own (a layer whose KV heads live on several GPUs runs them around an
// all-gather): group scores a (and c unless null), and the flattened adaptive allocation over a[nb, Hkv, n].
cudaError_t launch_group_scores(const Dims& d, const float* attn, const float* vnorm, float* a, float* c,
                                cudaStream_t st, int* launches);
cudaError_t launch_allocate_budgets(const Dims& d, const float* a_all, int32_t* budgets_out, int smem_optin,
                                    cudaStream_t st, int* launches);
// What the selection launcher needs to know about the device and the caller's wishes.
struct SelectDevice {
  int sm_count;
  int smem_optin;    // largest dynamic shared memory a CTA may ask for
  int allow_fused;   // 0: always the multi-kernel path (CKV_FLAG_SELECT_MULTIPASS)
  int prefer_fused;  // 1: the single kernel also for few heads (CKV_FLAG_SELECT_SINGLE_KERNEL)
  int allow_cluster; // 0: one CTA per head in the multi-kernel path (CKV_FLAG_SELECT_NO_CLUSTER)
};
// *fused = 1 when the single-kernel path ran, 2 when the two-stage top-k ran with a cluster per head, else 0.
cudaError_t launch_select(const Dims& d, const float* attn, const float* vnorm, const int32_t* budgets_in,
                          int32_t* idx, int32_t* offsets, uint8_t* stage, const SelectWorkspace& ws,
                          const SelectDevice& dev, cudaStream_t st, int* launches, int* status_word, int* fused);
// Steps 3-4 as one kernel.  cudaErrorNotSupported = the shape is outside what it handles or the cooperative launch is
// not available; no kernel has been launched then.
cudaError_t launch_select_fused(const Dims& d, const float* attn, const float* vnorm, const int32_t* budgets_in,
                                int32_t* idx, int32_t* offsets, uint8_t* stage, const SelectWorkspace& ws,
                                const SelectDevice& dev, cudaStream_t st, int* launches, int* status_word);
cudaError_t launch_compact(const Dims& d, const void* K, const void* V, const int32_t* idx, const int32_t* offsets,
                           void* K_out, void* V_out, int sm_count, int* status_word, cudaStream_t st, int* launches);

cudaError_t launch_gather_positions(const Dims& d, const int32_t* pos_in, const int32_t* idx, const int32_t* offsets,
                                    int32_t* pos_out, int sm_count, int* status_word, cudaStream_t st, int* launches);
// Dynamic shared memory the multi-kernel two-stage selection needs for a head of n entries.
size_t two_stage_smem_bytes(int n);
// The two-stage top-k with a thread-block cluster per (nb slice, KV head), for calls with few heads (a, c: the group
// scores of launch_group_scores, or null: computed in the kernel from attn and vnorm).  cudaErrorNotSupported = not launched (shape or device): use the one-CTA kernel.
bool two_stage_cluster_applies(const Dims& d, const SelectDevice& dev);
cudaError_t launch_two_stage_cluster(const Dims& d, const float* attn, const float* vnorm, const float* a,
                                     const float* c, const int32_t* budgets, int32_t* idx, int32_t* offsets,
                                     uint8_t* stage, const SelectDevice& dev, cudaStream_t st, int* launches,
                                     int* status_word);

}  // namespace ckv
