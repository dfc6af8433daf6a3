/*
 * criticalkv.h -- C ABI of the CriticalKV prefill-time KV-cache compression step for NVIDIA B200 (sm_100a).
 *
 * The library implements one layer-level operation of "Optimizing KV Cache Eviction from an Output Perturbation
 * Perspective": score every cached KV entry of every head, keep a budgeted subset with the paper's two-stage
 * perturbation-constrained rule, and compact K/V.  The three entry points follow the paper's problem statement
 * (Algorithm 1 inputs: budget b, query state, K, V, W^O, alpha; Algorithm 2 inputs: Q, K, V, window size):
 *
 *   criticalkv_score    steps 1-2   window attention (Algorithm 2) and the projected value-row norm (Algorithm 1)
 *   criticalkv_select   steps 3-4   scores per KV head, budgets, two-stage top-k (Algorithm 1)
 *   criticalkv_compact  step  5     gather of the retained rows (Algorithm 1, the step that appends the selected entries to the retained cache)
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer unless the argument is documented as host memory.  The caller owns all
 *     buffers, including the workspace; the library allocates device memory only in criticalkv_create (one status
 *     word).
 *   - Calls only enqueue work on the given CUDA stream (a cudaStream_t passed as void*, NULL = legacy default stream)
 *     and return; they never synchronise, except criticalkv_device_status and criticalkv_compress_host.
 *   - Return value: a criticalkv_status.  Argument errors are found on the host before any launch.  A device-side
 *     anomaly (a bounded wait that ran out) sets the handle's device status word; kernels still terminate.
 *   - Identical inputs give bit-identical outputs (no order-dependent floating-point atomics).
 *   - Data pointers must be 16-byte aligned; strides (in elements) must keep every row 16-byte aligned.
 *   - One handle per host thread / stream.
 *
 * Layouts (innermost index contiguous; nb = batch x layers handled by one call)
 *   Qw  [nb, Hq,  w, dh]   the last w query rows of each query head (the observation window)
 *   K,V [nb, Hkv, n, dh]   the KV cache; query head h reads KV head h / (Hq/Hkv)
 *   WO  [nbw, Hq, dh, dm]  head h's rows h*dh .. (h+1)*dh-1 of the (Hq*dh) x dm output projection (Eq. 2: o = A V W^O);
 *                          nbw = nb, or 1 when CKV_FLAG_WO_SHARED is set
 *   attn, vnorm [nb, Hq, n] float32
 *   idx [nb, Btot] int32, offsets [nb, Hkv+1] int32, stage [nb, Btot] uint8 (1 = stage 1, 2 = stage 2)
 *   K_out, V_out [nb, Btot, dh], same element type as K, V
 *   Btot = Hkv * budget (uniform), budget (flattened adaptive), or the capacity given by the caller (given budgets).
 */
#ifndef CRITICALKV_H_
#define CRITICALKV_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define CKV_API __attribute__((visibility("default")))
#else
#define CKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct criticalkv_handle_s* criticalkv_handle;

typedef enum {
  CKV_OK = 0,
  CKV_EINVAL = -1,      /* bad argument (null pointer, shape, budget out of range)            */
  CKV_ENOTSUP = -2,     /* valid request this build does not implement                        */
  CKV_EALIGN = -3,      /* pointer or stride not 16-byte aligned                              */
  CKV_EWORKSPACE = -4,  /* workspace smaller than criticalkv_workspace_bytes reports          */
  CKV_ECUDA = -5,       /* a CUDA runtime/driver call failed (see criticalkv_last_cuda_error) */
  CKV_ETIMEOUT = -6,    /* a bounded device-side wait ran out (read via criticalkv_device_status) */
  CKV_EBOUNDS = -7      /* CKV_FLAG_DEBUG_CHECKS: a kernel met an index, offset or count outside its buffer; the
                           access was skipped (read via criticalkv_device_status)                */
} criticalkv_status;

typedef enum { CKV_F32 = 0, CKV_BF16 = 1 } criticalkv_dtype;
typedef enum { CKV_BUDGET_UNIFORM = 0, CKV_BUDGET_FLAT_ADAPTIVE = 1, CKV_BUDGET_GIVEN = 2 } criticalkv_budget_mode;
/* CKV_NORM_L1: the paper's method.  CKV_NORM_L2: vnorm = ||V W^O_h||_2 (appendix on the distance metric), computed
   through the Gram matrix W^O_h W^O_h^T, d_model / head_dim times fewer flops than the L1 projection. */
typedef enum { CKV_NORM_L1 = 0, CKV_NORM_L2 = 1 } criticalkv_norm;

enum {
  CKV_FLAG_WO_SHARED = 1u << 0,   /* WO has no nb dimension (one projection for the whole call)             */
  CKV_FLAG_FORCE_SIMT = 1u << 1,  /* bf16 only: use the CUDA-core kernels instead of the tensor-core ones   */
  CKV_FLAG_PROTECT_WINDOW = 1u << 3, /* always keep the last w entries (the observation window): their scores are
                                     raised to the largest float32 in both stages, so they fill stage 1 first and
                                     count against the budget                                                   */
  CKV_FLAG_WO_GROUP_SUM = 1u << 2, /* grouped-query shortcut of step 2: the W^O slices of a KV group are added
                                     (float32, heads ascending, rounded once to the storage type) and each value
                                     row is projected once per KV head.  vnorm then is [nb, Hkv, n] and
                                     c_g = (a_g + eps) * vnorm_g in criticalkv_select.  Hq/Hkv times fewer flops;
                                     not the per-head norm of Algorithm 1 but the norm of the group's summed
                                     projection (the heads of a group share V, so their outputs add in Eq. 2).  */
  CKV_FLAG_SELECT_MULTIPASS = 1u << 5, /* criticalkv_select: always run steps 3-4 as separate kernels (group scores,
                                     budget allocation, two-stage top-k over score arrays in the workspace) even
                                     when a head's scores fit in shared memory and the single-kernel path applies.
                                     Same results bit for bit                                                   */
  CKV_FLAG_SELECT_SINGLE_KERNEL = 1u << 4, /* criticalkv_select: take the single kernel (one CTA per KV head) also for
                                     calls with few heads (nb * Hkv at most half the number of SMs), which by
                                     default run the separate kernels with a thread-block cluster per head: a
                                     layer at a time that is about twice as fast.  Same results bit for bit      */
  CKV_FLAG_SELECT_NO_CLUSTER = 1u << 8, /* criticalkv_select: no thread-block clusters in steps 3-4 (the separate
                                     kernels then give every head one CTA), for contexts where cluster launches are
                                     not wanted.  Same results bit for bit                                      */
  CKV_FLAG_DEBUG_CHECKS = 1u << 6, /* device-side checks in criticalkv_select, criticalkv_compact and
                                     criticalkv_gather_positions: every index read from idx / offsets / budgets and
                                     every output position is tested against the bounds the descriptor implies
                                     before it is used; a violation skips that access, sets the status word to
                                     CKV_EBOUNDS and lets the kernel finish (no trap).  Without the flag the same
                                     accesses are skipped silently.  Meant for bring-up of a caller: the stand-in
                                     for a memory checker where none can be run                                  */
  CKV_FLAG_REQUIRE_TENSOR_CORES = 1u << 7 /* criticalkv_score: return CKV_ENOTSUP instead of running the CUDA-core
                                     kernels when a bf16 problem is outside what the tensor-core kernels take
                                     (window attention: w in {16, 32, 64, 128, 256} and a layout a tensor map can
                                     express; they are 20 times faster, so a silent change of path is a
                                     performance cliff; criticalkv_last_path tells which kernels ran)          */
};

/* Problem descriptor (plain data, copied by every call). */
typedef struct {
  int32_t nb;            /* >= 1                                                                        */
  int32_t Hq, Hkv;       /* Hq % Hkv == 0, Hkv <= 64                                                    */
  int32_t dh;            /* head dim: 64 or 128                                                         */
  int32_t dm;            /* model dim, multiple of 8                                                    */
  int32_t n;             /* cached entries per head, >= w                                               */
  int32_t w;             /* observation window (Algorithm 2: n'), 1..256 (criticalkv_diagnose: 1..64)   */
  int32_t pool_k;        /* max-pool kernel, odd, 1..63 (Algorithm 2: maxpooling; 7 in the paper)       */
  int32_t dtype;         /* criticalkv_dtype of Qw, K, V, WO, K_out, V_out                              */
  float scale;           /* logit scale of Eq. 2; <= 0 selects 1/sqrt(dh)                               */
  float alpha;           /* stage split of Algorithm 1 in [0,1]: b' = floor(alpha*b), b'' = b - b'      */
  float eps;             /* Algorithm 1: (A + eps) * norm; the paper uses 1e-4                          */
  int32_t budget_mode;   /* criticalkv_budget_mode                                                      */
  int32_t norm;          /* criticalkv_norm                                                             */
  int64_t budget;        /* UNIFORM: B per KV head (<= n); FLAT_ADAPTIVE: B_total per nb slice
                            (<= Hkv*n); GIVEN: capacity Btot of idx per nb slice (>= sum of budgets)    */
  uint32_t flags;        /* CKV_FLAG_*                                                                  */
  uint32_t reserved;     /* must be 0                                                                   */
  /* Element strides of Qw / K / V for the nb, head and row (token) index; 0 selects the dense default. */
  int64_t q_stride[3];
  int64_t k_stride[3];
  int64_t v_stride[3];
  float adaptive_floor;  /* FLAT_ADAPTIVE only, in [0,1]: every KV head is first guaranteed
                            floor(adaptive_floor * budget / Hkv) entries, the rest of the budget goes to the
                            flattened top-k, and a head's budget is capped at n.  0 in the paper's settings.   */
  uint32_t reserved2;    /* must be 0                                                                   */
  const int32_t* valid_from; /* NULL, or device int32 [nb,Hkv]: KV head g of slice b holds its entries right-aligned,
                            rows i < valid_from[b,g] of K and V are padding (0 <= valid_from <= n - w).  Padding
                            is invisible to the window queries, gets attn = 0 and the scores a = c = -1, below
                            every real entry, so it is selected only if a head's budget exceeds its n -
                            valid_from real entries (the caller's to avoid; adaptive allocation never does while
                            budget <= number of real entries).  This is the ragged cache that adaptive budgets
                            leave between the chunks of a chunked prefill.  Not accepted by
                            criticalkv_compress_host and criticalkv_diagnose.                              */
} criticalkv_desc;

/* Create / destroy a handle bound to CUDA device `device`.  create allocates one device status word. */
CKV_API int criticalkv_create(criticalkv_handle* out, int device);
CKV_API int criticalkv_destroy(criticalkv_handle h);

/* Workspace sizes in bytes for score and select (host computation, no CUDA call); compact needs none. */
CKV_API int criticalkv_workspace_bytes(const criticalkv_desc* d, size_t* score_bytes, size_t* select_bytes);

/*
 * Steps 1-2.  attn[nb,Hq,n]: per query head the causal softmax of the w window queries over all n keys (window row
 * j sits at position n-w+j and sees keys i <= n-w+j), averaged over the window and max-pooled along the sequence
 * (Algorithm 2; Eq. 2).  vnorm[nb,Hq,n]: L1 norm of each value row projected through that head's slice of W^O
 * (Algorithm 1, "L1 norm of each row of V W^O"; Theorem 3.3).  The n x dm product is never written to memory.
 * Either output may be NULL to skip that half.  ws: workspace of at least score_bytes, 256-byte aligned.
 */
CKV_API int criticalkv_score(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K,
                             const void* V, const void* WO, float* attn, float* vnorm, void* ws, size_t ws_bytes,
                             void* stream);

/*
 * Steps 3-4.  Per KV head g: a_g = mean over the group's query heads of attn, c_g = mean of (attn + eps) * vnorm
 * (Algorithm 1), each +, *, / a separately rounded float32 operation, heads summed in increasing order.  Budgets:
 * uniform, flattened top-B_total of a over (g, i) counted per head (Algorithm 2, budget allocation), or read from
 * budgets_in[nb,Hkv] (device).  Then stage 1 keeps the b' largest a_g, stage 2 the b'' largest c_g among the rest
 * (Algorithm 1); ties go to the lower index; idx is ascending inside each head's segment
 * [offsets[g], offsets[g+1]).  stage may be NULL.  With given budgets whose sum is below the capacity the tail of
 * idx is left untouched; budgets outside [0, n] or beyond the capacity are clipped and flagged in the status word.
 * Three implementations give the same bits: one kernel with a CTA per head (default when nb * Hkv exceeds half the
 * number of SMs), separate kernels with a thread-block cluster per head (default for fewer heads, i.e. a layer at a
 * time), separate kernels with a CTA per head (heads too long for the other two); CKV_FLAG_SELECT_* override the
 * choice and criticalkv_last_path reports it.
 */
CKV_API int criticalkv_select(criticalkv_handle h, const criticalkv_desc* d, const float* attn, const float* vnorm,
                              const int32_t* budgets_in, int32_t* idx, int32_t* offsets, uint8_t* stage, void* ws,
                              size_t ws_bytes, void* stream);

/*
 * The two front steps of criticalkv_select on their own, for a layer whose KV heads are spread over several GPUs
 * (each GPU holds some KV heads, their query heads and their rows of W^O).  Uniform budgets need nothing from other
 * GPUs.  The flattened adaptive allocation (Algorithm 2, budget allocation) ranks the group attention scores of ALL
 * heads of the layer, so each GPU
 *   1. criticalkv_score on its heads, then criticalkv_group_scores: a_out[nb,Hkv_local,n] (and c_out, which may be
 *      NULL) from attn and vnorm exactly as criticalkv_select computes them;
 *   2. all-gathers a over the head axis (the caller's collective: Hkv*n floats per layer);
 *   3. criticalkv_allocate_budgets with the descriptor of the WHOLE layer (Hkv, budget = B_total, CKV_BUDGET_FLAT_
 *      ADAPTIVE; Hq, dh, dm only need to be consistent): budgets_out[nb,Hkv] int32, identical on every GPU;
 *   4. criticalkv_select with its local descriptor in CKV_BUDGET_GIVEN mode and its slice of the budgets.
 * The result equals, head for head, that of one GPU holding the whole layer.  All pointers are device memory,
 * a/attn/vnorm 16-byte aligned; neither call needs a workspace.
 */
CKV_API int criticalkv_group_scores(criticalkv_handle h, const criticalkv_desc* d, const float* attn,
                                    const float* vnorm, float* a_out, float* c_out, void* stream);
CKV_API int criticalkv_allocate_budgets(criticalkv_handle h, const criticalkv_desc* d, const float* a,
                                        int32_t* budgets_out, void* stream);

/*
 * Allocation-free variant of criticalkv_select (the paper has no counterpart: this is a packaging of steps 3-4 for
 * callers that cannot provide a workspace).  Some hosts of this library may not allocate device memory at the point
 * where they compress a cache: a serving engine that reserved all of HBM for its own pools at start-up has nothing
 * left for cudaMalloc, and a latency-critical loop cannot afford the device-wide synchronisation an allocation or a
 * free implies.  This entry point therefore takes no workspace: the group scores and per-head budgets go to a fixed
 * array of CKV_STATIC_SCRATCH_BYTES that lives inside the library image (every GPU that loads the library keeps
 * that much memory until the process exits).  Arguments and results are those of criticalkv_select.
 *   - The request must fit: if the select_bytes that criticalkv_workspace_bytes reports exceeds
 *     CKV_STATIC_SCRATCH_BYTES (about nb*Hkv*n > 2^20 scored entries) the call returns CKV_EWORKSPACE, launches
 *     nothing, and criticalkv_last_cuda_error describes the sizes.
 *   - The first call on each device looks up the array's device address (once, with that device current); make that
 *     first call outside any stream capture.  No call allocates or frees device memory.
 *   - All calls, from every handle and stream of the process, share the one array per device.  Nothing is read from
 *     it before this call has written it, so stale contents are harmless, but two calls whose kernels may overlap on
 *     the GPU (different streams) race on it: order them on one stream or with events.
 */
#define CKV_STATIC_SCRATCH_BYTES ((size_t)((8u << 20) + (64u << 10)))
CKV_API int criticalkv_select_static(criticalkv_handle h, const criticalkv_desc* d, const float* attn,
                                     const float* vnorm, const int32_t* budgets_in, int32_t* idx, int32_t* offsets,
                                     uint8_t* stage, void* stream);

/* Step 5.  K_out[nb, r, :] = K[nb, g, idx[nb, r], :] for r in head g's segment, same for V (bit copy). */
CKV_API int criticalkv_compact(criticalkv_handle h, const criticalkv_desc* d, const void* K, const void* V,
                               const int32_t* idx, const int32_t* offsets, void* K_out, void* V_out, void* stream);

/*
 * Companion of criticalkv_compact for chunked prefill (the paper's long-context deployment: the cache is compressed
 * after every prefill chunk and later chunks see [retained entries ; new chunk]).  pos_in[nb,Hkv,n] int32 holds the
 * original token position of every cached entry; pos_out[nb, r] = pos_in[nb, g, idx[nb, r]] keeps them attached to
 * the retained rows.
 */
CKV_API int criticalkv_gather_positions(criticalkv_handle h, const criticalkv_desc* d, const int32_t* pos_in,
                                        const int32_t* idx, const int32_t* offsets, int32_t* pos_out, void* stream);

/* The three calls above back to back on one stream.  ws must hold max(score_bytes, select_bytes). */
CKV_API int criticalkv_compress(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K,
                                const void* V, const void* WO, const int32_t* budgets_in, float* attn, float* vnorm,
                                int32_t* idx, int32_t* offsets, uint8_t* stage, void* K_out, void* V_out, void* ws,
                                size_t ws_bytes, void* stream);

/*
 * The whole path for callers whose tensors live in HOST memory (pinned memory recommended): Qw, K, V, WO,
 * budgets_in (given budgets only) are host arrays in the dense layouts above, idx [nb,Btot], offsets [nb,Hkv+1],
 * K_out, V_out [nb,Btot,dh] are host arrays that receive the result.  The nb slices are streamed one at a time
 * through two device staging buffers on two internal streams, so that the upload of slice b+1, the kernels of slice b
 * and the download of slice b-1 overlap.  `staging` is DEVICE memory of at least criticalkv_host_staging_bytes(d),
 * 256-byte aligned, owned by the caller; the call allocates no device memory (its first use on a handle creates two
 * streams and three events).  Work starts after everything already queued on `stream`; unlike the other calls this
 * one returns only when the results are in host memory.  Element strides in the descriptor must be 0 (dense).
 */
CKV_API int criticalkv_host_staging_bytes(const criticalkv_desc* d, size_t* bytes);
CKV_API int criticalkv_compress_host(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K,
                                     const void* V, const void* WO, const int32_t* budgets_in, int32_t* idx,
                                     int32_t* offsets, void* K_out, void* V_out, void* staging,
                                     size_t staging_bytes, void* stream);

/*
 * Perturbation diagnostics of Section 3 for a finished selection (not on the hot path).  For every query head and
 * window row j, with A the causal softmax row of that query and nu = vnorm of the head:
 *   diag[nb,Hq,w,10] = sigma (attention mass of the stage-1 set, Assumption 3.4), retained mass, C = sum_i A_i nu_i,
 *   its parts over stage 1 and stage 2, min_i nu_i, L = ||(A - A') V W^O||_1 (Definition 3.1 with A' of Theorem 3.2),
 *   theta (Theorem 3.3), theta_hat (Theorem 3.5), theta_relax (relaxed bound of the appendix).
 * vnorm is the per-head output of criticalkv_score (CKV_ENOTSUP with CKV_FLAG_WO_GROUP_SUM or w > 64); idx, offsets
 * and stage (required) come from criticalkv_select.  ws: criticalkv_diagnose_workspace_bytes, 256-byte aligned.
 */
#define CKV_DIAG_FIELDS 10
CKV_API int criticalkv_diagnose_workspace_bytes(const criticalkv_desc* d, size_t* bytes);
CKV_API int criticalkv_diagnose(criticalkv_handle h, const criticalkv_desc* d, const void* Qw, const void* K,
                                const void* V, const void* WO, const float* vnorm, const int32_t* idx,
                                const int32_t* offsets, const uint8_t* stage, float* diag, void* ws, size_t ws_bytes,
                                void* stream);

/*
 * Self-test of the bounded device-side wait every tensor-core kernel uses: launches one CTA that waits, for at most
 * limit_ns nanoseconds, on a barrier nothing will ever signal.  The kernel must give up, write 0 to *observed_device
 * (a device int; 1 would mean the wait claimed success), set the status word to CKV_ETIMEOUT and end normally.
 * limit_ns above CKV_SELFTEST_MAX_WAIT_NS (100 ms) is refused with CKV_EINVAL: no wait of this library may hold an SM
 * for long.
 */
#define CKV_SELFTEST_MAX_WAIT_NS 100000000ull
CKV_API int criticalkv_selftest_bounded_wait(criticalkv_handle h, uint64_t limit_ns, int* observed_device,
                                             void* stream);

/* Reads the device status word (synchronises `stream` first), clears it, and returns it in *out. */
CKV_API int criticalkv_device_status(criticalkv_handle h, void* stream, int* out);

CKV_API const char* criticalkv_status_string(int status);
/* Last CUDA error string (or size diagnostic of criticalkv_select_static) seen by this handle ("" if none); valid
   until the next call on the handle. */
CKV_API const char* criticalkv_last_cuda_error(criticalkv_handle h);
/* Which kernels the last criticalkv_score on this handle launched: bit0 tensor-core window attention,
   bit1 tensor-core projection norm, bit2 CUDA-core window attention, bit3 CUDA-core projection norm,
   bit5: the last criticalkv_select (or
   criticalkv_select_static) ran as the single kernel; bit6: its two-stage top-k ran with a cluster per head. */
CKV_API int criticalkv_last_path(criticalkv_handle h);
/* Number of kernel launches this handle has issued since it was created. */
CKV_API int64_t criticalkv_launch_count(criticalkv_handle h);

#ifdef __cplusplus
}
#endif
#endif /* CRITICALKV_H_ */
