// Steps 3-4: scores per KV head, budgets, and the two-stage top-k of Algorithm 1.
//
//   group_reduce : a_g = mean_h attn_h, c_g = mean_h (attn_h + eps) * vnorm_h over the query heads of a KV group,
//                  every operation a separately rounded float32 op in a fixed order (the selection is decided in
//                  exactly this arithmetic)
//   adaptive     : flattened top-B_total of a over (g, i), counted per head (Algorithm 2, budget allocation)
//   two_stage    : per (nb, KV head): stage 1 = b' largest a_g, stage 2 = b'' largest c_g among the rest,
//                  b' = floor(alpha * b); ties go to the lower index; indices written in ascending order
//
// Top-k is a radix *select* (4 passes of 8 bits over order-preserving integer keys) followed by an ordered walk that
// resolves ties by index and compacts with warp ballots: no sort, no floating-point atomics, bit-reproducible.
#include <cooperative_groups.h>

#include "ckv_internal.h"
#include "select_common.cuh"

namespace ckv {
namespace {

__global__ void group_reduce_kernel(GroupScoreArgs p, float* __restrict__ a, float* __restrict__ c) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= p.n) return;
  const int g = blockIdx.y, b = blockIdx.z;
  float av, cv;
  group_scores_of(p, b, g, i, &av, &cv);
  const long long o = ((long long)b * p.Hkv + g) * p.n + i;
  a[o] = av;
  if (c != nullptr) c[o] = cv;
}

struct TwoStageArgs {
  const float* a;
  const float* c;
  const int32_t* budgets;  // [nb, Hkv] or nullptr for uniform
  int32_t* idx;
  int32_t* offsets;
  uint8_t* stage;
  int* status;
  int Hkv, n;
  long long uniform_b, btot;
  float alpha;
  int debug;   // CKV_FLAG_DEBUG_CHECKS: report a skipped write
};

__global__ void __launch_bounds__(kSelThreads) two_stage_kernel(TwoStageArgs p) {
  extern __shared__ __align__(16) uint32_t dyn[];
  __shared__ SelectShared sh;
  const int g = blockIdx.x, b = blockIdx.y;
  const int n = p.n;
  const int nwords = (n + 31) / 32;
  uint32_t* sel1 = dyn;
  uint32_t* sel2 = dyn + nwords;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // this head's budget and the start of its segment
  long long off = 0, bud;
  bool clipped = false;
  if (p.budgets == nullptr) {
    bud = p.uniform_b;
    off = (long long)g * bud;
  } else {
    const int32_t* bb = p.budgets + (long long)b * p.Hkv;
    for (int q = 0; q < g; ++q) off += min(max((long long)bb[q], 0LL), (long long)n);
    bud = bb[g];
    if (bud < 0 || bud > n) { bud = min(max(bud, 0LL), (long long)n); clipped = true; }
    if (off > p.btot) { off = p.btot; clipped = true; }
    if (off + bud > p.btot) { bud = p.btot - off; clipped = true; }
  }
  if (clipped && threadIdx.x == 0) atomicExch(p.status, (int)CKV_EINVAL);
  long long b1 = (long long)floor((double)p.alpha * (double)bud);
  b1 = min(max(b1, 0LL), bud);
  const long long b2 = bud - b1;

  const float* ag = p.a + ((long long)b * p.Hkv + g) * n;
  const float* cg = p.c + ((long long)b * p.Hkv + g) * n;

  uint32_t T = 0, r = 0;
  if (b1 > 0) radix_select(ag, n, nullptr, (uint32_t)b1, sh, &T, &r);
  mark_selected(ag, n, nullptr, T, r, b1 > 0, sel1, sh);
  if (b2 > 0) radix_select(cg, n, sel1, (uint32_t)b2, sh, &T, &r);
  mark_selected(cg, n, sel1, T, r, b2 > 0, sel2, sh);

  // ordered compaction of sel1 | sel2
  const int wpw = (nwords + kSelWarps - 1) / kSelWarps;
  const int w0 = min(warp * wpw, nwords), w1 = min(w0 + wpw, nwords);
  uint32_t cnt = 0;
  for (int q = w0 + lane; q < w1; q += 32) cnt += __popc(sel1[q] | sel2[q]);
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if (lane == 0) sh.warp_cnt[warp] = cnt;
  __syncthreads();
  uint32_t running = 0;
  for (int q = 0; q < warp; ++q) running += sh.warp_cnt[q];
  int32_t* idx = p.idx + (long long)b * p.btot + off;
  uint8_t* stage = p.stage ? p.stage + (long long)b * p.btot + off : nullptr;
  for (int q = w0; q < w1; ++q) {
    const uint32_t s1 = sel1[q], word = s1 | sel2[q];
    if ((word >> lane) & 1u) {
      const uint32_t pos = running + __popc(word & ((1u << lane) - 1u));
      if ((long long)pos < bud) {   // a selection larger than the budget never writes past the head's segment
        idx[pos] = q * 32 + lane;
        if (stage) stage[pos] = ((s1 >> lane) & 1u) ? 1 : 2;
      } else if (p.debug) {
        atomicExch(p.status, (int)CKV_EBOUNDS);
      }
    }
    running += __popc(word);
  }
  if (threadIdx.x == 0) {
    p.offsets[(long long)b * (p.Hkv + 1) + g] = (int32_t)off;
    if (g == p.Hkv - 1) p.offsets[(long long)b * (p.Hkv + 1) + p.Hkv] = (int32_t)(off + bud);
  }
}

// Flattened top-B_total over a[nb, Hkv*n]: budgets[g] = #{i : key > T} + the first ties in (g, i) order.
__global__ void __launch_bounds__(kSelThreads) adaptive_budget_kernel(const float* __restrict__ a,
                                                                      int32_t* __restrict__ budgets, int Hkv, int n,
                                                                      long long btotal, int floor_b) {
  __shared__ SelectShared sh;
  __shared__ uint32_t cnt_gt[64], cnt_eq[64];
  const int b = blockIdx.x;
  const float* ab = a + (long long)b * Hkv * n;
  int32_t* out = budgets + (long long)b * Hkv;
  if (btotal <= 0) {  // nothing left for the flattened top-k: every head gets its guaranteed share
    if (threadIdx.x < Hkv) out[threadIdx.x] = min(floor_b, n);
    return;
  }
  uint32_t T, r;
  radix_select(ab, (long long)Hkv * n, nullptr, (uint32_t)btotal, sh, &T, &r);
  if (threadIdx.x < 64) { cnt_gt[threadIdx.x] = 0; cnt_eq[threadIdx.x] = 0; }
  __syncthreads();
  for (int g = 0; g < Hkv; ++g) {
    uint32_t gt = 0, eq = 0;
    scan_keys(ab + (long long)g * n, n, [&](long long, float x) {
      const uint32_t key = order_key(x);
      gt += key > T;
      eq += key == T;
    });
    gt = __reduce_add_sync(0xffffffffu, gt);
    eq = __reduce_add_sync(0xffffffffu, eq);
    if ((threadIdx.x & 31) == 0) {
      if (gt) atomicAdd(&cnt_gt[g], gt);
      if (eq) atomicAdd(&cnt_eq[g], eq);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t rem = r;
    for (int g = 0; g < Hkv; ++g) {
      const uint32_t take = min(cnt_eq[g], rem);
      out[g] = (int32_t)min((long long)cnt_gt[g] + take + floor_b, (long long)n);
      rem -= take;
    }
  }
}

// The same allocation spread over a thread-block cluster: CTA r of the cluster owns Hkv / cluster_size whole KV heads of
// one nb slice, builds the digit histogram of its share, and every CTA sums the histograms of all ranks through
// distributed shared memory, so all of them walk the same radix-select decisions without any broadcast.  Two hardware
// cluster barriers per pass (histograms complete / histograms consumed).  Rank 0 finally reads every rank's per-head
// counts and hands out the ties in flattened (g, i) order.
struct ClusterShared {
  uint32_t hist[kSelWarps][256];
  uint32_t total[256];    // this CTA's histogram of the current pass (read by the peers)
  uint32_t gtotal[256];   // sum over the cluster
  uint32_t cnt_gt[64], cnt_eq[64];
  uint32_t prefix, krem;
};

__global__ void __launch_bounds__(kSelThreads) adaptive_budget_cluster_kernel(const float* __restrict__ a,
                                                                              int32_t* __restrict__ budgets, int Hkv,
                                                                              int n, long long btotal, int floor_b,
                                                                              int cached) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ ClusterShared sh;
  extern __shared__ __align__(16) uint32_t kcache[];   // cached != 0: the integer keys of this CTA's share
  const int cs = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int b = blockIdx.x / cs;
  const int heads = Hkv / cs, g0 = rank * heads;
  const float* ab = a + (long long)b * Hkv * n;
  int32_t* out = budgets + (long long)b * Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (btotal <= 0) {   // uniform across the cluster: nobody reaches a cluster barrier
    if (tid < heads) out[g0 + tid] = min(floor_b, n);
    return;
  }
  const long long count = (long long)heads * n;
  const float* mine = ab + (long long)g0 * n;
  if (tid == 0) { sh.prefix = 0; sh.krem = (uint32_t)btotal; }
  // the five walks over this CTA's share read it from shared memory when it fits (a layer at a time), else from L2
  if (cached) scan_keys(mine, count, [&](long long i, float x) { kcache[i] = order_key(x); });
  auto each_key = [&](long long first, long long cnt, auto&& f) {
    if (cached) {
      for (long long i = tid; i < cnt; i += kSelThreads) f(kcache[first + i]);
    } else {
      scan_keys(mine + first, cnt, [&](long long, float x) { f(order_key(x)); });
    }
  };
  uint32_t known = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int e = tid; e < kSelWarps * 256; e += kSelThreads) (&sh.hist[0][0])[e] = 0;
    __syncthreads();
    const uint32_t prefix = sh.prefix;
    each_key(0, count, [&](uint32_t key) {
      if ((key & known) == prefix) atomicAdd(&sh.hist[warp][(key >> shift) & 255u], 1u);
    });
    __syncthreads();
    if (tid < 256) {
      uint32_t s = 0;
      for (int wq = 0; wq < kSelWarps; ++wq) s += sh.hist[wq][tid];
      sh.total[tid] = s;
    }
    cluster.sync();   // every rank's total[] is complete
    if (tid < 256) {
      uint32_t s = 0;
      for (int q = 0; q < cs; ++q) s += cluster.map_shared_rank(sh.total, q)[tid];
      sh.gtotal[tid] = s;
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t m = 0;
      for (int q = 0; q < 8; ++q) m += sh.gtotal[lane * 8 + q];
      uint32_t above = m;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, above, o);
        if (lane + o < 32) above += v;
      }
      above -= m;
      const uint32_t krem = sh.krem;
      if (above < krem && krem <= above + m) {
        uint32_t acc = above;
        for (int q = 7; q >= 0; --q) {
          const uint32_t cnt = sh.gtotal[lane * 8 + q];
          if (acc + cnt >= krem) {
            sh.prefix = prefix | ((uint32_t)(lane * 8 + q) << shift);
            sh.krem = krem - acc;
            break;
          }
          acc += cnt;
        }
      }
    }
    known |= 0xffu << shift;
    cluster.sync();   // peers are done reading total[] before the next pass rewrites it
  }
  const uint32_t T = sh.prefix, r = sh.krem;
  if (tid < 64) { sh.cnt_gt[tid] = 0; sh.cnt_eq[tid] = 0; }
  __syncthreads();
  for (int g = 0; g < heads; ++g) {
    uint32_t gt = 0, eq = 0;
    each_key((long long)g * n, n, [&](uint32_t key) {
      gt += key > T;
      eq += key == T;
    });
    gt = __reduce_add_sync(0xffffffffu, gt);
    eq = __reduce_add_sync(0xffffffffu, eq);
    if (lane == 0) {
      if (gt) atomicAdd(&sh.cnt_gt[g], gt);
      if (eq) atomicAdd(&sh.cnt_eq[g], eq);
    }
  }
  cluster.sync();
  if (rank == 0 && tid == 0) {
    uint32_t rem = r;
    for (int q = 0; q < cs; ++q) {
      const uint32_t* pgt = cluster.map_shared_rank(sh.cnt_gt, q);
      const uint32_t* peq = cluster.map_shared_rank(sh.cnt_eq, q);
      for (int g = 0; g < heads; ++g) {
        const uint32_t take = min(peq[g], rem);
        out[q * heads + g] = (int32_t)min((long long)pgt[g] + take + floor_b, (long long)n);
        rem -= take;
      }
    }
  }
  cluster.sync();   // rank 0 has read the peers' counts
}

}  // namespace

size_t two_stage_smem_bytes(int n) {
  // two bit masks of n bits (dynamic) next to the kernel's static histograms
  return (size_t)2 * ((n + 31) / 32) * sizeof(uint32_t) + sizeof(SelectShared) + 1024;
}

cudaError_t launch_group_scores(const Dims& d, const float* attn, const float* vnorm, float* a, float* c,
                                cudaStream_t st, int* launches) {
  dim3 rgrid((d.n + 255) / 256, d.Hkv, d.nb);
  group_reduce_kernel<<<rgrid, 256, 0, st>>>(group_score_args(d, attn, vnorm), a, c);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_allocate_budgets(const Dims& d, const float* a_all, int32_t* budgets_out, int smem_optin,
                                    cudaStream_t st, int* launches) {
  const long long b_adapt = d.budget - d.Hkv * d.floor_b;
  int cs = 8;
  while (cs > 1 && d.Hkv % cs != 0) cs >>= 1;
  bool launched = false;
  if (cs > 1) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(d.nb * cs));
    cfg.blockDim = dim3(kSelThreads);
    const size_t share = (size_t)(d.Hkv / cs) * d.n * sizeof(uint32_t);
    int cached = share + sizeof(ClusterShared) + 1024 <= (size_t)smem_optin ? 1 : 0;
    if (cached && cudaFuncSetAttribute(adaptive_budget_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)share) != cudaSuccess) {
      (void)cudaGetLastError();
      cached = 0;
    }
    cfg.dynamicSmemBytes = cached ? share : 0;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = (unsigned)cs;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const cudaError_t ec = cudaLaunchKernelEx(&cfg, adaptive_budget_cluster_kernel, a_all, budgets_out, d.Hkv, d.n,
                                              b_adapt, (int)d.floor_b, cached);
    if (ec == cudaSuccess) launched = true;
    else (void)cudaGetLastError();   // no cluster launch on this device: use the single-CTA kernel
  }
  if (!launched)
    adaptive_budget_kernel<<<d.nb, kSelThreads, 0, st>>>(a_all, budgets_out, d.Hkv, d.n, b_adapt, (int)d.floor_b);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_select(const Dims& d, const float* attn, const float* vnorm, const int32_t* budgets_in,
                          int32_t* idx, int32_t* offsets, uint8_t* stage, const SelectWorkspace& ws,
                          const SelectDevice& dev, cudaStream_t st, int* launches, int* status_word, int* fused) {
  *fused = 0;
  // few heads (a layer at a time): the separate kernels with a cluster of CTAs per head beat one CTA per head
  const bool few_heads = two_stage_cluster_applies(d, dev);
  if (dev.allow_fused && (dev.prefer_fused || !few_heads)) {
    // one kernel when the shape allows it; otherwise the three kernels below
    const cudaError_t ef = launch_select_fused(d, attn, vnorm, budgets_in, idx, offsets, stage, ws, dev, st, launches,
                                               status_word);
    if (ef == cudaSuccess) {
      *fused = 1;
      return ef;
    }
    if (ef != cudaErrorNotSupported) return ef;
  }
  cudaError_t e;
  if (few_heads && d.budget_mode != CKV_BUDGET_FLAT_ADAPTIVE) {
    // uniform or given budgets: the cluster kernel computes the group scores itself
    e = launch_two_stage_cluster(d, attn, vnorm, nullptr, nullptr,
                                 d.budget_mode == CKV_BUDGET_GIVEN ? budgets_in : nullptr, idx, offsets, stage, dev, st,
                                 launches, status_word);
    if (e == cudaSuccess) *fused = 2;
    if (e != cudaErrorNotSupported) return e;
  }
  e = launch_group_scores(d, attn, vnorm, ws.a, ws.c, st, launches);
  if (e != cudaSuccess) return e;
  const int32_t* budgets = nullptr;
  if (d.budget_mode == CKV_BUDGET_FLAT_ADAPTIVE) {
    if ((e = launch_allocate_budgets(d, ws.a, ws.budgets, dev.smem_optin, st, launches)) != cudaSuccess) return e;
    budgets = ws.budgets;
  } else if (d.budget_mode == CKV_BUDGET_GIVEN) {
    budgets = budgets_in;
  }
  if (dev.allow_cluster) {
    e = launch_two_stage_cluster(d, attn, vnorm, ws.a, ws.c, budgets, idx, offsets, stage, dev, st, launches,
                                 status_word);
    if (e == cudaSuccess) *fused = 2;
    if (e != cudaErrorNotSupported) return e;
  }
  TwoStageArgs p;
  p.a = ws.a; p.c = ws.c; p.budgets = budgets; p.idx = idx; p.offsets = offsets; p.stage = stage;
  p.status = status_word;
  p.Hkv = d.Hkv; p.n = d.n; p.uniform_b = d.budget; p.btot = d.btot; p.alpha = d.alpha;
  p.debug = d.debug_checks;
  const size_t dyn = (size_t)2 * ((d.n + 31) / 32) * sizeof(uint32_t);
  e = cudaFuncSetAttribute(two_stage_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
  if (e != cudaSuccess) return e;
  dim3 tgrid(d.Hkv, d.nb);
  two_stage_kernel<<<tgrid, kSelThreads, dyn, st>>>(p);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace ckv
