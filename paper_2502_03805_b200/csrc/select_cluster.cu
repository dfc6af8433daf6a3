// Step 4 for calls with few KV heads (one layer at a time): the two-stage top-k of Algorithm 1 (stage 1 by attention,
// stage 2 by the perturbation-aware score among the rest) with one thread-block CLUSTER per (nb slice, KV head), so
// that a single layer's eight heads occupy 64 SMs instead of 8 (8, 4 or 2 CTAs per head, as many as are resident at once).
//
// CTA r of a head's cluster owns the contiguous index range [r * m, (r + 1) * m) and keeps the order-preserving integer
// keys of a_g and c_g of that range in shared memory for the whole kernel (the scores cross L2 once; unless the budgets
// are the flattened adaptive ones, which need a_g of all heads first, the group scores are computed here as well).  A top-k is a
// radix select in four passes of 8 bits: every CTA histograms its own keys, all CTAs read every peer's histogram
// through distributed shared memory and so walk the same decisions without any broadcast (two hardware cluster
// barriers per pass).  Ties go to the lower index: a CTA learns through the same exchange how many entries equal to
// the threshold the lower ranks hold.  The ascending index list is written with a cluster-wide prefix of the per-CTA
// counts.  Same keys, same tie rule, same budget arithmetic as the one-CTA-per-head kernel: identical results.
#include <cooperative_groups.h>

#include "ckv_internal.h"
#include "select_common.cuh"

namespace ckv {
namespace {

namespace cg = cooperative_groups;

constexpr int kMaxClusterSize = 8;   // portable maximum

struct HeadShared {
  uint32_t hist[kSelWarps][256];
  uint32_t total[256];    // this CTA's histogram of the current pass (read by the peers)
  uint32_t gtotal[256];   // sum over the cluster
  uint32_t warp_cnt[kSelWarps];
  uint32_t xchg;          // one count per CTA, read by the peers
  uint32_t prefix, krem;
};

struct ClusterArgs {
  GroupScoreArgs gs;       // a == nullptr: the group scores are computed here from attn and vnorm
  const float* a;
  const float* c;
  const int32_t* budgets;  // [nb, Hkv] or nullptr for uniform
  int32_t* idx;
  int32_t* offsets;
  uint8_t* stage;
  int* status;
  int Hkv, n, m;           // m: entries per CTA, a multiple of 32
  long long uniform_b, btot;
  float alpha;
  int debug;
};

__device__ __forceinline__ bool bit_set(const uint32_t* mask, int i) { return (mask[i >> 5] >> (i & 31)) & 1u; }

// k-th largest key over the cluster's candidates (local entries [0, cnt) whose bit in excl is clear); every CTA of the
// cluster calls it with its own keys and returns the same (T, r): r entries equal to T belong to the top k.
__device__ void cluster_radix_select(cg::cluster_group& cluster, const uint32_t* keys, int cnt, const uint32_t* excl,
                                     uint32_t k, HeadShared& sh, uint32_t* T, uint32_t* r) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { sh.prefix = 0; sh.krem = k; }
  uint32_t known = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int e = tid; e < kSelWarps * 256; e += kSelThreads) (&sh.hist[0][0])[e] = 0;
    __syncthreads();
    const uint32_t prefix = sh.prefix;
    for (int i = tid; i < cnt; i += kSelThreads) {
      if (excl != nullptr && bit_set(excl, i)) continue;
      const uint32_t key = keys[i];
      if ((key & known) == prefix) atomicAdd(&sh.hist[warp][(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 256) {
      uint32_t s = 0;
      for (int wq = 0; wq < kSelWarps; ++wq) s += sh.hist[wq][tid];
      sh.total[tid] = s;
    }
    cluster.sync();   // every rank's total[] is complete
    if (tid < 256) {
      uint32_t s = 0;
      for (int q = 0; q < (int)cluster.num_blocks(); ++q) s += cluster.map_shared_rank(sh.total, q)[tid];
      sh.gtotal[tid] = s;
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns digits 8l .. 8l+7; find the digit at which the count from the top reaches krem
      uint32_t mine = 0;
      for (int q = 0; q < 8; ++q) mine += sh.gtotal[lane * 8 + q];
      uint32_t above = mine;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, above, o);
        if (lane + o < 32) above += v;
      }
      above -= mine;
      const uint32_t krem = sh.krem;
      if (above < krem && krem <= above + mine) {
        uint32_t acc = above;
        for (int q = 7; q >= 0; --q) {
          const uint32_t c8 = sh.gtotal[lane * 8 + q];
          if (acc + c8 >= krem) {
            sh.prefix = prefix | ((uint32_t)(lane * 8 + q) << shift);
            sh.krem = krem - acc;
            break;
          }
          acc += c8;
        }
      }
    }
    known |= 0xffu << shift;
    cluster.sync();   // peers are done reading total[] before the next pass rewrites it; prefix / krem are written
  }
  *T = sh.prefix;
  *r = sh.krem;
}

// Sum of v over the CTAs of lower rank (all threads get it).  Two cluster barriers.
__device__ uint32_t cluster_exclusive(cg::cluster_group& cluster, uint32_t v, HeadShared& sh) {
  if (threadIdx.x == 0) sh.xchg = v;
  cluster.sync();
  uint32_t before = 0;
  const int rank = (int)cluster.block_rank();
  for (int q = 0; q < rank; ++q) before += *cluster.map_shared_rank(&sh.xchg, q);
  cluster.sync();
  return before;
}

// Bit i of out[] is set iff key_i > T, or key_i == T and fewer than r equal candidates precede i in the cluster's
// index order.  Warp q owns the contiguous word range [q * wpw, (q + 1) * wpw) of this CTA's entries.
__device__ void cluster_mark(cg::cluster_group& cluster, const uint32_t* keys, int cnt, int words, const uint32_t* excl,
                             uint32_t T, uint32_t r, bool any, uint32_t* out, HeadShared& sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wpw = (words + kSelWarps - 1) / kSelWarps;
  const int w0 = min(warp * wpw, words), w1 = min(w0 + wpw, words);
  uint32_t eq_count = 0;
  for (int q = w0; q < w1; ++q) {
    const int i = q * 32 + lane;
    const bool valid = any && i < cnt && !(excl != nullptr && bit_set(excl, i));
    eq_count += __popc(__ballot_sync(0xffffffffu, valid && keys[i] == T));
  }
  __syncthreads();
  if (lane == 0) sh.warp_cnt[warp] = eq_count;
  __syncthreads();
  uint32_t running = 0, mine = 0;
  for (int q = 0; q < kSelWarps; ++q) {
    const uint32_t w = sh.warp_cnt[q];
    if (q < warp) running += w;
    mine += w;
  }
  running += cluster_exclusive(cluster, mine, sh);
  for (int q = w0; q < w1; ++q) {
    const int i = q * 32 + lane;
    const bool valid = any && i < cnt && !(excl != nullptr && bit_set(excl, i));
    const uint32_t key = valid ? keys[i] : 0u;
    const bool eq = valid && key == T;
    const uint32_t eqm = __ballot_sync(0xffffffffu, eq);
    const bool take = eq && (running + __popc(eqm & ((1u << lane) - 1u)) < r);
    const uint32_t word = __ballot_sync(0xffffffffu, (valid && key > T) || take);
    if (lane == 0) out[q] = word;
    running += __popc(eqm);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads) two_stage_cluster_kernel(ClusterArgs p) {
  extern __shared__ __align__(16) uint32_t dyn[];
  __shared__ HeadShared sh;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.x / (int)cluster.num_blocks();
  const int g = head % p.Hkv, b = head / p.Hkv;
  const int n = p.n, m = p.m, words = m / 32;
  uint32_t* ka = dyn;
  uint32_t* kc = dyn + m;
  uint32_t* sel1 = dyn + 2 * m;
  uint32_t* sel2 = sel1 + words;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // this head's budget and the start of its segment (the arithmetic of the one-CTA kernel)
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
  if (clipped && rank == 0 && threadIdx.x == 0) atomicExch(p.status, (int)CKV_EINVAL);
  long long b1 = (long long)floor((double)p.alpha * (double)bud);
  b1 = min(max(b1, 0LL), bud);
  const long long b2 = bud - b1;

  // this CTA's entries
  const int i0 = rank * m;
  const int cnt = max(0, min(m, n - i0));
  if (p.a != nullptr) {
    const float* ag = p.a + ((long long)b * p.Hkv + g) * n + i0;
    const float* cg_ = p.c + ((long long)b * p.Hkv + g) * n + i0;
    for (int i = threadIdx.x; i < m; i += kSelThreads) {
      ka[i] = i < cnt ? order_key(ag[i]) : 0u;
      kc[i] = i < cnt ? order_key(cg_[i]) : 0u;
    }
  } else {
    for (int i = threadIdx.x; i < m; i += kSelThreads) {
      float av = 0.f, cv = 0.f;
      if (i < cnt) group_scores_of(p.gs, b, g, i0 + i, &av, &cv);
      ka[i] = i < cnt ? order_key(av) : 0u;
      kc[i] = i < cnt ? order_key(cv) : 0u;
    }
  }
  __syncthreads();

  uint32_t T = 0, r = 0;
  if (b1 > 0) cluster_radix_select(cluster, ka, cnt, nullptr, (uint32_t)b1, sh, &T, &r);   // b1 is the same in every CTA
  cluster_mark(cluster, ka, cnt, words, nullptr, T, r, b1 > 0, sel1, sh);
  if (b2 > 0) cluster_radix_select(cluster, kc, cnt, sel1, (uint32_t)b2, sh, &T, &r);
  cluster_mark(cluster, kc, cnt, words, sel1, T, r, b2 > 0, sel2, sh);

  // ordered compaction of sel1 | sel2 across the cluster
  const int wpw = (words + kSelWarps - 1) / kSelWarps;
  const int w0 = min(warp * wpw, words), w1 = min(w0 + wpw, words);
  uint32_t wc = 0;
  for (int q = w0 + lane; q < w1; q += 32) wc += __popc(sel1[q] | sel2[q]);
  wc = __reduce_add_sync(0xffffffffu, wc);
  __syncthreads();
  if (lane == 0) sh.warp_cnt[warp] = wc;
  __syncthreads();
  uint32_t running = 0, mine = 0;
  for (int q = 0; q < kSelWarps; ++q) {
    const uint32_t w = sh.warp_cnt[q];
    if (q < warp) running += w;
    mine += w;
  }
  running += cluster_exclusive(cluster, mine, sh);
  int32_t* idx = p.idx + (long long)b * p.btot + off;
  uint8_t* stage = p.stage ? p.stage + (long long)b * p.btot + off : nullptr;
  for (int q = w0; q < w1; ++q) {
    const uint32_t s1 = sel1[q], word = s1 | sel2[q];
    if ((word >> lane) & 1u) {
      const uint32_t pos = running + __popc(word & ((1u << lane) - 1u));
      if ((long long)pos < bud) {   // a selection larger than the budget never writes past the head's segment
        idx[pos] = i0 + q * 32 + lane;
        if (stage) stage[pos] = ((s1 >> lane) & 1u) ? 1 : 2;
      } else if (p.debug) {
        atomicExch(p.status, (int)CKV_EBOUNDS);
      }
    }
    running += __popc(word);
  }
  if (rank == 0 && threadIdx.x == 0) {
    p.offsets[(long long)b * (p.Hkv + 1) + g] = (int32_t)off;
    if (g == p.Hkv - 1) p.offsets[(long long)b * (p.Hkv + 1) + p.Hkv] = (int32_t)(off + bud);
  }
}

// CTAs per head (8, 4 or 2: as many as keeps all clusters of the call resident at once) and entries per CTA; false when
// the call has too many heads or a CTA's share does not fit in shared memory.
bool cluster_shape(const Dims& d, const SelectDevice& dev, int* cs_out, int* m_out, size_t* dyn_out) {
  const long long heads = (long long)d.nb * d.Hkv;
  int cs = kMaxClusterSize;
  while (cs > 2 && heads * cs > (long long)dev.sm_count * 3 / 4) cs >>= 1;
  if (heads * cs > (long long)dev.sm_count) return false;
  const int m = ((d.n + cs - 1) / cs + 31) / 32 * 32;
  const size_t dyn = ((size_t)2 * m + 2 * (m / 32)) * sizeof(uint32_t);
  if (dyn + sizeof(HeadShared) + 1024 > (size_t)dev.smem_optin) return false;
  *cs_out = cs;
  *m_out = m;
  *dyn_out = dyn;
  return true;
}

}  // namespace

bool two_stage_cluster_applies(const Dims& d, const SelectDevice& dev) {
  int cs, m;
  size_t dyn;
  return dev.allow_cluster && cluster_shape(d, dev, &cs, &m, &dyn);
}

// cudaErrorNotSupported: the shape does not fit or the device refuses the cluster launch; nothing has been launched.
cudaError_t launch_two_stage_cluster(const Dims& d, const float* attn, const float* vnorm, const float* a,
                                     const float* c, const int32_t* budgets, int32_t* idx, int32_t* offsets,
                                     uint8_t* stage, const SelectDevice& dev, cudaStream_t st, int* launches,
                                     int* status_word) {
  int cs, m;
  size_t dyn;
  if (!cluster_shape(d, dev, &cs, &m, &dyn)) return cudaErrorNotSupported;
  const long long heads = (long long)d.nb * d.Hkv;
  ClusterArgs p;
  p.gs = group_score_args(d, attn, vnorm);
  p.a = a; p.c = c; p.budgets = budgets; p.idx = idx; p.offsets = offsets; p.stage = stage; p.status = status_word;
  p.Hkv = d.Hkv; p.n = d.n; p.m = m; p.uniform_b = d.budget; p.btot = d.btot; p.alpha = d.alpha;
  p.debug = d.debug_checks;
  if (cudaFuncSetAttribute(two_stage_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) !=
      cudaSuccess) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(heads * cs));
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = (unsigned)cs;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, two_stage_cluster_kernel, p) != cudaSuccess) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  *launches += 1;
  return cudaSuccess;
}

}  // namespace ckv
