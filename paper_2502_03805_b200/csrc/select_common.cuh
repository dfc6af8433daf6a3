// Device-side pieces shared by the selection kernels (steps 3-4): order-preserving integer keys, the 8-bit radix
// select over a key array in global memory, and the ordered walk that resolves ties by index.
#pragma once
#include <stdint.h>

#include "ckv_internal.h"

namespace ckv {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Group scores of entry i of KV head g in slice b (Algorithm 1: attention and perturbation-aware score of a KV group):
// a = mean_h attn_h, c = mean_h (attn_h + eps) * vnorm_h over the group's query heads (group_sum: c = (a + eps) * the
// one norm of the KV head), every operation a separately rounded float32 op in this fixed order: the selection is
// decided in exactly this arithmetic by every kernel.
struct GroupScoreArgs {
  const float* attn;
  const float* vnorm;
  const int32_t* valid_from;   // [nb, Hkv] or null
  int Hq, Hkv, G, n;
  float eps;
  int group_sum;
  int protect_from;            // entries >= protect_from are raised to the largest float32 (n when nothing is protected)
};
inline GroupScoreArgs group_score_args(const Dims& d, const float* attn, const float* vnorm) {
  GroupScoreArgs p;
  p.attn = attn; p.vnorm = vnorm; p.valid_from = d.valid_from;
  p.Hq = d.Hq; p.Hkv = d.Hkv; p.G = d.G; p.n = d.n; p.eps = d.eps; p.group_sum = d.group_sum;
  p.protect_from = d.protect_window ? d.n - d.w : d.n;
  return p;
}
__device__ __forceinline__ void group_scores_of(const GroupScoreArgs& p, int b, int g, int i, float* a_out,
                                                float* c_out) {
  const long long n = p.n;
  const long long h0 = (long long)b * p.Hq + (long long)g * p.G;
  const float Gf = (float)p.G;
  float av, cv;
  if (p.group_sum) {
    float sa = p.attn[h0 * n + i];
    for (int q = 1; q < p.G; ++q) sa = __fadd_rn(sa, p.attn[(h0 + q) * n + i]);
    av = __fdiv_rn(sa, Gf);
    cv = __fmul_rn(__fadd_rn(av, p.eps), p.vnorm[((long long)b * p.Hkv + g) * n + i]);
  } else {
    float x = p.attn[h0 * n + i];
    float sa = x;
    float sc = __fmul_rn(__fadd_rn(x, p.eps), p.vnorm[h0 * n + i]);
    for (int q = 1; q < p.G; ++q) {
      x = p.attn[(h0 + q) * n + i];
      sa = __fadd_rn(sa, x);
      sc = __fadd_rn(sc, __fmul_rn(__fadd_rn(x, p.eps), p.vnorm[(h0 + q) * n + i]));
    }
    av = __fdiv_rn(sa, Gf);
    cv = __fdiv_rn(sc, Gf);
  }
  if (i >= p.protect_from) av = cv = 3.402823466e+38f;  // protected observation window: largest float32
  // padding in front of a right-aligned head: below every real score (those are >= 0), so it is taken last
  if (p.valid_from != nullptr && i < p.valid_from[b * p.Hkv + g]) av = cv = -1.0f;
  if (av == 0.f) av = 0.f;  // -0 and +0 must order alike
  if (cv == 0.f) cv = 0.f;
  *a_out = av;
  *c_out = cv;
}

struct SelectShared {
  uint32_t hist[kSelWarps][256];
  uint32_t total[256];
  uint32_t warp_cnt[kSelWarps];
  uint32_t prefix;
  uint32_t krem;
};

__device__ __forceinline__ bool excluded(const uint32_t* excl, long long i) {
  return excl != nullptr && ((excl[i >> 5] >> (i & 31)) & 1u);
}

// Applies f(index, value) to keys[0 .. count) with the CTA's threads striding over the array; eight independent loads
// are issued before any of them is used, so the walk is not serialised on memory latency.
template <typename F>
__device__ __forceinline__ void scan_keys(const float* __restrict__ keys, long long count, F&& f) {
  long long i = threadIdx.x;
  for (; i + 7LL * kSelThreads < count; i += 8LL * kSelThreads) {
    float v[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = keys[i + (long long)q * kSelThreads];
#pragma unroll
    for (int q = 0; q < 8; ++q) f(i + (long long)q * kSelThreads, v[q]);
  }
  for (; i < count; i += kSelThreads) f(i, keys[i]);
}

// Finds the k-th largest key among the candidates (all i in [0, count) not excluded), 1 <= k <= #candidates.
// On return (all threads): *T = that key, *r = how many entries equal to T belong to the top k.
__device__ void radix_select(const float* __restrict__ keys, long long count, const uint32_t* excl, uint32_t k,
                             SelectShared& sh, uint32_t* T, uint32_t* r) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { sh.prefix = 0; sh.krem = k; }
  uint32_t known = 0;  // mask of the key bits fixed so far
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int e = tid; e < kSelWarps * 256; e += kSelThreads) (&sh.hist[0][0])[e] = 0;
    __syncthreads();
    const uint32_t prefix = sh.prefix;
    scan_keys(keys, count, [&](long long i, float x) {
      if (excluded(excl, i)) return;
      const uint32_t key = order_key(x);
      if ((key & known) == prefix) atomicAdd(&sh.hist[warp][(key >> shift) & 255u], 1u);
    });
    __syncthreads();
    if (tid < 256) {
      uint32_t s = 0;
      for (int wq = 0; wq < kSelWarps; ++wq) s += sh.hist[wq][tid];
      sh.total[tid] = s;
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns digits 8l .. 8l+7; find the digit at which the count from the top reaches krem
      uint32_t mine = 0;
      for (int q = 0; q < 8; ++q) mine += sh.total[lane * 8 + q];
      uint32_t above = mine;  // inclusive suffix sum over lanes >= lane
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, above, o);
        if (lane + o < 32) above += v;
      }
      above -= mine;  // keys in strictly higher lanes
      const uint32_t krem = sh.krem;
      if (above < krem && krem <= above + mine) {
        uint32_t acc = above;
        for (int q = 7; q >= 0; --q) {
          const uint32_t cnt = sh.total[lane * 8 + q];
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
    __syncthreads();
  }
  *T = sh.prefix;
  *r = sh.krem;
  __syncthreads();
}

// Ordered walk over [0, n): sets bit i of out[] iff key_i > T, or key_i == T and fewer than r equal candidates
// precede i.  Warp q owns the contiguous word range [q * wpw, (q + 1) * wpw).
__device__ void mark_selected(const float* __restrict__ keys, int n, const uint32_t* excl, uint32_t T, uint32_t r,
                              bool any, uint32_t* out, SelectShared& sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nwords = (n + 31) / 32;
  const int wpw = (nwords + kSelWarps - 1) / kSelWarps;
  const int w0 = min(warp * wpw, nwords), w1 = min(w0 + wpw, nwords);
  uint32_t eq_count = 0;
  for (int q0 = w0; q0 < w1; q0 += 4) {
    float x[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {   // independent loads first
      const int i = (q0 + u) * 32 + lane;
      x[u] = (any && q0 + u < w1 && i < n) ? keys[i] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = (q0 + u) * 32 + lane;
      const bool valid = any && q0 + u < w1 && i < n && !excluded(excl, i);
      eq_count += __popc(__ballot_sync(0xffffffffu, valid && order_key(x[u]) == T));
    }
  }
  if (lane == 0) sh.warp_cnt[warp] = eq_count;
  __syncthreads();
  uint32_t running = 0;
  for (int q = 0; q < warp; ++q) running += sh.warp_cnt[q];
  for (int q0 = w0; q0 < w1; q0 += 4) {
    float x[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = (q0 + u) * 32 + lane;
      x[u] = (any && q0 + u < w1 && i < n) ? keys[i] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int q = q0 + u;
      if (q >= w1) break;   // uniform across the warp
      const int i = q * 32 + lane;
      const bool valid = any && i < n && !excluded(excl, i);
      const uint32_t key = valid ? order_key(x[u]) : 0u;
      const bool eq = valid && key == T;
      const uint32_t eqm = __ballot_sync(0xffffffffu, eq);
      const bool take = eq && (running + __popc(eqm & ((1u << lane) - 1u)) < r);
      const uint32_t word = __ballot_sync(0xffffffffu, (valid && key > T) || take);
      if (lane == 0) out[q] = word;
      running += __popc(eqm);
    }
  }
  __syncthreads();
}

}  // namespace
}  // namespace ckv
