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
