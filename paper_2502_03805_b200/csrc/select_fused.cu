// Steps 3-4 in ONE kernel (Algorithm 1: scores, b' = floor(alpha b), stage 1 by attention, stage 2 by the
// perturbation-aware score among the rest; Algorithm 2: budget allocation across the heads of a layer).
//
// A CTA works on one (nb slice, KV head) at a time; attn and vnorm cross HBM exactly once:
//   reduce   : a_g, c_g from the group's query heads in the fixed float32 operation order of the selection (see
//              select.cu), turned into order-preserving integer keys and written to a scratch array in a
//              word-transposed layout (entry i = 32 t + j lives at [j][t]), so that later walks give every thread
//              whole 32-entry words with coalesced loads; the 12-bit first-digit histogram of a_g is built on the way
//   budgets  : flattened adaptive allocation over the KV heads of a slice, i.e. over several CTAs: three radix rounds
//              (12 + 10 + 10 bits) whose histograms are summed in a small per-slice block of global memory; the CTAs
//              of a slice meet at four bounded barriers (the launch is cooperative, so all of them are resident)
//   stage 1  : the first round is the histogram already built; the second walks the keys once, also collecting the
//              keys of the threshold bin; the third runs on that short list; an ordered marking walk (ties to the
//              lower index) writes the stage-1 bit mask and builds the first-digit histogram of c over the entries
//              stage 1 leaves
//   stage 2  : one walk over c marks the entries above the threshold bin and collects the entries inside it; the
//              remaining digits and the index tie-break run on the list
//   output   : ordered compaction of the two bit masks into ascending indices
// The scratch arrays are re-read from L2 (a up to four times, c twice); two CTAs share an SM.  Every decision is taken
// on the same integer keys and with the same tie rule as the multi-kernel path: both give identical results.  Scores
// must not be NaN (the padding of the last word uses the key 0, which only a NaN bit pattern maps to).
#include "ckv_internal.h"
#include "select_common.cuh"
#include "sm100_ptx.cuh"

namespace ckv {
namespace {

constexpr int kFT = 512;                       // threads per CTA
constexpr int kFW = kFT / 32;
constexpr int kD1Shift = 20, kD1Bins = 4096;   // first digit: sign, exponent and 3 mantissa bits
constexpr int kD2Bins = 1024;                  // second and third digit: 10 bits each
constexpr int kCandCap = 2048;                 // keys of a threshold bin kept in shared memory
constexpr int kMaxWords = kD1Bins;             // 32-entry words per head (n <= 131072)
constexpr int kMaxHeads = 64;

// Per nb slice, zeroed before the launch (adaptive budgets only).
struct LayerSync {
  uint32_t hist1[kD1Bins];
  uint32_t hist2[kD2Bins];
  uint32_t hist3[kD2Bins];
  uint32_t cnt[kMaxHeads][2];   // keys above / equal to the flattened threshold per KV head
  uint32_t arrive[4];           // one counter per barrier
  uint32_t pad[28];
};
static_assert(sizeof(LayerSync) % 16 == 0, "slices of the sync block stay 16-byte aligned");

struct FusedArgs {
  const float* attn;
  const float* vnorm;
  const int32_t* budgets_in;   // given budgets [nb, Hkv] or null
  uint32_t* a_t;               // scratch: keys of a, [nb*Hkv][32][nw]
  uint32_t* c_t;               // scratch: keys of c, same layout
  LayerSync* sync;             // [nb] (adaptive only)
  int32_t* budgets_out;        // [nb, Hkv]: the budgets used (adaptive mode), may be null
  int32_t* idx;
  int32_t* offsets;
  uint8_t* stage;
  int* status;
  const int32_t* valid_from;
  int Hq, Hkv, G, n, nw;       // nw: words per head, even
  int group_sum, protect_from;
  int debug;                   // CKV_FLAG_DEBUG_CHECKS: report a skipped write
  long long nitems;
  long long uniform_b, btot, b_adapt;
  int floor_b;
  float alpha, eps;
};

struct FusedShared {
  uint32_t hist_a[kD1Bins];    // first-digit histogram of a; afterwards scratch (tie prefixes of the stage-2 walk)
  uint32_t hist_w[kD1Bins];    // working histogram
  uint32_t cand_key[kCandCap];
  uint32_t cand_idx[kCandCap];
  uint32_t cand_c[kCandCap];   // stage 1: the c key of every candidate
  uint32_t wtot[kFW];
  uint32_t res_bin, res_k, cand_count, flag;
  uint32_t red[4];
};

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Bin of the k-th largest key in a histogram spread over the CTA: thread t holds bins t*PER .. t*PER+PER-1 (higher
// bin = larger key).  Returns the bin and k minus the keys in higher bins (all threads).
template <int PER>
__device__ __forceinline__ void find_bin(const uint32_t (&v)[PER], uint32_t k, FusedShared& sh, uint32_t* bin,
                                         uint32_t* krem) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t s = 0;
#pragma unroll
  for (int q = 0; q < PER; ++q) s += v[q];
  uint32_t x = s;   // inclusive suffix sum over the lanes >= lane
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_down_sync(0xffffffffu, x, o);
    if (lane + o < 32) x += y;
  }
  if (lane == 0) sh.wtot[warp] = x;
  __syncthreads();
  // the result words are written only between the two barriers: a thread that is still reading the previous call's
  // result has not reached the first one yet
  uint32_t above = x - s;
  for (int q = warp + 1; q < kFW; ++q) above += sh.wtot[q];
  if (tid == 0 && (k == 0 || k > above + s)) {   // thread 0 sees the total: k outside the histogram
    sh.res_bin = 0;
    sh.res_k = 0;
  }
  if (s > 0 && above < k && k <= above + s) {
    uint32_t acc = above;
#pragma unroll
    for (int q = PER - 1; q >= 0; --q) {
      if (acc + v[q] >= k) {
        sh.res_bin = (uint32_t)(tid * PER + q);
        sh.res_k = k - acc;
        break;
      }
      acc += v[q];
    }
  }
  __syncthreads();
  *bin = sh.res_bin;
  *krem = sh.res_k;
}
// The same over a histogram in shared memory.
__device__ __forceinline__ void find_bin_d1(const uint32_t* hist, uint32_t k, FusedShared& sh, uint32_t* bin,
                                            uint32_t* krem) {
  uint32_t v[8];
  const uint4 x = *reinterpret_cast<const uint4*>(hist + 8 * threadIdx.x);
  const uint4 y = *reinterpret_cast<const uint4*>(hist + 8 * threadIdx.x + 4);
  v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w; v[4] = y.x; v[5] = y.y; v[6] = y.z; v[7] = y.w;
  find_bin<8>(v, k, sh, bin, krem);
}
__device__ __forceinline__ void find_bin_d2(const uint32_t* hist, uint32_t k, FusedShared& sh, uint32_t* bin,
                                            uint32_t* krem) {
  uint32_t v[2] = {hist[2 * threadIdx.x], hist[2 * threadIdx.x + 1]};
  find_bin<2>(v, k, sh, bin, krem);
}

// Exclusive prefix of v over the threads of the CTA (thread order) and the CTA-wide total.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, FusedShared& sh, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) sh.wtot[warp] = x;
  __syncthreads();
  uint32_t before = 0, all = 0;
  for (int q = 0; q < kFW; ++q) {
    const uint32_t w = sh.wtot[q];
    if (q < warp) before += w;
    all += w;
  }
  __syncthreads();
  *total = all;
  return before + x - v;
}
__device__ __forceinline__ uint32_t block_sum(uint32_t v, FusedShared& sh) {
  uint32_t total;
  (void)block_excl_scan(v, sh, &total);
  return total;
}

__device__ __forceinline__ void zero_words(uint32_t* p, int count) {
  for (int e = threadIdx.x; e < count; e += kFT) p[e] = 0;
}

// The CTAs that work on the heads of one slice meet here.  Bounded: gives up after two seconds (false).
__device__ __forceinline__ bool layer_barrier(uint32_t* counter, uint32_t target, FusedShared& sh) {
  __syncthreads();   // every thread's writes and reductions to the slice's block are issued
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(counter, 1u);
    bool ok = true;
    if (ld_acquire(counter) < target) {
      const uint64_t t0 = ptx::global_timer_ns();
      for (uint32_t spin = 1;; ++spin) {
        if (ld_acquire(counter) >= target) break;
        if ((spin & 63u) == 0 && ptx::global_timer_ns() - t0 > 2000000000ull) {
          ok = false;
          break;
        }
      }
    }
    __threadfence();
    sh.flag = ok ? 1u : 0u;
  }
  __syncthreads();
  return sh.flag != 0;
}

// One entry of the group reduce: the sums over the group's heads are finished into (a, c), the special scores of the
// protected window and of the padding are applied, and -0 is folded into +0.
__device__ __forceinline__ void finish_entry(float sa, float sc, float Gf, float invG, bool pow2, float eps,
                                             int group_sum, float vg, int i, int protect_from, int vf,
                                             uint32_t* ka, uint32_t* kc) {
  // dividing by a power of two and multiplying by its reciprocal round the same exact value
  float av = pow2 ? __fmul_rn(sa, invG) : __fdiv_rn(sa, Gf);
  float cv = group_sum ? __fmul_rn(__fadd_rn(av, eps), vg) : (pow2 ? __fmul_rn(sc, invG) : __fdiv_rn(sc, Gf));
  if (i >= protect_from) av = cv = 3.402823466e+38f;
  if (i < vf) av = cv = -1.0f;
  if (av == 0.f) av = 0.f;
  if (cv == 0.f) cv = 0.f;
  *ka = order_key(av);
  *kc = order_key(cv);
}

// Four consecutive keys into a first-digit histogram: neighbours mostly share a bin (the scores are max-pooled), one
// atomic per run.  (Adding up the counts of the lanes of a warp that share a bin first, with a warp match, was
// measured slower.)
__device__ __forceinline__ void count_digits4(uint32_t* hist, const uint32_t (&k)[4]) {
  uint32_t cur = k[0] >> kD1Shift, run = 1;
#pragma unroll
  for (int j = 1; j < 4; ++j) {
    const uint32_t bin = k[j] >> kD1Shift;
    if (bin == cur) {
      ++run;
    } else {
      atomicAdd(&hist[cur], run);
      cur = bin;
      run = 1;
    }
  }
  atomicAdd(&hist[cur], run);
}

// Applies f(key0, key1, j) to the entries j = 0..31 of the word pair (2 wp, 2 wp + 1); eight loads in flight.
template <typename F>
__device__ __forceinline__ void walk_pair(const uint32_t* __restrict__ arr, int nw, int wp, F&& f) {
  const uint2* p = reinterpret_cast<const uint2*>(arr) + wp;
  const size_t row = (size_t)(nw >> 1);
#pragma unroll 1
  for (int j0 = 0; j0 < 32; j0 += 8) {
    uint2 k[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) k[u] = __ldcg(p + (size_t)(j0 + u) * row);
#pragma unroll
    for (int u = 0; u < 8; ++u) f(k[u].x, k[u].y, j0 + u);
  }
}
template <typename F>
__device__ __forceinline__ void walk_pair2(const uint32_t* __restrict__ arr_a, const uint32_t* __restrict__ arr_b,
                                           int nw, int wp, F&& f) {
  const uint2* pa = reinterpret_cast<const uint2*>(arr_a) + wp;
  const uint2* pb = reinterpret_cast<const uint2*>(arr_b) + wp;
  const size_t row = (size_t)(nw >> 1);
#pragma unroll 1
  for (int j0 = 0; j0 < 32; j0 += 4) {
    uint2 ka[4], kb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      ka[u] = __ldcg(pa + (size_t)(j0 + u) * row);
      kb[u] = __ldcg(pb + (size_t)(j0 + u) * row);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) f(ka[u].x, ka[u].y, kb[u].x, kb[u].y, j0 + u);
  }
}

// Second and third radix round over the keys of `arr` (entries excluded by `excl` skipped) whose first digit is bin1;
// the first round's result (bin1, krem) comes from a histogram the caller already has.  With kSync the histograms of
// the rounds are summed over the CTAs of the slice (barriers arrive[1], arrive[2]).  Returns the threshold key T, how
// many of the keys equal to T belong to the top k (r), how many keys equal T in this CTA's array (own_eq), and adds
// this CTA's keys in higher bins of rounds two and three to *own_gt.  Uses cand_key as list.  false = a barrier
// timed out.
template <bool kExcl, bool kSync>
__device__ __forceinline__ bool refine_threshold(const uint32_t* __restrict__ arr, int nw, const uint32_t* excl,
                                                 uint32_t bin1, uint32_t krem, LayerSync* ls, uint32_t target,
                                                 FusedShared& sh, uint32_t* T, uint32_t* r, uint32_t* own_eq,
                                                 uint32_t* own_gt) {
  const int tid = threadIdx.x;
  zero_words(sh.hist_w, kD2Bins);
  if (tid == 0) sh.cand_count = 0;
  __syncthreads();
  for (int wp = tid; wp < (nw >> 1); wp += kFT) {
    uint32_t e0 = 0, e1 = 0;
    if (kExcl) { e0 = excl[2 * wp]; e1 = excl[2 * wp + 1]; }
    // candidate masks first (no divergence inside the walk), then the few candidates one by one
    uint32_t c0 = 0, c1 = 0;
    walk_pair(arr, nw, wp, [&](uint32_t k0, uint32_t k1, int j) {
      c0 |= (uint32_t)((k0 >> kD1Shift) == bin1) << j;
      c1 |= (uint32_t)((k1 >> kD1Shift) == bin1) << j;
    });
    c0 &= ~e0;
    c1 &= ~e1;
    for (int half = 0; half < 2; ++half) {
      uint32_t cm = half ? c1 : c0;
      while (cm) {
        const int j = __ffs(cm) - 1;
        cm &= cm - 1;
        const uint32_t key = __ldcg(arr + (size_t)j * nw + 2 * wp + half);
        atomicAdd(&sh.hist_w[(key >> 10) & (kD2Bins - 1)], 1u);
        const uint32_t slot = atomicAdd(&sh.cand_count, 1u);
        if (slot < (uint32_t)kCandCap) sh.cand_key[slot] = key;
      }
    }
  }
  __syncthreads();
  const uint32_t ncand = sh.cand_count;
  uint32_t prefix = bin1;
  uint32_t gt = 0;
  for (int round = 0; round < 2; ++round) {
    if (round == 1) {
      zero_words(sh.hist_w, kD2Bins);
      __syncthreads();
      if (ncand <= (uint32_t)kCandCap) {
        for (uint32_t e = tid; e < ncand; e += kFT) {
          const uint32_t key = sh.cand_key[e];
          if ((key >> 10) == prefix) atomicAdd(&sh.hist_w[key & (kD2Bins - 1)], 1u);
        }
      } else {
        for (int wp = tid; wp < (nw >> 1); wp += kFT) {
          uint32_t e0 = 0, e1 = 0;
          if (kExcl) { e0 = excl[2 * wp]; e1 = excl[2 * wp + 1]; }
          walk_pair(arr, nw, wp, [&](uint32_t k0, uint32_t k1, int j) {
            if ((k0 >> 10) == prefix && !((e0 >> j) & 1u)) atomicAdd(&sh.hist_w[k0 & (kD2Bins - 1)], 1u);
            if ((k1 >> 10) == prefix && !((e1 >> j) & 1u)) atomicAdd(&sh.hist_w[k1 & (kD2Bins - 1)], 1u);
          });
        }
      }
      __syncthreads();
    }
    const uint32_t own[2] = {sh.hist_w[2 * tid], sh.hist_w[2 * tid + 1]};
    uint32_t v[2] = {own[0], own[1]};
    if (kSync) {
      uint32_t* gh = round == 0 ? ls->hist2 : ls->hist3;
      if (own[0]) atomicAdd(&gh[2 * tid], own[0]);
      if (own[1]) atomicAdd(&gh[2 * tid + 1], own[1]);
      if (!layer_barrier(&ls->arrive[1 + round], target, sh)) return false;
      const uint2 x = __ldcg(reinterpret_cast<const uint2*>(gh) + tid);
      v[0] = x.x;
      v[1] = x.y;
    }
    uint32_t bin;
    find_bin<2>(v, krem, sh, &bin, &krem);
    if ((uint32_t)(2 * tid) > bin) gt += own[0];
    if ((uint32_t)(2 * tid + 1) > bin) gt += own[1];
    if (round == 1 && (uint32_t)tid == (bin >> 1)) sh.red[2] = own[bin & 1u];
    prefix = (prefix << 10) | bin;
  }
  __syncthreads();
  *T = prefix;
  *r = krem;
  *own_eq = sh.red[2];
  *own_gt += gt;
  return true;
}

// Ordered marking walk over the keys of `arr`: bit (t, j) of out is set iff the entry is not excluded and its key is
// above T, or equal to T with fewer than r equal (not excluded) entries before it.  `ties` = number of such equal
// entries; when all of them are taken no ordering is needed.  With kHist the first digit of `other`'s key of every
// entry left unmarked is counted in hist.  tmp: nw words of scratch.
template <bool kExcl, bool kHist>
__device__ __forceinline__ void mark_walk(const uint32_t* __restrict__ arr, const uint32_t* __restrict__ other, int nw,
                                          const uint32_t* excl, bool any, uint32_t T, uint32_t r, uint32_t ties,
                                          uint32_t* out, uint32_t* tmp, uint32_t* hist, FusedShared& sh) {
  const int tid = threadIdx.x;
  const bool ordered = any && r < ties;
  if (ordered) {
    uint32_t carry = 0;
    for (int base = 0; base < (nw >> 1); base += kFT) {
      const int wp = base + tid;
      uint32_t q0 = 0, q1 = 0;
      if (wp < (nw >> 1)) {
        uint32_t e0 = 0, e1 = 0;
        if (kExcl) { e0 = excl[2 * wp]; e1 = excl[2 * wp + 1]; }
        walk_pair(arr, nw, wp, [&](uint32_t k0, uint32_t k1, int j) {
          q0 += (k0 == T) & !((e0 >> j) & 1u);
          q1 += (k1 == T) & !((e1 >> j) & 1u);
        });
      }
      uint32_t total;
      const uint32_t before = carry + block_excl_scan(q0 + q1, sh, &total);
      if (wp < (nw >> 1)) {
        tmp[2 * wp] = before;
        tmp[2 * wp + 1] = before + q0;
      }
      carry += total;
    }
    __syncthreads();
  }
  for (int wp = tid; wp < (nw >> 1); wp += kFT) {
    uint32_t e0 = 0, e1 = 0;
    if (kExcl) { e0 = excl[2 * wp]; e1 = excl[2 * wp + 1]; }
    uint32_t run0 = 0, run1 = 0;
    if (ordered) { run0 = tmp[2 * wp]; run1 = tmp[2 * wp + 1]; }
    uint32_t w0 = 0, w1 = 0;
    auto decide = [&](uint32_t key, uint32_t e, int j, uint32_t& run) -> uint32_t {
      const uint32_t free_ = !((e >> j) & 1u);
      const uint32_t eq = (key == T) & free_;
      const uint32_t take = ordered ? (eq & (run < r)) : eq;
      run += eq;
      return any ? (((key > T) & free_) | take) : 0u;
    };
    if (kHist) {
      walk_pair2(arr, other, nw, wp, [&](uint32_t k0, uint32_t k1, uint32_t o0, uint32_t o1, int j) {
        const uint32_t m0 = decide(k0, e0, j, run0), m1 = decide(k1, e1, j, run1);
        w0 |= m0 << j;
        w1 |= m1 << j;
        if (!m0) atomicAdd(&hist[o0 >> kD1Shift], 1u);
        if (!m1) atomicAdd(&hist[o1 >> kD1Shift], 1u);
      });
    } else {
      walk_pair(arr, nw, wp, [&](uint32_t k0, uint32_t k1, int j) {
        w0 |= decide(k0, e0, j, run0) << j;
        w1 |= decide(k1, e1, j, run1) << j;
      });
    }
    out[2 * wp] = w0;
    out[2 * wp + 1] = w1;
  }
  __syncthreads();
}

// Finishes a selection on a list of candidates that all share the first digit: `hist2` holds the histogram of their
// second digit (bits 19..10), k = how many of them belong to the selection.  Returns the threshold key T and the
// index limit for the ties: a candidate is selected iff key > T, or key == T and 0xfffff - index >= tie_limit (the
// lowest indices win).  scratch: kD2Bins words that may alias hist2.
__device__ __forceinline__ void finish_on_list(const uint32_t* list_key, const uint32_t* list_idx, uint32_t ncand,
                                               uint32_t bin1, uint32_t* hist2, uint32_t k, uint32_t* scratch,
                                               FusedShared& sh, uint32_t* T_out, uint32_t* tie_limit_out) {
  const int tid = threadIdx.x;
  uint32_t bin2, bin3, krem;
  find_bin_d2(hist2, k, sh, &bin2, &krem);
  const uint32_t prefix22 = (bin1 << 10) | bin2;
  zero_words(scratch, kD2Bins);
  __syncthreads();
  for (uint32_t e = tid; e < ncand; e += kFT) {
    const uint32_t key = list_key[e];
    if ((key >> 10) == prefix22) atomicAdd(&scratch[key & (kD2Bins - 1)], 1u);
  }
  __syncthreads();
  find_bin_d2(scratch, krem, sh, &bin3, &krem);
  const uint32_t T = (prefix22 << 10) | bin3;
  const uint32_t r = krem, ties = scratch[bin3];
  __syncthreads();
  uint32_t tie_limit = 0;
  if (r < ties) {
    // the r lowest indices among the ties: two more rounds over the 20-bit key (0xfffff - index)
    uint32_t pre = 0, kk = r;
    for (int round = 0; round < 2; ++round) {
      const int shift = round == 0 ? 10 : 0;
      zero_words(scratch, kD2Bins);
      __syncthreads();
      for (uint32_t e = tid; e < ncand; e += kFT) {
        if (list_key[e] != T) continue;
        const uint32_t ik = 0xfffffu - list_idx[e];
        if (round == 0 || (ik >> 10) == pre) atomicAdd(&scratch[(ik >> shift) & (kD2Bins - 1)], 1u);
      }
      __syncthreads();
      uint32_t binx;
      find_bin_d2(scratch, kk, sh, &binx, &kk);
      pre = (pre << 10) | binx;
    }
    tie_limit = pre;
  }
  *T_out = T;
  *tie_limit_out = tie_limit;
}

template <bool kAdaptive>
__global__ void __launch_bounds__(kFT, 2) select_fused_kernel(FusedArgs p) {
  extern __shared__ __align__(16) uint8_t fused_smem[];
  FusedShared& sh = *reinterpret_cast<FusedShared*>(fused_smem);
  const int n = p.n, nw = p.nw;
  uint32_t* sel1 = reinterpret_cast<uint32_t*>(fused_smem + ((sizeof(FusedShared) + 15) / 16) * 16);
  uint32_t* sel2 = sel1 + nw;
  const int tid = threadIdx.x;
  const int G = p.G;
  const float Gf = (float)G, invG = 1.0f / Gf;
  const bool pow2 = (G & (G - 1)) == 0;
  const size_t head_words = (size_t)32 * nw;

  for (long long item = blockIdx.x; item < p.nitems; item += gridDim.x) {
    const int b = (int)(item / p.Hkv), g = (int)(item % p.Hkv);
    const long long h0 = (long long)b * p.Hq + (long long)g * G;
    const int vf = p.valid_from ? p.valid_from[b * p.Hkv + g] : 0;
    uint32_t* a_t = p.a_t + (size_t)item * head_words;
    uint32_t* c_t = p.c_t + (size_t)item * head_words;
    LayerSync* ls = kAdaptive ? p.sync + b : nullptr;

    __syncthreads();   // the previous item's shared state is no longer read
    zero_words(sh.hist_a, kD1Bins);
    __syncthreads();

    // ---------------- reduce: one pass over attn and vnorm ----------------
    const float* vg_row = p.group_sum ? p.vnorm + ((long long)b * p.Hkv + g) * n : nullptr;
    if ((n & 3) == 0) {
      const int n4 = n >> 2;
      for (int i4 = tid; i4 < n4; i4 += kFT) {
        const int word = i4 >> 3, quad = i4 & 7;
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int q0 = 0; q0 < G; q0 += 4) {
          float4 pa[4], pv[4];
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            if (q0 + v < G) {
              pa[v] = __ldcs(reinterpret_cast<const float4*>(p.attn + (h0 + q0 + v) * n) + i4);
              if (!p.group_sum) pv[v] = __ldcs(reinterpret_cast<const float4*>(p.vnorm + (h0 + q0 + v) * n) + i4);
            }
          }
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            if (q0 + v < G) {
              const float a4[4] = {pa[v].x, pa[v].y, pa[v].z, pa[v].w};
              float v4[4] = {0.f, 0.f, 0.f, 0.f};
              if (!p.group_sum) { v4[0] = pv[v].x; v4[1] = pv[v].y; v4[2] = pv[v].z; v4[3] = pv[v].w; }
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float prod = __fmul_rn(__fadd_rn(a4[j], p.eps), v4[j]);
                if (q0 + v == 0) { sa[j] = a4[j]; sc[j] = prod; }
                else { sa[j] = __fadd_rn(sa[j], a4[j]); sc[j] = __fadd_rn(sc[j], prod); }
              }
            }
          }
        }
        float4 vg4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.group_sum) vg4 = __ldcs(reinterpret_cast<const float4*>(vg_row) + i4);
        const float vgs[4] = {vg4.x, vg4.y, vg4.z, vg4.w};
        uint32_t ka[4], kc[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          finish_entry(sa[j], sc[j], Gf, invG, pow2, p.eps, p.group_sum, vgs[j], 4 * i4 + j, p.protect_from, vf,
                       &ka[j], &kc[j]);
          a_t[(size_t)(4 * quad + j) * nw + word] = ka[j];
          c_t[(size_t)(4 * quad + j) * nw + word] = kc[j];
        }
        count_digits4(sh.hist_a, ka);
      }
    } else {
      for (int i = tid; i < n; i += kFT) {
        float sa = 0.f, sc = 0.f;
        for (int q = 0; q < G; ++q) {
          const float a1 = p.attn[(h0 + q) * n + i];
          const float v1 = p.group_sum ? 0.f : p.vnorm[(h0 + q) * n + i];
          const float prod = __fmul_rn(__fadd_rn(a1, p.eps), v1);
          if (q == 0) { sa = a1; sc = prod; }
          else { sa = __fadd_rn(sa, a1); sc = __fadd_rn(sc, prod); }
        }
        uint32_t ka, kc;
        finish_entry(sa, sc, Gf, invG, pow2, p.eps, p.group_sum, p.group_sum ? vg_row[i] : 0.f, i, p.protect_from,
                     vf, &ka, &kc);
        a_t[(size_t)(i & 31) * nw + (i >> 5)] = ka;
        c_t[(size_t)(i & 31) * nw + (i >> 5)] = kc;
        atomicAdd(&sh.hist_a[ka >> kD1Shift], 1u);
      }
    }
    // the tail of the last word and the padding words: key 0, below every real key
    for (int i = n + tid; i < 32 * nw; i += kFT) {
      a_t[(size_t)(i & 31) * nw + (i >> 5)] = 0u;
      c_t[(size_t)(i & 31) * nw + (i >> 5)] = 0u;
    }
    __syncthreads();

    // ---------------- this head's budget and the start of its segment ----------------
    long long off = 0, bud = 0;
    bool clipped = false, failed = false;
    if (kAdaptive) {
      if (p.b_adapt > 0) {
        // flattened top-b_adapt over the keys of every head of the slice
        const uint32_t Hkv = (uint32_t)p.Hkv;
        for (int e = tid; e < kD1Bins; e += kFT) {
          const uint32_t v = sh.hist_a[e];
          if (v) atomicAdd(&ls->hist1[e], v);
        }
        failed = !layer_barrier(&ls->arrive[0], Hkv, sh);
        uint32_t T = 0, r = 0, own_eq = 0, own_gt = 0;
        if (!failed) {
          uint32_t v[8];
          const uint4 x = __ldcg(reinterpret_cast<const uint4*>(ls->hist1) + 2 * tid);
          const uint4 y = __ldcg(reinterpret_cast<const uint4*>(ls->hist1) + 2 * tid + 1);
          v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w; v[4] = y.x; v[5] = y.y; v[6] = y.z; v[7] = y.w;
          uint32_t bin1, krem1;
          find_bin<8>(v, (uint32_t)p.b_adapt, sh, &bin1, &krem1);
#pragma unroll
          for (int q = 0; q < 8; ++q)
            if ((uint32_t)(8 * tid + q) > bin1) own_gt += sh.hist_a[8 * tid + q];
          failed = !refine_threshold<false, true>(a_t, nw, nullptr, bin1, krem1, ls, Hkv, sh, &T, &r, &own_eq,
                                                  &own_gt);
        }
        if (!failed) {
          const uint32_t total = block_sum(own_gt, sh);
          if (tid == 0) {
            ls->cnt[g][0] = total;
            ls->cnt[g][1] = own_eq;
          }
          failed = !layer_barrier(&ls->arrive[3], Hkv, sh);
        }
        if (!failed) {
          uint32_t rem = r;
          for (int q = 0; q <= g; ++q) {
            const uint2 c2 = __ldcg(reinterpret_cast<const uint2*>(&ls->cnt[q][0]));
            const uint32_t take = min(c2.y, rem);
            const long long bq = min((long long)c2.x + take + p.floor_b, (long long)n);
            rem -= take;
            if (q < g) off += bq;
            else bud = bq;
          }
        }
      } else {
        bud = min((long long)p.floor_b, (long long)n);
        off = (long long)g * bud;
      }
      if (off > p.btot) { off = p.btot; clipped = true; }
      if (off + bud > p.btot) { bud = p.btot - off; clipped = true; }
      if (p.budgets_out != nullptr && tid == 0) p.budgets_out[(long long)b * p.Hkv + g] = (int32_t)bud;
    } else if (p.budgets_in == nullptr) {
      bud = p.uniform_b;
      off = (long long)g * bud;
    } else {
      const int32_t* bb = p.budgets_in + (long long)b * p.Hkv;
      for (int q = 0; q < g; ++q) off += min(max((long long)bb[q], 0LL), (long long)n);
      bud = bb[g];
      if (bud < 0 || bud > n) { bud = min(max(bud, 0LL), (long long)n); clipped = true; }
      if (off > p.btot) { off = p.btot; clipped = true; }
      if (off + bud > p.btot) { bud = p.btot - off; clipped = true; }
    }
    if (failed) {   // a barrier ran out: report and stop (the CTAs that wait for this one run out as well)
      if (tid == 0) atomicExch(p.status, (int)CKV_ETIMEOUT);
      break;
    }
    if (clipped && tid == 0) atomicExch(p.status, (int)CKV_EINVAL);
    long long b1 = (long long)floor((double)p.alpha * (double)bud);
    b1 = min(max(b1, 0LL), bud);
    const long long b2 = bud - b1;

    // ---------------- stage 1: the b1 largest a; first digits of c over the entries it leaves ----------------
    // One walk over a and c: entries above the threshold bin of a are taken, entries inside it are collected (their
    // remaining digits and the index tie-break run on the list), and the first digit of c is counted for the entries
    // below it; the candidates that the list rounds reject are counted afterwards.
    uint32_t bin1 = kD1Bins, krem1 = 0;      // b1 == 0: no first digit is above or inside the threshold bin
    if (b1 > 0) find_bin_d1(sh.hist_a, (uint32_t)b1, sh, &bin1, &krem1);
    zero_words(sh.hist_w, kD1Bins);
    zero_words(sh.hist_a, kD2Bins);          // from here on: second-digit histogram of the stage-1 candidates
    if (tid == 0) sh.cand_count = 0;
    __syncthreads();
    for (int wp = tid; wp < (nw >> 1); wp += kFT) {
      uint32_t w0 = 0, w1 = 0, c0 = 0, c1 = 0;
      if (b2 > 0) {
        walk_pair2(a_t, c_t, nw, wp, [&](uint32_t k0, uint32_t k1, uint32_t o0, uint32_t o1, int j) {
          const uint32_t d0 = k0 >> kD1Shift, d1 = k1 >> kD1Shift;
          w0 |= (uint32_t)(d0 > bin1) << j;
          w1 |= (uint32_t)(d1 > bin1) << j;
          c0 |= (uint32_t)(d0 == bin1) << j;
          c1 |= (uint32_t)(d1 == bin1) << j;
          if (d0 < bin1) atomicAdd(&sh.hist_w[o0 >> kD1Shift], 1u);
          if (d1 < bin1) atomicAdd(&sh.hist_w[o1 >> kD1Shift], 1u);
        });
      } else {
        walk_pair(a_t, nw, wp, [&](uint32_t k0, uint32_t k1, int j) {
          const uint32_t d0 = k0 >> kD1Shift, d1 = k1 >> kD1Shift;
          w0 |= (uint32_t)(d0 > bin1) << j;
          w1 |= (uint32_t)(d1 > bin1) << j;
          c0 |= (uint32_t)(d0 == bin1) << j;
          c1 |= (uint32_t)(d1 == bin1) << j;
        });
      }
      sel1[2 * wp] = w0;
      sel1[2 * wp + 1] = w1;
      for (int half = 0; half < 2; ++half) {
        uint32_t cm = half ? c1 : c0;
        while (cm) {
          const int j = __ffs(cm) - 1;
          cm &= cm - 1;
          const size_t at = (size_t)j * nw + 2 * wp + half;
          const uint32_t key = __ldcg(a_t + at);
          atomicAdd(&sh.hist_a[(key >> 10) & (kD2Bins - 1)], 1u);
          const uint32_t slot = atomicAdd(&sh.cand_count, 1u);
          if (slot < (uint32_t)kCandCap) {
            sh.cand_key[slot] = key;
            sh.cand_idx[slot] = (uint32_t)(64 * wp + 32 * half + j);
            sh.cand_c[slot] = b2 > 0 ? __ldcg(c_t + at) : 0u;
          }
        }
      }
    }
    __syncthreads();
    const uint32_t ncand1 = sh.cand_count;
    if (ncand1 > (uint32_t)kCandCap) {
      // the threshold bin of a holds more entries than the list: radix rounds and an ordered walk over the arrays
      uint32_t T1, r1, ties1, unused = 0;
      refine_threshold<false, false>(a_t, nw, nullptr, bin1, krem1, nullptr, 0u, sh, &T1, &r1, &ties1, &unused);
      zero_words(sh.hist_w, kD1Bins);
      __syncthreads();
      if (b2 > 0)
        mark_walk<false, true>(a_t, c_t, nw, nullptr, true, T1, r1, ties1, sel1, sel2, sh.hist_w, sh);
      else
        mark_walk<false, false>(a_t, nullptr, nw, nullptr, true, T1, r1, ties1, sel1, sel2, nullptr, sh);
    } else if (ncand1 > 0) {
      uint32_t T1, tie_limit;
      finish_on_list(sh.cand_key, sh.cand_idx, ncand1, bin1, sh.hist_a, krem1, sh.hist_a, sh, &T1, &tie_limit);
      for (uint32_t e = tid; e < ncand1; e += kFT) {
        const uint32_t key = sh.cand_key[e], i = sh.cand_idx[e];
        if (key > T1 || (key == T1 && 0xfffffu - i >= tie_limit)) atomicOr(&sel1[i >> 5], 1u << (i & 31));
        else if (b2 > 0) atomicAdd(&sh.hist_w[sh.cand_c[e] >> kD1Shift], 1u);
      }
      __syncthreads();
    }
    const uint32_t k2 = (uint32_t)b2;

    // ---------------- stage 2: the b2 largest c among the entries stage 1 left ----------------
    if (b2 > 0) {
      uint32_t bin2, krem2;
      find_bin_d1(sh.hist_w, k2, sh, &bin2, &krem2);
      zero_words(sh.hist_w, kD2Bins);
      if (tid == 0) sh.cand_count = 0;
      __syncthreads();
      // one walk over c: entries above the threshold bin are taken, entries inside it become candidates
      for (int wp = tid; wp < (nw >> 1); wp += kFT) {
        const uint32_t e0 = sel1[2 * wp], e1 = sel1[2 * wp + 1];
        uint32_t w0 = 0, w1 = 0;
        uint32_t c0 = 0, c1 = 0;
        walk_pair(c_t, nw, wp, [&](uint32_t k0, uint32_t k1, int j) {
          const uint32_t dd0 = k0 >> kD1Shift, dd1 = k1 >> kD1Shift;
          w0 |= (uint32_t)(dd0 > bin2) << j;
          w1 |= (uint32_t)(dd1 > bin2) << j;
          c0 |= (uint32_t)(dd0 == bin2) << j;
          c1 |= (uint32_t)(dd1 == bin2) << j;
        });
        w0 &= ~e0;
        w1 &= ~e1;
        c0 &= ~e0;
        c1 &= ~e1;
        for (int half = 0; half < 2; ++half) {
          uint32_t cm = half ? c1 : c0;
          while (cm) {
            const int j = __ffs(cm) - 1;
            cm &= cm - 1;
            const uint32_t key = __ldcg(c_t + (size_t)j * nw + 2 * wp + half);
            atomicAdd(&sh.hist_w[(key >> 10) & (kD2Bins - 1)], 1u);
            const uint32_t slot = atomicAdd(&sh.cand_count, 1u);
            if (slot < (uint32_t)kCandCap) {
              sh.cand_key[slot] = key;
              sh.cand_idx[slot] = (uint32_t)(64 * wp + 32 * half + j);
            }
          }
        }
        sel2[2 * wp] = w0;
        sel2[2 * wp + 1] = w1;
      }
      __syncthreads();
      const uint32_t ncand2 = sh.cand_count;
      if (ncand2 > (uint32_t)kCandCap) {
        // more entries share the threshold bin than the list holds: radix rounds and an ordered walk over all of c
        uint32_t T2, r2, ties2, unused = 0;
        refine_threshold<true, false>(c_t, nw, sel1, bin2, krem2, nullptr, 0u, sh, &T2, &r2, &ties2, &unused);
        mark_walk<true, false>(c_t, nullptr, nw, sel1, true, T2, r2, ties2, sel2, sh.hist_a, nullptr, sh);
      } else {
        uint32_t T2, tie_limit;
        finish_on_list(sh.cand_key, sh.cand_idx, ncand2, bin2, sh.hist_w, krem2, sh.hist_w, sh, &T2, &tie_limit);
        for (uint32_t e = tid; e < ncand2; e += kFT) {
          const uint32_t kc = sh.cand_key[e], i = sh.cand_idx[e];
          if (kc > T2 || (kc == T2 && 0xfffffu - i >= tie_limit)) atomicOr(&sel2[i >> 5], 1u << (i & 31));
        }
        __syncthreads();
      }
    } else {
      for (int q = tid; q < nw; q += kFT) sel2[q] = 0;
      __syncthreads();
    }

    // ---------------- output: ascending indices of sel1 | sel2 ----------------
    int32_t* idx = p.idx + (long long)b * p.btot + off;
    uint8_t* stage = p.stage ? p.stage + (long long)b * p.btot + off : nullptr;
    uint32_t carry = 0;
    for (int base = 0; base < nw; base += kFT) {
      const int q = base + tid;
      const uint32_t s1 = q < nw ? sel1[q] : 0u;
      uint32_t word = q < nw ? (s1 | sel2[q]) : 0u;
      uint32_t total;
      uint32_t pos = carry + block_excl_scan((uint32_t)__popc(word), sh, &total);
      while (word) {
        const int j = __ffs(word) - 1;
        word &= word - 1;
        if ((long long)pos < bud) {   // a selection larger than the budget never writes past the head's segment
          idx[pos] = q * 32 + j;
          if (stage) stage[pos] = ((s1 >> j) & 1u) ? 1 : 2;
        } else if (p.debug) {
          atomicExch(p.status, (int)CKV_EBOUNDS);
        }
        ++pos;
      }
      carry += total;
    }
    if (tid == 0) {
      p.offsets[(long long)b * (p.Hkv + 1) + g] = (int32_t)off;
      if (g == p.Hkv - 1) p.offsets[(long long)b * (p.Hkv + 1) + p.Hkv] = (int32_t)(off + bud);
    }
  }
}

}  // namespace

size_t select_sync_bytes(const Dims& d) {
  return d.budget_mode == CKV_BUDGET_FLAT_ADAPTIVE ? (size_t)d.nb * sizeof(LayerSync) : 0;
}

cudaError_t launch_select_fused(const Dims& d, const float* attn, const float* vnorm, const int32_t* budgets_in,
                                int32_t* idx, int32_t* offsets, uint8_t* stage, const SelectWorkspace& ws,
                                const SelectDevice& dev, cudaStream_t st, int* launches, int* status_word) {
  const bool adaptive = d.budget_mode == CKV_BUDGET_FLAT_ADAPTIVE;
  const int nw = (int)(select_head_stride(d.n) / 32);
  if (nw > kMaxWords || d.Hkv > kMaxHeads) return cudaErrorNotSupported;
  if (adaptive && ws.sync == nullptr) return cudaErrorNotSupported;
  const size_t smem = (sizeof(FusedShared) + 15) / 16 * 16 + (size_t)2 * nw * sizeof(uint32_t);
  if (smem > (size_t)dev.smem_optin) return cudaErrorNotSupported;

  FusedArgs p;
  p.attn = attn; p.vnorm = vnorm;
  p.budgets_in = d.budget_mode == CKV_BUDGET_GIVEN ? budgets_in : nullptr;
  p.a_t = reinterpret_cast<uint32_t*>(ws.a);
  p.c_t = reinterpret_cast<uint32_t*>(ws.c);
  p.sync = adaptive ? reinterpret_cast<LayerSync*>(ws.sync) : nullptr;
  p.budgets_out = adaptive ? ws.budgets : nullptr;
  p.idx = idx; p.offsets = offsets; p.stage = stage; p.status = status_word;
  p.valid_from = d.valid_from;
  p.Hq = d.Hq; p.Hkv = d.Hkv; p.G = d.G; p.n = d.n; p.nw = nw;
  p.group_sum = d.group_sum;
  p.debug = d.debug_checks;
  p.protect_from = d.protect_window ? d.n - d.w : d.n;
  p.nitems = (long long)d.nb * d.Hkv;
  p.uniform_b = d.budget; p.btot = d.btot;
  p.b_adapt = d.budget - (long long)d.Hkv * d.floor_b;
  p.floor_b = (int)d.floor_b;
  p.alpha = d.alpha; p.eps = d.eps;

  auto kernel = adaptive ? select_fused_kernel<true> : select_fused_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  int per_sm = 0;
  if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kFT, smem);
  if (e != cudaSuccess || per_sm < 1) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  // every CTA of the grid is resident (the adaptive allocation waits across CTAs); a slice's heads are handled by
  // neighbouring CTAs of the same round when the grid is a multiple of Hkv
  long long grid = (long long)per_sm * dev.sm_count;
  if (grid > p.nitems) grid = p.nitems;
  if (adaptive) {
    grid -= grid % d.Hkv;
    if (grid < d.Hkv) return cudaErrorNotSupported;
    // histograms and counters of every slice start at zero
    e = cudaMemsetAsync(ws.sync, 0, select_sync_bytes(d), st);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kFT);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeCooperative;
  attr.val.cooperative = adaptive ? 1 : 0;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, kernel, p);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  *launches += 1;
  return cudaSuccess;
}

}  // namespace ckv
