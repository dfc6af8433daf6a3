// Steps 3-4 in ONE kernel for heads whose attention keys fit in shared memory (Algorithm 1: scores, b' = floor(alpha b),
// stage 1 by attention, stage 2 by the perturbation-aware score among the rest; Algorithm 2: budget allocation).
//
// One CTA per (nb slice, KV head).  attn and vnorm are read from memory exactly once:
//   reduce   : a_g, c_g from the group's query heads in the fixed float32 operation order of the selection (see
//              select.cu); the order-preserving integer keys of a_g stay in shared memory, c_g goes to a scratch
//              array that this CTA alone re-reads (twice, from L2); the 12-bit first-digit histogram of a_g is built
//              on the way
//   budgets  : flattened adaptive allocation across the KV heads of a slice = the CTAs of one thread-block cluster:
//              three radix rounds (12 + 10 + 10 bits), histograms summed through distributed shared memory
//   stage 1  : radix select on the shared-memory keys (first round = the histogram already built), ordered marking
//              walk (ties to the lower index) that at the same time builds the first-digit histogram of c over the
//              entries stage 1 left
//   stage 2  : one walk over c marks the entries above the threshold bin and collects the entries inside it; the
//              remaining digits and the index tie-break run on that short list
//   output   : ordered compaction of the two bit masks into ascending indices
// Every decision is taken on the same integer keys and with the same tie rule as the multi-kernel path, so both give
// identical results.  Shapes that do not fit (keys beyond shared memory, more KV heads than a portable cluster) are
// left to the multi-kernel path.
#include <cooperative_groups.h>

#include "ckv_internal.h"
#include "select_common.cuh"

namespace ckv {
namespace {

namespace cg = cooperative_groups;

constexpr int kD1Shift = 20, kD1Bins = 4096;   // first digit: sign, exponent and 3 mantissa bits
constexpr int kD2Bins = 1024;                  // second and third digit: 10 bits each
constexpr int kMaxCluster = 8;                 // portable cluster size

struct FusedArgs {
  const float* attn;
  const float* vnorm;
  const int32_t* budgets_in;   // given budgets [nb, Hkv] or null
  float* c;                    // scratch [nb, Hkv, n]
  int32_t* budgets_out;        // [nb, Hkv]: the budgets actually used (adaptive mode), may be null
  int32_t* idx;
  int32_t* offsets;
  uint8_t* stage;
  int* status;
  const int32_t* valid_from;
  int Hq, Hkv, G, n;
  int group_sum, protect_from;
  int cand_cap;
  long long uniform_b, btot, b_adapt;
  int floor_b;
  float alpha, eps;
};

struct FusedFixed {
  SelectShared old;          // hist[0..15] = first-digit histogram of a, hist[16..31] = working histogram
  uint32_t wtot[kSelWarps];
  uint32_t res_bin, res_k;
  uint32_t cand_count;
  uint32_t cnt[2];           // this head's keys above / equal to the flattened threshold (read by the cluster)
};

// k-th largest position in a histogram spread over the CTA: thread t holds the counts of bins t*PER .. t*PER+PER-1
// (higher bin = larger key).  Returns the bin that holds the k-th largest key and k minus the keys in higher bins.
template <int PER>
__device__ __forceinline__ void find_bin(const uint32_t (&v)[PER], uint32_t k, FusedFixed& sh, uint32_t* bin,
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
  if (tid == 0) { sh.res_bin = 0; sh.res_k = 0; }
  __syncthreads();
  uint32_t above = x - s;
  for (int q = warp + 1; q < kSelWarps; ++q) above += sh.wtot[q];
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

__device__ __forceinline__ void zero_words(uint32_t* p, int count) {
  for (int e = threadIdx.x; e < count; e += kSelThreads) p[e] = 0;
}

// One entry of the group reduce: the sums over the group's heads are finished into (a, c), the special scores of the
// protected window and of the padding are applied, and -0 is folded into +0.
__device__ __forceinline__ void finish_entry(float sa, float sc, float Gf, float eps, int group_sum, float vg, int i,
                                             int protect_from, int vf, float* av_out, float* cv_out) {
  float av = __fdiv_rn(sa, Gf);
  float cv = group_sum ? __fmul_rn(__fadd_rn(av, eps), vg) : __fdiv_rn(sc, Gf);
  if (i >= protect_from) av = cv = 3.402823466e+38f;
  if (i < vf) av = cv = -1.0f;
  if (av == 0.f) av = 0.f;
  if (cv == 0.f) cv = 0.f;
  *av_out = av;
  *cv_out = cv;
}

template <bool kCluster>
__global__ void __launch_bounds__(kSelThreads, 1) select_fused_kernel(FusedArgs p) {
  extern __shared__ __align__(16) uint8_t fused_smem[];
  FusedFixed& sh = *reinterpret_cast<FusedFixed*>(fused_smem);
  const int n = p.n;
  const int nwords = (n + 31) / 32;
  uint32_t* keys = reinterpret_cast<uint32_t*>(fused_smem + ((sizeof(FusedFixed) + 15) / 16) * 16);
  uint32_t* sel1 = keys + ((n + 3) / 4) * 4;
  uint32_t* sel2 = sel1 + nwords;
  uint32_t* cand_key = sel2 + nwords;
  uint32_t* cand_idx = cand_key + p.cand_cap;
  uint32_t* hist_d1 = &sh.old.hist[0][0];
  uint32_t* hist_w = &sh.old.hist[kSelWarps / 2][0];
  static_assert(kSelWarps * 256 == 2 * kD1Bins, "the two histograms alias the 8-bit select's per-warp histograms");

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x / p.Hkv, g = blockIdx.x % p.Hkv;
  const int G = p.G;
  const long long h0 = (long long)b * p.Hq + (long long)g * G;
  const float Gf = (float)G;
  const int vf = p.valid_from ? p.valid_from[b * p.Hkv + g] : 0;
  float* cg_out = p.c + ((long long)b * p.Hkv + g) * n;

  zero_words(hist_d1, 2 * kD1Bins);
  if (tid == 0) { sh.cand_count = 0; sh.cnt[0] = 0; sh.cnt[1] = 0; }
  __syncthreads();

  // ---------------- reduce: one pass over attn and vnorm ----------------
  const float* vg_row = p.group_sum ? p.vnorm + ((long long)b * p.Hkv + g) * n : nullptr;
  if ((n & 3) == 0) {
    const int n4 = n >> 2;
    for (int i4 = tid; i4 < n4; i4 += kSelThreads) {
      float sa[4] = {0.f, 0.f, 0.f, 0.f}, sc[4] = {0.f, 0.f, 0.f, 0.f};
      for (int q0 = 0; q0 < G; q0 += 4) {
        float4 pa[4], pv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (q0 + u < G) {
            pa[u] = __ldcs(reinterpret_cast<const float4*>(p.attn + (h0 + q0 + u) * n) + i4);
            if (!p.group_sum) pv[u] = __ldcs(reinterpret_cast<const float4*>(p.vnorm + (h0 + q0 + u) * n) + i4);
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (q0 + u < G) {
            const float a4[4] = {pa[u].x, pa[u].y, pa[u].z, pa[u].w};
            float v4[4] = {0.f, 0.f, 0.f, 0.f};
            if (!p.group_sum) { v4[0] = pv[u].x; v4[1] = pv[u].y; v4[2] = pv[u].z; v4[3] = pv[u].w; }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float prod = __fmul_rn(__fadd_rn(a4[j], p.eps), v4[j]);
              if (q0 + u == 0) { sa[j] = a4[j]; sc[j] = prod; }
              else { sa[j] = __fadd_rn(sa[j], a4[j]); sc[j] = __fadd_rn(sc[j], prod); }
            }
          }
        }
      }
      float4 vg4 = make_float4(0.f, 0.f, 0.f, 0.f);
      if (p.group_sum) vg4 = __ldcs(reinterpret_cast<const float4*>(vg_row) + i4);
      const float vgs[4] = {vg4.x, vg4.y, vg4.z, vg4.w};
      float cv[4];
      uint32_t ka[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float av;
        finish_entry(sa[j], sc[j], Gf, p.eps, p.group_sum, vgs[j], 4 * i4 + j, p.protect_from, vf, &av, &cv[j]);
        ka[j] = order_key(av);
      }
      *reinterpret_cast<uint4*>(keys + 4 * i4) = make_uint4(ka[0], ka[1], ka[2], ka[3]);
      *reinterpret_cast<float4*>(cg_out + 4 * i4) = make_float4(cv[0], cv[1], cv[2], cv[3]);
      // neighbouring entries mostly share a bin (the scores are max-pooled): one atomic per run
      uint32_t cur = ka[0] >> kD1Shift, run = 1;
#pragma unroll
      for (int j = 1; j < 4; ++j) {
        const uint32_t bin = ka[j] >> kD1Shift;
        if (bin == cur) {
          ++run;
        } else {
          atomicAdd(&hist_d1[cur], run);
          cur = bin;
          run = 1;
        }
      }
      atomicAdd(&hist_d1[cur], run);
    }
  } else {
    for (int i = tid; i < n; i += kSelThreads) {
      float sa = 0.f, sc = 0.f;
      for (int q = 0; q < G; ++q) {
        const float a1 = p.attn[(h0 + q) * n + i];
        const float v1 = p.group_sum ? 0.f : p.vnorm[(h0 + q) * n + i];
        const float prod = __fmul_rn(__fadd_rn(a1, p.eps), v1);
        if (q == 0) { sa = a1; sc = prod; }
        else { sa = __fadd_rn(sa, a1); sc = __fadd_rn(sc, prod); }
      }
      float av, cv;
      finish_entry(sa, sc, Gf, p.eps, p.group_sum, p.group_sum ? vg_row[i] : 0.f, i, p.protect_from, vf, &av, &cv);
      const uint32_t ka = order_key(av);
      keys[i] = ka;
      cg_out[i] = cv;
      atomicAdd(&hist_d1[ka >> kD1Shift], 1u);
    }
  }
  __syncthreads();

  // ---------------- this head's budget and the start of its segment ----------------
  long long off = 0, bud = 0;
  bool clipped = false;
  if (kCluster) {
    // flattened top-b_adapt over the keys of every head of the slice (the CTAs of this cluster)
    cg::cluster_group cluster = cg::this_cluster();
    const int cs = (int)cluster.num_blocks();
    uint32_t T = 0, r = 0;
    if (p.b_adapt > 0) {
      cluster.sync();   // every head's first-digit histogram is complete
      uint32_t v4[4] = {0u, 0u, 0u, 0u};
      for (int q = 0; q < cs; ++q) {
        const uint4 x = *reinterpret_cast<const uint4*>(cluster.map_shared_rank(hist_d1, q) + 4 * tid);
        v4[0] += x.x; v4[1] += x.y; v4[2] += x.z; v4[3] += x.w;
      }
      uint32_t bin, krem;
      find_bin<4>(v4, (uint32_t)p.b_adapt, sh, &bin, &krem);
      uint32_t prefix = bin;   // the key bits fixed so far, right-aligned
      for (int round = 0; round < 2; ++round) {
        const int shift = round == 0 ? 10 : 0;
        zero_words(hist_w, kD2Bins);
        __syncthreads();
        for (int i = tid; i < n; i += kSelThreads) {
          const uint32_t key = keys[i];
          if ((key >> (shift + 10)) == prefix) atomicAdd(&hist_w[(key >> shift) & (kD2Bins - 1)], 1u);
        }
        cluster.sync();   // every rank's working histogram is complete
        uint32_t v1[1] = {0u};
        for (int q = 0; q < cs; ++q) v1[0] += cluster.map_shared_rank(hist_w, q)[tid];
        cluster.sync();   // ... and has been read by everyone before the next round clears it
        find_bin<1>(v1, krem, sh, &bin, &krem);
        prefix = (prefix << 10) | bin;
      }
      T = prefix;
      r = krem;
      uint32_t gt = 0, eq = 0;
      for (int i = tid; i < n; i += kSelThreads) {
        const uint32_t key = keys[i];
        gt += key > T;
        eq += key == T;
      }
      gt = __reduce_add_sync(0xffffffffu, gt);
      eq = __reduce_add_sync(0xffffffffu, eq);
      if (lane == 0) {
        if (gt) atomicAdd(&sh.cnt[0], gt);
        if (eq) atomicAdd(&sh.cnt[1], eq);
      }
      cluster.sync();   // every head's counts are complete
      uint32_t rem = r;
      for (int q = 0; q < cs; ++q) {
        const uint32_t* pc = cluster.map_shared_rank(sh.cnt, q);
        const uint32_t take = min(pc[1], rem);
        const long long bq = min((long long)pc[0] + take + p.floor_b, (long long)n);
        rem -= take;
        if (q < g) off += bq;
        if (q == g) bud = bq;
      }
      cluster.sync();   // nobody leaves (or rewrites cnt) while a peer still reads its shared memory
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
  if (clipped && tid == 0) atomicExch(p.status, (int)CKV_EINVAL);
  long long b1 = (long long)floor((double)p.alpha * (double)bud);
  b1 = min(max(b1, 0LL), bud);
  const long long b2 = bud - b1;

  // ---------------- stage 1: the b1 largest a (keys in shared memory) ----------------
  uint32_t T1 = 0, r1 = 0;
  if (b1 > 0) {
    uint32_t v4[4];
    {
      const uint4 x = *reinterpret_cast<const uint4*>(hist_d1 + 4 * tid);
      v4[0] = x.x; v4[1] = x.y; v4[2] = x.z; v4[3] = x.w;
    }
    uint32_t bin, krem;
    find_bin<4>(v4, (uint32_t)b1, sh, &bin, &krem);
    uint32_t prefix = bin;
    for (int round = 0; round < 2; ++round) {
      const int shift = round == 0 ? 10 : 0;
      zero_words(hist_w, kD2Bins);
      __syncthreads();
      for (int i = tid; i < n; i += kSelThreads) {
        const uint32_t key = keys[i];
        if ((key >> (shift + 10)) == prefix) atomicAdd(&hist_w[(key >> shift) & (kD2Bins - 1)], 1u);
      }
      __syncthreads();
      uint32_t v1[1] = {hist_w[tid]};
      find_bin<1>(v1, krem, sh, &bin, &krem);
      prefix = (prefix << 10) | bin;
    }
    T1 = prefix;
    r1 = krem;
  }

  // ordered marking walk: warp q owns the words [q * wpw, (q + 1) * wpw); entries stage 1 leaves feed the first-digit
  // histogram of c
  const int wpw = (nwords + kSelWarps - 1) / kSelWarps;
  const int w0 = min(warp * wpw, nwords), w1 = min(w0 + wpw, nwords);
  {
    uint32_t eq_count = 0;
    if (b1 > 0) {
      for (int q = w0; q < w1; ++q) {
        const int i = q * 32 + lane;
        eq_count += __popc(__ballot_sync(0xffffffffu, i < n && keys[i] == T1));
      }
    }
    if (lane == 0) sh.old.warp_cnt[warp] = eq_count;
    zero_words(hist_w, kD1Bins);
    __syncthreads();
    uint32_t running = 0;
    for (int q = 0; q < warp; ++q) running += sh.old.warp_cnt[q];
    for (int q0 = w0; q0 < w1; q0 += 4) {
      float cv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = (q0 + u) * 32 + lane;
        cv[u] = (b2 > 0 && q0 + u < w1 && i < n) ? __ldcg(cg_out + i) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int q = q0 + u;
        if (q >= w1) break;   // uniform across the warp
        const int i = q * 32 + lane;
        const bool valid = i < n;
        const uint32_t key = valid ? keys[i] : 0u;
        const bool eq = b1 > 0 && valid && key == T1;
        const uint32_t eqm = __ballot_sync(0xffffffffu, eq);
        const bool take = eq && (running + __popc(eqm & ((1u << lane) - 1u)) < r1);
        const bool in1 = b1 > 0 && valid && (key > T1 || take);
        const uint32_t word = __ballot_sync(0xffffffffu, in1);
        if (lane == 0) sel1[q] = word;
        running += __popc(eqm);
        if (b2 > 0 && valid && !in1) atomicAdd(&hist_w[order_key(cv[u]) >> kD1Shift], 1u);
      }
    }
    __syncthreads();
  }

  // ---------------- stage 2: the b2 largest c among the entries stage 1 left ----------------
  if (b2 > 0) {
    uint32_t v4[4];
    {
      const uint4 x = *reinterpret_cast<const uint4*>(hist_w + 4 * tid);
      v4[0] = x.x; v4[1] = x.y; v4[2] = x.z; v4[3] = x.w;
    }
    uint32_t bin1, krem;
    find_bin<4>(v4, (uint32_t)b2, sh, &bin1, &krem);
    zero_words(hist_w, kD2Bins);
    __syncthreads();
    // one walk over c: entries above the threshold bin are taken, entries inside it become candidates
    for (int q0 = w0; q0 < w1; q0 += 4) {
      float cv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = (q0 + u) * 32 + lane;
        cv[u] = (q0 + u < w1 && i < n) ? __ldcg(cg_out + i) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int q = q0 + u;
        if (q >= w1) break;
        const int i = q * 32 + lane;
        const bool valid = i < n && !((sel1[q] >> lane) & 1u);
        const uint32_t kc = order_key(cv[u]);
        const uint32_t d = kc >> kD1Shift;
        const uint32_t word = __ballot_sync(0xffffffffu, valid && d > bin1);
        if (lane == 0) sel2[q] = word;
        const bool cand = valid && d == bin1;
        const uint32_t cm = __ballot_sync(0xffffffffu, cand);
        if (cm) {
          uint32_t base = 0;
          if (lane == 0) base = atomicAdd(&sh.cand_count, (uint32_t)__popc(cm));
          base = __shfl_sync(0xffffffffu, base, 0);
          if (cand) {
            const uint32_t slot = base + __popc(cm & ((1u << lane) - 1u));
            if (slot < (uint32_t)p.cand_cap) {
              cand_key[slot] = kc;
              cand_idx[slot] = (uint32_t)i;
            }
            atomicAdd(&hist_w[(kc >> 10) & (kD2Bins - 1)], 1u);
          }
        }
      }
    }
    __syncthreads();
    const uint32_t ncand = sh.cand_count;
    if (ncand > (uint32_t)p.cand_cap) {
      // more entries share the threshold bin than the list holds: full-array select and walk over c
      uint32_t T2, r2;
      radix_select(cg_out, n, sel1, (uint32_t)b2, sh.old, &T2, &r2);
      mark_selected(cg_out, n, sel1, T2, r2, true, sel2, sh.old);
    } else {
      uint32_t bin2, bin3;
      {
        uint32_t v1[1] = {hist_w[tid]};
        find_bin<1>(v1, krem, sh, &bin2, &krem);
      }
      zero_words(hist_w, kD2Bins);
      __syncthreads();
      for (uint32_t e = tid; e < ncand; e += kSelThreads) {
        const uint32_t kc = cand_key[e];
        if (((kc >> 10) & (kD2Bins - 1)) == bin2) atomicAdd(&hist_w[kc & (kD2Bins - 1)], 1u);
      }
      __syncthreads();
      {
        uint32_t v1[1] = {hist_w[tid]};
        find_bin<1>(v1, krem, sh, &bin3, &krem);
      }
      const uint32_t T2 = (bin1 << kD1Shift) | (bin2 << 10) | bin3;
      const uint32_t r2 = krem;                 // how many of the entries equal to T2 are taken
      const uint32_t ties = hist_w[bin3];
      uint32_t tie_limit = 0;                   // ties with (0xfffff - index) >= tie_limit are taken
      if (r2 < ties) {
        // the r2 lowest indices among the ties: two more rounds over the 20-bit key (0xfffff - index)
        uint32_t pre = 0, kk = r2;
        for (int round = 0; round < 2; ++round) {
          const int shift = round == 0 ? 10 : 0;
          __syncthreads();   // everyone has read the previous histogram
          zero_words(hist_w, kD2Bins);
          __syncthreads();
          for (uint32_t e = tid; e < ncand; e += kSelThreads) {
            if (cand_key[e] != T2) continue;
            const uint32_t ik = 0xfffffu - cand_idx[e];
            if (round == 0 || (ik >> 10) == pre) atomicAdd(&hist_w[(ik >> shift) & (kD2Bins - 1)], 1u);
          }
          __syncthreads();
          uint32_t v1[1] = {hist_w[tid]};
          uint32_t binx;
          find_bin<1>(v1, kk, sh, &binx, &kk);
          pre = (pre << 10) | binx;
        }
        tie_limit = pre;
      }
      for (uint32_t e = tid; e < ncand; e += kSelThreads) {
        const uint32_t kc = cand_key[e], i = cand_idx[e];
        if (kc > T2 || (kc == T2 && 0xfffffu - i >= tie_limit)) atomicOr(&sel2[i >> 5], 1u << (i & 31));
      }
      __syncthreads();
    }
  } else {
    for (int q = w0 + lane; q < w1; q += 32) sel2[q] = 0;
    __syncthreads();
  }

  // ---------------- output: ascending indices of sel1 | sel2 ----------------
  uint32_t cnt = 0;
  for (int q = w0 + lane; q < w1; q += 32) cnt += __popc(sel1[q] | sel2[q]);
  cnt = __reduce_add_sync(0xffffffffu, cnt);
  if (lane == 0) sh.old.warp_cnt[warp] = cnt;
  __syncthreads();
  uint32_t running = 0;
  for (int q = 0; q < warp; ++q) running += sh.old.warp_cnt[q];
  int32_t* idx = p.idx + (long long)b * p.btot + off;
  uint8_t* stage = p.stage ? p.stage + (long long)b * p.btot + off : nullptr;
  for (int q = w0; q < w1; ++q) {
    const uint32_t s1 = sel1[q], word = s1 | sel2[q];
    if ((word >> lane) & 1u) {
      const uint32_t pos = running + __popc(word & ((1u << lane) - 1u));
      idx[pos] = q * 32 + lane;
      if (stage) stage[pos] = ((s1 >> lane) & 1u) ? 1 : 2;
    }
    running += __popc(word);
  }
  if (tid == 0) {
    p.offsets[(long long)b * (p.Hkv + 1) + g] = (int32_t)off;
    if (g == p.Hkv - 1) p.offsets[(long long)b * (p.Hkv + 1) + p.Hkv] = (int32_t)(off + bud);
  }
}

size_t fused_smem_bytes(int n, int cand_cap) {
  const size_t fixed = (sizeof(FusedFixed) + 15) / 16 * 16;
  const size_t nwords = (size_t)(n + 31) / 32;
  return fixed + (size_t)((n + 3) / 4) * 16 + 2 * nwords * 4 + (size_t)cand_cap * 8;
}

}  // namespace

cudaError_t launch_select_fused(const Dims& d, const float* attn, const float* vnorm, const int32_t* budgets_in,
                                int32_t* idx, int32_t* offsets, uint8_t* stage, const SelectWorkspace& ws,
                                int smem_limit, cudaStream_t st, int* launches, int* status_word) {
  const bool adaptive = d.budget_mode == CKV_BUDGET_FLAT_ADAPTIVE;
  if (adaptive && d.Hkv > kMaxCluster) return cudaErrorNotSupported;
  if (d.n > (1 << 20) - 1) return cudaErrorNotSupported;   // the index tie-break works on 20-bit keys
  int cap = 4096;
  while (cap >= 1024 && fused_smem_bytes(d.n, cap) > (size_t)smem_limit) cap >>= 1;
  if (cap < 1024) return cudaErrorNotSupported;
  const size_t smem = fused_smem_bytes(d.n, cap);

  FusedArgs p;
  p.attn = attn; p.vnorm = vnorm;
  p.budgets_in = d.budget_mode == CKV_BUDGET_GIVEN ? budgets_in : nullptr;
  p.c = ws.c; p.budgets_out = adaptive ? ws.budgets : nullptr;
  p.idx = idx; p.offsets = offsets; p.stage = stage; p.status = status_word;
  p.valid_from = d.valid_from;
  p.Hq = d.Hq; p.Hkv = d.Hkv; p.G = d.G; p.n = d.n;
  p.group_sum = d.group_sum;
  p.protect_from = d.protect_window ? d.n - d.w : d.n;
  p.cand_cap = cap;
  p.uniform_b = d.budget; p.btot = d.btot;
  p.b_adapt = d.budget - (long long)d.Hkv * d.floor_b;
  p.floor_b = (int)d.floor_b;
  p.alpha = d.alpha; p.eps = d.eps;

  auto kernel = adaptive ? select_fused_kernel<true> : select_fused_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((long long)d.nb * d.Hkv));
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = (unsigned)(adaptive ? d.Hkv : 1);
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  if (adaptive) {
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg);
    if (e != cudaSuccess || clusters < 1) {
      (void)cudaGetLastError();
      return cudaErrorNotSupported;
    }
  }
  e = cudaLaunchKernelEx(&cfg, kernel, p);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  *launches += 1;
  return cudaSuccess;
}

}  // namespace ckv
