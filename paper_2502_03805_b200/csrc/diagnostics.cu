// Perturbation diagnostics of Section 3 for a finished selection, per query head and window row j:
//   sigma (Assumption 3.4), retained attention mass, C = sum_i A_i nu_i and its parts over the two stages, min_i nu_i,
//   L = || (A - A') V W^O ||_1 (Definition 3.1, A' by Theorem 3.2), theta (Theorem 3.3), theta_hat (Theorem 3.5) and
//   the relaxed bound of the appendix.
// A is the causal softmax row of window query j (not the pooled mean): the theory is stated for one query.
// Not on the hot path: one CTA per (nb slice, query head) walks all keys in chunks of 256 (one thread per key for the
// logits, then a small P^T V product from shared memory for the two output vectors), float32 throughout, fixed
// summation order.
#include <cuda_bf16.h>
#include <math.h>

#include "ckv_internal.h"
#include "simt_common.cuh"

namespace ckv {
namespace {

constexpr int kDiagFields = 10;

struct DiagArgs {
  const void* Qw;
  const void* K;
  const void* V;
  const void* WO;
  const float* vnorm;
  const uint8_t* stage_of;  // [nb, Hkv, n]: 0 evicted, 1 / 2 kept by that stage
  const float* rowstat;     // [nb*Hq*w, 2]: (max, 1 / (w * sum)) of every window row
  float* diag;              // [nb, Hq, w, kDiagFields]
  int Hq, Hkv, G, n, w, dm;
  float scale;
  long long qs[3], ks[3], vs[3];
  long long wo_nb_stride;
};

__global__ void scatter_stage_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ offsets,
                                     const uint8_t* __restrict__ stage, uint8_t* __restrict__ stage_of, int Hkv, int n,
                                     long long btot) {
  __shared__ int32_t offs[65];
  const int b = blockIdx.y;
  for (int q = threadIdx.x; q <= Hkv; q += blockDim.x) offs[q] = offsets[(long long)b * (Hkv + 1) + q];
  __syncthreads();
  const long long total = min((long long)offs[Hkv], btot);
  for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < total; r += (long long)gridDim.x * blockDim.x) {
    int g = 0;
    while (g + 1 < Hkv && r >= offs[g + 1]) ++g;
    const int src = idx[(long long)b * btot + r];
    if (src >= 0 && src < n) stage_of[((long long)b * Hkv + g) * n + src] = stage[(long long)b * btot + r];
  }
}

template <typename T, int DH, int WT>
__global__ void __launch_bounds__(kThreads) diag_kernel(DiagArgs a) {
  extern __shared__ __align__(16) float smem[];
  float* q_s = smem;                              // [WT][DH]
  float* P = q_s + WT * DH;                       // [256][WT]   weights of the chunk (later: d[DH][WT])
  float* accum = P + kThreads * WT;               // [WT][8]     running scalar sums
  float* stat = accum + WT * 8;                   // [WT][2]
  float* nus = stat + WT * 2;                     // [256]
  float* red = nus + kThreads;                    // [8][WT]
  uint8_t* msk = reinterpret_cast<uint8_t*>(red + 8 * WT);          // [256]
  T* Vs = reinterpret_cast<T*>(msk + kThreads);                     // [128][DH]

  const int h = blockIdx.x, b = blockIdx.y;
  const int g = h / a.G;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long row0 = (long long)(b * a.Hq + h) * a.w;

  {
    const T* q = reinterpret_cast<const T*>(a.Qw) + b * a.qs[0] + h * a.qs[1];
    for (int e = tid; e < WT * DH; e += kThreads) {
      const int j = e / DH, t = e % DH;
      q_s[e] = (j < a.w) ? to_float(q[j * a.qs[2] + t]) : 0.f;
    }
    for (int e = tid; e < WT * 8; e += kThreads) accum[e] = 0.f;
    for (int e = tid; e < 2 * a.w; e += kThreads) stat[e] = a.rowstat[row0 * 2 + e];
  }
  __syncthreads();

  constexpr int RG = kThreads / DH;      // row groups of the P^T V product
  constexpr int RPG = WT / RG;           // window rows per thread
  const int t_col = tid % DH, rg = tid / DH;
  float acc_o[RPG], acc_s[RPG];
#pragma unroll
  for (int r = 0; r < RPG; ++r) acc_o[r] = acc_s[r] = 0.f;
  float nu_min = INFINITY;
  const int first_pos = a.n - a.w;
  const T* Kg = reinterpret_cast<const T*>(a.K) + b * a.ks[0] + g * a.ks[1];
  const T* Vg = reinterpret_cast<const T*>(a.V) + b * a.vs[0] + g * a.vs[1];

  for (int c0 = 0; c0 < a.n; c0 += kThreads) {
    const int i = c0 + tid;
    const bool in_range = i < a.n;
    {
      float acc[WT];
      if (in_range) {
        key_logits<T, DH, WT>(Kg + (long long)i * a.ks[2], q_s, acc);
      } else {
#pragma unroll
        for (int j = 0; j < WT; ++j) acc[j] = 0.f;
      }
#pragma unroll
      for (int j = 0; j < WT; ++j) {
        const bool visible = in_range && j < a.w && i <= first_pos + j;
        // rowstat holds 1 / (w * sum): the plain softmax weight needs the factor w back
        P[tid * WT + j] = visible ? expf(acc[j] * a.scale - stat[2 * j]) * stat[2 * j + 1] * (float)a.w : 0.f;
      }
    }
    const float nu_i = in_range ? a.vnorm[(long long)(b * a.Hq + h) * a.n + i] : 0.f;
    if (in_range) nu_min = fminf(nu_min, nu_i);
    nus[tid] = nu_i;
    msk[tid] = in_range ? a.stage_of[((long long)b * a.Hkv + g) * a.n + i] : (uint8_t)0;
    __syncthreads();

    // scalar sums: warp q owns rows q, q + 8, ...
    for (int j = warp; j < a.w; j += 8) {
      float s1 = 0.f, sk = 0.f, c = 0.f, c1 = 0.f, c2 = 0.f, m2 = 0.f;
      for (int ii = lane; ii < kThreads; ii += 32) {
        const float p = P[ii * WT + j], pn = p * nus[ii];
        const int st = msk[ii];
        s1 += st == 1 ? p : 0.f;
        m2 += st == 2 ? p : 0.f;
        sk += st != 0 ? p : 0.f;
        c += pn;
        c1 += st == 1 ? pn : 0.f;
        c2 += st == 2 ? pn : 0.f;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
        m2 += __shfl_xor_sync(0xffffffffu, m2, o);
        sk += __shfl_xor_sync(0xffffffffu, sk, o);
        c += __shfl_xor_sync(0xffffffffu, c, o);
        c1 += __shfl_xor_sync(0xffffffffu, c1, o);
        c2 += __shfl_xor_sync(0xffffffffu, c2, o);
      }
      if (lane == 0) {
        accum[j * 8 + 0] += s1;
        accum[j * 8 + 1] += sk;
        accum[j * 8 + 2] += c;
        accum[j * 8 + 3] += c1;
        accum[j * 8 + 4] += c2;
        accum[j * 8 + 5] += m2;
      }
    }

    // o += P^T V and o_kept += (P masked)^T V, 128 keys at a time
    for (int half = 0; half < 2; ++half) {
      const int k0 = c0 + half * 128;
      for (int e = tid; e < 128 * DH; e += kThreads) {
        const int r = e / DH, t = e % DH;
        Vs[e] = (k0 + r < a.n) ? Vg[(long long)(k0 + r) * a.vs[2] + t] : T(0.f);
      }
      __syncthreads();
      for (int ii = 0; ii < 128; ++ii) {
        const int il = half * 128 + ii;
        const float v = to_float(Vs[ii * DH + t_col]);
        const float vk = msk[il] ? v : 0.f;
        const float* prow = P + il * WT + rg * RPG;
#pragma unroll
        for (int r = 0; r < RPG; r += 4) {
          const float4 p4 = *reinterpret_cast<const float4*>(prow + r);
          acc_o[r] = fmaf(p4.x, v, acc_o[r]);         acc_s[r] = fmaf(p4.x, vk, acc_s[r]);
          acc_o[r + 1] = fmaf(p4.y, v, acc_o[r + 1]); acc_s[r + 1] = fmaf(p4.y, vk, acc_s[r + 1]);
          acc_o[r + 2] = fmaf(p4.z, v, acc_o[r + 2]); acc_s[r + 2] = fmaf(p4.z, vk, acc_s[r + 2]);
          acc_o[r + 3] = fmaf(p4.w, v, acc_o[r + 3]); acc_s[r + 3] = fmaf(p4.w, vk, acc_s[r + 3]);
        }
      }
      __syncthreads();
    }
  }

  // min over the block
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) nu_min = fminf(nu_min, __shfl_xor_sync(0xffffffffu, nu_min, o));
  if (lane == 0) red[warp] = nu_min;
  // d[t][j] = o_j[t] - o_kept_j[t] / retained mass   (P's storage is free now)
  float* dvec = P;
#pragma unroll
  for (int r = 0; r < RPG; ++r) {
    const int j = rg * RPG + r;
    const float mass = accum[j * 8 + 1];
    dvec[t_col * WT + j] = acc_o[r] - (mass > 0.f ? acc_s[r] / mass : 0.f);
  }
  __syncthreads();
  if (tid == 0) {
    float m = red[0];
    for (int q = 1; q < 8; ++q) m = fminf(m, red[q]);
    nus[0] = m;
  }
  __syncthreads();
  nu_min = nus[0];
  __syncthreads();

  // L_j = sum_c | sum_t d_j[t] W[t][c] |
  const T* W = reinterpret_cast<const T*>(a.WO) + b * a.wo_nb_stride + (long long)h * DH * a.dm;
  float accL[WT];
#pragma unroll
  for (int j = 0; j < WT; ++j) accL[j] = 0.f;
  for (int c = tid; c < a.dm; c += kThreads) {
    float dot[WT];
#pragma unroll
    for (int j = 0; j < WT; ++j) dot[j] = 0.f;
    for (int t = 0; t < DH; ++t) {
      const float wv = to_float(W[(long long)t * a.dm + c]);
      const float4* d4 = reinterpret_cast<const float4*>(dvec + t * WT);
#pragma unroll
      for (int j = 0; j < WT; j += 4) {
        const float4 d = d4[j / 4];
        dot[j] = fmaf(d.x, wv, dot[j]);
        dot[j + 1] = fmaf(d.y, wv, dot[j + 1]);
        dot[j + 2] = fmaf(d.z, wv, dot[j + 2]);
        dot[j + 3] = fmaf(d.w, wv, dot[j + 3]);
      }
    }
#pragma unroll
    for (int j = 0; j < WT; ++j) accL[j] += fabsf(dot[j]);
  }
#pragma unroll
  for (int j = 0; j < WT; ++j) {
    float s = accL[j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) red[warp * WT + j] = s;
  }
  __syncthreads();
  if (tid < a.w) {
    const int j = tid;
    float L = 0.f;
    for (int q = 0; q < 8; ++q) L += red[q * WT + j];
    const float sigma = accum[j * 8 + 0], mass = accum[j * 8 + 1], C = accum[j * 8 + 2], C1 = accum[j * 8 + 3],
                C2 = accum[j * 8 + 4], m2 = accum[j * 8 + 5];
    const float f_all = mass > 0.f ? 2.f - 1.f / mass : -INFINITY;
    const float f_s1 = sigma > 0.f ? 2.f - 1.f / sigma : -INFINITY;
    float* o = a.diag + (row0 + j) * kDiagFields;
    o[0] = sigma; o[1] = mass; o[2] = C; o[3] = C1; o[4] = C2; o[5] = nu_min; o[6] = L;
    o[7] = C - f_all * (C1 + C2);
    o[8] = C - f_s1 * (C1 + C2);
    o[9] = C - f_s1 * C1 - nu_min * f_s1 * m2;
  }
}

template <typename T, int DH, int WT>
cudaError_t run(const Dims& d, const DiagArgs& a, cudaStream_t st) {
  const size_t smem = (size_t)(WT * DH + kThreads * WT + WT * 8 + WT * 2 + kThreads + 8 * WT) * sizeof(float) +
                      kThreads + (size_t)128 * DH * sizeof(T) + 16;
  auto k = diag_kernel<T, DH, WT>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(d.Hq, d.nb);
  k<<<grid, kThreads, smem, st>>>(a);
  return cudaGetLastError();
}

template <typename T, int DH>
cudaError_t run_w(const Dims& d, const DiagArgs& a, cudaStream_t st) {
  if (d.w <= 16) return run<T, DH, 16>(d, a, st);
  if (d.w <= 32) return run<T, DH, 32>(d, a, st);
  return run<T, DH, 64>(d, a, st);
}

}  // namespace

cudaError_t launch_diagnostics(const Dims& d, const void* Qw, const void* K, const void* V, const void* WO,
                               const float* vnorm, const int32_t* idx, const int32_t* offsets, const uint8_t* stage,
                               float* diag, const ScoreWorkspace& ws, uint8_t* stage_of, cudaStream_t st,
                               int* launches) {
  cudaError_t e = cudaMemsetAsync(stage_of, 0, (size_t)d.nb * d.Hkv * d.n, st);
  if (e != cudaSuccess) return e;
  if (d.btot > 0) {
    long long ctas = (d.btot + 255) / 256;
    if (ctas > 148 * 8) ctas = 148 * 8;
    dim3 sgrid((unsigned)ctas, d.nb);
    scatter_stage_kernel<<<sgrid, 256, 0, st>>>(idx, offsets, stage, stage_of, d.Hkv, d.n, d.btot);
    *launches += 1;
  }
  if ((e = launch_window_stats_simt(d, Qw, K, ws, st, launches)) != cudaSuccess) return e;
  DiagArgs a;
  a.Qw = Qw; a.K = K; a.V = V; a.WO = WO; a.vnorm = vnorm; a.stage_of = stage_of; a.rowstat = ws.rowstat;
  a.diag = diag;
  a.Hq = d.Hq; a.Hkv = d.Hkv; a.G = d.G; a.n = d.n; a.w = d.w; a.dm = d.dm;
  a.scale = d.scale;
  for (int i = 0; i < 3; ++i) { a.qs[i] = d.qs[i]; a.ks[i] = d.ks[i]; a.vs[i] = d.vs[i]; }
  a.wo_nb_stride = d.wo_shared ? 0 : (long long)d.Hq * d.dh * d.dm;
  if (d.dtype == CKV_F32)
    e = d.dh == 64 ? run_w<float, 64>(d, a, st) : run_w<float, 128>(d, a, st);
  else
    e = d.dh == 64 ? run_w<__nv_bfloat16, 64>(d, a, st) : run_w<__nv_bfloat16, 128>(d, a, st);
  *launches += 1;
  return e;
}

}  // namespace ckv
