// Step 2 on CUDA cores: nu[h, i] = sum_c | sum_t V[g, i, t] * WO[h, t, c] |  -- the L1 norm of each value row
// projected through head h's slice of W^O (Algorithm 1, "L1 norm of each row of V W^O"; Theorem 3.3).
//
// float32 path and bf16 fallback.  One CTA owns 64 tokens of one query head and walks the dm columns in blocks
// of 64: a 64 x 64 x dh product per block from shared memory (4 x 4 outputs per thread), absolute values summed into
// per-thread row accumulators, so the n x dm product only ever exists as registers.  Fixed summation order.
#include <cuda_bf16.h>

#include "ckv_internal.h"

namespace ckv {
namespace {

constexpr int BM = 64, BN = 64, kThreads = 256, PAD = 4;

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }

struct VnormArgs {
  const void* V;
  const void* WO;
  float* vnorm;
  int Hq, G, n, dm;
  long long vs[3];
  long long wo_nb_stride;  // 0 when W^O is shared by the whole call
};

template <typename T, int DH>
__global__ void __launch_bounds__(kThreads) vnorm_simt_kernel(VnormArgs a) {
  extern __shared__ __align__(16) float smem[];
  float* Vs = smem;                       // [DH][BM + PAD]   (token index contiguous)
  float* Ws = smem + DH * (BM + PAD);     // [DH][BN]
  const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int g = h / a.G;
  const int row0 = tile * BM;
  const T* Vg = reinterpret_cast<const T*>(a.V) + b * a.vs[0] + g * a.vs[1];
  const T* W = reinterpret_cast<const T*>(a.WO) + b * a.wo_nb_stride + (long long)h * DH * a.dm;

  for (int e = threadIdx.x; e < BM * DH; e += kThreads) {
    const int r = e / DH, t = e % DH;
    const int i = row0 + r;
    Vs[t * (BM + PAD) + r] = (i < a.n) ? ldf(Vg + (long long)i * a.vs[2] + t) : 0.f;
  }

  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // 16 column groups x 16 row groups
  float rowsum[4] = {0.f, 0.f, 0.f, 0.f};

  for (int c0 = 0; c0 < a.dm; c0 += BN) {
    __syncthreads();  // previous block's reads of Ws are done (and Vs is complete on the first trip)
    for (int e = threadIdx.x; e < DH * BN; e += kThreads) {
      const int t = e / BN, c = e % BN;
      Ws[e] = (c0 + c < a.dm) ? ldf(W + (long long)t * a.dm + c0 + c) : 0.f;
    }
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
#pragma unroll 8
    for (int t = 0; t < DH; ++t) {
      const float4 v = *reinterpret_cast<const float4*>(Vs + t * (BM + PAD) + ty * 4);
      const float4 w = *reinterpret_cast<const float4*>(Ws + t * BN + tx * 4);
      const float vr[4] = {v.x, v.y, v.z, v.w};
      const float wc[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(vr[r], wc[c], acc[r][c]);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) rowsum[r] += fabsf(acc[r][c]);
  }
  // the 16 column groups of a row are 16 consecutive lanes
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    float s = rowsum[r];
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const int i = row0 + ty * 4 + r;
    if (tx == 0 && i < a.n) a.vnorm[(long long)(b * a.Hq + h) * a.n + i] = s;
  }
}

// out[bw, g, :] = round_to_T(W[bw, g*G] + W[bw, g*G+1] + ...) in float32, heads in increasing order.
template <typename T>
__global__ void wo_group_sum_kernel(const T* __restrict__ W, T* __restrict__ out, int G, long long per_head,
                                    long long total) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // element of out
  if (e >= total) return;
  const long long grp = e / per_head, r = e % per_head;
  const T* src = W + grp * G * per_head + r;
  float acc = ldf(src);
  for (int q = 1; q < G; ++q) acc = __fadd_rn(acc, ldf(src + q * per_head));
  out[e] = T(acc);
}

template <typename T, int DH>
cudaError_t run(const Dims& d, const VnormArgs& a, cudaStream_t st, int* launches) {
  const size_t smem = (size_t)(DH * (BM + PAD) + DH * BN) * sizeof(float);
  auto k = vnorm_simt_kernel<T, DH>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((d.n + BM - 1) / BM, d.Hq, d.nb);
  k<<<grid, kThreads, smem, st>>>(a);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_wo_group_sum(const Dims& d, const void* WO, void* wsum, cudaStream_t st, int* launches) {
  const long long per_head = (long long)d.dh * d.dm;
  const long long total = (long long)(d.wo_shared ? 1 : d.nb) * d.Hkv * per_head;
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (d.dtype == CKV_F32)
    wo_group_sum_kernel<float><<<blocks, 256, 0, st>>>((const float*)WO, (float*)wsum, d.G, per_head, total);
  else
    wo_group_sum_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)WO, (__nv_bfloat16*)wsum, d.G,
                                                              per_head, total);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_vnorm_simt(const Dims& d, const void* V, const void* WO, float* vnorm, cudaStream_t st,
                              int* launches) {
  VnormArgs a;
  a.V = V; a.WO = WO; a.vnorm = vnorm;
  a.Hq = d.Hq; a.G = d.G; a.n = d.n; a.dm = d.dm;
  for (int i = 0; i < 3; ++i) a.vs[i] = d.vs[i];
  a.wo_nb_stride = d.wo_shared ? 0 : (long long)d.Hq * d.dh * d.dm;
  if (d.dtype == CKV_F32) return d.dh == 64 ? run<float, 64>(d, a, st, launches) : run<float, 128>(d, a, st, launches);
  return d.dh == 64 ? run<__nv_bfloat16, 64>(d, a, st, launches) : run<__nv_bfloat16, 128>(d, a, st, launches);
}

}  // namespace ckv
