// Pieces shared by the CUDA-core kernels that walk the keys one thread per key.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "ckv_internal.h"

namespace ckv {
namespace {

constexpr int kThreads = kAttnChunk;  // one key per thread

template <typename T>
struct Vec16;  // 16-byte global load, widened to float
template <>
struct Vec16<float> {
  static constexpr int kElems = 4;
  __device__ static void load(const float* p, float* out) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void load(const __nv_bfloat16* p, float* out) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(u[i] << 16);
      out[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
  }
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// Logits of window rows 0..WT-1 for this thread's key; rows >= w come out as 0 (their queries are zero-filled).
template <typename T, int DH, int WT>
__device__ __forceinline__ void key_logits(const T* krow, const float* q_s, float (&acc)[WT]) {
#pragma unroll
  for (int j = 0; j < WT; ++j) acc[j] = 0.f;
  constexpr int E = Vec16<T>::kElems;
#pragma unroll 1
  for (int t = 0; t < DH; t += E) {
    float kf[E];
    Vec16<T>::load(krow + t, kf);
#pragma unroll
    for (int j = 0; j < WT; ++j) {
      const float4* qv = reinterpret_cast<const float4*>(q_s + j * DH + t);
#pragma unroll
      for (int e4 = 0; e4 < E / 4; ++e4) {
        float4 q = qv[e4];
        acc[j] = fmaf(q.x, kf[4 * e4 + 0], acc[j]);
        acc[j] = fmaf(q.y, kf[4 * e4 + 1], acc[j]);
        acc[j] = fmaf(q.z, kf[4 * e4 + 2], acc[j]);
        acc[j] = fmaf(q.w, kf[4 * e4 + 3], acc[j]);
      }
    }
  }
}

}  // namespace
}  // namespace ckv
