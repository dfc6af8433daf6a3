// Step 1 on CUDA cores: observation-window attention (Algorithm 2: softmax of the last w queries over all keys,
// mean over the window, max-pool along the sequence; softmax and scale as in Eq. 2).
//
// Used for float32 inputs and as the bf16 fallback.  Four launches:
//   partial : one CTA per (256-key chunk, query head, nb): logits of the w window rows against the chunk's keys,
//             per-row maximum and sum of exponentials of the chunk
//   combine : per (query head, nb): merges the chunk partials into each row's (max, 1 / (w * sum))
//   prob    : recomputes the same logits, normalises, sums the w rows -> window-mean attention
//   pool    : stride-1 centred max-pool with clipped borders
// A thread owns one key; the w logits of that key live in registers.  The two logit computations run the same
// instruction sequence, so a logit never exceeds the maximum found for its row.
#include <cuda_bf16.h>
#include <math.h>

#include "ckv_internal.h"
#include "simt_common.cuh"

namespace ckv {
namespace {


struct AttnArgs {
  const void* Qw;
  const void* K;
  float* part_m;
  float* part_l;
  float* rowstat;
  float* abar;
  int Hq, G, n, w, nchunks;
  const int32_t* valid_from;   // [nb, Hkv] or null: first real key of every KV head
  float scale;
  long long qs[3], ks[3];
};

// Window rows j0 .. j0+WT-1 of query head h as floats; rows past w are zero-filled.
template <typename T, int DH, int WT>
__device__ __forceinline__ void stage_queries(const AttnArgs& a, int b, int h, int j0, float* q_s) {
  const T* q = reinterpret_cast<const T*>(a.Qw) + b * a.qs[0] + h * a.qs[1];
  for (int e = threadIdx.x; e < WT * DH; e += kThreads) {
    int j = j0 + e / DH, t = e % DH;
    q_s[e] = (j < a.w) ? to_float(q[j * a.qs[2] + t]) : 0.f;
  }
}

template <typename T, int DH, int WT, bool kProb>
__global__ void __launch_bounds__(kThreads) attn_pass_kernel(AttnArgs a) {
  extern __shared__ __align__(16) float smem[];
  float* q_s = smem;                         // [WT][DH]
  float* red = smem + WT * DH;               // [8 warps][WT]
  float* stat = red + (kThreads / 32) * WT;  // [WT][2]
  const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int g = h / a.G;
  const int i = chunk * kAttnChunk + threadIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  const long long row = (long long)(b * a.Hq + h) * a.w;
  const bool in_range = i < a.n;
  const int first_pos = a.n - a.w;  // sequence position of window row 0
  const int vf = a.valid_from ? a.valid_from[b * (a.Hq / a.G) + g] : 0;   // keys before vf are padding
  float s = 0.f;                    // second pass: sum of the normalised weights over the window rows
  // the window is walked in blocks of WT rows (one block unless w > 64)
  for (int j0 = 0; j0 < a.w; j0 += WT) {
    if (j0 > 0) __syncthreads();    // the previous block's queries and scratch are no longer read
    stage_queries<T, DH, WT>(a, b, h, j0, q_s);
    const int wb = min(WT, a.w - j0);
    if constexpr (kProb) {
      for (int e = threadIdx.x; e < 2 * wb; e += kThreads) stat[e] = a.rowstat[(row + j0) * 2 + e];
    }
    __syncthreads();

    float acc[WT];
    if (in_range) {
      const T* krow = reinterpret_cast<const T*>(a.K) + b * a.ks[0] + g * a.ks[1] + (long long)i * a.ks[2];
      key_logits<T, DH, WT>(krow, q_s, acc);
    } else {
#pragma unroll
      for (int j = 0; j < WT; ++j) acc[j] = 0.f;
    }
#pragma unroll
    for (int j = 0; j < WT; ++j) {
      const bool visible = in_range && j < wb && i <= first_pos + j0 + j && i >= vf;
      acc[j] = visible ? acc[j] * a.scale : -INFINITY;
    }

    if constexpr (kProb) {
      // normalise with the final row statistics and sum the window rows in increasing row order
#pragma unroll
      for (int j = 0; j < WT; ++j) {
        if (j < wb) {
          float p = (acc[j] == -INFINITY) ? 0.f : expf(acc[j] - stat[2 * j]) * stat[2 * j + 1];
          s += p;
        }
      }
    } else {
      // chunk maximum per row
#pragma unroll
      for (int j = 0; j < WT; ++j) {
        float m = acc[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) red[warp * WT + j] = m;
      }
      __syncthreads();
      if (threadIdx.x < WT) {
        float m = red[threadIdx.x];
        for (int wq = 1; wq < kThreads / 32; ++wq) m = fmaxf(m, red[wq * WT + threadIdx.x]);
        stat[threadIdx.x] = m;
      }
      __syncthreads();
      // chunk sum of exp(logit - chunk max)
#pragma unroll
      for (int j = 0; j < WT; ++j) {
        float e = (acc[j] == -INFINITY) ? 0.f : expf(acc[j] - stat[j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
        if (lane == 0) red[warp * WT + j] = e;
      }
      __syncthreads();
      if (threadIdx.x < wb) {
        float l = red[threadIdx.x];
        for (int wq = 1; wq < kThreads / 32; ++wq) l += red[wq * WT + threadIdx.x];
        const long long o = (row + j0 + threadIdx.x) * a.nchunks + chunk;
        a.part_m[o] = stat[threadIdx.x];
        a.part_l[o] = l;
      }
    }
  }
  if constexpr (kProb) {
    if (in_range) a.abar[(long long)(b * a.Hq + h) * a.n + i] = s;
  }
}

// Merge chunk partials: M = max_c m_c, L = sum_c l_c * exp(m_c - M); store (M, 1 / (w * L)).  One warp per row, lanes
// across the partials (a layer at a time a row has up to n / 256 + 2 of them, and a thread walking them one after
// another took longer than a sweep); the sum runs over each lane's partials in ascending order and then over the
// lanes in a fixed butterfly, so it is the same on every run.
constexpr int kCombineThreads = 128;
__global__ void __launch_bounds__(kCombineThreads) attn_combine_kernel(const float* __restrict__ part_m,
                                                                       const float* __restrict__ part_l,
                                                                       float* __restrict__ rowstat, int rows,
                                                                       int nchunks, int w) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * (kCombineThreads / 32) + (threadIdx.x >> 5);
  if (r >= rows) return;   // whole warps leave
  const float* pm = part_m + (long long)r * nchunks;
  const float* pl = part_l + (long long)r * nchunks;
  float M = -INFINITY;
  for (int c = lane; c < nchunks; c += 128) {
    float m4[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) m4[q] = c + 32 * q < nchunks ? pm[c + 32 * q] : -INFINITY;
#pragma unroll
    for (int q = 0; q < 4; ++q) M = fmaxf(M, m4[q]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float L = 0.f;
  for (int c = lane; c < nchunks; c += 128) {
    float m4[4], l4[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const bool in = c + 32 * q < nchunks;
      m4[q] = in ? pm[c + 32 * q] : -INFINITY;
      l4[q] = in ? pl[c + 32 * q] : 0.f;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (m4[q] != -INFINITY) L += l4[q] * expf(m4[q] - M);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
  if (lane == 0) {
    rowstat[2 * r] = M;
    rowstat[2 * r + 1] = 1.0f / (L * (float)w);
  }
}

// A CTA pools 4096 consecutive positions of one row from a shared-memory copy (with a halo of (kp-1)/2 on both sides),
// so every input is read from global memory once.  The tile is fetched with four 16-byte loads per thread issued
// before any of them is used; a thread then produces 16 outputs a CTA-width apart, so that neither its shared-memory
// reads nor its stores conflict.
constexpr int kPoolTile = 4096;
constexpr int kPoolThreads = 256;
template <int R>
__global__ void __launch_bounds__(kPoolThreads) maxpool_kernel(const float* __restrict__ abar, float* __restrict__ attn,
                                                               int n, int kp) {
  __shared__ __align__(16) float tile[kPoolTile + 64];   // tile[32 + e] = input i0 + e; halo of at most 31 around it
  const long long base = (long long)blockIdx.y * n;
  const int r = (kp - 1) / 2;          // <= 31
  const int i0 = blockIdx.x * kPoolTile;
  const int tid = threadIdx.x;
  const float* row = abar + base;
  if ((n & 3) == 0 && i0 + kPoolTile <= n) {
    float4 v[kPoolTile / (4 * kPoolThreads)];
#pragma unroll
    for (int q = 0; q < kPoolTile / (4 * kPoolThreads); ++q)
      v[q] = __ldcs(reinterpret_cast<const float4*>(row + i0) + q * kPoolThreads + tid);
#pragma unroll
    for (int q = 0; q < kPoolTile / (4 * kPoolThreads); ++q)
      *reinterpret_cast<float4*>(tile + 32 + 4 * (q * kPoolThreads + tid)) = v[q];
  } else {
    for (int e = tid; e < kPoolTile; e += kPoolThreads) {
      const int i = i0 + e;
      tile[32 + e] = i < n ? row[i] : -INFINITY;   // outside the sequence: never the maximum
    }
  }
  if (tid < 2 * r) {
    const int e = tid < r ? tid - r : kPoolTile + (tid - r);
    const int i = i0 + e;
    tile[32 + e] = (i >= 0 && i < n) ? row[i] : -INFINITY;
  }
  __syncthreads();
  if (R >= 0 && (n & 3) == 0 && i0 + kPoolTile <= n) {
    // small kernels (the paper's 7 included): four neighbouring outputs per thread from three 16-byte reads of the
    // tile, one 16-byte store
#pragma unroll
    for (int q = 0; q < kPoolTile / (4 * kPoolThreads); ++q) {
      const int e = 4 * (q * kPoolThreads + tid);
      float v[12];
#pragma unroll
      for (int u = 0; u < 3; ++u) {
        const float4 x = *reinterpret_cast<const float4*>(tile + 32 + e - 4 + 4 * u);
        v[4 * u] = x.x; v[4 * u + 1] = x.y; v[4 * u + 2] = x.z; v[4 * u + 3] = x.w;
      }
      float o[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float m = v[4 + c - (R >= 0 ? R : 0)];
#pragma unroll
        for (int k = 1; k <= 2 * (R >= 0 ? R : 0); ++k) m = fmaxf(m, v[4 + c - (R >= 0 ? R : 0) + k]);
        o[c] = m;
      }
      __stcs(reinterpret_cast<float4*>(attn + base + i0 + e), make_float4(o[0], o[1], o[2], o[3]));
    }
    return;
  }
  for (int e = tid; e < kPoolTile; e += kPoolThreads) {
    const int i = i0 + e;
    if (i >= n) break;
    float m = tile[32 + e - r];
    for (int k = 1; k <= 2 * r; ++k) m = fmaxf(m, tile[32 + e - r + k]);
    __stcs(attn + base + i, m);
  }
}

// R = (kp - 1) / 2 known at compile time for the small kernels, -1 otherwise
static void launch_maxpool_kernel(dim3 grid, cudaStream_t st, const float* abar, float* attn, int n, int kp) {
  switch ((kp - 1) / 2) {
    case 0: maxpool_kernel<0><<<grid, kPoolThreads, 0, st>>>(abar, attn, n, kp); break;
    case 1: maxpool_kernel<1><<<grid, kPoolThreads, 0, st>>>(abar, attn, n, kp); break;
    case 2: maxpool_kernel<2><<<grid, kPoolThreads, 0, st>>>(abar, attn, n, kp); break;
    case 3: maxpool_kernel<3><<<grid, kPoolThreads, 0, st>>>(abar, attn, n, kp); break;
    case 4: maxpool_kernel<4><<<grid, kPoolThreads, 0, st>>>(abar, attn, n, kp); break;
    default: maxpool_kernel<-1><<<grid, kPoolThreads, 0, st>>>(abar, attn, n, kp); break;
  }
}

template <typename T, int DH, int WT>
cudaError_t run(const Dims& d, const AttnArgs& a, float* attn, cudaStream_t st, int* launches) {
  const size_t smem = (size_t)(WT * DH + (kThreads / 32) * WT + 2 * WT) * sizeof(float);
  auto k1 = attn_pass_kernel<T, DH, WT, false>;
  auto k2 = attn_pass_kernel<T, DH, WT, true>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  dim3 grid(a.nchunks, d.Hq, d.nb);
  k1<<<grid, kThreads, smem, st>>>(a);
  const int rows = d.nb * d.Hq * d.w;
  attn_combine_kernel<<<(rows + kCombineThreads / 32 - 1) / (kCombineThreads / 32), kCombineThreads, 0, st>>>(a.part_m, a.part_l, a.rowstat, rows, a.nchunks, d.w);
  k2<<<grid, kThreads, smem, st>>>(a);
  dim3 pgrid((d.n + kPoolTile - 1) / kPoolTile, d.nb * d.Hq);
  launch_maxpool_kernel(pgrid, st, a.abar, attn, d.n, d.kp);
  *launches += 4;
  return cudaGetLastError();
}

// Only the row statistics (max, 1 / (w * sum)) of every window row: first pass and merge.
template <typename T, int DH, int WT>
cudaError_t run_stats(const Dims& d, const AttnArgs& a, cudaStream_t st, int* launches) {
  const size_t smem = (size_t)(WT * DH + (kThreads / 32) * WT + 2 * WT) * sizeof(float);
  auto k1 = attn_pass_kernel<T, DH, WT, false>;
  cudaError_t e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(a.nchunks, d.Hq, d.nb);
  k1<<<grid, kThreads, smem, st>>>(a);
  const int rows = d.nb * d.Hq * d.w;
  attn_combine_kernel<<<(rows + kCombineThreads / 32 - 1) / (kCombineThreads / 32), kCombineThreads, 0, st>>>(a.part_m, a.part_l, a.rowstat, rows, a.nchunks, d.w);
  *launches += 2;
  return cudaGetLastError();
}

template <typename T, int DH>
cudaError_t run_stats_w(const Dims& d, const AttnArgs& a, cudaStream_t st, int* launches) {
  if (d.w <= 16) return run_stats<T, DH, 16>(d, a, st, launches);
  if (d.w <= 32) return run_stats<T, DH, 32>(d, a, st, launches);
  return run_stats<T, DH, 64>(d, a, st, launches);
}

template <typename T, int DH>
cudaError_t run_w(const Dims& d, const AttnArgs& a, float* attn, cudaStream_t st, int* launches) {
  if (d.w <= 16) return run<T, DH, 16>(d, a, attn, st, launches);
  if (d.w <= 32) return run<T, DH, 32>(d, a, attn, st, launches);
  return run<T, DH, 64>(d, a, attn, st, launches);
}

}  // namespace

cudaError_t launch_attn_combine(const float* part_m, const float* part_l, float* rowstat, int rows, int nchunks,
                                int w, cudaStream_t st) {
  attn_combine_kernel<<<(rows + kCombineThreads / 32 - 1) / (kCombineThreads / 32), kCombineThreads, 0, st>>>(part_m, part_l, rowstat, rows, nchunks, w);
  return cudaGetLastError();
}

cudaError_t launch_maxpool(const float* abar, float* attn, int n, int kp, int nrows, cudaStream_t st) {
  dim3 pgrid((n + kPoolTile - 1) / kPoolTile, nrows);
  launch_maxpool_kernel(pgrid, st, abar, attn, n, kp);
  return cudaGetLastError();
}

static AttnArgs make_attn_args(const Dims& d, const void* Qw, const void* K, const ScoreWorkspace& ws) {
  AttnArgs a;
  a.Qw = Qw; a.K = K;
  a.part_m = ws.part_m; a.part_l = ws.part_l; a.rowstat = ws.rowstat; a.abar = ws.abar;
  a.Hq = d.Hq; a.G = d.G; a.n = d.n; a.w = d.w;
  a.nchunks = (d.n + kAttnChunk - 1) / kAttnChunk;
  a.valid_from = d.valid_from;
  a.scale = d.scale;
  for (int i = 0; i < 3; ++i) { a.qs[i] = d.qs[i]; a.ks[i] = d.ks[i]; }
  return a;
}

cudaError_t launch_window_stats_simt(const Dims& d, const void* Qw, const void* K, const ScoreWorkspace& ws,
                                     cudaStream_t st, int* launches) {
  const AttnArgs a = make_attn_args(d, Qw, K, ws);
  if (d.dtype == CKV_F32)
    return d.dh == 64 ? run_stats_w<float, 64>(d, a, st, launches) : run_stats_w<float, 128>(d, a, st, launches);
  return d.dh == 64 ? run_stats_w<__nv_bfloat16, 64>(d, a, st, launches)
                    : run_stats_w<__nv_bfloat16, 128>(d, a, st, launches);
}

cudaError_t launch_window_attn_simt(const Dims& d, const void* Qw, const void* K, float* attn,
                                    const ScoreWorkspace& ws, cudaStream_t st, int* launches) {
  const AttnArgs a = make_attn_args(d, Qw, K, ws);
  if (d.dtype == CKV_F32) {
    return d.dh == 64 ? run_w<float, 64>(d, a, attn, st, launches) : run_w<float, 128>(d, a, attn, st, launches);
  }
  return d.dh == 64 ? run_w<__nv_bfloat16, 64>(d, a, attn, st, launches)
                    : run_w<__nv_bfloat16, 128>(d, a, attn, st, launches);
}

}  // namespace ckv
