// Step 2 with the L2 distance (the paper's appendix on the choice of distance metric: the framework also works with
// ||.||_2 and gives similar quality): nu2[h, i] = || V[g, i, :] W^O_h ||_2.
//
// By the Gram identity ||v W||_2^2 = v (W W^T) v^T the n x dh x dm contraction of the L1 path becomes
//   (1) G_h = W^O_h W^O_h^T                 dh x dh x dm per head, independent of n
//   (2) nu2[h, i] = sqrt(v_i G_h v_i^T)      n x dh x dh per head, dm / dh times cheaper than the L1 projection
// bf16, dh = 128: both run on tcgen05.  (1) uses the same shared-memory tile as A and B operand; its float32 result
// is split into two bf16 matrices G = G_hi + G_lo so that (2) keeps about 16 bits of G.  (2) accumulates
// V G_hi + V G_lo in tensor memory and the epilogue dots every row with the value row itself.
// float32 inputs and dh = 64 use plain CUDA-core kernels.
#include <cuda_bf16.h>
#include <math.h>

#include "ckv_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace ckv {
namespace {

using namespace ptx;

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// ---------------------------------------------------------------------------------------------------------------
// CUDA-core fallbacks (float32 arithmetic)
// ---------------------------------------------------------------------------------------------------------------
// G[hh][t][u] = sum_c W[hh][t][c] * W[hh][u][c]; one CTA per (head, 16 x 16 block of G), columns in chunks of 64.
template <typename T>
__global__ void __launch_bounds__(256) gram_simt_kernel(const T* __restrict__ W, float* __restrict__ G, int dh, int dm) {
  __shared__ float A[16][65], Bm[16][65];
  const long long hh = blockIdx.z;
  const int t0 = blockIdx.y * 16, u0 = blockIdx.x * 16;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const T* Wh = W + hh * (long long)dh * dm;
  float acc = 0.f;
  for (int c0 = 0; c0 < dm; c0 += 64) {
    for (int e = threadIdx.x; e < 16 * 64; e += 256) {
      const int r = e / 64, c = e % 64;
      const bool ok = c0 + c < dm;
      A[r][c] = ok ? ldf(Wh + (long long)(t0 + r) * dm + c0 + c) : 0.f;
      Bm[r][c] = ok ? ldf(Wh + (long long)(u0 + r) * dm + c0 + c) : 0.f;
    }
    __syncthreads();
#pragma unroll 16
    for (int c = 0; c < 64; ++c) acc = fmaf(A[ty][c], Bm[tx][c], acc);
    __syncthreads();
  }
  G[hh * dh * dh + (long long)(t0 + ty) * dh + u0 + tx] = acc;
}

// nu2[b, h, i] = sqrt(v G v^T): one warp per token, lanes over the columns of G.
template <typename T>
__global__ void __launch_bounds__(256) quad_simt_kernel(const T* __restrict__ V, const float* __restrict__ G,
                                                        float* __restrict__ vnorm, int Hq, int Gsz, int n, int dh,
                                                        long long vs0, long long vs1, long long vs2,
                                                        long long g_nb_stride) {
  extern __shared__ float Gs[];  // [dh][dh]
  const int h = blockIdx.y, b = blockIdx.z;
  const float* Gh = G + b * g_nb_stride + (long long)h * dh * dh;
  for (int e = threadIdx.x; e < dh * dh; e += 256) Gs[e] = Gh[e];
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* Vg = V + b * vs0 + (h / Gsz) * vs1;
  for (int i = blockIdx.x * 8 + warp; i < n; i += gridDim.x * 8) {
    const T* v = Vg + (long long)i * vs2;
    float total = 0.f;
    for (int u = lane; u < dh; u += 32) {
      float y = 0.f;
      for (int t = 0; t < dh; ++t) y = fmaf(ldf(v + t), Gs[t * dh + u], y);
      total = fmaf(y, ldf(v + u), total);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    if (lane == 0) vnorm[((long long)b * Hq + h) * n + i] = sqrtf(fmaxf(total, 0.f));
  }
}

// ---------------------------------------------------------------------------------------------------------------
// (1) Gram matrix on tcgen05, dh = 128: one CTA per (nbw slice, head).
// ---------------------------------------------------------------------------------------------------------------
constexpr int kGramStages = 8;
constexpr int kGramThreads = 6 * 32;   // warp 0 TMA, warp 1 MMA, warps 2-5 epilogue
constexpr int kGramStageBytes = 128 * 128;  // 128 rows x 64 bf16

struct GramArgs {
  __nv_bfloat16* ghi;   // [nbw, Hq, 128, 128]
  __nv_bfloat16* glo;
  int* status;
  int Hq, dm;
};

__global__ void __launch_bounds__(kGramThreads, 1)
gram_umma_kernel(const __grid_constant__ CUtensorMap mapW, GramArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_addr(smem);
  const uint32_t bars = sbase + kGramStages * kGramStageBytes;
  auto full = [&](int s) { return bars + 8u * s; };
  auto empty = [&](int s) { return bars + 8u * (kGramStages + s); };
  const uint32_t done_bar = bars + 8u * (2 * kGramStages);
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem + kGramStages * kGramStageBytes + (2 * kGramStages + 1) * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* never = tmem_slot + 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.x, bw = blockIdx.y;
  const int ksteps = (a.dm + 63) / 64;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGramStages; ++s) {
      mbar_init(full(s), 1);
      mbar_init(empty(s), 1);
    }
    mbar_init(done_bar, 1);
    *abort_flag = 0;
    *never = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_addr(const_cast<uint32_t*>(tmem_slot)), 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tensormap(&mapW);
      uint32_t armed = 0, last_phase = 0;
      for (int k = 0; k < ksteps; ++k) {
        const int s = k % kGramStages;
        const uint32_t ph = (k / kGramStages) & 1u;
        if (!mbar_wait_bounded(empty(s), ph ^ 1u, abort_flag)) { failed = true; break; }
        mbar_arrive_expect_tx(full(s), kGramStageBytes);
        tma_load_4d(sbase + s * kGramStageBytes, &mapW, k * 64, 0, h, bw, full(s));
        armed |= 1u << s;
        last_phase = (last_phase & ~(1u << s)) | (ph << s);
      }
      if (failed)
        for (int s = 0; s < kGramStages; ++s)
          if (armed & (1u << s)) mbar_wait_bounded(full(s), (last_phase >> s) & 1u, never, 200000000ull);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(128, 128, 0);
      for (int k = 0; k < ksteps; ++k) {
        const int s = k % kGramStages;
        if (!mbar_wait_bounded(full(s), (k / kGramStages) & 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t tile = sbase + s * kGramStageBytes;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          // the same 128 x 64 tile of W^O_h is both operands: rows t of A, rows u of B, 16 columns per step
          const uint64_t desc = smem_desc_sw128(tile + kk * 32, 16, 1024);
          umma_f16(tmem_base, desc, desc, idesc, (k | kk) ? 1u : 0u);
        }
        umma_commit(empty(s));
      }
      umma_commit(done_bar);
      if (failed) mbar_wait_bounded(done_bar, 0, never, 500000000ull);
    }
  } else {
    // epilogue: lane = row u of G (G is symmetric, so the TMEM row is also the column); split into hi + lo bf16
    const int quad = warp & 3;
    if (!__all_sync(0xffffffffu, mbar_wait_bounded(done_bar, 0, abort_flag, 4000000000ull))) {
      failed = true;
    } else {
      tc_fence_after();
      const int u = quad * 32 + lane;
      const long long row = (((long long)bw * a.Hq + h) * 128 + u) * 128;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float v[32];
        tmem_ld_32cols(tmem_base + ((uint32_t)(quad * 32) << 16) + q * 32, v);
        tc_wait_ld();
        __align__(16) __nv_bfloat16 hi[32], lo[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          hi[e] = __float2bfloat16_rn(v[e]);
          lo[e] = __float2bfloat16_rn(v[e] - __bfloat162float(hi[e]));
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          reinterpret_cast<uint4*>(a.ghi + row + q * 32)[e] = reinterpret_cast<const uint4*>(hi)[e];
          reinterpret_cast<uint4*>(a.glo + row + q * 32)[e] = reinterpret_cast<const uint4*>(lo)[e];
        }
      }
    }
  }
  if (failed) {
    *abort_flag = 1;
    atomicExch(a.status, (int)CKV_ETIMEOUT);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 128);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// (2) quadratic form on tcgen05, dh = 128.  Persistent; a work item is (nb slice, query head, run of token tiles).
//     warp 0: G_hi, G_lo of the item's head (TMA, once per item)   warp 1: MMA issuer   warp 2: V tiles (TMA ring)
//     warps 3-6: epilogue, one per 32-lane quarter of tensor memory
// ---------------------------------------------------------------------------------------------------------------
constexpr int kQuadThreads = 7 * 32;
constexpr int kQuadStages = 4;             // V tile ring
constexpr int kQuadSlots = 4;              // accumulators of 128 columns
constexpr int kQuadTile = 128 * 128 * 2;   // bytes of a 128 x 128 bf16 tile (two 64-column panels)

struct QuadArgs {
  const __nv_bfloat16* V;
  float* vnorm;
  int* status;
  int Hq, Hkv, G, n, g_shared;
  int ntiles, tiles_per_item, chunks;
  long long vs[3];
  long long nitems;
};

struct QItem { int b, h, g, t0, t1; };
__device__ __forceinline__ QItem decode_qitem(long long item, const QuadArgs& a) {
  QItem it;
  const int chunk = (int)(item % a.chunks);
  const long long r = item / a.chunks;
  it.h = (int)(r % a.Hq);
  it.b = (int)(r / a.Hq);
  it.g = it.h / a.G;
  it.t0 = chunk * a.tiles_per_item;
  it.t1 = min(it.t0 + a.tiles_per_item, a.ntiles);
  return it;
}

__global__ void __launch_bounds__(kQuadThreads, 1)
quad_umma_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapGhi,
                 const __grid_constant__ CUtensorMap mapGlo, QuadArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_addr(smem);
  const uint32_t g_addr = sbase;                              // G_hi then G_lo
  const uint32_t v_addr = sbase + 2 * kQuadTile;              // ring of V tiles
  const uint32_t bars = v_addr + kQuadStages * kQuadTile;
  const uint32_t g_full = bars, g_empty = bars + 8;
  auto v_full = [&](int s) { return bars + 8u * (2 + s); };
  auto v_empty = [&](int s) { return bars + 8u * (2 + kQuadStages + s); };
  auto t_full = [&](int s) { return bars + 8u * (2 + 2 * kQuadStages + s); };
  auto t_empty = [&](int s) { return bars + 8u * (2 + 2 * kQuadStages + kQuadSlots + s); };
  const uint32_t drain_bar = bars + 8u * (2 + 2 * kQuadStages + 2 * kQuadSlots);
  constexpr int kBars = 3 + 2 * kQuadStages + 2 * kQuadSlots;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + (2 + kQuadStages) * kQuadTile + kBars * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* never = tmem_slot + 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(g_full, 1);
    mbar_init(g_empty, 1);
    for (int s = 0; s < kQuadStages; ++s) { mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1); }
    for (int s = 0; s < kQuadSlots; ++s) { mbar_init(t_full(s), 1); mbar_init(t_empty(s), 4); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    *never = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_addr(const_cast<uint32_t*>(tmem_slot)), kQuadSlots * 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tensormap(&mapGhi);
      prefetch_tensormap(&mapGlo);
      uint32_t item_cnt = 0;
      bool armed = false;
      for (long long item = blockIdx.x; item < a.nitems; item += gridDim.x, ++item_cnt) {
        const QItem w = decode_qitem(item, a);
        if (!mbar_wait_bounded(g_empty, (item_cnt & 1u) ^ 1u, abort_flag)) { failed = true; break; }
        mbar_arrive_expect_tx(g_full, 2 * kQuadTile);
        const int bg = a.g_shared ? 0 : w.b;
#pragma unroll
        for (int p = 0; p < 2; ++p) {
          tma_load_4d(g_addr + p * (128 * 128), &mapGhi, p * 64, 0, w.h, bg, g_full);
          tma_load_4d(g_addr + kQuadTile + p * (128 * 128), &mapGlo, p * 64, 0, w.h, bg, g_full);
        }
        armed = true;
      }
      if (failed && armed) mbar_wait_bounded(g_full, (item_cnt - 1) & 1u, never, 200000000ull);
    }
  } else if (warp == 2) {
    if (lane == 0) {
      prefetch_tensormap(&mapV);
      uint32_t it_v = 0, armed = 0, last_phase = 0;
      for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x) {
        const QItem w = decode_qitem(item, a);
        for (int t = w.t0; t < w.t1; ++t, ++it_v) {
          const int s = it_v % kQuadStages;
          const uint32_t ph = (it_v / kQuadStages) & 1u;
          if (!mbar_wait_bounded(v_empty(s), ph ^ 1u, abort_flag)) { failed = true; break; }
          mbar_arrive_expect_tx(v_full(s), kQuadTile);
#pragma unroll
          for (int p = 0; p < 2; ++p)
            tma_load_4d(v_addr + s * kQuadTile + p * (128 * 128), &mapV, p * 64, t * 128, w.g, w.b, v_full(s));
          armed |= 1u << s;
          last_phase = (last_phase & ~(1u << s)) | (ph << s);
        }
      }
      if (failed)
        for (int s = 0; s < kQuadStages; ++s)
          if (armed & (1u << s)) mbar_wait_bounded(v_full(s), (last_phase >> s) & 1u, never, 200000000ull);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(128, 128, 0);
      uint32_t it_v = 0, item_cnt = 0;
      for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x, ++item_cnt) {
        const QItem w = decode_qitem(item, a);
        if (!mbar_wait_bounded(g_full, item_cnt & 1u, abort_flag)) { failed = true; break; }
        for (int t = w.t0; t < w.t1; ++t, ++it_v) {
          const int s = it_v % kQuadStages, slot = it_v % kQuadSlots;
          if (!mbar_wait_bounded(v_full(s), (it_v / kQuadStages) & 1u, abort_flag)) { failed = true; break; }
          if (!mbar_wait_bounded(t_empty(slot), ((it_v / kQuadSlots) & 1u) ^ 1u, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t va = v_addr + s * kQuadTile;
          // y = v G_hi + v G_lo: rows = tokens (A, K-major), B row u = G[u][:] (symmetric, so K-major as stored)
#pragma unroll
          for (int part = 0; part < 2; ++part)
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint32_t off = (kk / 4) * (128 * 128) + (kk % 4) * 32;
              umma_f16(tmem_base + slot * 128, smem_desc_sw128(va + off, 16, 1024),
                       smem_desc_sw128(g_addr + part * kQuadTile + off, 16, 1024), idesc, (part | kk) ? 1u : 0u);
            }
          umma_commit(t_full(slot));
          umma_commit(v_empty(s));
        }
        if (failed) break;
        umma_commit(g_empty);
      }
      umma_commit(drain_bar);
      mbar_wait_bounded(drain_bar, 0, never, 500000000ull);
    }
  } else {
    const int quad = warp & 3;
    uint32_t it_v = 0;
    for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x) {
      const QItem w = decode_qitem(item, a);
      const __nv_bfloat16* Vg = a.V + w.b * a.vs[0] + w.g * a.vs[1];
      for (int t = w.t0; t < w.t1; ++t, ++it_v) {
        const int slot = it_v % kQuadSlots;
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(t_full(slot), (it_v / kQuadSlots) & 1u, abort_flag))) {
          failed = true;
          break;
        }
        tc_fence_after();
        const int i = t * 128 + quad * 32 + lane;
        const uint4* vrow = reinterpret_cast<const uint4*>(Vg + (long long)min(i, a.n - 1) * a.vs[2]);
        float total = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float y[32];
          tmem_ld_32cols(tmem_base + ((uint32_t)(quad * 32) << 16) + slot * 128 + q * 32, y);
          tc_wait_ld();
          if (q == 3) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(t_empty(slot));
          }
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint4 pk = vrow[q * 4 + e];
            const uint32_t u[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
            for (int z = 0; z < 4; ++z) {
              s0 = fmaf(y[e * 8 + 2 * z], __uint_as_float(u[z] << 16), s0);
              s1 = fmaf(y[e * 8 + 2 * z + 1], __uint_as_float(u[z] & 0xffff0000u), s1);
            }
          }
          total += s0 + s1;
        }
        if (i < a.n) a.vnorm[((long long)w.b * a.Hq + w.h) * a.n + i] = sqrtf(fmaxf(total, 0.f));
      }
    }
  }
  if (failed) {
    *abort_flag = 1;
    atomicExch(a.status, (int)CKV_ETIMEOUT);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kQuadSlots * 128);
  }
}

}  // namespace

size_t vnorm_l2_workspace_bytes(const Dims& d) {
  return (size_t)(d.wo_shared ? 1 : d.nb) * d.Hq * d.dh * d.dh * 4;   // float32 G, or bf16 G_hi + G_lo
}

cudaError_t launch_vnorm_l2(const Dims& d, const void* V, const void* WO, float* vnorm, void* gram, int sm_count,
                            int cc_major, bool force_simt, int* status_word, cudaStream_t st, int* launches,
                            int* used_tensor_cores) {
  const int nbw = d.wo_shared ? 1 : d.nb;
  *used_tensor_cores = 0;
  const bool tc = d.dtype == CKV_BF16 && d.dh == 128 && !force_simt && cc_major == 10 && tma_encode_fn() != nullptr;
  if (tc) {
    CUtensorMap mw, mv, mhi, mlo;
    const long long per = (long long)nbw * d.Hq * 128 * 128;
    __nv_bfloat16* ghi = (__nv_bfloat16*)gram;
    __nv_bfloat16* glo = ghi + per;
    const cuuint64_t wdims[4] = {(cuuint64_t)d.dm, (cuuint64_t)d.dh, (cuuint64_t)d.Hq, (cuuint64_t)nbw};
    const long long wstr[3] = {d.dm, (long long)d.dh * d.dm, (long long)d.Hq * d.dh * d.dm};
    const cuuint32_t box[4] = {64, 128, 1, 1};
    const cuuint64_t gdims[4] = {128, 128, (cuuint64_t)d.Hq, (cuuint64_t)nbw};
    const long long gstr[3] = {128, 128 * 128, (long long)d.Hq * 128 * 128};
    const cuuint64_t vdims[4] = {(cuuint64_t)d.dh, (cuuint64_t)d.n, (cuuint64_t)d.Hkv, (cuuint64_t)d.nb};
    const long long vstr[3] = {d.vs[2], d.vs[1], d.vs[0]};
    if (make_bf16_map_4d(&mw, WO, wdims, wstr, box) && make_bf16_map_4d(&mhi, ghi, gdims, gstr, box) &&
        make_bf16_map_4d(&mlo, glo, gdims, gstr, box) && make_bf16_map_4d(&mv, V, vdims, vstr, box)) {
      cudaError_t e;
      {
        const int smem = kGramStages * kGramStageBytes + (2 * kGramStages + 1) * 8 + 16 + 1024;
        if ((e = cudaFuncSetAttribute(gram_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) !=
            cudaSuccess)
          return e;
        GramArgs ga{ghi, glo, status_word, d.Hq, d.dm};
        gram_umma_kernel<<<dim3(d.Hq, nbw), kGramThreads, smem, st>>>(mw, ga);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
      }
      QuadArgs qa;
      qa.V = (const __nv_bfloat16*)V; qa.vnorm = vnorm; qa.status = status_word;
      qa.Hq = d.Hq; qa.Hkv = d.Hkv; qa.G = d.G; qa.n = d.n; qa.g_shared = d.wo_shared;
      qa.ntiles = (d.n + 127) / 128;
      long long want = 4LL * sm_count;
      int tpi = (int)(((long long)d.nb * d.Hq * qa.ntiles + want - 1) / want);
      if (tpi < 8) tpi = 8;
      if (tpi > 64) tpi = 64;
      qa.tiles_per_item = tpi;
      qa.chunks = (qa.ntiles + tpi - 1) / tpi;
      qa.nitems = (long long)d.nb * d.Hq * qa.chunks;
      for (int i = 0; i < 3; ++i) qa.vs[i] = d.vs[i];
      const int smem = (2 + kQuadStages) * kQuadTile + (3 + 2 * kQuadStages + 2 * kQuadSlots) * 8 + 16 + 1024;
      if ((e = cudaFuncSetAttribute(quad_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) !=
          cudaSuccess)
        return e;
      const int grid = (int)(qa.nitems < sm_count ? qa.nitems : sm_count);
      quad_umma_kernel<<<grid, kQuadThreads, smem, st>>>(mv, mhi, mlo, qa);
      *launches += 2;
      *used_tensor_cores = 1;
      return cudaGetLastError();
    }
  }
  // CUDA-core path
  float* G = (float*)gram;
  dim3 ggrid(d.dh / 16, d.dh / 16, nbw * d.Hq);
  const size_t qsmem = (size_t)d.dh * d.dh * sizeof(float);
  dim3 qgrid(128, d.Hq, d.nb);
  const long long gstride = d.wo_shared ? 0 : (long long)d.Hq * d.dh * d.dh;
  cudaError_t e;
  if (d.dtype == CKV_F32) {
    gram_simt_kernel<float><<<ggrid, 256, 0, st>>>((const float*)WO, G, d.dh, d.dm);
    if ((e = cudaFuncSetAttribute(quad_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)qsmem)) != cudaSuccess)
      return e;
    quad_simt_kernel<float><<<qgrid, 256, qsmem, st>>>((const float*)V, G, vnorm, d.Hq, d.G, d.n, d.dh, d.vs[0],
                                                       d.vs[1], d.vs[2], gstride);
  } else {
    gram_simt_kernel<__nv_bfloat16><<<ggrid, 256, 0, st>>>((const __nv_bfloat16*)WO, G, d.dh, d.dm);
    if ((e = cudaFuncSetAttribute(quad_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)qsmem)) != cudaSuccess)
      return e;
    quad_simt_kernel<__nv_bfloat16><<<qgrid, 256, qsmem, st>>>((const __nv_bfloat16*)V, G, vnorm, d.Hq, d.G, d.n,
                                                               d.dh, d.vs[0], d.vs[1], d.vs[2], gstride);
  }
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace ckv
