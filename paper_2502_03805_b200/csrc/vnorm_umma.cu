// Step 2 on the tensor cores: nu[h, i] = sum_c | sum_t V[g, i, t] * WO[h, t, c] |  (Algorithm 1, "L1 norm of each
// row of V W^O"; Theorem 3.3), bf16 inputs, float32 accumulation in tensor memory, and an epilogue that reduces every
// output row to its L1 norm so the n x dm product never leaves the SM.
//
// Persistent kernel, one CTA per SM, 11 warps with fixed roles:
//   warp 0  B producer : TMA loads of W^O_h column chunks (kNC columns x dh), kStages deep
//   warp 1  MMA issuer : tcgen05.mma 128 x kNC x 16, dh/16 per (chunk, token tile); owns the TMEM allocation
//   warp 2  A producer : TMA loads of the work item's kTiles token tiles of V (128 tokens x dh each), resident for
//                        the whole item
//   warps 3-10 epilogue: two sets of four warps (one warp per 32-lane quarter of tensor memory); set s takes the
//                        token tiles with (tile & 1) == s: tcgen05.ld of a finished 128 x kNC accumulator, |x| summed
//                        into one register per row
// A work item is (nb slice, query head, block of kTiles*128 tokens).  Each W^O chunk fetched from L2 is used by all
// kTiles token tiles, which cuts the shared-memory fill per flop by kTiles; the kTiles accumulators (kTiles * kNC =
// 512 columns, all of tensor memory) let the epilogue of one tile overlap the MMAs of the next.
// Shape choice (measured): with 128 x 128 x 16 MMAs both operands stream from shared memory at 128 B/cycle, the
// whole shared-memory bandwidth of the SM, and the tensor pipe idles half of the time (1150 TFLOP/s); 128 x 256 x 16
// needs 96 B/cycle and reaches 1500 TFLOP/s.  Hence kNC = 256 with two token tiles and a two-deep W^O ring.
// Operand layouts: V rows are K-major (dh contiguous); W^O_h is N-major (dm contiguous), consumed directly through an
// MN-major shared-memory descriptor, so no transposed copy of W^O is ever made.  128-byte swizzle on both.
// Every wait is bounded: when one runs out the kernel records CKV_ETIMEOUT in the status word, drains what it has in
// flight, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include "ckv_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace ckv {
namespace {

using namespace ptx;

#ifndef CKV_VN_TILES
#define CKV_VN_TILES 2
#endif
#ifndef CKV_VN_NC
#define CKV_VN_NC 256
#endif
#ifndef CKV_VN_STAGES
#define CKV_VN_STAGES 2
#endif
constexpr int kTiles = CKV_VN_TILES;    // token tiles (128 rows) per work item
constexpr int kNC = CKV_VN_NC;          // W^O columns per chunk = MMA N
constexpr int kStages = CKV_VN_STAGES;  // W^O chunk ring
static_assert(kTiles * kNC <= 512 && kNC % 128 == 0 && kNC <= 256, "accumulators must fit tensor memory");
constexpr int kThreads = 11 * 32;
constexpr int kTmemCols = kTiles * kNC;  // 512

struct UmmaArgs {
  float* vnorm;
  int* status;
  int Hq, Hkv, G, n, dm, nb;
  int wo_shared;
  int mblocks;      // ceil(n / (kTiles*128))
  long long nitems;
};

template <int DH>
struct SmemLayout {
  static constexpr int kATile = 128 * DH * 2;       // bytes of one token tile
  static constexpr int kBStage = kNC * DH * 2;      // bytes of one W^O chunk
  static constexpr int kAOff = 0;
  static constexpr int kBOff = kTiles * kATile;
  static constexpr int kBarOff = kBOff + kStages * kBStage;
  static constexpr int kNumBars = 2 * kTiles + 2 * kStages + 2 * kTiles + 1;
  static constexpr int kTotal = kBarOff + kNumBars * 8 + 16;
};

struct Item {
  int b, g, h, row0, tiles;
};
__device__ __forceinline__ Item decode_item(long long item, const UmmaArgs& a) {
  Item it;
  const int q = (int)(item % a.G);
  long long r = item / a.G;
  const int mblk = (int)(r % a.mblocks);
  r /= a.mblocks;
  it.g = (int)(r % a.Hkv);
  it.b = (int)(r / a.Hkv);
  it.h = it.g * a.G + q;
  it.row0 = mblk * kTiles * 128;
  const int left = a.n - it.row0;
  it.tiles = left >= kTiles * 128 ? kTiles : (left + 127) / 128;
  return it;
}

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
vnorm_umma_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapW, UmmaArgs a) {
  using L = SmemLayout<DH>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // 128-byte swizzle wants 1024-byte aligned tiles
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_addr(smem);
  const uint32_t bars = sbase + L::kBarOff;
  auto a_full = [&](int m) { return bars + 8u * m; };
  auto a_empty = [&](int m) { return bars + 8u * (kTiles + m); };
  auto b_full = [&](int s) { return bars + 8u * (2 * kTiles + s); };
  auto b_empty = [&](int s) { return bars + 8u * (2 * kTiles + kStages + s); };
  auto t_full = [&](int m) { return bars + 8u * (2 * kTiles + 2 * kStages + m); };
  auto t_empty = [&](int m) { return bars + 8u * (3 * kTiles + 2 * kStages + m); };
  const uint32_t drain_bar = bars + 8u * (4 * kTiles + 2 * kStages);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::kBarOff + L::kNumBars * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* never = tmem_slot + 2;   // stays 0: for the drain waits, which must not be cut short

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nchunks = (a.dm + kNC - 1) / kNC;
  constexpr int kKSteps = DH / 16;
  constexpr int kPanels = DH / 64;            // 64-element (128-byte) K panels of an A tile

  if (threadIdx.x == 0) {
    for (int m = 0; m < kTiles; ++m) {
      mbar_init(a_full(m), 1);
      mbar_init(a_empty(m), 1);
      mbar_init(t_full(m), 1);
      mbar_init(t_empty(m), 4);
    }
    for (int s = 0; s < kStages; ++s) {
      mbar_init(b_full(s), 1);
      mbar_init(b_empty(s), 1);
    }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    *never = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  bool failed = false;

  if (warp == 0) {
    // ---------------- B producer: W^O chunks ----------------
    if (lane == 0) {
      prefetch_tensormap(&mapW);
      uint32_t it_b = 0;
      uint32_t armed = 0;            // bit s set: stage s has been armed at least once
      uint32_t last_phase = 0;       // bit s: parity of the phase stage s was last armed for
      for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x) {
        const Item w = decode_item(item, a);
        const int bw = a.wo_shared ? 0 : w.b;
        for (int j = 0; j < nchunks; ++j, ++it_b) {
          const int s = it_b % kStages;
          const uint32_t ph = (it_b / kStages) & 1u;
          if (!mbar_wait_bounded(b_empty(s), ph ^ 1u, abort_flag)) { failed = true; break; }
          mbar_arrive_expect_tx(b_full(s), L::kBStage);
          const uint32_t dst = sbase + L::kBOff + s * L::kBStage;
#pragma unroll
          for (int nbk = 0; nbk < kNC / 64; ++nbk)
            tma_load_4d(dst + nbk * (DH * 128), &mapW, j * kNC + nbk * 64, 0, w.h, bw, b_full(s));
          armed |= 1u << s;
          last_phase = (last_phase & ~(1u << s)) | (ph << s);
        }
      }
      if (failed) {
        // a consumer may never look at these stages again: wait for the copies themselves before leaving
        for (int s = 0; s < kStages; ++s)
          if (armed & (1u << s)) mbar_wait_bounded(b_full(s), (last_phase >> s) & 1u, never, 200000000ull);
      }
    }
  } else if (warp == 2) {
    // ---------------- A producer: token tiles of V ----------------
    if (lane == 0) {
      prefetch_tensormap(&mapV);
      uint32_t item_cnt = 0;
      int last_tiles = 0;
      for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x, ++item_cnt) {
        const Item w = decode_item(item, a);
        for (int m = 0; m < w.tiles; ++m) {
          if (!mbar_wait_bounded(a_empty(m), (item_cnt & 1u) ^ 1u, abort_flag)) { failed = true; break; }
          mbar_arrive_expect_tx(a_full(m), L::kATile);
          const uint32_t dst = sbase + L::kAOff + m * L::kATile;
#pragma unroll
          for (int p = 0; p < kPanels; ++p)
            tma_load_4d(dst + p * (128 * 128), &mapV, p * 64, w.row0 + m * 128, w.g, w.b, a_full(m));
          last_tiles = m + 1;
        }
        // tiles beyond the sequence end are skipped by every role, but their phase must still advance
        for (int m = w.tiles; m < kTiles && !failed; ++m) {
          if (!mbar_wait_bounded(a_empty(m), (item_cnt & 1u) ^ 1u, abort_flag)) { failed = true; break; }
          mbar_arrive(a_full(m));
        }
        if (failed) break;   // keep item_cnt at the failing item
      }
      if (failed) {
        for (int m = 0; m < last_tiles; ++m) mbar_wait_bounded(a_full(m), item_cnt & 1u, never, 200000000ull);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(128, kNC, 1);
      uint32_t it_b = 0, item_cnt = 0;
      uint32_t use[kTiles];
#pragma unroll
      for (int m = 0; m < kTiles; ++m) use[m] = 0;
      for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x, ++item_cnt) {
        const Item w = decode_item(item, a);
        for (int j = 0; j < nchunks && !failed; ++j, ++it_b) {
          const int s = it_b % kStages;
          const uint32_t ph = (it_b / kStages) & 1u;
          if (!mbar_wait_bounded(b_full(s), ph, abort_flag)) { failed = true; break; }
          const uint32_t b_addr = sbase + L::kBOff + s * L::kBStage;
#pragma unroll
          for (int m = 0; m < kTiles; ++m) {
            if (j == 0) {
              if (!mbar_wait_bounded(a_full(m), item_cnt & 1u, abort_flag)) { failed = true; break; }
            }
            if (m < w.tiles) {
              if (!mbar_wait_bounded(t_empty(m), (use[m] & 1u) ^ 1u, abort_flag)) { failed = true; break; }
              tc_fence_after();
              const uint32_t a_addr = sbase + L::kAOff + m * L::kATile;
#pragma unroll
              for (int kk = 0; kk < kKSteps; ++kk) {
                // A: K-major, 8-row groups 1024 bytes apart; step of 16 elements = 32 bytes inside a 128-byte row,
                //    next 64-element panel = next 128-row block.  B: N-major, 64-column blocks DH*128 bytes apart
                //    (leading offset), 8-row K groups 1024 bytes apart (stride offset); 16 K rows = 2048 bytes.
                const uint64_t ad = smem_desc_sw128(a_addr + (kk / 4) * (128 * 128) + (kk % 4) * 32, 16, 1024);
                const uint64_t bd = smem_desc_sw128(b_addr + kk * 2048, DH * 128, 1024);
                umma_f16(tmem_base + m * kNC, ad, bd, idesc, kk > 0 ? 1u : 0u);
              }
              umma_commit(t_full(m));
              ++use[m];
            }
            if (j == nchunks - 1) umma_commit(a_empty(m));
          }
          if (failed) break;
          umma_commit(b_empty(s));
        }
      }
      // every MMA issued so far must have retired before tensor memory is released
      umma_commit(drain_bar);
      mbar_wait_bounded(drain_bar, 0, never, 500000000ull);
    }
  } else {
    // ---------------- epilogue: a warp owns TMEM lanes 32*(warp%4) .. +31 of the tiles of its set ----------------
    const int quad = warp & 3;
    const int set = (warp - 3) >> 2;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t use[kTiles];
#pragma unroll
    for (int m = 0; m < kTiles; ++m) use[m] = 0;
    for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x) {
      const Item w = decode_item(item, a);
      float acc[kTiles];
#pragma unroll
      for (int m = 0; m < kTiles; ++m) acc[m] = 0.f;
      for (int j = 0; j < nchunks && !failed; ++j) {
#pragma unroll
        for (int m = 0; m < kTiles; ++m) {
          if ((m & 1) != set || m >= w.tiles) continue;
          // the warp must stay converged for the .sync.aligned loads: all lanes succeed or all give up
          if (!__all_sync(0xffffffffu, mbar_wait_bounded(t_full(m), use[m] & 1u, abort_flag))) { failed = true; break; }
          ++use[m];
          tc_fence_after();
#pragma unroll
          for (int half = 0; half < kNC / 128; ++half) {
            float v[4][32];
#pragma unroll
            for (int q = 0; q < 4; ++q) tmem_ld_32cols(lane_base + m * kNC + half * 128 + q * 32, v[q]);
            tc_wait_ld();
            if (half == kNC / 128 - 1) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(t_empty(m));
            }
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              s0 += fabsf(v[0][e]);
              s1 += fabsf(v[1][e]);
              s2 += fabsf(v[2][e]);
              s3 += fabsf(v[3][e]);
            }
            acc[m] += (s0 + s1) + (s2 + s3);
          }
        }
      }
      if (!failed) {
#pragma unroll
        for (int m = 0; m < kTiles; ++m) {
          const int i = w.row0 + m * 128 + quad * 32 + lane;
          if ((m & 1) == set && m < w.tiles && i < a.n) a.vnorm[((long long)w.b * a.Hq + w.h) * a.n + i] = acc[m];
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
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int DH>
cudaError_t run(const Dims& d, const CUtensorMap& mv, const CUtensorMap& mw, const UmmaArgs& a, int sm_count,
                cudaStream_t st) {
  using L = SmemLayout<DH>;
  const int smem = L::kTotal + 1024;
  auto k = vnorm_umma_kernel<DH>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  const long long grid = a.nitems < sm_count ? a.nitems : sm_count;
  k<<<(unsigned)grid, kThreads, smem, st>>>(mv, mw, a);
  return cudaGetLastError();
}

}  // namespace

bool vnorm_umma_supported(const Dims& d) {
  return d.dtype == CKV_BF16 && (d.dh == 64 || d.dh == 128) && d.vs[2] >= d.dh && tma_encode_fn() != nullptr;
}

// Returns cudaErrorNotSupported when the tensor maps cannot be encoded for this layout (caller falls back to the
// CUDA-core kernel); any other error is a real launch failure.
cudaError_t launch_vnorm_umma(const Dims& d, const void* V, const void* WO, float* vnorm, int sm_count,
                              int* status_word, cudaStream_t st, int* launches) {
  if (!vnorm_umma_supported(d)) return cudaErrorNotSupported;
  CUtensorMap mv, mw;
  const cuuint64_t vdims[4] = {(cuuint64_t)d.dh, (cuuint64_t)d.n, (cuuint64_t)d.Hkv, (cuuint64_t)d.nb};
  const long long vstr[3] = {d.vs[2], d.vs[1], d.vs[0]};
  const cuuint32_t vbox[4] = {64, 128, 1, 1};
  if (!make_bf16_map_4d(&mv, V, vdims, vstr, vbox)) return cudaErrorNotSupported;
  const int nbw = d.wo_shared ? 1 : d.nb;
  const cuuint64_t wdims[4] = {(cuuint64_t)d.dm, (cuuint64_t)d.dh, (cuuint64_t)d.Hq, (cuuint64_t)nbw};
  const long long wstr[3] = {d.dm, (long long)d.dh * d.dm, (long long)d.Hq * d.dh * d.dm};
  const cuuint32_t wbox[4] = {64, (cuuint32_t)d.dh, 1, 1};
  if (!make_bf16_map_4d(&mw, WO, wdims, wstr, wbox)) return cudaErrorNotSupported;
  UmmaArgs a;
  a.vnorm = vnorm; a.status = status_word;
  a.Hq = d.Hq; a.Hkv = d.Hkv; a.G = d.G; a.n = d.n; a.dm = d.dm; a.nb = d.nb;
  a.wo_shared = d.wo_shared;
  a.mblocks = (d.n + kTiles * 128 - 1) / (kTiles * 128);
  a.nitems = (long long)d.nb * d.Hq * a.mblocks;
  cudaError_t e = d.dh == 64 ? run<64>(d, mv, mw, a, sm_count, st) : run<128>(d, mv, mw, a, sm_count, st);
  if (e == cudaSuccess) *launches += 1;
  return e;
}

}  // namespace ckv
