// Step 2 on the tensor cores with CTA pairs (opt-in variant, CKV_FLAG_CTA_PAIR_MMA): nu[h, i] = sum_c | sum_t
// V[g, i, t] * WO[h, t, c] |  (Algorithm 1, "L1 norm of each row of V W^O"; Theorem 3.3).  Same contraction, epilogue
// and summation order as the single-CTA kernel, but two CTAs of a thread-block cluster share every MMA (tcgen05
// cta_group::2): one instruction covers 256 tokens x kNC columns, each CTA supplies its own 128 tokens of V and only
// HALF of the W^O chunk, which halves the W^O bytes a CTA pulls from L2 and reads from shared memory.
//
// Measured on B200 (head_dim 128, d_model 4096): slower than the single-CTA kernel (27.5 against 24.4 ms per 32
// layers).  With K = head_dim = 128 an accumulator is complete after only eight MMAs, so the hand-over of finished
// accumulators to the epilogue and back is on the critical path; tensor memory holds just two 256-column accumulators,
// and the hand-over now crosses the cluster twice (multicast commit to the partner's epilogue, remote arrival back at
// the leader): the issuing thread waits for a free accumulator 41 % of the time.  Four 128-column accumulators remove
// the wait but 256 x 128 x 16 MMAs run at half rate (operand delivery, as for 128 x 128 x 16 in one CTA).  Kept as a
// tested variant for shapes with a longer K loop per accumulator.
//
// Cluster of two CTAs (rank 0 = leader), persistent, 11 warps per CTA with the roles of the single-CTA kernel:
//   warp 0  B producer : this CTA's half (kNC / 2 columns x dh) of every W^O chunk, kStages deep
//   warp 1  MMA issuer : leader only; owns the (paired) tensor-memory allocation in both CTAs
//   warp 2  A producer : this CTA's kTiles token tiles of the work item
//   warps 3-10 epilogue: two sets of four warps (one warp per 32-lane quarter of tensor memory); set s takes the
//                        accumulators with (m & 1) == s: tcgen05.ld of a finished accumulator, |x| summed into one
//                        register per row
// A work item is (nb slice, query head, block of kTiles * 256 tokens); token tile (2m + rank) belongs to accumulator m
// of CTA `rank`.
// Barriers: "full" barriers (A tiles, W^O stages) live in the leader and collect the bytes of BOTH CTAs' copies (each
// copy names the leader's barrier); "empty" and "accumulator full" barriers exist in both CTAs and are signalled by
// one multicast tcgen05.commit; "accumulator empty" lives in the leader and counts the epilogue warps of both CTAs.
// No copy is multicast: every CTA fetches exactly the bytes it needs itself.
// Every wait is bounded; a CTA that gives up records CKV_ETIMEOUT, lets its copies land, and still takes part in the
// cluster barrier and the paired tensor-memory release at the end.
#include <cuda_bf16.h>

#include "ckv_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace ckv {
namespace {

using namespace ptx;

#ifndef CKV_VP_TILES
#define CKV_VP_TILES 2
#endif
#ifndef CKV_VP_NC
#define CKV_VP_NC 256
#endif
#ifndef CKV_VP_STAGES
#define CKV_VP_STAGES 4
#endif
constexpr int kTiles = CKV_VP_TILES;   // accumulators per CTA = token tiles per CTA and work item
constexpr int kNC = CKV_VP_NC;         // W^O columns per chunk = MMA N (each CTA stages kNC / 2 of them)
constexpr int kStages = CKV_VP_STAGES; // W^O half-chunk ring
static_assert(kTiles * kNC <= 512 && (kNC == 128 || kNC == 256), "accumulators must fit tensor memory");
constexpr int kThreads = 11 * 32;
constexpr int kTmemCols = 512;             // all of tensor memory
constexpr int kItemRows = kTiles * 256;   // tokens per work item

struct PairArgs {
  float* vnorm;
  int* status;
  int Hq, Hkv, G, n, dm, nb;
  int wo_shared;
  int mblocks;      // ceil(n / kItemRows)
  long long nitems;
};

template <int DH>
struct SmemLayout {
  static constexpr int kATile = 128 * DH * 2;          // bytes of one token tile
  static constexpr int kBStage = (kNC / 2) * DH * 2;   // bytes of this CTA's half of a W^O chunk
  static constexpr int kAOff = 0;
  static constexpr int kBOff = kTiles * kATile;
  static constexpr int kBarOff = kBOff + kStages * kBStage;
  static constexpr int kNumBars = 4 * kTiles + 2 * kStages + 1;
  static constexpr int kTotal = kBarOff + kNumBars * 8 + 16;
};

struct Item {
  int b, g, h, row0, pairs;
};
__device__ __forceinline__ Item decode_item(long long item, const PairArgs& a) {
  Item it;
  const int q = (int)(item % a.G);
  long long r = item / a.G;
  const int mblk = (int)(r % a.mblocks);
  r /= a.mblocks;
  it.g = (int)(r % a.Hkv);
  it.b = (int)(r / a.Hkv);
  it.h = it.g * a.G + q;
  it.row0 = mblk * kItemRows;
  const int left = a.n - it.row0;
  it.pairs = left >= kItemRows ? kTiles : (left + 255) / 256;   // 256-token MMA tiles that hold any token
  return it;
}

// Lets copies that were issued shortly before a failure land before the CTA leaves (they are credited to a barrier
// this CTA cannot wait on).
__device__ __forceinline__ void settle_copies() {
  const uint64_t t0 = global_timer_ns();
  while (global_timer_ns() - t0 < 1000000ull) __nanosleep(1000);
}

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
vnorm_umma_pair_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapW,
                       PairArgs a) {
  using L = SmemLayout<DH>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
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
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const long long cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;
  const int nchunks = (a.dm + kNC - 1) / kNC;
  constexpr int kKSteps = DH / 16;
  constexpr int kPanels = DH / 64;

  if (threadIdx.x == 0) {
    for (int m = 0; m < kTiles; ++m) {
      mbar_init(a_full(m), 1);
      mbar_init(a_empty(m), 1);
      mbar_init(t_full(m), 1);
      mbar_init(t_empty(m), 8);      // four epilogue warps of each CTA (used in the leader only)
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
    tmem_alloc_pair(smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers exist before any remote arrival or copy can reach them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  bool failed = false;

  if (warp == 0) {
    // ---------------- B producer: this CTA's half of every W^O chunk ----------------
    if (lane == 0) {
      prefetch_tensormap(&mapW);
      uint32_t it_b = 0;
      uint32_t armed = 0, last_phase = 0;
      bool issued = false;
      for (long long item = cluster_id; item < a.nitems && !failed; item += nclusters) {
        const Item w = decode_item(item, a);
        const int bw = a.wo_shared ? 0 : w.b;
        for (int j = 0; j < nchunks; ++j, ++it_b) {
          const int s = it_b % kStages;
          const uint32_t ph = (it_b / kStages) & 1u;
          if (!mbar_wait_bounded(b_empty(s), ph ^ 1u, abort_flag)) { failed = true; break; }
          if (leader) mbar_arrive_expect_tx(b_full(s), 2 * L::kBStage);
          const uint32_t full_in_leader = map_to_cta(b_full(s), 0);
          const uint32_t dst = sbase + L::kBOff + s * L::kBStage;
#pragma unroll
          for (int nbk = 0; nbk < kNC / 128; ++nbk)   // 64-column blocks of this CTA's half
            tma_load_4d_pair(dst + nbk * (DH * 128), &mapW, j * kNC + (int)rank * (kNC / 2) + nbk * 64, 0, w.h, bw,
                             full_in_leader);
          issued = true;
          armed |= 1u << s;
          last_phase = (last_phase & ~(1u << s)) | (ph << s);
        }
      }
      if (failed) {
        if (leader) {
          for (int s = 0; s < kStages; ++s)
            if (armed & (1u << s)) mbar_wait_bounded(b_full(s), (last_phase >> s) & 1u, never, 200000000ull);
        } else if (issued) {
          settle_copies();
        }
      }
    }
  } else if (warp == 2) {
    // ---------------- A producer: this CTA's token tiles ----------------
    if (lane == 0) {
      prefetch_tensormap(&mapV);
      uint32_t item_cnt = 0;
      int last_tiles = 0;
      for (long long item = cluster_id; item < a.nitems && !failed; item += nclusters, ++item_cnt) {
        const Item w = decode_item(item, a);
        for (int m = 0; m < kTiles; ++m) {
          if (!mbar_wait_bounded(a_empty(m), (item_cnt & 1u) ^ 1u, abort_flag)) { failed = true; break; }
          if (m < w.pairs) {
            if (leader) mbar_arrive_expect_tx(a_full(m), 2 * L::kATile);
            const uint32_t full_in_leader = map_to_cta(a_full(m), 0);
            const uint32_t dst = sbase + L::kAOff + m * L::kATile;
            // rows past the end of the sequence read as zero
#pragma unroll
            for (int p = 0; p < kPanels; ++p)
              tma_load_4d_pair(dst + p * (128 * 128), &mapV, p * 64, w.row0 + (2 * m + (int)rank) * 128, w.g, w.b,
                               full_in_leader);
            last_tiles = m + 1;
          } else if (leader) {
            mbar_arrive(a_full(m));   // tile pair beyond the sequence end: skipped by every role, phase advances
          }
        }
        if (failed) break;   // keep item_cnt at the failing item
      }
      if (failed) {
        if (leader) {
          for (int m = 0; m < last_tiles; ++m) mbar_wait_bounded(a_full(m), item_cnt & 1u, never, 200000000ull);
        } else if (last_tiles > 0) {
          settle_copies();
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = idesc_bf16_f32(256, kNC, 1);
      uint32_t it_b = 0, item_cnt = 0;
      uint32_t use[kTiles];
#pragma unroll
      for (int m = 0; m < kTiles; ++m) use[m] = 0;
      for (long long item = cluster_id; item < a.nitems && !failed; item += nclusters, ++item_cnt) {
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
            if (m < w.pairs) {
              if (!mbar_wait_bounded_cluster(t_empty(m), (use[m] & 1u) ^ 1u, abort_flag)) { failed = true; break; }
              tc_fence_after();
              const uint32_t a_addr = sbase + L::kAOff + m * L::kATile;
#pragma unroll
              for (int kk = 0; kk < kKSteps; ++kk) {
                // descriptors are shared-memory offsets, valid in both CTAs (identical carve-up).  A: K-major 128 rows
                // per CTA.  B: N-major, this CTA's 128 columns as two 64-column blocks DH*128 bytes apart.
                const uint64_t ad = smem_desc_sw128(a_addr + (kk / 4) * (128 * 128) + (kk % 4) * 32, 16, 1024);
                const uint64_t bd = smem_desc_sw128(b_addr + kk * 2048, DH * 128, 1024);
                umma_f16_pair(tmem_base + m * kNC, ad, bd, idesc, kk > 0 ? 1u : 0u);
              }
              umma_commit_pair(t_full(m), 3);
              ++use[m];
            }
            if (j == nchunks - 1) umma_commit_pair(a_empty(m), 3);
          }
          if (failed) break;
          umma_commit_pair(b_empty(s), 3);
        }
      }
      // every MMA issued so far must have retired before tensor memory is released
      umma_commit_pair(drain_bar, 1);
      mbar_wait_bounded(drain_bar, 0, never, 500000000ull);
    }
  } else {
    // ---------------- epilogue: a warp owns TMEM lanes 32*(warp%4) .. +31 of the accumulators of its set ----------
    const int quad = warp & 3;
    const int set = (warp - 3) >> 2;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t empty_in_leader[kTiles];
#pragma unroll
    for (int m = 0; m < kTiles; ++m) empty_in_leader[m] = map_to_cta(t_empty(m), 0);
    uint32_t use = 0;   // bit m: parity of the next phase of t_full(m)
    for (long long item = cluster_id; item < a.nitems && !failed; item += nclusters) {
      const Item w = decode_item(item, a);
      float acc[kTiles];
#pragma unroll
      for (int m = 0; m < kTiles; ++m) acc[m] = 0.f;
      for (int j = 0; j < nchunks && !failed; ++j) {
#pragma unroll
        for (int m = 0; m < kTiles; ++m) {
          if ((m & 1) != set || m >= w.pairs) continue;
          if (!__all_sync(0xffffffffu, mbar_wait_bounded(t_full(m), (use >> m) & 1u, abort_flag))) { failed = true; break; }
          use ^= 1u << m;
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
              if (lane == 0) mbar_arrive_cluster(empty_in_leader[m]);
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
          const int i = w.row0 + (2 * m + (int)rank) * 128 + quad * 32 + lane;
          if ((m & 1) == set && m < w.pairs && i < a.n) a.vnorm[((long long)w.b * a.Hq + w.h) * a.n + i] = acc[m];
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
  cluster_sync_all();   // no CTA leaves (or frees tensor memory) while its partner may still signal or read it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

template <int DH>
cudaError_t run(const CUtensorMap& mv, const CUtensorMap& mw, const PairArgs& a, int sm_count, cudaStream_t st) {
  using L = SmemLayout<DH>;
  const int smem = L::kTotal + 1024;
  auto k = vnorm_umma_pair_kernel<DH>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)(sm_count & ~1));
  int max_clusters = 0;
  e = cudaOccupancyMaxActiveClusters(&max_clusters, k, &cfg);
  if (e != cudaSuccess || max_clusters < 1) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  long long clusters = max_clusters;
  if (clusters > sm_count / 2) clusters = sm_count / 2;
  if (clusters > a.nitems) clusters = a.nitems;
  cfg.gridDim = dim3((unsigned)(2 * clusters));
  e = cudaLaunchKernelEx(&cfg, k, mv, mw, a);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return cudaErrorNotSupported;
  }
  return cudaGetLastError();
}

}  // namespace

// Same contract as launch_vnorm_umma: cudaErrorNotSupported when this layout, device or launch shape cannot take
// the paired kernel (the caller then uses the single-CTA kernel).
cudaError_t launch_vnorm_umma_pair(const Dims& d, const void* V, const void* WO, float* vnorm, int sm_count,
                                   int* status_word, cudaStream_t st, int* launches) {
  if (!vnorm_umma_supported(d) || sm_count < 2) return cudaErrorNotSupported;
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
  PairArgs a;
  a.vnorm = vnorm; a.status = status_word;
  a.Hq = d.Hq; a.Hkv = d.Hkv; a.G = d.G; a.n = d.n; a.dm = d.dm; a.nb = d.nb;
  a.wo_shared = d.wo_shared;
  a.mblocks = (d.n + kItemRows - 1) / kItemRows;
  a.nitems = (long long)d.nb * d.Hq * a.mblocks;
  cudaError_t e = d.dh == 64 ? run<64>(mv, mw, a, sm_count, st) : run<128>(mv, mw, a, sm_count, st);
  if (e == cudaSuccess) *launches += 1;
  return e;
}

}  // namespace ckv
