// Step 1 on the tensor cores (bf16): observation-window attention of Algorithm 2 (softmax and scale as in Eq. 2).
//
// The logits of a KV group (G query heads x w window rows, e.g. 4 x 32 = 128 rows) against a tile of 128 keys are one
// tcgen05 MMA shape, so QK^T runs on the tensor cores and the K stream stays memory-bound.  Softmax needs every row's
// maximum and sum before any weight can be normalised, hence two sweeps over K (the second is served from L2 when the
// working set allows):
//   sweep 1 (kStats) : D = Q_g K_tile^T, rows = query rows.  A thread owns one query row, keeps its running (max, sum)
//                      over the key columns it reads from tensor memory, and stores one partial per work item.
//                      The partials are merged by the same combine kernel the CUDA-core path uses.
//   sweep 2 (kProbs) : D = K_tile Q_g^T, rows = keys.  A thread owns one key and sums the normalised weights of the w
//                      window rows of each head straight from its tensor-memory lane: the window mean comes out
//                      without any cross-lane traffic and is written coalesced along the sequence.
// Max-pooling runs afterwards in the shared pooling kernel.
// Windows of 128 or 256 rows: a work item covers only as many query heads of the group as fit 384 query rows (two
// heads, or one), the parts of a group stream the KV head's keys one after another, and sweep 2 reads an accumulator
// in chunks of 64 columns.  Right-aligned ragged heads (valid_from): keys before a head's first real row are masked
// like the causally invisible ones.
//
// Persistent kernel, one CTA per SM: warp 0 streams K tiles (and the group's Q rows, once per work item) with TMA,
// warp 1 issues the MMAs (warps 2-3 only fill the role warpgroup, which gives its registers to the others with
// setmaxnreg), warps 4-11 are two sets of four softmax warps that take alternating accumulators (two
// 256-column TMEM slots), so that the exponentials of one tile overlap the MMAs and TMEM loads of the next.
// The per-element work is one fma and one exp (plus a max in sweep 1): the normaliser 1 / (w * sum) enters sweep 2
// as log2 in the exponent's bias, and every reduction runs as four independent chains.
// All waits are bounded (status word CKV_ETIMEOUT, tensor memory freed, normal return).
#include <cuda_bf16.h>
#include <math.h>

#include "ckv_internal.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace ckv {
namespace {

using namespace ptx;

constexpr int kKeyTile = 128;
// softmax warps per (accumulator, TMEM lane quarter); 2 (columns split between two warps) measured no faster
constexpr int kHalves = 1;
constexpr int kThreads = (4 + 8 * kHalves) * 32;   // warpgroup 0: producer, MMA issuer, two idle warps; then softmax warps
// launch bounds of 384 threads give every thread 168 registers; the role warpgroup hands most of its share to the
// softmax warpgroups, whose 128 accumulator values per thread otherwise leave no room to pipeline the exponentials
constexpr int kRoleRegs = 56, kSoftmaxRegs = 224;
static_assert(kHalves == 1 && 128 * kRoleRegs + 256 * kSoftmaxRegs <= 65536, "register budget of one CTA per SM");
constexpr int kSlotCols = 256;
constexpr int kMaxRowBlocks = 3;  // query rows per work item <= 384
constexpr float kLog2e = 1.4426950408889634f;

enum { kStats = 1, kProbs = 2 };

struct AttnUmmaArgs {
  float* part_m;
  float* part_l;
  const float* rowstat;
  float* abar;
  const int32_t* valid_from;   // [nb, Hkv] or null: first real key of every KV head (keys before it are padding)
  int* status;
  int Hq, Hkv, G, n, nb;
  int Gi;              // query heads per work item: the largest divisor of G with Gi * w <= 384
  int subgroups;       // G / Gi work items share a KV head's key tiles
  int rows;            // Gi * w
  int row_blocks;      // ceil(rows / 128)                          (sweep 1 sub-tiles per key tile)
  int heads_per_group; // heads per MMA in sweep 2 (hg * w <= 256)
  int head_groups;     // ceil(Gi / heads_per_group)                (sweep 2 sub-tiles per key tile)
  int ntiles;          // ceil(n / 128)
  int tiles_per_item;
  int chunks_per_bg;   // work items per (nb, KV head, subgroup)
  int part_stride;     // partial slots per row = 2 * chunks_per_bg
  int kstages;
  int qbufs;           // 1 or 2 shared-memory copies of the group's Q rows (and statistics)
  float c;             // scale * log2(e)
  float scale;
  long long nitems;
};

struct Item {
  int b, g, chunk, t0, t1;
  int h0;   // first query head of the item
};
__device__ __forceinline__ Item decode_item(long long item, const AttnUmmaArgs& a) {
  Item it;
  it.chunk = (int)(item % a.chunks_per_bg);
  long long r = item / a.chunks_per_bg;
  const int sg = (int)(r % a.subgroups);
  r /= a.subgroups;
  it.g = (int)(r % a.Hkv);
  it.b = (int)(r / a.Hkv);
  it.h0 = it.g * a.G + sg * a.Gi;
  it.t0 = it.chunk * a.tiles_per_item;
  it.t1 = min(it.t0 + a.tiles_per_item, a.ntiles);
  return it;
}

// Shared-memory carve-up (byte offsets from the 1024-aligned base).
template <int DH>
struct Layout {
  int q_panel;   // bytes between the 64-element K panels of the Q rows
  int q_bytes;
  int k_off, k_stage;
  int stats_off;  // two buffers of rows * 8 bytes
  int bar_off;
  int total;
  __host__ __device__ Layout(int rows, int kstages, int qbufs) {
    q_panel = rows * 128;
    q_bytes = (q_panel * (DH / 64) + 1023) / 1024 * 1024;
    k_off = qbufs * q_bytes;
    k_stage = kKeyTile * DH * 2;
    stats_off = k_off + kstages * k_stage;
    bar_off = stats_off + 2 * rows * 8;
    bar_off = (bar_off + 15) / 16 * 16;
    total = bar_off + 25 * 8 + 16;
  }
};

template <int DH, int W, int PASS>
__global__ void __launch_bounds__(kThreads, 1)
window_attn_umma_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                        AttnUmmaArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const Layout<DH> L(a.rows, a.kstages, a.qbufs);
  const uint32_t sbase = smem_addr(smem);
  const uint32_t bars = sbase + L.bar_off;
  auto q_full = [&](int s) { return bars + 8u * s; };
  auto q_empty = [&](int s) { return bars + 8u * (2 + s); };
  auto k_full = [&](int s) { return bars + 8u * (4 + s); };
  auto k_empty = [&](int s) { return bars + 8u * (12 + s); };
  auto t_full = [&](int s) { return bars + 8u * (20 + s); };
  auto t_empty = [&](int s) { return bars + 8u * (22 + s); };
  const uint32_t drain_bar = bars + 8u * 24;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L.bar_off + 25 * 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* never = tmem_slot + 2;
  float* stats = reinterpret_cast<float*>(smem + L.stats_off);  // [2][rows]: -max * log2e + log2(1 / (w * sum))

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kKSteps = DH / 16;
  constexpr int kPanels = DH / 64;
  const int nsub = PASS == kStats ? a.row_blocks : a.head_groups;
  const bool flip_tiles = (nsub & 1) == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(q_full(s), 1);
      // a Q buffer is free again when the MMAs of its item have retired and, in the second sweep, when all eight
      // softmax warps are done with the item's statistics
      mbar_init(q_empty(s), PASS == kProbs ? 1 + 8 * kHalves : 1);
    }
    for (int s = 0; s < 8; ++s) {
      mbar_init(k_full(s), 1);
      mbar_init(k_empty(s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(t_full(s), 1);
      mbar_init(t_empty(s), 4 * kHalves);
    }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    *never = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_addr(const_cast<uint32_t*>(tmem_slot)), 2 * kSlotCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  bool failed = false;

  if (warp < 4) {
  warpgroup_reg_dealloc<kRoleRegs>();
  if (warp == 0) {
    // ---------------- producer: Q rows (+ row statistics) per item, K tiles ----------------
    if (lane == 0) {
      prefetch_tensormap(&mapQ);
      prefetch_tensormap(&mapK);
    }
    uint32_t it_k = 0, item_cnt = 0;
    uint32_t armed = 0, last_phase = 0;
    bool q_armed = false;
    uint32_t q_last = 0;
    for (long long item = blockIdx.x; item < a.nitems; item += gridDim.x, ++item_cnt) {
      const Item w = decode_item(item, a);
      const int qb = item_cnt % a.qbufs;
      const uint32_t qph = (item_cnt / a.qbufs) & 1u;
      bool ok = true;
      if (lane == 0) ok = mbar_wait_bounded(q_empty(qb), qph ^ 1u, abort_flag);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { failed = true; break; }
      if (PASS == kProbs) {
        // the normalisation constants of the group's rows, next to the Q buffer they belong to
        float* dst = stats + qb * a.rows;
        for (int r = lane; r < a.rows; r += 32) {
          const long long rowg = ((long long)w.b * a.Hq + w.h0 + r / W) * W + r % W;
          dst[r] = fmaf(-a.rowstat[2 * rowg], kLog2e, log2f(a.rowstat[2 * rowg + 1]));
        }
        __syncwarp();
      }
      if (lane == 0) {
        mbar_arrive_expect_tx(q_full(qb), (uint32_t)(a.rows * DH * 2));
#pragma unroll
        for (int p = 0; p < kPanels; ++p)
          tma_load_4d(sbase + qb * L.q_bytes + p * L.q_panel, &mapQ, p * 64, 0, w.h0, w.b, q_full(qb));
        q_armed = true;
        q_last = (uint32_t)qb | (qph << 1);
        for (int t = w.t0; t < w.t1; ++t, ++it_k) {
          const int s = it_k % a.kstages;
          const uint32_t ph = (it_k / a.kstages) & 1u;
          if (!mbar_wait_bounded(k_empty(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          mbar_arrive_expect_tx(k_full(s), (uint32_t)L.k_stage);
          const uint32_t dst = sbase + L.k_off + s * L.k_stage;
#pragma unroll
          for (int p = 0; p < kPanels; ++p)
            tma_load_4d(dst + p * (kKeyTile * 128), &mapK, p * 64, t * kKeyTile, w.g, w.b, k_full(s));
          armed |= 1u << s;
          last_phase = (last_phase & ~(1u << s)) | (ph << s);
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { failed = true; break; }
    }
    if (failed && lane == 0) {
      if (q_armed) mbar_wait_bounded(q_full(q_last & 1u), q_last >> 1, never, 200000000ull);
      for (int s = 0; s < a.kstages; ++s)
        if (armed & (1u << s)) mbar_wait_bounded(k_full(s), (last_phase >> s) & 1u, never, 200000000ull);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      uint32_t it_k = 0, item_cnt = 0, t = 0;
      uint32_t slot_uses[2] = {0, 0};
      for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x, ++item_cnt) {
        const Item w = decode_item(item, a);
        const int qb = item_cnt % a.qbufs;
        const uint32_t q_addr = sbase + qb * L.q_bytes;
        if (!mbar_wait_bounded(q_full(qb), (item_cnt / a.qbufs) & 1u, abort_flag)) { failed = true; break; }
        for (int kt = w.t0; kt < w.t1 && !failed; ++kt, ++it_k) {
          const int s = it_k % a.kstages;
          if (!mbar_wait_bounded(k_full(s), (it_k / a.kstages) & 1u, abort_flag)) { failed = true; break; }
          const uint32_t k_addr = sbase + L.k_off + s * L.k_stage;
          for (int sub = 0; sub < nsub; ++sub, ++t) {
            // with an even number of sub-tiles per key tile a plain alternation would hand every set the same
            // sub-tiles for ever (e.g. always the wide head group): the assignment flips from tile to tile
            const uint32_t slot = (t + (flip_tiles ? it_k : 0u)) & 1u;
            if (!mbar_wait_bounded(t_empty(slot), (slot_uses[slot] & 1u) ^ 1u, abort_flag)) { failed = true; break; }
            ++slot_uses[slot];
            tc_fence_after();
            uint32_t idesc, a_addr, b_addr, a_panel, b_panel;
            if (PASS == kStats) {
              // rows = query rows [sub*128, sub*128+128) of the group, columns = the 128 keys of the tile
              idesc = idesc_bf16_f32(128, kKeyTile, 0);
              a_addr = q_addr + sub * (128 * 128);
              a_panel = L.q_panel;
              b_addr = k_addr;
              b_panel = kKeyTile * 128;
            } else {
              // rows = the 128 keys of the tile, columns = the window rows of this head group
              const int h0 = sub * a.heads_per_group;
              const int ncols = min(a.heads_per_group, a.Gi - h0) * W;
              idesc = idesc_bf16_f32(128, ncols, 0);
              a_addr = k_addr;
              a_panel = kKeyTile * 128;
              b_addr = q_addr + h0 * W * 128;
              b_panel = L.q_panel;
            }
#pragma unroll
            for (int kk = 0; kk < kKSteps; ++kk) {
              const uint64_t ad = smem_desc_sw128(a_addr + (kk / 4) * a_panel + (kk % 4) * 32, 16, 1024);
              const uint64_t bd = smem_desc_sw128(b_addr + (kk / 4) * b_panel + (kk % 4) * 32, 16, 1024);
              umma_f16(tmem_base + slot * kSlotCols, ad, bd, idesc, kk > 0 ? 1u : 0u);
            }
            umma_commit(t_full(slot));
          }
          if (failed) break;
          umma_commit(k_empty(s));
        }
        if (failed) break;
        umma_commit(q_empty(qb));
      }
      umma_commit(drain_bar);
      mbar_wait_bounded(drain_bar, 0, never, 500000000ull);
    }
  }
  } else {
    warpgroup_reg_alloc<kSoftmaxRegs>();
    // ---------------- softmax warps ----------------
    // warp e = warp - 4: TMEM lane quarter = warp % 4 (fixed by the hardware), accumulator slot ("set") = (e / 4) % 2,
    // column half = e / 8.  A set takes the accumulators with t % 2 == set; its kHalves warps per lane quarter split
    // the columns (sweep 1: keys, sweep 2: heads) between them.
    const int e_id = warp - 4;
    const uint32_t set = (uint32_t)(e_id >> 2) & 1u;
    const int half = e_id >> 3;
    const int quad = warp & 3;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16) + set * kSlotCols;
    const int first_pos = a.n - W;  // sequence position of window row 0
    uint32_t item_cnt = 0, t = 0, uses = 0, tile_cnt = 0;
    for (long long item = blockIdx.x; item < a.nitems && !failed; item += gridDim.x, ++item_cnt) {
      const Item w = decode_item(item, a);
      const int qb = item_cnt % a.qbufs;
      if (PASS == kProbs) {
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(q_full(qb), (item_cnt / a.qbufs) & 1u, abort_flag))) {
          failed = true;
          break;
        }
      }
      const float* st = stats + qb * a.rows;
      const int vf = a.valid_from ? a.valid_from[w.b * a.Hkv + w.g] : 0;
      float rm[kMaxRowBlocks], rl[kMaxRowBlocks];
#pragma unroll
      for (int rb = 0; rb < kMaxRowBlocks; ++rb) { rm[rb] = -INFINITY; rl[rb] = 0.f; }

      for (int kt = w.t0; kt < w.t1 && !failed; ++kt, ++tile_cnt) {
        const int key0 = kt * kKeyTile;
        // some (key, row) pair of this tile is masked: causally (last tiles) or as padding (first tiles)
        const bool tail = key0 + kKeyTile - 1 > first_pos || key0 < vf;
#pragma unroll 1
        for (int sub = 0; sub < nsub; ++sub, ++t) {
          if (((t + (flip_tiles ? tile_cnt : 0u)) & 1u) != set) continue;
          if (!__all_sync(0xffffffffu, mbar_wait_bounded(t_full(set), uses & 1u, abort_flag))) { failed = true; break; }
          ++uses;
          tc_fence_after();
          if (PASS == kStats) {
            constexpr int CW = kKeyTile / kHalves;                // key columns per warp
            const int r = sub * 128 + quad * 32 + lane;           // query row of the group
            const bool warp_live = sub * 128 + quad * 32 < a.rows;
            const int c0 = half * CW;
            float v[CW / 32][32];
            if (warp_live) {
#pragma unroll
              for (int q = 0; q < CW / 32; ++q) tmem_ld_32cols(lane_base + c0 + q * 32, v[q]);
              tc_wait_ld();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(t_empty(set));
            if (warp_live && r < a.rows) {
              if (tail) {
                const int lim = min(first_pos + r % W, a.n - 1);  // last visible key of this row
#pragma unroll
                for (int q = 0; q < CW / 32; ++q)
#pragma unroll
                  for (int e = 0; e < 32; ++e)
                    if (key0 + c0 + q * 32 + e > lim || key0 + c0 + q * 32 + e < vf) v[q][e] = -INFINITY;
              }
              float x0 = -INFINITY, x1 = -INFINITY, x2 = -INFINITY, x3 = -INFINITY;
#pragma unroll
              for (int q = 0; q < CW / 32; ++q)
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                  x0 = fmaxf(x0, v[q][e]);
                  x1 = fmaxf(x1, v[q][e + 1]);
                  x2 = fmaxf(x2, v[q][e + 2]);
                  x3 = fmaxf(x3, v[q][e + 3]);
                }
              const float mx = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
              float m_old = -INFINITY, l_old = 0.f;
#pragma unroll
              for (int rb = 0; rb < kMaxRowBlocks; ++rb)
                if (rb == sub) { m_old = rm[rb]; l_old = rl[rb]; }
              const float m_new = fmaxf(m_old, mx);
              if (m_new > -INFINITY) {
                const float mc = m_new * a.c;
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                for (int q = 0; q < CW / 32; ++q)
#pragma unroll
                  for (int e = 0; e < 32; e += 4) {
                    s0 += ex2_approx(fmaf(v[q][e], a.c, -mc));
                    s1 += ex2_approx(fmaf(v[q][e + 1], a.c, -mc));
                    s2 += ex2_approx(fmaf(v[q][e + 2], a.c, -mc));
                    s3 += ex2_approx(fmaf(v[q][e + 3], a.c, -mc));
                  }
                l_old = l_old * ex2_approx((m_old - m_new) * a.c) + ((s0 + s1) + (s2 + s3));
                m_old = m_new;
              }
#pragma unroll
              for (int rb = 0; rb < kMaxRowBlocks; ++rb)
                if (rb == sub) { rm[rb] = m_old; rl[rb] = l_old; }
            }
          } else {
            const int i = key0 + quad * 32 + lane;               // this thread's key
            const int h0 = sub * a.heads_per_group;
            const int nh = min(a.heads_per_group, a.Gi - h0);
            const int hph = (a.heads_per_group + kHalves - 1) / kHalves;   // heads per column half
            const int hq0 = half * hph, hq1 = min(nh, hq0 + hph);
            if (hq0 >= hq1) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(t_empty(set));
            }
            // the W weights of a (key, head) pair are read from tensor memory in chunks of at most 64 columns
            constexpr int JC = W < 64 ? W : 64;
            for (int hq = hq0; hq < hq1; ++hq) {
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 1
              for (int jc = 0; jc < W; jc += JC) {
                float v[JC / 16][16];
#pragma unroll
                for (int q = 0; q < JC / 16; ++q) tmem_ld_16cols(lane_base + hq * W + jc + q * 16, v[q]);
                tc_wait_ld();
                if (hq == hq1 - 1 && jc + JC >= W) {
                  tc_fence_before();
                  __syncwarp();
                  if (lane == 0) mbar_arrive(t_empty(set));
                }
                // bias_j = -max_j * log2e + log2(1 / (w * sum_j)): one fma and one exp per weight
                const float4* sr = reinterpret_cast<const float4*>(st + (h0 + hq) * W + jc);
                if (!tail) {
#pragma unroll
                  for (int j = 0; j < JC; j += 4) {
                    const float4 bz = sr[j / 4];
                    a0 += ex2_approx(fmaf(v[j / 16][j % 16], a.c, bz.x));
                    a1 += ex2_approx(fmaf(v[(j + 1) / 16][(j + 1) % 16], a.c, bz.y));
                    a2 += ex2_approx(fmaf(v[(j + 2) / 16][(j + 2) % 16], a.c, bz.z));
                    a3 += ex2_approx(fmaf(v[(j + 3) / 16][(j + 3) % 16], a.c, bz.w));
                  }
                } else {
                  // rows jc + j with j < jmin do not see key i; a padding key is seen by no row
                  const int jmin = i >= vf ? i - first_pos - jc : W;
#pragma unroll
                  for (int j = 0; j < JC; j += 4) {
                    const float4 bz = sr[j / 4];
                    a0 += j >= jmin ? ex2_approx(fmaf(v[j / 16][j % 16], a.c, bz.x)) : 0.f;
                    a1 += j + 1 >= jmin ? ex2_approx(fmaf(v[(j + 1) / 16][(j + 1) % 16], a.c, bz.y)) : 0.f;
                    a2 += j + 2 >= jmin ? ex2_approx(fmaf(v[(j + 2) / 16][(j + 2) % 16], a.c, bz.z)) : 0.f;
                    a3 += j + 3 >= jmin ? ex2_approx(fmaf(v[(j + 3) / 16][(j + 3) % 16], a.c, bz.w)) : 0.f;
                  }
                }
              }
              if (i < a.n) a.abar[((long long)w.b * a.Hq + w.h0 + h0 + hq) * a.n + i] = (a0 + a1) + (a2 + a3);
            }
          }
        }
      }
      if (PASS == kProbs && !failed) {
        __syncwarp();
        if (lane == 0) mbar_arrive(q_empty(qb));
      }
      if (PASS == kStats && !failed) {
#pragma unroll
        for (int rb = 0; rb < kMaxRowBlocks; ++rb) {
          const int r = rb * 128 + quad * 32 + lane;
          if (rb < a.row_blocks && r < a.rows) {
            const long long rowg = ((long long)w.b * a.Hq + w.h0 + r / W) * W + r % W;
            const long long o = rowg * a.part_stride + (w.chunk * 2 + set) * kHalves + half;
            a.part_m[o] = rm[rb] * a.scale;
            a.part_l[o] = rl[rb];
          }
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
    tmem_dealloc(tmem_base, 2 * kSlotCols);
  }
}

template <int DH, int W, int PASS>
cudaError_t run_pass(const CUtensorMap& mq, const CUtensorMap& mk, const AttnUmmaArgs& a, int grid,
                     cudaStream_t st) {
  const Layout<DH> L(a.rows, a.kstages, a.qbufs);
  const int smem = L.total + 1024;
  auto k = window_attn_umma_kernel<DH, W, PASS>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  k<<<grid, kThreads, smem, st>>>(mq, mk, a);
  return cudaGetLastError();
}

template <int DH, int W>
cudaError_t run_both(const Dims& d, const CUtensorMap& mq, const CUtensorMap& mk, AttnUmmaArgs& a, int grid,
                     float* attn, const ScoreWorkspace& ws, cudaStream_t st, int* launches) {
  cudaError_t e = run_pass<DH, W, kStats>(mq, mk, a, grid, st);
  if (e != cudaSuccess) return e;
  e = launch_attn_combine(ws.part_m, ws.part_l, ws.rowstat, d.nb * d.Hq * d.w, a.part_stride, d.w, st);
  if (e != cudaSuccess) return e;
  e = run_pass<DH, W, kProbs>(mq, mk, a, grid, st);
  if (e != cudaSuccess) return e;
  e = launch_maxpool(ws.abar, attn, d.n, d.kp, d.nb * d.Hq, st);
  *launches += 4;
  return e;
}

}  // namespace

cudaError_t launch_window_attn_umma(const Dims& d, const void* Qw, const void* K, float* attn,
                                    const ScoreWorkspace& ws, int sm_count, int* status_word, cudaStream_t st,
                                    int* launches) {
  if (d.dtype != CKV_BF16 || tma_encode_fn() == nullptr) return cudaErrorNotSupported;
  if (d.w != 16 && d.w != 32 && d.w != 64 && d.w != 128 && d.w != 256) return cudaErrorNotSupported;
  // a work item covers Gi query heads of a KV head; with long windows the group is split and every part streams
  // the KV head's keys again (from L2 when they are still there)
  int Gi = d.G;
  while (Gi > 1 && (d.G % Gi != 0 || Gi * d.w > 128 * kMaxRowBlocks)) --Gi;
  const int rows = Gi * d.w;
  if (rows > 128 * kMaxRowBlocks) return cudaErrorNotSupported;

  AttnUmmaArgs a;
  a.part_m = ws.part_m; a.part_l = ws.part_l; a.rowstat = ws.rowstat; a.abar = ws.abar; a.status = status_word;
  a.valid_from = d.valid_from;
  a.Hq = d.Hq; a.Hkv = d.Hkv; a.G = d.G; a.n = d.n; a.nb = d.nb;
  a.Gi = Gi;
  a.subgroups = d.G / Gi;
  a.rows = rows;
  a.row_blocks = (rows + 127) / 128;
  // sweep 2: as few MMAs per key tile as an accumulator slot allows, with the heads spread evenly over them (the two
  // sets of softmax warps take turns on the sub-tiles)
  const int max_hpg = kSlotCols / d.w < Gi ? kSlotCols / d.w : Gi;
  a.head_groups = (Gi + max_hpg - 1) / max_hpg;
  a.heads_per_group = (Gi + a.head_groups - 1) / a.head_groups;
  a.ntiles = (d.n + kKeyTile - 1) / kKeyTile;
  // Work items: a KV group's key tiles are cut into chunks of tiles_per_item; CTA x takes the items x, x + grid, ...
  // The sweep lasts as long as the CTA with the most tiles, so the chunk length is chosen to make the last round of
  // items as full as possible (cost of a candidate = rounds * (tiles per item + about half a tile per item for the Q
  // reload and the pipeline restart)); at least 4 key tiles per item, so that the partial statistics (two per item)
  // fit the workspace sized for one partial per 256 keys.
  const long long groups = (long long)d.nb * d.Hkv * a.subgroups;
  const int max_stride = (d.n + kAttnChunk - 1) / kAttnChunk + 2;
  int tpi = 0;
  long long best_cost = 0;
  for (int cand = 4 * kHalves; cand <= 64; ++cand) {
    const long long chunks = (a.ntiles + cand - 1) / cand;
    if (2 * kHalves * chunks > max_stride) continue;
    const long long items = groups * chunks;
    const long long grid_c = items < sm_count ? items : sm_count;
    const long long rounds = (items + grid_c - 1) / grid_c;
    const long long cost = rounds * (2 * (long long)(cand < a.ntiles ? cand : a.ntiles) + 1);
    if (tpi == 0 || cost < best_cost) { tpi = cand; best_cost = cost; }
  }
  if (tpi == 0) return cudaErrorNotSupported;   // workspace layout
  a.tiles_per_item = tpi;
  a.chunks_per_bg = (a.ntiles + tpi - 1) / tpi;
  a.part_stride = 2 * kHalves * a.chunks_per_bg;
  a.nitems = groups * a.chunks_per_bg;
  a.scale = d.scale;
  a.c = d.scale * kLog2e;
  // shared memory: Q rows, then as many K stages as fit (2..8)
  const int q_bytes = ((rows * 128 * (d.dh / 64)) + 1023) / 1024 * 1024;
  const int k_stage = kKeyTile * d.dh * 2;
  const int budget = 225 * 1024 - 2 * rows * 8 - 1024;
  a.qbufs = (budget - 2 * q_bytes) / k_stage >= 3 ? 2 : 1;
  int ks = (budget - a.qbufs * q_bytes) / k_stage;
  if (ks > 8) ks = 8;
  if (ks < 2) return cudaErrorNotSupported;
  a.kstages = ks;

  CUtensorMap mq, mk;
  const cuuint64_t qdims[4] = {(cuuint64_t)d.dh, (cuuint64_t)d.w, (cuuint64_t)d.Hq, (cuuint64_t)d.nb};
  const long long qstr[3] = {d.qs[2], d.qs[1], d.qs[0]};
  const cuuint32_t qbox[4] = {64, (cuuint32_t)d.w, (cuuint32_t)Gi, 1};
  if (!make_bf16_map_4d(&mq, Qw, qdims, qstr, qbox)) return cudaErrorNotSupported;
  const cuuint64_t kdims[4] = {(cuuint64_t)d.dh, (cuuint64_t)d.n, (cuuint64_t)d.Hkv, (cuuint64_t)d.nb};
  const long long kstr[3] = {d.ks[2], d.ks[1], d.ks[0]};
  const cuuint32_t kbox[4] = {64, kKeyTile, 1, 1};
  if (!make_bf16_map_4d(&mk, K, kdims, kstr, kbox)) return cudaErrorNotSupported;

  const int grid = (int)(a.nitems < sm_count ? a.nitems : sm_count);
#define CKV_ATTN_CASE(DHV, WV) \
  if (d.dh == DHV && d.w == WV) return run_both<DHV, WV>(d, mq, mk, a, grid, attn, ws, st, launches);
  CKV_ATTN_CASE(128, 16) CKV_ATTN_CASE(128, 32) CKV_ATTN_CASE(128, 64) CKV_ATTN_CASE(128, 128) CKV_ATTN_CASE(128, 256)
  CKV_ATTN_CASE(64, 16) CKV_ATTN_CASE(64, 32) CKV_ATTN_CASE(64, 64) CKV_ATTN_CASE(64, 128) CKV_ATTN_CASE(64, 256)
#undef CKV_ATTN_CASE
  return cudaErrorNotSupported;
}

}  // namespace ckv
