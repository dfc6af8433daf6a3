// Step 5: compaction of the retained entries (Algorithm 1, the steps that append the selected entries to the retained cache).
// K_out[nb, r, :] = K[nb, g, idx[nb, r], :] for every r in head g's segment [offsets[g], offsets[g+1]); same for V.
// Pure data movement: every row is copied as 16-byte vectors, one lane per vector, consecutive lanes on consecutive
// vectors of a row (a 256-byte bf16 row of head_dim 128 is 16 lanes), rows of one head read in ascending order.
#include "ckv_internal.h"

namespace ckv {
namespace {

struct CompactArgs {
  const char* K;
  const char* V;
  const int32_t* idx;
  const int32_t* offsets;
  char* K_out;
  char* V_out;
  int Hkv, n;
  int vec_per_row;          // 16-byte vectors per row
  long long btot;
  long long ks[3], vs[3];   // byte strides: nb, head, row
  int* status;              // CKV_FLAG_DEBUG_CHECKS: where a violated bound is reported; null otherwise
};

// offsets must start at 0, never decrease and end within the capacity of idx
__device__ __forceinline__ bool offsets_sane(const int32_t* offs, int Hkv, long long btot) {
  bool ok = offs[0] == 0 && (long long)offs[Hkv] <= btot;
  for (int q = 0; q < Hkv; ++q) ok = ok && offs[q] <= offs[q + 1];
  return ok;
}

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads) compact_kernel(CompactArgs p) {
  __shared__ int32_t offs[65];
  const int b = blockIdx.y;
  for (int q = threadIdx.x; q <= p.Hkv; q += kThreads) offs[q] = p.offsets[(long long)b * (p.Hkv + 1) + q];
  __syncthreads();
  if (p.status != nullptr && threadIdx.x == 0 && blockIdx.x == 0 && !offsets_sane(offs, p.Hkv, p.btot))
    atomicExch(p.status, (int)CKV_EBOUNDS);
  const long long total = min(max((long long)offs[p.Hkv], 0LL), p.btot);
  const int rows_per_cta = kThreads / p.vec_per_row;
  const int lane = threadIdx.x % p.vec_per_row, sub = threadIdx.x / p.vec_per_row;
  if (sub >= rows_per_cta) return;
  for (long long r = (long long)blockIdx.x * rows_per_cta + sub; r < total; r += (long long)gridDim.x * rows_per_cta) {
    int g = 0;
    while (g + 1 < p.Hkv && r >= offs[g + 1]) ++g;
    const int src = p.idx[(long long)b * p.btot + r];
    if (src < 0 || src >= p.n) {   // never read outside the cache; reported when the caller asked for checks
      if (p.status != nullptr && lane == 0) atomicExch(p.status, (int)CKV_EBOUNDS);
      continue;
    }
    const long long ko = b * p.ks[0] + g * p.ks[1] + (long long)src * p.ks[2] + lane * 16LL;
    const long long vo = b * p.vs[0] + g * p.vs[1] + (long long)src * p.vs[2] + lane * 16LL;
    const long long oo = ((long long)b * p.btot + r) * p.vec_per_row * 16LL + lane * 16LL;
    const uint4 kv = *reinterpret_cast<const uint4*>(p.K + ko);
    const uint4 vv = *reinterpret_cast<const uint4*>(p.V + vo);
    *reinterpret_cast<uint4*>(p.K_out + oo) = kv;
    *reinterpret_cast<uint4*>(p.V_out + oo) = vv;
  }
}

__global__ void gather_positions_kernel(const int32_t* __restrict__ pos_in, const int32_t* __restrict__ idx,
                                        const int32_t* __restrict__ offsets, int32_t* __restrict__ pos_out, int Hkv,
                                        int n, long long btot, int* status) {
  __shared__ int32_t offs[65];
  const int b = blockIdx.y;
  for (int q = threadIdx.x; q <= Hkv; q += blockDim.x) offs[q] = offsets[(long long)b * (Hkv + 1) + q];
  __syncthreads();
  if (status != nullptr && threadIdx.x == 0 && blockIdx.x == 0 && !offsets_sane(offs, Hkv, btot))
    atomicExch(status, (int)CKV_EBOUNDS);
  const long long total = min(max((long long)offs[Hkv], 0LL), btot);
  for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < total; r += (long long)gridDim.x * blockDim.x) {
    int g = 0;
    while (g + 1 < Hkv && r >= offs[g + 1]) ++g;
    const int src = idx[(long long)b * btot + r];
    if (src >= 0 && src < n) pos_out[(long long)b * btot + r] = pos_in[((long long)b * Hkv + g) * n + src];
    else if (status != nullptr) atomicExch(status, (int)CKV_EBOUNDS);
  }
}

}  // namespace

cudaError_t launch_gather_positions(const Dims& d, const int32_t* pos_in, const int32_t* idx, const int32_t* offsets,
                                    int32_t* pos_out, int sm_count, int* status_word, cudaStream_t st,
                                    int* launches) {
  long long ctas = (d.btot + 255) / 256;
  if (ctas < 1) ctas = 1;
  if (ctas > (long long)sm_count * 8) ctas = (long long)sm_count * 8;
  dim3 grid((unsigned)ctas, d.nb);
  gather_positions_kernel<<<grid, 256, 0, st>>>(pos_in, idx, offsets, pos_out, d.Hkv, d.n, d.btot,
                                                d.debug_checks ? status_word : nullptr);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_compact(const Dims& d, const void* K, const void* V, const int32_t* idx, const int32_t* offsets,
                           void* K_out, void* V_out, int sm_count, int* status_word, cudaStream_t st,
                           int* launches) {
  const int es = d.dtype == CKV_F32 ? 4 : 2;
  CompactArgs p;
  p.K = (const char*)K; p.V = (const char*)V; p.idx = idx; p.offsets = offsets;
  p.K_out = (char*)K_out; p.V_out = (char*)V_out;
  p.Hkv = d.Hkv; p.n = d.n; p.btot = d.btot;
  p.status = d.debug_checks ? status_word : nullptr;
  p.vec_per_row = d.dh * es / 16;
  for (int i = 0; i < 3; ++i) { p.ks[i] = d.ks[i] * es; p.vs[i] = d.vs[i] * es; }
  const int rows_per_cta = kThreads / p.vec_per_row;
  long long ctas = (d.btot + rows_per_cta - 1) / rows_per_cta;
  if (ctas < 1) ctas = 1;
  if (ctas > (long long)sm_count * 16) ctas = (long long)sm_count * 16;   // a few waves, grid-stride beyond
  dim3 grid((unsigned)ctas, d.nb);
  compact_kernel<<<grid, kThreads, 0, st>>>(p);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace ckv
