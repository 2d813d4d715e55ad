// Stage 4+5: pixel-to-instance assignment (Eq. 4, Eq. 7, Eq. 8) and the label-map write.
//
// Scores are computed in binary32 in the direct-difference form, in one fixed order, so that every
// variant of this kernel gives the same bits for the same (pixel, peak):
//   sx = 0; for c = 0..2F-1: t = xhat_c - P_w[a][c]; sx = fma(t, t, sx)      (likewise sy)
//   d  = sqrt(sx) + sqrt(sy)
// The smallest d wins; on equal d the lowest k.
#pragma once

#include "cpe_common.cuh"

namespace cpe {

constexpr int kAssignThreads = 256;
constexpr int kPeakChunk = 32;  // peaks staged in shared memory per pass

// `bound`: the caller only needs to know d if d < bound.  sqrt(sx) alone already bounds d from below, so when
// sqrt(sx) >= bound the y half is skipped and +inf is returned (the peak cannot beat `bound`; on equality it
// would lose the tie to the earlier peak anyway).  Whenever a finite value is returned it is the full score.
template <int D>
__device__ __forceinline__ float score_direct(const float (&e)[D], const float* __restrict__ pk, float bound) {
  float sx = 0.0f, sy = 0.0f;
#pragma unroll
  for (int c = 0; c < D / 2; c += 4) {
    const float4 a = *reinterpret_cast<const float4*>(pk + c);
    float t;
    t = __fsub_rn(e[c + 0], a.x); sx = __fmaf_rn(t, t, sx);
    t = __fsub_rn(e[c + 1], a.y); sx = __fmaf_rn(t, t, sx);
    t = __fsub_rn(e[c + 2], a.z); sx = __fmaf_rn(t, t, sx);
    t = __fsub_rn(e[c + 3], a.w); sx = __fmaf_rn(t, t, sx);
  }
  const float dx = __fsqrt_rn(sx);
  // warp-uniform skip: the y half is only worth its 2F fused multiply-adds if some lane can still use it
  if (!__any_sync(__activemask(), dx < bound)) return __int_as_float(0x7f800000);
#pragma unroll
  for (int c = 0; c < D / 2; c += 4) {
    const float4 g = *reinterpret_cast<const float4*>(pk + D / 2 + c);
    float t;
    t = __fsub_rn(e[D / 2 + c + 0], g.x); sy = __fmaf_rn(t, t, sy);
    t = __fsub_rn(e[D / 2 + c + 1], g.y); sy = __fmaf_rn(t, t, sy);
    t = __fsub_rn(e[D / 2 + c + 2], g.z); sy = __fmaf_rn(t, t, sy);
    t = __fsub_rn(e[D / 2 + c + 3], g.w); sy = __fmaf_rn(t, t, sy);
  }
  return __fadd_rn(dx, __fsqrt_rn(sy));
}

// Generic-F version of the same arithmetic (any F in [1,16]); e lives in local memory.
__device__ __forceinline__ float score_direct_rt(const float* e, const float* __restrict__ pk, int F) {
  float sx = 0.0f, sy = 0.0f;
  for (int c = 0; c < 2 * F; ++c) {
    const float t = __fsub_rn(e[c], pk[c]);
    sx = __fmaf_rn(t, t, sx);
  }
  for (int c = 0; c < 2 * F; ++c) {
    const float t = __fsub_rn(e[2 * F + c], pk[2 * F + c]);
    sy = __fmaf_rn(t, t, sy);
  }
  return __fadd_rn(__fsqrt_rn(sx), __fsqrt_rn(sy));
}

// One thread per pixel; the pixel's 4F values stay in registers while the peaks stream through shared
// memory in chunks (the paper's mask-aggregation design point: all candidates of a pixel are evaluated
// by one thread with the pixel's data held on chip).  FT in {4, 8, 16} fixes F; FT = 0 is the generic path.
template <typename T, int FT>
__global__ void __launch_bounds__(kAssignThreads)
assign_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F_rt, int K_max,
              const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau,
              int32_t* __restrict__ labels, float* __restrict__ best, float* __restrict__ second,
              uint32_t* __restrict__ counters, uint32_t* __restrict__ votes, int cells, int k_limit) {
  constexpr int DT = FT > 0 ? 4 * FT : 64;
  const int F = FT > 0 ? FT : F_rt;
  const int D = 4 * F;
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  const long long n = (long long)blockIdx.x * kAssignThreads + tid;
  const size_t plane = (size_t)HW;
  const int K = count_ptr[b];
  if (K > k_limit) return;   // this image is left to the tensor-core kernel launched next to this one
  const float* pk_img = peak_emb + (size_t)b * K_max * D;

  __shared__ __align__(16) float s_pk[kPeakChunk * 64];
  __shared__ uint32_t s_rejected;
  if (tid == 0) s_rejected = 0;
  // the vote map has no reader left: leave it zero for the next decode (votes == NULL keeps it)
  if (votes) zero_votes_share(votes + (size_t)b * cells, cells, (int)blockIdx.x, (int)gridDim.x);

  bool act = n < HW;
  if (act && fg) act = __ldg(fg + (size_t)b * plane + n) != 0;
  float e[DT];
  if (act) {
    const T* p = emb + (size_t)b * D * plane + n;
    bool ok = true;
    if constexpr (FT > 0) {
#pragma unroll
      for (int c = 0; c < DT; ++c) e[c] = Elem<T>::load1(p + (size_t)c * plane);
#pragma unroll
      for (int c = 0; c < DT; c += 2) ok = ok && pair_finite(e[c], e[c + 1]);
    } else {
      for (int c = 0; c < D; ++c) e[c] = Elem<T>::load1(p + (size_t)c * plane);
      for (int c = 0; c < D; c += 2) ok = ok && pair_finite(e[c], e[c + 1]);
    }
    act = ok;
  }

  const float inf = __int_as_float(0x7f800000);
  float d1 = inf, d2 = inf;
  int k1 = -1;
  for (int k0 = 0; k0 < K; k0 += kPeakChunk) {
    const int kn = min(kPeakChunk, K - k0);
    __syncthreads();
    for (int i = tid; i < kn * D; i += kAssignThreads) s_pk[i] = pk_img[(size_t)k0 * D + i];
    __syncthreads();
    if (act) {
      for (int kk = 0; kk < kn; ++kk) {
        float d;
        // only distances below the current runner-up (or best, when no scores are stored) matter
        if constexpr (FT > 0) d = score_direct<DT>(e, s_pk + kk * DT, best ? d2 : d1);
        else d = score_direct_rt(e, s_pk + kk * D, F);
        if (d < d1) { d2 = d1; d1 = d; k1 = k0 + kk; }
        else if (d < d2) { d2 = d; }
      }
    }
  }

  int label = 0;
  bool rejected = false;
  if (act && k1 >= 0) {
    if (d1 < tau) label = k1 + 1;
    else rejected = true;
  }
  if (n < HW) {
    const size_t o = (size_t)b * plane + n;
    labels[o] = label;
    if (best) {
      best[o] = act ? d1 : inf;
      second[o] = act ? d2 : inf;
    }
  }
  const uint32_t rej = __ballot_sync(0xffffffffu, rejected);
  if (rej && (tid & 31) == 0) atomicAdd(&s_rejected, (uint32_t)__popc(rej));
  __syncthreads();
  if (tid == 0 && s_rejected) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_TAU_REJECTED], s_rejected);
}

}  // namespace cpe
