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

constexpr int kAssignThreads = 128;
constexpr int kPeakChunk = 32;  // peaks staged in shared memory per pass

// The x chain and the y chain of one (pixel, peak) pair advance together as the two lanes of packed binary32
// instructions: e2[c] = (xhat_c, yhat_c), pk2[c] = (P_w[a][c], P_h[b][c]).  Each lane performs exactly the scalar
// sequence above, so the result has the same bits.
//
// `bound2`: the caller only needs d if d < bound, and passes bound^2 (rounded up).  Since sx + sy <= d^2, a pair with
// sx + sy > bound2 cannot get below the bound: +inf is returned without taking the two IEEE square roots.
template <int D>
__device__ __forceinline__ float score_direct(const float2 (&e2)[D / 2], const float2* __restrict__ pk2, float bound2) {
  float2 s = make_float2(0.0f, 0.0f);
#pragma unroll
  for (int c = 0; c < D / 2; c += 2) {
    const float4 q = *reinterpret_cast<const float4*>(pk2 + c);
    float2 t = sub2_rn(e2[c], make_float2(q.x, q.y));
    s = fma2_rn(t, t, s);
    t = sub2_rn(e2[c + 1], make_float2(q.z, q.w));
    s = fma2_rn(t, t, s);
  }
  if (s.x + s.y > bound2) return __int_as_float(0x7f800000);
  return __fadd_rn(__fsqrt_rn(s.x), __fsqrt_rn(s.y));
}

// Four peaks at once: four independent chains keep the FMA pipe busy (one chain alone waits on its own latency).
// Peaks beyond `kn` must not be passed (the caller pads the shared-memory chunk with copies of a valid peak).
// ROW2 = distance between two of the four rows, in float2 units.
template <int D, int ROW2 = D / 2>
__device__ __forceinline__ void score_direct4(const float2 (&e2)[D / 2], const float2* __restrict__ pk2, float bound2,
                                              float (&d)[4]) {
  float2 s[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) s[j] = make_float2(0.0f, 0.0f);
#pragma unroll
  for (int c = 0; c < D / 2; c += 2) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 q = *reinterpret_cast<const float4*>(pk2 + j * ROW2 + c);
      float2 t = sub2_rn(e2[c], make_float2(q.x, q.y));
      s[j] = fma2_rn(t, t, s[j]);
      t = sub2_rn(e2[c + 1], make_float2(q.z, q.w));
      s[j] = fma2_rn(t, t, s[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j)
    d[j] = (s[j].x + s[j].y > bound2) ? __int_as_float(0x7f800000) : __fadd_rn(__fsqrt_rn(s[j].x), __fsqrt_rn(s[j].y));
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

// One thread per pixel (a CTA walks blocks of 128 pixels); the pixel's 4F values stay in registers while the peaks
// stream through shared memory in chunks (the paper's mask-aggregation design point: all candidates of a pixel are evaluated
// by one thread with the pixel's data held on chip).  FT in {4, 8, 16} fixes F; FT = 0 is the generic path.
template <typename T, int FT>
__global__ void __launch_bounds__(kAssignThreads)
assign_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F_rt, int K_max,
              const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau,
              int32_t* __restrict__ labels, float* __restrict__ best, float* __restrict__ second,
              uint32_t* __restrict__ counters, uint32_t* __restrict__ votes, int cells, int k_limit) {
  grid_dependency_sync();
  constexpr int DT = FT > 0 ? 4 * FT : 64;
  const int F = FT > 0 ? FT : F_rt;
  const int D = 4 * F;
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  const size_t plane = (size_t)HW;
  const int K = count_ptr[b];
  if (K > k_limit) return;   // this image is left to the tensor-core kernel launched next to this one
  const float* pk_img = peak_emb + (size_t)b * K_max * D;

  __shared__ __align__(16) float s_pk[kPeakChunk * 64];
  __shared__ uint32_t s_rejected;
  if (tid == 0) s_rejected = 0;
  // the vote map has no reader left: leave it zero for the next decode (votes == NULL keeps it)
  if (votes) zero_votes_share(votes + (size_t)b * cells, cells, (int)blockIdx.x, (int)gridDim.x);

  // peaks k0 .. k0 + kn - 1 into shared memory
  auto stage_peaks = [&](int k0, int kn) {
    if constexpr (FT > 0) {
      // interleave the peak's two halves: s_pk[kk][2c] = P_w[a][c], s_pk[kk][2c+1] = P_h[b][c]
      for (int i = tid; i < kn * D; i += kAssignThreads) {
        const int kk = i / D, j = i - kk * D, c = j >> 1;
        s_pk[i] = pk_img[(size_t)(k0 + kk) * D + ((j & 1) ? D / 2 + c : c)];
      }
    } else {
      for (int i = tid; i < kn * D; i += kAssignThreads) s_pk[i] = pk_img[(size_t)k0 * D + i];
    }
  };
  const bool one_chunk = K <= kPeakChunk;     // the usual case: staged once for all of this CTA's pixel blocks
  if (one_chunk) stage_peaks(0, K);
  __syncthreads();

  const float inf = __int_as_float(0x7f800000);
  uint32_t n_rejected = 0;
  const long long n_blocks = ((long long)HW + kAssignThreads - 1) / kAssignThreads;
  // a CTA walks pixel blocks with the grid's stride (the grid is a few CTAs per SM: an image that is not this
  // kernel's costs a handful of CTAs that exit, not one per 128 pixels)
  for (long long blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
    const long long n = blk * kAssignThreads + tid;
    bool act = n < HW;
    if (act && fg) act = __ldg(fg + (size_t)b * plane + n) != 0;
    float e[FT > 0 ? 1 : DT];          // generic path: channel order
    float2 e2[DT / 2];                 // fixed-F path: (x channel c, y channel c) pairs
    if (act) {
      const T* p = emb + (size_t)b * D * plane + n;
      bool ok = true;
      if constexpr (FT > 0) {
#pragma unroll
        for (int c = 0; c < DT / 2; ++c) {
          e2[c].x = Elem<T>::load1(p + (size_t)c * plane);
          e2[c].y = Elem<T>::load1(p + (size_t)(DT / 2 + c) * plane);
        }
#pragma unroll
        for (int c = 0; c < DT / 2; c += 2) {
          ok = ok && pair_finite(e2[c].x, e2[c + 1].x);
          ok = ok && pair_finite(e2[c].y, e2[c + 1].y);
        }
      } else {
        for (int c = 0; c < D; ++c) e[c] = Elem<T>::load1(p + (size_t)c * plane);
        for (int c = 0; c < D; c += 2) ok = ok && pair_finite(e[c], e[c + 1]);
      }
      act = ok;
    }

    float d1 = inf, d2 = inf;
    float bound2 = inf;   // square of the distance a peak has to beat (the runner-up when scores are stored), rounded up
    int k1 = -1;
    for (int k0 = 0; k0 < K; k0 += kPeakChunk) {
      const int kn = min(kPeakChunk, K - k0);
      if (!one_chunk) {
        __syncthreads();
        stage_peaks(k0, kn);
        __syncthreads();
      }
      if (act) {
        int kk = 0;
        if constexpr (FT > 0) {
          for (; kk + 4 <= kn; kk += 4) {
            float d[4];
            score_direct4<DT>(e2, reinterpret_cast<const float2*>(s_pk + kk * DT), bound2, d);
#pragma unroll
            for (int j = 0; j < 4; ++j) {     // in ascending k: the lowest k keeps an exact tie
              if (d[j] < d1) { d2 = d1; d1 = d[j]; k1 = k0 + kk + j; }
              else if (d[j] < d2) { d2 = d[j]; }
            }
            const float bound = best ? d2 : d1;
            bound2 = bound * bound * (1.0f + 1e-6f);
          }
        }
        for (; kk < kn; ++kk) {
          float d;
          if constexpr (FT > 0) d = score_direct<DT>(e2, reinterpret_cast<const float2*>(s_pk + kk * DT), bound2);
          else d = score_direct_rt(e, s_pk + kk * D, F);
          if (d < d1) { d2 = d1; d1 = d; k1 = k0 + kk; }
          else if (d < d2) { d2 = d; }
          const float bound = best ? d2 : d1;
          bound2 = bound * bound * (1.0f + 1e-6f);
        }
      }
    }

    int label = 0;
    if (act && k1 >= 0) {
      if (d1 < tau) label = k1 + 1;
      else ++n_rejected;
    }
    if (n < HW) {
      const size_t o = (size_t)b * plane + n;
      labels[o] = label;
      if (best) {
        best[o] = act ? d1 : inf;
        second[o] = act ? d2 : inf;
      }
    }
  }
  const uint32_t rej = __reduce_add_sync(0xffffffffu, n_rejected);
  if (rej && (tid & 31) == 0) atomicAdd(&s_rejected, rej);
  __syncthreads();
  if (tid == 0 && s_rejected) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_TAU_REJECTED], s_rejected);
}

}  // namespace cpe
