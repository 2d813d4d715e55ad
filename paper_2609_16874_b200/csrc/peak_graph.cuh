// Between stage 3 and stage 4: for every peak, the short list of candidates that can win the arg-min of Eq. 7 for a
// pixel near that peak.
//
// Let g be any vector ("reference point") and e_k the candidate rows.  With the per-axis norms of Eq. 4,
//     G_k = ||g_x - e_k,x|| + ||g_y - e_k,y||        t = ||xhat - g_x|| + ||yhat - g_y||
// the triangle inequality gives, axis by axis, |d_k - G_k| <= t for the pixel's distance d_k to candidate k.  So once
// some candidate has been scored exactly with distance U, every k with G_k - t > U is out, whatever the pixel.  G
// depends on the peaks only: this kernel computes it for g = the reference point of peak k0 (gamma of the mean
// estimate of the peak's 3x3 window of bins, the refined centroid) against all candidates of the image, and keeps the
// kNbrCap smallest in ascending order (a sort in shared memory), so that the assignment scans a list until G exceeds U + t and stops.
//
// A list entry is (Gq << 12) | k with Gq = floor(G * 2^16 * (1 - 2^-15)), i.e. G rounded DOWN by more than its own
// rounding error (at most (2F + 3) units in the last place), as the bound needs; entries ascend as plain integers.
// Unused entries are 0xffffffff.  Also written: the reference and candidate rows with their x and y halves
// interleaved, row[2c] = x channel c, row[2c + 1] = y channel c, the operand layout of score_direct, and binary16
// copies of the rows in plain order for the streaming kernel's bounds.
#pragma once

#include <cuda_fp16.h>

#include "cpe_common.cuh"

namespace cpe {

constexpr int kGraphThreads = 256;
constexpr uint32_t kNbrEnd = 0xffffffffu;

// One CTA per peak k0 (the grid strides over the peaks); its threads share the candidates.
template <int FT>
__global__ void __launch_bounds__(kGraphThreads)
peak_graph_kernel(const float* __restrict__ ref_emb, const float* __restrict__ cand_emb,
                  const int32_t* __restrict__ count_ptr, int K_max, int k_min, float* __restrict__ ref2,
                  float* __restrict__ cand2, __half* __restrict__ ref_h, __half* __restrict__ cand_h,
                  uint32_t* __restrict__ nbr, long long* __restrict__ sums_to_zero, int cells) {
  constexpr int D = 4 * FT, D2 = 2 * FT;
  __shared__ __align__(16) float s_ref[D];                    // plain order: x half, y half
  __shared__ __align__(16) uint32_t s_keys[kNearMaxPeaks];
  grid_dependency_sync();
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  // the per-bin sums have no reader left (the kernel before this one was the last): this CTA's share of them is left
  // zero for the next decode, which then needs no clearing pass (sums_to_zero == NULL keeps them)
  if (sums_to_zero) {
    uint4* z = reinterpret_cast<uint4*>(sums_to_zero + (size_t)b * cells * 2);      // 16 bytes per bin
    for (int i = blockIdx.x * kGraphThreads + tid; i < cells; i += gridDim.x * kGraphThreads) z[i] = make_uint4(0, 0, 0, 0);
  }
  const int K = count_ptr[b];
  if (K < k_min || K > kNearMaxPeaks) return;
  const float* ref_img = ref_emb + (size_t)b * K_max * D;
  const float* cand_img = cand_emb + (size_t)b * K_max * D;
  const bool same = ref2 == cand2;
  const int Kpad = (K + 3) & ~3;

  for (int k0 = blockIdx.x; k0 < K; k0 += gridDim.x) {
    // this peak's rows: a plain copy for the distances below, interleaved copies for the assignment
    for (int c = tid; c < D; c += kGraphThreads) {
      const float r = ref_img[(size_t)k0 * D + c];
      s_ref[c] = r;
      const int dst = c < D2 ? 2 * c : 2 * (c - D2) + 1;
      ref2[((size_t)b * K_max + k0) * D + dst] = r;
      ref_h[((size_t)b * K_max + k0) * D + c] = __float2half_rn(r);
      if (!same) {
        const float e = cand_img[(size_t)k0 * D + c];
        cand2[((size_t)b * K_max + k0) * D + dst] = e;
        cand_h[((size_t)b * K_max + k0) * D + c] = __float2half_rn(e);
      }
    }
    __syncthreads();
    // G(k0, k) for this thread's candidates: a row is fetched with independent 128-bit loads
    for (int k = tid; k < Kpad; k += kGraphThreads) {
      uint32_t key = kNbrEnd;                                  // padding up to a multiple of four
      if (k < K) {
        const float4* e = reinterpret_cast<const float4*>(cand_img + (size_t)k * D);
        float4 row[D / 4];
#pragma unroll
        for (int q = 0; q < D / 4; ++q) row[q] = __ldg(e + q);
        float sx = 0.0f, sy = 0.0f;
#pragma unroll
        for (int q = 0; q < D2 / 4; ++q) {
          const float4 gx = *reinterpret_cast<const float4*>(&s_ref[4 * q]);
          const float4 gy = *reinterpret_cast<const float4*>(&s_ref[D2 + 4 * q]);
          const float4 ex = row[q], ey = row[D2 / 4 + q];
          float t;
          t = gx.x - ex.x; sx = fmaf(t, t, sx);
          t = gx.y - ex.y; sx = fmaf(t, t, sx);
          t = gx.z - ex.z; sx = fmaf(t, t, sx);
          t = gx.w - ex.w; sx = fmaf(t, t, sx);
          t = gy.x - ey.x; sy = fmaf(t, t, sy);
          t = gy.y - ey.y; sy = fmaf(t, t, sy);
          t = gy.z - ey.z; sy = fmaf(t, t, sy);
          t = gy.w - ey.w; sy = fmaf(t, t, sy);
        }
        const float G = sqrtf(sx) + sqrtf(sy);
        const float q = floorf(G * (65536.0f * (1.0f - 1.0f / 32768.0f)));
        const uint32_t Gq = (uint32_t)fminf(q, 1048575.0f);
        key = (Gq << 12) | (uint32_t)k;
      }
      s_keys[k] = key;
    }
    __syncthreads();
    // the kNbrCap smallest keys in ascending order: a bitonic sort of the keys, padded with end marks to a power of two
    // (keys are distinct -- k is part of them -- so the order is unique)
    int n = kNbrCap;
    while (n < K) n <<= 1;
    for (int k = Kpad + tid; k < n; k += kGraphThreads) s_keys[k] = kNbrEnd;
    __syncthreads();
    // Thread t takes the pairs t, t + 256, ...: while the pair distance j is at most 32, the pairs of a warp lie in 64
    // consecutive keys that no other warp touches, so those steps need no CTA-wide barrier.
    for (int kk = 2; kk <= n; kk <<= 1) {
      for (int j = kk >> 1; j > 0; j >>= 1) {
        for (int t = tid; t < n / 2; t += kGraphThreads) {
          const int i = 2 * t - (t & (j - 1));                 // the pair's lower index: bit j clear
          const uint32_t a = s_keys[i], c = s_keys[i + j];
          const bool ascending = (i & kk) == 0;
          if ((a > c) == ascending) {
            s_keys[i] = c;
            s_keys[i + j] = a;
          }
        }
        if (j > 32 || (j == 1 && kk >= 64)) __syncthreads();   // (the next step's j is kk: beyond the warp's keys)
        else __syncwarp();
      }
    }
    __syncthreads();
    uint32_t* out = nbr + ((size_t)b * K_max + k0) * kNbrCap;
    for (int r = tid; r < kNbrCap; r += kGraphThreads) out[r] = s_keys[r];
    __syncthreads();
  }
}

}  // namespace cpe
