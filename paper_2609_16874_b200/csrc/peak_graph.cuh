// Between stage 3 and stage 4: for every peak, the short list of candidates that can win the arg-min of Eq. 7 for a
// pixel near that peak.
//
// Let g be any vector ("reference point") and e_k the candidate rows.  With the per-axis norms of Eq. 4,
//     G_k = ||g_x - e_k,x|| + ||g_y - e_k,y||        t = ||xhat - g_x|| + ||yhat - g_y||
// the triangle inequality gives, axis by axis, |d_k - G_k| <= t for the pixel's distance d_k to candidate k.  So once
// some candidate has been scored exactly with distance U, every k with G_k - t > U is out, whatever the pixel.  G
// depends on the peaks only: this kernel computes it for g = the reference point of peak k0 (gamma of the mean
// estimate of the peak's 3x3 window of bins, the refined centroid) against all candidates of the image, and keeps the
// kNbrCap smallest in ascending order, so that the assignment scans a list until G exceeds U + t and stops.
//
// A list entry is (Gq << 12) | k with Gq = floor(G * 2^16 * (1 - 2^-15)), i.e. G rounded DOWN by more than its own
// rounding error (at most (2F + 3) units in the last place), as the bound needs; entries ascend as plain integers.
// Unused entries are 0xffffffff.  Also written: the reference and candidate rows with their x and y halves
// interleaved, row[2c] = x channel c, row[2c + 1] = y channel c, the operand layout of score_direct.
#pragma once

#include "cpe_common.cuh"

namespace cpe {

constexpr int kGraphThreads = 256;
constexpr uint32_t kNbrEnd = 0xffffffffu;

// One warp per peak k0; lanes share the candidates.  Dynamic shared memory: (8 warps) x K_cap keys.
__global__ void __launch_bounds__(kGraphThreads)
peak_graph_kernel(const float* __restrict__ ref_emb, const float* __restrict__ cand_emb,
                  const int32_t* __restrict__ count_ptr, int K_max, int F, int k_min, float* __restrict__ ref2,
                  float* __restrict__ cand2, uint32_t* __restrict__ nbr) {
  extern __shared__ uint32_t s_keys_all[];
  __shared__ float s_ref[kGraphThreads / 32][64];
  grid_dependency_sync();
  const int b = blockIdx.y;
  const int K = count_ptr[b];
  if (K < k_min || K > kNearMaxPeaks) return;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int D = 4 * F, D2 = 2 * F;
  const float* ref_img = ref_emb + (size_t)b * K_max * D;
  const float* cand_img = cand_emb + (size_t)b * K_max * D;
  uint32_t* keys = s_keys_all + (size_t)wid * kNearMaxPeaks;
  const bool same = ref2 == cand2;

  for (int k0 = blockIdx.x * (kGraphThreads / 32) + wid; k0 < K; k0 += gridDim.x * (kGraphThreads / 32)) {
    // this peak's rows, interleaved
    for (int c = lane; c < D; c += 32) {
      const int src = (c & 1) ? D2 + (c >> 1) : (c >> 1);
      const float r = ref_img[(size_t)k0 * D + src];
      s_ref[wid][c] = r;
      ref2[((size_t)b * K_max + k0) * D + c] = r;
      if (!same) cand2[((size_t)b * K_max + k0) * D + c] = cand_img[(size_t)k0 * D + src];
    }
    __syncwarp();
    // G(k0, k) for the lane's candidates
    for (int k = lane; k < K; k += 32) {
      const float* e = cand_img + (size_t)k * D;
      float sx = 0.0f, sy = 0.0f;
      for (int c = 0; c < D2; ++c) {
        const float tx = s_ref[wid][2 * c] - e[c];
        const float ty = s_ref[wid][2 * c + 1] - e[D2 + c];
        sx = fmaf(tx, tx, sx);
        sy = fmaf(ty, ty, sy);
      }
      const float G = sqrtf(sx) + sqrtf(sy);
      const float q = floorf(G * (65536.0f * (1.0f - 1.0f / 32768.0f)));
      const uint32_t Gq = (uint32_t)fminf(q, 1048575.0f);
      keys[k] = (Gq << 12) | (uint32_t)k;
    }
    __syncwarp();
    // the kNbrCap smallest keys in ascending order (keys are distinct: k is part of them)
    uint32_t* out = nbr + ((size_t)b * K_max + k0) * kNbrCap;
    uint32_t last = 0;
    bool first = true;
    for (int j = 0; j < kNbrCap; ++j) {
      uint32_t m = kNbrEnd;
      for (int k = lane; k < K; k += 32) {
        const uint32_t v = keys[k];
        if ((first || v > last) && v < m) m = v;
      }
      m = __reduce_min_sync(0xffffffffu, m);
      if (lane == 0) out[j] = m;
      if (m == kNbrEnd) {          // fewer candidates than entries: the rest are end markers
        for (int jj = j + 1 + lane; jj < kNbrCap; jj += 32) out[jj] = kNbrEnd;
        break;
      }
      last = m;
      first = false;
    }
    __syncwarp();
  }
}

}  // namespace cpe
