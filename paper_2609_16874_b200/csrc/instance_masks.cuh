// The paper's output form of the assignment (Sec. 3.2 "Mask aggregation", Eq. 8): one binary mask plane per candidate
// centroid and a counter of the pixels that went to it, expanded from the label map that the assignment writes.
// A store-bound pass: 4 bytes read and n_planes bytes written per pixel.  A thread takes 16 consecutive pixels: four
// 128-bit label loads, then one 128-bit store per plane (consecutive threads -> consecutive 16 bytes of a plane).
// Counters: a per-CTA histogram in shared memory, flushed with one global atomic per label seen.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cpe {

constexpr int kImThreads = 256;
constexpr int kImPixels = 16;        // per thread

__global__ void __launch_bounds__(kImThreads)
instance_masks_kernel(const int32_t* __restrict__ labels, int HW, int n_planes, int vec, uint8_t* __restrict__ planes,
                      uint32_t* __restrict__ pixels) {
  extern __shared__ uint32_t s_hist[];                 // [n_planes + 1], only when counters are wanted
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  const int32_t* lab = labels + (size_t)b * HW;
  if (pixels) {
    for (int i = tid; i <= n_planes; i += kImThreads) s_hist[i] = 0u;
    __syncthreads();
  }
  const long long n_chunks = ((long long)HW + kImPixels - 1) / kImPixels;
  for (long long ch = (long long)blockIdx.x * kImThreads + tid; ch < n_chunks; ch += (long long)gridDim.x * kImThreads) {
    const long long p0 = ch * kImPixels;
    int32_t l[kImPixels];
    if (vec && p0 + kImPixels <= HW) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int4 v = __ldg(reinterpret_cast<const int4*>(lab + p0) + q);
        l[4 * q] = v.x; l[4 * q + 1] = v.y; l[4 * q + 2] = v.z; l[4 * q + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < kImPixels; ++i) l[i] = p0 + i < HW ? __ldg(lab + p0 + i) : 0;
    }
    if (pixels) {
      // runs of equal labels are the rule: one shared-memory atomic per run
      int run_label = l[0], run = 1;
#pragma unroll
      for (int i = 1; i < kImPixels; ++i) {
        if (l[i] == run_label) { ++run; continue; }
        if (run_label >= 1 && run_label <= n_planes) atomicAdd(&s_hist[run_label], (uint32_t)run);
        run_label = l[i];
        run = 1;
      }
      if (run_label >= 1 && run_label <= n_planes) atomicAdd(&s_hist[run_label], (uint32_t)run);
    }
    if (planes) {
      uint8_t* base = planes + (size_t)b * n_planes * HW + p0;
      for (int m = 0; m < n_planes; ++m) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          w[q] = (l[4 * q] == m + 1 ? 1u : 0u) | (l[4 * q + 1] == m + 1 ? 0x100u : 0u) |
                 (l[4 * q + 2] == m + 1 ? 0x10000u : 0u) | (l[4 * q + 3] == m + 1 ? 0x1000000u : 0u);
        uint8_t* dst = base + (size_t)m * HW;
        if (vec && p0 + kImPixels <= HW) {
          *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
          for (int i = 0; i < kImPixels && p0 + i < HW; ++i) dst[i] = (uint8_t)((w[i >> 2] >> (8 * (i & 3))) & 1u);
        }
      }
    }
  }
  if (pixels) {
    __syncthreads();
    for (int i = tid; i < n_planes; i += kImThreads)
      if (s_hist[i + 1]) atomicAdd(&pixels[(size_t)b * n_planes + i], s_hist[i + 1]);
  }
}

}  // namespace cpe
