// Channels-last input (the paper writes the prediction as H_O x W_O x 4L, Sec. 3.1): conversion to the planar
// [B][4F][H][W] layout that the decode kernels read.  A tiled transpose through shared memory: a CTA takes 128 pixels
// x all 4F channels of one image; global reads are 128-bit pieces of the contiguous pixel-major source, global writes
// are 128-bit pieces (8 or 4 consecutive pixels) of one plane.  Bound: HBM (one read and one write of the embedding).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cpe {

constexpr int kLyThreads = 256;
constexpr int kLyPixels = 128;     // pixels per CTA tile

template <typename T>
__global__ void __launch_bounds__(kLyThreads)
channels_last_to_planar_kernel(const T* __restrict__ src, T* __restrict__ dst, int HW, int D, int vec_in, int vec_out) {
  constexpr int VEC = 16 / (int)sizeof(T);
  extern __shared__ __align__(16) unsigned char ly_smem[];
  T* tile = reinterpret_cast<T*>(ly_smem);            // [kLyPixels][D + 1]: the pad spreads a plane's column over banks
  const int b = blockIdx.y;
  const long long p0 = (long long)blockIdx.x * kLyPixels;
  const int np = (int)min((long long)kLyPixels, (long long)HW - p0);
  const T* s = src + ((size_t)b * HW + p0) * D;
  const int pitch = D + 1;
  const int n = np * D;
  if (vec_in) {
    // the tile's source is contiguous: 128-bit loads, elements scattered into the padded tile
    for (int i = threadIdx.x * VEC; i < n; i += kLyThreads * VEC) {
      T v[VEC];
      if (i + VEC <= n) {
        *reinterpret_cast<uint4*>(v) = __ldg(reinterpret_cast<const uint4*>(s + i));
      } else {
        for (int j = 0; j < VEC; ++j) v[j] = i + j < n ? s[i + j] : T();
      }
      int p = i / D, c = i - p * D;
#pragma unroll
      for (int j = 0; j < VEC; ++j) {
        if (i + j < n) tile[p * pitch + c] = v[j];
        if (++c == D) { c = 0; ++p; }
      }
    }
  } else {
    for (int i = threadIdx.x; i < n; i += kLyThreads) {
      const int p = i / D, c = i - p * D;
      tile[p * pitch + c] = s[i];
    }
  }
  __syncthreads();
  T* d = dst + (size_t)b * D * HW + p0;
  if (vec_out && np == kLyPixels) {
    // VEC consecutive pixels of one plane per store; consecutive threads -> consecutive pieces of the plane
    constexpr int kPieces = kLyPixels / VEC;
    for (int i = threadIdx.x; i < kPieces * D; i += kLyThreads) {
      const int c = i / kPieces, p = (i - c * kPieces) * VEC;
      T v[VEC];
#pragma unroll
      for (int j = 0; j < VEC; ++j) v[j] = tile[(p + j) * pitch + c];
      *reinterpret_cast<uint4*>(d + (size_t)c * HW + p) = *reinterpret_cast<const uint4*>(v);
    }
  } else {
    for (int i = threadIdx.x; i < n; i += kLyThreads) {
      const int c = i / np, p = i - c * np;
      d[(size_t)c * HW + p] = tile[p * pitch + c];
    }
  }
}

}  // namespace cpe
