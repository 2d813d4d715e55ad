// Channels-last input (the paper writes the prediction as H_O x W_O x 4L, Sec. 3.1): conversion to the planar
// [B][4F][H][W] layout that the decode kernels read.  A tiled transpose through shared memory: a CTA takes 128 pixels
// x all 4F channels of one image; global reads are 128-bit pieces of the contiguous pixel-major source, global writes
// are 128-bit pieces (8 or 4 consecutive pixels) of one plane.  Bound: HBM (one read and one write of the embedding).
// This element-wise kernel serves any shape; the unit-wise kernels below serve the aligned ones at HBM speed.
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


// ------------------------------------------------------------------------------------------------
// Fast variants for the aligned case (both pointers 16-byte aligned, H*W a multiple of the tile, D a multiple of the
// unit): the generic kernel above moves single elements through shared memory and is bound by its own instruction
// count; these move 64- and 128-bit units, and the element-level transpose happens in registers.
//
// binary16: a unit is 4 channels of one pixel (8 bytes).  A tile is 256 pixels; shared memory holds it pixel-major,
// unit u of pixel r at r * (D/4) + (u ^ swz(r)) with swz(r) = (r / 8) mod (D/4): the eight-pixel groups that 32
// consecutive lanes read for one unit then fall on different banks.  A thread takes one (group of 8 pixels, unit):
// 8 x 64-bit loads = 4 channels x 8 pixels, 16 byte-permutes, and one 128-bit store per channel; consecutive lanes
// write consecutive 16-byte pieces of the same plane.
constexpr int kLyFastPixels16 = 256;
constexpr int kLyFastPixels32 = 128;

__global__ void __launch_bounds__(kLyThreads)
channels_last_to_planar_f16_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int HW, int D) {
  extern __shared__ __align__(16) unsigned char ly_smem[];
  uint2* tile = reinterpret_cast<uint2*>(ly_smem);
  const int b = blockIdx.y;
  const long long p0 = (long long)blockIdx.x * kLyFastPixels16;
  const int U = D >> 2;                                   // units per pixel
  const uint4* s4 = reinterpret_cast<const uint4*>(src + ((size_t)b * HW + p0) * D);
  const int n16 = kLyFastPixels16 * D / 8;                // 16-byte pieces of the tile (contiguous in the source)
  for (int i0 = threadIdx.x; i0 < n16; i0 += 4 * kLyThreads) {
    uint4 raw[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (i0 + k * kLyThreads < n16) raw[k] = __ldg(s4 + i0 + k * kLyThreads);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k * kLyThreads;
      if (i < n16) {
        const int r = i / (U >> 1), u = (i - r * (U >> 1)) * 2;
        const int sw = (r >> 3) & (U - 1);
        tile[r * U + (u ^ sw)] = make_uint2(raw[k].x, raw[k].y);
        tile[r * U + ((u + 1) ^ sw)] = make_uint2(raw[k].z, raw[k].w);
      }
    }
  }
  __syncthreads();
  uint16_t* d = dst + (size_t)b * D * HW + p0;
  constexpr int G = kLyFastPixels16 / 8;                  // groups of 8 pixels: 32, one per lane
  for (int it = threadIdx.x; it < G * U; it += kLyThreads) {
    const int u = it / G, g = it - u * G;
    const int sw = g & (U - 1);                            // swz of the rows 8g .. 8g+7
    uint2 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = tile[(8 * g + j) * U + (u ^ sw)];
    // v[j] = pixel j: x = channels (4u, 4u+1), y = channels (4u+2, 4u+3)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t w[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t a = (c & 2) ? v[2 * q].y : v[2 * q].x, bb = (c & 2) ? v[2 * q + 1].y : v[2 * q + 1].x;
        w[q] = __byte_perm(a, bb, (c & 1) ? 0x7632 : 0x5410);      // (pixel 2q, pixel 2q+1) of channel 4u+c
      }
      *reinterpret_cast<uint4*>(d + (size_t)(4 * u + c) * HW + 8 * g) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// binary32: a unit is 4 channels of one pixel (16 bytes), a tile 128 pixels, unit u of pixel r at
// r * (D/4) + (u ^ ((r / 4) mod (D/4))).  A thread takes one (group of 4 pixels, unit): 4 x 128-bit loads, a 4 x 4
// transpose in registers, one 128-bit store per channel.
__global__ void __launch_bounds__(kLyThreads)
channels_last_to_planar_f32_kernel(const float* __restrict__ src, float* __restrict__ dst, int HW, int D) {
  extern __shared__ __align__(16) unsigned char ly_smem[];
  float4* tile = reinterpret_cast<float4*>(ly_smem);
  const int b = blockIdx.y;
  const long long p0 = (long long)blockIdx.x * kLyFastPixels32;
  const int U = D >> 2;
  const float4* s4 = reinterpret_cast<const float4*>(src + ((size_t)b * HW + p0) * D);
  const int n16 = kLyFastPixels32 * U;
  for (int i0 = threadIdx.x; i0 < n16; i0 += 4 * kLyThreads) {
    float4 raw[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (i0 + k * kLyThreads < n16) raw[k] = __ldg(s4 + i0 + k * kLyThreads);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k * kLyThreads;
      if (i < n16) {
        const int r = i / U, u = i - r * U;
        tile[r * U + (u ^ ((r >> 2) & (U - 1)))] = raw[k];
      }
    }
  }
  __syncthreads();
  float* d = dst + (size_t)b * D * HW + p0;
  constexpr int G = kLyFastPixels32 / 4;                  // groups of 4 pixels: 32, one per lane
  for (int it = threadIdx.x; it < G * U; it += kLyThreads) {
    const int u = it / G, g = it - u * G;
    const int sw = g & (U - 1);
    float4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = tile[(4 * g + j) * U + (u ^ sw)];
    float* o = d + (size_t)(4 * u) * HW + 4 * g;
    *reinterpret_cast<float4*>(o) = make_float4(v[0].x, v[1].x, v[2].x, v[3].x);
    *reinterpret_cast<float4*>(o + (size_t)HW) = make_float4(v[0].y, v[1].y, v[2].y, v[3].y);
    *reinterpret_cast<float4*>(o + 2 * (size_t)HW) = make_float4(v[0].z, v[1].z, v[2].z, v[3].z);
    *reinterpret_cast<float4*>(o + 3 * (size_t)HW) = make_float4(v[0].w, v[1].w, v[2].w, v[3].w);
  }
}

}  // namespace cpe
