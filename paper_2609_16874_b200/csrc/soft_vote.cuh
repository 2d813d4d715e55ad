// Second vote mode: the paper's soft-vote histogram (Eq. 4-6) in its factorised form (Eq. 10-11),
//     H(a, b) = sum over participating pixels of E_x(p, a) E_y(p, b),   E_x(p, a) = exp(-||xhat_p - P_w[a]||),
// as two tensor-core contractions per tile of 128 pixels, with E_x and E_y never leaving the SM:
//   GEMM 1   D_x = Xhat (-2 P_w)^T  [128 pixels x 128 bins], D_y likewise: binary16 operands split into a high and a
//            low part (pixel and palette), three tcgen05.mma per k-step, binary32 accumulators in tensor memory, so
//            that ||xhat - P_w[a]||^2 = ||xhat||^2 + F + D_x is good to ~1e-6 relative before the square root.
//   epilogue two threads own one pixel row (one per axis, in warps that share the row's tensor-memory lanes): each
//            reads its D row (tcgen05.ld), forms exp(-sqrt(.)) and stores it, rounded to binary16, straight into the
//            operand layout of GEMM 2 (bin-major core matrices).  Two warps per scheduler keep the special-function
//            unit, which bounds this kernel, busier than one can.
//   GEMM 2   H_block += E_x^T E_y  [128 x 128 bins], K = the tile's 128 pixels, accumulated in tensor memory over all
//            the tiles that the CTA sees; at the end the block is added to the histogram in global memory
//            (binary32 atomics: the split over CTAs is a split-K reduction whose order is not fixed).
// A CTA serves one 128 x 128 block of bins of one image and a share of its pixels; the pixel side (spans, mask,
// compaction of participating 8-pixel groups, 16-byte gathers into the A-operand layout, squared norms) is the
// producer role of the assignment kernel with two tile buffers.  Needs 16-byte aligned planes.
// Error budget: binary16 rounding of E_x and E_y (2^-11 each, relative) dominates: |H - H_exact| <= 1.1e-3 H.
#pragma once

#include "assign_tc.cuh"
#include "cpe_common.cuh"

namespace cpe {

constexpr int kSvThreads = 384;     // warps 0-3: pixel rows, x axis (and MMA issue); warps 4-7: producers;
                                    // warps 8-11: the same pixel rows, y axis
constexpr int kSvBins = 128;        // bins per block side
constexpr int kSvTiles = 2;         // pixel tile buffers
constexpr int kSvFlushTiles = 8;    // tiles accumulated in tensor memory between two flushes of the H block
constexpr int kSvCols = 512;        // tensor-memory columns: D_x [0,128), D_y [128,256), H block [256,384)

struct SvSmem {
  int tiles, pw, ph, ex, ey, exl, eyl, ring, ringbits, rnx, rny, rflags, misc, total;
};
__host__ __device__ inline SvSmem sv_smem_layout(int KA) {
  SvSmem s;
  int off = 0;
  s.tiles = off;    off += kSvTiles * 2 * (2 * KA * kTcRows * 2);   // per buffer: high parts, low parts
  s.pw = off;       off += 2 * kSvBins * KA * 2;                    // -2 P_w block: high, low (K-major rows)
  s.ph = off;       off += 2 * kSvBins * KA * 2;
  s.ex = off;       off += kTcRows * kSvBins * 2;                   // E_x tile, operand layout of GEMM 2
  s.ey = off;       off += kTcRows * kSvBins * 2;
  // low parts of the two E tiles (F <= 8 only: with F > 8 the pixel tiles leave no room for them)
  s.exl = off;      off += KA == 16 ? kTcRows * kSvBins * 2 : 0;
  s.eyl = off;      off += KA == 16 ? kTcRows * kSvBins * 2 : 0;
  s.ring = off;     off += kTcRing * 4;
  s.ringbits = off; off += kTcRing;
  s.rnx = off;      off += kSvTiles * kTcRows * 4;
  s.rny = off;      off += kSvTiles * kTcRows * 4;
  s.rflags = off;   off += kSvTiles * kTcRows * 4;
  s.misc = off;     off += 256;
  s.total = off;
  return s;
}

// Instruction descriptors of kind::f16, binary32 accumulate, M = 128, N = 128: GEMM 1 takes A pixel-major and B
// K-major; GEMM 2 takes both operands with the M / N index contiguous (bits 15 and 16).
constexpr uint32_t kSvIdesc1 = (1u << 4) | (1u << 15) | ((uint32_t)(kSvBins >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t kSvIdesc2 = kSvIdesc1 | (1u << 16);

// Barrier among the 256 row threads of both axes (barrier resource 2)
__device__ __forceinline__ void sv_consumers_sync() { asm volatile("barrier.cta.sync 2, 256;" ::: "memory"); }

template <typename T, int KA>
__global__ void __launch_bounds__(kSvThreads, 1)
soft_vote_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F, int bins_w, int bins_h,
                 const float* __restrict__ pal_w, const float* __restrict__ pal_h, int vec_mask, float* __restrict__ hist,
                 uint32_t* __restrict__ status_all, uint32_t* __restrict__ acc) {
  constexpr int KS = KA / 16;                       // k-steps per axis
  constexpr int kPartHalves = 2 * KA * kTcRows;     // one tile part (high or low)
  constexpr uint32_t kTileLbo = kTcRows * 16;       // bytes between core matrices along K in a pixel tile
  constexpr uint32_t kPalLbo = kSvBins * 16;        // ... in a palette block
  constexpr uint32_t kELbo = (kSvBins / 8) * 128;   // ... (along the pixels) in an E tile
  constexpr bool kSplitPixel = sizeof(T) == 4;      // binary32 pixels carry a low part
  constexpr bool kSplitE = KA == 16;                // the weights go to GEMM 2 as binary16 high + low parts
  extern __shared__ __align__(1024) unsigned char sv_smem[];
  const SvSmem L = sv_smem_layout(KA);
  __half* s_tiles = reinterpret_cast<__half*>(sv_smem + L.tiles);
  __half* s_pw = reinterpret_cast<__half*>(sv_smem + L.pw);
  __half* s_ph = reinterpret_cast<__half*>(sv_smem + L.ph);
  __half* s_ex = reinterpret_cast<__half*>(sv_smem + L.ex);
  __half* s_ey = reinterpret_cast<__half*>(sv_smem + L.ey);
  __half* s_exl = reinterpret_cast<__half*>(sv_smem + L.exl);      // (only with kSplitE)
  __half* s_eyl = reinterpret_cast<__half*>(sv_smem + L.eyl);
  uint32_t* s_ring = reinterpret_cast<uint32_t*>(sv_smem + L.ring);
  uint8_t* s_ringbits = reinterpret_cast<uint8_t*>(sv_smem + L.ringbits);
  float* s_rnx = reinterpret_cast<float*>(sv_smem + L.rnx);               // per tile buffer and row: ||xhat||^2
  float* s_rny = reinterpret_cast<float*>(sv_smem + L.rny);               // ... ||yhat||^2
  uint32_t* s_rflags = reinterpret_cast<uint32_t*>(sv_smem + L.rflags);   // ... kRfLive / kRfEnd
  int* s_scan = reinterpret_cast<int*>(sv_smem + L.misc);
  volatile int* s_abort = s_scan + 8;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_scan + 9);
  const uint32_t mbar0 = (uint32_t)__cvta_generic_to_shared(sv_smem + L.misc + 64);
  // mbarriers: tile buffer filled [2], tile buffer read by GEMM 1 [2], GEMM 1 done, GEMM 2 done
  const uint32_t mb_meta = mbar0, mb_tile = mbar0 + 16, mb_d = mbar0 + 32, mb_e = mbar0 + 40;

  const int img = blockIdx.z;
  const int nab = (bins_w + kSvBins - 1) / kSvBins;
  const int a0 = ((int)blockIdx.y % nab) * kSvBins, b0 = ((int)blockIdx.y / nab) * kSvBins;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  uint32_t* status = status_all + img;
  const size_t plane = (size_t)HW;
  const int D = 4 * F;
  const T* e_img = emb + (size_t)img * D * plane;
  const uint8_t* fg_img = fg ? fg + (size_t)img * plane : nullptr;
  const float inf = __int_as_float(0x7f800000);

  // ---- set-up: tensor memory, barriers, zeroed tile buffers (padding k-slots stay zero), palette blocks
  if (wid == 0) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(s_tmem);
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst), "r"(kSvCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < kSvTiles; ++i) {
      mbar_init(mb_meta + 8 * i, 4);    // one arrival per producer warp
      mbar_init(mb_tile + 8 * i, 1);    // the MMA commit
    }
    mbar_init(mb_d, 1);
    mbar_init(mb_e, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < kSvTiles * 2 * kPartHalves / 2; i += kSvThreads) reinterpret_cast<uint32_t*>(s_tiles)[i] = 0u;
  for (int i = tid; i < (kSplitE ? 2 : 1) * kTcRows * kSvBins; i += kSvThreads) {      // E_x, E_y (and their low parts) are contiguous
    reinterpret_cast<uint32_t*>(s_ex)[i] = 0u;
  }
  // -2 P rows of this block, split into binary16 high and low parts; K-major core matrices: (bin n, slot s) at
  // (s / 8) * (128 * 8) + n * 8 + s % 8.  Bins beyond the map are zero rows (their H entries are never stored).
  // (four elements per thread and round, so that their loads are in flight together)
  for (int i0 = tid; i0 < 2 * kSvBins * KA; i0 += 4 * kSvThreads) {
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * kSvThreads;
      const int axis = i / (kSvBins * KA), j = i - axis * kSvBins * KA;
      const int n = j / KA, s = j - n * KA;
      const int bin = (axis ? b0 : a0) + n, nbins = axis ? bins_h : bins_w;
      v[u] = 0.0f;
      if (i < 2 * kSvBins * KA && bin < nbins && s < 2 * F) v[u] = -2.0f * __ldg((axis ? pal_h : pal_w) + (size_t)bin * 2 * F + s);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * kSvThreads;
      if (i >= 2 * kSvBins * KA) break;
      const int axis = i / (kSvBins * KA), j = i - axis * kSvBins * KA;
      const int n = j / KA, s = j - n * KA;
      const __half hi = __float2half_rn(v[u]);
      const __half lo = __float2half_rn(v[u] - __half2float(hi));
      __half* dst = axis ? s_ph : s_pw;
      const int o = (s >> 3) * (kSvBins * 8) + n * 8 + (s & 7);
      dst[o] = hi;
      dst[kSvBins * KA + o] = lo;
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  if (wid >= 4 && wid < 8) {
    // =============================================================================================== producers
    const int ptid = tid - 128, pw = ptid >> 5;
    const int gl = ptid >> 3, cq = ptid & 7;        // lane cq fetches channels cq, cq+8, ... of group gl, owns row ptid
    const int n_spans = (HW + kTcSpan - 1) / kTcSpan;
    uint32_t t = 0;                                 // tiles handed over
    uint32_t ring_head = 0, ring_tail = 0;
    bool bad = false, my_bad = false;

    auto slot_of = [&](int c) { return c >= 2 * F ? KA + (c - 2 * F) : c; };
    auto unit_ptr = [&](__half* tile, int c) {
      const int s = slot_of(c);
      return tile + (s >> 3) * (kTcRows * 8) + gl * 64 + (s & 7) * 8;
    };
    // one tile: ng groups from ring position head into buffer t % 2, norms, row data, hand-over
    auto emit = [&](int ng) {
      const int us = (int)(t % kSvTiles);
      __half* tile = s_tiles + (size_t)us * 2 * kPartHalves;
      if (!my_bad && !mbar_wait(mb_tile + 8 * us, ((t / kSvTiles) & 1u) ^ 1u, s_abort)) {   // GEMM 1 of its previous tile is done
        my_bad = true;
        *s_abort = 1;
      }
      float ax[8], ay[8];
#pragma unroll
      for (int r = 0; r < 8; ++r) ax[r] = ay[r] = 0.0f;
      uint32_t bits = 0;
      if (gl < ng && !my_bad) {
        const uint32_t grp = s_ring[(ring_head + gl) & (kTcRing - 1)];
        bits = s_ringbits[(ring_head + gl) & (kTcRing - 1)];
        const T* src0 = e_img + (size_t)grp * 8;
        constexpr int kIt = 2 * KA / 8;                 // channels per lane at most (D <= 2 KA)
        // every load of this lane is issued before the first value is used
        uint4 raw[kIt * (sizeof(T) == 2 ? 1 : 2)];
#pragma unroll
        for (int it = 0; it < kIt; ++it) {
          const int c = cq + 8 * it;
          if (c < D) {
            const uint4* src = reinterpret_cast<const uint4*>(src0 + (size_t)c * plane);
            if constexpr (sizeof(T) == 2) {
              raw[it] = __ldg(src);
            } else {
              raw[2 * it] = __ldg(src);
              raw[2 * it + 1] = __ldg(src + 1);
            }
          }
        }
#pragma unroll
        for (int it = 0; it < kIt; ++it) {
          const int c = cq + 8 * it;
          if (c >= D) break;
          float f[8];
          if constexpr (sizeof(T) == 2) {
            const uint4 q = raw[it];
            *reinterpret_cast<uint4*>(unit_ptr(tile, c)) = q;
            const __half2* h = reinterpret_cast<const __half2*>(&q);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 v = __half22float2(h[i]);
              f[2 * i] = v.x;
              f[2 * i + 1] = v.y;
            }
          } else {
            const float4 lo4 = *reinterpret_cast<const float4*>(&raw[2 * it]);
            const float4 hi4 = *reinterpret_cast<const float4*>(&raw[2 * it + 1]);
            f[0] = lo4.x; f[1] = lo4.y; f[2] = lo4.z; f[3] = lo4.w;
            f[4] = hi4.x; f[5] = hi4.y; f[6] = hi4.z; f[7] = hi4.w;
            __half hh[8], hl[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              hh[i] = __float2half_rn(f[i]);
              hl[i] = __float2half_rn(f[i] - __half2float(hh[i]));
            }
            *reinterpret_cast<uint4*>(unit_ptr(tile, c)) = *reinterpret_cast<const uint4*>(hh);
            *reinterpret_cast<uint4*>(unit_ptr(tile + kPartHalves, c)) = *reinterpret_cast<const uint4*>(hl);
          }
          if (c < 2 * F) {
#pragma unroll
            for (int r = 0; r < 8; ++r) ax[r] = fmaf(f[r], f[r], ax[r]);
          } else {
#pragma unroll
            for (int r = 0; r < 8; ++r) ay[r] = fmaf(f[r], f[r], ay[r]);
          }
        }
      }
      fence_async_smem();
      const float nx = reduce_scatter8(ax, cq), ny = reduce_scatter8(ay, cq);
      const bool present = gl < ng && ((bits >> cq) & 1u);
      // a value beyond the binary16 range would poison the row's dot products: such a pixel is left out (its weights
      // exp(-d), d > 6e4, are zero in binary32 anyway)
      const bool finite = (nx + ny) < inf && (sizeof(T) == 2 || (nx < 4.0e9f && ny < 4.0e9f));
      s_rnx[us * kTcRows + ptid] = nx;
      s_rny[us * kTcRows + ptid] = ny;
      s_rflags[us * kTcRows + ptid] = (present && finite) ? kRfLive : 0u;
      if (acc && blockIdx.y == 0) {
        // the decode's counters (the CTAs of the first block of bins see every pixel once): pixels that take part, and
        // participating pixels with a channel that is not finite
        const bool any_nonfinite = !((nx + ny) < inf);
        const uint32_t bv = __ballot_sync(0xffffffffu, present && !any_nonfinite);
        const uint32_t bn = __ballot_sync(0xffffffffu, present && any_nonfinite);
        if (lane == 0) {
          if (bv) atomicAdd(&acc[img * kAccStride + kAccVoting], (uint32_t)__popc(bv));
          if (bn) atomicAdd(&acc[img * kAccStride + kAccNonfinite], (uint32_t)__popc(bn));
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(mb_meta + 8 * us);
      ring_head += (uint32_t)ng;
      ++t;
    };

    for (int sp = blockIdx.x; sp < n_spans && !bad; sp += gridDim.x) {
      const long long p0 = (long long)sp * kTcSpan + (long long)ptid * 8;
      uint32_t bits = 0;
      if (p0 < HW) {                                  // HW is a multiple of 8: the whole group is inside
        if (!fg_img) {
          bits = 0xffu;
        } else if (vec_mask) {
          const uint2 w = __ldg(reinterpret_cast<const uint2*>(fg_img + p0));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            bits |= (((w.x >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
            bits |= (((w.y >> (8 * j)) & 0xffu) ? 1u : 0u) << (4 + j);
          }
        } else {
          for (int j = 0; j < 8; ++j)
            if (__ldg(fg_img + p0 + j)) bits |= 1u << j;
        }
      }
      const uint32_t gm = __ballot_sync(0xffffffffu, bits != 0);
      if (lane == 0) s_scan[pw] = __popc(gm);
      bad = producers_sync_or(my_bad);
      if (bad) break;
      int before = 0, total = 0;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int v = s_scan[w];
        if (w < pw) before += v;
        total += v;
      }
      if (bits) {
        const uint32_t pos = ring_tail + (uint32_t)before + (uint32_t)__popc(gm & ((1u << lane) - 1u));
        s_ring[pos & (kTcRing - 1)] = (uint32_t)(p0 >> 3);
        s_ringbits[pos & (kTcRing - 1)] = (uint8_t)bits;
      }
      bad = producers_sync_or(my_bad);
      if (bad) break;
      ring_tail += (uint32_t)total;
      while (ring_tail - ring_head >= (uint32_t)kTcGroups) emit(kTcGroups);
    }
    if (!bad && ring_tail != ring_head) emit((int)(ring_tail - ring_head));
    if (!bad) {
      // end marker, once the buffer's previous tile has been worked off
      const int us = (int)(t % kSvTiles);
      if (!my_bad && !mbar_wait(mb_tile + 8 * us, ((t / kSvTiles) & 1u) ^ 1u, s_abort)) {
        my_bad = true;
        *s_abort = 1;
      }
      s_rflags[us * kTcRows + ptid] = kRfEnd;
      __syncwarp();
      if (lane == 0) mbar_arrive(mb_meta + 8 * us);
    }
    if (bad || my_bad) {
      *s_abort = 1;
      am_ok(false, 12u, status);
    }
  } else {
    // =============================================================================================== pixel rows
    const int axis_y = wid >= 8 ? 1 : 0;                 // which of the two distance accumulators this thread reads
    const int row = tid & 127;                           // warps 8-11 start at thread 256
    const uint32_t t_lane = tmem + ((uint32_t)((wid & 3) * 32) << 16);
    const uint64_t d_tile0 = tc_desc((uint32_t)__cvta_generic_to_shared(s_tiles), kTileLbo, 128u);
    const uint64_t d_pw = tc_desc((uint32_t)__cvta_generic_to_shared(s_pw), kPalLbo, 128u);
    const uint64_t d_ph = tc_desc((uint32_t)__cvta_generic_to_shared(s_ph), kPalLbo, 128u);
    const uint64_t d_ex = tc_desc((uint32_t)__cvta_generic_to_shared(s_ex), kELbo, 128u);
    const uint64_t d_ey = tc_desc((uint32_t)__cvta_generic_to_shared(s_ey), kELbo, 128u);
    const uint64_t d_exl = tc_desc((uint32_t)__cvta_generic_to_shared(s_exl), kELbo, 128u);
    const uint64_t d_eyl = tc_desc((uint32_t)__cvta_generic_to_shared(s_eyl), kELbo, 128u);
    constexpr uint64_t kLoPal = (uint64_t)((kSvBins * KA * 2) >> 4);        // low part of a palette block
    constexpr uint64_t kLoTile = (uint64_t)((kPartHalves * 2) >> 4);        // low part of a pixel tile
    uint32_t t = 0;
    bool bad = false;
    const float log2e_sq = 2.0813689810056077f;         // log2(e)^2
    const int na = min(kSvBins, bins_w - a0), nb = min(kSvBins, bins_h - b0);   // bins of this block that exist

    // exp(-sqrt(|c + D|)) for 8 consecutive bins, rounded to binary16, as 2^(-sqrt(|c + D| log2(e)^2)): one fused
    // multiply-add, two special-function results.  (The squared distance is non-negative up to the rounding of its
    // three terms, about 1e-6; its magnitude stands in for max(., 0) and costs nothing.)  The special-function unit's
    // approximations (sqrt, 2^x: about 2^-22 relative each) are far inside the binary16 rounding that follows; the
    // flush-to-zero forms are single instructions (a subnormal argument or result is below anything binary16 holds:
    // its smallest subnormal is e^-16.6).  A row without a pixel is masked after packing.  `ck` = c log2(e)^2.
    // With kSplitE a weight w goes to GEMM 2 as two binary16 numbers, hi = fl16(w) and lo = fl16(w - hi), and the product
    // of two weights as hi hi + hi lo + lo hi (what is dropped, lo lo, is 2^-22 of it): the histogram is then good to
    // about 1e-5 instead of the 1e-3 of a single binary16 rounding.  The weights are also scaled by 2^14 (added to the
    // exponent argument, so it costs nothing), which keeps the low parts of small weights out of binary16's subnormal
    // range; the block is scaled back by 2^-28 when it is added to the histogram.
    constexpr float kEScale = kSplitE ? 14.0f : 0.0f;
    auto weights8 = [&](const float* v, float ck, bool live, uint4& lo_out) -> uint4 {
      uint32_t w[4], wl[4];
      const uint32_t keep = live ? 0xffffffffu : 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float d0, d1, e0, e1;
        asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(d0) : "f"(fabsf(fmaf(v[2 * i], log2e_sq, ck))));
        asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(d1) : "f"(fabsf(fmaf(v[2 * i + 1], log2e_sq, ck))));
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(kEScale - d0));
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(kEScale - d1));
        const __half2 h = __floats2half2_rn(e0, e1);
        w[i] = *reinterpret_cast<const uint32_t*>(&h) & keep;
        if constexpr (kSplitE) {
          const float2 hf = __half22float2(h);
          const __half2 l = __floats2half2_rn(e0 - hf.x, e1 - hf.y);
          wl[i] = *reinterpret_cast<const uint32_t*>(&l) & keep;
        } else {
          wl[i] = 0u;
        }
      }
      lo_out = make_uint4(wl[0], wl[1], wl[2], wl[3]);
      return make_uint4(w[0], w[1], w[2], w[3]);
    };

    // GEMM 1 of tile `tt` (buffer `us`): D_x, D_y = pixel tile (high [+ low]) x palette block (high + low)
    auto issue_gemm1 = [&](int us) {
      const uint64_t da = d_tile0 + (uint64_t)(((uint32_t)us * 2u * (kPartHalves * 2)) >> 4);
#pragma unroll
      for (int axis = 0; axis < 2; ++axis) {
        const uint64_t db = axis ? d_ph : d_pw;
        bool acc = false;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          const uint64_t ka = da + (uint64_t)(((axis * KS + ks) * 2u * kTileLbo) >> 4);
          const uint64_t kb = db + (uint64_t)((ks * 2u * kPalLbo) >> 4);
          tc_mma(tmem + (uint32_t)(axis * 128), ka, kb, kSvIdesc1, acc);
          acc = true;
          tc_mma(tmem + (uint32_t)(axis * 128), ka, kb + kLoPal, kSvIdesc1, true);
          if (kSplitPixel) tc_mma(tmem + (uint32_t)(axis * 128), ka + kLoTile, kb, kSvIdesc1, true);
        }
      }
      tc_commit(mb_d);
      tc_commit(mb_tile + 8 * us);
    };
    // row data of tile `tt`: false when the wait ran out
    uint32_t flags = 0;
    float cn = 0.0f;
    auto fetch_row = [&](uint32_t tt) -> bool {
      const int us = (int)(tt % kSvTiles);
      const bool ok = mbar_wait(mb_meta + 8 * us, (tt / kSvTiles) & 1u, s_abort);
      if (!__all_sync(0xffffffffu, ok)) return false;
      flags = s_rflags[us * kTcRows + row];
      cn = (axis_y ? s_rny : s_rnx)[us * kTcRows + row] + (float)F;
      return true;
    };

    // The H block goes to the histogram (thread = bin a, the tensor-memory lane; columns = bins b) every kSvFlushTiles
    // tiles and at the end.  The tensor pipe adds into its binary32 accumulator with a small systematic loss per
    // addition (measured: about 2^-23 of the running sum, all of one sign), so a block that ran over a CTA's whole
    // share of a large image (a hundred tiles, thousands of additions) came out 1.7e-4 low; restarting it every
    // eight tiles bounds the loss at 192 additions (2.3e-5) and leaves the long sum to the round-to-nearest atomics.
    uint32_t t_flushed = 0;
    auto flush_block = [&]() {
      const bool ok = mbar_wait(mb_e, (t - 1) & 1u, s_abort);   // GEMM 2 of tile t - 1 is done
      if (!__all_sync(0xffffffffu, ok)) { bad = true; return; }
      tc_fence_after();
      const int a = a0 + row;
      float* h_img = hist + (size_t)img * bins_w * bins_h;
      // the two threads of a row share its columns
      for (int c0 = axis_y * (kSvBins / 2); c0 < (axis_y + 1) * (kSvBins / 2); c0 += 32) {
        float v[32];
        tc_ld32(t_lane + 256u + (uint32_t)c0, v);
        if (a < bins_w) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (b0 + c0 + j < bins_h)
              atomicAdd(h_img + (size_t)(b0 + c0 + j) * bins_w + a, kSplitE ? v[j] * 3.7252902984619140625e-9f : v[j]);   // 2^-28
        }
      }
      t_flushed = t;
    };

    // The loop is software-pipelined by one tile: the thread that issues GEMM 2 of tile t issues GEMM 1 of tile t + 1
    // right behind it, so the tensor pipe runs them back to back while the row threads are between two epilogues,
    // and one wait (GEMM 1 done: the MMAs complete in issue order, so GEMM 2 of the tile before is done as well)
    // and one barrier per tile are enough.
    if (!fetch_row(0)) bad = true;
    if (!bad && !(flags & kRfEnd)) {
      tc_fence_before();
      sv_consumers_sync();        // every row thread has read its row data
      if (tid == 0) {
        tc_fence_after();
        issue_gemm1(0);
      }
      __syncwarp();
    }
    while (!bad && !(flags & kRfEnd)) {
      const bool live = (flags & kRfLive) != 0;
      const float c_row = cn * log2e_sq;
      {
        const bool ok = mbar_wait(mb_d, t & 1u, s_abort);   // GEMM 1 of this tile (and every MMA before it) is done
        if (!__all_sync(0xffffffffu, ok)) { bad = true; break; }
      }
      tc_fence_after();
      // ---- epilogue: this row's weights into the operand tiles of GEMM 2: element (bin n, pixel p) at
      // (p / 8) * kELbo + (n / 8) * 128 + (p % 8) * 16 + (n % 8) * 2 bytes
      {
        unsigned char* e_row = reinterpret_cast<unsigned char*>(axis_y ? s_ey : s_ex) + (row >> 3) * kELbo + (row & 7) * 16;
        unsigned char* e_row_lo = reinterpret_cast<unsigned char*>(axis_y ? s_eyl : s_exl) + (row >> 3) * kELbo + (row & 7) * 16;
        // only the bins that exist (in steps of 32): the rest of the E tiles stays zero
        const int nbins = axis_y ? nb : na;
        for (int c0 = 0; c0 < nbins; c0 += 32) {
          float v[32];
          tc_ld32(t_lane + (uint32_t)(axis_y * 128 + c0), v);
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 lo;
            *reinterpret_cast<uint4*>(e_row + ((c0 >> 3) + g) * 128) = weights8(v + 8 * g, c_row, live, lo);
            if constexpr (kSplitE) *reinterpret_cast<uint4*>(e_row_lo + ((c0 >> 3) + g) * 128) = lo;
          }
        }
      }
      // the next tile's row data (the producers are a tile ahead), before the barrier that frees D and publishes E
      if (!fetch_row(t + 1)) { bad = true; break; }
      fence_async_smem();
      tc_fence_before();
      sv_consumers_sync();
      if (tid == 0) {
        tc_fence_after();
        // GEMM 2: H_block += E_x^T E_y over the tile's 128 pixels (8 k-steps of 16)
#pragma unroll
        for (int ks = 0; ks < kTcRows / 16; ++ks) {
          const uint64_t o = (uint64_t)((ks * 2u * kELbo) >> 4);
          tc_mma(tmem + 256u, d_ex + o, d_ey + o, kSvIdesc2, t > t_flushed || ks > 0);
          if constexpr (kSplitE) {
            tc_mma(tmem + 256u, d_ex + o, d_eyl + o, kSvIdesc2, true);
            tc_mma(tmem + 256u, d_exl + o, d_ey + o, kSvIdesc2, true);
          }
        }
        tc_commit(mb_e);
        if (!(flags & kRfEnd)) issue_gemm1((int)((t + 1) % kSvTiles));
      }
      __syncwarp();
      ++t;
      // the reads of the block are ordered before the next GEMM 2 (which starts it afresh) by the next tile's barrier
      if (t - t_flushed == (uint32_t)kSvFlushTiles && !(flags & kRfEnd)) flush_block();
    }
    if (!bad && t > t_flushed) flush_block();
    if (bad) {
      *s_abort = 1;
      am_ok(false, 13u, status);
    }
  }

  // ---- tear-down
  tc_fence_before();
  __syncthreads();
  if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kSvCols) : "memory");
}

}  // namespace cpe
