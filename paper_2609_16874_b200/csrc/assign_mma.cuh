// Stage 4+5, fast path: pixel-to-instance assignment (Eq. 4, Eq. 7, Eq. 8) with the pixels x D x K score
// contraction on the tensor cores as a FILTER, and the decision taken exactly in binary32.
//
// For a pixel with halves xhat, yhat and a peak k with palette rows ex = P_w(a_k), ey = P_h(b_k):
//     A_k = ||xhat - ex||^2 = ||xhat||^2 + ||ex||^2 - 2 xhat.ex ,   B_k likewise,   d_k = sqrt(A_k) + sqrt(B_k).
// ||ex||^2 = F up to rounding (sin^2 + cos^2 per harmonic), so A_k and B_k are two dot products away from
// per-pixel constants.  The dot products are taken by mma.sync (binary16 operands, binary32 accumulators)
// with the accumulators pre-loaded with a LOWER bound ||xhat||^2 + F - delta, where delta bounds every error of
// the approximation (binary16 rounding of the palette and, for binary32 inputs, of the pixel; accumulation).
// From the bounds  Alo <= A <= Alo + 2 delta  follow  dlo_k <= d_k <= dhi_k.  U = min_k dhi_k bounds the best
// distance from above, and only peaks with dlo_k <= U can be the arg-min: those few candidates are re-scored
// in binary32 in the one fixed operation order (score_direct_rt) that defines the result.  A cheap test
// without square roots,  A + B + 2 min(A, B) <= d^2,  rejects almost every (pixel, peak) pair first.
//
// Work decomposition: a CTA walks spans of consecutive pixels; it compacts the span's participating pixels,
// gathers them 256 at a time into a binary16 shared-memory tile [channel][pixel], and each warp sweeps its
// 2 x 16 pixels over all peaks (peak operand resident in shared memory, B fragments shared by both m-tiles).
#pragma once

#include "assign.cuh"
#include "cpe_common.cuh"

namespace cpe {

constexpr int kAmThreads = 256;
constexpr int kAmSpan = 2048;               // pixels per span
constexpr int kAmMT = 256;                  // participating pixels per tile: 8 warps x 2 m-tiles x 16 rows
constexpr int kAmTilePitch = kAmMT + 8;     // halves; +8 keeps ldmatrix rows on distinct banks
constexpr int kAmPeakCap = 512;             // peaks resident in shared memory at a time

struct AmSmem {
  int list, lab, tile, peaks, cxlo, cylo, d2x, d2y, flag, scan, total;
};

__host__ __device__ inline AmSmem am_smem_layout(int KA, int peak_cap) {
  AmSmem s;
  int off = 0;
  s.list = off;  off += kAmSpan * 2;
  s.lab = off;   off += kAmSpan * 4;
  s.tile = off;  off += 2 * KA * kAmTilePitch * 2;
  s.peaks = off; off += peak_cap * (2 * KA + 8) * 2;
  s.cxlo = off;  off += kAmMT * 4;
  s.cylo = off;  off += kAmMT * 4;
  s.d2x = off;   off += kAmMT * 4;
  s.d2y = off;   off += kAmMT * 4;
  s.flag = off;  off += kAmMT * 4;
  s.scan = off;  off += 64;
  s.total = off;
  return s;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
// d += a (16x16, row) * b (16x8, col), binary16 operands, binary32 accumulate
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

constexpr uint32_t kRowValid = 1u;   // the row holds a participating, finite pixel
constexpr uint32_t kRowHard = 2u;    // the filter cannot be trusted for this pixel: score every peak exactly

// Per-row filter state of one thread (a row is shared by the 4 threads of a quad; each sees 2 of 8 columns).
template <int NC>
struct RowState {
  float U1, U2;      // smallest and second smallest upper bound dhi among this thread's own (row, peak) pairs
  float G1, G2;      // the same over the whole quad, as of the last exchange (the quad's pairs are disjoint)
  float Um;          // candidate threshold with rounding margin
  float thr2;        // Um^2: threshold of the square-root-free test
  float cd[NC];      // candidates: lower bounds
  int ck[NC];        //             peak indices (-1: empty)
  uint32_t hard;
};

template <int NC, bool WANT2>
__device__ __forceinline__ void row_retune(RowState<NC>& s) {
  // any upper bound of the (second) smallest distance is a valid threshold: own and shared lists may overlap,
  // so they are not merged here; the second smallest of either list bounds the second smallest of the union
  const float Uth = WANT2 ? fminf(s.U2, s.G2) : fminf(s.U1, s.G1);
  s.Um = Uth * (1.0f + 4e-5f) + 1e-6f;
  s.thr2 = s.Um * s.Um * (1.0f + 1e-6f);
}

template <int NC, bool WANT2>
__device__ __forceinline__ void row_consider(RowState<NC>& s, int k, float Alo, float Blo, float d2x, float d2y) {
  const float dlo = (__fsqrt_rn(fmaxf(Alo, 0.0f)) + __fsqrt_rn(fmaxf(Blo, 0.0f))) * (1.0f - 2e-6f);
  const float dhi = (__fsqrt_rn(fmaxf(Alo + d2x, 0.0f)) + __fsqrt_rn(fmaxf(Blo + d2y, 0.0f))) * (1.0f + 2e-6f);
  if (dhi < s.U1) { s.U2 = s.U1; s.U1 = dhi; }
  else if (dhi < s.U2) { s.U2 = dhi; }
  row_retune<NC, WANT2>(s);
  if (dlo <= s.Um) {
    // a stored candidate whose lower bound now exceeds the threshold can never win: its slot is free
    int slot = -1;
#pragma unroll
    for (int i = NC - 1; i >= 0; --i)
      if (s.ck[i] < 0 || s.cd[i] > s.Um) slot = i;
    if (slot < 0) {
      s.hard = 1u;
    } else {
#pragma unroll
      for (int i = 0; i < NC; ++i)
        if (i == slot) { s.ck[i] = k; s.cd[i] = dlo; }
    }
  }
}

// (d, k) lexicographic "less": smaller distance, then lower peak index
__device__ __forceinline__ bool dk_less(float d1, int k1, float d2, int k2) {
  return d1 < d2 || (d1 == d2 && k1 < k2);
}

// Keeps the two lexicographically smallest (d, k) pairs.
__device__ __forceinline__ void top2_push(float& d1, int& k1, float& d2, int& k2, float d, int k) {
  if (dk_less(d, k, d1, k1)) { d2 = d1; k2 = k1; d1 = d; k1 = k; }
  else if (dk_less(d, k, d2, k2)) { d2 = d; k2 = k; }
}

template <typename T, int KA, bool WANT2>
__global__ void __launch_bounds__(kAmThreads, 2)
assign_mma_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F, int K_max,
                  const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau, int need_exact,
                  int peak_cap, int vec_mask, int32_t* __restrict__ labels, float* __restrict__ best,
                  float* __restrict__ second, uint32_t* __restrict__ counters) {
  constexpr int NC = WANT2 ? 3 : 2;
  constexpr int PKP = 2 * KA + 8;     // peak row pitch in halves
  constexpr int KS = KA / 16;         // k-steps per axis
  extern __shared__ __align__(16) unsigned char smem[];
  const AmSmem L = am_smem_layout(KA, peak_cap);
  uint16_t* s_list = reinterpret_cast<uint16_t*>(smem + L.list);
  int32_t* s_lab = reinterpret_cast<int32_t*>(smem + L.lab);
  __half* s_tile = reinterpret_cast<__half*>(smem + L.tile);
  __half* s_pk = reinterpret_cast<__half*>(smem + L.peaks);
  float* s_cxlo = reinterpret_cast<float*>(smem + L.cxlo);
  float* s_cylo = reinterpret_cast<float*>(smem + L.cylo);
  float* s_d2x = reinterpret_cast<float*>(smem + L.d2x);
  float* s_d2y = reinterpret_cast<float*>(smem + L.d2y);
  uint32_t* s_flag = reinterpret_cast<uint32_t*>(smem + L.flag);
  int* s_scan = reinterpret_cast<int*>(smem + L.scan);

  const int b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const size_t plane = (size_t)HW;
  const int D = 4 * F;
  const T* e_img = emb + (size_t)b * D * plane;
  const uint8_t* fg_img = fg ? fg + (size_t)b * plane : nullptr;
  const float* pk_img = peak_emb + (size_t)b * K_max * D;
  const int K = count_ptr[b];
  const float inf = __int_as_float(0x7f800000);
  const int n_spans = (HW + kAmSpan - 1) / kAmSpan;
  const int n_pchunks = K > 0 ? (K + peak_cap - 1) / peak_cap : 0;
  int32_t* lab_img = labels + (size_t)b * plane;
  float* best_img = best ? best + (size_t)b * plane : nullptr;
  float* second_img = second ? second + (size_t)b * plane : nullptr;

  // zero the tile once: padding rows (channels beyond 2F of each axis) must stay zero
  for (int i = tid; i < 2 * KA * kAmTilePitch / 2; i += kAmThreads) reinterpret_cast<uint32_t*>(s_tile)[i] = 0u;

  // peak operand: row k = [-2 ex (2F), 0.., -2 ey (2F), 0..] in binary16 (the factor -2 is exact)
  auto load_peaks = [&](int pc) {
    const int k0 = pc * peak_cap;
    const int kn = min(peak_cap, K - k0);
    const int kn8 = (kn + 7) & ~7;
    for (int i = tid; i < kn8 * 2 * KA; i += kAmThreads) {
      const int k = i / (2 * KA), c = i - k * 2 * KA;
      const int axis = c / KA, cc = c - axis * KA;
      float v = 0.0f;
      if (k < kn && cc < 2 * F) v = -2.0f * pk_img[(size_t)(k0 + k) * D + axis * 2 * F + cc];
      s_pk[k * PKP + c] = __float2half_rn(v);
    }
  };
  if (n_pchunks == 1) load_peaks(0);
  __syncthreads();

  uint32_t rejected = 0;
  int start_tile = 0;

  for (int sp = blockIdx.x; sp < n_spans; sp += gridDim.x) {
    // later spans first: the tail of the voting pass is what is still in L2
    const long long span0 = (long long)(n_spans - 1 - sp) * kAmSpan;
    const int span_len = (int)min((long long)kAmSpan, (long long)HW - span0);

    // ---- compaction of the span's participating pixels; background pixels get their outputs here
    {
      const long long p0 = span0 + (long long)tid * 8;
      uint32_t bits = 0;
      if (p0 < HW) {
        if (!fg_img) {
          const long long left = HW - p0;
          bits = left >= 8 ? 0xffu : ((1u << (int)left) - 1u);
        } else if (vec_mask && p0 + 8 <= HW) {
          const uint2 w = __ldg(reinterpret_cast<const uint2*>(fg_img + p0));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            bits |= (((w.x >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
            bits |= (((w.y >> (8 * j)) & 0xffu) ? 1u : 0u) << (4 + j);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (p0 + j < HW && __ldg(fg_img + p0 + j)) bits |= 1u << j;
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        s_lab[tid * 8 + j] = 0;
        if (best_img && p0 + j < HW && (K == 0 || !((bits >> j) & 1u))) {
          best_img[p0 + j] = inf;
          second_img[p0 + j] = inf;
        }
      }
      const int mine = __popc(bits);
      int incl = mine;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
      }
      if (lane == 31) s_scan[wid] = incl;
      __syncthreads();
      if (tid == 0) {
        int run = 0;
#pragma unroll
        for (int w = 0; w < kAmThreads / 32; ++w) {
          const int v = s_scan[w];
          s_scan[w] = run;
          run += v;
        }
        s_scan[kAmThreads / 32] = run;
      }
      __syncthreads();
      int slot = s_scan[wid] + incl - mine;
      while (bits) {
        const int j = __ffs(bits) - 1;
        bits &= bits - 1;
        s_list[slot++] = (uint16_t)(tid * 8 + j);
      }
      __syncthreads();
    }
    const int n_active = s_scan[kAmThreads / 32];

    for (int chunk0 = 0; chunk0 < n_active && K > 0; chunk0 += kAmMT) {
      const int nrows = min(kAmMT, n_active - chunk0);
      __syncthreads();   // the previous tile is no longer read
      // ---- gather: thread j brings pixel j of the tile, all channels; norms and error bounds on the fly
      {
        uint32_t flag = 0;
        if (tid < nrows) {
          const T* src = e_img + span0 + (int)s_list[chunk0 + tid];
          float n2[2] = {0.0f, 0.0f}, n1[2] = {0.0f, 0.0f};
          float fin = 0.0f, big = 0.0f;
#pragma unroll
          for (int axis = 0; axis < 2; ++axis) {
            const T* sa = src + (size_t)axis * 2 * F * plane;
            __half* ta = s_tile + (size_t)axis * KA * kAmTilePitch + tid;
#pragma unroll 4
            for (int l = 0; l < F; ++l) {
              const float s = Elem<T>::load1(sa + (size_t)(2 * l) * plane);
              const float c = Elem<T>::load1(sa + (size_t)(2 * l + 1) * plane);
              fin = fold_finite(fin, s, c);
              n2[axis] = fmaf(s, s, fmaf(c, c, n2[axis]));
              n1[axis] += fabsf(s) + fabsf(c);
              big = fmaxf(big, fmaxf(fabsf(s), fabsf(c)));
              ta[(2 * l) * kAmTilePitch] = __float2half_rn(s);
              ta[(2 * l + 1) * kAmTilePitch] = __float2half_rn(c);
            }
          }
          const bool finite = fin == fin;
          if (finite) {
            flag = kRowValid;
            // binary32 inputs are rounded to binary16 for the filter: that error joins the bound, and values
            // outside the binary16 range make the filter useless for this pixel
            if (sizeof(T) == 4 && !(big < 60000.0f)) flag |= kRowHard;
            const float kappa = (sizeof(T) == 4 ? 3.0f : 1.0f) * 4.93e-4f;   // 2^-11 * 1.01
#pragma unroll
            for (int axis = 0; axis < 2; ++axis) {
              const float cfull = n2[axis] + (float)F;
              const float delta = kappa * n1[axis] + 1e-5f * (cfull + 2.0f * n1[axis] + 2.0f);
              (axis == 0 ? s_cxlo : s_cylo)[tid] = cfull - delta;
              (axis == 0 ? s_d2x : s_d2y)[tid] = 2.0f * delta;
            }
          }
        }
        s_flag[tid] = flag;
      }
      __syncthreads();

      // ---- per-warp sweep: rows m = wid*32 + mt*16 + half*8 + g
      RowState<NC> st[4];
      float cx[4], cy[4];
      uint32_t rflag[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int m = wid * 32 + (r >> 1) * 16 + (r & 1) * 8 + g;
        rflag[r] = s_flag[m];
        const bool live = (rflag[r] & kRowValid) && !(rflag[r] & kRowHard);
        cx[r] = live ? s_cxlo[m] : 0.0f;
        cy[r] = live ? s_cylo[m] : 0.0f;
        st[r].U1 = st[r].U2 = st[r].G1 = st[r].G2 = inf;
        st[r].Um = inf;
        st[r].thr2 = live ? inf : -inf;   // dead rows never pass the test
        st[r].hard = (rflag[r] & kRowHard) ? 1u : 0u;
#pragma unroll
        for (int i = 0; i < NC; ++i) { st[r].ck[i] = -1; st[r].cd[i] = inf; }
      }
      // A fragments of both m-tiles and both axes stay in registers for the whole sweep
      uint32_t af[2][2][KS][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int axis = 0; axis < 2; ++axis)
#pragma unroll
          for (int ks = 0; ks < KS; ++ks) {
            const int mat = lane >> 3, rr = lane & 7;
            const int krow = axis * KA + ks * 16 + rr + (mat >> 1) * 8;
            const int mcol = wid * 32 + mt * 16 + (mat & 1) * 8;
            ldmatrix_x4_trans(af[mt][axis][ks], s_tile + (size_t)krow * kAmTilePitch + mcol);
          }

      for (int pc = 0; pc < n_pchunks; ++pc) {
        if (n_pchunks > 1) {
          __syncthreads();
          load_peaks(pc);
          __syncthreads();
        }
        const int k0 = pc * peak_cap;
        const int kn = min(peak_cap, K - k0);
        const int n_tiles = (kn + 7) >> 3;
        const int first = (n_pchunks == 1 && start_tile < n_tiles) ? start_tile : 0;
        for (int it = 0; it < n_tiles; ++it) {
          int nt = it + first;
          if (nt >= n_tiles) nt -= n_tiles;
          uint32_t bf[2][KS][2];
          {
            const __half* prow = s_pk + (size_t)(nt * 8 + (lane & 7)) * PKP + (lane >> 3) * 8;
            if constexpr (KS == 1) {
              uint32_t q[4];
              ldmatrix_x4(q, prow);
              bf[0][0][0] = q[0]; bf[0][0][1] = q[1]; bf[1][0][0] = q[2]; bf[1][0][1] = q[3];
            } else {
              uint32_t q[4];
              ldmatrix_x4(q, prow);
              bf[0][0][0] = q[0]; bf[0][0][1] = q[1]; bf[0][1][0] = q[2]; bf[0][1][1] = q[3];
              ldmatrix_x4(q, prow + KA);
              bf[1][0][0] = q[0]; bf[1][0][1] = q[1]; bf[1][1][0] = q[2]; bf[1][1][1] = q[3];
            }
          }
          const bool ragged = nt * 8 + 8 > kn;
          bool slow = false;
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            float ax[4] = {cx[mt * 2], cx[mt * 2], cx[mt * 2 + 1], cx[mt * 2 + 1]};
            float ay[4] = {cy[mt * 2], cy[mt * 2], cy[mt * 2 + 1], cy[mt * 2 + 1]};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
              mma_16816(ax, af[mt][0][ks], bf[0][ks][0], bf[0][ks][1]);
              mma_16816(ay, af[mt][1][ks], bf[1][ks][0], bf[1][ks][1]);
            }
            bool pass[4];
            bool any = false;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int r = mt * 2 + (i >> 1);
              const float S = ax[i] + ay[i];
              const float Lb = fmaf(2.0f, fminf(ax[i], ay[i]), S);   // A + B + 2 min(A,B) <= (sqrt A + sqrt B)^2
              pass[i] = Lb <= st[r].thr2;
              if (ragged && nt * 8 + 2 * t4 + (i & 1) >= kn) pass[i] = false;
              any = any || pass[i];
            }
            if (any) {
              slow = true;
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                if (pass[i]) {
                  const int r = mt * 2 + (i >> 1);
                  const int m = wid * 32 + mt * 16 + (i >> 1) * 8 + g;
                  row_consider<NC, WANT2>(st[r], k0 + nt * 8 + 2 * t4 + (i & 1), ax[i], ay[i], s_d2x[m], s_d2y[m]);
                }
              }
            }
          }
          if (__any_sync(0xffffffffu, slow)) {
            // the 4 threads of a quad own the same rows and disjoint peaks: merge their own top-2 lists
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              float m1 = st[r].U1, m2 = st[r].U2;
#pragma unroll
              for (int x = 1; x <= 2; x <<= 1) {
                const float o1 = __shfl_xor_sync(0xffffffffu, m1, x);
                const float o2 = __shfl_xor_sync(0xffffffffu, m2, x);
                const float lo = fminf(m1, o1), hi = fmaxf(m1, o1);
                m2 = fminf(hi, fminf(m2, o2));
                m1 = lo;
              }
              st[r].G1 = m1;
              st[r].G2 = m2;
              if (st[r].thr2 > -inf) row_retune<NC, WANT2>(st[r]);
            }
          }
        }
      }

      // ---- decision per row: exact binary32 scores of the surviving candidates
      int lane0_k = -1;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int m = wid * 32 + (r >> 1) * 16 + (r & 1) * 8 + g;
        const bool valid = (rflag[r] & kRowValid) != 0;          // same for the 4 threads of the quad
        uint32_t hard = st[r].hard;
        hard |= __shfl_xor_sync(0xffffffffu, hard, 1);
        hard |= __shfl_xor_sync(0xffffffffu, hard, 2);
        int mine = 0;
#pragma unroll
        for (int i = 0; i < NC; ++i)
          if (st[r].ck[i] >= 0 && st[r].cd[i] <= st[r].Um) ++mine; else st[r].ck[i] = -1;
        int tot = mine;
        tot += __shfl_xor_sync(0xffffffffu, tot, 1);
        tot += __shfl_xor_sync(0xffffffffu, tot, 2);

        const int off = valid ? (int)s_list[chunk0 + m] : 0;
        const T* src = e_img + span0 + off;
        auto pixel = [&](int axis, int c) -> float {
          if constexpr (sizeof(T) == 2) return __half2float(s_tile[(size_t)(axis * KA + c) * kAmTilePitch + m]);
          else return Elem<T>::load1(src + (size_t)(axis * 2 * F + c) * plane);
        };
        auto exact = [&](int k) -> float {
          const float* pk = pk_img + (size_t)k * D;
          float sx = 0.0f, sy = 0.0f;
          for (int c = 0; c < 2 * F; ++c) {
            const float v = __fsub_rn(pixel(0, c), __ldg(pk + c));
            sx = __fmaf_rn(v, v, sx);
          }
          for (int c = 0; c < 2 * F; ++c) {
            const float v = __fsub_rn(pixel(1, c), __ldg(pk + 2 * F + c));
            sy = __fmaf_rn(v, v, sy);
          }
          return __fadd_rn(__fsqrt_rn(sx), __fsqrt_rn(sy));
        };

        float d1 = inf, d2 = inf;
        int k1 = 0x7fffffff, k2 = 0x7fffffff;
        const bool all_k = valid && hard;                         // quad-uniform
        const bool shortcut = valid && !hard && !need_exact && !WANT2 && tot == 1;
        if (all_k) {
          for (int k = t4; k < K; k += 4) top2_push(d1, k1, d2, k2, exact(k), k);
        } else if (shortcut) {
#pragma unroll
          for (int i = 0; i < NC; ++i)
            if (st[r].ck[i] >= 0) { d1 = 0.0f; k1 = st[r].ck[i]; }
        } else if (valid) {
#pragma unroll
          for (int i = 0; i < NC; ++i)
            if (st[r].ck[i] >= 0) top2_push(d1, k1, d2, k2, exact(st[r].ck[i]), st[r].ck[i]);
        }
        // merge the quad's top-2 lists
#pragma unroll
        for (int x = 1; x <= 2; x <<= 1) {
          const float od1 = __shfl_xor_sync(0xffffffffu, d1, x), od2 = __shfl_xor_sync(0xffffffffu, d2, x);
          const int ok1 = __shfl_xor_sync(0xffffffffu, k1, x), ok2 = __shfl_xor_sync(0xffffffffu, k2, x);
          top2_push(d1, k1, d2, k2, od1, ok1);
          top2_push(d1, k1, d2, k2, od2, ok2);
        }
        if (!valid && t4 == 0 && m < nrows && best_img) {   // participating but not finite: no label, no score
          const int o = (int)s_list[chunk0 + m];
          best_img[span0 + o] = inf;
          second_img[span0 + o] = inf;
        }
        if (valid && t4 == 0) {
          int label = 0;
          if (k1 != 0x7fffffff) {
            if (shortcut || d1 < tau) label = k1 + 1;
            else ++rejected;
          }
          s_lab[off] = label;
          if (best_img) {
            best_img[span0 + off] = (k1 != 0x7fffffff) ? d1 : inf;
            second_img[span0 + off] = (k2 != 0x7fffffff) ? d2 : inf;
          }
        }
        if (r == 0) lane0_k = (valid && k1 != 0x7fffffff) ? k1 : -1;
      }
      // the next tile's pixels are this tile's neighbours: start its sweep at the peak that won here
      {
        const int kk = __shfl_sync(0xffffffffu, lane0_k, 0);
        if (kk >= 0) start_tile = (kk % peak_cap) >> 3;
      }
    }
    __syncthreads();
    // ---- label map of the span: every pixel written, 128-bit stores when the span is aligned
    if ((span_len & 3) == 0 && ((uintptr_t)(lab_img + span0) & 15u) == 0) {
      for (int i = tid; i < span_len / 4; i += kAmThreads)
        reinterpret_cast<int4*>(lab_img + span0)[i] = reinterpret_cast<const int4*>(s_lab)[i];
    } else {
      for (int i = tid; i < span_len; i += kAmThreads) lab_img[span0 + i] = s_lab[i];
    }
    __syncthreads();
  }
  const uint32_t wr = __reduce_add_sync(0xffffffffu, rejected);
  if (wr && lane == 0) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_TAU_REJECTED], wr);
}

}  // namespace cpe
