// Stage 4+5, fast path: pixel-to-instance assignment (Eq. 4, Eq. 7, Eq. 8) with the pixels x D x K score
// contraction on the tensor cores as a FILTER, and the decision taken exactly in binary32.
//
// For a pixel with halves xhat, yhat and a peak k with palette rows ex = P_w(a_k), ey = P_h(b_k):
//     A_k = ||xhat - ex||^2 = ||xhat||^2 + ||ex||^2 - 2 xhat.ex ,   B_k likewise,   d_k = sqrt(A_k) + sqrt(B_k).
// ||ex||^2 = F up to rounding (sin^2 + cos^2 per harmonic), so A_k, B_k and S_k = A_k + B_k are dot products
// away from per-pixel constants.  mma.sync (binary16 operands, binary32 accumulators) takes the dot products
// with the accumulators pre-loaded with LOWER bounds ||.||^2 + F - delta, where delta bounds every error of the
// approximation (binary16 rounding of the palette and, for binary32 inputs, of the pixel; accumulation).
//
//   sweep 1   S_k for every peak; the smallest one, S_min, bounds the best distance: since S <= d^2 <= 2 S,
//             d_best^2 <= 2 (S_min + slack) =: T, and a peak with S_k > T cannot be the arg-min.
//   sweep 2   S_k again, plus A_k; the test S_k <= T is ONE compare per (pixel, peak) pair.  The few pairs that
//             pass (and also pass S + 2 min(A,B) <= T, a tighter bound of d^2 without square roots) are queued.
//   drain     the queue is worked off with all lanes busy: bounds dlo <= d <= dhi per entry, U = min dhi per
//             pixel, candidates are the entries with dlo <= U; a single candidate decides the pixel, several
//             are re-scored in binary32 in the one fixed operation order that defines the result.
//
// Work decomposition: a CTA walks spans of consecutive pixels; it compacts the span's participating pixels,
// gathers them 256 at a time into a binary16 shared-memory tile [channel][pixel], and each warp sweeps its
// 2 x 16 pixels over all peaks (peak operand resident in shared memory, B fragments shared by both m-tiles).
#pragma once

#include "assign.cuh"
#include "cpe_common.cuh"

namespace cpe {

constexpr int kAmThreads = 256;
constexpr int kAmSpanMax = 2048;            // pixels per span (512 for small images: more CTAs)
constexpr int kAmMT = 256;                  // participating pixels per tile: 8 warps x 2 m-tiles x 16 rows
constexpr int kAmTilePitch = kAmMT + 8;     // halves; +8 keeps ldmatrix rows on distinct banks
constexpr int kAmQueue = 128;               // queued (pixel, peak) pairs per warp and tile

struct AmSmem {
  int list, lab, tile, tile2, peaks, rowoff, glist, gbits, d2x, d2y, flag, best, second, u1, u2, nc, ck, queue, scan, total;
};

__host__ __device__ inline AmSmem am_smem_layout(int KA, int peak_cap, int span, int two_tiles) {
  AmSmem s;
  int off = 0;
  s.list = off;   off += span * 2;
  s.lab = off;    off += span * 4;
  s.tile = off;   off += 2 * KA * kAmTilePitch * 2;
  s.tile2 = off;  off += two_tiles ? 2 * KA * kAmTilePitch * 2 : 0;
  s.peaks = off;  off += peak_cap * (2 * KA + 8) * 2;
  s.rowoff = off; off += kAmMT * 2;
  s.glist = off;  off += 256 * 2;
  s.gbits = off;  off += 256;
  s.d2x = off;    off += kAmMT * 4;
  s.d2y = off;    off += kAmMT * 4;
  s.flag = off;   off += kAmMT * 4;
  s.nc = off;     off += kAmMT * 4;
  s.ck = off;     off += kAmMT * 4;
  off = (off + 15) & ~15;
  s.best = off;   off += kAmMT * 8;
  s.second = off; off += kAmMT * 8;
  s.u1 = off;     off += kAmMT * 8;
  s.u2 = off;     off += kAmMT * 8;
  s.queue = off;  off += (kAmThreads / 32) * kAmQueue * 16;
  s.scan = off;   off += 128;   // block-scan scratch (16 ints) and the warps' queue counters (8 ints)
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
constexpr unsigned long long kPackEmpty = ~0ull;

// (distance, peak) as one integer whose order is the lexicographic order (distances are >= +0)
__device__ __forceinline__ unsigned long long pack_dk(float d, int k) {
  return ((unsigned long long)__float_as_uint(d) << 32) | (unsigned int)k;
}
__device__ __forceinline__ float pack_d(unsigned long long p) { return __uint_as_float((unsigned int)(p >> 32)); }
__device__ __forceinline__ int pack_k(unsigned long long p) { return (int)(unsigned int)(p & 0xffffffffu); }

struct __align__(16) AmEntry {
  int rk;        // row within the CTA's tile (8 bits) << 24 | "bounds evaluated" mark (bit 23) | peak index
  float a, b;    // lower bounds Alo, Blo; later: a = dlo, b = exact score
  float hi;      // upper bound dhi
};
constexpr int kEntryDone = 1 << 23;    // the entry's bounds have been evaluated (a = dlo, hi = dhi)
constexpr int kEntryKMask = (1 << 23) - 1;

// Index self-check: a violated bound is recorded in the status word (bit 2 plus a site code) and the access is
// skipped; it never becomes a wild access.
__device__ __forceinline__ bool am_ok(bool ok, uint32_t site, uint32_t* status) {
  if (!ok) atomicOr(status, (uint32_t)CPE_STATUS_INTERNAL | (site << 8));
  return ok;
}

template <typename T, int KA, bool WANT2>
__device__ __forceinline__ void
assign_mma_body(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F, int K_max,
                  const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau, int need_exact,
                  int peak_cap, int span, int vec_mask, int vec_gather, int32_t* __restrict__ labels, float* __restrict__ best,
                  float* __restrict__ second, uint32_t* __restrict__ counters, uint32_t* __restrict__ status_all,
                  uint32_t* __restrict__ votes, int cells, int k_min) {
  constexpr int PKP = 2 * KA + 8;     // peak row pitch in halves
  constexpr int KS = KA / 16;         // k-steps per axis
  extern __shared__ __align__(16) unsigned char smem[];
  const int two_tiles = (vec_gather && sizeof(T) == 2 && KA == 16) ? 1 : 0;   // prefetch the next tile while this one is swept
  const AmSmem L = am_smem_layout(KA, peak_cap, span, two_tiles);
  uint16_t* s_list = reinterpret_cast<uint16_t*>(smem + L.list);
  int32_t* s_lab = reinterpret_cast<int32_t*>(smem + L.lab);
  __half* s_tile0 = reinterpret_cast<__half*>(smem + L.tile);
  __half* s_tile = s_tile0;                                            // the tile being swept
  __half* s_pk = reinterpret_cast<__half*>(smem + L.peaks);
  uint16_t* s_rowoff = reinterpret_cast<uint16_t*>(smem + L.rowoff);   // row -> pixel offset in the span, 0xffff: no pixel
  uint16_t* s_glist = reinterpret_cast<uint16_t*>(smem + L.glist);     // participating 8-pixel groups of the span
  uint8_t* s_gbits = reinterpret_cast<uint8_t*>(smem + L.gbits);       // which of a group's 8 pixels participate
  float* s_d2x = reinterpret_cast<float*>(smem + L.d2x);
  float* s_d2y = reinterpret_cast<float*>(smem + L.d2y);
  uint32_t* s_flag = reinterpret_cast<uint32_t*>(smem + L.flag);
  uint32_t* s_nc = reinterpret_cast<uint32_t*>(smem + L.nc);
  int32_t* s_ck = reinterpret_cast<int32_t*>(smem + L.ck);
  unsigned long long* s_best = reinterpret_cast<unsigned long long*>(smem + L.best);
  unsigned long long* s_second = reinterpret_cast<unsigned long long*>(smem + L.second);
  unsigned long long* s_u1 = reinterpret_cast<unsigned long long*>(smem + L.u1);
  unsigned long long* s_u2 = reinterpret_cast<unsigned long long*>(smem + L.u2);
  AmEntry* s_queue = reinterpret_cast<AmEntry*>(smem + L.queue);
  int* s_scan = reinterpret_cast<int*>(smem + L.scan);

  const int b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  uint32_t* status = status_all + b;
  // the vote map has no reader left: leave it zero for the next decode (votes == NULL keeps it)
  if (votes) zero_votes_share(votes + (size_t)b * cells, cells, (int)blockIdx.x, (int)gridDim.x);
  const size_t plane = (size_t)HW;
  const int D = 4 * F;
  const T* e_img = emb + (size_t)b * D * plane;
  const uint8_t* fg_img = fg ? fg + (size_t)b * plane : nullptr;
  const float* pk_img = peak_emb + (size_t)b * K_max * D;
  const int K = count_ptr[b];
  if (K < k_min) return;     // few peaks: this image is done by the plain all-pairs kernel launched next to this one
  const float inf = __int_as_float(0x7f800000);
  const int n_spans = (HW + span - 1) / span;
  const int n_pchunks = K > 0 ? (K + peak_cap - 1) / peak_cap : 0;
  int32_t* lab_img = labels + (size_t)b * plane;
  float* best_img = best ? best + (size_t)b * plane : nullptr;
  float* second_img = second ? second + (size_t)b * plane : nullptr;
  AmEntry* my_queue = s_queue + wid * kAmQueue;
  const int ppt = span / kAmThreads;   // pixels per thread in the mask pass: 8 or 2

  // zero the tile once: padding rows (channels beyond 2F of each axis) must stay zero
  for (int i = tid; i < (1 + two_tiles) * 2 * KA * kAmTilePitch / 2; i += kAmThreads)
    reinterpret_cast<uint32_t*>(s_tile0)[i] = 0u;

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

  uint32_t rejected = 0, n_pairs = 0, n_rescored = 0, n_full = 0;

  for (int sp = blockIdx.x; sp < n_spans; sp += gridDim.x) {
    // later spans first: the tail of the voting pass is what is still in L2
    const long long span0 = (long long)(n_spans - 1 - sp) * span;
    const int span_len = (int)min((long long)span, (long long)HW - span0);

    // ---- compaction of the span's participating pixels; background pixels get their outputs here
    {
      const long long p0 = span0 + (long long)tid * ppt;
      uint32_t bits = 0;
      if (p0 < HW) {
        if (!fg_img) {
          const long long left = HW - p0;
          bits = left >= ppt ? ((1u << ppt) - 1u) : ((1u << (int)left) - 1u);
        } else if (ppt == 8 && vec_mask && p0 + 8 <= HW) {
          const uint2 w = __ldg(reinterpret_cast<const uint2*>(fg_img + p0));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            bits |= (((w.x >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
            bits |= (((w.y >> (8 * j)) & 0xffu) ? 1u : 0u) << (4 + j);
          }
        } else {
          for (int j = 0; j < ppt; ++j)
            if (p0 + j < HW && __ldg(fg_img + p0 + j)) bits |= 1u << j;
        }
      }
      for (int j = 0; j < ppt; ++j) {
        s_lab[tid * ppt + j] = 0;
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
      uint32_t rest = bits;
      while (rest) {
        const int j = __ffs(rest) - 1;
        rest &= rest - 1;
        s_list[slot++] = (uint16_t)(tid * ppt + j);
      }
      const int n_act = s_scan[kAmThreads / 32];
      __syncthreads();
      if (vec_gather) {
        // second compaction, of whole 8-pixel groups (thread t owns group t of the span)
        const uint32_t gm = __ballot_sync(0xffffffffu, bits != 0);
        if (lane == 0) s_scan[wid] = __popc(gm);
        __syncthreads();
        if (tid == 0) {
          int run = 0;
#pragma unroll
          for (int w = 0; w < kAmThreads / 32; ++w) {
            const int v = s_scan[w];
            s_scan[w] = run;
            run += v;
          }
          s_scan[kAmThreads / 32 + 1] = run;
        }
        __syncthreads();
        if (bits) {
          const int gi = s_scan[wid] + __popc(gm & ((1u << lane) - 1u));
          s_glist[gi] = (uint16_t)tid;
          s_gbits[gi] = (uint8_t)bits;
        }
        if (tid == 0) s_scan[kAmThreads / 32] = n_act;
        __syncthreads();
      }
    }
    const int n_active = s_scan[kAmThreads / 32];
    const int n_groups = vec_gather ? s_scan[kAmThreads / 32 + 1] : 0;
    const int n_chunks = K > 0 ? (vec_gather ? (n_groups + 31) / 32 : (n_active + kAmMT - 1) / kAmMT) : 0;

    // Asynchronous 16-byte copies of one tile (32 groups x 4F channels) straight into shared memory.
    auto issue_gather = [&](int ci, __half* dst_tile) {
      if constexpr (sizeof(T) == 2) {
        const int ng = min(32, n_groups - ci * 32);
        for (int i = tid; i < ng * D; i += kAmThreads) {
          const int gl = i % ng, c = i / ng;               // consecutive lanes -> consecutive groups of one channel
          const int grp = s_glist[ci * 32 + gl];
          const int axis = c >= 2 * F ? 1 : 0;
          const __half* dst = dst_tile + (size_t)(axis * KA + (c - axis * 2 * F)) * kAmTilePitch + gl * 8;
          const T* src = e_img + (size_t)c * plane + span0 + grp * 8;
          const uint32_t d32 = (uint32_t)__cvta_generic_to_shared(dst);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d32), "l"(src));
        }
      }
      asm volatile("cp.async.commit_group;\n" ::);
    };
    if (vec_gather && sizeof(T) == 2 && n_chunks > 0) issue_gather(0, s_tile0);

    for (int ci = 0; ci < n_chunks; ++ci) {
      const int chunk0 = ci * kAmMT;
      __syncthreads();   // the previous tile and its row state are no longer read
      // ---- gather
      {
        int off = 0xffff;
        if (vec_gather) {
          // rows = the pixels of 32 participating groups; a row whose pixel does not participate stays empty
          const int gl = tid >> 3, j = tid & 7, gi = ci * 32 + gl;
          if (gi < n_groups && ((s_gbits[gi] >> j) & 1u)) off = (int)s_glist[gi] * 8 + j;
          if constexpr (sizeof(T) == 2) {
            s_tile = two_tiles ? s_tile0 + (size_t)(ci & 1) * 2 * KA * kAmTilePitch : s_tile0;
            if (!two_tiles && ci > 0) issue_gather(ci, s_tile);
            asm volatile("cp.async.wait_group 0;\n" ::);
          } else {
            // binary32: two 128-bit loads per (group, channel), rounded to binary16 on the way
            const int ng = min(32, n_groups - ci * 32);
            for (int i = tid; i < ng * D; i += kAmThreads) {
              const int gq = i % ng, c = i / ng;
              const int grp = s_glist[ci * 32 + gq];
              const int axis = c >= 2 * F ? 1 : 0;
              __half* dst = s_tile + (size_t)(axis * KA + (c - axis * 2 * F)) * kAmTilePitch + gq * 8;
              const float4* src = reinterpret_cast<const float4*>(e_img + (size_t)c * plane + span0 + grp * 8);
              const float4 lo = __ldg(src), hi = __ldg(src + 1);
              __half2 h[4] = {__floats2half2_rn(lo.x, lo.y), __floats2half2_rn(lo.z, lo.w),
                              __floats2half2_rn(hi.x, hi.y), __floats2half2_rn(hi.z, hi.w)};
              *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(h);
            }
          }
        } else {
          // thread j copies pixel j of the tile, all channels (binary32 inputs are rounded to binary16)
          if (chunk0 + tid < n_active) off = (int)s_list[chunk0 + tid];
          if (off != 0xffff && am_ok(off < span_len, 1u, status)) {
            const T* src = e_img + span0 + off;
            constexpr int FMAX = KA / 2;       // F <= FMAX for this instantiation
#pragma unroll
            for (int axis = 0; axis < 2; ++axis) {
              const T* sa = src + (size_t)axis * 2 * F * plane;
              __half* ta = s_tile + (size_t)axis * KA * kAmTilePitch + tid;
              // every plane load of this axis is issued before the first value is stored
              __half hv[2 * FMAX];
#pragma unroll
              for (int c = 0; c < 2 * FMAX; ++c) {
                hv[c] = __ushort_as_half((unsigned short)0);
                if (c < 2 * F) {
                  if constexpr (sizeof(T) == 2)
                    hv[c] = __ushort_as_half(__ldg(reinterpret_cast<const unsigned short*>(sa + (size_t)c * plane)));
                  else
                    hv[c] = __float2half_rn(__ldg(reinterpret_cast<const float*>(sa + (size_t)c * plane)));
                }
              }
#pragma unroll
              for (int c = 0; c < 2 * FMAX; ++c)
                if (c < 2 * F) ta[c * kAmTilePitch] = hv[c];
            }
          }
        }
        s_rowoff[tid] = (uint16_t)off;
        s_nc[tid] = 0;
        s_ck[tid] = -1;
        s_best[tid] = kPackEmpty;
        s_second[tid] = kPackEmpty;
        s_u1[tid] = kPackEmpty;
        s_u2[tid] = kPackEmpty;
      }
      __syncthreads();
      // the other tile buffer was last read before the barrier above: fill it while this tile is swept
      if (two_tiles && ci + 1 < n_chunks)
        issue_gather(ci + 1, s_tile0 + (size_t)((ci + 1) & 1) * 2 * KA * kAmTilePitch);

      // ---- per-warp sweeps: rows m = wid*32 + mt*16 + half*8 + g
      // A fragments of both m-tiles and both axes stay in registers for the whole tile
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
      // ||xhat||^2 and ||yhat||^2 of every row from the tensor cores as well: the diagonal of tile x tile^T
      // (the B operand of a row block is that block's own A fragment: {a0, a2} for rows 0-7, {a1, a3} for 8-15)
      float cs[4], cx[4], cy[4], thr[4];
      bool live[4];
      {
        float n2[2][4];   // [axis][row r]
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int axis = 0; axis < 2; ++axis) {
            float glo[4] = {0.0f, 0.0f, 0.0f, 0.0f}, ghi[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
              mma_16816(glo, af[mt][axis][ks], af[mt][axis][ks][0], af[mt][axis][ks][2]);
              mma_16816(ghi, af[mt][axis][ks], af[mt][axis][ks][1], af[mt][axis][ks][3]);
            }
            // row g's diagonal element sits in the quad's thread g/2 (c0 or c1); row g+8's in the same thread (c2 or c3)
            const float dlo_ = (g & 1) ? glo[1] : glo[0];
            const float dhi_ = (g & 1) ? ghi[3] : ghi[2];
            const int owner = (lane & ~3) | (g >> 1);
            n2[axis][mt * 2 + 0] = __shfl_sync(0xffffffffu, dlo_, owner);
            n2[axis][mt * 2 + 1] = __shfl_sync(0xffffffffu, dhi_, owner);
          }
        const float kappa = (sizeof(T) == 4 ? 3.0f : 1.0f) * 4.93e-4f;   // 2^-11 * 1.01 (x3: pixel rounding too)
        const float sq2f = sqrtf(2.0f * (float)F);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int m = wid * 32 + (r >> 1) * 16 + (r & 1) * 8 + g;
          const bool present = s_rowoff[m] != 0xffffu;
          const bool finite = (n2[0][r] + n2[1][r]) < inf;
          // binary16 pixels: a non-finite norm is a non-finite pixel.  binary32 pixels: it may also be a value
          // beyond the binary16 range, so the row is scored exactly (and its finiteness checked there).
          uint32_t flag = 0;
          if (present) flag = finite ? kRowValid : (sizeof(T) == 4 ? (kRowValid | kRowHard) : 0u);
          live[r] = present && finite;
          float cfull[2], delta[2];
#pragma unroll
          for (int axis = 0; axis < 2; ++axis) {
            const float nn = live[r] ? n2[axis][r] : 0.0f;
            const float n1 = sq2f * sqrtf(nn) * 1.0001f;          // sum |v| <= sqrt(2F) ||v||
            cfull[axis] = nn + (float)F;
            delta[axis] = kappa * n1 + 1e-5f * (cfull[axis] + 2.0f * n1 + 2.0f);
          }
          cx[r] = cfull[0] - delta[0];
          cy[r] = cfull[1] - delta[1];
          cs[r] = (cfull[0] - delta[0]) + (cfull[1] - delta[1]) - 1e-6f * (cfull[0] + cfull[1]);
          if (t4 == 0) {
            s_flag[m] = flag;
            s_d2x[m] = 2.0f * delta[0];
            s_d2y[m] = 2.0f * delta[1] + 4e-6f * (cfull[0] + cfull[1]);   // B is recovered as S - A: one more rounding
          }
        }
      }
      __syncwarp();
      auto load_b = [&](int nt, uint32_t (&bf)[2][KS][2]) {
        const __half* prow = s_pk + (size_t)(nt * 8 + (lane & 7)) * PKP + (lane >> 3) * 8;
        uint32_t q[4];
        ldmatrix_x4(q, prow);
        if constexpr (KS == 1) {
          bf[0][0][0] = q[0]; bf[0][0][1] = q[1]; bf[1][0][0] = q[2]; bf[1][0][1] = q[3];
        } else {
          bf[0][0][0] = q[0]; bf[0][0][1] = q[1]; bf[0][1][0] = q[2]; bf[0][1][1] = q[3];
          ldmatrix_x4(q, prow + KA);
          bf[1][0][0] = q[0]; bf[1][0][1] = q[1]; bf[1][1][0] = q[2]; bf[1][1][1] = q[3];
        }
      };

      // sweep 1: the smallest (and, if the runner-up is wanted, second smallest) S_k of every row
      float s1[4], s2[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) s1[r] = s2[r] = inf;
      for (int pc = 0; pc < n_pchunks; ++pc) {
        if (n_pchunks > 1) { __syncthreads(); load_peaks(pc); __syncthreads(); }
        const int kn = min(peak_cap, K - pc * peak_cap);
        const int n_tiles = (kn + 7) >> 3;
        for (int nt = 0; nt < n_tiles; ++nt) {
          uint32_t bf[2][KS][2];
          load_b(nt, bf);
          const bool ragged = nt * 8 + 8 > kn;
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            float as[4] = {cs[mt * 2], cs[mt * 2], cs[mt * 2 + 1], cs[mt * 2 + 1]};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
              mma_16816(as, af[mt][0][ks], bf[0][ks][0], bf[0][ks][1]);
              mma_16816(as, af[mt][1][ks], bf[1][ks][0], bf[1][ks][1]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int r = mt * 2 + (i >> 1);
              float v = as[i];
              if (ragged && nt * 8 + 2 * t4 + (i & 1) >= kn) v = inf;
              if constexpr (WANT2) {
                const float lo = fminf(s1[r], v), hi = fmaxf(s1[r], v);
                s1[r] = lo;
                s2[r] = fminf(s2[r], hi);
              } else {
                s1[r] = fminf(s1[r], v);
              }
            }
          }
        }
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
#pragma unroll
        for (int x = 1; x <= 2; x <<= 1) {   // the quad's peaks are disjoint: merge the top-2 lists
          const float o1 = __shfl_xor_sync(0xffffffffu, s1[r], x);
          const float o2 = __shfl_xor_sync(0xffffffffu, s2[r], x);
          const float lo = fminf(s1[r], o1), hi = fmaxf(s1[r], o1);
          s2[r] = fminf(hi, fminf(s2[r], o2));
          s1[r] = lo;
        }
        const int m = wid * 32 + (r >> 1) * 16 + (r & 1) * 8 + g;
        // d^2 <= 2 S_true <= 2 (S_lo + slack);  slack = 2 delta_x + 2 delta_y (+ rounding, in d2y)
        const float sref = WANT2 ? s2[r] : s1[r];
        // rows without a usable pixel get a NaN threshold: no comparison with it is ever true (their accumulators
        // may hold anything, -inf included, because the tile column is stale or non-finite)
        thr[r] = live[r] ? 2.0f * (fmaxf(sref, 0.0f) + s_d2x[m] + s_d2y[m]) * (1.0f + 1e-4f) + 1e-6f
                         : __int_as_float(0x7fc00000);
      }

      // sweep 2: one compare per pair; the few pairs that pass go to the warp's queue
      int q_tail = 0;
      bool q_over = false;
      const int row_l = wid * 32 + lane;                 // lane <-> one of the warp's 32 rows

      // Evaluates the bounds of the queued pairs, takes the smallest upper bound U of every row, drops the pairs
      // whose lower bound exceeds U (they can never win) and tightens the rows' thresholds to U^2.  Thresholds
      // only ever shrink, so dropping is final.  All 32 lanes take part.
      auto tighten = [&]() {
        for (int e = lane; e < q_tail; e += 32) {
          const AmEntry en = my_queue[e];
          const int m = (en.rk >> 24) & 0xff, k = en.rk & kEntryKMask;
          float dhi = en.hi;
          if (!(en.rk & kEntryDone)) {
            const float dlo = (__fsqrt_rn(fmaxf(en.a, 0.0f)) + __fsqrt_rn(fmaxf(en.b, 0.0f))) * (1.0f - 2e-6f);
            dhi = (__fsqrt_rn(fmaxf(en.a + s_d2x[m], 0.0f)) + __fsqrt_rn(fmaxf(en.b + s_d2y[m], 0.0f))) *
                  (1.0f + 2e-6f);
            my_queue[e].a = dlo;
            my_queue[e].hi = dhi;
            my_queue[e].rk = en.rk | kEntryDone;
          }
          atomicMin(&s_u1[m], pack_dk(dhi, k));
        }
        if constexpr (WANT2) {
          s_u2[row_l] = kPackEmpty;
          __syncwarp();
          for (int e = lane; e < q_tail; e += 32) {
            const AmEntry en = my_queue[e];
            const int m = (en.rk >> 24) & 0xff, k = en.rk & kEntryKMask;
            if (k != pack_k(s_u1[m])) atomicMin(&s_u2[m], pack_dk(en.hi, k));
          }
        }
        __syncwarp();
        int kept = 0;
        for (int base = 0; base < q_tail; base += 32) {
          const int e = base + lane;
          AmEntry en;
          bool keep = false;
          if (e < q_tail) {
            en = my_queue[e];
            const int m = (en.rk >> 24) & 0xff;
            const unsigned long long u = WANT2 ? s_u2[m] : s_u1[m];
            const float Um = (u == kPackEmpty) ? inf : pack_d(u) * (1.0f + 4e-5f) + 1e-6f;
            keep = en.a <= Um;
          }
          const uint32_t km = __ballot_sync(0xffffffffu, keep);
          __syncwarp();
          if (keep && am_ok(kept + __popc(km & ((1u << lane) - 1u)) < kAmQueue, 5u, status))
            my_queue[kept + __popc(km & ((1u << lane) - 1u))] = en;
          kept += __popc(km);
          __syncwarp();
        }
        q_tail = kept;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int m = wid * 32 + (r >> 1) * 16 + (r & 1) * 8 + g;
          const unsigned long long u = WANT2 ? s_u2[m] : s_u1[m];
          if (u != kPackEmpty && live[r]) {
            const float Um = pack_d(u) * (1.0f + 4e-5f) + 1e-6f;
            thr[r] = fminf(thr[r], Um * Um * (1.0f + 1e-6f));
          }
        }
      };

      // The first pair of a row that passes stays in this thread's registers: most rows have exactly one such
      // pair in the whole sweep, and are then decided without touching the queue.
      const bool force_queue = WANT2 || need_exact;       // scores wanted: every row goes through the queue
      int rk_[4] = {-1, -1, -1, -1};
      float ra_[4] = {0.0f, 0.0f, 0.0f, 0.0f}, rb_[4] = {0.0f, 0.0f, 0.0f, 0.0f};
      uint32_t extra = 0;                                   // 8 bits per row: pairs of mine that went to the queue

      // Appends the marked slots (bit j of `mask` <-> prk[j], pa[j], pb[j]) to the warp's queue, in lane order.
      auto queue_push = [&](uint32_t mask, const int (&prk)[8], const float (&pa)[8], const float (&pb)[8], int total,
                            int excl) {
        int pos = q_tail + excl;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if ((mask >> j) & 1u) {
            AmEntry e;
            e.rk = prk[j];
            e.a = pa[j];
            e.b = pb[j];
            e.hi = 0.0f;
            if (am_ok(pos >= 0 && pos < kAmQueue, 2u, status)) my_queue[pos] = e;
            ++pos;
            ++n_pairs;
          }
        q_tail += total;
        __syncwarp();
      };
      auto warp_scan = [&](int cnt, int& excl, int& total) {
        int incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += v;
        }
        total = __shfl_sync(0xffffffffu, incl, 31);
        excl = incl - cnt;
      };

      for (int pc = 0; pc < n_pchunks; ++pc) {
        if (n_pchunks > 1) { __syncthreads(); load_peaks(pc); __syncthreads(); }
        const int k0 = pc * peak_cap;
        const int kn = min(peak_cap, K - k0);
        const int n_tiles = (kn + 7) >> 3;
        for (int nt = 0; nt < n_tiles; ++nt) {
          uint32_t bf[2][KS][2];
          load_b(nt, bf);
          const bool ragged = nt * 8 + 8 > kn;
          // A and B separately (the legacy tensor path is the scarce resource here: two MMAs and an add per
          // pair are cheaper than a third MMA that would deliver S directly)
          float as[2][4], ax[2][4];
          bool any = false;
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            float ay[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              ax[mt][i] = cx[mt * 2 + (i >> 1)];
              ay[i] = cy[mt * 2 + (i >> 1)];
            }
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
              mma_16816(ax[mt], af[mt][0][ks], bf[0][ks][0], bf[0][ks][1]);
              mma_16816(ay, af[mt][1][ks], bf[1][ks][0], bf[1][ks][1]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              as[mt][i] = ax[mt][i] + ay[i];
              // the test of pass_mask below, evaluated here already: on workloads whose candidates all lie at about
              // the same distance the coarser S <= thr alone passes for nearly every pair
              const float S = as[mt][i], A = ax[mt][i];
              any = any || (fmaf(2.0f, fminf(A, S - A), S) <= thr[mt * 2 + (i >> 1)]);
            }
          }
          if (__any_sync(0xffffffffu, any)) {
            auto pass_mask = [&]() {
              uint32_t pm = 0;
#pragma unroll
              for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int r = mt * 2 + (i >> 1);
                  const float S = as[mt][i], A = ax[mt][i], Bv = S - A;
                  bool p = S <= thr[r];
                  // S + 2 min(A, B) <= (sqrt A + sqrt B)^2 as well
                  p = p && (fmaf(2.0f, fminf(A, Bv), S) <= thr[r]);
                  if (ragged && nt * 8 + 2 * t4 + (i & 1) >= kn) p = false;
                  if (p) pm |= 1u << (mt * 4 + i);
                }
              return pm;
            };
            uint32_t passmask = pass_mask();
            uint32_t taken = 0;
            if (!force_queue) {
#pragma unroll
              for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int r = mt * 2 + (i >> 1), j = mt * 4 + i;
                  if (((passmask >> j) & 1u) && rk_[r] < 0) {
                    rk_[r] = k0 + nt * 8 + 2 * t4 + (i & 1);
                    ra_[r] = ax[mt][i];
                    rb_[r] = as[mt][i] - ax[mt][i];
                    taken |= 1u << j;
                  }
                }
              passmask &= ~taken;
            }
            if (__any_sync(0xffffffffu, passmask != 0) && !q_over) {
              int excl = 0, total = 0;
              warp_scan(__popc(passmask), excl, total);
              if (q_tail + total > kAmQueue) {
                tighten();
                passmask = pass_mask() & ~taken;
                warp_scan(__popc(passmask), excl, total);
                if (q_tail + total > kAmQueue) q_over = true;
              }
              if (!q_over) {
                int prk[8];
                float pa[8], pb[8];
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const int j = mt * 4 + i;
                    const int row = wid * 32 + mt * 16 + (i >> 1) * 8 + g;
                    prk[j] = (row << 24) | (k0 + nt * 8 + 2 * t4 + (i & 1));
                    pa[j] = ax[mt][i];
                    pb[j] = as[mt][i] - ax[mt][i];
                    if ((passmask >> j) & 1u) extra += 1u << (8 * (mt * 2 + (i >> 1)));
                  }
                queue_push(passmask, prk, pa, pb, total, excl);
              }
            }
          }
        }
      }
      __syncwarp();

      // ---- rows with a single surviving pair in the whole quad are decided here; the others go to the queue
      {
        uint32_t packed = extra;
#pragma unroll
        for (int r = 0; r < 4; ++r) packed += (rk_[r] >= 0 ? 1u : 0u) << (8 * r);
        uint32_t mine_cnt = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) mine_cnt += (rk_[r] >= 0 ? 1u : 0u);
        n_pairs += mine_cnt;
        packed += __shfl_xor_sync(0xffffffffu, packed, 1);
        packed += __shfl_xor_sync(0xffffffffu, packed, 2);
        uint32_t pushmask = 0;
        int prk[8];
        float pa[8], pb[8];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int m = wid * 32 + (r >> 1) * 16 + (r & 1) * 8 + g;
          prk[r] = (m << 24) | (rk_[r] & kEntryKMask);
          pa[r] = ra_[r];
          pb[r] = rb_[r];
          prk[r + 4] = 0; pa[r + 4] = 0.0f; pb[r + 4] = 0.0f;
          if (rk_[r] >= 0) {
            if (((packed >> (8 * r)) & 0xffu) == 1u && !q_over) {
              const int o = (int)s_rowoff[m];
              if (am_ok(o < span_len, 3u, status)) s_lab[o] = rk_[r] + 1;
            }
            else pushmask |= 1u << r;
          }
        }
        if (__any_sync(0xffffffffu, pushmask != 0) && !q_over) {
          int excl = 0, total = 0;
          warp_scan(__popc(pushmask), excl, total);
          if (q_tail + total > kAmQueue) {
            tighten();
            if (q_tail + total > kAmQueue) q_over = true;
          }
          if (!q_over) queue_push(pushmask, prk, pa, pb, total, excl);
        }
      }
      const bool any_hard = __any_sync(0xffffffffu, (s_flag[row_l] & kRowHard) != 0) || q_over;
      if (q_tail == 0 && !any_hard && !best_img) continue;   // warp-uniform: nothing left for this warp in this tile

      // ---- drain: all lanes busy on the warp's queue
      auto pixel = [&](int m, const T* src, int axis, int c) -> float {
        if constexpr (sizeof(T) == 2) return __half2float(s_tile[(size_t)(axis * KA + c) * kAmTilePitch + m]);
        else return Elem<T>::load1(src + (size_t)(axis * 2 * F + c) * plane);
      };
      auto exact = [&](int m, int k) -> float {
        if (!am_ok(m >= 0 && m < kAmMT && k >= 0 && k < K && (int)s_rowoff[m] < span_len, 4u, status)) return inf;
        const T* src = e_img + span0 + (int)s_rowoff[m];
        const float* pk = pk_img + (size_t)k * D;
        float sx = 0.0f, sy = 0.0f;
        for (int c = 0; c < 2 * F; ++c) {
          const float v = __fsub_rn(pixel(m, src, 0, c), __ldg(pk + c));
          sx = __fmaf_rn(v, v, sx);
        }
        for (int c = 0; c < 2 * F; ++c) {
          const float v = __fsub_rn(pixel(m, src, 1, c), __ldg(pk + 2 * F + c));
          sy = __fmaf_rn(v, v, sy);
        }
        return __fadd_rn(__fsqrt_rn(sx), __fsqrt_rn(sy));
      };

      tighten();                                          // what is left in the queue are the candidates
      for (int e = lane; e < q_tail; e += 32) {
        const AmEntry en = my_queue[e];
        const int m = (en.rk >> 24) & 0xff;
        atomicAdd(&s_nc[m], 1u);
        s_ck[m] = en.rk & kEntryKMask;                   // used only when it is the row's single candidate
      }
      __syncwarp();
      // exact scores where a row has several candidates (or the score itself is wanted)
      for (int e = lane; e < q_tail; e += 32) {
        const AmEntry en = my_queue[e];
        const int m = (en.rk >> 24) & 0xff, k = en.rk & kEntryKMask;
        if (!WANT2 && !need_exact && s_nc[m] == 1u) continue;
        const float f = exact(m, k);
        my_queue[e].b = f;
        atomicMin(&s_best[m], pack_dk(f, k));
      }
      __syncwarp();
      if constexpr (WANT2) {
        for (int e = lane; e < q_tail; e += 32) {
          const AmEntry en = my_queue[e];
          const int m = (en.rk >> 24) & 0xff, k = en.rk & kEntryKMask;
          if (k != pack_k(s_best[m])) atomicMin(&s_second[m], pack_dk(en.b, k));
        }
        __syncwarp();
      }
      // rows that must score every peak: out-of-range pixels, or a queue that overflowed
      {
        const uint32_t f = s_flag[row_l];
        const bool hard = (f & kRowValid) && ((f & kRowHard) || q_over);
        uint32_t hmask = __ballot_sync(0xffffffffu, hard);
        while (hmask) {
          const int hl = __ffs(hmask) - 1;
          hmask &= hmask - 1;
          const int m = wid * 32 + hl;
          if constexpr (sizeof(T) == 4) {
            // the binary16 copy could not tell an out-of-range value from a non-finite one: look at the originals
            const T* src = e_img + span0 + (int)s_rowoff[m];
            float fin = 0.0f;
            if (am_ok((int)s_rowoff[m] < span_len, 7u, status))
            for (int l = lane; l < 2 * F; l += 32)
              fin = fold_finite(fin, Elem<T>::load1(src + (size_t)(2 * l) * plane),
                                Elem<T>::load1(src + (size_t)(2 * l + 1) * plane));
            if (__any_sync(0xffffffffu, fin != fin)) {
              if (lane == 0) { s_flag[m] = 0; s_best[m] = kPackEmpty; s_second[m] = kPackEmpty; s_nc[m] = 0; }
              __syncwarp();
              continue;
            }
          }
          if (lane == 0) { s_best[m] = kPackEmpty; s_second[m] = kPackEmpty; s_nc[m] = 2u; ++n_full; }
          __syncwarp();
          for (int k = lane; k < K; k += 32) atomicMin(&s_best[m], pack_dk(exact(m, k), k));
          __syncwarp();
          if constexpr (WANT2) {
            const int kb = pack_k(s_best[m]);
            for (int k = lane; k < K; k += 32)
              if (k != kb) atomicMin(&s_second[m], pack_dk(exact(m, k), k));
            __syncwarp();
          }
        }
      }
      // one lane per row writes the outcome of the rows that went through the queue
      if (s_rowoff[row_l] != 0xffffu && am_ok((int)s_rowoff[row_l] < span_len, 6u, status)) {
        const uint32_t f = s_flag[row_l];
        const int off = (int)s_rowoff[row_l];
        float d1 = inf, d2 = inf;
        if (f & kRowValid) {
          const unsigned long long bb = s_best[row_l];
          if (bb != kPackEmpty) {
            d1 = pack_d(bb);
            if (d1 < tau) s_lab[off] = pack_k(bb) + 1; else ++rejected;
            if (s_nc[row_l] > 1u) ++n_rescored;
            if (WANT2 && s_second[row_l] != kPackEmpty) d2 = pack_d(s_second[row_l]);
          } else if (s_nc[row_l] == 1u) {
            s_lab[off] = s_ck[row_l] + 1;                // decided by the filter alone (tau = +inf, no scores)
          }
        }
        if (best_img) {
          best_img[span0 + off] = d1;
          second_img[span0 + off] = d2;
        }
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
  const uint32_t wp = __reduce_add_sync(0xffffffffu, n_pairs);
  const uint32_t ws = __reduce_add_sync(0xffffffffu, n_rescored);
  const uint32_t wf = __reduce_add_sync(0xffffffffu, n_full);
  if (lane == 0) {
    if (wr) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_TAU_REJECTED], wr);
    if (wp) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_FILTER_PAIRS], wp);
    if (ws) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_RESCORED], ws);
    if (wf) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_FULL_SCORED], wf);
  }
}

template <typename T, int KA, bool WANT2>
__global__ void __launch_bounds__(kAmThreads, 2)
assign_mma_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F, int K_max,
                  const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau, int need_exact,
                  int peak_cap, int span, int vec_mask, int vec_gather, int32_t* __restrict__ labels, float* __restrict__ best,
                  float* __restrict__ second, uint32_t* __restrict__ counters, uint32_t* __restrict__ status_all,
                  uint32_t* __restrict__ votes, int cells, int k_min, const uint32_t* __restrict__ near_state) {
  grid_dependency_sync();
  // after the pruned assignment (near_state given) this kernel only takes the images which that one handed on
  if (near_state) {
    if (blockIdx.x == 0 && threadIdx.x == 0) fold_near_counters(near_state, counters, blockIdx.y);
    if (!near_state[blockIdx.y * kNearStride + kNearGiveUp]) k_min = 0x7fffffff;
  }
  assign_mma_body<T, KA, WANT2>(emb, fg, HW, F, K_max, peak_emb, count_ptr, tau, need_exact, peak_cap, span, vec_mask, vec_gather, labels, best, second, counters, status_all, votes, cells, k_min);
}

}  // namespace cpe
