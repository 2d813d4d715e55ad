// Stage 4+5 with pruned candidates: pixel-to-instance assignment (Eq. 4, Eq. 7, Eq. 8) that scores, for every
// participating pixel, only the peaks that can still win, and the label-map write.
//
// The voting kernel left every pixel's bin in `pix_cell`; the peak kernel mapped bins to the peak k0 whose 3x3 window
// holds them (`cell_peak`); peak_graph_kernel listed, per k0, the candidates in ascending G (see peak_graph.cuh).  A
// pixel computes t, its distance to k0's reference point, and walks the list: a candidate is scored exactly -- in the
// one fixed binary32 order that every assignment kernel of this library uses, so the winner, its distance and the
// runner-up are the same bits as in the all-pairs kernel -- as long as G <= (U + t)(1 + 2e-5), where U is the best
// (with scores wanted: the second best) exact distance so far; the first entry beyond that ends the walk, because
// every later one has d >= G - t > U.  The slack covers the rounding of G (stored rounded down), t and U.
//
// A pixel whose bin belongs to no peak's window, or whose list runs out before the bound closes it, is "hard": it is
// scored against every peak.  When more than an eighth of an image's pixels turn out hard (candidates that no bound
// separates: a vote map too coarse for the harmonics, heavy noise), the image is handed to the tensor-core filtered
// kernel launched after this one (`near_state[kNearGiveUp]`), which then redoes it as a whole; both kernels compute
// the same bits, so pixels already written are simply written again.
#pragma once

#include "assign.cuh"
#include "cpe_common.cuh"
#include "peak_graph.cuh"

namespace cpe {

constexpr int kNearThreads = 256;
constexpr float kNearSlack = 1.00002f;

template <typename T, int FT, bool WANT2>
__global__ void __launch_bounds__(kNearThreads, FT == 16 ? 2 : 3)
assign_near_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int K_max,
                   const float* __restrict__ ref2, const float* __restrict__ cand2, const uint32_t* __restrict__ nbr,
                   const int32_t* __restrict__ cell_peak, const uint32_t* __restrict__ pix_cell, int cells,
                   const int32_t* __restrict__ count_ptr, float tau, int32_t* __restrict__ labels,
                   float* __restrict__ best, float* __restrict__ second, uint32_t* __restrict__ near_state,
                   int k_min) {
  grid_dependency_sync();
  constexpr int D = 4 * FT;
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  const size_t plane = (size_t)HW;
  const int K = count_ptr[b];
  if (K < k_min) return;                       // few peaks: the all-pairs kernel's image
  uint32_t* state = near_state + b * kNearStride;
  if (K > kNearMaxPeaks) {                      // no lists were made: the filtered kernel's image
    if (tid == 0 && blockIdx.x == 0) state[kNearGiveUp] = 1u;
    return;
  }
  const bool same_rows = ref2 == cand2;
  const float* ref_img = ref2 + (size_t)b * K_max * D;
  const float* cand_img = cand2 + (size_t)b * K_max * D;
  const uint32_t* nbr_img = nbr + (size_t)b * K_max * kNbrCap;
  const int32_t* cp_img = cell_peak + (size_t)b * cells;
  const float inf = __int_as_float(0x7f800000);

  __shared__ uint32_t s_stop;
  uint32_t n_rejected = 0, n_pairs = 0, n_multi = 0, n_full = 0;
  const long long n_blocks = ((long long)HW + kNearThreads - 1) / kNearThreads;
  for (long long blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
    const long long n = blk * kNearThreads + tid;
    bool act = n < HW;
    if (act && fg) act = __ldg(fg + (size_t)b * plane + n) != 0;
    uint32_t cell = 0xffffffffu;
    if (act) cell = __ldg(pix_cell + (size_t)b * plane + n);
    act = act && cell != 0xffffffffu && (int)cell < cells;    // no vote: a non-finite pixel
    int k0 = -1;
    float2 e2[D / 2];
    if (act) {
      k0 = __ldg(cp_img + cell);
      const T* p = emb + (size_t)b * D * plane + n;
#pragma unroll
      for (int c = 0; c < D / 2; ++c) {
        e2[c].x = Elem<T>::load1(p + (size_t)c * plane);
        e2[c].y = Elem<T>::load1(p + (size_t)(D / 2 + c) * plane);
      }
    }

    float d1 = inf, d2 = inf;
    int k1 = -1;
    bool hard = act && (k0 < 0 || k0 >= K);
    uint32_t scored = 0;
    if (act && !hard) {
      const float t = score_direct<D>(e2, reinterpret_cast<const float2*>(ref_img + (size_t)k0 * D), inf);
      const uint32_t* list = nbr_img + (size_t)k0 * kNbrCap;
      float bound2 = inf;
      int j = 0;
      for (; j < kNbrCap; ++j) {
        const uint32_t ent = __ldg(list + j);
        if (ent == kNbrEnd) break;                                   // every candidate of the image has been seen
        const float G = (float)(ent >> 12) * (1.0f / 65536.0f);
        const float U = WANT2 ? d2 : d1;
        if (G > (U + t) * kNearSlack) break;                         // this one and all later ones: d >= G - t > U
        const int k = (int)(ent & 0xfffu);
        const float d = (same_rows && k == k0)
                            ? t
                            : score_direct<D>(e2, reinterpret_cast<const float2*>(cand_img + (size_t)k * D), bound2);
        ++scored;
        if (d < d1 || (d == d1 && k < k1)) { d2 = d1; d1 = d; k1 = k; }   // the lowest k keeps an exact tie
        else if (d < d2) { d2 = d; }
        const float bound = WANT2 ? d2 : d1;
        bound2 = bound * bound * (1.0f + 1e-6f);
      }
      hard = (j == kNbrCap) && K > kNbrCap;                          // the list ran out before the bound closed it
    }

    // hard pixels: count them, let the image go to the filtered kernel if there are too many, else score every peak
    // (the ratio is taken over all pixels visited, participating or not)
    const int n_hard = __syncthreads_count(hard);
    if (n_hard) {
      if (tid == 0) {
        const uint32_t proc = atomicAdd(&state[kNearProcessed], (uint32_t)kNearThreads) + (uint32_t)kNearThreads;
        const uint32_t hd = atomicAdd(&state[kNearHard], (uint32_t)n_hard) + (uint32_t)n_hard;
        uint32_t stop = *reinterpret_cast<volatile uint32_t*>(&state[kNearGiveUp]);
        if (!stop && proc >= 8192u && hd > proc / 8u) {
          atomicExch(&state[kNearGiveUp], 1u);
          stop = 1u;
        }
        s_stop = stop;
      }
      __syncthreads();
      if (s_stop) return;                                            // the filtered kernel redoes the whole image
      if (hard) {
        d1 = d2 = inf;
        k1 = -1;
        float bound2 = inf;
        for (int k = 0; k < K; ++k) {
          const float d = score_direct<D>(e2, reinterpret_cast<const float2*>(cand_img + (size_t)k * D), bound2);
          if (d < d1) { d2 = d1; d1 = d; k1 = k; }
          else if (d < d2) { d2 = d; }
          const float bound = WANT2 ? d2 : d1;
          bound2 = bound * bound * (1.0f + 1e-6f);
        }
        scored = (uint32_t)K;
        ++n_full;
      }
    } else if (tid == 0) {
      atomicAdd(&state[kNearProcessed], (uint32_t)kNearThreads);
    }

    int label = 0;
    if (act && k1 >= 0) {
      if (d1 < tau) label = k1 + 1;
      else ++n_rejected;
    }
    n_pairs += scored;
    if (scored > 1 && !hard) ++n_multi;
    if (n < HW) {
      const size_t o = (size_t)b * plane + n;
      labels[o] = label;
      if (WANT2) {
        best[o] = act ? d1 : inf;
        second[o] = act ? d2 : inf;
      }
    }
  }
  // counters: one atomic per warp and counter, into this kernel's own words; the last kernel of the chain folds them
  // into the image's counters unless the image was handed on (a CTA that returned above has dropped its share)
  const uint32_t rej = __reduce_add_sync(0xffffffffu, n_rejected), prs = __reduce_add_sync(0xffffffffu, n_pairs),
                 mul = __reduce_add_sync(0xffffffffu, n_multi), ful = __reduce_add_sync(0xffffffffu, n_full);
  if ((tid & 31) == 0) {
    if (rej) atomicAdd(&state[kNearCnt + 0], rej);
    if (prs) atomicAdd(&state[kNearCnt + 1], prs);
    if (mul) atomicAdd(&state[kNearCnt + 2], mul);
    if (ful) atomicAdd(&state[kNearCnt + 3], ful);
  }
}

}  // namespace cpe
