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
//
// Three kernels.  assign_near_stream_kernel (16-byte aligned planes, no scores wanted) streams the embedding the way
// the voting kernel does -- a thread takes (8-pixel group, axis), 128-bit plane loads, background never fetched --
// and only certifies, from cheap upper bounds of t and of the distance to the first candidate of k0's list, that the
// second list entry is already out of reach (nearly every pixel when the candidates sit on the voted centroids):
// the label is then final.  The other pixels are decided exactly by a walk of the list, one thread per pixel: a warp's
// first few by the warp itself once it has streamed its share, the rest through a queue in global memory by
// assign_near_walk_kernel.  assign_near_kernel is that walk for every pixel: any alignment, and scores.
#pragma once

#include "assign.cuh"
#include "cpe_common.cuh"
#include "peak_graph.cuh"

namespace cpe {

constexpr int kNearThreads = 256;
constexpr int kWarpQueue = 64;         // pixels that a warp of the streaming kernel keeps for its own walks
constexpr float kNearSlack = 1.00002f;
constexpr int kNearWalkMax = 12;     // list entries one thread walks before the pixel goes to the warp-wide scan

// The walk of one pixel, given its 4F values as (x channel c, y channel c) pairs.
template <int D, bool WANT2>
__device__ __forceinline__ void near_walk(const float2 (&e2)[D / 2], int k0, int K, bool same_rows,
                                          const float* __restrict__ ref_img, const float* __restrict__ cand_img,
                                          const uint32_t* __restrict__ nbr_img, float& d1, float& d2, int& k1, bool& hard,
                                          uint32_t& scored) {
  const float inf = __int_as_float(0x7f800000);
  const float t = score_direct<D>(e2, reinterpret_cast<const float2*>(ref_img + (size_t)k0 * D), inf);
  const uint32_t* list = nbr_img + (size_t)k0 * kNbrCap;
  float bound2 = inf;
  int j = 0;
  constexpr int kWalkMax = WANT2 ? kNbrCap : kNearWalkMax;       // (the runner-up alone needs a longer walk)
  for (; j < kNbrCap && j < kWalkMax; ++j) {
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
  // the list ran out before the bound closed it, or the walk is getting long: a thread's walk is a chain of dependent
  // row fetches, and a pixel far from its reference point (large t) would go through most of the list that way -- it
  // is handed to the warp-wide scan instead
  hard = (j == kNbrCap && K > kNbrCap) || (!WANT2 && j == kWalkMax);
}

// Every peak of an image for one pixel (a hard pixel), by a whole warp (every lane passes the same pixel): a lane
// scores the peaks k_first, k_first + k_stride, ... (lane, 32 for a warp on its own; several warps may share one pixel)
// with the pixel's values fetched by every lane (the same addresses: one transaction per load), then the lanes' results
// are merged -- smaller distance first, lower k on equal distances, which is what the serial scan in ascending k gives.
// A single thread scanning hundreds of peaks is a chain of dependent row fetches that takes as long as the rest of the
// kernel; 32 lanes share it.
template <typename T, int D, bool WANT2>
__device__ __forceinline__ void near_full_scan_warp(const T* __restrict__ p, size_t plane, int K,
                                                    const float* __restrict__ cand_img, float& d1, float& d2, int& k1,
                                                    int k_first, int k_stride) {
  const float inf = __int_as_float(0x7f800000);
  float2 e2[D / 2];
#pragma unroll
  for (int c = 0; c < D / 2; ++c) {
    e2[c].x = Elem<T>::load1(p + (size_t)c * plane);
    e2[c].y = Elem<T>::load1(p + (size_t)(D / 2 + c) * plane);
  }
  d1 = d2 = inf;
  k1 = 0x7fffffff;
  float bound2 = inf;
  for (int k = k_first; k < K; k += k_stride) {
    const float d = score_direct<D>(e2, reinterpret_cast<const float2*>(cand_img + (size_t)k * D), bound2);
    if (d < d1) { d2 = d1; d1 = d; k1 = k; }
    else if (d < d2) { d2 = d; }
    const float bound = WANT2 ? d2 : d1;
    bound2 = bound * bound * (1.0f + 1e-6f);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float od1 = __shfl_xor_sync(0xffffffffu, d1, off), od2 = __shfl_xor_sync(0xffffffffu, d2, off);
    const int ok1 = __shfl_xor_sync(0xffffffffu, k1, off);
    const bool other_wins = od1 < d1 || (od1 == d1 && ok1 < k1);
    const float loser = other_wins ? d1 : od1;       // the larger of the two best distances is a runner-up candidate
    if (other_wins) { d1 = od1; k1 = ok1; }
    d2 = fminf(fminf(d2, od2), loser);
  }
  if (k1 == 0x7fffffff) k1 = -1;
}

// Called by one thread of a CTA with the hard pixels it has just found among `visited` pixels: updates the image's
// totals and decides whether the image is handed on.  Returns the stop flag.
// (Hard pixels come in clusters -- an instance whose peak a stronger neighbour suppressed --, so the ratio is only
// looked at once an eighth of the image has been visited.)
// (proc_floor: the caller's own estimate of the pixels visited so far by everybody, for callers that report pixels
// without hard ones only now and then -- the counter alone would then lag behind the hard pixels' count.)
__device__ __forceinline__ uint32_t near_account(uint32_t* state, uint32_t visited, uint32_t n_hard, uint32_t min_proc,
                                                 uint32_t proc_floor = 0u) {
  const uint32_t proc = max(atomicAdd(&state[kNearProcessed], visited) + visited, proc_floor);
  if (!n_hard) return *reinterpret_cast<volatile uint32_t*>(&state[kNearGiveUp]);
  const uint32_t hd = atomicAdd(&state[kNearHard], n_hard) + n_hard;
  uint32_t stop = *reinterpret_cast<volatile uint32_t*>(&state[kNearGiveUp]);
  if (!stop && proc >= min_proc && hd > proc / 8u) {
    atomicExch(&state[kNearGiveUp], 1u);
    stop = 1u;
  }
  return stop;
}

__device__ __forceinline__ void near_flush_counters(uint32_t* state, uint32_t n_rejected, uint32_t n_pairs,
                                                    uint32_t n_multi, uint32_t n_full) {
  // one atomic per warp and counter, into this kernel's own words; the last kernel of the chain folds them into the
  // image's counters unless the image was handed on (a CTA that returned early has dropped its share)
  const uint32_t rej = __reduce_add_sync(0xffffffffu, n_rejected), prs = __reduce_add_sync(0xffffffffu, n_pairs),
                 mul = __reduce_add_sync(0xffffffffu, n_multi), ful = __reduce_add_sync(0xffffffffu, n_full);
  if ((threadIdx.x & 31) == 0) {
    if (rej) atomicAdd(&state[kNearCnt + 0], rej);
    if (prs) atomicAdd(&state[kNearCnt + 1], prs);
    if (mul) atomicAdd(&state[kNearCnt + 2], mul);
    if (ful) atomicAdd(&state[kNearCnt + 3], ful);
  }
}

// ------------------------------------------------------------------------------------------------ one thread per pixel

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
  if (K < k_min) {
    // Not this kernel's image -- unless it has no peak at all and this chain serves every image (k_min = 1): then
    // every pixel's label is 0 and its scores are +inf.
    if (K == 0 && k_min == 1) {
      const float inf0 = __int_as_float(0x7f800000);
      for (long long n = (long long)blockIdx.x * kNearThreads + tid; n < HW; n += (long long)gridDim.x * kNearThreads) {
        const size_t o = (size_t)b * plane + n;
        labels[o] = 0;
        if (WANT2) {
          best[o] = inf0;
          second[o] = inf0;
        }
      }
    }
    return;
  }
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
    if (act && !hard) near_walk<D, WANT2>(e2, k0, K, same_rows, ref_img, cand_img, nbr_img, d1, d2, k1, hard, scored);

    // hard pixels: count them, let the image go to the filtered kernel if there are too many, else score every peak
    // (the ratio is taken over all pixels visited, participating or not)
    const int n_hard = __syncthreads_count(hard);
    if (n_hard) {
      if (tid == 0) s_stop = near_account(state, (uint32_t)kNearThreads, (uint32_t)n_hard, max(8192u, (uint32_t)HW / 8u));
      __syncthreads();
      if (s_stop) return;                                            // the filtered kernel redoes the whole image
      // every peak, by the whole warp, one hard pixel after the other
      uint32_t hm = __ballot_sync(0xffffffffu, hard);
      while (hm) {
        const int src_lane = __ffs(hm) - 1;
        hm &= hm - 1;
        const long long nn = __shfl_sync(0xffffffffu, n, src_lane);
        float w1, w2;
        int wk;
        near_full_scan_warp<T, D, WANT2>(emb + (size_t)b * D * plane + nn, plane, K, cand_img, w1, w2, wk, (int)(threadIdx.x & 31), 32);
        if ((tid & 31) == src_lane) {
          d1 = w1;
          d2 = w2;
          k1 = wk;
          scored = (uint32_t)K;
          ++n_full;
        }
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
  near_flush_counters(state, n_rejected, n_pairs, n_multi, n_full);
}

// ------------------------------------------------------------------------------------------------ the streaming kernel

// Square root to within 2^-21 relative (the special-function unit's), for bounds that carry their own slack.
__device__ __forceinline__ float fast_sqrt(float x) {
  float r;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

// Shuffles of packed binary16 pairs as plain 32-bit words.
__device__ __forceinline__ uint32_t h2_bits(__half2 v) {
  return (uint32_t)__half_as_ushort(__low2half(v)) | ((uint32_t)__half_as_ushort(__high2half(v)) << 16);
}
__device__ __forceinline__ __half2 bits_h2(uint32_t w) {
  return __halves2half2(__ushort_as_half((unsigned short)(w & 0xffffu)), __ushort_as_half((unsigned short)(w >> 16)));
}
__device__ __forceinline__ __half2 shfl_xor_h2(__half2 v, int off) {
  return bits_h2(__shfl_xor_sync(0xffffffffu, h2_bits(v), off));
}
__device__ __forceinline__ __half2 shfl_h2(__half2 v, int src) {
  return bits_h2(__shfl_sync(0xffffffffu, h2_bits(v), src));
}

constexpr int kStreamThreads = 256;
// Two CTAs per SM (the step's working set needs more than the 85 registers that three would leave: it spilled), and
// the plane loads of this many harmonics in flight per thread.
__host__ __device__ constexpr int stream_ctas_per_sm(int) { return 2; }
__host__ __device__ constexpr int stream_level_batch(int ft) { return ft >= 4 ? 4 : ft; }
// What turns a distance accumulated in packed binary16 into an upper bound of the true one.  Per axis the sum has at
// most 32 non-negative terms: each rounding (difference, fused multiply-add) is within 2^-11 relative, so the sum is
// within 34 * 2^-11 < 1.7 %, its root within 0.85 %; the candidate rows are rounded to binary16 (2^-12 per component,
// |r| <= 1: at most sqrt(32) * 2^-12 = 0.0014 on the norm); binary32 pixels are rounded to binary16 first (2^-11
// relative per component: at most 0.0005 ||v||, with ||v|| <= 8 for anything that is not far from every row anyway).
// Non-finite sums (overflow) fail every comparison and send the pixel to the exact walk.
constexpr float kHalfRel = 1.01f, kHalfAbs = 0.008f;

// Warps stream the embedding with 128-bit plane loads, a thread per (8-pixel group, axis) -- the access pattern of the
// voting kernel -- and only have to CERTIFY, per pixel, that the second entry of its peak's list is out of reach:
//     G_2 > (d_ub + t_ub) * slack,   t_ub >= t (distance to the reference point),  d_ub >= d (to the first candidate).
// Upper bounds need no exact arithmetic: the sums of squares are accumulated in packed binary16 (two pixels per
// instruction, no widening of the loaded values) and inflated by their worst-case error.  A certified pixel gets the
// first candidate's label; every other pixel -- not certified, no peak for its bin, tau finite (the exact distance is
// then needed) -- is decided exactly by a walk of its list: the first kWarpQueue of a warp by the warp itself when its
// share of the image is done, the rest (and all of them when tau is finite) appended to the image's queue in global
// memory (`slow_q`, capacity q_cap; its fill is near_state[kNearQueue]) for assign_near_walk_kernel.  A queue that
// overflows hands the image to the filtered kernel, like too many hard pixels do.
//
// Dynamic shared memory (`smem_rows_bytes`): binary16 copies of the reference rows [K][D] and, unless SAME, of the
// candidate rows; an image whose rows do not fit reads them from global memory (`ref_h` / `cand_h`, [K][D] binary16,
// written by peak_graph_kernel).  Needs 16-byte aligned planes, mask and labels, and H*W a multiple of the group size.
template <typename T, int FT, bool SAME>
__global__ void __launch_bounds__(kStreamThreads, stream_ctas_per_sm(FT))
assign_near_stream_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int K_max,
                          const __half* __restrict__ ref_h, const __half* __restrict__ cand_h,
                          const uint32_t* __restrict__ nbr, const int32_t* __restrict__ cell_peak,
                          const uint32_t* __restrict__ pix_cell, int cells, const int32_t* __restrict__ count_ptr, float tau,
                          int32_t* __restrict__ labels, uint32_t* __restrict__ near_state, uint32_t* __restrict__ slow_q,
                          int q_cap, int k_min, int smem_rows_bytes, const float* __restrict__ ref2,
                          const float* __restrict__ cand2, uint32_t* __restrict__ hard_q) {
  extern __shared__ __align__(16) unsigned char near_smem[];
  // A warp keeps the first kWarpQueue pixels that it cannot certify to itself and walks their lists when its share of
  // the image is done (a lane per pixel, as assign_near_walk_kernel does for the rest): the walks are chains of
  // dependent fetches, which hide behind the other warps' streaming instead of waiting for a kernel of their own.
  __shared__ uint32_t s_wq[kStreamThreads / 32][kWarpQueue];
  grid_dependency_sync();
  constexpr int VEC = Elem<T>::kVec;           // pixels per 128-bit load
  constexpr int H2 = VEC / 2;
  constexpr int F = FT, D = 4 * FT, D2 = 2 * FT;
  const int b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const size_t plane = (size_t)HW;
  const int K = count_ptr[b];
  if (K < k_min) {
    // Not this kernel's image -- unless it has no peak at all and this chain serves every image (k_min = 1): then
    // every pixel's label is 0 (the label map is 16-byte aligned and H*W a multiple of four here).
    if (K == 0 && k_min == 1) {
      int4* z = reinterpret_cast<int4*>(labels + (size_t)b * plane);
      for (long long i = (long long)blockIdx.x * kStreamThreads + tid; i < (long long)HW / 4; i += (long long)gridDim.x * kStreamThreads)
        z[i] = make_int4(0, 0, 0, 0);
    }
    return;
  }
  uint32_t* state = near_state + b * kNearStride;
  if (K > kNearMaxPeaks) {                      // no lists were made: the filtered kernel's image
    if (tid == 0 && blockIdx.x == 0) state[kNearGiveUp] = 1u;
    return;
  }
  const T* e_img = emb + (size_t)b * D * plane;
  const uint32_t* nbr_img = nbr + (size_t)b * K_max * kNbrCap;
  const int32_t* cp_img = cell_peak + (size_t)b * cells;
  const uint32_t* pc_img = pix_cell + (size_t)b * plane;
  int32_t* lab_img = labels + (size_t)b * plane;
  uint32_t* q_img = slow_q + (size_t)b * q_cap;

  // the rows this CTA bounds against (binary16): in shared memory if this image's peaks fit
  const bool rows_in_smem = (size_t)K * D * sizeof(__half) * (SAME ? 1 : 2) <= (size_t)smem_rows_bytes;
  const __half* rows_ref = rows_in_smem ? reinterpret_cast<const __half*>(near_smem) : ref_h + (size_t)b * K_max * D;
  const __half* rows_cand = SAME ? rows_ref
                                 : (rows_in_smem ? reinterpret_cast<const __half*>(near_smem) + (size_t)K * D
                                                 : cand_h + (size_t)b * K_max * D);
  if (rows_in_smem) {
    const uint4* g_ref = reinterpret_cast<const uint4*>(ref_h + (size_t)b * K_max * D);
    const uint4* g_cand = reinterpret_cast<const uint4*>(cand_h + (size_t)b * K_max * D);
    uint4* dst = reinterpret_cast<uint4*>(near_smem);
    const int n16 = K * D * (int)sizeof(__half) / 16;
    for (int i = tid; i < n16; i += kStreamThreads) {
      dst[i] = __ldg(g_ref + i);
      if (!SAME) dst[n16 + i] = __ldg(g_cand + i);
    }
    __syncthreads();
  }

  const bool certify = !(tau < __int_as_float(0x7f800000));   // with a finite tau every pixel needs its exact distance
  const uint32_t min_proc = max(8192u, (uint32_t)HW / 8u);
  uint32_t n_pairs = 0;
  uint32_t wq_n = 0;                            // fill of this warp's own queue (uniform over the warp)
  uint32_t visited = 0, hard_acc = 0;          // lane 0: not yet added to the image's totals
  uint32_t visited_all = 0;                     // pixels this warp has been through
  const int axis = lane & 1;                    // lanes 2j and 2j+1 share a group
  const long long n_groups = (long long)HW / VEC;
  const long long n_steps = (n_groups + 15) / 16;
  const long long warp0 = (long long)blockIdx.x * (kStreamThreads / 32) + wid, n_warps = (long long)gridDim.x * (kStreamThreads / 32);

  auto load_take = [&](long long step) -> uint32_t {      // participation bits of this lane's group in that step
    const long long grp = step * 16 + (lane >> 1);
    if (step < 0 || grp >= n_groups) return 0u;
    if (!fg) return (1u << VEC) - 1u;
    const uint8_t* m = fg + (size_t)b * plane + (size_t)grp * VEC;
    uint32_t take = 0;
    if constexpr (VEC == 8) {
      const uint2 w = __ldg(reinterpret_cast<const uint2*>(m));
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        take |= (((w.x >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
        take |= (((w.y >> (8 * j)) & 0xffu) ? 1u : 0u) << (4 + j);
      }
    } else {
      const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(m));
#pragma unroll
      for (int j = 0; j < 4; ++j) take |= (((w >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
    }
    return take;
  };

  // from the end of the image backwards: what the voting kernel read last may still be in L2
  long long step = n_steps - 1 - warp0;
  uint32_t take_next = load_take(step);
  for (; step >= 0; step -= n_warps) {
    const long long grp = step * 16 + (lane >> 1);
    const bool in_range = grp < n_groups;
    const size_t pix0 = (size_t)(in_range ? grp : 0) * VEC;
    const uint32_t take = take_next;
    take_next = load_take(step - n_warps);      // the next step's mask is on its way while this step runs
    const bool have = take != 0;
    const T* src = e_img + pix0 + (size_t)axis * D2 * plane;

    // the first plane loads and the bins go out together
    constexpr int LB = F < stream_level_batch(FT) ? F : stream_level_batch(FT);   // harmonics whose plane loads are in flight together (2 loads each)
    uint4 raw[2 * LB];
    // a lane looks up, and later finishes, its half of the group's pixels: the axis-0 lane the first half
    uint32_t cell[H2];
    if (have) {
#pragma unroll
      for (int q = 0; q < 2 * LB; ++q) raw[q] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)q * plane));
      if constexpr (H2 == 4) {
        const uint4 c4 = __ldg(reinterpret_cast<const uint4*>(pc_img + pix0 + axis * H2));
        cell[0] = c4.x; cell[1] = c4.y; cell[2] = c4.z; cell[3] = c4.w;
      } else {
        const uint2 c2 = __ldg(reinterpret_cast<const uint2*>(pc_img + pix0 + axis * H2));
        cell[0] = c2.x; cell[1] = c2.y;
      }
    }
    // bins -> peaks.  Pixels of one group nearly always share their peak (ku); at an instance border there is a second
    // one (kv); with more than two the group's pixels are left to the exact walk.
    int kpix[H2];
    uint32_t voted = 0;                         // bit jj: pixel jj of this lane's half participates and voted
    bool many = false;
    int ku = -1, kv = -1;
    auto add_peak = [&](int k) {
      if (k >= 0) {
        if (ku < 0) ku = k;
        else if (k != ku) {
          if (kv < 0) kv = k;
          else if (k != kv) many = true;
        }
      }
    };
    {
      const uint32_t take_h = (take >> (axis * H2)) & ((1u << H2) - 1u);
#pragma unroll
      for (int jj = 0; jj < H2; ++jj) {
        int k = -1;
        if (((take_h >> jj) & 1u) && cell[jj] != 0xffffffffu && (int)cell[jj] < cells) {
          voted |= 1u << jj;
          k = (jj > 0 && cell[jj] == cell[jj - 1] && ((voted >> (jj - 1)) & 1u)) ? kpix[jj - 1] : __ldg(cp_img + cell[jj]);
          if (k >= K) k = -1;
          add_peak(k);
        }
        kpix[jj] = k;
      }
      // the two halves' peaks become the group's, the first half's first, so that both lanes name them alike
      const uint32_t mine = ((uint32_t)ku & 0xfffu) | (((uint32_t)kv & 0xfffu) << 12) | (many ? 1u << 24 : 0u);
      const uint32_t other = __shfl_xor_sync(0xffffffffu, mine, 1);
      const uint32_t first = axis ? other : mine, second = axis ? mine : other;
      auto peak_of = [](uint32_t v) { return v == 0xfffu ? -1 : (int)v; };   // (K <= 1024: 0xfff is no peak index)
      ku = peak_of(first & 0xfffu);
      kv = peak_of((first >> 12) & 0xfffu);
      many = ((first | second) >> 24) & 1u;
      add_peak(peak_of(second & 0xfffu));
      add_peak(peak_of((second >> 12) & 0xfffu));
    }
    if (many) ku = kv = -1;
    // the first two entries of the peaks' lists
    uint2 e01u = make_uint2(0u, kNbrEnd), e01v = make_uint2(0u, kNbrEnd);
    if (ku >= 0) e01u = __ldg(reinterpret_cast<const uint2*>(nbr_img + (size_t)ku * kNbrCap));
    if (kv >= 0) e01v = __ldg(reinterpret_cast<const uint2*>(nbr_img + (size_t)kv * kNbrCap));
    const int kfu = (int)(e01u.x & 0xfffu), kfv = (int)(e01v.x & 0xfffu);

    // sums of squares, two pixels per register: against the reference row and the first candidate of ku, and of kv
    __half2 s[H2], sc[H2], sv[H2], scv[H2];
#pragma unroll
    for (int j = 0; j < H2; ++j) s[j] = sc[j] = sv[j] = scv[j] = __float2half2_rn(0.0f);
    // widening-free view of one 128-bit load as pixel pairs
    auto pairs_of = [](const uint4& r, __half2 (&v)[H2]) {
      if constexpr (sizeof(T) == 2) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < H2; ++j) v[j] = *reinterpret_cast<const __half2*>(&w[j]);
      } else {
        v[0] = __floats2half2_rn(__uint_as_float(r.x), __uint_as_float(r.y));
        v[1] = __floats2half2_rn(__uint_as_float(r.z), __uint_as_float(r.w));
      }
    };
    // all pixels of the group against the rows of one peak (row values splat over the pixel pairs); `first`: the first
    // batch of plane loads is already in `raw`
    auto accumulate = [&](int kref, int kcand, __half2 (&acc)[H2], __half2 (&accc)[H2], bool first) {
      const __half* rr = rows_ref + (size_t)kref * D + axis * D2;
      const __half* rc = rows_cand + (size_t)kcand * D + axis * D2;
#pragma unroll
      for (int l0 = 0; l0 < F; l0 += LB) {
        if (l0 > 0 || !first) {
#pragma unroll
          for (int q = 0; q < 2 * LB; ++q)
            raw[q] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)(2 * l0 + q) * plane));
        }
#pragma unroll
        for (int q = 0; q < 2 * LB; q += 2) {
          const int c = 2 * l0 + q;                // channels c and c + 1: one 32-bit row load serves both
          const __half2 r2 = *reinterpret_cast<const __half2*>(rr + c);
          const __half2 r_lo = __low2half2(r2), r_hi = __high2half2(r2);
          __half2 v0[H2], v1[H2];
          pairs_of(raw[q], v0);
          pairs_of(raw[q + 1], v1);
#pragma unroll
          for (int j = 0; j < H2; ++j) {
            const __half2 d = __hsub2(v0[j], r_lo);
            acc[j] = __hfma2(d, d, acc[j]);
          }
#pragma unroll
          for (int j = 0; j < H2; ++j) {
            const __half2 d = __hsub2(v1[j], r_hi);
            acc[j] = __hfma2(d, d, acc[j]);
          }
          if constexpr (!SAME) {
            const __half2 q2 = *reinterpret_cast<const __half2*>(rc + c);
            const __half2 q_lo = __low2half2(q2), q_hi = __high2half2(q2);
#pragma unroll
            for (int j = 0; j < H2; ++j) {
              const __half2 d = __hsub2(v0[j], q_lo);
              accc[j] = __hfma2(d, d, accc[j]);
            }
#pragma unroll
            for (int j = 0; j < H2; ++j) {
              const __half2 d = __hsub2(v1[j], q_hi);
              accc[j] = __hfma2(d, d, accc[j]);
            }
          }
        }
      }
    };
    if (ku >= 0) accumulate(ku, kfu, s, sc, true);
    // An instance border: a group with a second peak.  Nearly every step of a large image has one such group, so the
    // second pass over it is shared by the whole warp instead of being run by the group's two lanes while thirty wait:
    // lane (pixel pair, axis, part of the axis' planes) re-reads its 32-bit pieces (cache hits), the parts are summed
    // with shuffles and handed to the group's lanes in the layout of the first pass.
    {
      constexpr int NPQ = 16 / H2;               // parts that an axis' planes are split into
      constexpr int PL = D2 / NPQ;               // planes per lane
      static_assert(PL >= 1 && PL * NPQ == D2, "the planes divide among the lanes");
      uint32_t border = __ballot_sync(0xffffffffu, kv >= 0 && axis == 0);
      const int pp = lane & (H2 - 1), a2 = (lane / H2) & 1, pq = lane / (2 * H2);
#pragma unroll 1
      while (border) {
        const int src_lane = __ffs(border) - 1;
        border &= border - 1;
        const int kvb = __shfl_sync(0xffffffffu, kv, src_lane);
        const int kfb = __shfl_sync(0xffffffffu, kfv, src_lane);
        const uint32_t gb = __shfl_sync(0xffffffffu, (uint32_t)(pix0 / VEC), src_lane);   // group index (< 2^28)
        const int c0 = a2 * D2 + pq * PL;
        const T* pb = e_img + (size_t)gb * VEC + 2 * pp + (size_t)c0 * plane;
        const __half* rr = rows_ref + (size_t)kvb * D + c0;
        const __half* rc = rows_cand + (size_t)kfb * D + c0;
        __half2 v[PL];
#pragma unroll
        for (int i = 0; i < PL; ++i) {
          if constexpr (sizeof(T) == 2) {
            const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(pb + (size_t)i * plane));
            v[i] = *reinterpret_cast<const __half2*>(&w);
          } else {
            const float2 f = __ldg(reinterpret_cast<const float2*>(pb + (size_t)i * plane));
            v[i] = __floats2half2_rn(f.x, f.y);
          }
        }
        __half2 acc = __float2half2_rn(0.0f), accc = acc;
#pragma unroll
        for (int i = 0; i < PL; ++i) {
          const __half2 d = __hsub2(v[i], __half2half2(rr[i]));
          acc = __hfma2(d, d, acc);
          if constexpr (!SAME) {
            const __half2 dc = __hsub2(v[i], __half2half2(rc[i]));
            accc = __hfma2(dc, dc, accc);
          }
        }
#pragma unroll
        for (int off = 2 * H2; off < 32; off <<= 1) {
          acc = __hadd2(acc, shfl_xor_h2(acc, off));
          if constexpr (!SAME) accc = __hadd2(accc, shfl_xor_h2(accc, off));
        }
        // lane (pp, axis) of part 0 holds the sums of pixel pair pp on that axis
        const bool mine = (lane >> 1) == (src_lane >> 1);
#pragma unroll
        for (int j = 0; j < H2; ++j) {
          const __half2 t = shfl_h2(acc, axis * H2 + j);
          if (mine) sv[j] = t;
          if constexpr (!SAME) {
            const __half2 tc = shfl_h2(accc, axis * H2 + j);
            if (mine) scv[j] = tc;
          }
        }
      }
    }
    // per pixel, pick the sums of its own peak first (register pairs hold two pixels: blend the halves).  The shuffle
    // is executed by every lane: a group's two lanes share kv, the lanes of other groups do not.
    {
      uint32_t use_h = 0;
#pragma unroll
      for (int jj = 0; jj < H2; ++jj)
        if (kv >= 0 && kpix[jj] == kv) use_h |= 1u << jj;
      const uint32_t use_o = __shfl_xor_sync(0xffffffffu, use_h, 1);
      const uint32_t use_v = axis ? (use_o | (use_h << H2)) : (use_h | (use_o << H2));
      if (use_v) {
#pragma unroll
        for (int j = 0; j < H2; ++j) {
          const bool lo = (use_v >> (2 * j)) & 1u, hi = (use_v >> (2 * j + 1)) & 1u;
          s[j] = __halves2half2(lo ? __low2half(sv[j]) : __low2half(s[j]), hi ? __high2half(sv[j]) : __high2half(s[j]));
          if constexpr (!SAME)
            sc[j] = __halves2half2(lo ? __low2half(scv[j]) : __low2half(sc[j]), hi ? __high2half(scv[j]) : __high2half(sc[j]));
        }
      }
    }
    // swap with the partner lane: each lane keeps its own axis' sums of its half of the pixels and gets the partner's
    // (the distances below are symmetric in the two axes, so which one is x does not matter)
    constexpr int Q2 = H2 / 2;                  // half2 registers per half of the group (2 for binary16, 1 for binary32)
    float2 own[Q2], oth[Q2], cwn[Q2], cth[Q2];
#pragma unroll
    for (int i = 0; i < Q2; ++i) {
      const __half2 send = axis ? s[i] : s[Q2 + i];
      const __half2 keep = axis ? s[Q2 + i] : s[i];
      own[i] = __half22float2(keep);
      oth[i] = __half22float2(shfl_xor_h2(send, 1));
      if constexpr (!SAME) {
        const __half2 sendc = axis ? sc[i] : sc[Q2 + i];
        const __half2 keepc = axis ? sc[Q2 + i] : sc[i];
        cwn[i] = __half22float2(keepc);
        cth[i] = __half22float2(shfl_xor_h2(sendc, 1));
      } else {
        cwn[i] = own[i];
        cth[i] = oth[i];
      }
    }
    int my_label[H2];
    uint32_t n_likely_hard = 0;
#pragma unroll
    for (int jj = 0; jj < H2; ++jj) {
      const int j = axis * H2 + jj;              // the pixel's place in the group
      const float sa = (jj & 1) ? own[jj / 2].y : own[jj / 2].x, sb = (jj & 1) ? oth[jj / 2].y : oth[jj / 2].x;
      const float ca = (jj & 1) ? cwn[jj / 2].y : cwn[jj / 2].x, cb = (jj & 1) ? cth[jj / 2].y : cth[jj / 2].x;
      const int k0j = kpix[jj];
      int label = 0;
      bool slow = false;
      if ((voted >> jj) & 1u) {
        slow = true;
        bool likely_hard = k0j < 0;
        if (k0j >= 0 && !many) {
          const uint2 e01 = k0j == ku ? e01u : e01v;
          const int kfj = (int)(e01.x & 0xfffu);
          const float t = (fast_sqrt(sa) + fast_sqrt(sb)) * kHalfRel + kHalfAbs;
          const float dub = SAME ? t : (fast_sqrt(ca) + fast_sqrt(cb)) * kHalfRel + kHalfAbs;
          const float reach = (dub + t) * kNearSlack;
          // the list's first entry is the candidate bounded above (with refined candidates that must be k0 itself:
          // an identical row with a lower index may precede it); the second entry decides whether the walk is over
          const bool first_ok = !SAME || kfj == k0j;
          const bool closed = e01.y == kNbrEnd || (float)(e01.y >> 12) * (1.0f / 65536.0f) > reach;
          if (certify && first_ok && closed) {
            label = kfj + 1;
            slow = false;
            ++n_pairs;
          } else if (K > kNbrCap) {
            const uint32_t el = __ldg(nbr_img + (size_t)k0j * kNbrCap + kNbrCap - 1);
            // (a comparison that a non-finite bound fails counts as likely hard)
            likely_hard = el != kNbrEnd && !((float)(el >> 12) * (1.0f / 65536.0f) > reach);
          }
        }
        if (likely_hard) ++n_likely_hard;
      }
      my_label[jj] = label;
      // queue the pixel: one atomic per warp and round
      const uint32_t sm = __ballot_sync(0xffffffffu, slow);
      if (sm && certify && wq_n + (uint32_t)__popc(sm) <= (uint32_t)kWarpQueue) {
        if (slow) s_wq[wid][wq_n + (uint32_t)__popc(sm & ((1u << lane) - 1u))] = (uint32_t)(pix0 + j);
        wq_n += (uint32_t)__popc(sm);
      } else if (sm) {
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(&state[kNearQueue], (uint32_t)__popc(sm));
        base = __shfl_sync(0xffffffffu, base, 0);
        if (slow) {
          const uint32_t at = base + (uint32_t)__popc(sm & ((1u << lane) - 1u));
          if (at < (uint32_t)q_cap) q_img[at] = (uint32_t)(pix0 + j);
        }
        if (lane == 0 && base + (uint32_t)__popc(sm) > (uint32_t)q_cap) atomicExch(&state[kNearGiveUp], 1u);
      }
    }
    if (in_range) {
      int32_t* dst = lab_img + pix0 + (size_t)axis * H2;
      if constexpr (VEC == 8)
        *reinterpret_cast<int4*>(dst) = make_int4(my_label[0], my_label[1], my_label[2], my_label[3]);
      else
        *reinterpret_cast<int2*>(dst) = make_int2(my_label[0], my_label[1]);
    }
    // ---- hand the image on if too many pixels cannot be closed by the bounds (before the walks are paid for)
    const uint32_t nh = __reduce_add_sync(0xffffffffu, n_likely_hard);
    visited += 16u * VEC;
    visited_all += 16u * VEC;
    hard_acc += nh;
    uint32_t stop = 0;
    if (lane == 0 && (hard_acc || visited >= 4096u)) {
      // hard pixels are reported at once, the others now and then: the share is taken of what all warps have visited
      // by now, estimated from this warp's own progress (the warps walk the image in step)
      const uint32_t everybody = (uint32_t)min((unsigned long long)visited_all * (unsigned long long)n_warps, (unsigned long long)HW);
      stop = near_account(state, visited, hard_acc, min_proc, everybody);
      visited = hard_acc = 0;
    }
    if (__shfl_sync(0xffffffffu, stop, 0)) return;     // the filtered kernel redoes the whole image
  }
  if (lane == 0 && visited) near_account(state, visited, hard_acc, min_proc);

  // ---- this warp's own queue: exact walks, a lane per pixel
  uint32_t n_multi = 0;
  __syncwarp();
  if (wq_n) {
    const float* ref_img = ref2 + (size_t)b * K_max * D;
    const float* cand_img = cand2 + (size_t)b * K_max * D;
    for (uint32_t i0 = 0; i0 < wq_n; i0 += 32u) {
      const bool have = i0 + lane < wq_n;
      const size_t n = have ? s_wq[wid][i0 + lane] : 0;
      float d1 = __int_as_float(0x7f800000), d2 = d1;
      int k1 = -1;
      bool hard = false;
      uint32_t scored = 0;
      if (have) {
        const uint32_t cell = __ldg(pc_img + n);
        int k0 = (cell != 0xffffffffu && (int)cell < cells) ? __ldg(cp_img + cell) : -1;
        if (k0 >= K) k0 = -1;
        hard = k0 < 0;
        if (!hard) {
          const T* p = e_img + n;
          float2 e2[D / 2];
#pragma unroll
          for (int c = 0; c < D / 2; ++c) {
            e2[c].x = Elem<T>::load1(p + (size_t)c * plane);
            e2[c].y = Elem<T>::load1(p + (size_t)(D / 2 + c) * plane);
          }
          near_walk<D, false>(e2, k0, K, SAME, ref_img, cand_img, nbr_img, d1, d2, k1, hard, scored);
        }
      }
      const uint32_t hm = __ballot_sync(0xffffffffu, hard);
      if (hm) {
        uint32_t hbase = 0;
        if (lane == 0) hbase = atomicAdd(&state[kNearHardQueue], (uint32_t)__popc(hm));
        hbase = __shfl_sync(0xffffffffu, hbase, 0);
        const uint32_t at = hbase + (uint32_t)__popc(hm & ((1u << lane) - 1u));
        if (hard && at < (uint32_t)q_cap) hard_q[(size_t)b * q_cap + at] = (uint32_t)n;
        if (lane == 0 && hbase + (uint32_t)__popc(hm) > (uint32_t)q_cap) atomicExch(&state[kNearGiveUp], 1u);
      }
      if (have && !hard) {
        if (scored > 1) ++n_multi;
        n_pairs += scored;
        lab_img[n] = k1 >= 0 ? k1 + 1 : 0;        // (tau is infinite here: nothing is rejected)
      }
    }
  }
  near_flush_counters(state, 0u, n_pairs, n_multi, 0u);
}

// The walk of the pixels that the streaming kernel queued, one thread per pixel.
template <typename T, int FT>
__global__ void __launch_bounds__(kNearThreads, FT == 16 ? 2 : 3)
assign_near_walk_kernel(const T* __restrict__ emb, int HW, int K_max, const float* __restrict__ ref2,
                        const float* __restrict__ cand2, const uint32_t* __restrict__ nbr,
                        const int32_t* __restrict__ cell_peak, const uint32_t* __restrict__ pix_cell, int cells,
                        const int32_t* __restrict__ count_ptr, float tau, int32_t* __restrict__ labels,
                        uint32_t* __restrict__ near_state, const uint32_t* __restrict__ slow_q,
                        uint32_t* __restrict__ hard_q, int q_cap, int k_min) {
  grid_dependency_sync();
  constexpr int D = 4 * FT;
  const int b = blockIdx.y;
  const size_t plane = (size_t)HW;
  const int K = count_ptr[b];
  if (K < k_min || K > kNearMaxPeaks) return;
  uint32_t* state = near_state + b * kNearStride;
  if (state[kNearGiveUp]) return;                // the filtered kernel redoes the whole image
  const int n_q = (int)min(state[kNearQueue], (uint32_t)q_cap);
  const bool same_rows = ref2 == cand2;
  const float* ref_img = ref2 + (size_t)b * K_max * D;
  const float* cand_img = cand2 + (size_t)b * K_max * D;
  const uint32_t* nbr_img = nbr + (size_t)b * K_max * kNbrCap;
  const int32_t* cp_img = cell_peak + (size_t)b * cells;
  const float inf = __int_as_float(0x7f800000);
  uint32_t n_rejected = 0, n_pairs = 0, n_multi = 0, n_full = 0;
  const int lane = threadIdx.x & 31;
  for (int base = blockIdx.x * kNearThreads; base < n_q; base += gridDim.x * kNearThreads) {   // uniform per CTA
    const int i = base + threadIdx.x;
    const bool have = i < n_q;
    const size_t n = have ? slow_q[(size_t)b * q_cap + i] : 0;
    const T* p = emb + (size_t)b * D * plane + n;
    float d1 = inf, d2 = inf;
    int k1 = -1;
    bool hard = false;
    uint32_t scored = 0;
    if (have) {
      const uint32_t cell = __ldg(pix_cell + (size_t)b * plane + n);
      int k0 = (cell != 0xffffffffu && (int)cell < cells) ? __ldg(cp_img + cell) : -1;
      if (k0 >= K) k0 = -1;
      hard = k0 < 0;
      if (!hard) {
        float2 e2[D / 2];
#pragma unroll
        for (int c = 0; c < D / 2; ++c) {
          e2[c].x = Elem<T>::load1(p + (size_t)c * plane);
          e2[c].y = Elem<T>::load1(p + (size_t)(D / 2 + c) * plane);
        }
        near_walk<D, false>(e2, k0, K, same_rows, ref_img, cand_img, nbr_img, d1, d2, k1, hard, scored);
      }
    }
    // hard pixels (no peak for the bin, list run out, long walk): every peak has to be scored, which a warp does
    // together.  They come in runs (an instance without a peak of its own), so they go to a second queue from which
    // assign_near_hard_kernel deals them out one per warp, instead of being done here, a run at a time by one warp.
    const uint32_t hm = __ballot_sync(0xffffffffu, hard);
    if (hm) {
      uint32_t hbase = 0;
      if (lane == 0) hbase = atomicAdd(&state[kNearHardQueue], (uint32_t)__popc(hm));
      hbase = __shfl_sync(0xffffffffu, hbase, 0);
      // (the streaming kernel's warps append here too: the bound is checked, and an overflow hands the image on)
      const uint32_t at = hbase + (uint32_t)__popc(hm & ((1u << lane) - 1u));
      if (hard && at < (uint32_t)q_cap) hard_q[(size_t)b * q_cap + at] = (uint32_t)n;
      if (lane == 0 && hbase + (uint32_t)__popc(hm) > (uint32_t)q_cap) atomicExch(&state[kNearGiveUp], 1u);
    }
    if (have && !hard) {
      if (scored > 1) ++n_multi;
      n_pairs += scored;
      int label = 0;
      if (k1 >= 0) {
        if (d1 < tau) label = k1 + 1;
        else ++n_rejected;
      }
      labels[(size_t)b * plane + n] = label;
    }
  }
  near_flush_counters(state, n_rejected, n_pairs, n_multi, n_full);
}

// The pixels that the walk left over are scored against every peak: a whole CTA per pixel while there are fewer pixels
// than CTAs, else eight lanes per pixel with the rows staged in shared memory.
template <typename T, int FT>
__global__ void __launch_bounds__(kNearThreads, FT == 16 ? 1 : 4)   // (a CTA is a chain of latencies: many resident ones)
assign_near_hard_kernel(const T* __restrict__ emb, int HW, int K_max, const float* __restrict__ cand2,
                        const int32_t* __restrict__ count_ptr, float tau, int32_t* __restrict__ labels,
                        uint32_t* __restrict__ near_state, const uint32_t* __restrict__ hard_q, int q_cap, int k_min) {
  grid_dependency_sync();
  constexpr int D = 4 * FT;
  const int b = blockIdx.y;
  const size_t plane = (size_t)HW;
  const int K = count_ptr[b];
  if (K < k_min || K > kNearMaxPeaks) return;
  uint32_t* state = near_state + b * kNearStride;
  if (state[kNearGiveUp]) return;                // the filtered kernel redoes the whole image
  const int n_h = (int)min(state[kNearHardQueue], (uint32_t)q_cap);
  const float* cand_img = cand2 + (size_t)b * K_max * D;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  constexpr int kWarps = kNearThreads / 32;
  uint32_t n_rejected = 0, n_full = 0;
  auto finish = [&](size_t n, float d1, int k1) {
    ++n_full;
    int label = 0;
    if (k1 >= 0) {
      if (d1 < tau) label = k1 + 1;
      else ++n_rejected;
    }
    labels[(size_t)b * plane + n] = label;
  };
  if (n_h <= (int)gridDim.x) {
    // Few pixels (the usual case: a handful per image): a pixel's scan is a chain of K / 32 dependent row fetches for
    // one warp, so a whole CTA shares it, thread t scoring the peaks t, t + 256, ...; the warps' results are merged
    // with the same rule as the lanes' (smaller distance, then lower k).
    __shared__ float s_d1[kWarps], s_d2[kWarps];
    __shared__ int s_k1[kWarps];
    for (int i = blockIdx.x; i < n_h; i += gridDim.x) {       // (at most one round)
      const size_t n = hard_q[(size_t)b * q_cap + i];
      float d1, d2;
      int k1;
      near_full_scan_warp<T, D, false>(emb + (size_t)b * D * plane + n, plane, K, cand_img, d1, d2, k1, (int)threadIdx.x,
                                       kNearThreads);
      if (lane == 0) {
        s_d1[wid] = d1;
        s_d2[wid] = d2;
        s_k1[wid] = k1 < 0 ? 0x7fffffff : k1;
      }
      __syncthreads();
      if (wid == 0) {
        static_assert(kWarps <= 32, "one lane per warp result");
        const float inf = __int_as_float(0x7f800000);
        d1 = lane < kWarps ? s_d1[lane] : inf;
        d2 = lane < kWarps ? s_d2[lane] : inf;
        k1 = lane < kWarps ? s_k1[lane] : 0x7fffffff;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          const float od1 = __shfl_xor_sync(0xffffffffu, d1, off), od2 = __shfl_xor_sync(0xffffffffu, d2, off);
          const int ok1 = __shfl_xor_sync(0xffffffffu, k1, off);
          const bool other_wins = od1 < d1 || (od1 == d1 && ok1 < k1);
          const float loser = other_wins ? d1 : od1;
          if (other_wins) { d1 = od1; k1 = ok1; }
          d2 = fminf(fminf(d2, od2), loser);
        }
        if (lane == 0) finish(n, d1, k1 == 0x7fffffff ? -1 : k1);
      }
      __syncthreads();
    }
  } else {
    // Many pixels (an instance without a peak of its own sends all of its pixels here): the all-pairs scheme with
    // eight lanes per pixel.  The candidate rows pass through shared memory in chunks of 32; lane s of a pixel scores
    // the rows s, s + 8, s + 16, s + 24 of a chunk against the pixel's values in its registers (a row is padded to
    // D + 4 floats, so the eight rows that a warp reads at a time sit in different banks), and the eight results are
    // merged like the lanes' of the warp-wide scan: smaller distance first, lower k on equal distances -- what the
    // serial scan in ascending k with a strict comparison gives.  (One thread per pixel scoring every peak left most
    // of the GPU idle: a few thousand threads, each a chain of a hundred dependent scores.)
    constexpr int kChunk = 32, kSlices = 8, kRow = D + 4;
    constexpr int kPixPerCta = kNearThreads / kSlices;
    __shared__ __align__(16) float s_rows[kChunk * kRow];
    const float inf = __int_as_float(0x7f800000);
    const int slice = lane & (kSlices - 1);
    for (int base = blockIdx.x * kPixPerCta; base < n_h; base += gridDim.x * kPixPerCta) {   // uniform per CTA
      const int i = base + (int)(threadIdx.x / kSlices);
      const bool have = i < n_h;
      const size_t n = have ? hard_q[(size_t)b * q_cap + i] : 0;
      float2 e2[D / 2];
      if (have) {
        const T* p = emb + (size_t)b * D * plane + n;
#pragma unroll
        for (int c = 0; c < D / 2; ++c) {
          e2[c].x = Elem<T>::load1(p + (size_t)c * plane);
          e2[c].y = Elem<T>::load1(p + (size_t)(D / 2 + c) * plane);
        }
      }
      float d1 = inf, bound2 = inf;
      int k1 = 0x7fffffff;
      for (int k0 = 0; k0 < K; k0 += kChunk) {
        const int kn = min(kChunk, K - k0);
        __syncthreads();
        // (rows past the last peak are copies of the chunk's first row: scored, never taken)
        for (int j = threadIdx.x; j < kChunk * (D / 4); j += kNearThreads) {
          const int r = j / (D / 4), q = j % (D / 4);
          reinterpret_cast<float4*>(s_rows + r * kRow)[q] =
              __ldg(reinterpret_cast<const float4*>(cand_img + (size_t)(k0 + (r < kn ? r : 0)) * D) + q);
        }
        __syncthreads();
        if (have) {
          float d[4];
          score_direct4<D, kSlices * kRow / 2>(e2, reinterpret_cast<const float2*>(s_rows + slice * kRow), bound2, d);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (slice + kSlices * j < kn && d[j] < d1) { d1 = d[j]; k1 = k0 + slice + kSlices * j; }
          bound2 = d1 * d1 * (1.0f + 1e-6f);
        }
      }
      // (every lane of the warp takes part: lanes without a pixel carry +inf)
#pragma unroll
      for (int off = 1; off < kSlices; off <<= 1) {
        const float od1 = __shfl_xor_sync(0xffffffffu, d1, off);
        const int ok1 = __shfl_xor_sync(0xffffffffu, k1, off);
        if (od1 < d1 || (od1 == d1 && ok1 < k1)) { d1 = od1; k1 = ok1; }
      }
      if (have && slice == 0) finish(n, d1, k1 == 0x7fffffff ? -1 : k1);
    }
  }
  near_flush_counters(state, n_rejected, n_full * (uint32_t)K, 0u, n_full);
}

}  // namespace cpe
