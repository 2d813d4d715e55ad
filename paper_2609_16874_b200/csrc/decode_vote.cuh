// Stage 1+2: per-pixel centroid estimate and hard-vote accumulation (hard-vote form of Eq. 6 on the
// Eq. 9 bins).
//
// A CTA owns a span of consecutive pixels.  It first compacts the span's participating pixels into a
// shared-memory list (mask bytes read with 64-bit loads), then walks that list with all lanes busy:
// lane i of a warp decodes the i-th participating pixel, so background pixels cost neither arithmetic
// nor embedding traffic (32-byte sectors that hold no participating pixel are never requested), and
// consecutive lanes read consecutive addresses of each channel plane.  Votes are aggregated per warp
// (one bin per warp is the common case), cached per CTA in a small shared-memory (bin -> count) table
// and flushed with one global atomic per distinct bin per CTA.
#pragma once

#include "cpe_common.cuh"
#include "peaks.cuh"

namespace cpe {

constexpr int kVoteThreads = 256;
constexpr int kVoteSpan = 2048;       // pixels per CTA (8 per thread in the mask pass)
constexpr int kVotePix = 2;           // pixels decoded per thread per sweep of the list (independent chains)
constexpr int kHashSlots = 512;       // per-CTA (bin -> count) cache in shared memory
constexpr int kHashProbes = 16;
constexpr uint32_t kHashEmpty = 0xffffffffu;

// Adds n votes for `cell` to the CTA's cache; falls back to the global map if the cache is crowded.
__device__ __forceinline__ void vote_cache_add(uint32_t* keys, uint32_t* cnts, uint32_t cell, uint32_t n,
                                               uint32_t* votes_img) {
  uint32_t h = (cell * 2654435761u) >> 23;  // 9 bits
#pragma unroll 1
  for (int i = 0; i < kHashProbes; ++i) {
    const uint32_t old = atomicCAS(&keys[h], kHashEmpty, cell);
    if (old == kHashEmpty || old == cell) {
      atomicAdd(&cnts[h], n);
      return;
    }
    h = (h + 1) & (kHashSlots - 1);
  }
  atomicAdd(&votes_img[cell], n);
}

// Sub-cell refinement: next to the count, a bin also gets the sum of the estimates that fell into it, as integers so
// that the result does not depend on the order of addition.  An estimate p in [-1, 1) is taken as rint(p * 2^24)
// (exact for |p| >= 1/4).  Lanes of the warp that name the same bin are summed first (at most 32 x 2^24 fits in 32
// bits), then one lane per distinct bin adds the pair to the bin's 64-bit sums in global memory (fire-and-forget
// reductions).  Called by all 32 lanes; cell < 0 = this lane has no vote.
constexpr float kRefineScale = 16777216.0f;  // 2^24

// What a voting kernel records besides the vote map (template parameter MODE, a bit set):
constexpr int kVoteSums = 1;    // the per-bin fixed-point sums of the estimates
constexpr int kVotePeaks = 4;   // the last CTA of an image to finish also searches its (small) vote map for the peaks:
                                // peaks_image with one CTA per image, instead of a launch of peaks_kernel
constexpr int kVoteCells = 2;   // every participating pixel's bin (uint32 [B][H*W]; 0xffffffff: it did not vote), which the
                                // pruned assignment looks its candidate list up with

__device__ __forceinline__ void vote_sums_add(long long* __restrict__ sums_img, int cell, float px, float py,
                                              bool one_bin, uint32_t voters) {
  const int lane = threadIdx.x & 31;
  const int fx = cell >= 0 ? __float2int_rn(__fmul_rn(px, kRefineScale)) : 0;
  const int fy = cell >= 0 ? __float2int_rn(__fmul_rn(py, kRefineScale)) : 0;
  if (one_bin) {
    const int sx = __reduce_add_sync(0xffffffffu, fx), sy = __reduce_add_sync(0xffffffffu, fy);
    if (lane == __ffs(voters) - 1) {
      atomicAdd(reinterpret_cast<unsigned long long*>(sums_img + 2 * (size_t)cell), (unsigned long long)(long long)sx);
      atomicAdd(reinterpret_cast<unsigned long long*>(sums_img + 2 * (size_t)cell + 1),
                (unsigned long long)(long long)sy);
    }
  } else {
    const uint32_t same = __match_any_sync(0xffffffffu, cell);   // the lanes without a vote form a group of their own
    const int sx = __reduce_add_sync(same, fx), sy = __reduce_add_sync(same, fy);
    if (cell >= 0 && lane == __ffs(same) - 1) {
      atomicAdd(reinterpret_cast<unsigned long long*>(sums_img + 2 * (size_t)cell), (unsigned long long)(long long)sx);
      atomicAdd(reinterpret_cast<unsigned long long*>(sums_img + 2 * (size_t)cell + 1),
                (unsigned long long)(long long)sy);
    }
  }
}

// With kVotePeaks: called by every thread of a voting CTA after its votes and counts have gone to global memory.  The
// last CTA of image b to get here (ticket counter, no waiting) runs the peak search on the finished map.
template <int THREADS>
__device__ __forceinline__ void vote_then_peaks(const PeakArgs& pa, int b, uint32_t* acc, uint32_t* s_map) {
  __shared__ int s_vote_last;
  __threadfence();              // this CTA's votes are visible device-wide before its ticket is taken
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t ticket = atomicAdd(&acc[b * kAccStride + kAccTicket], 1u);
    s_vote_last = ticket == gridDim.x - 1;
  }
  __syncthreads();
  if (!s_vote_last) return;
  __threadfence();              // and the other CTAs' votes are visible to this one
  peaks_image<THREADS>(pa, b, 0, 1, s_map);      // (leaves the ticket zero for the next decode)
}

// Compacts the participating pixels of the CTA's span into s_list (offsets within the span, ascending).
// Returns the number of entries.  `fg` may be NULL (all pixels participate).  Uses s_scan[9] as scratch.
__device__ __forceinline__ int compact_span(const uint8_t* __restrict__ fg_img, long long span0, int HW, bool vec_mask,
                                            uint16_t* s_list, int* s_scan) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const long long p0 = span0 + (long long)tid * 8;
  uint32_t bits = 0;  // bit j: pixel p0 + j participates
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
  const int mine = __popc(bits);
  int incl = mine;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) s_scan[wid] = incl;
  __syncthreads();
  if (tid == 0) {
    int run = 0;
#pragma unroll
    for (int w = 0; w < kVoteThreads / 32; ++w) {
      const int t = s_scan[w];
      s_scan[w] = run;
      run += t;
    }
    s_scan[kVoteThreads / 32] = run;
  }
  __syncthreads();
  int slot = s_scan[wid] + incl - mine;
  while (bits) {
    const int j = __ffs(bits) - 1;
    bits &= bits - 1;
    s_list[slot++] = (uint16_t)(tid * 8 + j);
  }
  __syncthreads();
  return s_scan[kVoteThreads / 32];
}

// Scalar-load variant: any F, any alignment, any H*W.  FT > 0 fixes F at compile time.
template <typename T, int FT, int MODE>
__global__ void __launch_bounds__(kVoteThreads)
decode_vote_scalar_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F_rt, int levels,
                   int bins_w, int bins_h, int vec_mask, uint32_t* __restrict__ votes,
                   uint32_t* __restrict__ acc, long long* __restrict__ sums, uint32_t* __restrict__ pix_cell,
                   const PeakArgs pa) {
  constexpr bool REFINE = (MODE & kVoteSums) != 0;
  constexpr bool CELLS = (MODE & kVoteCells) != 0;
  extern __shared__ uint32_t s_vote_map[];       // with kVotePeaks: room for the vote map
  grid_dependency_sync();
  const int F = FT > 0 ? FT : F_rt;
  const int Fu = (levels > 0 && levels < F) ? levels : F;
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const size_t plane = (size_t)HW;
  const T* e = emb + (size_t)b * 4 * F * plane;
  const uint8_t* fg_img = fg ? fg + (size_t)b * plane : nullptr;
  uint32_t* votes_img = votes + (size_t)b * bins_w * bins_h;
  long long* sums_img = REFINE ? sums + (size_t)b * bins_w * bins_h * 2 : nullptr;
  const long long span0 = (long long)blockIdx.x * kVoteSpan;

  __shared__ uint32_t s_keys[kHashSlots];
  __shared__ uint32_t s_cnts[kHashSlots];
  __shared__ uint16_t s_list[kVoteSpan];
  __shared__ int s_scan[kVoteThreads / 32 + 1];
  __shared__ uint32_t s_nonfinite, s_voting;
  for (int i = tid; i < kHashSlots; i += kVoteThreads) {
    s_keys[i] = kHashEmpty;
    s_cnts[i] = 0;
  }
  if (tid == 0) s_nonfinite = s_voting = 0;

  const int n_active = compact_span(fg_img, span0, HW, vec_mask != 0, s_list, s_scan);  // has __syncthreads

  const float half_w = (float)(bins_w + 1) * 0.5f, half_h = (float)(bins_h + 1) * 0.5f;
  uint32_t nonfinite = 0, voted = 0;

  // all threads of a warp run the same number of sweeps (warp collectives inside)
  for (int base = 0; base < n_active; base += kVoteThreads * kVotePix) {
    bool have[kVotePix];
    const T* src[kVotePix];
#pragma unroll
    for (int q = 0; q < kVotePix; ++q) {
      const int i = base + q * kVoteThreads + tid;
      have[q] = i < n_active;
      const int off = have[q] ? (int)s_list[i] : 0;
      src[q] = e + span0 + off;
    }
    float p[kVotePix][2];
    float fin[kVotePix];
#pragma unroll
    for (int q = 0; q < kVotePix; ++q) fin[q] = 0.0f;
#pragma unroll
    for (int axis = 0; axis < 2; ++axis) {
#pragma unroll
      for (int l = 0; l < (FT > 0 ? FT : 16); ++l) {
        if (FT == 0 && l >= F) break;
        const size_t ch = ((size_t)axis * 2 * F + 2 * l) * plane;
        float s[kVotePix], c[kVotePix];
#pragma unroll
        for (int q = 0; q < kVotePix; ++q) {
          s[q] = have[q] ? Elem<T>::load1(src[q] + ch) : 0.0f;
          c[q] = have[q] ? Elem<T>::load1(src[q] + ch + plane) : 1.0f;
        }
#pragma unroll
        for (int q = 0; q < kVotePix; ++q) {
          fin[q] = fold_finite(fin[q], s[q], c[q]);
          if (l < Fu) {
            const float u = atan2_ht(s[q], c[q]);
            p[q][axis] = (l == 0) ? u : refine_scaled(p[q][axis], u);
          }
        }
      }
    }
    const float unscale = pow2f(1 - Fu);
#pragma unroll
    for (int q = 0; q < kVotePix; ++q) {
      int cell = -1;
      float ux = 0.0f, uy = 0.0f;
      if (have[q]) {
        if (fin[q] == fin[q]) {
          ux = wrap_unit(__fmul_rn(p[q][0], unscale));
          uy = wrap_unit(__fmul_rn(p[q][1], unscale));
          const int cx = cell_of(ux, half_w, bins_w);
          const int cy = cell_of(uy, half_h, bins_h);
          cell = cy * bins_w + cx;
          ++voted;
        } else {
          ++nonfinite;
        }
        if constexpr (CELLS)
          pix_cell[(size_t)b * plane + (size_t)(src[q] - e)] = (uint32_t)cell;   // 0xffffffff: no vote
      }
      // warp-aggregated insertion; fast path: every voting lane of the warp names the same bin
      const uint32_t voters = __ballot_sync(0xffffffffu, cell >= 0);
      if (voters) {
        const int leader = __ffs(voters) - 1;
        const int ref = __shfl_sync(0xffffffffu, cell, leader);
        const bool one_bin = __all_sync(0xffffffffu, cell < 0 || cell == ref);
        if constexpr (REFINE) vote_sums_add(sums_img, cell, ux, uy, one_bin, voters);
        if (one_bin) {
          if (lane == leader) vote_cache_add(s_keys, s_cnts, (uint32_t)ref, (uint32_t)__popc(voters), votes_img);
        } else {
          const uint32_t same = __match_any_sync(0xffffffffu, cell);
          if (cell >= 0 && lane == __ffs(same) - 1)
            vote_cache_add(s_keys, s_cnts, (uint32_t)cell, (uint32_t)__popc(same), votes_img);
        }
      }
    }
  }
  const uint32_t wv = __reduce_add_sync(0xffffffffu, voted);
  const uint32_t wb = __reduce_add_sync(0xffffffffu, nonfinite);
  if (lane == 0) {
    if (wv) atomicAdd(&s_voting, wv);
    if (wb) atomicAdd(&s_nonfinite, wb);
  }
  __syncthreads();

  // Flush: one global atomic per distinct bin per CTA.
  for (int i = tid; i < kHashSlots; i += kVoteThreads) {
    const uint32_t k = s_keys[i];
    if (k != kHashEmpty) atomicAdd(&votes_img[k], s_cnts[i]);
  }
  if (tid == 0 && s_voting) atomicAdd(&acc[b * kAccStride + kAccVoting], s_voting);
  if (tid == 0 && s_nonfinite) atomicAdd(&acc[b * kAccStride + kAccNonfinite], s_nonfinite);
  if constexpr ((MODE & kVotePeaks) != 0) vote_then_peaks<kVoteThreads>(pa, b, acc, s_vote_map);
}

// ------------------------------------------------------------------------------------------------
// Vector-load variant (the fast path): needs 16-byte aligned planes (emb 16-byte aligned, H*W a
// multiple of the vector width) and F fixed at compile time.
//
// The unit of work is (group, axis): VEC consecutive pixels (one 128-bit load per channel plane) and
// one of the two coordinate axes.  A CTA compacts the groups of its span that hold at least one
// participating pixel, then each thread takes one (group, axis) item: it issues all 2F plane loads of
// its axis at once (the only long-latency step), runs the coarse-to-fine estimate for its VEC pixels,
// swaps results with its partner lane (same group, other axis) and turns half of the pixels into bins.
constexpr int kVecGroupsMax = 256;   // groups per CTA: 256, 128 or 64 (template parameter GROUPS; the launcher takes the
                                     // largest that still gives a full wave of CTAs -- small images are latency-bound
                                     // and want many short CTAs, large ones want fewer fixed costs)
// harmonics whose plane loads are in flight together (2 loads each); four CTAs per SM at 64 registers
template <typename T> __host__ __device__ constexpr int vec_level_batch() { return 4; }

template <typename T, int FT, int MODE, int GROUPS>
__global__ void __launch_bounds__(kVoteThreads, 4)
decode_vote_vec_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int levels, int bins_w,
                       int bins_h, uint32_t* __restrict__ votes, uint32_t* __restrict__ acc,
                       long long* __restrict__ sums, uint32_t* __restrict__ pix_cell, const PeakArgs pa) {
  constexpr bool REFINE = (MODE & kVoteSums) != 0;
  constexpr bool CELLS = (MODE & kVoteCells) != 0;
  extern __shared__ uint32_t s_vote_map[];       // with kVotePeaks: room for the vote map
  grid_dependency_sync();
  constexpr int VEC = Elem<T>::kVec;
  constexpr int F = FT;
  const int Fu = (levels > 0 && levels < F) ? levels : F;
  const int b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const size_t plane = (size_t)HW;
  const T* e = emb + (size_t)b * 4 * F * plane;
  uint32_t* votes_img = votes + (size_t)b * bins_w * bins_h;
  long long* sums_img = REFINE ? sums + (size_t)b * bins_w * bins_h * 2 : nullptr;
  static_assert(GROUPS <= kVecGroupsMax && GROUPS <= kVoteThreads, "one thread looks at one group");
  const long long span0 = (long long)blockIdx.x * GROUPS * VEC;

  __shared__ uint32_t s_keys[kHashSlots];
  __shared__ uint32_t s_cnts[kHashSlots];
  __shared__ uint16_t s_grp[GROUPS];   // low 8 bits: group index in the span; high 8 bits: participation bits
  __shared__ int s_scan[kVoteThreads / 32 + 1];
  __shared__ uint32_t s_nonfinite, s_voting;
  for (int i = tid; i < kHashSlots; i += kVoteThreads) {
    s_keys[i] = kHashEmpty;
    s_cnts[i] = 0;
  }
  if (tid == 0) s_nonfinite = s_voting = 0;

  // ---- which groups of the span hold a participating pixel (thread t looks at group t)
  uint32_t bits = 0;
  {
    const long long p0 = span0 + (long long)tid * VEC;
    if (tid < GROUPS && p0 < HW) {  // H*W is a multiple of VEC: a group is never cut by the end of the image
      if (!fg) {
        bits = (1u << VEC) - 1u;
      } else {
        const uint8_t* m = fg + (size_t)b * plane + p0;
        if constexpr (VEC == 8) {
          const uint2 w = __ldg(reinterpret_cast<const uint2*>(m));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            bits |= (((w.x >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
            bits |= (((w.y >> (8 * j)) & 0xffu) ? 1u : 0u) << (4 + j);
          }
        } else {
          const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(m));
#pragma unroll
          for (int j = 0; j < 4; ++j) bits |= (((w >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
        }
      }
    }
  }
  const uint32_t act = __ballot_sync(0xffffffffu, bits != 0);
  if (lane == 0) s_scan[wid] = __popc(act);
  __syncthreads();
  // every thread adds up the warps' counts itself (eight shared-memory reads): no serial step, one barrier fewer
  int before = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kVoteThreads / 32; ++w) {
    const int t = s_scan[w];
    if (w < wid) before += t;
    total += t;
  }
  if (bits) s_grp[before + __popc(act & ((1u << lane) - 1u))] = (uint16_t)(tid | (bits << 8));
  __syncthreads();
  const int n_items = 2 * total;

  const float half_w = (float)(bins_w + 1) * 0.5f, half_h = (float)(bins_h + 1) * 0.5f;
  uint32_t nonfinite = 0, voted = 0;

  for (int base = 0; base < n_items; base += kVoteThreads) {   // warp-uniform trip count
    const int i = base + tid;
    const bool have = i < n_items;
    const uint32_t ent = have ? (uint32_t)s_grp[i >> 1] : 0u;
    const int axis = i & 1;                    // lanes 2j and 2j+1 share a group
    const uint32_t take = ent >> 8;
    const T* src = e + span0 + (size_t)(ent & 0xffu) * VEC + (size_t)axis * 2 * F * plane;

    float p[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) p[j] = 0.0f;   // the first harmonic's step from 0 returns its own estimate u
    uint32_t okbits = (1u << VEC) - 1u;
    if (have) {
      // validity accumulators: binary32 inputs fold |s| + |c| per pixel (fold_finite); binary16 inputs are finite iff
      // every element is (their sums cannot overflow binary32), so a running packed maximum of the absolute values in
      // the form that propagates NaNs is enough: one instruction per two pixels and harmonic
      float fin[VEC];
      __half2 rmax[VEC / 2];
#pragma unroll
      for (int j = 0; j < VEC; ++j) fin[j] = 0.0f;
#pragma unroll
      for (int j = 0; j < VEC / 2; ++j) rmax[j] = __float2half2_rn(0.0f);
      // The plane loads of a batch of harmonics are in flight together, kept raw in registers.  The loop over the
      // batches is not unrolled: the body for one batch (VEC pixels x LB harmonics) then stays in the instruction
      // cache, which the fully unrolled chain of all F harmonics overflowed.
      constexpr int LB = F < vec_level_batch<T>() ? F : vec_level_batch<T>();
      const T* ptr = src;
#pragma unroll 1
      for (int l0 = 0; l0 < F; l0 += LB, ptr += (size_t)(2 * LB) * plane) {
        uint4 raw[2 * LB];
#pragma unroll
        for (int i = 0; i < 2 * LB; ++i) raw[i] = __ldg(reinterpret_cast<const uint4*>(ptr + (size_t)i * plane));
#pragma unroll
        for (int ll = 0; ll < LB; ++ll) {
          if constexpr (sizeof(T) == 2) {
            // two pixels at a time, from the packed pairs as they were loaded (atan2_ht_pair_hw)
            const uint32_t ws[4] = {raw[2 * ll].x, raw[2 * ll].y, raw[2 * ll].z, raw[2 * ll].w};
            const uint32_t wc[4] = {raw[2 * ll + 1].x, raw[2 * ll + 1].y, raw[2 * ll + 1].z, raw[2 * ll + 1].w};
#pragma unroll
            for (int j = 0; j < VEC / 2; ++j) {
              const __half2 ys = *reinterpret_cast<const __half2*>(&ws[j]), xs = *reinterpret_cast<const __half2*>(&wc[j]);
              const __half2 ay = __habs2(ys), ax = __habs2(xs);
              const __half2 mxn = __hmax2_nan(ax, ay);
              rmax[j] = __hmax2_nan(rmax[j], mxn);
              if (l0 + ll < Fu) {
                const float2 u = atan2_ht_pair_hw(ys, xs, ay, ax, mxn);
                const float2 v = refine_scaled_pair(make_float2(p[2 * j], p[2 * j + 1]), u);
                p[2 * j] = v.x;
                p[2 * j + 1] = v.y;
              }
            }
          } else {
            float s[VEC], c[VEC];
            unpack_vec<T>(raw[2 * ll], s);
            unpack_vec<T>(raw[2 * ll + 1], c);
#pragma unroll
            for (int j = 0; j < VEC; ++j) fin[j] = fold_finite(fin[j], s[j], c[j]);
            if (l0 + ll < Fu) {
              // two pixels at a time: the polynomial and the coarse-to-fine step as packed instructions
#pragma unroll
              for (int j = 0; j < VEC; j += 2) {
                const float2 u = atan2_ht_pair(s[j], c[j], s[j + 1], c[j + 1]);
                const float2 v = refine_scaled_pair(make_float2(p[j], p[j + 1]), u);
                p[j] = v.x;
                p[j + 1] = v.y;
              }
            }
          }
        }
      }
      const float unscale = pow2f(1 - Fu);
#pragma unroll
      for (int j = 0; j < VEC; ++j) {
        p[j] = __fmul_rn(p[j], unscale);
        bool bad = fin[j] != fin[j];
        if constexpr (sizeof(T) == 2)   // the running maximum is infinite or a NaN: exponent field all ones
          bad = ((*reinterpret_cast<const uint32_t*>(&rmax[j / 2]) >> (16 * (j & 1))) & 0x7c00u) == 0x7c00u;
        if (bad) okbits &= ~(1u << j);
      }
    }
    // swap with the partner lane: afterwards every lane knows both coordinates of its half of the pixels
    const uint32_t ok_other = __shfl_xor_sync(0xffffffffu, okbits, 1);
    const uint32_t ok_both = okbits & ok_other;
    float other[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) other[j] = __shfl_xor_sync(0xffffffffu, p[j], 1);
    uint32_t my_cells[VEC / 2];
#pragma unroll
    for (int jj = 0; jj < VEC / 2; ++jj) {
      const int j = axis * (VEC / 2) + jj;       // axis-0 lane finishes the first half, axis-1 lane the second
      float px = axis == 0 ? p[jj] : other[VEC / 2 + jj];
      float py = axis == 0 ? other[jj] : p[VEC / 2 + jj];
      int cell = -1;
      if (have && ((take >> j) & 1u)) {
        if ((ok_both >> j) & 1u) {
          px = wrap_unit(px);
          py = wrap_unit(py);
          const int cx = cell_of(px, half_w, bins_w);
          const int cy = cell_of(py, half_h, bins_h);
          cell = cy * bins_w + cx;
          ++voted;
        } else {
          ++nonfinite;
        }
      }
      my_cells[jj] = (uint32_t)cell;
      const uint32_t voters = __ballot_sync(0xffffffffu, cell >= 0);
      if (voters) {
        const int leader = __ffs(voters) - 1;
        const int ref = __shfl_sync(0xffffffffu, cell, leader);
        const bool one_bin = __all_sync(0xffffffffu, cell < 0 || cell == ref);
        if constexpr (REFINE) vote_sums_add(sums_img, cell, px, py, one_bin, voters);
        if (one_bin) {
          if (lane == leader) vote_cache_add(s_keys, s_cnts, (uint32_t)ref, (uint32_t)__popc(voters), votes_img);
        } else {
          const uint32_t same = __match_any_sync(0xffffffffu, cell);
          if (cell >= 0 && lane == __ffs(same) - 1)
            vote_cache_add(s_keys, s_cnts, (uint32_t)cell, (uint32_t)__popc(same), votes_img);
        }
      }
    }
    if constexpr (CELLS) {
      // this lane's half of the group: VEC/2 consecutive pixels, one 16-byte (fp16) or 8-byte (fp32) store
      if (have) {
        uint32_t* dst = pix_cell + (size_t)b * plane + (size_t)span0 + (size_t)(ent & 0xffu) * VEC + (size_t)axis * (VEC / 2);
        if constexpr (VEC == 8)
          *reinterpret_cast<uint4*>(dst) = make_uint4(my_cells[0], my_cells[1], my_cells[2], my_cells[3]);
        else
          *reinterpret_cast<uint2*>(dst) = make_uint2(my_cells[0], my_cells[1]);
      }
    }
  }
  const uint32_t wv = __reduce_add_sync(0xffffffffu, voted);
  const uint32_t wb = __reduce_add_sync(0xffffffffu, nonfinite);
  if (lane == 0) {
    if (wv) atomicAdd(&s_voting, wv);
    if (wb) atomicAdd(&s_nonfinite, wb);
  }
  __syncthreads();
  for (int i = tid; i < kHashSlots; i += kVoteThreads) {
    const uint32_t k = s_keys[i];
    if (k != kHashEmpty) atomicAdd(&votes_img[k], s_cnts[i]);
  }
  if (tid == 0 && s_voting) atomicAdd(&acc[b * kAccStride + kAccVoting], s_voting);
  if (tid == 0 && s_nonfinite) atomicAdd(&acc[b * kAccStride + kAccNonfinite], s_nonfinite);
  if constexpr ((MODE & kVotePeaks) != 0) vote_then_peaks<kVoteThreads>(pa, b, acc, s_vote_map);
}

}  // namespace cpe
