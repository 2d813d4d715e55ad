// Stage 1+2: per-pixel centroid estimate and hard-vote accumulation (hard-vote form of Eq. 6 on the
// Eq. 9 bins).  HBM-bound: each participating pixel's 4F channel values are read once with 128-bit
// loads from the channel planes; groups of pixels that do not participate are never fetched.
#pragma once

#include "cpe_common.cuh"

namespace cpe {

constexpr int kVoteThreads = 256;
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

// One thread owns VEC consecutive pixels (one 128-bit load per channel plane when VEC is the vector
// width).  FT > 0 fixes F at compile time.
template <typename T, int VEC, int FT>
__global__ void __launch_bounds__(kVoteThreads)
decode_vote_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F_rt, int levels,
                   int bins_w, int bins_h, uint32_t* __restrict__ votes, uint32_t* __restrict__ counters,
                   uint32_t* __restrict__ status) {
  const int F = FT > 0 ? FT : F_rt;
  const int Fu = (levels > 0 && levels < F) ? levels : F;
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const size_t plane = (size_t)HW;
  const T* e = emb + (size_t)b * 4 * F * plane;
  uint32_t* votes_img = votes + (size_t)b * bins_w * bins_h;

  __shared__ uint32_t s_keys[kHashSlots];
  __shared__ uint32_t s_cnts[kHashSlots];
  __shared__ uint32_t s_nonfinite, s_voting;
  for (int i = tid; i < kHashSlots; i += kVoteThreads) {
    s_keys[i] = kHashEmpty;
    s_cnts[i] = 0;
  }
  if (tid == 0) s_nonfinite = s_voting = 0;
  __syncthreads();

  const long long n0 = ((long long)blockIdx.x * kVoteThreads + tid) * VEC;
  bool take[VEC];
  bool any = false;
#pragma unroll
  for (int j = 0; j < VEC; ++j) take[j] = false;
  if (n0 < HW) {
    if (fg) {
      const uint8_t* m = fg + (size_t)b * plane + n0;
      if constexpr (VEC == 8) {
        const uint2 w = __ldg(reinterpret_cast<const uint2*>(m));
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          take[j] = ((w.x >> (8 * j)) & 0xffu) != 0;
          take[4 + j] = ((w.y >> (8 * j)) & 0xffu) != 0;
        }
      } else if constexpr (VEC == 4) {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(m));
#pragma unroll
        for (int j = 0; j < 4; ++j) take[j] = ((w >> (8 * j)) & 0xffu) != 0;
      } else {
        take[0] = __ldg(m) != 0;
      }
    } else {
#pragma unroll
      for (int j = 0; j < VEC; ++j) take[j] = true;
    }
#pragma unroll
    for (int j = 0; j < VEC; ++j) any |= take[j];
  }

  int cell[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) cell[j] = -1;
  uint32_t nonfinite = 0;

  if (any) {
    float p[2][VEC];
    bool ok[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) ok[j] = true;
#pragma unroll
    for (int axis = 0; axis < 2; ++axis) {
      const T* ea = e + (size_t)axis * 2 * F * plane + n0;
#pragma unroll 2
      for (int l = 0; l < F; ++l) {
        float s[VEC], c[VEC];
        load_elems<T, VEC>(ea + (size_t)(2 * l) * plane, s);
        load_elems<T, VEC>(ea + (size_t)(2 * l + 1) * plane, c);
        const float scale = pow2f(l), inv = pow2f(-l);
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
          ok[j] = ok[j] && pair_finite(s[j], c[j]);
          if (l < Fu) {
            const float u = atan2_ht(s[j], c[j]);
            p[axis][j] = (l == 0) ? u : refine(p[axis][j], u, scale, inv);
          }
        }
      }
    }
    const float half_w = (float)(bins_w + 1) * 0.5f, half_h = (float)(bins_h + 1) * 0.5f;
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      if (take[j]) {
        if (ok[j]) {
          const int cx = cell_of(wrap_unit(p[0][j]), half_w, bins_w);
          const int cy = cell_of(wrap_unit(p[1][j]), half_h, bins_h);
          cell[j] = cy * bins_w + cx;
        } else {
          ++nonfinite;
        }
      }
    }
  }

  // Warp-aggregated insertion into the CTA's cache.  Fast path: the whole warp votes for one bin.
  {
    int first = -1;
    uint32_t mine = 0;
    bool uniform = true;
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      if (cell[j] >= 0) {
        if (first < 0) first = cell[j];
        uniform = uniform && (cell[j] == first);
        ++mine;
      }
    }
    const uint32_t voters = __ballot_sync(0xffffffffu, mine > 0);
    if (voters) {
      const uint32_t warp_votes = __reduce_add_sync(0xffffffffu, mine);
      if (lane == 0) atomicAdd(&s_voting, warp_votes);
      const int leader = __ffs(voters) - 1;
      const int ref = __shfl_sync(0xffffffffu, first, leader);
      const bool warp_uniform = __all_sync(0xffffffffu, mine == 0 || (uniform && first == ref));
      if (warp_uniform) {
        if (lane == leader) vote_cache_add(s_keys, s_cnts, (uint32_t)ref, warp_votes, votes_img);
      } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
          const int key = cell[j];
          const uint32_t same = __match_any_sync(0xffffffffu, key);
          if (key >= 0 && lane == __ffs(same) - 1)
            vote_cache_add(s_keys, s_cnts, (uint32_t)key, (uint32_t)__popc(same), votes_img);
        }
      }
    }
    const uint32_t bad = __reduce_add_sync(0xffffffffu, nonfinite);
    if (bad && lane == 0) atomicAdd(&s_nonfinite, bad);
  }
  __syncthreads();

  // Flush: one global atomic per distinct bin per CTA.
  for (int i = tid; i < kHashSlots; i += kVoteThreads) {
    const uint32_t k = s_keys[i];
    if (k != kHashEmpty) atomicAdd(&votes_img[k], s_cnts[i]);
  }
  if (tid == 0 && s_voting) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_VOTING], s_voting);
  if (tid == 0 && s_nonfinite) {
    atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_NONFINITE], s_nonfinite);
    atomicOr(status, (uint32_t)CPE_STATUS_NONFINITE);
  }
}

}  // namespace cpe
