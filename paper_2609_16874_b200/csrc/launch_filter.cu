// Launchers of the tensor-core filtered assignment (stage 4+5): the merged tcgen05 / mma.sync kernel for 16-byte
// aligned planes, the mma.sync kernel alone otherwise.
#include <math.h>

#include <algorithm>

#include "assign_mma.cuh"
#include "assign_tc.cuh"
#include "launch.h"

namespace cpe {
namespace host {

namespace {

template <typename T, int KA, bool WANT2>
int launch_assign_mma_t(cudaStream_t st, const T* e, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                        const float* peak_emb, const int32_t* count, int32_t* labels, float* best, float* second,
                        uint32_t* counters, uint32_t* status, uint32_t* votes_to_zero, int cells, int k_min,
                        const uint32_t* near_state) {
  // small inputs get short spans so that there are enough CTAs to fill the GPU
  const int span = ((long long)B * HW >= (1 << 20)) ? cpe::kAmSpanMax : 512;
  // 16-byte gathers of whole 8-pixel groups need aligned planes and the long span
  const int vec_gather = (span == cpe::kAmSpanMax) && ((uintptr_t)e % 16 == 0) && (HW % 8 == 0);
  const int two_tiles = (vec_gather && sizeof(T) == 2 && KA == 16) ? 1 : 0;
  // as many peaks resident in shared memory as leave room for two CTAs per SM
  int peak_cap = (p->max_instances + 7) & ~7;
  const int budget = 110 * 1024;
  const int fixed = cpe::am_smem_layout(KA, 0, span, two_tiles).total;
  peak_cap = std::max(8, std::min(peak_cap, ((budget - fixed) / ((2 * KA + 8) * 2)) & ~7));
  const int smem = cpe::am_smem_layout(KA, peak_cap, span, two_tiles).total;
  auto kern = cpe::assign_mma_kernel<T, KA, WANT2>;
  static bool configured[64] = {};
  CPE_CUDA(allow_dynamic_smem(kern, 160 * 1024, configured));
  const int n_spans = (HW + span - 1) / span;
  const int per_image = std::max(1, (2 * sm_count() + B - 1) / B);
  dim3 grid((unsigned)std::min(n_spans, per_image), (unsigned)B);
  const int vec_mask = fg && ((uintptr_t)fg % 8 == 0) && (HW % 8 == 0);
  const int need_exact = p->tau < INFINITY ? 1 : 0;
  CPE_CUDA(launch_dependent(plain_launch(p), kern, grid, cpe::kAmThreads, smem, st, e, fg, HW, F, p->max_instances,
                            peak_emb, count, p->tau, need_exact, peak_cap, span, vec_mask, vec_gather, labels, best, second,
                            counters, status, votes_to_zero, cells, k_min, near_state));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

// The filtered assignment for 16-byte aligned planes: one launch, the tcgen05 pipeline for the images whose peaks
// fit one of its rounds, the mma.sync body for the others (the choice is made on the device, per image).
template <typename T, int KA, bool WANT2>
int launch_assign_filter_t(cudaStream_t st, const T* e, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                           const float* peak_emb, const int32_t* count, int32_t* labels, float* best, float* second,
                           uint32_t* counters, uint32_t* status, uint32_t* votes_to_zero, int cells, int k_min, uint32_t* acc,
                           const uint32_t* near_state) {
  // tcgen05 body: as many peaks resident in shared memory as leave room for two CTAs per SM (each CTA holds half of
  // the SM's tensor memory, so there must never be more than two)
  const int budget = 104 * 1024;
  int tc_cap = (p->max_instances + cpe::kTcRound - 1) / cpe::kTcRound * cpe::kTcRound;
  const int tc_fixed = cpe::tc_smem_layout(KA, 0).total;
  tc_cap = std::max(cpe::kTcRound, std::min(tc_cap, (budget - tc_fixed) / (2 * KA * 2) / cpe::kTcRound * cpe::kTcRound));
  // up to 128 peaks fit the two tensor-memory stages at once; beyond that the mma.sync body is the faster one
  // (CPE_FLAG_TC_ALL_ROUNDS lifts the limit, CPE_FLAG_TC_ONE_STAGE keeps it at one stage: tests, comparisons)
  const int tc_k_max = (p->flags & CPE_FLAG_TC_ALL_ROUNDS)  ? tc_cap
                       : (p->flags & CPE_FLAG_TC_ONE_STAGE) ? std::min(tc_cap, cpe::kTcRound)
                                                            : std::min(tc_cap, 2 * cpe::kTcRound);
  const int tc_smem = cpe::tc_smem_layout(KA, tc_cap).total;
  // mma.sync body
  const int span = ((long long)B * HW >= (1 << 20)) ? cpe::kAmSpanMax : 512;
  const int vec_gather = span == cpe::kAmSpanMax ? 1 : 0;
  const int two_tiles = (vec_gather && sizeof(T) == 2 && KA == 16) ? 1 : 0;
  int mma_cap = (p->max_instances + 7) & ~7;
  const int mma_fixed = cpe::am_smem_layout(KA, 0, span, two_tiles).total;
  mma_cap = std::max(8, std::min(mma_cap, ((110 * 1024 - mma_fixed) / ((2 * KA + 8) * 2)) & ~7));
  const int mma_smem = cpe::am_smem_layout(KA, mma_cap, span, two_tiles).total;
  const int smem = std::max(std::max(tc_smem, mma_smem), 78 * 1024);
  auto kern = cpe::assign_filter_kernel<T, KA, WANT2>;
  static bool configured[64] = {};
  CPE_CUDA(allow_dynamic_smem(kern, 160 * 1024, configured));
  const int n_spans = (HW + cpe::kTcSpan - 1) / cpe::kTcSpan;
  const int per_image = std::max(1, (2 * sm_count() + B - 1) / B);
  dim3 grid((unsigned)std::min(n_spans, per_image), (unsigned)B);
  const int vec_mask = fg && ((uintptr_t)fg % 8 == 0) ? 1 : 0;
  const int need_exact = p->tau < INFINITY ? 1 : 0;
  CPE_CUDA(launch_dependent(plain_launch(p), kern, grid, cpe::kTcThreads, smem, st, e, fg, HW, F, p->max_instances,
                            peak_emb, count, p->tau, need_exact, tc_cap, tc_k_max, vec_mask, mma_cap, span, vec_mask,
                            vec_gather, labels, best, second, counters, status, votes_to_zero, cells, k_min, acc,
                            near_state, (p->flags & CPE_FLAG_TEST_STALL) ? 1 : 0));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

template <typename T>
int launch_assign_filtered_t(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F,
                             const cpe_params* p, const float* peak_emb, const int32_t* count, int32_t* labels, float* best,
                             float* second, uint32_t* counters, uint32_t* status, uint32_t* votes_to_zero, int cells,
                             int k_min, uint32_t* acc, const uint32_t* near_state) {
  const T* e = static_cast<const T*>(emb);
  const bool want2 = best != nullptr;
  // CPE_FLAG_MMA_ASSIGN keeps the mma.sync kernel everywhere (comparisons)
  const bool aligned = (uintptr_t)e % 16 == 0 && HW % 8 == 0;
  if (aligned && !(p->flags & CPE_FLAG_MMA_ASSIGN)) {
    if (F <= 8)
      return want2 ? launch_assign_filter_t<T, 16, true>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second,
                                                         counters, status, votes_to_zero, cells, k_min, acc, near_state)
                   : launch_assign_filter_t<T, 16, false>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second,
                                                          counters, status, votes_to_zero, cells, k_min, acc, near_state);
    return want2 ? launch_assign_filter_t<T, 32, true>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second,
                                                       counters, status, votes_to_zero, cells, k_min, acc, near_state)
                 : launch_assign_filter_t<T, 32, false>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second,
                                                        counters, status, votes_to_zero, cells, k_min, acc, near_state);
  }
  if (F <= 8) {
    return want2 ? launch_assign_mma_t<T, 16, true>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                                    status, votes_to_zero, cells, k_min, near_state)
                 : launch_assign_mma_t<T, 16, false>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second,
                                                     counters, status, votes_to_zero, cells, k_min, near_state);
  }
  return want2 ? launch_assign_mma_t<T, 32, true>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                                  status, votes_to_zero, cells, k_min, near_state)
               : launch_assign_mma_t<T, 32, false>(st, e, fg, B, HW, F, p, peak_emb, count, labels, best, second,
                                                   counters, status, votes_to_zero, cells, k_min, near_state);
}

}  // namespace

int launch_assign_filtered(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                           const float* peak_emb, const int32_t* count, int32_t* labels, float* best, float* second,
                           uint32_t* counters, uint32_t* status, uint32_t* votes_to_zero, int cells, int k_min,
                           uint32_t* acc, const uint32_t* near_state) {
  return p->dtype == CPE_F32
             ? launch_assign_filtered_t<float>(st, emb, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                               status, votes_to_zero, cells, k_min, acc, near_state)
             : launch_assign_filtered_t<__half>(st, emb, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                                status, votes_to_zero, cells, k_min, acc, near_state);
}

}  // namespace host
}  // namespace cpe
