// Launchers of the pruned assignment: the per-peak candidate lists, and the kernel that walks them.
#include <algorithm>

#include "assign_near.cuh"
#include "launch.h"
#include "peak_graph.cuh"

namespace cpe {
namespace host {

int launch_peak_graph(cudaStream_t st, int B, int F, const cpe_params* p, const float* ref_emb, const float* cand_emb,
                      const int32_t* count, int k_min, float* ref2, float* cand2, uint32_t* nbr) {
  // one warp per peak; no image has more than min(max_instances, kNearMaxPeaks) peaks to list
  const int warps = cpe::kGraphThreads / 32;
  const int k_cap = std::min(p->max_instances, cpe::kNearMaxPeaks);
  const int per_image = std::max(1, (4 * sm_count() + B - 1) / B);
  dim3 grid((unsigned)std::min((k_cap + warps - 1) / warps, per_image), (unsigned)B);
  const size_t smem = sizeof(uint32_t) * (size_t)warps * cpe::kNearMaxPeaks;
  CPE_CUDA(launch_dependent(plain_launch(p), cpe::peak_graph_kernel, grid, cpe::kGraphThreads, smem, st, ref_emb, cand_emb,
                            count, p->max_instances, F, k_min, ref2, cand2, nbr));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

namespace {

template <typename T, int FT, bool WANT2>
int launch_assign_near_t(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, const cpe_params* p,
                         const float* ref2, const float* cand2, const uint32_t* nbr, const int32_t* cell_peak,
                         const uint32_t* pix_cell, int cells, const int32_t* count, int32_t* labels, float* best,
                         float* second, uint32_t* near_state, int k_min) {
  // a bounded grid (a few CTAs per SM, shared among the images) walks the pixel blocks
  const long long n_blocks = ((long long)HW + cpe::kNearThreads - 1) / cpe::kNearThreads;
  const int resident = FT == 16 ? 2 : 3;
  const long long per_image = std::max(1, (2 * resident * sm_count() + B - 1) / B);
  dim3 grid((unsigned)std::min(n_blocks, per_image), (unsigned)B);
  CPE_CUDA(launch_dependent(plain_launch(p), cpe::assign_near_kernel<T, FT, WANT2>, grid, cpe::kNearThreads, 0, st,
                            static_cast<const T*>(emb), fg, HW, p->max_instances, ref2, cand2, nbr, cell_peak, pix_cell,
                            cells, count, p->tau, labels, best, second, near_state, k_min));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

template <typename T, bool WANT2>
int launch_assign_near_f(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                         const float* ref2, const float* cand2, const uint32_t* nbr, const int32_t* cell_peak,
                         const uint32_t* pix_cell, int cells, const int32_t* count, int32_t* labels, float* best,
                         float* second, uint32_t* near_state, int k_min) {
#define CPE_NEAR(FT_)                                                                                                  \
  return launch_assign_near_t<T, FT_, WANT2>(st, emb, fg, B, HW, p, ref2, cand2, nbr, cell_peak, pix_cell, cells, count, \
                                             labels, best, second, near_state, k_min)
  switch (F) {
    case 4: CPE_NEAR(4);
    case 8: CPE_NEAR(8);
    case 16: CPE_NEAR(16);
    default: return CPE_ERR_SIZE;     // the caller enables the pruned assignment for these F only
  }
#undef CPE_NEAR
}

}  // namespace

int launch_assign_near(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                       const float* ref2, const float* cand2, const uint32_t* nbr, const int32_t* cell_peak,
                       const uint32_t* pix_cell, int cells, const int32_t* count, int32_t* labels, float* best,
                       float* second, uint32_t* near_state, int k_min) {
  const bool want2 = best != nullptr;
  if (p->dtype == CPE_F32)
    return want2 ? launch_assign_near_f<float, true>(st, emb, fg, B, HW, F, p, ref2, cand2, nbr, cell_peak, pix_cell, cells,
                                                     count, labels, best, second, near_state, k_min)
                 : launch_assign_near_f<float, false>(st, emb, fg, B, HW, F, p, ref2, cand2, nbr, cell_peak, pix_cell,
                                                      cells, count, labels, best, second, near_state, k_min);
  return want2 ? launch_assign_near_f<__half, true>(st, emb, fg, B, HW, F, p, ref2, cand2, nbr, cell_peak, pix_cell, cells,
                                                    count, labels, best, second, near_state, k_min)
               : launch_assign_near_f<__half, false>(st, emb, fg, B, HW, F, p, ref2, cand2, nbr, cell_peak, pix_cell,
                                                     cells, count, labels, best, second, near_state, k_min);
}

}  // namespace host
}  // namespace cpe
