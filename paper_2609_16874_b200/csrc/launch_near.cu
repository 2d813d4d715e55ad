// Launchers of the pruned assignment: the per-peak candidate lists, and the kernel that walks them.
#include <algorithm>

#include "assign_near.cuh"
#include "launch.h"
#include "peak_graph.cuh"

namespace cpe {
namespace host {

int launch_peak_graph(cudaStream_t st, int B, int F, const cpe_params* p, const float* ref_emb, const float* cand_emb,
                      const int32_t* count, int k_min, float* ref2, float* cand2, void* ref_h, void* cand_h, uint32_t* nbr,
                      long long* sums_to_zero, int cells) {
  // one CTA per peak; no image has more than min(max_instances, kNearMaxPeaks) peaks to list
  const int k_cap = std::min(p->max_instances, cpe::kNearMaxPeaks);
  const int per_image = std::max(1, (8 * sm_count() + B - 1) / B);
  dim3 grid((unsigned)std::min(k_cap, per_image), (unsigned)B);
  const size_t smem = 0;
#define CPE_GRAPH(FT_)                                                                                               \
  CPE_CUDA(launch_dependent(plain_launch(p), cpe::peak_graph_kernel<FT_>, grid, cpe::kGraphThreads, smem, st, ref_emb, \
                            cand_emb, count, p->max_instances, k_min, ref2, cand2,             \
                            static_cast<__half*>(ref_h), static_cast<__half*>(cand_h), nbr, sums_to_zero, cells))
  switch (F) {
    case 4: CPE_GRAPH(4); break;
    case 8: CPE_GRAPH(8); break;
    case 16: CPE_GRAPH(16); break;
    default: return CPE_ERR_SIZE;     // the caller enables the pruned assignment for these F only
  }
#undef CPE_GRAPH
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

namespace {

struct NearArgs {
  const void* emb;
  const uint8_t* fg;
  int B, HW;
  const cpe_params* p;
  const float *ref_emb, *cand_emb, *ref2, *cand2;
  const uint32_t* nbr;
  const int32_t* cell_peak;
  const uint32_t* pix_cell;
  int cells;
  const int32_t* count;
  int32_t* labels;
  float *best, *second;
  uint32_t* near_state;
  int k_min;
  uint32_t* slow_q;
  int q_cap;
  uint32_t* status;
  const void *ref_h, *cand_h;
  uint32_t* hard_q;
  int W;
};

template <typename T, int FT, bool WANT2>
int launch_walk_t(cudaStream_t st, const NearArgs& a) {
  // a bounded grid (a few CTAs per SM, shared among the images) walks the pixel blocks
  const long long n_blocks = ((long long)a.HW + cpe::kNearThreads - 1) / cpe::kNearThreads;
  const int resident = FT == 16 ? 2 : 3;
  const long long per_image = std::max(1, (2 * resident * sm_count() + a.B - 1) / a.B);
  dim3 grid((unsigned)std::min(n_blocks, per_image), (unsigned)a.B);
  CPE_CUDA(launch_dependent(plain_launch(a.p), cpe::assign_near_kernel<T, FT, WANT2>, grid, cpe::kNearThreads, 0, st,
                            static_cast<const T*>(a.emb), a.fg, a.HW, a.p->max_instances, a.ref2, a.cand2, a.nbr,
                            a.cell_peak, a.pix_cell, a.cells, a.count, a.p->tau, a.labels, a.best, a.second, a.near_state,
                            a.k_min));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

template <typename T, int FT, bool SAME>
int launch_stream_t(cudaStream_t st, const NearArgs& a) {
  constexpr int VEC = cpe::Elem<T>::kVec;
  constexpr int D = 4 * FT;
  // shared memory for the binary16 rows: what max_instances peaks need, at most what leaves room for three CTAs per SM
  const size_t want = (size_t)std::min(a.p->max_instances, cpe::kNearMaxPeaks) * D * 2 * (SAME ? 1 : 2);
  const int smem = (int)std::min<size_t>(want, 72 * 1024);
  auto kern = cpe::assign_near_stream_kernel<T, FT, SAME>;
  static bool configured[64] = {};
  CPE_CUDA(allow_dynamic_smem(kern, 72 * 1024, configured));
  // a warp takes 16 groups per step; a bounded grid (three CTAs per SM), shared among the images
  const long long n_steps = ((long long)a.HW / VEC + 15) / 16;
  const long long ctas = (n_steps + cpe::kStreamThreads / 32 - 1) / (cpe::kStreamThreads / 32);
  const long long per_image = std::max(1, (cpe::stream_ctas_per_sm(FT) * sm_count() + a.B - 1) / a.B);
  dim3 grid((unsigned)std::min(ctas, per_image), (unsigned)a.B);
  CPE_CUDA(launch_dependent(plain_launch(a.p), kern, grid, cpe::kStreamThreads, (size_t)smem, st,
                            static_cast<const T*>(a.emb), a.fg, a.HW, a.p->max_instances,
                            static_cast<const __half*>(a.ref_h), static_cast<const __half*>(a.cand_h), a.nbr, a.cell_peak,
                            a.pix_cell, a.cells, a.count, a.p->tau, a.labels, a.near_state, a.slow_q, a.q_cap, a.k_min,
                            smem, a.ref2, a.cand2, a.hard_q));
  CPE_CUDA(cudaGetLastError());
  // the pixels it queued
  const long long walk_ctas = std::max(1, ((FT == 16 ? 2 : 3) * sm_count() + a.B - 1) / a.B);
  dim3 wgrid((unsigned)std::min<long long>(walk_ctas, (a.q_cap + cpe::kNearThreads - 1) / cpe::kNearThreads), (unsigned)a.B);
  CPE_CUDA(launch_dependent(plain_launch(a.p), cpe::assign_near_walk_kernel<T, FT>, wgrid, cpe::kNearThreads, 0, st,
                            static_cast<const T*>(a.emb), a.HW, a.p->max_instances, a.ref2, a.cand2, a.nbr, a.cell_peak,
                            a.pix_cell, a.cells, a.count, a.p->tau, a.labels, a.near_state, a.slow_q, a.hard_q, a.q_cap,
                            a.k_min));
  CPE_CUDA(cudaGetLastError());
  // ... and the pixels that the walk left to the scan of every peak, one warp each
  // (a pixel keeps its warp for a few microseconds of dependent fetches: as many warps as the SMs hold)
  const long long hard_ctas = std::max(1, (8 * sm_count() + a.B - 1) / a.B);
  dim3 hgrid((unsigned)std::min<long long>(hard_ctas, (a.q_cap + 7) / 8), (unsigned)a.B);
  CPE_CUDA(launch_dependent(plain_launch(a.p), cpe::assign_near_hard_kernel<T, FT>, hgrid, cpe::kNearThreads, 0, st,
                            static_cast<const T*>(a.emb), a.HW, a.p->max_instances, a.cand2, a.count, a.p->tau, a.labels,
                            a.near_state, a.hard_q, a.q_cap, a.k_min));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

template <typename T, int FT>
int launch_near_ft(cudaStream_t st, const NearArgs& a) {
  const bool want2 = a.best != nullptr;
  const bool same = a.ref2 == a.cand2;
  constexpr int VEC = cpe::Elem<T>::kVec;
  // the streaming kernel: 128-bit plane loads, 128-bit label and bin accesses, no scores
  const bool vec = !want2 && ((uintptr_t)a.emb % 16 == 0) && (a.HW % VEC == 0) && (!a.fg || (uintptr_t)a.fg % VEC == 0) &&
                   ((uintptr_t)a.labels % 16 == 0) && !(a.p->flags & CPE_FLAG_PRUNE_WALK_ONLY);
  if (vec) return same ? launch_stream_t<T, FT, true>(st, a) : launch_stream_t<T, FT, false>(st, a);
  return want2 ? launch_walk_t<T, FT, true>(st, a) : launch_walk_t<T, FT, false>(st, a);
}

template <typename T>
int launch_near_f(cudaStream_t st, int F, const NearArgs& a) {
  switch (F) {
    case 4: return launch_near_ft<T, 4>(st, a);
    case 8: return launch_near_ft<T, 8>(st, a);
    case 16: return launch_near_ft<T, 16>(st, a);
    default: return CPE_ERR_SIZE;     // the caller enables the pruned assignment for these F only
  }
}

}  // namespace

int launch_assign_near(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                       const float* ref_emb, const float* cand_emb, const float* ref2, const float* cand2,
                       const uint32_t* nbr, const int32_t* cell_peak, const uint32_t* pix_cell, int cells,
                       const int32_t* count, int32_t* labels, float* best, float* second, uint32_t* near_state, int k_min,
                       uint32_t* slow_q, int q_cap, uint32_t* status, const void* ref_h, const void* cand_h,
                       uint32_t* hard_q, int W) {
  const NearArgs a{emb, fg, B, HW, p, ref_emb, cand_emb, ref2, cand2, nbr, cell_peak, pix_cell, cells, count, labels, best,
                   second, near_state, k_min, slow_q, q_cap, status, ref_h, cand_h, hard_q, W};
  return p->dtype == CPE_F32 ? launch_near_f<float>(st, F, a) : launch_near_f<__half>(st, F, a);
}

}  // namespace host
}  // namespace cpe
