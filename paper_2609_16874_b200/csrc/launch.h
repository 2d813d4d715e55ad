// Host-side plumbing shared by the translation units of the library: error bookkeeping, the dependent-launch
// helper, and the launchers that each unit exports to the C ABI in cpe_api.cu.  (The kernels are templates in the
// .cuh files; every launcher lives in the one unit that instantiates its kernels, so the units compile in parallel.)
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "cpe.h"
#include "cpe_common.cuh"

namespace cpe {
namespace host {

// Records the CUDA error behind the calling thread's CPE_ERR_CUDA and returns that code.
int cuda_fail(cudaError_t e);

#define CPE_CUDA(call)                                        \
  do {                                                        \
    cudaError_t e_ = (call);                                  \
    if (e_ != cudaSuccess) return ::cpe::host::cuda_fail(e_); \
  } while (0)

// SMs of the current device (cached per device).
int sm_count();

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per (kernel instantiation, device): the attribute belongs
// to the device's copy of the function.  `done` is a per-instantiation table indexed by the device ordinal.
template <typename K>
cudaError_t allow_dynamic_smem(K kern, int bytes, bool (&done)[64]) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
  return e;
}

// Launch of a kernel that consumes what the kernel before it in the stream wrote, with programmatic stream
// serialisation: its CTAs may be scheduled while the predecessor is still running and wait on the device
// (grid_dependency_sync at the top of every kernel of the chain).  `plain` launches without the attribute.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(bool plain, void (*kern)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t st,
                             Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = plain ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

inline bool plain_launch(const cpe_params* p) { return (p->flags & CPE_FLAG_NO_PDL) != 0; }

// ---- stage 1+2 (launch_vote.cu).  sums: per-bin fixed-point sums or NULL; pix_cell: per-pixel bin or NULL;
// fused_peaks: not NULL = the last CTA of each image also runs the peak search (stage 3) on its small map, and
// launch_peaks is not called.
int launch_decode_vote(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                       uint32_t* votes, uint32_t* acc, long long* sums, uint32_t* pix_cell,
                       const cpe::PeakArgs* fused_peaks);
// Whether launch_decode_vote can take stage 3 along for this problem.
bool vote_can_fuse_peaks(int B, int HW, int words, const cpe_params* p);

// ---- stage 3 (launch_vote.cu): the peak search, and (pruned assignment) the kernel that writes the peaks' rows
int launch_peaks(cudaStream_t st, int B, const cpe_params* p, const cpe::PeakArgs& a);
int launch_peak_rows(cudaStream_t st, int B, int F, const cpe_params* p, const uint32_t* votes, const long long* sums, int H,
                     int W, const int32_t* peak_cell, const int32_t* count, int refine_out, float* gamma_out,
                     float* out_centroids, const float* pal_w, const float* pal_h, float* peak_emb);

// ---- stage 4+5, tensor-core filtered kernels (launch_filter.cu): images with at least k_min peaks.
int launch_assign_filtered(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                           const float* peak_emb, const int32_t* count, int32_t* labels, float* best, float* second,
                           uint32_t* counters, uint32_t* status, uint32_t* votes_to_zero, int cells, int k_min,
                           uint32_t* acc, const uint32_t* near_state);

// ---- the pruned assignment (launch_near.cu): candidate lists per peak, then the kernel that walks them.  Images with
// fewer than k_min peaks are left alone; near_state tells the filtered kernel, launched afterwards, which images it
// is handed.
int launch_peak_graph(cudaStream_t st, int B, int F, const cpe_params* p, const float* ref_emb, const float* cand_emb,
                      const int32_t* count, int k_min, float* ref2, float* cand2, void* ref_h, void* cand_h, uint32_t* nbr,
                      long long* sums_to_zero, int cells);
int launch_assign_near(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                       const float* ref_emb, const float* cand_emb, const float* ref2, const float* cand2,
                       const uint32_t* nbr, const int32_t* cell_peak, const uint32_t* pix_cell, int cells,
                       const int32_t* count, int32_t* labels, float* best, float* second, uint32_t* near_state, int k_min,
                       uint32_t* slow_q, int q_cap, uint32_t* status, const void* ref_h, const void* cand_h,
                       uint32_t* hard_q, int W);

// ---- second vote mode (launch_soft.cu).  acc: the per-image accumulators that the peak kernel folds into the
// counters (participating / non-finite pixels), or NULL.
int launch_soft_votes(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                      const float* pal_w, const float* pal_h, float* hist, uint32_t* status, uint32_t* acc);

}  // namespace host
}  // namespace cpe
