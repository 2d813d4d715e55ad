// Launcher of the second vote mode (soft-vote histogram, Eq. 6 / Eq. 10-11).
#include <algorithm>

#include "launch.h"
#include "soft_vote.cuh"

namespace cpe {
namespace host {

namespace {
template <typename T, int KA>
int launch_soft_votes_t(cudaStream_t st, const T* e, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                        const float* pal_w, const float* pal_h, float* hist, uint32_t* status, uint32_t* acc) {
  const int smem = cpe::sv_smem_layout(KA).total;
  auto kern = cpe::soft_vote_kernel<T, KA>;
  static bool configured[64] = {};
  CPE_CUDA(allow_dynamic_smem(kern, 200 * 1024, configured));
  // one CTA per SM (it holds all of the SM's tensor memory): the SMs are shared among the images and the
  // 128 x 128 blocks of bins, the CTAs of one block split the pixels
  const int n_blocks = ((p->bins_w + cpe::kSvBins - 1) / cpe::kSvBins) * ((p->bins_h + cpe::kSvBins - 1) / cpe::kSvBins);
  const int n_spans = (HW + cpe::kTcSpan - 1) / cpe::kTcSpan;
  const int split = std::max(1, std::min(n_spans, sm_count() / std::max(1, n_blocks * B)));
  dim3 grid((unsigned)split, (unsigned)n_blocks, (unsigned)B);
  const int vec_mask = fg && ((uintptr_t)fg % 8 == 0) ? 1 : 0;
  kern<<<grid, cpe::kSvThreads, smem, st>>>(e, fg, HW, F, p->bins_w, p->bins_h, pal_w, pal_h, vec_mask, hist, status, acc);
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}
}  // namespace

int launch_soft_votes(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                      const float* pal_w, const float* pal_h, float* hist, uint32_t* status, uint32_t* acc) {
  if (p->dtype == CPE_F32)
    return F <= 8 ? launch_soft_votes_t<float, 16>(st, static_cast<const float*>(emb), fg, B, HW, F, p, pal_w, pal_h, hist,
                                                   status, acc)
                  : launch_soft_votes_t<float, 32>(st, static_cast<const float*>(emb), fg, B, HW, F, p, pal_w, pal_h, hist,
                                                   status, acc);
  return F <= 8 ? launch_soft_votes_t<__half, 16>(st, static_cast<const __half*>(emb), fg, B, HW, F, p, pal_w, pal_h, hist,
                                                  status, acc)
                : launch_soft_votes_t<__half, 32>(st, static_cast<const __half*>(emb), fg, B, HW, F, p, pal_w, pal_h, hist,
                                                  status, acc);
}

}  // namespace host
}  // namespace cpe
