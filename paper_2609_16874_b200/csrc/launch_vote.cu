// Launcher of stage 1+2 (per-pixel estimate and hard vote): picks the vectorised or the scalar-load kernel.
#include <algorithm>

#include "decode_vote.cuh"
#include "launch.h"

namespace cpe {
namespace host {

namespace {

template <typename T>
int launch_decode_vote_t(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                         uint32_t* votes, uint32_t* acc, long long* sums, uint32_t* pix_cell,
                         const cpe::PeakArgs* fused) {
  const T* e = static_cast<const T*>(emb);
  const cpe::PeakArgs pa = fused ? *fused : cpe::PeakArgs{};
  // the fused search works on a copy of the vote map in shared memory
  const size_t map_smem = fused ? 4 * (size_t)p->bins_w * p->bins_h : 0;
  if (fused && map_smem > 48 * 1024) return CPE_ERR_SIZE;     // (callers ask vote_can_fuse_peaks first)
  constexpr int V = cpe::Elem<T>::kVec;
  // 128-bit plane loads: every plane of every image must start on a 16-byte boundary
  const bool vec = ((uintptr_t)emb % 16 == 0) && (HW % V == 0) && (!fg || (uintptr_t)fg % V == 0) &&
                   (F == 4 || F == 8 || F == 16);
  if (vec) {
    const long long groups = (long long)HW / V;
    // the largest span that still gives one full wave of CTAs (four resident per SM), else the smallest
    const long long wave = 4LL * sm_count();
    const int span = fused ? 64 : (groups + 255) / 256 * B >= wave ? 256 : (groups + 127) / 128 * B >= wave ? 128 : 64;
    dim3 grid((unsigned)((groups + span - 1) / span), (unsigned)B);
#define CPE_LAUNCH_VOTE_G(FT_, RF_, G_)                                                                              \
  cpe::decode_vote_vec_kernel<T, FT_, RF_, G_><<<grid, cpe::kVoteThreads, map_smem, st>>>(                            \
      e, fg, HW, p->levels, p->bins_w, p->bins_h, votes, acc, sums, pix_cell, pa)
#define CPE_LAUNCH_VOTE_R(FT_, RF_)                                                                                   \
  switch (span) {                                                                                                     \
    case 256: CPE_LAUNCH_VOTE_G(FT_, RF_, 256); break;                                                                \
    case 128: CPE_LAUNCH_VOTE_G(FT_, RF_, 128); break;                                                                \
    default: CPE_LAUNCH_VOTE_G(FT_, RF_, 64); break;                                                                  \
  }
#define CPE_LAUNCH_VOTE(FT_)                                                                                          \
  if (fused) {                                                                                                        \
    if (sums) CPE_LAUNCH_VOTE_G(FT_, 5, 64); else CPE_LAUNCH_VOTE_G(FT_, 4, 64);                                      \
  } else if (pix_cell) { CPE_LAUNCH_VOTE_R(FT_, 3) } else if (sums) { CPE_LAUNCH_VOTE_R(FT_, 1) } else { CPE_LAUNCH_VOTE_R(FT_, 0) }
    switch (F) {
      case 4: CPE_LAUNCH_VOTE(4); break;
      case 8: CPE_LAUNCH_VOTE(8); break;
      default: CPE_LAUNCH_VOTE(16); break;
    }
#undef CPE_LAUNCH_VOTE
#undef CPE_LAUNCH_VOTE_R
#undef CPE_LAUNCH_VOTE_G
  } else {
    // 64-bit mask loads need every image's mask to start on an 8-byte boundary
    const int vec_mask = fg && ((uintptr_t)fg % 8 == 0) && (HW % 8 == 0);
    dim3 grid((unsigned)(((long long)HW + cpe::kVoteSpan - 1) / cpe::kVoteSpan), (unsigned)B);
#define CPE_LAUNCH_VOTE_M(FT_, M_)                                                                                       \
  cpe::decode_vote_scalar_kernel<T, FT_, M_><<<grid, cpe::kVoteThreads, map_smem, st>>>(                                 \
      e, fg, HW, F, p->levels, p->bins_w, p->bins_h, vec_mask, votes, acc, sums, pix_cell, pa)
#define CPE_LAUNCH_VOTE(FT_)                                                                                             \
  if (fused) { if (sums) CPE_LAUNCH_VOTE_M(FT_, 5); else CPE_LAUNCH_VOTE_M(FT_, 4); }                                    \
  else if (pix_cell) CPE_LAUNCH_VOTE_M(FT_, 3); else if (sums) CPE_LAUNCH_VOTE_M(FT_, 1); else CPE_LAUNCH_VOTE_M(FT_, 0)
    switch (F) {
      case 4: CPE_LAUNCH_VOTE(4); break;
      case 8: CPE_LAUNCH_VOTE(8); break;
      case 16: CPE_LAUNCH_VOTE(16); break;
      default: CPE_LAUNCH_VOTE(0); break;
    }
#undef CPE_LAUNCH_VOTE
#undef CPE_LAUNCH_VOTE_M
  }
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

}  // namespace

int launch_decode_vote(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                       uint32_t* votes, uint32_t* acc, long long* sums, uint32_t* pix_cell, const cpe::PeakArgs* fused) {
  return p->dtype == CPE_F32 ? launch_decode_vote_t<float>(st, emb, fg, B, HW, F, p, votes, acc, sums, pix_cell, fused)
                             : launch_decode_vote_t<__half>(st, emb, fg, B, HW, F, p, votes, acc, sums, pix_cell, fused);
}

// On request (CPE_FLAG_FUSE_PEAKS) and for small inputs only: there the launch saved is a sizeable part of the decode,
// and the voting CTAs are short anyway (the fused variant always takes the shortest spans).
bool vote_can_fuse_peaks(int B, int HW, int words, const cpe_params* p) {
  return (p->flags & CPE_FLAG_FUSE_PEAKS) && words <= cpe::kPeakStageWords && (long long)B * HW <= (1 << 20);
}

int launch_peaks(cudaStream_t st, int B, const cpe_params* p, const cpe::PeakArgs& a) {
  const int warps_per_cta = cpe::kPeakThreads / 32;
  // small maps: one CTA per image does both phases without the cross-CTA hand-over, on a copy of the vote map in
  // shared memory (at most 32 KB)
  const int ctas = a.staged ? 1 : (a.words + warps_per_cta - 1) / warps_per_cta;
  const size_t map_smem = a.staged ? 4 * (size_t)a.bins_w * a.bins_h : 0;
  CPE_CUDA(launch_dependent(plain_launch(p), cpe::peaks_kernel, dim3((unsigned)ctas, (unsigned)B), cpe::kPeakThreads,
                            map_smem, st, a));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

int launch_peak_rows(cudaStream_t st, int B, int F, const cpe_params* p, const uint32_t* votes, const long long* sums, int H,
                     int W, const int32_t* peak_cell, const int32_t* count, int refine_out, float* gamma_out,
                     float* out_centroids, const float* pal_w, const float* pal_h, float* peak_emb) {
  // gamma of every peak's mean estimate (the bounds' reference points; the candidates too when they are refined),
  // a thread per (peak, axis, harmonic) over as many CTAs as the largest image can need
  const int k_cap = std::min(p->max_instances, cpe::kNearMaxPeaks);
  const int ctas = std::max(1, std::min((k_cap * 2 * F + cpe::kRowsThreads - 1) / cpe::kRowsThreads, 4 * sm_count()));
  CPE_CUDA(launch_dependent(plain_launch(p), cpe::peak_rows_kernel, dim3((unsigned)ctas, (unsigned)B), cpe::kRowsThreads, 0,
                            st, votes, sums, p->bins_w, p->bins_h, p->max_instances, F, H, W, peak_cell, count, refine_out,
                            gamma_out, out_centroids, pal_w, pal_h, peak_emb));
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

}  // namespace host
}  // namespace cpe
