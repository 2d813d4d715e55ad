// Launcher of stage 1+2 (per-pixel estimate and hard vote): picks the vectorised or the scalar-load kernel.
#include "decode_vote.cuh"
#include "launch.h"

namespace cpe {
namespace host {

namespace {

template <typename T>
int launch_decode_vote_t(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                         uint32_t* votes, uint32_t* acc, long long* sums, uint32_t* pix_cell) {
  const T* e = static_cast<const T*>(emb);
  constexpr int V = cpe::Elem<T>::kVec;
  // 128-bit plane loads: every plane of every image must start on a 16-byte boundary
  const bool vec = ((uintptr_t)emb % 16 == 0) && (HW % V == 0) && (!fg || (uintptr_t)fg % V == 0) &&
                   (F == 4 || F == 8 || F == 16);
  if (vec) {
    const long long groups = (long long)HW / V;
    // the largest span that still gives one full wave of CTAs (four resident per SM), else the smallest
    const long long wave = 4LL * sm_count();
    const int span = (groups + 255) / 256 * B >= wave ? 256 : (groups + 127) / 128 * B >= wave ? 128 : 64;
    dim3 grid((unsigned)((groups + span - 1) / span), (unsigned)B);
#define CPE_LAUNCH_VOTE_G(FT_, RF_, G_)                                                                              \
  cpe::decode_vote_vec_kernel<T, FT_, RF_, G_><<<grid, cpe::kVoteThreads, 0, st>>>(e, fg, HW, p->levels, p->bins_w,   \
                                                                                  p->bins_h, votes, acc, sums, pix_cell)
#define CPE_LAUNCH_VOTE_R(FT_, RF_)                                                                                   \
  switch (span) {                                                                                                     \
    case 256: CPE_LAUNCH_VOTE_G(FT_, RF_, 256); break;                                                                \
    case 128: CPE_LAUNCH_VOTE_G(FT_, RF_, 128); break;                                                                \
    default: CPE_LAUNCH_VOTE_G(FT_, RF_, 64); break;                                                                  \
  }
#define CPE_LAUNCH_VOTE(FT_)                                                                                          \
  if (pix_cell) { CPE_LAUNCH_VOTE_R(FT_, 3) } else if (sums) { CPE_LAUNCH_VOTE_R(FT_, 1) } else { CPE_LAUNCH_VOTE_R(FT_, 0) }
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
  cpe::decode_vote_scalar_kernel<T, FT_, M_><<<grid, cpe::kVoteThreads, 0, st>>>(e, fg, HW, F, p->levels, p->bins_w,      \
                                                                                 p->bins_h, vec_mask, votes, acc, sums,   \
                                                                                 pix_cell)
#define CPE_LAUNCH_VOTE(FT_)                                                                                             \
  if (pix_cell) CPE_LAUNCH_VOTE_M(FT_, 3); else if (sums) CPE_LAUNCH_VOTE_M(FT_, 1); else CPE_LAUNCH_VOTE_M(FT_, 0)
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
                       uint32_t* votes, uint32_t* acc, long long* sums, uint32_t* pix_cell) {
  return p->dtype == CPE_F32 ? launch_decode_vote_t<float>(st, emb, fg, B, HW, F, p, votes, acc, sums, pix_cell)
                             : launch_decode_vote_t<__half>(st, emb, fg, B, HW, F, p, votes, acc, sums, pix_cell);
}

}  // namespace host
}  // namespace cpe
