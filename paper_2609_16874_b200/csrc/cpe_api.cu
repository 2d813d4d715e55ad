// C ABI of the decoder: argument checks, workspace layout, launch geometry, CUDA-graph and host-buffer
// helpers.  Every entry point that takes a stream only enqueues work.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include "assign.cuh"
#include "cpe.h"
#include "cpe_common.cuh"
#include "instance_masks.cuh"
#include "launch.h"
#include "layout.cuh"

namespace {
thread_local int g_last_cuda = 0;
}

namespace cpe {
namespace host {

int cuda_fail(cudaError_t e) {
  g_last_cuda = (int)e;
  return CPE_ERR_CUDA;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (!cached[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace host
}  // namespace cpe

namespace {

using cpe::host::cuda_fail;
using cpe::host::launch_dependent;
using cpe::host::plain_launch;
using cpe::host::sm_count;

inline size_t elem_size(int dtype) { return dtype == CPE_F32 ? 4 : 2; }

int check_shape(int B, int H, int W, int F, const cpe_params* p) {
  if (!p) return CPE_ERR_NULL;
  if (p->struct_size != sizeof(cpe_params)) return CPE_ERR_PARAM;
  if (p->dtype != CPE_F32 && p->dtype != CPE_F16) return CPE_ERR_DTYPE;
  if (B < 1 || H < 1 || W < 1 || F < 1 || F > 16) return CPE_ERR_SIZE;
  if ((long long)H * W > 0x7fffffffLL || B > 65535) return CPE_ERR_SIZE;
  if (p->bins_w < 1 || p->bins_w > 4096 || p->bins_h < 1 || p->bins_h > 4096) return CPE_ERR_SIZE;
  if (p->vote_threshold < 0 || p->max_instances < 1 || p->max_instances > (1 << 20)) return CPE_ERR_PARAM;
  if (p->levels < 0) return CPE_ERR_PARAM;
  if (p->tau != p->tau) return CPE_ERR_PARAM;  // NaN
  if (p->flags & CPE_FLAG_SOFT_VOTE) {
    if (p->flags & CPE_FLAG_REFINE) return CPE_ERR_PARAM;
    if (!(p->soft_threshold >= 0.0f) || !(p->soft_threshold < INFINITY)) return CPE_ERR_PARAM;
  }
  return CPE_OK;
}

int check_workspace(int B, int H, int W, int F, const cpe_params* p, cpe::Layout* L) {
  int rc = check_shape(B, H, W, F, p);
  if (rc) return rc;
  *L = cpe::make_layout(B, H, W, F, p);
  if (!p->workspace || ((uintptr_t)p->workspace & 255u) || p->workspace_bytes < L->total) return CPE_ERR_WORKSPACE;
  return CPE_OK;
}

template <typename T>
int launch_assign_exact(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                        const float* peak_emb, const int32_t* count, int32_t* labels, float* best, float* second,
                        uint32_t* counters, uint32_t* votes_to_zero, int cells, int k_limit) {
  const T* e = static_cast<const T*>(emb);
  // eight CTAs of 128 threads per SM, shared among the images, walk the pixel blocks
  const long long n_blocks = ((long long)HW + cpe::kAssignThreads - 1) / cpe::kAssignThreads;
  const long long per_image = std::max(1, (8 * sm_count() + B - 1) / B);
  dim3 grid((unsigned)std::min(n_blocks, per_image), (unsigned)B);
#define CPE_LAUNCH_ASSIGN(FT_)                                                                                          \
  CPE_CUDA(launch_dependent(plain_launch(p), cpe::assign_kernel<T, FT_>, grid, cpe::kAssignThreads, 0, st, e, fg, HW, F, \
                            p->max_instances, peak_emb, count, p->tau, labels, best, second, counters, votes_to_zero,   \
                            cells, k_limit))
  switch (F) {
    case 4: CPE_LAUNCH_ASSIGN(4); break;
    case 8: CPE_LAUNCH_ASSIGN(8); break;
    case 16: CPE_LAUNCH_ASSIGN(16); break;
    default: CPE_LAUNCH_ASSIGN(0); break;
  }
#undef CPE_LAUNCH_ASSIGN
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

// What the pruned assignment reads and writes besides the outputs (all inside the workspace).
struct PruneArgs {
  const float* ref_emb = nullptr;
  float* ref2 = nullptr;
  float* cand2 = nullptr;
  uint32_t* nbr = nullptr;
  const int32_t* cell_peak = nullptr;
  const uint32_t* pix_cell = nullptr;
  uint32_t* near_state = nullptr;
  uint32_t* slow_q = nullptr;
  int q_cap = 0;
  int H = 0, W = 0;
  // what the kernel that evaluates gamma of the peaks' mean estimates reads and writes
  const uint32_t* votes = nullptr;
  const long long* sums = nullptr;
  const int32_t* peak_cell = nullptr;
  float* gamma_out = nullptr;       // peak_emb with refined candidates, else ref_emb
  float* out_centroids = nullptr;
  int refine_out = 0;
  const float *pal_w = nullptr, *pal_h = nullptr;
  float* peak_emb = nullptr;
  long long* sums_to_zero = nullptr;   // the list kernel leaves the sums zero for the next decode (NULL: kept)
  void* ref_h = nullptr;
  void* cand_h = nullptr;
  uint32_t* hard_q = nullptr;
};

// Stage 4+5.  The number of peaks is only known on the device, so several kernels are enqueued and every image is
// done by exactly one of them; the CTAs of the others exit at once:
//   - all pairs on the plain ALUs when an image has few peaks (the fixed costs of the others do not pay);
//   - else, with pruning enabled, the kernel that walks per-peak candidate lists (after the kernel that makes them);
//   - else (pruning disabled, or that kernel handed the image on) the tensor-core filtered kernel.
// `ev_lists`: an event recorded between the list kernel and the assignment kernels (per-stage timing).
template <typename T>
int launch_assign(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int HW, int F, const cpe_params* p,
                  const float* peak_emb, const int32_t* count, int32_t* labels, float* best, float* second,
                  uint32_t* counters, uint32_t* status, uint32_t* votes_to_zero, int cells, uint32_t* acc,
                  const PruneArgs* pr, cudaEvent_t ev_lists) {
  if (p->flags & CPE_FLAG_EXACT_ASSIGN) {
    if (ev_lists) CPE_CUDA(cudaEventRecord(ev_lists, st));
    return launch_assign_exact<T>(st, emb, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                  votes_to_zero, cells, 0x7fffffff);
  }
  const int k_limit = cpe::all_pairs_limit(F, p);
  // A caller whose max_instances already is within the all-pairs range needs no second kernel: no image can have
  // more peaks than that (the list is truncated to max_instances), so the chain is shorter.
  if (p->max_instances <= k_limit) {
    if (ev_lists) CPE_CUDA(cudaEventRecord(ev_lists, st));
    return launch_assign_exact<T>(st, emb, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                  votes_to_zero, cells, 0x7fffffff);
  }
  int rc = CPE_OK;
  if (pr) {
    // gamma of every peak's mean estimate (the bounds' reference points; the candidates too when they are refined),
    // a thread per (peak, axis, harmonic) over as many CTAs as the largest image can need
    rc = cpe::host::launch_peak_rows(st, B, F, p, pr->votes, pr->sums, pr->H, pr->W, pr->peak_cell, count, pr->refine_out,
                                     pr->gamma_out, pr->out_centroids, pr->pal_w, pr->pal_h, pr->peak_emb);
    if (rc) return rc;
    rc = cpe::host::launch_peak_graph(st, B, F, p, pr->ref_emb, peak_emb, count, 1, pr->ref2, pr->cand2, pr->ref_h,
                                      pr->cand_h, pr->nbr, pr->sums_to_zero, cells);
    if (rc) return rc;
  }
  if (ev_lists) CPE_CUDA(cudaEventRecord(ev_lists, st));
  if (pr) {
    rc = cpe::host::launch_assign_near(st, emb, fg, B, HW, F, p, pr->ref_emb, peak_emb, pr->ref2, pr->cand2, pr->nbr,
                                       pr->cell_peak, pr->pix_cell, cells, count, labels, best, second, pr->near_state,
                                       1, pr->slow_q, pr->q_cap, status, pr->ref_h, pr->cand_h, pr->hard_q, pr->W);
    if (rc) return rc;
    // The pruned chain serves every image, whatever its number of peaks (an image without any gets its all-zero label
    // map from it): no all-pairs launch.  The filtered kernel follows for the images that were handed on, and it
    // leaves the vote map zero.
    return cpe::host::launch_assign_filtered(st, emb, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                             status, votes_to_zero, cells, 1, acc, pr->near_state);
  }
  // (also with a limit of 0: an image without any peak still gets its all-zero label map from this kernel)
  rc = launch_assign_exact<T>(st, emb, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters, nullptr,
                              cells, k_limit);
  if (rc) return rc;
  return cpe::host::launch_assign_filtered(st, emb, fg, B, HW, F, p, peak_emb, count, labels, best, second, counters,
                                           status, votes_to_zero, cells, k_limit + 1, acc, nullptr);
}

// Debug builds only (-DCPE_DEBUG_SYNC): wait after every stage and name the stage whose kernel failed (never
// inside stream capture).  The product build compiles this to nothing.
int debug_stage_check(cudaStream_t st, const char* stage) {
#ifndef CPE_DEBUG_SYNC
  (void)st;
  (void)stage;
  return CPE_OK;
#else
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone) return CPE_OK;
  cudaError_t e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    fprintf(stderr, "[cpe] stage %s failed: %s\n", stage, cudaGetErrorString(e));
    return cuda_fail(e);
  }
  return CPE_OK;
#endif
}

// The chain.  `ev`, when given, holds CPE_STAGE_N + 1 events recorded around the stages.
int decode_impl(cudaStream_t st, const void* emb, const uint8_t* fg, int B, int H, int W, int F, const cpe_params* p,
                int32_t* out_labels, float* out_centroids, int32_t* out_count, cudaEvent_t* ev) {
  if (!emb || !out_labels || !out_centroids || !out_count) return CPE_ERR_NULL;
  cpe::Layout L;
  int rc = check_workspace(B, H, W, F, p, &L);
  if (rc) return rc;
  if ((uintptr_t)emb % elem_size(p->dtype) || (uintptr_t)out_labels % 4 || (uintptr_t)out_centroids % 4 ||
      (uintptr_t)out_count % 4)
    return CPE_ERR_ALIGN;
  char* ws = static_cast<char*>(p->workspace);
  uint32_t* status = reinterpret_cast<uint32_t*>(ws + L.status);
  uint32_t* counters = reinterpret_cast<uint32_t*>(ws + L.counters);
  uint32_t* votes = reinterpret_cast<uint32_t*>(ws + L.votes);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(ws + L.bitmap);
  int32_t* peak_cell = reinterpret_cast<int32_t*>(ws + L.peak_cell);
  uint32_t* peak_votes = reinterpret_cast<uint32_t*>(ws + L.peak_votes);
  float* peak_emb = reinterpret_cast<float*>(ws + L.peak_emb);
  const float* pal_w = reinterpret_cast<const float*>(ws + L.pal_w);
  const float* pal_h = reinterpret_cast<const float*>(ws + L.pal_h);
  float* best = (p->flags & CPE_FLAG_WRITE_SCORES) ? reinterpret_cast<float*>(ws + L.best) : nullptr;
  float* second = (p->flags & CPE_FLAG_WRITE_SCORES) ? reinterpret_cast<float*>(ws + L.second) : nullptr;
  const int HW = H * W;

  uint32_t* acc = reinterpret_cast<uint32_t*>(ws + L.acc);
  const bool keep_votes = (p->flags & CPE_FLAG_KEEP_VOTES) != 0;

  if (ev) CPE_CUDA(cudaEventRecord(ev[CPE_STAGE_CLEAR], st));
  // Normally the map is already zero (cpe_init_workspace, then the previous decode's last kernel).
  if (keep_votes) CPE_CUDA(cudaMemsetAsync(ws + L.votes, 0, L.votes_end - L.votes, st));
  // The per-bin sums of the refinement: a small map, which one CTA of the peak kernel handles per image, is cleared
  // by that CTA after its last read; otherwise (or when the intermediates are to stay readable) they are cleared here.
  const bool refine = (p->flags & CPE_FLAG_REFINE) != 0;
  long long* sums = (refine || L.prune) ? reinterpret_cast<long long*>(ws + L.sums) : nullptr;
  PruneArgs pr;
  if (L.prune) {
    pr.ref_emb = reinterpret_cast<const float*>(ws + L.ref_emb);
    pr.ref2 = reinterpret_cast<float*>(ws + L.ref2);
    pr.cand2 = reinterpret_cast<float*>(ws + L.cand2);
    pr.nbr = reinterpret_cast<uint32_t*>(ws + L.nbr);
    pr.cell_peak = reinterpret_cast<const int32_t*>(ws + L.cell_peak);
    pr.pix_cell = reinterpret_cast<const uint32_t*>(ws + L.pix_cell);
    pr.near_state = reinterpret_cast<uint32_t*>(ws + L.near_state);
    pr.slow_q = reinterpret_cast<uint32_t*>(ws + L.slow_q);
    pr.q_cap = L.q_cap;
    pr.H = H;
    pr.W = W;
    pr.votes = votes;
    pr.sums = sums;
    pr.peak_cell = peak_cell;
    pr.refine_out = refine ? 1 : 0;
    pr.gamma_out = refine ? peak_emb : reinterpret_cast<float*>(ws + L.ref_emb);
    pr.out_centroids = out_centroids;
    pr.pal_w = pal_w;
    pr.pal_h = pal_h;
    pr.peak_emb = peak_emb;
    pr.sums_to_zero = keep_votes ? nullptr : sums;
    pr.hard_q = reinterpret_cast<uint32_t*>(ws + L.hard_q);
    pr.ref_h = ws + L.ref_h;
    pr.cand_h = ws + L.cand_h;
  }
  const bool one_peak_cta = L.words <= cpe::kPeakStageWords;
  // (with the pruned assignment the sums are read by a later kernel: they are cleared at the start instead)
  const bool sums_cleared_by_peaks = sums && one_peak_cta && !keep_votes && !L.prune;
  const bool sums_cleared_by_lists = sums && L.prune && !keep_votes;
  if (sums && !sums_cleared_by_peaks && !sums_cleared_by_lists)
    CPE_CUDA(cudaMemsetAsync(ws + L.sums, 0, L.sums_end - L.sums, st));

  if (ev) CPE_CUDA(cudaEventRecord(ev[CPE_STAGE_DECODE_VOTE], st));
  // From here on the vote map and the accumulators may hold this decode's votes.  If a later enqueue fails, the
  // kernel that would have left them zero for the next decode never runs: clear them here instead.
  auto fail_after_votes = [&](int code) {
    cudaMemsetAsync(ws + L.acc, 0, L.votes_end - L.acc, st);
    if (sums) cudaMemsetAsync(ws + L.sums, 0, L.sums_end - L.sums, st);
    return code;
  };
  // Stage 3's arguments (the voting kernel takes them along when it runs the search itself)
  cpe::PeakArgs pk{};
  pk.votes = votes;
  pk.bins_w = p->bins_w;
  pk.bins_h = p->bins_h;
  pk.words = L.words;
  pk.bitmap = bitmap;
  pk.K_max = p->max_instances;
  pk.F = F;
  pk.H = H;
  pk.W = W;
  pk.pal_w = pal_w;
  pk.pal_h = pal_h;
  pk.peak_cell = peak_cell;
  pk.peak_votes = peak_votes;
  pk.peak_emb = peak_emb;
  pk.out_centroids = out_centroids;
  pk.out_count = out_count;
  pk.acc = acc;
  pk.counters = counters;
  pk.status = status;
  pk.sums = L.prune ? nullptr : sums;
  pk.zero_sums = sums_cleared_by_peaks ? 1 : 0;
  pk.staged = one_peak_cta ? 1 : 0;
  pk.refine_out = refine ? 1 : 0;
  pk.skip_rows = L.prune ? 1 : 0;
  pk.ref_emb = L.prune ? reinterpret_cast<float*>(ws + L.ref_emb) : nullptr;
  pk.cell_peak = L.prune ? reinterpret_cast<int32_t*>(ws + L.cell_peak) : nullptr;
  pk.near_state = pr.near_state;
  // Vote: by default the hard vote (each pixel's centroid estimate, one count).  With CPE_FLAG_SOFT_VOTE the map holds
  // the binary32 histogram of Eq. 6 instead: non-negative binary32 values order like their bit patterns and 0.0f is
  // all-zero bits, so the zeroing conventions and the peak kernel's comparisons carry over to it unchanged.
  const bool soft = (p->flags & CPE_FLAG_SOFT_VOTE) != 0;
  pk.T_v = (uint32_t)p->vote_threshold;
  pk.strict = soft ? 1 : 0;
  bool peaks_done = false;
  if (soft) {
    if ((uintptr_t)emb % 16 || HW % 8) return CPE_ERR_ALIGN;
    memcpy(&pk.T_v, &p->soft_threshold, sizeof pk.T_v);
    // the soft-vote kernel only ever ORs into the status words; the peak kernel then ORs too
    CPE_CUDA(cudaMemsetAsync(status, 0, sizeof(uint32_t) * (size_t)B, st));
    rc = cpe::host::launch_soft_votes(st, emb, fg, B, HW, F, p, pal_w, pal_h, reinterpret_cast<float*>(votes), status, acc);
  } else {
    // small maps without the pruned chain: the voting kernel's last CTA of an image searches the map itself
    peaks_done = one_peak_cta && !L.prune && cpe::host::vote_can_fuse_peaks(B, HW, L.words, p);
    rc = cpe::host::launch_decode_vote(st, emb, fg, B, HW, F, p, votes, acc, sums,
                                       L.prune ? reinterpret_cast<uint32_t*>(ws + L.pix_cell) : nullptr,
                                       peaks_done ? &pk : nullptr);
  }
  if (rc) return fail_after_votes(rc);
  if ((rc = debug_stage_check(st, "decode_vote"))) return rc;

  if (ev) CPE_CUDA(cudaEventRecord(ev[CPE_STAGE_PEAKS], st));
  if (!peaks_done) {
    rc = cpe::host::launch_peaks(st, B, p, pk);
    if (rc) return fail_after_votes(rc);
  }
  if ((rc = debug_stage_check(st, "peaks"))) return rc;
  if (ev) CPE_CUDA(cudaEventRecord(ev[CPE_STAGE_LISTS], st));
  uint32_t* votes_to_zero = keep_votes ? nullptr : votes;
  const PruneArgs* prp = L.prune ? &pr : nullptr;
  cudaEvent_t ev_lists = ev ? ev[CPE_STAGE_ASSIGN] : nullptr;
  rc = p->dtype == CPE_F32 ? launch_assign<float>(st, emb, fg, B, HW, F, p, peak_emb, out_count, out_labels, best, second,
                                                  counters, status, votes_to_zero, L.cells, acc, prp, ev_lists)
                           : launch_assign<__half>(st, emb, fg, B, HW, F, p, peak_emb, out_count, out_labels, best,
                                                   second, counters, status, votes_to_zero, L.cells, acc, prp, ev_lists);
  if (rc) return fail_after_votes(rc);
  if ((rc = debug_stage_check(st, "assign"))) return rc;
  if (ev) CPE_CUDA(cudaEventRecord(ev[CPE_STAGE_N], st));
  return CPE_OK;
}

}  // namespace

struct cpe_graph {
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  int kernel_nodes = 0;
};

struct HostSlot {
  cpe_params params{};
  cudaStream_t stream = nullptr;
  void* d_emb = nullptr;
  uint8_t* d_fg = nullptr;
  int32_t* d_labels = nullptr;
  float* d_centroids = nullptr;
  int32_t* d_count = nullptr;
  void* d_ws = nullptr;
  cpe_graph* graph = nullptr;
};

// Two slots, each with its own stream, device buffers, workspace and captured graph: while one slot's decode and
// read-back run, the other slot's inputs are already on their way to the device.
struct cpe_host_ctx {
  int B = 0, H = 0, W = 0, F = 0, has_mask = 0;
  HostSlot slot[2];
  unsigned submitted = 0, waited = 0;     // calls so far; submitted - waited <= 2 are in flight
  size_t emb_bytes = 0, fg_bytes = 0, labels_bytes = 0, centroids_bytes = 0, count_bytes = 0;
};

extern "C" {

size_t cpe_workspace_size(int B, int H, int W, int F, const cpe_params* params) {
  if (check_shape(B, H, W, F, params) != CPE_OK) return 0;
  return cpe::make_layout(B, H, W, F, params).total;
}

int cpe_init_workspace(cpe_stream_t stream, int B, int H, int W, int F, const cpe_params* params) {
  cpe::Layout L;
  int rc = check_workspace(B, H, W, F, params, &L);
  if (rc) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(params->workspace);
  CPE_CUDA(cudaMemsetAsync(ws, 0, L.total, st));
  // Eq. 9 positions through Eq. 2, evaluated in double and rounded once to binary32.
  const double pi = 3.14159265358979323846;
  for (int axis = 0; axis < 2; ++axis) {
    const int n = axis == 0 ? params->bins_w : params->bins_h;
    std::vector<float> pal((size_t)n * 2 * F);
    for (int i = 1; i <= n; ++i) {
      const double pos = -1.0 + 2.0 * (double)i / (double)(n + 1);
      for (int l = 0; l < F; ++l) {
        const double arg = pi * ldexp(1.0, l) * pos;
        pal[(size_t)(i - 1) * 2 * F + 2 * l] = (float)sin(arg);
        pal[(size_t)(i - 1) * 2 * F + 2 * l + 1] = (float)cos(arg);
      }
    }
    // pageable source: the runtime stages the data before returning, so `pal` may go out of scope
    CPE_CUDA(cudaMemcpyAsync(ws + (axis == 0 ? L.pal_w : L.pal_h), pal.data(), pal.size() * sizeof(float),
                             cudaMemcpyHostToDevice, st));
    CPE_CUDA(cudaStreamSynchronize(st));
  }
  return CPE_OK;
}

int cpe_decode(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
               const cpe_params* params, int32_t* out_labels, float* out_centroids, int32_t* out_count) {
  return decode_impl(reinterpret_cast<cudaStream_t>(stream), emb, fg_mask, B, H, W, F, params, out_labels,
                     out_centroids, out_count, nullptr);
}

int cpe_get_intermediate(const cpe_params* params, int which, int B, int H, int W, int F, void** device_ptr,
                         size_t* bytes) {
  if (!device_ptr || !bytes) return CPE_ERR_NULL;
  cpe::Layout L;
  int rc = check_workspace(B, H, W, F, params, &L);
  if (rc) return rc;
  const size_t Kmax = (size_t)params->max_instances, HW = (size_t)H * W;
  size_t off = 0, sz = 0;
  switch (which) {
    case CPE_INT_VOTES:
      if (!(params->flags & CPE_FLAG_KEEP_VOTES)) return CPE_ERR_WHICH;
      off = L.votes;
      sz = 4 * (size_t)L.cells * B;
      break;
    case CPE_INT_PEAK_CELLS: off = L.peak_cell; sz = 4 * Kmax * B; break;
    case CPE_INT_PEAK_VOTES: off = L.peak_votes; sz = 4 * Kmax * B; break;
    case CPE_INT_PEAK_EMB: off = L.peak_emb; sz = 4 * Kmax * 4 * F * B; break;
    case CPE_INT_PALETTE_W: off = L.pal_w; sz = 4 * (size_t)params->bins_w * 2 * F; break;
    case CPE_INT_PALETTE_H: off = L.pal_h; sz = 4 * (size_t)params->bins_h * 2 * F; break;
    case CPE_INT_BEST_SCORE:
    case CPE_INT_SECOND_SCORE:
      if (!(params->flags & CPE_FLAG_WRITE_SCORES)) return CPE_ERR_WHICH;
      off = which == CPE_INT_BEST_SCORE ? L.best : L.second;
      sz = 4 * HW * B;
      break;
    case CPE_INT_STATUS: off = L.status; sz = 4 * (size_t)B; break;
    case CPE_INT_COUNTERS: off = L.counters; sz = 4 * (size_t)CPE_CNT_N * B; break;
    case CPE_INT_VOTE_SUMS:
      if (!(params->flags & CPE_FLAG_REFINE) || !(params->flags & CPE_FLAG_KEEP_VOTES)) return CPE_ERR_WHICH;
      off = L.sums;
      sz = 16 * (size_t)L.cells * B;
      break;
    case CPE_INT_PRUNE_STATE:
      if (!L.prune) return CPE_ERR_WHICH;
      off = L.near_state;
      sz = 4 * (size_t)cpe::kNearStride * B;
      break;
    default: return CPE_ERR_WHICH;
  }
  *device_ptr = static_cast<char*>(params->workspace) + off;
  *bytes = sz;
  return CPE_OK;
}

const char* cpe_strerror(int code) {
  switch (code) {
    case CPE_OK: return "ok";
    case CPE_ERR_NULL: return "a required pointer is NULL";
    case CPE_ERR_SIZE: return "a size is out of range (B, H, W >= 1; 1 <= F <= 16; 1 <= bins <= 4096)";
    case CPE_ERR_DTYPE: return "unknown element type";
    case CPE_ERR_ALIGN: return "a buffer is not aligned to its element size";
    case CPE_ERR_WORKSPACE: return "workspace missing, not 256-byte aligned, or too small";
    case CPE_ERR_PARAM: return "invalid cpe_params (struct_size, threshold, max_instances, levels or tau)";
    case CPE_ERR_CUDA: return "a CUDA runtime call failed";
    case CPE_ERR_WHICH: return "unknown or unavailable intermediate";
    case CPE_ERR_NOMEM: return "allocation failed";
    case CPE_ERR_STATIC_LIMIT: return "the problem needs more scratch (or more bins) than cpe_decode_static provides";
    case CPE_ERR_BUSY: return "the host front end already has its two calls in flight";
    default: return "unknown error code";
  }
}

int cpe_last_cuda_error(void) { return g_last_cuda; }

// ------------------------------------------------------------------------------------ graph helper

int cpe_graph_create(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
                     const cpe_params* params, int32_t* out_labels, float* out_centroids, int32_t* out_count,
                     cpe_graph** out_graph) {
  if (!out_graph) return CPE_ERR_NULL;
  *out_graph = nullptr;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cpe_graph* g = new (std::nothrow) cpe_graph();
  if (!g) return CPE_ERR_NOMEM;
  cudaError_t e = cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal);
  if (e != cudaSuccess) { delete g; return cuda_fail(e); }
  int rc = decode_impl(st, emb, fg_mask, B, H, W, F, params, out_labels, out_centroids, out_count, nullptr);
  e = cudaStreamEndCapture(st, &g->graph);
  if (rc != CPE_OK || e != cudaSuccess) {
    if (g->graph) cudaGraphDestroy(g->graph);
    delete g;
    return rc != CPE_OK ? rc : cuda_fail(e);
  }
  e = cudaGraphInstantiate(&g->exec, g->graph, 0);
  if (e != cudaSuccess) { cudaGraphDestroy(g->graph); delete g; return cuda_fail(e); }
  size_t n = 0;
  if (cudaGraphGetNodes(g->graph, nullptr, &n) == cudaSuccess && n) {
    std::vector<cudaGraphNode_t> nodes(n);
    if (cudaGraphGetNodes(g->graph, nodes.data(), &n) == cudaSuccess) {
      for (size_t i = 0; i < n; ++i) {
        cudaGraphNodeType t;
        if (cudaGraphNodeGetType(nodes[i], &t) == cudaSuccess && t == cudaGraphNodeTypeKernel) ++g->kernel_nodes;
      }
    }
  }
  *out_graph = g;
  return CPE_OK;
}

int cpe_graph_launch(cpe_graph* graph, cpe_stream_t stream) {
  if (!graph || !graph->exec) return CPE_ERR_NULL;
  CPE_CUDA(cudaGraphLaunch(graph->exec, reinterpret_cast<cudaStream_t>(stream)));
  return CPE_OK;
}

void cpe_graph_destroy(cpe_graph* graph) {
  if (!graph) return;
  if (graph->exec) cudaGraphExecDestroy(graph->exec);
  if (graph->graph) cudaGraphDestroy(graph->graph);
  delete graph;
}

int cpe_graph_kernel_nodes(const cpe_graph* graph) { return graph ? graph->kernel_nodes : 0; }

// ------------------------------------------------------------------------------------ per-stage timing

int cpe_profile_decode(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
                       const cpe_params* params, int32_t* out_labels, float* out_centroids, int32_t* out_count,
                       int iters, float* stage_ms) {
  if (!stage_ms) return CPE_ERR_NULL;
  if (iters < 1) return CPE_ERR_SIZE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int per = CPE_STAGE_N + 1;
  std::vector<cudaEvent_t> ev((size_t)iters * per, nullptr);
  int rc = CPE_OK;
  for (auto& x : ev) {
    cudaError_t e = cudaEventCreate(&x);
    if (e != cudaSuccess) { rc = cuda_fail(e); break; }
  }
  for (int it = 0; rc == CPE_OK && it < iters; ++it)
    rc = decode_impl(st, emb, fg_mask, B, H, W, F, params, out_labels, out_centroids, out_count, &ev[(size_t)it * per]);
  if (rc == CPE_OK) {
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) rc = cuda_fail(e);
  }
  if (rc == CPE_OK) {
    for (int s = 0; s < CPE_STAGE_N; ++s) {
      double sum = 0.0;
      for (int it = 0; it < iters; ++it) {
        float ms = 0.0f;
        cudaEventElapsedTime(&ms, ev[(size_t)it * per + s], ev[(size_t)it * per + s + 1]);
        sum += ms;
      }
      stage_ms[s] = (float)(sum / iters);
    }
  }
  for (auto& x : ev)
    if (x) cudaEventDestroy(x);
  return rc;
}

// ------------------------------------------------------------------------------------ host-buffer front end

void cpe_host_ctx_destroy(cpe_host_ctx* c) {
  if (!c) return;
  for (HostSlot& sl : c->slot) {
    if (sl.stream) cudaStreamSynchronize(sl.stream);
    if (sl.graph) cpe_graph_destroy(sl.graph);
    cudaFree(sl.d_emb);
    cudaFree(sl.d_fg);
    cudaFree(sl.d_labels);
    cudaFree(sl.d_centroids);
    cudaFree(sl.d_count);
    cudaFree(sl.d_ws);
    if (sl.stream) cudaStreamDestroy(sl.stream);
  }
  delete c;
}

int cpe_host_ctx_create(int B, int H, int W, int F, const cpe_params* params, int has_mask, cpe_host_ctx** out_ctx) {
  if (!out_ctx) return CPE_ERR_NULL;
  *out_ctx = nullptr;
  int rc = check_shape(B, H, W, F, params);
  if (rc) return rc;
  cpe_host_ctx* c = new (std::nothrow) cpe_host_ctx();
  if (!c) return CPE_ERR_NOMEM;
  c->B = B; c->H = H; c->W = W; c->F = F; c->has_mask = has_mask ? 1 : 0;
  const size_t HW = (size_t)H * W;
  c->emb_bytes = (size_t)B * 4 * F * HW * elem_size(params->dtype);
  c->fg_bytes = has_mask ? (size_t)B * HW : 0;
  c->labels_bytes = (size_t)B * HW * 4;
  c->centroids_bytes = (size_t)B * params->max_instances * 2 * 4;
  c->count_bytes = (size_t)B * 4;
  for (HostSlot& sl : c->slot) {
    sl.params = *params;
    sl.params.workspace_bytes = cpe::make_layout(B, H, W, F, params).total;
    cudaError_t e = cudaStreamCreateWithFlags(&sl.stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaMalloc(&sl.d_emb, c->emb_bytes);
    if (e == cudaSuccess && has_mask) e = cudaMalloc((void**)&sl.d_fg, c->fg_bytes);
    if (e == cudaSuccess) e = cudaMalloc((void**)&sl.d_labels, c->labels_bytes);
    if (e == cudaSuccess) e = cudaMalloc((void**)&sl.d_centroids, c->centroids_bytes);
    if (e == cudaSuccess) e = cudaMalloc((void**)&sl.d_count, c->count_bytes);
    if (e == cudaSuccess) e = cudaMalloc(&sl.d_ws, sl.params.workspace_bytes);
    if (e != cudaSuccess) {
      cuda_fail(e);
      cpe_host_ctx_destroy(c);
      return e == cudaErrorMemoryAllocation ? CPE_ERR_NOMEM : CPE_ERR_CUDA;
    }
    sl.params.workspace = sl.d_ws;
    cpe_stream_t s = reinterpret_cast<cpe_stream_t>(sl.stream);
    rc = cpe_init_workspace(s, B, H, W, F, &sl.params);
    if (rc == CPE_OK && cudaMemsetAsync(sl.d_centroids, 0, c->centroids_bytes, sl.stream) != cudaSuccess) rc = CPE_ERR_CUDA;
    if (rc == CPE_OK)
      rc = cpe_graph_create(s, sl.d_emb, sl.d_fg, B, H, W, F, &sl.params, sl.d_labels, sl.d_centroids, sl.d_count,
                            &sl.graph);
    if (rc != CPE_OK) { cpe_host_ctx_destroy(c); return rc; }
  }
  *out_ctx = c;
  return CPE_OK;
}

int cpe_host_submit(cpe_host_ctx* c, const void* emb_host, const uint8_t* fg_mask_host, int32_t* labels_host,
                    float* centroids_host, int32_t* count_host) {
  if (!c || !emb_host || !labels_host || !centroids_host || !count_host) return CPE_ERR_NULL;
  if (c->has_mask && !fg_mask_host) return CPE_ERR_NULL;
  if (c->submitted - c->waited >= 2u) return CPE_ERR_BUSY;
  HostSlot& sl = c->slot[c->submitted & 1u];
  CPE_CUDA(cudaMemcpyAsync(sl.d_emb, emb_host, c->emb_bytes, cudaMemcpyHostToDevice, sl.stream));
  if (c->has_mask) CPE_CUDA(cudaMemcpyAsync(sl.d_fg, fg_mask_host, c->fg_bytes, cudaMemcpyHostToDevice, sl.stream));
  int rc = cpe_graph_launch(sl.graph, reinterpret_cast<cpe_stream_t>(sl.stream));
  if (rc) return rc;
  CPE_CUDA(cudaMemcpyAsync(labels_host, sl.d_labels, c->labels_bytes, cudaMemcpyDeviceToHost, sl.stream));
  CPE_CUDA(cudaMemcpyAsync(centroids_host, sl.d_centroids, c->centroids_bytes, cudaMemcpyDeviceToHost, sl.stream));
  CPE_CUDA(cudaMemcpyAsync(count_host, sl.d_count, c->count_bytes, cudaMemcpyDeviceToHost, sl.stream));
  ++c->submitted;
  return CPE_OK;
}

int cpe_host_wait(cpe_host_ctx* c) {
  if (!c) return CPE_ERR_NULL;
  if (c->submitted == c->waited) return CPE_ERR_PARAM;
  HostSlot& sl = c->slot[c->waited & 1u];
  ++c->waited;
  CPE_CUDA(cudaStreamSynchronize(sl.stream));
  return CPE_OK;
}

int cpe_host_decode(cpe_host_ctx* c, const void* emb_host, const uint8_t* fg_mask_host, int32_t* labels_host,
                    float* centroids_host, int32_t* count_host) {
  if (!c) return CPE_ERR_NULL;
  if (c->submitted != c->waited) return CPE_ERR_BUSY;
  int rc = cpe_host_submit(c, emb_host, fg_mask_host, labels_host, centroids_host, count_host);
  if (rc) return rc;
  return cpe_host_wait(c);
}

int cpe_host_ctx_traffic(const cpe_host_ctx* c, size_t* h2d_bytes, size_t* d2h_bytes) {
  if (!c || !h2d_bytes || !d2h_bytes) return CPE_ERR_NULL;
  *h2d_bytes = c->emb_bytes + c->fg_bytes;
  *d2h_bytes = c->labels_bytes + c->centroids_bytes + c->count_bytes;
  return CPE_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------ decode without allocation

// The scratch of cpe_decode_static lives in the library image.  In host code this name is only a handle for
// cudaGetSymbolAddress: it is not a device address and must never be handed to a kernel as one.
static __device__ __align__(256) unsigned char g_static_scratch[CPE_STATIC_SCRATCH_BYTES];

namespace {

struct StaticSlot {
  void* ptr = nullptr;                 // device address of g_static_scratch on this device
  int F = 0, bins_w = 0, bins_h = 0;   // palettes currently uploaded ...
  size_t off_w = 0, off_h = 0;         // ... and where (the layout moves with B, bins and max_instances)
};
StaticSlot g_static_slot[64];
// host staging for one palette: static storage, so the set-up allocates nothing either
float g_static_palette[CPE_STATIC_MAX_BINS * 32];
std::mutex g_static_mutex;

}  // namespace

extern "C" int cpe_decode_static(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W,
                                 int F, const cpe_params* params, int32_t* out_labels, float* out_centroids,
                                 int32_t* out_count) {
  int rc = check_shape(B, H, W, F, params);
  if (rc) return rc;
  if (!emb || !out_labels || !out_centroids || !out_count) return CPE_ERR_NULL;
  cpe_params p = *params;
  if (p.flags & CPE_FLAG_WRITE_SCORES) return CPE_ERR_STATIC_LIMIT;
  p.flags |= CPE_FLAG_KEEP_VOTES;   // the vote map is cleared at the start of every call instead of at the end
  p.flags |= CPE_FLAG_NO_PRUNE;     // the pruned assignment keeps per-pixel scratch, which the built-in array has no room for
  p.workspace = nullptr;
  p.workspace_bytes = 0;
  const cpe::Layout L = cpe::make_layout(B, H, W, F, &p);
  if (L.total > (size_t)CPE_STATIC_SCRATCH_BYTES || p.bins_w > CPE_STATIC_MAX_BINS || p.bins_h > CPE_STATIC_MAX_BINS)
    return CPE_ERR_STATIC_LIMIT;

  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int dev = 0;
  CPE_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return CPE_ERR_SIZE;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticSlot& slot = g_static_slot[dev];
  if (!slot.ptr) {
    // once per device, with that device current: the device address behind the symbol
    void* ptr = nullptr;
    CPE_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
    slot.ptr = ptr;
  }
  char* ws = static_cast<char*>(slot.ptr);
  if (slot.F != F || slot.bins_w != p.bins_w || slot.bins_h != p.bins_h || slot.off_w != L.pal_w ||
      slot.off_h != L.pal_h) {
    // the set-up copies from a host staging buffer and waits for the stream: impossible while the stream is being
    // captured (the wait would invalidate the capture), so such a call is refused and enqueues nothing
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    CPE_CUDA(cudaStreamIsCapturing(st, &cs));
    if (cs != cudaStreamCaptureStatusNone) return CPE_ERR_PARAM;
    // Eq. 9 positions through Eq. 2, in double, rounded once to binary32 (as cpe_init_workspace does)
    const double pi = 3.14159265358979323846;
    for (int axis = 0; axis < 2; ++axis) {
      const int n = axis == 0 ? p.bins_w : p.bins_h;
      for (int i = 1; i <= n; ++i) {
        const double pos = -1.0 + 2.0 * (double)i / (double)(n + 1);
        for (int l = 0; l < F; ++l) {
          const double arg = pi * ldexp(1.0, l) * pos;
          g_static_palette[(size_t)(i - 1) * 2 * F + 2 * l] = (float)sin(arg);
          g_static_palette[(size_t)(i - 1) * 2 * F + 2 * l + 1] = (float)cos(arg);
        }
      }
      CPE_CUDA(cudaMemcpyAsync(ws + (axis == 0 ? L.pal_w : L.pal_h), g_static_palette,
                               sizeof(float) * (size_t)n * 2 * F, cudaMemcpyHostToDevice, st));
      CPE_CUDA(cudaStreamSynchronize(st));   // the staging buffer is reused for the other axis
    }
    slot.F = F;
    slot.bins_w = p.bins_w;
    slot.bins_h = p.bins_h;
    slot.off_w = L.pal_w;
    slot.off_h = L.pal_h;
  }
  // what must start at zero: the voting accumulators and the peak kernel's ticket (the vote map is cleared by
  // the decode itself because of CPE_FLAG_KEEP_VOTES); an earlier call with other sizes may have left anything
  CPE_CUDA(cudaMemsetAsync(ws + L.acc, 0, L.votes - L.acc, st));
  p.workspace = slot.ptr;
  p.workspace_bytes = CPE_STATIC_SCRATCH_BYTES;
  return decode_impl(st, emb, fg_mask, B, H, W, F, &p, out_labels, out_centroids, out_count, nullptr);
}

namespace cpe {
// Self-test of div2_half_operands: CTA i takes the denominator with binary16 bit pattern i (0 .. 0x7bff: zero and every
// positive finite value), its threads all numerators up to it; counts the results whose bits differ from __fdiv_rn's.
__global__ void half_division_selftest_kernel(unsigned long long* __restrict__ mismatches) {
  const uint32_t bi = blockIdx.x;
  if (bi > 0x7bffu) return;
  const float floor_b = 9.31322574615478515625e-10f;
  const float b = fmaxf(__half2float(__ushort_as_half((unsigned short)bi)), floor_b);
  unsigned long long n = 0;
  for (uint32_t ai = 2 * threadIdx.x; ai <= bi; ai += 2 * blockDim.x) {
    const float a0 = __half2float(__ushort_as_half((unsigned short)ai));
    const float a1 = __half2float(__ushort_as_half((unsigned short)min(ai + 1u, bi)));
    const float2 got = div2_half_operands(make_float2(a0, a1), make_float2(b, b));
    n += __float_as_uint(got.x) != __float_as_uint(__fdiv_rn(a0, b));
    n += __float_as_uint(got.y) != __float_as_uint(__fdiv_rn(a1, b));
  }
  if (n) atomicAdd(mismatches, n);
}
}  // namespace cpe

extern "C" int cpe_selftest_half_division(cpe_stream_t stream, unsigned long long* out_mismatches) {
  if (!out_mismatches) return CPE_ERR_NULL;
  if ((uintptr_t)out_mismatches % 8) return CPE_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  CPE_CUDA(cudaMemsetAsync(out_mismatches, 0, sizeof(unsigned long long), st));
  cpe::half_division_selftest_kernel<<<0x7c00, 256, 0, st>>>(out_mismatches);
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

extern "C" int cpe_soft_votes(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
                   const cpe_params* params, float* out_hist) {
  if (!emb || !out_hist) return CPE_ERR_NULL;
  cpe::Layout L;
  int rc = check_workspace(B, H, W, F, params, &L);
  if (rc) return rc;
  const long long HW = (long long)H * W;
  if ((uintptr_t)emb % 16 || HW % 8 || (uintptr_t)out_hist % 4) return CPE_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(params->workspace);
  const float* pal_w = reinterpret_cast<const float*>(ws + L.pal_w);
  const float* pal_h = reinterpret_cast<const float*>(ws + L.pal_h);
  uint32_t* status = reinterpret_cast<uint32_t*>(ws + L.status);
  CPE_CUDA(cudaMemsetAsync(out_hist, 0, sizeof(float) * (size_t)B * params->bins_w * params->bins_h, st));
  return cpe::host::launch_soft_votes(st, emb, fg_mask, B, (int)HW, F, params, pal_w, pal_h, out_hist, status, nullptr);
}

extern "C" int cpe_instance_masks(cpe_stream_t stream, const int32_t* labels, int B, int H, int W, int n_planes,
                                  uint8_t* out_planes, uint32_t* out_pixels) {
  if (!labels || (!out_planes && !out_pixels)) return CPE_ERR_NULL;
  if (B < 1 || H < 1 || W < 1 || n_planes < 1 || n_planes > 8191 || (long long)H * W > 0x7fffffffLL) return CPE_ERR_SIZE;
  if ((uintptr_t)labels % 4 || (uintptr_t)out_pixels % 4) return CPE_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int HW = H * W;
  if (out_pixels) CPE_CUDA(cudaMemsetAsync(out_pixels, 0, sizeof(uint32_t) * (size_t)B * n_planes, st));
  // 128-bit accesses need aligned rows of every image and plane
  const int vec = ((uintptr_t)labels % 16 == 0) && (HW % 16 == 0) && (!out_planes || (uintptr_t)out_planes % 16 == 0);
  const long long n_chunks = ((long long)HW + cpe::kImPixels - 1) / cpe::kImPixels;
  const long long ctas = (n_chunks + cpe::kImThreads - 1) / cpe::kImThreads;
  const long long per_image = std::max(1, (8 * sm_count() + B - 1) / B);
  dim3 grid((unsigned)std::min(ctas, per_image), (unsigned)B);
  const size_t smem = out_pixels ? sizeof(uint32_t) * (size_t)(n_planes + 1) : 0;
  cpe::instance_masks_kernel<<<grid, cpe::kImThreads, smem, st>>>(labels, HW, n_planes, vec, out_planes, out_pixels);
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}

extern "C" int cpe_channels_last_to_planar(cpe_stream_t stream, const void* emb_nhwc, void* emb_planar, int B, int H,
                                           int W, int F, int dtype) {
  if (!emb_nhwc || !emb_planar) return CPE_ERR_NULL;
  if (B < 1 || H < 1 || W < 1 || F < 1 || F > 16 || (long long)H * W > 0x7fffffffLL) return CPE_ERR_SIZE;
  if (dtype != CPE_F32 && dtype != CPE_F16) return CPE_ERR_DTYPE;
  const size_t esz = dtype == CPE_F32 ? 4 : 2;
  if ((uintptr_t)emb_nhwc % esz || (uintptr_t)emb_planar % esz) return CPE_ERR_ALIGN;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int HW = H * W, D = 4 * F;
  dim3 grid((unsigned)((HW + cpe::kLyPixels - 1) / cpe::kLyPixels), (unsigned)B);
  const size_t smem = (size_t)cpe::kLyPixels * (D + 1) * esz;
  // 128-bit accesses: every tile of the source starts on a 16-byte boundary iff 128 * D * esz does (always) and the
  // base does; a plane piece does iff the base, the plane pitch H * W and the tile start are multiples of 16 bytes
  const int vec_in = (uintptr_t)emb_nhwc % 16 == 0 && ((size_t)HW * D * esz) % 16 == 0;
  const int vec_out = (uintptr_t)emb_planar % 16 == 0 && ((size_t)HW * esz) % 16 == 0;
  // aligned inputs with whole tiles and a power-of-two number of 4-channel units take the unit-wise kernels
  const int U = D / 4;
  const bool pow2_units = (U & (U - 1)) == 0;
  if (vec_in && vec_out && pow2_units && dtype == CPE_F16 && U >= 2 && HW % cpe::kLyFastPixels16 == 0) {
    dim3 g((unsigned)(HW / cpe::kLyFastPixels16), (unsigned)B);
    cpe::channels_last_to_planar_f16_kernel<<<g, cpe::kLyThreads, (size_t)cpe::kLyFastPixels16 * D * 2, st>>>(
        static_cast<const uint16_t*>(emb_nhwc), static_cast<uint16_t*>(emb_planar), HW, D);
    CPE_CUDA(cudaGetLastError());
    return CPE_OK;
  }
  if (vec_in && vec_out && pow2_units && dtype == CPE_F32 && HW % cpe::kLyFastPixels32 == 0) {
    dim3 g((unsigned)(HW / cpe::kLyFastPixels32), (unsigned)B);
    cpe::channels_last_to_planar_f32_kernel<<<g, cpe::kLyThreads, (size_t)cpe::kLyFastPixels32 * D * 4, st>>>(
        static_cast<const float*>(emb_nhwc), static_cast<float*>(emb_planar), HW, D);
    CPE_CUDA(cudaGetLastError());
    return CPE_OK;
  }
  if (dtype == CPE_F32)
    cpe::channels_last_to_planar_kernel<float><<<grid, cpe::kLyThreads, smem, st>>>(
        static_cast<const float*>(emb_nhwc), static_cast<float*>(emb_planar), HW, D, vec_in, vec_out);
  else
    cpe::channels_last_to_planar_kernel<__half><<<grid, cpe::kLyThreads, smem, st>>>(
        static_cast<const __half*>(emb_nhwc), static_cast<__half*>(emb_planar), HW, D, vec_in, vec_out);
  CPE_CUDA(cudaGetLastError());
  return CPE_OK;
}
