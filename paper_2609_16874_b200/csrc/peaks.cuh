// Stage 3: local-maximum test over the vote map (Sec. 3.2, "Local Maxima Search") and ordered
// compaction of the peaks into a device-side list, with centroids and peak embeddings - one kernel.
#pragma once

#include "cpe_common.cuh"

namespace cpe {

constexpr int kPeakThreads = 1024;   // wide CTAs: the last one of an image does the whole compaction
constexpr int kRefineChunk = 512;     // peaks whose refined positions are staged in shared memory at a time
constexpr int kPeakListStage = 1024;  // peak-list entries mirrored in shared memory when one CTA does the image

// Mean estimate of a peak on one axis, pooled over the 3x3 window of bins around it (`lin` is the peak's bin): the sum of
// the fixed-point sums over 2^24 times the sum of the counts, in binary64.  `vote_at(i)` reads the count of bin i.
template <typename VoteAt>
__device__ __forceinline__ double window_mean(VoteAt vote_at, const long long* __restrict__ S, int lin, int bins_w,
                                              int bins_h, int axis) {
  const int cy = lin / bins_w, cx = lin - cy * bins_w;
  long long s = 0, n = 0;
#pragma unroll
  for (int dy = -1; dy <= 1; ++dy) {
#pragma unroll
    for (int dx = -1; dx <= 1; ++dx) {
      const int ny = cy + dy, nx = cx + dx;
      if (ny < 0 || ny >= bins_h || nx < 0 || nx >= bins_w) continue;
      const int nlin = ny * bins_w + nx;
      n += (long long)vote_at(nlin);
      s += __ldcg(S + 2 * (size_t)nlin + axis);
    }
  }
  return __ddiv_rn((double)s, __dmul_rn((double)n, 16777216.0));
}
// The refined centroid in pixel units: pixel centres sit at x = -1 + (2 col + 1) / W.
__device__ __forceinline__ float mean_to_pixels(double m, int extent) {
  return (float)__dmul_rn(__dadd_rn(__dmul_rn(__dadd_rn(m, 1.0), (double)extent), -1.0), 0.5);
}

// Phase 1 (every CTA): one thread per bin, one warp per 32 consecutive bins; the warp's ballot is one word
// of the peak indicator bitmap (the paper's binary map H-bar, packed).  A bin is a peak iff V > T_v and it
// beats each existing 8-neighbour: larger count, or equal count and lower linear index.
//
// `strict` (the soft vote's real-valued map, whose non-negative binary32 values are compared through their bit
// patterns): the test as the paper prints it, a bin must exceed every existing neighbour; equal neighbours are both
// rejected.  The image's status word is then OR-ed into (the soft-vote kernel may have set bits) instead of written.
//
// Phase 2 (the last CTA of each image to finish phase 1; found with a ticket counter, no waiting): ordered
// compaction without atomics or sorting.  Every thread counts the set bits of its contiguous slice of the
// bitmap, an exclusive block scan gives each slice its first output slot, and the slices are written out in
// order, so the list is ascending in the linear bin index and, when there are more than K_max peaks, exactly
// the first K_max are kept.  Then the centroids (bin positions of Eq. 9 in pixel units) and the peak
// embeddings concat(P_w[cx], P_h[cy]) are gathered, and the image's counters and status word are written.
//
// With `sums` (sub-cell refinement; int64 [B][cells][2], the fixed-point sums of the estimates that fell into each
// bin) a peak is moved from its bin position to the mean estimate of its 3x3 neighbourhood -- a strict peak has no
// other peak there, so those votes are its own -- and its embedding is gamma(mean) of Eq. 2, evaluated in binary64
// and rounded once, the way the palette rows are made.  `zero_sums` (only with one CTA per image): the sums are cleared
// at the end, so that the decode needs no clearing pass for them.
//
// `refine_out` = 0 with `sums` (the pruned assignment of the unrefined decode): the peaks stay on their bin positions
// and keep their palette rows, and gamma(mean) goes to `ref_emb` instead, where the assignment uses it as the point
// its distance bounds are taken around.  `cell_peak` (with the pruned assignment): bin -> index of the peak whose 3x3
// window holds it, -1 where there is none; `near_state`: that kernel's per-image words, zeroed here.
//
// `skip_rows`: the peaks' embeddings and centroids are left to peak_rows_kernel (launched next), which spreads them over
// the GPU; this kernel's last CTA then ends with the peak list, the bin -> peak table and the counters.
//
// `staged` (only with one CTA per image; needs 4 * bins_w * bins_h bytes of dynamic shared memory): the CTA first
// copies the whole vote map into shared memory with independent loads -- one round trip to L2 instead of one or two
// per 32-bin word and warp iteration -- and keeps the bitmap and the head of the peak list there as well, so that
// the dependent steps of this latency-bound kernel stay on the SM.
// The search for image b by CTA `cta` of `n_ctas` (THREADS threads each); s_map: [cells] words of shared memory when
// a.staged.  peaks_kernel calls it with its grid's coordinates; the voting kernel's last CTA of an image calls it with
// n_ctas = 1 when the map is small (one launch fewer).
template <int THREADS>
__device__ __forceinline__ void peaks_image(const PeakArgs& a, int b, int cta, int n_ctas, uint32_t* s_map) {
  const uint32_t* __restrict__ votes = a.votes;
  const int bins_w = a.bins_w, bins_h = a.bins_h, words = a.words;
  const uint32_t T_v = a.T_v;
  const int strict = a.strict;
  uint32_t* __restrict__ bitmap = a.bitmap;
  const int K_max = a.K_max, F = a.F, H = a.H, W = a.W;
  const float* __restrict__ pal_w = a.pal_w;
  const float* __restrict__ pal_h = a.pal_h;
  int32_t* __restrict__ peak_cell = a.peak_cell;
  uint32_t* __restrict__ peak_votes = a.peak_votes;
  float* __restrict__ peak_emb = a.peak_emb;
  float* __restrict__ out_centroids = a.out_centroids;
  int32_t* __restrict__ out_count = a.out_count;
  uint32_t* __restrict__ acc = a.acc;
  uint32_t* __restrict__ counters = a.counters;
  uint32_t* __restrict__ status = a.status;
  long long* __restrict__ sums = a.sums;
  const int zero_sums = a.zero_sums, staged = a.staged, refine_out = a.refine_out, skip_rows = a.skip_rows;
  float* __restrict__ ref_emb = a.ref_emb;
  int32_t* __restrict__ cell_peak = a.cell_peak;
  uint32_t* __restrict__ near_state = a.near_state;
  __shared__ uint32_t s_bm[kPeakStageWords];
  __shared__ int s_pc[kPeakListStage];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int cells = bins_w * bins_h;
  const uint32_t* V = votes + (size_t)b * cells;
  uint32_t* bm = bitmap + (size_t)b * words;
  // the voting kernel's accumulators are wanted by thread 0 near the end: fetched now, off the critical path
  uint32_t acc_voting = 0, acc_nonfinite = 0;
  if (tid == 0) {
    acc_voting = __ldcg(&acc[b * kAccStride + kAccVoting]);
    acc_nonfinite = __ldcg(&acc[b * kAccStride + kAccNonfinite]);
  }
  if (staged) {
    for (int i = tid; i < cells; i += THREADS) s_map[i] = __ldcg(V + i);
    __syncthreads();
  }
  auto vote_at = [&](int i) -> uint32_t { return staged ? s_map[i] : __ldg(V + i); };
  auto bitmap_at = [&](int w) -> uint32_t { return staged ? s_bm[w] : __ldcg(bm + w); };
  auto cell_of = [&](const int32_t* list, int k) -> int { return (staged && k < kPeakListStage) ? s_pc[k] : list[k]; };

  // ---- phase 1 (a CTA takes the words cta*32 + wid, then strides by the grid: one CTA per image for small maps)
  for (int warp = cta * (THREADS / 32) + wid; warp < words; warp += n_ctas * (THREADS / 32)) {
    const int lin = warp * 32 + lane;
    bool peak = false;
    if (lin < cells) {
      const uint32_t v = vote_at(lin);
      if (v > T_v) {
        const int cy = lin / bins_w, cx = lin - cy * bins_w;
        peak = true;
#pragma unroll
        for (int dy = -1; dy <= 1; ++dy) {
#pragma unroll
          for (int dx = -1; dx <= 1; ++dx) {
            if (dx == 0 && dy == 0) continue;
            const int ny = cy + dy, nx = cx + dx;
            if (ny < 0 || ny >= bins_h || nx < 0 || nx >= bins_w) continue;
            const int nlin = ny * bins_w + nx;
            const uint32_t nv = vote_at(nlin);
            if (nv > v || (nv == v && (strict || nlin < lin))) peak = false;
          }
        }
      }
    }
    if (cell_peak && lin < cells) cell_peak[(size_t)b * cells + lin] = -1;
    const uint32_t word = __ballot_sync(0xffffffffu, peak);
    if (lane == 0) {
      bm[warp] = word;
      if (staged) s_bm[warp] = word;
    }
  }

  // ---- which CTA of this image is the last one?  (with one CTA per image there is nothing to ask)
  if (n_ctas > 1) {
    __shared__ int s_last;
    __threadfence();          // this CTA's bitmap words are visible device-wide before its ticket is taken
    __syncthreads();
    if (tid == 0) {
      const uint32_t ticket = atomicAdd(&acc[b * kAccStride + kAccTicket], 1u);
      s_last = ticket == (uint32_t)(n_ctas - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();          // and the other CTAs' words are visible to this one
  } else {
    __syncthreads();
  }

  // ---- phase 2
  int32_t* pc = peak_cell + (size_t)b * K_max;
  uint32_t* pv = peak_votes + (size_t)b * K_max;
  const int per = (words + THREADS - 1) / THREADS;
  const int w0 = min(words, tid * per), w1 = min(words, w0 + per);
  // (eight words at a time, fetched before the first is used: a thread's words come one round trip apart otherwise)
  int local = 0;
  for (int w = w0; w < w1; w += 8) {
    uint32_t v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = (w + u < w1) ? bitmap_at(w + u) : 0u;
#pragma unroll
    for (int u = 0; u < 8; ++u) local += __popc(v[u]);
  }

  __shared__ int s_warp[THREADS / 32];
  __shared__ int s_total;
  int incl = local;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) s_warp[wid] = incl;
  __syncthreads();
  if (wid == 0) {                      // exclusive scan of the warp totals by the first warp
    constexpr int NW = THREADS / 32;
    static_assert(NW <= 32, "one lane per warp total");
    const int mine = lane < NW ? s_warp[lane] : 0;
    int inc = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += t;
    }
    if (lane < NW) s_warp[lane] = inc - mine;
    if (lane == 31) s_total = inc;
  }
  __syncthreads();
  int slot = s_warp[wid] + incl - local;
  const int total = s_total;

  for (int w = w0; w < w1 && slot < K_max && local > 0; w += 8) {     // (a slice without a peak is not read again)
    uint32_t v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = (w + u < w1) ? bitmap_at(w + u) : 0u;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      uint32_t bits = v[u];
      while (bits && slot < K_max) {
        const int bit = __ffs(bits) - 1;
        bits &= bits - 1;
        const int lin = (w + u) * 32 + bit;
        pc[slot] = lin;
        if (staged && slot < kPeakListStage) s_pc[slot] = lin;
        pv[slot] = vote_at(lin);
        ++slot;
      }
    }
  }
  const int count = min(total, K_max);
  if (tid == 0) {
    out_count[b] = count;
    // fold the voting kernel's accumulators into this image's counters, and leave them zero for the next decode
    const uint32_t voting = acc_voting, nonfinite = acc_nonfinite;
    acc[b * kAccStride + kAccVoting] = 0u;
    acc[b * kAccStride + kAccNonfinite] = 0u;
    acc[b * kAccStride + kAccTicket] = 0u;
    acc[b * kAccStride + kAccSpan] = 0u;
    uint32_t* cnt = counters + b * CPE_CNT_N;
    cnt[CPE_CNT_VOTING] = voting;
    cnt[CPE_CNT_NONFINITE] = nonfinite;
    cnt[CPE_CNT_RAW_PEAKS] = (uint32_t)total;
    cnt[CPE_CNT_TRUNCATED] = (uint32_t)(total - count);
    cnt[CPE_CNT_TAU_REJECTED] = 0u;     // the assignment kernel adds to these four
    cnt[CPE_CNT_FILTER_PAIRS] = 0u;
    cnt[CPE_CNT_RESCORED] = 0u;
    cnt[CPE_CNT_FULL_SCORED] = 0u;
    if (near_state)
      for (int i = 0; i < kNearStride; ++i) near_state[b * kNearStride + i] = 0u;
    const uint32_t st_bits = (nonfinite ? (uint32_t)CPE_STATUS_NONFINITE : 0u) |
                             (total > K_max ? (uint32_t)CPE_STATUS_PEAK_OVERFLOW : 0u);
    if (strict) atomicOr(&status[b], st_bits);
    else status[b] = st_bits;
  }
  __syncthreads();  // the list written above is read below by other threads of this CTA

  const int D = 4 * F;
  float* pe = peak_emb + (size_t)b * K_max * D;
  if (cell_peak) {
    // every bin of a peak's 3x3 window names that peak (two peaks are never neighbours, so a peak's own bin is in no
    // other window; a bin between two peaks gets either)
    int32_t* cp = cell_peak + (size_t)b * cells;
    for (int k = tid; k < count; k += THREADS) {
      const int lin = cell_of(pc, k);
      const int cy = lin / bins_w, cx = lin - cy * bins_w;
#pragma unroll
      for (int dy = -1; dy <= 1; ++dy) {
#pragma unroll
        for (int dx = -1; dx <= 1; ++dx) {
          const int ny = cy + dy, nx = cx + dx;
          if (ny < 0 || ny >= bins_h || nx < 0 || nx >= bins_w) continue;
          cp[ny * bins_w + nx] = k;
        }
      }
    }
  }
  if (sums) {
    float* gm = refine_out ? pe : ref_emb + (size_t)b * K_max * D;   // where gamma(mean) goes
    __shared__ double s_mean[2 * kRefineChunk];
    long long* S = sums + (size_t)b * cells * 2;
    for (int k0 = 0; k0 < count; k0 += kRefineChunk) {
      const int nk = min(kRefineChunk, count - k0);
      for (int i = tid; i < 2 * nk; i += THREADS) {       // (peak, axis): pooled mean of the 3x3 window
        const int k = k0 + (i >> 1), axis = i & 1;
        const double m = window_mean(vote_at, S, cell_of(pc, k), bins_w, bins_h, axis);
        s_mean[i] = m;
        if (refine_out) out_centroids[((size_t)b * K_max + k) * 2 + axis] = mean_to_pixels(m, axis ? H : W);
      }
      __syncthreads();
      for (int i = tid; i < 2 * F * nk; i += THREADS) {   // (peak, axis, harmonic): sin and cos of pi 2^l mean
        const int kk = i / (2 * F), r = i - kk * 2 * F;
        const int axis = r / F, l = r - axis * F;
        double sn, cs;
        sincospi(scalbn(s_mean[2 * kk + axis], l), &sn, &cs);
        float* o = gm + (size_t)(k0 + kk) * D + axis * 2 * F + 2 * l;
        o[0] = (float)sn;
        o[1] = (float)cs;
      }
      __syncthreads();
    }
    // small maps (this CTA does the whole image): the sums have no reader left and are left zero for the next decode
    if (zero_sums)
      for (int i = tid; i < 2 * cells; i += THREADS) S[i] = 0;
    if (refine_out) return;
  }
  if (skip_rows) return;     // peak_rows_kernel writes the embeddings and the centroids
  for (int i = tid; i < count * D; i += THREADS) {
    const int k = i / D, c = i - k * D;
    const int lin = cell_of(pc, k);
    const int cy = lin / bins_w, cx = lin - cy * bins_w;
    pe[i] = (c < 2 * F) ? pal_w[cx * 2 * F + c] : pal_h[cy * 2 * F + (c - 2 * F)];
  }
  for (int k = tid; k < count; k += THREADS) {
    const int lin = cell_of(pc, k);
    const int cy = lin / bins_w, cx = lin - cy * bins_w;
    // bin position -1 + 2i/(n+1), i = c+1 (Eq. 9); pixel centres sit at x = -1 + (2 col + 1)/W
    const double x = -1.0 + 2.0 * (double)(cx + 1) / (double)(bins_w + 1);
    const double y = -1.0 + 2.0 * (double)(cy + 1) / (double)(bins_h + 1);
    float* o = out_centroids + ((size_t)b * K_max + k) * 2;
    o[0] = (float)(((x + 1.0) * (double)W - 1.0) * 0.5);
    o[1] = (float)(((y + 1.0) * (double)H - 1.0) * 0.5);
  }
}

__global__ void __launch_bounds__(kPeakThreads)
peaks_kernel(const PeakArgs a) {
  extern __shared__ uint32_t s_peak_map[];            // [cells] when a.staged
  grid_dependency_sync();
  peaks_image<kPeakThreads>(a, (int)blockIdx.y, (int)blockIdx.x, (int)gridDim.x, s_peak_map);
}

// gamma of the peaks' mean estimates as a kernel of its own, spread over the GPU: the binary64 sine and cosine of
// 2F arguments per peak take the last CTA of peaks_kernel longer than everything else it does once an image has
// hundreds of peaks.  A thread per (peak, axis, harmonic); `gm` [B][K_max][4F] receives gamma(mean) and, with
// `refine_out`, out_centroids the means in pixel units (the same operations as in peaks_kernel).  F a power of two.
constexpr int kRowsThreads = 128;
__global__ void __launch_bounds__(kRowsThreads)
peak_rows_kernel(const uint32_t* __restrict__ votes, const long long* __restrict__ sums, int bins_w, int bins_h, int K_max,
                 int F, int H, int W, const int32_t* __restrict__ peak_cell, const int32_t* __restrict__ count_ptr,
                 int refine_out, float* __restrict__ gm, float* __restrict__ out_centroids,
                 const float* __restrict__ pal_w, const float* __restrict__ pal_h, float* __restrict__ peak_emb) {
  grid_dependency_sync();
  const int b = blockIdx.y;
  const int cells = bins_w * bins_h;
  const int count = count_ptr[b];
  const uint32_t* V = votes + (size_t)b * cells;
  const long long* S = sums + (size_t)b * cells * 2;
  const int TP = 2 * F, D = 4 * F;                        // threads per peak (at most one warp)
  const int lane = threadIdx.x & 31;
  const int n_items = ((count * TP + 31) / 32) * 32;     // whole warps take part in the shuffle below
  for (int i = blockIdx.x * kRowsThreads + threadIdx.x; i < n_items; i += gridDim.x * kRowsThreads) {
    const int k = i / TP, r = i - k * TP;
    const int axis = r / F, l = r - axis * F;
    const bool have = k < count;
    double m = 0.0;
    const int lin = have ? peak_cell[(size_t)b * K_max + k] : 0;
    if (have && l == 0) {
      m = window_mean([&](int c) { return __ldcg(V + c); }, S, lin, bins_w, bins_h, axis);
      if (refine_out) out_centroids[((size_t)b * K_max + k) * 2 + axis] = mean_to_pixels(m, axis ? H : W);
    }
    if (have && !refine_out) {
      // the peak stays on its bin position: palette rows (Eq. 9) and the bin centre in pixel units
      const int cy = lin / bins_w, cx = lin - cy * bins_w;
      const int c = axis ? cy : cx, n = axis ? bins_h : bins_w;
      const float2 pr = *reinterpret_cast<const float2*>((axis ? pal_h : pal_w) + (size_t)c * 2 * F + 2 * l);
      *reinterpret_cast<float2*>(peak_emb + ((size_t)b * K_max + k) * D + axis * 2 * F + 2 * l) = pr;
      if (l == 0) {
        const double x = -1.0 + 2.0 * (double)(c + 1) / (double)(n + 1);
        out_centroids[((size_t)b * K_max + k) * 2 + axis] = (float)(((x + 1.0) * (double)(axis ? H : W) - 1.0) * 0.5);
      }
    }
    m = __shfl_sync(0xffffffffu, m, lane - l);             // from this (peak, axis)'s first thread
    if (have) {
      double sn, cs;
      sincospi(scalbn(m, l), &sn, &cs);
      float* o = gm + ((size_t)b * K_max + k) * D + axis * 2 * F + 2 * l;
      o[0] = (float)sn;
      o[1] = (float)cs;
    }
  }
}

}  // namespace cpe
