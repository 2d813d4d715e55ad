/*
 * CPU oracle for the centroid-positional-encoding decoder.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the decode
 * path computes.  Tests, the smoke check and the benchmark's CPU-baseline leg call it; the
 * product (the CUDA library) never does, and shares no code, header, table or constant
 * generator with it.  Build:  gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 *
 * What follows the paper and what is a stated reading of it:
 *   - gamma(p) = (sin(2^l pi p), cos(2^l pi p)), l = 0..F-1            Eq. 2   (F is the paper's L)
 *   - prediction split into an x half and a y half of 2F channels       Eq. 3
 *   - separable distance d = ||xhat - gamma(a)|| + ||yhat - gamma(b)||  Eq. 4   (Euclidean norms, not squared)
 *   - palettes P_n = { gamma(-1 + 2i/(n+1)) : i = 1..n }                Eq. 9   (taken as printed; no void bin, Sec. 3.2)
 *   - local maxima: strict maximum in the 8-connected neighbourhood
 *     above a threshold                                                 Sec. 3.2, "Local Maxima Search"
 *   - assignment m = argmin_k d(a_k, b_k), kept iff d < tau             Eq. 7, Eq. 8
 *   - soft-vote histogram H(a,b) = sum_ij exp(-d_ij(a,b))               Eq. 5, Eq. 6 (cpe_oracle_soft_votes; a second
 *     vote mode next to the hard vote, the plain definition in binary64)
 *   - the HARD vote (one integer vote per pixel into the nearest Eq. 9 bin of a per-pixel
 *     centroid estimate) replaces the soft vote of Eq. 5-6.  The paper does not define a
 *     per-pixel estimate; the one used here is coarse-to-fine phase unwrapping of the
 *     harmonics, fixed as an exact sequence of IEEE binary32 operations because an integer
 *     (the bin) is decided by it.                                       [parity unpinned by the paper;
 *                                                                        pinned by round trips and by the
 *                                                                        brute-force minimiser of Eq. 4]
 *   - integer ties between neighbouring cells (impossible with the paper's real-valued H)
 *     are broken towards the lower linear cell index.                   [reading]
 *   - ties in the argmin go to the lowest k.                            [reading]
 *
 * Layout: emb is planar [B][4F][H][W]; channel c = axis*2F + 2l + t, axis 0 = x (width),
 * axis 1 = y (height), t = 0 sin, t = 1 cos.  dtype 0 = binary32, 1 = binary16.
 * Floating point: the estimate and the bin decision are binary32 (round to nearest even,
 * no contraction; fmaf where an fma is meant).  Scores are binary64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_PI 3.14159265358979323846

static int g_threads = 1;

void cpe_oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }

int cpe_oracle_get_threads(void) {
#ifdef _OPENMP
  return g_threads;
#else
  return 1;
#endif
}

int cpe_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_num_procs();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------- O1: widen ---- */

/* binary16 -> binary32, exact. */
static float half_bits_to_float(uint16_t h) {
  uint32_t sign = (uint32_t)(h >> 15) & 1u;
  int32_t expo = (int32_t)((h >> 10) & 0x1Fu);
  uint32_t frac = (uint32_t)h & 0x3FFu;
  float v;
  if (expo == 0x1F) {
    v = frac ? NAN : INFINITY;
  } else if (expo == 0) {
    v = ldexpf((float)frac, -24); /* subnormal: frac * 2^-24 */
  } else {
    v = ldexpf((float)(frac | 0x400u), expo - 25); /* (1024+frac) * 2^(e-15-10) */
  }
  return sign ? -v : v;
}

void cpe_oracle_half_to_float_array(const uint16_t* h, int64_t n, float* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = half_bits_to_float(h[i]);
}

static float load_elem(const void* emb, int dtype, size_t idx) {
  if (dtype == 0) return ((const float*)emb)[idx];
  return half_bits_to_float(((const uint16_t*)emb)[idx]);
}

/* ------------------------------------------------- Eq. 9: bin positions, palettes ---- */

/* Position of bin i (1-based) of an n-bin palette, Eq. 9. */
static double bin_position(int n, int i) { return -1.0 + 2.0 * (double)i / (double)(n + 1); }

double cpe_oracle_bin_position(int n, int i) { return bin_position(n, i); }

/* out[(i-1)*2F + 2l + t] = (float) sin|cos(pi 2^l pos_n(i)); double evaluation, one rounding. Eq. 2, Eq. 9. */
void cpe_oracle_palette(int n, int F, float* out) {
  for (int i = 1; i <= n; ++i) {
    double pos = bin_position(n, i);
    for (int l = 0; l < F; ++l) {
      double arg = ORACLE_PI * ldexp(1.0, l) * pos;
      out[(size_t)(i - 1) * 2 * F + 2 * l + 0] = (float)sin(arg);
      out[(size_t)(i - 1) * 2 * F + 2 * l + 1] = (float)cos(arg);
    }
  }
}

/* ------------------------------------- O2: per-pixel centroid estimate (binary32) ---- */

/* Odd polynomial for atan(r)/pi on [0,1]: r*(C0 + C1 q + ... + C5 q^5), q = r*r. */
static const float AT_C0 = 0x1.45f12p-2f;
static const float AT_C1 = -0x1.b1ac3ap-4f;
static const float AT_C2 = 0x1.f8acc2p-5f;
static const float AT_C3 = -0x1.2f97d2p-5f;
static const float AT_C4 = 0x1.1290dap-6f;
static const float AT_C5 = -0x1.e8f09ap-9f;

/* atan2(y, x) in half-turns, result in [-1, 1]; inputs must be finite. */
float cpe_oracle_atan2_ht(float y, float x) {
  float ax = fabsf(x), ay = fabsf(y);
  float mx = ax > ay ? ax : ay;
  float mn = ax > ay ? ay : ax;
  if (mx == 0.0f) return 0.0f;
  float r = mn / mx;
  float q = r * r;
  float h = AT_C5;
  h = fmaf(h, q, AT_C4);
  h = fmaf(h, q, AT_C3);
  h = fmaf(h, q, AT_C2);
  h = fmaf(h, q, AT_C1);
  h = fmaf(h, q, AT_C0);
  h = h * r;
  if (ay > ax) h = 0.5f - h;
  if (x < 0.0f) h = 1.0f - h;
  if (y < 0.0f) h = -h;
  return h;
}

void cpe_oracle_atan2_ht_array(const float* y, const float* x, int64_t n, float* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = cpe_oracle_atan2_ht(y[i], x[i]);
}

/* A (sin, cos) pair takes part only if |s| + |c|, rounded to binary32, is finite. */
static int pair_is_finite(float s, float c) {
  float v = fabsf(s) + fabsf(c);
  return v < INFINITY; /* false for NaN and for +inf */
}

/*
 * Coarse-to-fine estimate of p in [-1, 1) from sc[2l] = sin, sc[2l+1] = cos, l = 0..F-1,
 * using harmonics 0..levels-1.  Harmonic 0 fixes p up to its own noise; every further
 * harmonic l knows p modulo 2^(1-l) more precisely, and the integer m picks the branch
 * nearest to the running estimate.
 */
float cpe_oracle_decode_axis(const float* sc, int F, int levels) {
  int Fu = (levels > 0 && levels < F) ? levels : F;
  float p = cpe_oracle_atan2_ht(sc[0], sc[1]);
  for (int l = 1; l < Fu; ++l) {
    float scale = ldexpf(1.0f, l);
    float inv = ldexpf(1.0f, -l);
    float u = cpe_oracle_atan2_ht(sc[2 * l], sc[2 * l + 1]);
    float t = p * scale;               /* exact */
    float m = rintf((t - u) * 0.5f);   /* one rounded subtraction; halving exact; ties to even */
    float w = u + 2.0f * m;            /* 2m exact; one rounded addition */
    p = w * inv;                       /* exact */
  }
  if (p < -1.0f) p = p + 2.0f;
  if (p >= 1.0f) p = p - 2.0f;
  return p;
}

/* sc is [n][2F]; out[i] = estimate of row i. */
void cpe_oracle_decode_axis_array(const float* sc, int64_t n, int F, int levels, float* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = cpe_oracle_decode_axis(sc + (size_t)i * 2 * F, F, levels);
}

/* O3: nearest Eq. 9 bin (0-based) of a coordinate estimate; the end bins also take what lies beyond them. */
int cpe_oracle_cell_of(float p, int n) {
  float half_np1 = (float)(n + 1) * 0.5f; /* exact for n <= 2^23 */
  float a = p + 1.0f;
  float g = a * half_np1;
  float r = rintf(g);
  int i = (int)r;
  if (i < 1) i = 1;
  if (i > n) i = n;
  return i - 1;
}

enum { CNT_VOTING = 0, CNT_NONFINITE = 1, CNT_RAW_PEAKS = 2, CNT_TRUNCATED = 3, CNT_TAU_REJECTED = 4, CNT_N = 8 };

/*
 * O2 + O3 for a whole batch.
 * votes    [B][bins_h][bins_w]  (zeroed here)
 * est      optional [B][H][W][2] (px, py) of each participating finite pixel, NaN elsewhere
 * cell     optional [B][H][W] linear cell cy*bins_w + cx, -1 for pixels that do not vote
 * counters optional [B][CNT_N]
 */
int cpe_oracle_votes(const void* emb, int dtype, const uint8_t* fg, int B, int H, int W, int F, int bins_w,
                     int bins_h, int levels, uint32_t* votes, float* est, int32_t* cell, int64_t* counters) {
  if (!emb || !votes || B < 1 || H < 1 || W < 1 || F < 1 || F > 16 || bins_w < 1 || bins_h < 1) return -1;
  size_t HW = (size_t)H * W;
  size_t cells = (size_t)bins_w * bins_h;
  memset(votes, 0, sizeof(uint32_t) * cells * B);
  int32_t* tmp_cell = cell ? cell : (int32_t*)malloc(sizeof(int32_t) * HW * B);
  if (!tmp_cell) return -2;
#pragma omp parallel for num_threads(g_threads) schedule(static)
  for (long long n = 0; n < (long long)(HW * B); ++n) {
    size_t b = (size_t)n / HW, pix = (size_t)n % HW;
    float sc[2][32];
    int take = fg ? (fg[n] != 0) : 1;
    int finite = 1;
    tmp_cell[n] = -1;
    if (est) est[2 * n] = est[2 * n + 1] = NAN;
    if (!take) continue;
    for (int axis = 0; axis < 2; ++axis)
      for (int j = 0; j < 2 * F; ++j)
        sc[axis][j] = load_elem(emb, dtype, (b * 4 * F + (size_t)axis * 2 * F + j) * HW + pix);
    for (int axis = 0; axis < 2; ++axis)
      for (int l = 0; l < F; ++l)
        if (!pair_is_finite(sc[axis][2 * l], sc[axis][2 * l + 1])) finite = 0;
    if (!finite) { tmp_cell[n] = -2; continue; }
    float px = cpe_oracle_decode_axis(sc[0], F, levels);
    float py = cpe_oracle_decode_axis(sc[1], F, levels);
    int cx = cpe_oracle_cell_of(px, bins_w);
    int cy = cpe_oracle_cell_of(py, bins_h);
    tmp_cell[n] = cy * bins_w + cx;
    if (est) { est[2 * n] = px; est[2 * n + 1] = py; }
  }
  for (size_t b = 0; b < (size_t)B; ++b) {
    int64_t voting = 0, nonfinite = 0;
    for (size_t pix = 0; pix < HW; ++pix) {
      int32_t c = tmp_cell[b * HW + pix];
      if (c >= 0) { votes[b * cells + (size_t)c] += 1u; ++voting; }
      else if (c == -2) { ++nonfinite; if (cell) tmp_cell[b * HW + pix] = -1; }
    }
    if (counters) { counters[b * CNT_N + CNT_VOTING] = voting; counters[b * CNT_N + CNT_NONFINITE] = nonfinite; }
  }
  if (!cell) free(tmp_cell);
  return 0;
}

/* ------------------------------------------------------------------ O4: peaks ---- */

/*
 * One image.  A cell is a peak iff V > T_v and it beats every existing 8-neighbour:
 * larger count, or equal count and lower linear index.  Peaks are listed by ascending
 * linear index; at most K_max are kept.  Returns the number kept; *raw_count = number found.
 */
int cpe_oracle_peaks(const uint32_t* V, int bins_w, int bins_h, int T_v, int K_max, int32_t* peak_cell,
                     uint32_t* peak_votes, int32_t* raw_count) {
  int kept = 0, raw = 0;
  for (int cy = 0; cy < bins_h; ++cy)
    for (int cx = 0; cx < bins_w; ++cx) {
      int lin = cy * bins_w + cx;
      uint32_t v = V[lin];
      if (T_v >= 0 && v <= (uint32_t)T_v) continue;
      int is_peak = 1;
      for (int dy = -1; dy <= 1 && is_peak; ++dy)
        for (int dx = -1; dx <= 1; ++dx) {
          if (!dx && !dy) continue;
          int ny = cy + dy, nx = cx + dx;
          if (ny < 0 || ny >= bins_h || nx < 0 || nx >= bins_w) continue;
          int nlin = ny * bins_w + nx;
          uint32_t nv = V[nlin];
          if (v > nv) continue;
          if (v == nv && lin < nlin) continue;
          is_peak = 0;
          break;
        }
      if (!is_peak) continue;
      if (kept < K_max) {
        if (peak_cell) peak_cell[kept] = lin;
        if (peak_votes) peak_votes[kept] = v;
        ++kept;
      }
      ++raw;
    }
  if (raw_count) *raw_count = raw;
  return kept;
}

/*
 * The local-maxima search as the paper prints it, on a real-valued map H (Sec. 3.2, "Local Maxima Search"): a bin
 * is a candidate centroid iff its value exceeds the threshold and is a STRICT maximum of its 8-connected
 * neighbourhood (neighbours outside the map do not exist).  Two equal neighbours are both rejected: the printed
 * test has no tie rule and real-valued sums do not tie.  Peaks are listed by ascending linear index, at most K_max.
 */
int cpe_oracle_real_peaks(const double* Hmap, int bins_w, int bins_h, double threshold, int K_max, int32_t* peak_cell,
                          int32_t* raw_count) {
  int kept = 0, raw = 0;
  for (int cy = 0; cy < bins_h; ++cy)
    for (int cx = 0; cx < bins_w; ++cx) {
      const int lin = cy * bins_w + cx;
      const double v = Hmap[lin];
      if (!(v > threshold)) continue;
      int is_peak = 1;
      for (int dy = -1; dy <= 1 && is_peak; ++dy)
        for (int dx = -1; dx <= 1; ++dx) {
          if (!dx && !dy) continue;
          const int ny = cy + dy, nx = cx + dx;
          if (ny < 0 || ny >= bins_h || nx < 0 || nx >= bins_w) continue;
          if (!(v > Hmap[ny * bins_w + nx])) { is_peak = 0; break; }
        }
      if (!is_peak) continue;
      if (kept < K_max && peak_cell) peak_cell[kept] = lin;
      if (kept < K_max) ++kept;
      ++raw;
    }
  if (raw_count) *raw_count = raw;
  return kept;
}

/* O5: pixel-unit centre of bin (cx, cy): normalised x = -1 + (2 col + 1)/W  <=>  col = ((x+1) W - 1)/2. */
void cpe_oracle_centroid_px(int cx, int cy, int bins_w, int bins_h, int H, int W, float* out_xy) {
  double x = bin_position(bins_w, cx + 1), y = bin_position(bins_h, cy + 1);
  out_xy[0] = (float)(((x + 1.0) * (double)W - 1.0) * 0.5);
  out_xy[1] = (float)(((y + 1.0) * (double)H - 1.0) * 0.5);
}

/* ------------------------------------------------------------- O6: assignment ---- */

/*
 * One image.  For the pixels listed in idx[0..n_idx) (all H*W pixels if idx is NULL):
 * label = 1 + argmin_k d_k if the pixel participates, is finite, count > 0 and d < tau; else 0.
 * best/second (optional, same indexing as labels) receive the smallest and second smallest d
 * (+inf where there is none).  Outputs are indexed by position in idx (or by pixel if idx is NULL).
 */
int cpe_oracle_assign_image(const void* emb_img, int dtype, const uint8_t* fg_img, int H, int W, int F,
                            const float* Pw, const float* Ph, int bins_w, const int32_t* peak_cell, int count,
                            double tau, const int64_t* idx, int64_t n_idx, int32_t* labels, double* best,
                            double* second, int64_t* tau_rejected, const float* peak_emb) {
  size_t HW = (size_t)H * W;
  int64_t N = idx ? n_idx : (int64_t)HW;
  int64_t rejected = 0;
#pragma omp parallel for num_threads(g_threads) schedule(static) reduction(+ : rejected)
  for (long long j = 0; j < (long long)N; ++j) {
    size_t pix = idx ? (size_t)idx[j] : (size_t)j;
    double xh[32], yh[32];
    double d1 = INFINITY, d2 = INFINITY;
    int k1 = -1;
    labels[j] = 0;
    if (best) best[j] = INFINITY;
    if (second) second[j] = INFINITY;
    if (fg_img && !fg_img[pix]) continue;
    int finite = 1;
    for (int c = 0; c < 2 * F; ++c) {
      float xv = load_elem(emb_img, dtype, (size_t)c * HW + pix);
      float yv = load_elem(emb_img, dtype, (size_t)(2 * F + c) * HW + pix);
      xh[c] = (double)xv;
      yh[c] = (double)yv;
    }
    for (int l = 0; l < F; ++l) {
      if (!pair_is_finite((float)xh[2 * l], (float)xh[2 * l + 1])) finite = 0;
      if (!pair_is_finite((float)yh[2 * l], (float)yh[2 * l + 1])) finite = 0;
    }
    if (!finite) continue;
    for (int k = 0; k < count; ++k) {
      int cx = peak_cell[k] % bins_w, cy = peak_cell[k] / bins_w;
      /* candidates are the palette rows of the peak's bin (Eq. 7), unless the caller hands in refined ones */
      const float* ex = peak_emb ? peak_emb + (size_t)k * 4 * F : Pw + (size_t)cx * 2 * F;
      const float* ey = peak_emb ? peak_emb + (size_t)k * 4 * F + 2 * F : Ph + (size_t)cy * 2 * F;
      double sx = 0.0, sy = 0.0;
      for (int c = 0; c < 2 * F; ++c) {
        double dx = xh[c] - (double)ex[c];
        double dy = yh[c] - (double)ey[c];
        sx += dx * dx;
        sy += dy * dy;
      }
      double d = sqrt(sx) + sqrt(sy); /* Eq. 4 */
      if (d < d1) { d2 = d1; d1 = d; k1 = k; }   /* strict: the lowest k keeps an exact tie */
      else if (d < d2) { d2 = d; }
    }
    if (best) best[j] = d1;
    if (second) second[j] = d2;
    if (k1 >= 0) {
      if (d1 < tau) labels[j] = k1 + 1; /* Eq. 8, strict */
      else ++rejected;
    }
  }
  if (tau_rejected) *tau_rejected = rejected;
  return 0;
}

/* ------------------------------------------------------------- the whole chain ---- */

/* ------------------------------------------------ Sec. 3.2 "Mask aggregation": per-instance outputs ---- */

/*
 * The paper's output form of the assignment: one binary mask per candidate centroid and a counter of the pixels
 * that went to it (Eq. 8; Sec. 3.2: "output masks ... and a counter").  From a label map (0 = none, m + 1 = mask m):
 * planes[b][m][i][j] = 1 iff labels[b][i][j] == m + 1, pixels[b][m] = number of such pixels, for m < n_planes.
 * Either output may be NULL.
 */
int cpe_oracle_instance_masks(const int32_t* labels, int B, int H, int W, int n_planes, uint8_t* planes,
                              uint32_t* pixels) {
  if (!labels || B < 1 || H < 1 || W < 1 || n_planes < 1) return -1;
  const size_t HW = (size_t)H * W;
  for (int b = 0; b < B; ++b)
    for (int m = 0; m < n_planes; ++m) {
      uint32_t cnt = 0;
      for (size_t p = 0; p < HW; ++p) {
        const int hit = labels[(size_t)b * HW + p] == m + 1;
        if (planes) planes[((size_t)b * n_planes + m) * HW + p] = (uint8_t)hit;
        cnt += (uint32_t)hit;
      }
      if (pixels) pixels[(size_t)b * n_planes + m] = cnt;
    }
  return 0;
}

/* ------------------------------------------- Eq. 4-6: the soft-vote histogram (binary64) ---- */

/*
 * The paper's coarse voting histogram, written out as printed: every participating pixel (i, j) adds the weight
 *     w_ij(a, b) = exp(-(||xhat(i,j) - P_w[a]|| + ||yhat(i,j) - P_h[b]||))          Eq. 4, Eq. 5
 * to bin (a, b):  H(a, b) = sum over the participating pixels of w_ij(a, b).          Eq. 6
 * (Eq. 10-11 factorise the same sum as E_x^T E_y; this is the unfactorised definition.)  Euclidean norms, not
 * squared.  A pixel takes part iff its mask byte is non-zero (all pixels if fg is NULL) and all its channels are
 * finite -- the same participating set as the hard vote.  Palette rows are the binary32 tables of Eq. 9.
 * out: [B][bins_h][bins_w] doubles, or, with n_sample > 0, [B][n_sample] for the linear cells b*bins_w + a listed
 * in sample_cells (so that a few bins of a large problem can be checked).
 */
int cpe_oracle_soft_votes(const void* emb, int dtype, const uint8_t* fg, int B, int H, int W, int F, int bins_w,
                          int bins_h, const int32_t* sample_cells, int n_sample, double* out) {
  if (!emb || !out || B < 1 || H < 1 || W < 1 || F < 1 || bins_w < 1 || bins_h < 1) return -1;
  float* Pw = (float*)malloc(sizeof(float) * (size_t)bins_w * 2 * F);
  float* Ph = (float*)malloc(sizeof(float) * (size_t)bins_h * 2 * F);
  if (!Pw || !Ph) { free(Pw); free(Ph); return -2; }
  cpe_oracle_palette(bins_w, F, Pw);
  cpe_oracle_palette(bins_h, F, Ph);
  const size_t HW = (size_t)H * W;
  const int n_cells = n_sample > 0 ? n_sample : bins_w * bins_h;
  for (int b = 0; b < B; ++b) {
    const size_t base = (size_t)b * 4 * F * HW;
#pragma omp parallel for schedule(dynamic, 1) num_threads(g_threads)
    for (int ci = 0; ci < n_cells; ++ci) {
      const int lin = n_sample > 0 ? sample_cells[ci] : ci;
      const int a = lin % bins_w, bb = lin / bins_w;
      double sum = 0.0;
      for (size_t p = 0; p < HW; ++p) {
        if (fg && !fg[(size_t)b * HW + p]) continue;
        int finite = 1;
        for (int l = 0; l < 2 * F && finite; ++l)
          finite = pair_is_finite(load_elem(emb, dtype, base + (size_t)(2 * l) * HW + p),
                                  load_elem(emb, dtype, base + (size_t)(2 * l + 1) * HW + p));
        if (!finite) continue;
        double sx = 0.0, sy = 0.0;
        for (int c = 0; c < 2 * F; ++c) {
          const double tx = (double)load_elem(emb, dtype, base + (size_t)c * HW + p) - (double)Pw[(size_t)a * 2 * F + c];
          const double ty = (double)load_elem(emb, dtype, base + (size_t)(2 * F + c) * HW + p) - (double)Ph[(size_t)bb * 2 * F + c];
          sx += tx * tx;
          sy += ty * ty;
        }
        sum += exp(-(sqrt(sx) + sqrt(sy)));
      }
      out[(size_t)b * n_cells + ci] = sum;
    }
  }
  free(Pw);
  free(Ph);
  return 0;
}

/*
 * Same argument order as the library's decode entry point, host pointers, plus the intermediates.
 * out_labels [B][H][W], out_centroids [B][K_max][2], out_count [B];
 * votes [B][bins_h][bins_w], peak_cell [B][K_max], peak_votes [B][K_max] (all required);
 * best/second optional [B][H][W] doubles; counters optional [B][CNT_N].
 */
int cpe_oracle_decode(const void* emb, const uint8_t* fg, int B, int H, int W, int F, int dtype, int bins_w,
                      int bins_h, int levels, int T_v, double tau, int K_max, int32_t* out_labels,
                      float* out_centroids, int32_t* out_count, uint32_t* votes, int32_t* peak_cell,
                      uint32_t* peak_votes, double* best, double* second, int64_t* counters) {
  if (!out_labels || !out_centroids || !out_count || !peak_cell || !peak_votes || K_max < 1) return -1;
  int rc = cpe_oracle_votes(emb, dtype, fg, B, H, W, F, bins_w, bins_h, levels, votes, NULL, NULL, counters);
  if (rc) return rc;
  float* Pw = (float*)malloc(sizeof(float) * (size_t)bins_w * 2 * F);
  float* Ph = (float*)malloc(sizeof(float) * (size_t)bins_h * 2 * F);
  if (!Pw || !Ph) { free(Pw); free(Ph); return -2; }
  cpe_oracle_palette(bins_w, F, Pw);
  cpe_oracle_palette(bins_h, F, Ph);
  size_t HW = (size_t)H * W, cells = (size_t)bins_w * bins_h;
  size_t esz = dtype == 0 ? 4 : 2;
  for (int b = 0; b < B; ++b) {
    int32_t raw = 0;
    int kept = cpe_oracle_peaks(votes + b * cells, bins_w, bins_h, T_v, K_max, peak_cell + (size_t)b * K_max,
                                peak_votes + (size_t)b * K_max, &raw);
    out_count[b] = kept;
    for (int k = 0; k < kept; ++k) {
      int lin = peak_cell[(size_t)b * K_max + k];
      cpe_oracle_centroid_px(lin % bins_w, lin / bins_w, bins_w, bins_h, H, W,
                             out_centroids + ((size_t)b * K_max + k) * 2);
    }
    int64_t rejected = 0;
    cpe_oracle_assign_image((const char*)emb + (size_t)b * 4 * F * HW * esz, dtype, fg ? fg + b * HW : NULL, H, W,
                            F, Pw, Ph, bins_w, peak_cell + (size_t)b * K_max, kept, tau, NULL, 0,
                            out_labels + b * HW, best ? best + b * HW : NULL, second ? second + b * HW : NULL,
                            &rejected, NULL);
    if (counters) {
      counters[b * CNT_N + CNT_RAW_PEAKS] = raw;
      counters[b * CNT_N + CNT_TRUNCATED] = raw - kept;
      counters[b * CNT_N + CNT_TAU_REJECTED] = rejected;
    }
  }
  free(Pw);
  free(Ph);
  return 0;
}

/* ------------------------------- sub-cell refined centroids (an extension of Sec. 3.2 / Eq. 7) ---- */

/*
 * The paper's candidates are bin positions, so a candidate is off the voted centroid by up to half a bin.  The
 * refinement keeps, next to every bin's count, the sum of the estimates that fell into it, and moves each peak to
 * the mean estimate of its 3x3 neighbourhood (a strict peak has no other peak there, so those votes are its own).
 *
 * Sums are integers so that they do not depend on the order of addition: every estimate is taken as the fixed-point
 * number rint(p * 2^24) (|p| <= 1: exact for |p| >= 1/4, otherwise rounded to 2^-24).
 *   est  [B][H*W][2] binary32 estimates and cell [B][H*W] (-1 = no vote), as cpe_oracle_votes returns them
 *   sums [B][cells][2] int64 (x, y)
 */
#define REFINE_SCALE 16777216.0 /* 2^24 */

int cpe_oracle_vote_sums(const float* est, const int32_t* cell, int B, int H, int W, int cells, int64_t* sums) {
  if (!est || !cell || !sums) return -1;
  size_t HW = (size_t)H * W;
  memset(sums, 0, sizeof(int64_t) * 2 * (size_t)cells * B);
  for (size_t b = 0; b < (size_t)B; ++b)
    for (size_t pix = 0; pix < HW; ++pix) {
      int32_t c = cell[b * HW + pix];
      if (c < 0) continue;
      for (int a = 0; a < 2; ++a)
        sums[(b * cells + (size_t)c) * 2 + a] += (int64_t)llrint((double)est[(b * HW + pix) * 2 + a] * REFINE_SCALE);
    }
  return 0;
}

/*
 * One image: for each listed peak, mean = (sum over the 3x3 window of sums) / (2^24 * sum over it of votes), per
 * axis, in binary64; the refined candidate is gamma(mean) of Eq. 2 (binary64 sin/cos, one rounding to binary32, the
 * way the palette of Eq. 9 is made) and the refined centroid is mean in pixel units.
 *   peak_emb [count][4F] (x block then y block), centroids [count][2], mean [count][2] (optional)
 */
int cpe_oracle_refined_peaks(const uint32_t* votes_img, const int64_t* sums_img, int bins_w, int bins_h,
                             const int32_t* peak_cell, int count, int F, int H, int W, float* peak_emb,
                             float* centroids, double* mean) {
  if (!votes_img || !sums_img || !peak_cell || !peak_emb || !centroids) return -1;
  for (int k = 0; k < count; ++k) {
    int cx = peak_cell[k] % bins_w, cy = peak_cell[k] / bins_w;
    int64_t s[2] = {0, 0}, n = 0;
    for (int dy = -1; dy <= 1; ++dy)
      for (int dx = -1; dx <= 1; ++dx) {
        int x = cx + dx, y = cy + dy;
        if (x < 0 || x >= bins_w || y < 0 || y >= bins_h) continue;
        size_t c = (size_t)y * bins_w + x;
        n += votes_img[c];
        s[0] += sums_img[2 * c];
        s[1] += sums_img[2 * c + 1];
      }
    double m[2];
    for (int a = 0; a < 2; ++a) {
      m[a] = (double)s[a] / ((double)n * REFINE_SCALE);
      if (mean) mean[2 * k + a] = m[a];
      for (int l = 0; l < F; ++l) {
        double arg = ORACLE_PI * ldexp(1.0, l) * m[a];
        peak_emb[(size_t)k * 4 * F + (size_t)a * 2 * F + 2 * l + 0] = (float)sin(arg);
        peak_emb[(size_t)k * 4 * F + (size_t)a * 2 * F + 2 * l + 1] = (float)cos(arg);
      }
    }
    centroids[2 * k + 0] = (float)(((m[0] + 1.0) * (double)W - 1.0) * 0.5);
    centroids[2 * k + 1] = (float)(((m[1] + 1.0) * (double)H - 1.0) * 0.5);
  }
  return 0;
}
