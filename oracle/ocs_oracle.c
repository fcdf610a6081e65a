/*
 * CPU checker for outlier channel splitting (arXiv:1901.09504).  TEST INFRASTRUCTURE ONLY:
 * plain scalar C, no blocking, no fusion; see ocs_oracle.h for the conventions.
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC (OpenMP is used
 * only on the outermost independent loop of the integer contractions).
 */
#include "ocs_oracle.h"

#include <math.h>
#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif
#ifndef M_E
#define M_E 2.71828182845904523536
#endif
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ Section 3.4: split count */
int ocs_oracle_num_splits(int C, double ratio) {
  if (C <= 0 || !(ratio > 0.0)) return 0;
  return (int)ceil(ratio * (double)C - 1e-9);
}

/* ------------------------------------------------------------------ Section 3.3: one split */
/* The two halves of one value.  d = 0 is the Net2WiderNet rule (w/2, w/2); d = half a grid
 * step is the quantization-aware rule ((w - 0.5)/2, (w + 0.5)/2) written in weight units.
 * Each operation rounds once to fp32. */
static inline float split_keep(float w, float d) {
  volatile float t = w - d;
  return t * 0.5f;
}
static inline float split_new(float w, float d) {
  volatile float t = w + d;
  return t * 0.5f;
}

static float channel_maxabs(const float* Wc, int O, int Ctot, int R, int j) {
  float m = 0.0f;
  for (int o = 0; o < O; ++o)
    for (int r = 0; r < R; ++r) {
      float a = fabsf(Wc[((size_t)o * Ctot + j) * R + r]);
      if (a > m) m = a;
    }
  return m;
}

static void split_channel(float* Wc, int O, int Ctot, int R, int j, int jnew, float d) {
  for (int o = 0; o < O; ++o)
    for (int r = 0; r < R; ++r) {
      size_t src = ((size_t)o * Ctot + j) * R + r;
      size_t dst = ((size_t)o * Ctot + jnew) * R + r;
      float w = Wc[src];
      Wc[src] = split_keep(w, d);
      Wc[dst] = split_new(w, d);
    }
}

static int split_common(const float* W, int O, int C, int R, int S, float qa_step, float* W_out,
                        int32_t* idx_map, int32_t* split_order, float* max_abs, int cached) {
  if (!W || !W_out || !idx_map || O <= 0 || C <= 0 || R <= 0 || S < 0 || !(qa_step >= 0.0f))
    return 1;
  const int Ctot = C + S;
  const float d = qa_step * 0.5f;
  /* current tensor: channels [0, C) hold W, [C, C+S) are not alive yet */
  for (int o = 0; o < O; ++o)
    for (int j = 0; j < Ctot; ++j)
      for (int r = 0; r < R; ++r)
        W_out[((size_t)o * Ctot + j) * R + r] =
            (j < C) ? W[((size_t)o * C + j) * R + r] : 0.0f;
  for (int j = 0; j < C; ++j) idx_map[j] = j;
  if (max_abs) {
    float m = 0.0f;
    for (int j = 0; j < C; ++j) {
      float c = channel_maxabs(W_out, O, Ctot, R, j);
      if (c > m) m = c;
    }
    max_abs[0] = m;
  }
  float* cmax = NULL;
  if (cached) {
    cmax = (float*)malloc(sizeof(float) * (size_t)Ctot);
    if (!cmax) return 2;
    for (int j = 0; j < C; ++j) cmax[j] = channel_maxabs(W_out, O, Ctot, R, j);
  }
  for (int s = 0; s < S; ++s) {
    const int alive = C + s;
    int jbest = 0;
    float best = -1.0f;
    for (int j = 0; j < alive; ++j) { /* ascending j + strict '>' : ties go to the smallest index */
      float c = cached ? cmax[j] : channel_maxabs(W_out, O, Ctot, R, j);
      if (c > best) { best = c; jbest = j; }
    }
    split_channel(W_out, O, Ctot, R, jbest, alive, d);
    idx_map[alive] = idx_map[jbest];
    if (split_order) split_order[s] = jbest;
    if (cached) {
      cmax[jbest] = channel_maxabs(W_out, O, Ctot, R, jbest);
      cmax[alive] = channel_maxabs(W_out, O, Ctot, R, alive);
    }
  }
  if (max_abs) {
    float m = 0.0f;
    for (int j = 0; j < Ctot; ++j) {
      float c = channel_maxabs(W_out, O, Ctot, R, j);
      if (c > m) m = c;
    }
    max_abs[1] = m;
  }
  free(cmax);
  return 0;
}

int ocs_oracle_split_literal(const float* W, int O, int C, int R, int S, float qa_step,
                             float* W_out, int32_t* idx_map, int32_t* split_order,
                             float* max_abs) {
  return split_common(W, O, C, R, S, qa_step, W_out, idx_map, split_order, max_abs, 0);
}
int ocs_oracle_split_cached(const float* W, int O, int C, int R, int S, float qa_step,
                            float* W_out, int32_t* idx_map, int32_t* split_order,
                            float* max_abs) {
  return split_common(W, O, C, R, S, qa_step, W_out, idx_map, split_order, max_abs, 1);
}

/* ------------------------------------------------------------------ Eq. 1: linear quantization */
float ocs_oracle_maxabs(const float* T, int64_t n) {
  float m = 0.0f;
  for (int64_t i = 0; i < n; ++i) {
    float a = fabsf(T[i]);
    if (a > m) m = a;
  }
  return m;
}

static int code_limit(int bits, int is_signed) {
  return is_signed ? (1 << (bits - 1)) - 1 : (1 << bits) - 1;
}

int ocs_oracle_quantize(const float* T, int64_t n, int bits, int is_signed, float alpha,
                        int8_t* codes, float* scale) {
  if (!T || !codes || n < 0 || bits < 2 || bits > 8 || !(alpha >= 0.0f)) return 1;
  const int L = code_limit(bits, is_signed);
  if (alpha == 0.0f) {
    memset(codes, 0, (size_t)n);
    if (scale) *scale = 0.0f;
    return 0;
  }
  volatile float step = alpha / (float)L;
  volatile float inv = (float)L / alpha;
  const float lo = is_signed ? -(float)L : 0.0f, hi = (float)L;
  for (int64_t i = 0; i < n; ++i) {
    volatile float t = T[i] * inv;
    float q = nearbyintf(t); /* default rounding mode: half to even */
    if (q < lo) q = lo;
    if (q > hi) q = hi;
    int c = (int)q;
    if (is_signed) codes[i] = (int8_t)c;
    else ((uint8_t*)codes)[i] = (uint8_t)c;
  }
  if (scale) *scale = step;
  return 0;
}

/* ------------------------------------------------------------------ Section 4.1: MSE clip search */
int ocs_oracle_clip_mse(const float* T, int64_t n, int bits, int is_signed, int n_bins,
                        int n_candidates, float* alpha, float* max_abs, uint64_t* hist,
                        double* scores) {
  if (!T || !alpha || n < 0 || bits < 2 || bits > 8 || n_bins < 1 || n_candidates < 1) return 1;
  const int L = code_limit(bits, is_signed);
  const int B = n_bins;
  const float m = ocs_oracle_maxabs(T, n);
  if (max_abs) *max_abs = m;
  uint64_t* h = (uint64_t*)calloc((size_t)B, sizeof(uint64_t));
  if (!h) return 2;
  if (m == 0.0f) {
    *alpha = 0.0f;
    if (hist) { memset(hist, 0, sizeof(uint64_t) * (size_t)B); hist[0] = (uint64_t)n; }
    if (scores) for (int c = 0; c < n_candidates; ++c) scores[c] = 0.0;
    free(h);
    return 0;
  }
  /* histogram of |x|: B equal bins on [0, m] */
  volatile float invw = (float)B / m;
  for (int64_t i = 0; i < n; ++i) {
    volatile float t = fabsf(T[i]) * invw;
    int b = (int)t; /* truncation */
    if (b > B - 1) b = B - 1;
    h[b] += 1;
  }
  if (hist) memcpy(hist, h, sizeof(uint64_t) * (size_t)B);
  const double width = (double)m / (double)B;
  const double lo = is_signed ? -(double)L : 0.0, hi = (double)L;
  double best = 0.0;
  int cbest = -1;
  for (int c = 1; c <= n_candidates; ++c) {
    const float alpha_c = (float)((double)m * (double)c / (double)n_candidates);
    const double step = (double)alpha_c / (double)L;
    double score = 0.0;
    for (int b = 0; b < B; ++b) {
      const double xb = ((double)b + 0.5) * width;
      double q = nearbyint(xb / step);
      if (q < lo) q = lo;
      if (q > hi) q = hi;
      const double e = xb - q * step;
      score += (double)h[b] * e * e;
    }
    if (scores) scores[c - 1] = score;
    if (cbest < 0 || score <= best) { best = score; cbest = c; } /* '<=' : ties to the largest alpha */
  }
  *alpha = (float)((double)m * (double)cbest / (double)n_candidates);
  free(h);
  return 0;
}

int ocs_oracle_clip_mse_exact(const float* T, int64_t n, int bits, int is_signed,
                              int n_candidates, float* alpha, double* scores) {
  if (!T || !alpha || n < 0 || bits < 2 || bits > 8 || n_candidates < 1) return 1;
  const int L = code_limit(bits, is_signed);
  const float m = ocs_oracle_maxabs(T, n);
  if (m == 0.0f) {
    *alpha = 0.0f;
    if (scores) for (int c = 0; c < n_candidates; ++c) scores[c] = 0.0;
    return 0;
  }
  const double lo = is_signed ? -(double)L : 0.0, hi = (double)L;
  double best = 0.0;
  int cbest = -1;
  for (int c = 1; c <= n_candidates; ++c) {
    const float alpha_c = (float)((double)m * (double)c / (double)n_candidates);
    const double step = (double)alpha_c / (double)L;
    double score = 0.0;
    for (int64_t i = 0; i < n; ++i) {
      const double x = (double)T[i];
      double q = nearbyint(x / step);
      if (q < lo) q = lo;
      if (q > hi) q = hi;
      const double e = x - q * step;
      score += e * e;
    }
    if (scores) scores[c - 1] = score;
    if (cbest < 0 || score <= best) { best = score; cbest = c; }
  }
  *alpha = (float)((double)m * (double)cbest / (double)n_candidates);
  return 0;
}

/* ------------------------------------------------------------------ Section 3.3: grid step of the QA split */
/* The half step of the quantization-aware split is half a step of the grid the split tensor will
 * be rounded on, and that grid depends on the split's outcome.  Reading taken ("two-pass rule"):
 * run the greedy loop once with plain halving, take max|W'| of that run, qa_step = that / L
 * (one fp32 division, L = 2^(bits-1) - 1), then run the loop again with d = qa_step / 2. */
int ocs_oracle_split_qa(const float* W, int O, int C, int R, int S, int qa_bits, float* W_out,
                        int32_t* idx_map, int32_t* split_order, float* max_abs3) {
  if (qa_bits < 2 || qa_bits > 8) return 1;
  float mx[2] = {0.0f, 0.0f};
  int rc = split_common(W, O, C, R, S, 0.0f, W_out, idx_map, split_order, mx, 1);
  if (rc) return rc;
  volatile float step = mx[1] / (float)code_limit(qa_bits, 1);
  rc = split_common(W, O, C, R, S, step, W_out, idx_map, split_order, mx, 1);
  if (rc) return rc;
  if (max_abs3) { max_abs3[0] = mx[0]; max_abs3[1] = mx[1]; max_abs3[2] = step; }
  return 0;
}

/* ------------------------------------------------------------------ Section 4.3: KL clip search */
/* histogram of |x| exactly as in the MSE search */
static uint64_t* abs_histogram(const float* T, int64_t n, int B, float m) {
  uint64_t* h = (uint64_t*)calloc((size_t)B, sizeof(uint64_t));
  if (!h) return NULL;
  volatile float invw = (float)B / m;
  for (int64_t i = 0; i < n; ++i) {
    volatile float t = fabsf(T[i]) * invw;
    int b = (int)t;
    if (b > B - 1) b = B - 1;
    h[b] += 1;
  }
  return h;
}

/* The paper describes the method only in general terms (histogram, candidate thresholds,
 * divergence between the float and the quantized distribution, a little probability mass moved
 * into empty bins so that the divergence is defined).  Reading taken, for candidate c of the
 * same candidate list as the MSE search (alpha_c = max * c / n_candidates):
 *   the first n_c = ceil(c * B / n_candidates) bins lie inside the threshold;
 *   P: those bins' counts, with the count of everything beyond them added to the last one
 *      (clipped values saturate), divided by the total count;
 *   Q: the same bins WITHOUT the clipped mass, quantized and expanded again: bin i belongs to
 *      level j(i) = clamp(rint(x_i / step_c)) (x_i the bin centre, step_c = alpha_c / L); a level's
 *      count is spread evenly over its non-empty bins; divided by the kept count;
 *   the only bin where P > 0 and Q = 0 can be the last one (empty itself, but holding clipped
 *      mass): it then gets eps = 1e-4 and every other entry of Q is scaled by (1 - eps);
 *   score_c = sum over bins with P > 0 of P * ln(P / Q), bins ascending, in double.
 * Smallest score wins, ties to the largest threshold; a candidate that keeps no value at all
 * scores +infinity. */
int ocs_oracle_clip_kl(const float* T, int64_t n, int bits, int is_signed, int n_bins,
                       int n_candidates, float* alpha, float* max_abs, uint64_t* hist,
                       double* scores) {
  if (!T || !alpha || n < 0 || bits < 2 || bits > 8 || n_bins < 1 || n_candidates < 1) return 1;
  const int L = code_limit(bits, is_signed);
  const int B = n_bins;
  const float m = ocs_oracle_maxabs(T, n);
  if (max_abs) *max_abs = m;
  if (m == 0.0f) {
    *alpha = 0.0f;
    if (hist) { memset(hist, 0, sizeof(uint64_t) * (size_t)B); hist[0] = (uint64_t)n; }
    if (scores) for (int c = 0; c < n_candidates; ++c) scores[c] = 0.0;
    return 0;
  }
  uint64_t* h = abs_histogram(T, n, B, m);
  uint64_t* level_count = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(L + 1));
  int* level_bins = (int*)malloc(sizeof(int) * (size_t)(L + 1));
  int* level_of = (int*)malloc(sizeof(int) * (size_t)B);
  if (!h || !level_count || !level_bins || !level_of) {
    free(h); free(level_count); free(level_bins); free(level_of);
    return 2;
  }
  if (hist) memcpy(hist, h, sizeof(uint64_t) * (size_t)B);
  uint64_t total = 0;
  for (int b = 0; b < B; ++b) total += h[b];
  const double width = (double)m / (double)B;
  const double eps = 1e-4;
  double best = 0.0;
  int cbest = -1;
  for (int c = 1; c <= n_candidates; ++c) {
    const float alpha_c = (float)((double)m * (double)c / (double)n_candidates);
    const double step = (double)alpha_c / (double)L;
    int nc = (int)(((int64_t)c * B + n_candidates - 1) / n_candidates);
    if (nc < 1) nc = 1;
    if (nc > B) nc = B;
    uint64_t kept = 0;
    for (int j = 0; j <= L; ++j) { level_count[j] = 0; level_bins[j] = 0; }
    for (int b = 0; b < nc; ++b) {
      const double xb = ((double)b + 0.5) * width;
      double q = nearbyint(xb / step);
      if (q < 0.0) q = 0.0;
      if (q > (double)L) q = (double)L;
      level_of[b] = (int)q;
      kept += h[b];
      level_count[(int)q] += h[b];
      if (h[b] > 0) level_bins[(int)q] += 1;
    }
    double score;
    if (kept == 0) {
      score = INFINITY;
    } else {
      const uint64_t clipped = total - kept;
      const int smooth = (h[nc - 1] == 0 && clipped > 0);
      score = 0.0;
      for (int b = 0; b < nc; ++b) {
        const uint64_t pb = h[b] + (b == nc - 1 ? clipped : 0);
        if (pb == 0) continue;
        const double p = (double)pb / (double)total;
        double q;
        if (h[b] == 0) {
          q = eps; /* the last bin: empty itself, but clipped values land on it */
        } else {
          const int j = level_of[b];
          q = ((double)level_count[j] / (double)level_bins[j]) / (double)kept;
          if (smooth) q = q * (1.0 - eps);
        }
        score += p * log(p / q);
      }
    }
    if (scores) scores[c - 1] = score;
    if (cbest < 0 || score <= best) { best = score; cbest = c; }
  }
  *alpha = (float)((double)m * (double)cbest / (double)n_candidates);
  free(h); free(level_count); free(level_bins); free(level_of);
  return 0;
}

/* ------------------------------------------------------------------ Section 4.2: ACIQ */
/* The threshold, in units of the fitted scale, that minimises the model error
 *     E(alpha) = (clipping noise of the fitted density beyond alpha) + step^2 / 12,
 * step = 2 * alpha / n_intervals (a uniform grid of n_intervals steps across [-alpha, alpha]).
 *   Laplace(0, b):  clipping noise 2 b^2 e^(-alpha/b);  dE/dalpha = 0  <=>  t e^t = 3 n_intervals^2,
 *                   t = alpha / b  (a Lambert-W value), solved by Newton on t + ln t = ln(3 n^2).
 *   Gauss(0, s):    clipping noise 2 [(s^2 + alpha^2) Qf(t) - alpha s phi(t)], t = alpha / s;
 *                   dE/dalpha = 0  <=>  4 [phi(t) - t Qf(t)] = 2 t / (3 n_intervals^2), by bisection
 *                   (the left side falls, the right side rises).
 * With 2^M intervals this is the published analysis of the method; the paper's grid of 2^M - 1
 * points has n_intervals = 2 L. */
double ocs_oracle_aciq_multiplier(double n_intervals, int laplace) {
  if (!(n_intervals > 0.0)) return 0.0;
  const double z = 3.0 * n_intervals * n_intervals;
  if (laplace) {
    const double lz = log(z);
    double t = lz > 1.0 ? lz : 1.0;
    for (int it = 0; it < 100; ++it) {
      const double g = t + log(t) - lz;
      const double tn = t - g / (1.0 + 1.0 / t);
      if (fabs(tn - t) <= 1e-16 * fabs(tn)) { t = tn; break; }
      t = tn > 1e-300 ? tn : 1e-300;
    }
    return t;
  }
  double lo = 0.0, hi = 40.0;
  for (int it = 0; it < 200; ++it) {
    const double t = 0.5 * (lo + hi);
    const double phi = exp(-0.5 * t * t) / sqrt(2.0 * M_PI);
    const double tail = 0.5 * erfc(t / sqrt(2.0));
    const double f = 4.0 * (phi - t * tail) - 2.0 * t / z;
    if (f > 0.0) lo = t; else hi = t;
  }
  return 0.5 * (lo + hi);
}

/* Reading taken (the paper gives no formula): the two candidate densities are zero-location and
 * are fitted to the histogram of |x| (same bins as the other searches, bin centres x_i):
 * b = sum h x_i / n, s = sqrt(sum h x_i^2 / n), the sums taken exactly in integers (x_i is an odd
 * multiple of half a bin width; n up to 2^38 values).  The density with
 * the larger likelihood at its own fit is taken: Laplace iff b / s < sqrt(pi / (2 e)).
 * alpha = multiplier(2 L) * (b or s), rounded to fp32, and never above max|x|.
 * stats (nullable) = {b, s, 1 if Laplace else 0, multiplier}. */
int ocs_oracle_clip_aciq(const float* T, int64_t n, int bits, int is_signed, int n_bins,
                         float* alpha, float* max_abs, uint64_t* hist, double* stats) {
  if (!T || !alpha || n < 0 || bits < 2 || bits > 8 || n_bins < 1) return 1;
  const int L = code_limit(bits, is_signed);
  const int B = n_bins;
  const float m = ocs_oracle_maxabs(T, n);
  if (max_abs) *max_abs = m;
  if (m == 0.0f) {
    *alpha = 0.0f;
    if (hist) { memset(hist, 0, sizeof(uint64_t) * (size_t)B); hist[0] = (uint64_t)n; }
    if (stats) { stats[0] = stats[1] = stats[2] = stats[3] = 0.0; }
    return 0;
  }
  uint64_t* h = abs_histogram(T, n, B, m);
  if (!h) return 2;
  if (hist) memcpy(hist, h, sizeof(uint64_t) * (size_t)B);
  /* moments of the bin centres x_i = (2i + 1) * width / 2 as exact integer sums (order-free):
   * sum h x_i = I1 * width / 2, sum h x_i^2 = I2 * width^2 / 4 */
  const double width = (double)m / (double)B;
  uint64_t cnt = 0, I1 = 0, I2 = 0;
  for (int b = 0; b < B; ++b) {
    const uint64_t odd = 2u * (uint64_t)b + 1u;
    cnt += h[b];
    I1 += h[b] * odd;
    I2 += h[b] * odd * odd;
  }
  free(h);
  const double bb = ((double)I1 / (2.0 * (double)cnt)) * width;
  const double sd = sqrt((double)I2 / (4.0 * (double)cnt)) * width;
  const int laplace = bb / sd < sqrt(M_PI / (2.0 * M_E));
  const double mult = ocs_oracle_aciq_multiplier(2.0 * (double)L, laplace);
  float a = (float)(mult * (laplace ? bb : sd));
  if (!(a < m)) a = m;
  *alpha = a;
  if (stats) { stats[0] = bb; stats[1] = sd; stats[2] = (double)laplace; stats[3] = mult; }
  return 0;
}

/* ------------------------------------------------------------------ Section 3.4: knapsack allocation */
/* curve[s] = max|W'| after s greedy plain-halving splits, s = 0..S_max: what the allocation's
 * reward is made of.  The channel maxima are all the greedy loop sees under plain halving. */
int ocs_oracle_range_curve(const float* W, int O, int C, int R, int S_max, float* curve) {
  if (!W || !curve || O <= 0 || C <= 0 || R <= 0 || S_max < 0) return 1;
  float* cmax = (float*)malloc(sizeof(float) * (size_t)(C + S_max));
  if (!cmax) return 2;
  for (int j = 0; j < C; ++j) cmax[j] = channel_maxabs(W, O, C, R, j);
  for (int s = 0; s <= S_max; ++s) {
    const int alive = C + s;
    int jbest = 0;
    float best = -1.0f;
    for (int j = 0; j < alive; ++j)
      if (cmax[j] > best) { best = cmax[j]; jbest = j; }
    curve[s] = best;
    if (s == S_max) break;
    volatile float half = best * 0.5f;
    cmax[jbest] = half;
    cmax[alive] = half;
  }
  free(cmax);
  return 0;
}

/* Section 3.4's alternative to ceil(r*C) per layer: choose the split counts of all layers at once.
 * reward_l(s) = (curve_l[0] - curve_l[s]) / curve_l[0], the fraction by which s splits shrink the
 * layer's dynamic range (0 for an all-zero layer); cost_l(s) = s * unit_cost[l] weight elements
 * (unit_cost = O * R, one more input channel).  Maximise sum_l reward_l(s_l) subject to
 * sum_l cost_l(s_l) <= budget, 0 <= s_l <= s_max[l]: a multiple-choice knapsack, solved exactly by
 * dynamic programming over the budget in units of gcd(unit_cost): layers in order,
 * best_l[b] = max over s (ascending; a later s must be strictly better) of
 * best_{l-1}[b - s * cost] + reward_l(s), in double.  curves holds the layers' curves back to back
 * (layer l at curve_off[l], s_max[l] + 1 entries).  S_out[l] = chosen count; *total_reward may be
 * NULL.  The paper states the objective and the constraint, not the solver: parity unpinned beyond
 * optimality. */
static int64_t gcd64(int64_t a, int64_t b) { while (b) { int64_t t = a % b; a = b; b = t; } return a; }

int ocs_oracle_knapsack(int n_layers, const float* curves, const int64_t* curve_off,
                        const int32_t* s_max, const int64_t* unit_cost, int64_t budget,
                        int32_t* S_out, double* total_reward) {
  if (n_layers <= 0 || !curves || !curve_off || !s_max || !unit_cost || !S_out || budget < 0) return 1;
  int64_t g = 0;
  for (int l = 0; l < n_layers; ++l) {
    if (unit_cost[l] <= 0 || s_max[l] < 0) return 1;
    g = gcd64(g, unit_cost[l]);
  }
  const int64_t Bu = budget / g; /* budget in units (a remainder cannot be spent) */
  if (Bu > (int64_t)1 << 26) return 3;
  double* prev = (double*)calloc((size_t)(Bu + 1), sizeof(double));
  double* cur = (double*)malloc(sizeof(double) * (size_t)(Bu + 1));
  int32_t* choice = (int32_t*)malloc(sizeof(int32_t) * (size_t)n_layers * (size_t)(Bu + 1));
  if (!prev || !cur || !choice) { free(prev); free(cur); free(choice); return 2; }
  for (int l = 0; l < n_layers; ++l) {
    const float* cv = curves + curve_off[l];
    const int64_t cu = unit_cost[l] / g;
    const double c0 = (double)cv[0];
    for (int64_t b = 0; b <= Bu; ++b) {
      double best = prev[b]; /* s = 0: reward 0 */
      int32_t sbest = 0;
      for (int s = 1; s <= s_max[l]; ++s) {
        if ((int64_t)s * cu > b) break;
        const double reward = c0 > 0.0 ? (c0 - (double)cv[s]) / c0 : 0.0;
        const double v = prev[b - (int64_t)s * cu] + reward;
        if (v > best) { best = v; sbest = s; }
      }
      cur[b] = best;
      choice[(size_t)l * (size_t)(Bu + 1) + (size_t)b] = sbest;
    }
    double* t = prev; prev = cur; cur = t;
  }
  if (total_reward) *total_reward = prev[Bu];
  int64_t b = Bu;
  for (int l = n_layers - 1; l >= 0; --l) {
    const int32_t sc = choice[(size_t)l * (size_t)(Bu + 1) + (size_t)b];
    S_out[l] = sc;
    b -= (int64_t)sc * (unit_cost[l] / g);
  }
  free(prev); free(cur); free(choice);
  return 0;
}

/* ------------------------------------------------------------------ Eq. 2 / Eq. 3 on codes */
static inline int32_t act_code(const void* A, int a_signed, size_t i) {
  return a_signed ? (int32_t)((const int8_t*)A)[i] : (int32_t)((const uint8_t*)A)[i];
}

static inline float dequant(int32_t acc, float a_scale, float w_scale, float bias) {
  volatile float s = a_scale * w_scale; /* one rounded multiply */
  return fmaf((float)acc, s, bias);
}

static int qlinear_one(const void* A, int a_signed, int C, const int8_t* Wc, int S,
                       const int32_t* idx_map, int m, int n, int32_t* out) {
  const int K = C + S;
  int64_t acc = 0;
  for (int j = 0; j < K; ++j) {
    const int src = idx_map[j];
    if (src < 0 || src >= C) return 3;
    acc += (int64_t)act_code(A, a_signed, (size_t)m * C + src) * (int64_t)Wc[(size_t)n * K + j];
  }
  if (acc > INT32_MAX || acc < INT32_MIN) return 4;
  *out = (int32_t)acc;
  return 0;
}

int ocs_oracle_qlinear(const void* A, int a_signed, float a_scale, int M, int C,
                       const int8_t* Wc, float w_scale, int N, int S, const int32_t* idx_map,
                       const float* bias, float* Y, int32_t* acc) {
  if (!A || !Wc || !idx_map || M < 0 || C <= 0 || N < 0 || S < 0) return 1;
  int err = 0;
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      int32_t v = 0;
      int e = qlinear_one(A, a_signed, C, Wc, S, idx_map, m, n, &v);
      if (e) {
#pragma omp atomic write
        err = e;
        continue;
      }
      if (acc) acc[(size_t)m * N + n] = v;
      if (Y) Y[(size_t)m * N + n] = dequant(v, a_scale, w_scale, bias ? bias[n] : 0.0f);
    }
  return err;
}

int ocs_oracle_qlinear_samples(const void* A, int a_signed, float a_scale, int M, int C,
                               const int8_t* Wc, float w_scale, int N, int S,
                               const int32_t* idx_map, const float* bias, const int32_t* ms,
                               const int32_t* ns, int count, float* Y, int32_t* acc) {
  if (!A || !Wc || !idx_map || !ms || !ns || C <= 0 || S < 0 || count < 0) return 1;
  for (int i = 0; i < count; ++i) {
    if (ms[i] < 0 || ms[i] >= M || ns[i] < 0 || ns[i] >= N) return 1;
    int32_t v = 0;
    int e = qlinear_one(A, a_signed, C, Wc, S, idx_map, ms[i], ns[i], &v);
    if (e) return e;
    if (acc) acc[i] = v;
    if (Y) Y[i] = dequant(v, a_scale, w_scale, bias ? bias[ns[i]] : 0.0f);
  }
  return 0;
}

int ocs_oracle_qconv(const void* X, int a_signed, float a_scale, int Nb, int H, int Wd, int C,
                     const int8_t* Wc, float w_scale, int O, int S, int kh, int kw, int stride,
                     int pad, const int32_t* idx_map, const float* bias, float* Y, int32_t* acc) {
  if (!X || !Wc || !idx_map || Nb < 0 || H <= 0 || Wd <= 0 || C <= 0 || O <= 0 || S < 0 ||
      kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
    return 1;
  const int K = C + S;
  const int Ho = (H + 2 * pad - kh) / stride + 1;
  const int Wo = (Wd + 2 * pad - kw) / stride + 1;
  if (Ho <= 0 || Wo <= 0) return 1;
  for (int j = 0; j < K; ++j)
    if (idx_map[j] < 0 || idx_map[j] >= C) return 3;
  int err = 0;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < Nb; ++n)
    for (int oh = 0; oh < Ho; ++oh)
      for (int ow = 0; ow < Wo; ++ow)
        for (int o = 0; o < O; ++o) {
          int64_t a = 0;
          for (int y = 0; y < kh; ++y)
            for (int x = 0; x < kw; ++x) {
              const int ih = oh * stride + y - pad, iw = ow * stride + x - pad;
              if (ih < 0 || ih >= H || iw < 0 || iw >= Wd) continue; /* zero padding */
              const size_t px = (((size_t)n * H + ih) * Wd + iw) * C;
              for (int j = 0; j < K; ++j)
                a += (int64_t)act_code(X, a_signed, px + idx_map[j]) *
                     (int64_t)Wc[(((size_t)o * K + j) * kh + y) * kw + x];
            }
          if (a > INT32_MAX || a < INT32_MIN) {
#pragma omp atomic write
            err = 4;
            continue;
          }
          const size_t oi = (((size_t)n * Ho + oh) * Wo + ow) * O + o;
          if (acc) acc[oi] = (int32_t)a;
          if (Y) Y[oi] = dequant((int32_t)a, a_scale, w_scale, bias ? bias[o] : 0.0f);
        }
  return err;
}

/* ------------------------------------------------------------------ folding duplicated codes */
int64_t ocs_oracle_fold_duplicates(const int8_t* Wc, int N, int C, int R, int S,
                                   const int32_t* idx_map, int8_t* Wf) {
  if (!Wc || !Wf || !idx_map || N <= 0 || C <= 0 || R <= 0 || S < 0) return -1;
  for (int j = 0; j < C + S; ++j)
    if (idx_map[j] < 0 || idx_map[j] >= C) return -1;
  int64_t overflow = 0;
  for (int n = 0; n < N; ++n)
    for (int i = 0; i < C; ++i)
      for (int r = 0; r < R; ++r) {
        int sum = 0;
        for (int j = 0; j < C + S; ++j)
          if (idx_map[j] == i) sum += Wc[((size_t)n * (C + S) + j) * R + r];
        if (sum > 127) { sum = 127; ++overflow; }
        if (sum < -128) { sum = -128; ++overflow; }
        Wf[((size_t)n * C + i) * R + r] = (int8_t)sum;
      }
  return overflow;
}

/* ------------------------------------------------------------------ Section 5.3: static activation OCS */
static int cmp_float_asc(const void* a, const void* b) {
  const float x = *(const float*)a, y = *(const float*)b;
  return (x > y) - (x < y);
}

int ocs_oracle_act_select(const float* P, int64_t rows, int C, int S, double quantile,
                          int32_t* sel, int64_t* counts, float* thr) {
  if (!P || !sel || rows <= 0 || C <= 0 || S < 0 || S > C) return 1;
  if (!(quantile > 0.0) || !(quantile <= 1.0)) return 1;
  const int64_t n = rows * (int64_t)C;
  float* v = (float*)malloc(sizeof(float) * (size_t)n);
  int64_t* cnt = (int64_t*)calloc((size_t)C, sizeof(int64_t));
  char* taken = (char*)calloc((size_t)C, 1);
  if (!v || !cnt || !taken) { free(v); free(cnt); free(taken); return 2; }
  for (int64_t i = 0; i < n; ++i) v[i] = fabsf(P[i]);
  qsort(v, (size_t)n, sizeof(float), cmp_float_asc);
  int64_t k = (int64_t)ceil(quantile * (double)n - 1e-9);
  if (k < 1) k = 1;
  if (k > n) k = n;
  const float t = v[k - 1];
  for (int64_t m = 0; m < rows; ++m)
    for (int c = 0; c < C; ++c)
      if (fabsf(P[m * C + c]) > t) cnt[c] += 1;
  for (int s = 0; s < S; ++s) {
    int best = -1;
    for (int c = 0; c < C; ++c)
      if (!taken[c] && (best < 0 || cnt[c] > cnt[best])) best = c;
    taken[best] = 1;
    sel[s] = best;
  }
  if (counts) memcpy(counts, cnt, sizeof(int64_t) * (size_t)C);
  if (thr) *thr = t;
  free(v); free(cnt); free(taken);
  return 0;
}

int ocs_oracle_act_split_static(const float* A, int64_t rows, int C, int S, const int32_t* sel,
                                float* A_out, int32_t* idx_map) {
  if (!A || !A_out || !idx_map || rows <= 0 || C <= 0 || S < 0 || S > C || (S > 0 && !sel)) return 1;
  char* chosen = (char*)calloc((size_t)C, 1);
  if (!chosen) return 2;
  for (int s = 0; s < S; ++s) {
    if (sel[s] < 0 || sel[s] >= C || chosen[sel[s]]) { free(chosen); return 1; }
    chosen[sel[s]] = 1;
  }
  for (int c = 0; c < C; ++c) idx_map[c] = c;
  for (int s = 0; s < S; ++s) idx_map[C + s] = sel[s];
  for (int64_t m = 0; m < rows; ++m) {
    const float* a = A + m * C;
    float* o = A_out + m * (int64_t)(C + S);
    for (int c = 0; c < C; ++c) o[c] = chosen[c] ? a[c] * 0.5f : a[c];
    for (int s = 0; s < S; ++s) o[C + s] = a[sel[s]] * 0.5f;
  }
  free(chosen);
  return 0;
}

/* ------------------------------------------------------------------ glue */
void ocs_oracle_relu(const float* x, int64_t n, float* y) {
  for (int64_t i = 0; i < n; ++i) y[i] = x[i] > 0.0f ? x[i] : 0.0f;
}

void ocs_oracle_add_relu(const float* a, const float* b, int64_t n, int relu, float* y) {
  for (int64_t i = 0; i < n; ++i) {
    volatile float s = a[i] + b[i];
    y[i] = (relu && !(s > 0.0f)) ? 0.0f : s;
  }
}

void ocs_oracle_maxpool3x3s2(const float* x, int Nb, int H, int Wd, int C, float* y) {
  const int Ho = (H + 2 - 3) / 2 + 1, Wo = (Wd + 2 - 3) / 2 + 1;
  for (int n = 0; n < Nb; ++n)
    for (int oh = 0; oh < Ho; ++oh)
      for (int ow = 0; ow < Wo; ++ow)
        for (int c = 0; c < C; ++c) {
          float m = -INFINITY;
          for (int dy = 0; dy < 3; ++dy)
            for (int dx = 0; dx < 3; ++dx) {
              const int ih = oh * 2 + dy - 1, iw = ow * 2 + dx - 1;
              if (ih < 0 || ih >= H || iw < 0 || iw >= Wd) continue; /* padding never wins */
              const float v = x[(((size_t)n * H + ih) * Wd + iw) * C + c];
              if (v > m) m = v;
            }
          y[(((size_t)n * Ho + oh) * Wo + ow) * C + c] = m;
        }
}

void ocs_oracle_global_avgpool(const float* x, int Nb, int H, int Wd, int C, float* y) {
  volatile float inv = 1.0f / (float)(H * Wd);
  for (int n = 0; n < Nb; ++n)
    for (int c = 0; c < C; ++c) {
      volatile float s = 0.0f;
      for (int h = 0; h < H; ++h)
        for (int w = 0; w < Wd; ++w) s = s + x[(((size_t)n * H + h) * Wd + w) * C + c];
      y[(size_t)n * C + c] = s * inv;
    }
}

void ocs_oracle_nchw_to_nhwc(const float* x, int Nb, int C, int H, int Wd, float* y) {
  for (int n = 0; n < Nb; ++n)
    for (int c = 0; c < C; ++c)
      for (int h = 0; h < H; ++h)
        for (int w = 0; w < Wd; ++w)
          y[(((size_t)n * H + h) * Wd + w) * C + c] = x[(((size_t)n * C + c) * H + h) * Wd + w];
}

/* exp(x) for x <= 0 clamped at -87: t = x*log2(e), n = rint(t), f = t - n in [-0.5, 0.5],
 * 2^f by a degree-6 Taylor polynomial in f*ln2 evaluated with fmaf (Horner), scaled by 2^n. */
static float exp_neg(float x) {
  if (x < -87.0f) x = -87.0f;
  volatile float t = x * 1.44269504088896341f;
  const float n = nearbyintf(t);
  volatile float f = t - n;
  volatile float g = f * 0.693147180559945309f;
  float p = 1.0f / 720.0f;
  p = fmaf(p, g, 1.0f / 120.0f);
  p = fmaf(p, g, 1.0f / 24.0f);
  p = fmaf(p, g, 1.0f / 6.0f);
  p = fmaf(p, g, 0.5f);
  p = fmaf(p, g, 1.0f);
  p = fmaf(p, g, 1.0f);
  return ldexpf(p, (int)n);
}

float ocs_oracle_sigmoid(float x) {
  /* 1/(1+e^-|x|) on the negative side, mirrored */
  const float e = exp_neg(-fabsf(x));
  volatile float den = 1.0f + e;
  volatile float s = 1.0f / den;        /* sigmoid(|x|) */
  if (x >= 0.0f) return s;
  volatile float r = e / den;           /* sigmoid(-|x|) */
  return r;
}

float ocs_oracle_tanh(float x) {
  volatile float a = -2.0f * fabsf(x);
  const float e = exp_neg(a);
  volatile float num = 1.0f - e;
  volatile float den = 1.0f + e;
  volatile float r = num / den;
  return x < 0.0f ? -r : r;
}

void ocs_oracle_lstm_cell(const float* g_ih, const float* g_hh, int batch, int hidden, float* c,
                          float* h) {
  for (int b = 0; b < batch; ++b)
    for (int k = 0; k < hidden; ++k) {
      const size_t base = (size_t)b * 4 * hidden;
      volatile float zi = g_ih[base + k] + g_hh[base + k];
      volatile float zf = g_ih[base + hidden + k] + g_hh[base + hidden + k];
      volatile float zg = g_ih[base + 2 * hidden + k] + g_hh[base + 2 * hidden + k];
      volatile float zo = g_ih[base + 3 * hidden + k] + g_hh[base + 3 * hidden + k];
      const float i = ocs_oracle_sigmoid(zi), f = ocs_oracle_sigmoid(zf);
      const float g = ocs_oracle_tanh(zg), o = ocs_oracle_sigmoid(zo);
      volatile float ig = i * g;
      const float cn = fmaf(f, c[(size_t)b * hidden + k], ig);
      c[(size_t)b * hidden + k] = cn;
      volatile float hn = o * ocs_oracle_tanh(cn);
      h[(size_t)b * hidden + k] = hn;
    }
}
