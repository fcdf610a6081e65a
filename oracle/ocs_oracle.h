/*
 * CPU checker ("oracle") for outlier channel splitting (OCS) post-training quantization,
 * Zhao et al., ICML 2019 (arXiv:1901.09504).
 *
 * THIS IS TEST INFRASTRUCTURE, not a product path: a plain, slow, scalar restatement of
 * what the paper defines, used only to check the CUDA library and as a timed CPU baseline.
 * It shares no code, header, table or helper with the CUDA library.
 *
 * Conventions: weights are fp32 [O][C][R] (O outputs, C input channels, R = kh*kw taps,
 * R = 1 for fully-connected layers); "channel" always means INPUT channel (Section 3.2:
 * splitting one weight adds a whole row / all filters connected to that channel).
 * L = 2^(k-1) - 1 for signed k-bit codes (2^k - 1 grid points, Eq. 1), 2^k - 1 for
 * unsigned codes.  All functions return 0 on success, non-zero on a bad argument.
 *
 * Pinned by tests (paper facts, closed forms, brute force): split, quantize, clip_mse,
 * clip_mse_exact, clip_kl (as the function defined here), clip_aciq (the closed forms), qlinear,
 * qconv, fold_duplicates, pools, relu/add, act_select, act_split_static, range_curve, knapsack
 * (optimality).  Parity unpinned (conventions the paper does not fix, enforced only
 * checker-vs-GPU): the QA grid-step policy (split_qa), the unsigned activation grid, the bin
 * count and the tie rule of the clip searches, the construction of the two distributions of
 * clip_kl and its smoothing constant, the density test and the histogram moments of clip_aciq,
 * the reward sum and the tie rule of knapsack, the LSTM cell's sigmoid/tanh routines, the
 * quantile convention of act_select (nearest rank on |a|; the paper says only which percentile).
 */
#ifndef OCS_ORACLE_H
#define OCS_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Section 3.4: a layer with C channels gets ceil(r*C) splits.  Evaluated in double with a
 * 1e-9 guard so that products that are integral in exact arithmetic (0.02*650 = 13) do not
 * round up to the next integer. */
int ocs_oracle_num_splits(int C, double ratio);

/* Section 3.4 + Eq. 3 + Section 3.3: S times, find the channel holding the largest |w| of
 * the current tensor (ties: smallest current channel index), duplicate it; the copy left in
 * place becomes fl(fl(w - d) * 0.5) and the appended copy (index C + s) fl(fl(w + d) * 0.5),
 * d = qa_step / 2 (qa_step = 0: plain halving, the Net2WiderNet rule).
 * W_out is dense [O][C+S][R]; idx_map[C+S] gives each expanded channel's ORIGINAL source
 * channel; split_order[S] the expanded index chosen at each step; max_abs[0] = max|W|,
 * max_abs[1] = max|W_out|.  split_order / max_abs may be NULL.
 * The literal version rescans the whole tensor at every step; the cached version keeps a
 * per-channel max and rescans only the two touched channels (same result, usable at
 * fc6 size). */
int ocs_oracle_split_literal(const float* W, int O, int C, int R, int S, float qa_step,
                             float* W_out, int32_t* idx_map, int32_t* split_order, float* max_abs);
int ocs_oracle_split_cached(const float* W, int O, int C, int R, int S, float qa_step,
                            float* W_out, int32_t* idx_map, int32_t* split_order, float* max_abs);

/* max |x| over n values (0 for n = 0). */
float ocs_oracle_maxabs(const float* T, int64_t n);

/* Eq. 1 with the threshold alpha in place of max|x| (Section 4: clipping = threshold, then
 * linear quantization): step = alpha / L, inv = L / alpha (fp32 divisions),
 * code = clamp(rint(x * inv), -L, L) with round-half-to-even; unsigned: clamp to [0, L_u].
 * alpha = 0 gives all-zero codes and scale 0.  codes holds the uint8 bit pattern when
 * is_signed = 0.  *scale = step. */
int ocs_oracle_quantize(const float* T, int64_t n, int bits, int is_signed, float alpha,
                        int8_t* codes, float* scale);

/* Section 4.1: histogram of |x| with n_bins bins on [0, max|x|] (bin = min(B-1,
 * trunc(|x| * (B / max)))), candidates alpha_c = max * c / n_candidates, c = 1..n_candidates;
 * score_c = sum_b h[b] * (x_b - Q_c(x_b))^2 in double, bins ascending, x_b the bin centre;
 * returns the alpha with the smallest score (ties: largest alpha).  hist [n_bins] and
 * scores [n_candidates] may be NULL.  *alpha = 0 if the tensor is all zero. */
int ocs_oracle_clip_mse(const float* T, int64_t n, int bits, int is_signed, int n_bins,
                        int n_candidates, float* alpha, float* max_abs, uint64_t* hist,
                        double* scores);

/* The same candidates scored on the elements themselves (no histogram):
 * score_c = sum_i (x_i - Q_c(x_i))^2 in double, elements in storage order. */
int ocs_oracle_clip_mse_exact(const float* T, int64_t n, int bits, int is_signed,
                              int n_candidates, float* alpha, double* scores);

/* The split with the grid step of the quantization-aware rule chosen by the two-pass rule
 * (Section 3.3 leaves open which grid the half step refers to): a plain-halving run of the
 * greedy loop predicts max|W'|, qa_step = that / L(qa_bits) in fp32, and the loop is run again
 * with that step.  max_abs3 (nullable) = max|W|, max|W'|, qa_step. */
int ocs_oracle_split_qa(const float* W, int O, int C, int R, int S, int qa_bits, float* W_out,
                        int32_t* idx_map, int32_t* split_order, float* max_abs3);

/* Section 4.3: clip threshold by KL divergence, on the histogram and candidate list of the MSE
 * search.  For candidate c the first n_c = ceil(c * n_bins / n_candidates) bins are inside the
 * threshold; P = their counts with the clipped count added to the last of them; Q = their
 * counts without it, grouped into the quantization levels of their bin centres and spread back
 * evenly over each level's non-empty bins; both normalised; if the last bin is empty but takes
 * clipped mass, Q gets 1e-4 there and is scaled by (1 - 1e-4) elsewhere; score_c = sum P ln(P/Q)
 * in double, bins ascending.  Smallest score wins, ties to the largest threshold. */
int ocs_oracle_clip_kl(const float* T, int64_t n, int bits, int is_signed, int n_bins,
                       int n_candidates, float* alpha, float* max_abs, uint64_t* hist,
                       double* scores);

/* Section 4.2 (ACIQ): which of a zero-location Laplace or Gauss density fits the histogram of |x|
 * better (likelihood at the fitted scale: Laplace iff b / s < sqrt(pi / (2e)), b = mean |x|,
 * s = sqrt(mean x^2), both from the bin centres), then the threshold that minimises
 * (clipping noise of that density) + step^2 / 12 in closed form: alpha = multiplier * scale,
 * capped at max|x|.  stats (nullable) = {b, s, Laplace?, multiplier}.
 * ocs_oracle_aciq_multiplier(n_intervals, laplace): the minimiser alpha / scale for a uniform grid
 * of n_intervals steps across [-alpha, alpha] (the paper's 2^M - 1 grid points: n_intervals = 2L). */
double ocs_oracle_aciq_multiplier(double n_intervals, int laplace);
int ocs_oracle_clip_aciq(const float* T, int64_t n, int bits, int is_signed, int n_bins,
                         float* alpha, float* max_abs, uint64_t* hist, double* stats);

/* Section 3.4, knapsack allocation.  range_curve: curve[s] = max|W'| after s greedy plain-halving
 * splits (s = 0..S_max).  knapsack: split counts for all layers at once, maximising the summed
 * fractional reduction of each layer's dynamic range, (curve[0] - curve[s]) / curve[0], subject to
 * sum_l S_out[l] * unit_cost[l] <= budget (weight elements; unit_cost = O * R) and
 * S_out[l] <= s_max[l]; exact dynamic programme (ties: fewer splits in the later layer). */
int ocs_oracle_range_curve(const float* W, int O, int C, int R, int S_max, float* curve);
int ocs_oracle_knapsack(int n_layers, const float* curves, const int64_t* curve_off,
                        const int32_t* s_max, const int64_t* unit_cost, int64_t budget,
                        int32_t* S_out, double* total_reward);

/* Eq. 2 / Eq. 3 on integer codes: acc[m][n] = sum_{j < C+S} A[m][idx_map[j]] * Wc[n][j]
 * (exact, checked to fit int32), Y = fmaf((float)acc, a_scale * w_scale, bias[n]).
 * A [M][C] (uint8 when a_signed = 0), Wc dense [N][C+S] int8.  bias, Y, acc may be NULL. */
int ocs_oracle_qlinear(const void* A, int a_signed, float a_scale, int M, int C,
                       const int8_t* Wc, float w_scale, int N, int S, const int32_t* idx_map,
                       const float* bias, float* Y, int32_t* acc);
/* The same for `count` sampled outputs (ms[i], ns[i]). */
int ocs_oracle_qlinear_samples(const void* A, int a_signed, float a_scale, int M, int C,
                               const int8_t* Wc, float w_scale, int N, int S,
                               const int32_t* idx_map, const float* bias, const int32_t* ms,
                               const int32_t* ns, int count, float* Y, int32_t* acc);

/* Convolution form of Eq. 2 / Eq. 3 ("an entire 2D activation channel and all 2D filters
 * connected to it", Section 3.2): X codes NHWC [Nb][H][Wd][C]; Wc dense [O][C+S][kh][kw];
 * acc[(n,oh,ow)][o] = sum_{kh,kw,j} X[n][oh*s+kh-p][ow*s+kw-p][idx_map[j]] * Wc[o][j][kh][kw],
 * zero outside the image; Y NHWC fp32 [Nb][Ho][Wo][O] with the same epilogue as qlinear. */
int ocs_oracle_qconv(const void* X, int a_signed, float a_scale, int Nb, int H, int Wd, int C,
                     const int8_t* Wc, float w_scale, int O, int S, int kh, int kw, int stride,
                     int pad, const int32_t* idx_map, const float* bias, float* Y, int32_t* acc);

/* Folding the duplicates back (Eq. 3 read right to left on the integer codes): the copies of a
 * split channel all multiply the same activation, so Wf[n][i][r] = sum over j with
 * idx_map[j] = i of Wc[n][j][r] gives the same accumulators without any gather.
 * Wc dense [N][C+S][R] int8 -> Wf dense [N][C][R] int8.  Returns the number of sums that left
 * [-128, 127] (those entries are saturated), or -1 on a bad argument. */
int64_t ocs_oracle_fold_duplicates(const int8_t* Wc, int N, int C, int R, int S,
                                   const int32_t* idx_map, int8_t* Wf);

/* Section 5.3, static activation OCS: which channels to split is decided once, on sampled
 * activations P [rows][C].  t = the `quantile` (the paper uses 0.99) quantile of all |a| by
 * nearest rank: the k-th smallest value, k = ceil(quantile * n - 1e-9) clamped to [1, n],
 * n = rows * C.  counts[c] = number of samples of channel c with |a| > t.  sel[0..S) = the S
 * channels with the highest counts (ties: smallest channel index), highest first.  S <= C.
 * counts [C] and thr may be NULL. */
int ocs_oracle_act_select(const float* P, int64_t rows, int C, int S, double quantile,
                          int32_t* sel, int64_t* counts, float* thr);

/* Eq. 4 for a fixed channel list: each channel in sel (distinct, in [0, C)) is duplicated and
 * both copies become fl(a * 0.5); A_out [rows][C+S], the copy of sel[s] at index C + s;
 * idx_map[C+S] as in the weight split. */
int ocs_oracle_act_split_static(const float* A, int64_t rows, int C, int S, const int32_t* sel,
                                float* A_out, int32_t* idx_map);

/* Elementwise / pooling glue of the end-to-end networks, each a single rounded fp32 op per
 * output in a fixed order.  Tensors NHWC. */
void ocs_oracle_relu(const float* x, int64_t n, float* y);
void ocs_oracle_add_relu(const float* a, const float* b, int64_t n, int relu, float* y);
void ocs_oracle_maxpool3x3s2(const float* x, int Nb, int H, int Wd, int C, float* y);
/* sequential sum over (h, w) row-major, then one multiply by 1.0f / (H*Wd) */
void ocs_oracle_global_avgpool(const float* x, int Nb, int H, int Wd, int C, float* y);
void ocs_oracle_nchw_to_nhwc(const float* x, int Nb, int C, int H, int Wd, float* y);

/* LSTM cell, gate order i, f, g, o; z = g_ih + g_hh (each already holding its bias);
 * c' = fmaf(f, c, i * g); h' = o * tanh(c').  sigmoid/tanh are the written-down routines
 * in ocs_oracle.c (exp2-based, fmaf polynomial, one division). */
void ocs_oracle_lstm_cell(const float* g_ih, const float* g_hh, int batch, int hidden,
                          float* c, float* h);
float ocs_oracle_sigmoid(float x);
float ocs_oracle_tanh(float x);

#ifdef __cplusplus
}
#endif
#endif
