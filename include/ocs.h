/*
 * ocs.h -- C ABI of the B200 (sm_100a) library for outlier channel splitting (OCS)
 * post-training quantization, after Zhao et al., "Improving Neural Network Quantization
 * without Retraining using Outlier Channel Splitting", ICML 2019 (arXiv:1901.09504).
 *
 * Common rules for every call
 *  - Every pointer is a DEVICE pointer owned by the caller unless it is marked "host".
 *    The library allocates nothing; scratch memory comes in through (ws, ws_bytes), whose
 *    minimum size the matching *_workspace_bytes() query returns (host call, no GPU work).
 *    ws must be 256-byte aligned.  Inputs are never modified and outputs must not alias inputs,
 *    unless an entry says otherwise (ocs_dup_weight_columns and ocs_add_relu work in place).
 *  - Every call only enqueues work on `stream` (a cudaStream_t passed as void*) and returns
 *    without synchronising.  Scalar results (scales, thresholds, maxima) are written to
 *    device memory.
 *  - The return value reports what the host can see before launching (ocs_status).
 *    Conditions only the device can see are OR-ed into the caller's device status word
 *    `dev_status` (OCS_DEV_* bits; may be NULL to ignore); read it with ocs_poll_status().
 *    A kernel that gives up on a bounded wait sets OCS_DEV_TIMEOUT and returns normally.
 *  - There is no CPU fallback: on a machine without an sm_100 GPU the calls return
 *    OCS_ERR_UNSUPPORTED or OCS_ERR_CUDA.
 *
 * Notation: W fp32 [O][C][R] (O outputs, C input channels, R = kh*kw filter taps, R = 1 for
 * fully-connected and LSTM matrices); "channel" = input channel (Section 3.2).  S splits
 * give C+S expanded channels.  L = 2^(k-1)-1 for signed k-bit codes (Eq. 1: 2^k-1 grid
 * points), L_u = 2^k-1 for unsigned codes.
 */
#ifndef OCS_H
#define OCS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  OCS_OK = 0,
  OCS_ERR_INVALID_ARG = 1, /* null pointer, bits outside [2,8], negative ratio, n_candidates < 1 ... */
  OCS_ERR_SHAPE = 2,       /* non-positive dims, leading dimension too small, misaligned pointer / ld */
  OCS_ERR_WORKSPACE = 3,   /* ws NULL, misaligned or smaller than the query result */
  OCS_ERR_UNSUPPORTED = 4, /* device is not sm_100, or a documented size limit is exceeded */
  OCS_ERR_CUDA = 5         /* a CUDA runtime / driver call failed */
} ocs_status;

/* bits of the device status word */
#define OCS_DEV_NONFINITE 1 /* an input held NaN or Inf; outputs unspecified */
#define OCS_DEV_BAD_INDEX 2 /* an idx_map entry was outside [0, C); it was read as channel 0 */
#define OCS_DEV_TIMEOUT 4   /* a bounded pipeline wait expired; outputs unspecified */
#define OCS_DEV_DEPTH 8     /* a channel was re-split more than 63 times under the QA rule */
#define OCS_DEV_OVERFLOW 16 /* a folded sum of duplicated codes left int8; it was saturated */

typedef enum {
  OCS_CLIP_NONE = 0,     /* alpha = max|T| (Eq. 1) */
  OCS_CLIP_MSE = 1,      /* histogram MSE search (Section 4.1) */
  OCS_CLIP_MSE_EXACT = 2,/* the same candidates scored on the elements themselves, no histogram */
  OCS_CLIP_KL = 3,       /* KL-divergence search on the same histogram and candidates (Section 4.3) */
  OCS_CLIP_ACIQ = 4      /* Laplace-or-Gauss fit and closed-form threshold (Section 4.2) */
} ocs_clip_mode;

/* Host helpers ------------------------------------------------------------------------- */

/* Section 3.4: number of splits for a layer with C channels at expansion ratio r,
 * ceil(r*C), evaluated in double as ceil(r*C - 1e-9) so that products that are integers in
 * exact arithmetic do not round up; 0 for r <= 0.  Host only. */
int ocs_num_splits(int C, double ratio);

/* Copies the device status word to *host_out (host pointer) after synchronising `stream`.
 * Returns OCS_ERR_CUDA if the copy fails. */
ocs_status ocs_poll_status(const int* dev_status, void* stream, int* host_out);

/* Version string of the build (host). */
const char* ocs_version(void);

/* Launch accounting and tracing (host; no counterpart in the paper, used by reports) ------
 * ocs_kernel_launches(): number of kernels this process has launched through the library.
 * ocs_trace_start(max_records): from now on every kernel launch of the library is bracketed
 * by a pair of CUDA events on its stream (at most max_records launches are recorded; the
 * events are created on first use and reused).  ocs_trace_stop(rows, capacity): ends the
 * trace, waits for the recorded launches and writes one row per kernel name (launch count,
 * summed device time in ms) into rows[0..capacity); returns the number of rows written, or
 * -1 if an event could not be read.  Tracing is process-wide and meant for one stream at a
 * time; it is off by default and costs nothing then. */
typedef struct {
  char name[48];
  long long launches;
  double total_ms;
} ocs_trace_row;
long long ocs_kernel_launches(void);
ocs_status ocs_trace_start(int max_records);
int ocs_trace_stop(ocs_trace_row* rows, int capacity);

/* ocs_selftest_wait_expiry (no counterpart in the paper; for tests of the failure path) -------
 * Every device-side wait of the library is bounded; when one runs out the kernel sets
 * OCS_DEV_TIMEOUT and returns.  This call shows that path without faulting or hanging anything:
 * it runs the row-staged copy of ocs_split on W [O][C] (C a multiple of 4, rows 16-byte aligned,
 * two rows must fit in shared memory) with no splits, but each CTA never requests its last row
 * group and waits for it for about a millisecond only.  Afterwards *dev_status has
 * OCS_DEV_TIMEOUT set, rows of the dropped groups of W_out are unwritten, no copy is in flight,
 * and the stream and context are as usable as before.  Workspace: ocs_split_workspace_bytes(O, C,
 * 1, 0) + 4*C rounded up to 256. */
ocs_status ocs_selftest_wait_expiry(const float* W, int O, int C, int64_t ld_in, float* W_out,
                                    int64_t ld_out, void* ws, size_t ws_bytes, int* dev_status,
                                    void* stream);

/* ocs_split -------------------------------------------------------------------------------
 * Weight OCS (Section 3.2 Eq. 3, Section 3.3, Section 3.4): S times, take the channel that
 * holds the largest |w| of the CURRENT expanded tensor (ties: the smallest current channel
 * index), duplicate it, and replace every value w of it by the pair
 *      kept in place  : fl(fl(w - d) * 0.5)        appended at index C+s : fl(fl(w + d) * 0.5)
 * with d = qa_step/2.  d = 0 is plain halving (Net2WiderNet); d = half a quantization step
 * is the quantization-aware split ((w-0.5)/2, (w+0.5)/2) of Section 3.3 in weight units.
 *   qa_bits = 0 : use the given qa_step (>= 0).
 *   qa_bits in [2,8] : the step is chosen on the device: the greedy loop is first run with
 *       d = 0 on the channel extrema, qa_step = (max|W'| predicted by that run) / L(qa_bits),
 *       then the loop is run again with that step (qa_step argument ignored).
 * Layouts: W [O][C][R] with row stride ld_in >= C*R floats; W_out [O][C+S][R] with row
 * stride ld_out >= (C+S)*R floats (when both strides are multiples of 4 and both bases are
 * 16-byte aligned the kernels use 128-bit accesses).  idx_map [C+S]: ORIGINAL source channel of
 * each expanded channel (idx_map[j] = j for j < C).  split_order [S] (nullable): expanded
 * index chosen at each step.  max_abs_out [3] (nullable): max|W|, max|W_out|, qa_step used.
 * Limits: C*R and (C+S)*R below 2^31; S may exceed C.
 * Errors: INVALID_ARG, SHAPE, WORKSPACE as above.  Device flags: NONFINITE, DEPTH. */
size_t ocs_split_workspace_bytes(int O, int C, int R, int S);
ocs_status ocs_split(const float* W, int O, int C, int R, int64_t ld_in, int S, float qa_step,
                     int qa_bits, float* W_out, int64_t ld_out, int32_t* idx_map,
                     int32_t* split_order, float* max_abs_out, void* ws, size_t ws_bytes,
                     int* dev_status, void* stream);

/* ocs_range_curve / ocs_knapsack_allocate ---------------------------------------------------
 * Section 3.4's second way of deciding how many channels each layer may add: instead of
 * ceil(r*C) per layer, the counts of all layers are chosen together as a knapsack problem whose
 * reward is the relative reduction of a layer's dynamic range and whose cost is the memory the
 * extra channels take, under one overall memory constraint.
 *   ocs_range_curve: curve (device, fp32 [S_max+1]), curve[s] = max|W'| after s steps of the
 *   greedy loop with plain halving (curve[0] = max|W|).  W, O, C, R, ld_in as in ocs_split.  One
 *   pass over W plus the split plan on channel maxima.  Device flag: NONFINITE.
 *   ocs_knapsack_allocate: n_layers layers; curves (device) holds their curves back to back,
 *   layer l at element curve_off[l] with s_max[l]+1 entries; unit_cost[l] = weight elements one
 *   more input channel adds to layer l (O*R); curve_off, s_max, unit_cost are HOST arrays, read
 *   before the call returns.  reward_l(s) = (curve_l[0] - curve_l[s]) / curve_l[0] (0 for an
 *   all-zero layer), in double.  S_out (device, int32 [n_layers]) maximises sum_l reward_l(S_out[l])
 *   subject to sum_l S_out[l]*unit_cost[l] <= budget (weight elements) and S_out[l] <= s_max[l]:
 *   exact dynamic programme over the budget in units of gcd(unit_cost), layers in order, a larger
 *   count taken only when strictly better.  total_reward (device, double [1], nullable) = the
 *   optimum.  Limits: budget/gcd <= 2^22, n_layers <= 4096 (else OCS_ERR_UNSUPPORTED).
 *   The paper states objective and constraint only (and reports no gain over the simple rule). */
size_t ocs_range_curve_workspace_bytes(int C, int R, int S_max);
ocs_status ocs_range_curve(const float* W, int O, int C, int R, int64_t ld_in, int S_max, float* curve,
                           void* ws, size_t ws_bytes, int* dev_status, void* stream);
size_t ocs_knapsack_workspace_bytes(int n_layers, const int64_t* unit_cost, int64_t budget);
ocs_status ocs_knapsack_allocate(int n_layers, const float* curves, const int64_t* curve_off,
                                 const int32_t* s_max, const int64_t* unit_cost, int64_t budget,
                                 int32_t* S_out, double* total_reward, void* ws, size_t ws_bytes,
                                 void* stream);

/* ocs_quantize ----------------------------------------------------------------------------
 * k-bit linear quantization (Eq. 1) with the clip threshold alpha in place of max|x|
 * (Section 4): step = alpha/L, inv = L/alpha (fp32), code = clamp(rint(x*inv), -L, L) with
 * round-half-to-even; unsigned (is_signed = 0): clamp to [0, L_u].  Codes live in 8-bit
 * containers for every k (uint8 bit pattern when unsigned).
 *   mode NONE: alpha = max|T|.   mode MSE (Section 4.1): histogram of |x| with n_bins equal
 *   bins on [0, max|T|]; candidates alpha_c = max*c/n_candidates, c = 1..n_candidates;
 *   score_c = sum_b h[b]*(x_b - Q_c(x_b))^2 at the bin centres x_b, in double; the smallest
 *   score wins, ties go to the largest alpha.   mode MSE_EXACT: the same candidates with
 *   score_c = sum_i (x_i - Q_c(x_i))^2 over the elements, in double (the MSE of Section 4.1
 *   without the histogram approximation; bound by fp64 arithmetic, not by memory).  For this
 *   mode n_bins is ignored and the workspace query is called with n_bins = 0.
 *   mode KL (Section 4.3; the paper names the ingredients -- histogram, candidates, divergence
 *   between the float and the quantized distribution, a little mass moved into empty bins --
 *   the details here are this library's): same histogram and candidates as MSE.  Candidate c
 *   keeps the first n_c = ceil(c*n_bins/n_candidates) bins.  P = their counts, with the count of
 *   everything beyond added to the last one, over the total count.  Q = their counts alone,
 *   grouped by the code of the bin centre (clamp(rint(x_b/step_c), 0, L)), each group's count
 *   spread evenly over its non-empty bins, over the kept count; if the last kept bin is empty but
 *   receives clipped mass, Q is 1e-4 there and scaled by (1 - 1e-4) elsewhere.  score_c =
 *   sum over bins with P > 0 of P*ln(P/Q) in double; smallest wins, ties to the largest alpha;
 *   a candidate that keeps no value scores +infinity.
 *   mode ACIQ (Section 4.2: decide between a Gaussian and a Laplacian, then an approximate
 *   closed form for the MSE-optimal threshold; the details are this library's): from the same
 *   histogram, b = mean|x| and s = sqrt(mean x^2) at the bin centres (exact integer sums; up to
 *   2^38 values); Laplace if b/s < sqrt(pi/2e) (the density with the larger likelihood at its own
 *   fit), else Gauss; alpha = t*b resp. t*s, capped at max|T|, where t minimises
 *   (clipping noise of the density) + step^2/12 for the grid of 2L intervals the codes span:
 *   t*exp(t) = 12 L^2 for Laplace, 4*(phi(t) - t*Qf(t)) = t/(6 L^2) for Gauss.  n_candidates is
 *   ignored (the workspace query takes 1).
 * T [rows][cols] fp32 with row stride ld_in; codes [rows][cols] with row stride ld_codes bytes
 * (bytes beyond cols in a row are left untouched).  max_abs_in (nullable): device scalar
 * holding max|T| if the caller already has it (saves one pass over T).  *scale = step,
 * *alpha = chosen threshold (device scalars; alpha nullable).  An all-zero tensor gives zero
 * codes, scale 0, alpha 0.  n_bins <= 4096, n_candidates <= 1024 (ignored for mode NONE).
 * Device flags: NONFINITE. */
size_t ocs_quantize_workspace_bytes(int n_bins, int n_candidates);
ocs_status ocs_quantize(const float* T, int64_t rows, int64_t cols, int64_t ld_in, int bits,
                        int is_signed, ocs_clip_mode mode, int n_candidates, int n_bins,
                        const float* max_abs_in, int8_t* codes, int64_t ld_codes, float* scale,
                        float* alpha, void* ws, size_t ws_bytes, int* dev_status, void* stream);

/* ocs_split_quantize -----------------------------------------------------------------------
 * ocs_split followed by ocs_quantize on its result (the split-then-clip order of Section 5.2;
 * Sections 3.2-3.4, Eq. 1, Section 4.1) in one call that never writes the fp32 W': the
 * expanded rows exist only in shared memory, from where they are histogrammed (mode MSE) and
 * quantized.  W is read three times (extrema, histogram, quantization) instead of W and W'
 * being read and written five times.  Results are bit-identical to the two separate calls:
 * codes int8 [O][(C+S)*R] in the split's layout with row stride ld_codes bytes, idx_map,
 * split_order (nullable), max_abs_out [3] (nullable), *scale, *alpha (nullable).
 * Arguments as in ocs_split and ocs_quantize (modes NONE, MSE, KL and ACIQ).
 * Applied to an ACTIVATION matrix [rows][C] (R = 1, qa_bits = 0) this is the activation side
 * of Eq. 4 with channels chosen on the batch at hand (the per-batch selection of Section 5.3):
 * the chosen channels are duplicated and halved, and the codes come out already expanded,
 * [rows][C+S]; ocs_dup_weight_columns provides the matching weight columns.
 * Limits: W 16-byte aligned, ld_in and C*R multiples of 4, and two expanded rows (plus the
 * histogram) must fit in shared memory ((C+S)*R up to about 27,000 floats); otherwise
 * OCS_ERR_UNSUPPORTED -- use the two separate calls.  Device flags: NONFINITE, DEPTH, TIMEOUT. */
size_t ocs_split_quantize_workspace_bytes(int O, int C, int R, int S, int n_bins, int n_candidates);
ocs_status ocs_split_quantize(const float* W, int O, int C, int R, int64_t ld_in, int S, float qa_step,
                              int qa_bits, int bits, int is_signed, ocs_clip_mode mode, int n_candidates, int n_bins,
                              int8_t* codes, int64_t ld_codes, int32_t* idx_map, int32_t* split_order,
                              float* max_abs_out, float* scale, float* alpha, void* ws, size_t ws_bytes,
                              int* dev_status, void* stream);

/* ocs_split_quantize_batch -------------------------------------------------------------------
 * ocs_split_quantize with plain halving and no clip search (Sections 3.2-3.4, Eq. 1) for all
 * the layers of a network at once: five launches in total instead of five per layer (one
 * extrema pass over all weights, the greedy plans side by side -- one CTA per layer --, one
 * code pass for the short-row layers and one for the long-row layers).  The results of every
 * layer are bit-identical to its own ocs_split_quantize call (qa_step = 0, qa_bits = 0, mode
 * OCS_CLIP_NONE).  layers: HOST array of n_layers descriptors (read before the call returns);
 * W dense [O][C][R]; codes [O][ld_codes]; idx_map [C+S]; scale [1]; max_abs3 [3] nullable.
 * Limits: n_layers <= 64; every layer must satisfy ocs_split_quantize's staging limits (W 16-byte
 * aligned, C*R a multiple of 4, two expanded rows in shared memory), otherwise
 * OCS_ERR_UNSUPPORTED -- prepare that layer with its own call.  Device flags: NONFINITE, TIMEOUT. */
typedef struct {
  const float* W;
  int O, C, R, S;
  int8_t* codes;
  int64_t ld_codes;
  int32_t* idx_map;
  float* scale;
  float* max_abs3;
} ocs_layer_desc;
size_t ocs_split_quantize_batch_workspace_bytes(const ocs_layer_desc* layers, int n_layers);
ocs_status ocs_split_quantize_batch(const ocs_layer_desc* layers, int n_layers, int bits, int is_signed,
                                    void* ws, size_t ws_bytes, int* dev_status, void* stream);

/* ocs_dup_weight_columns ------------------------------------------------------------------
 * Weight side of activation OCS (Eq. 4: the activation channel is halved in both copies, its
 * weights are duplicated unchanged).  W_codes (device) int8 [N][ldw >= (C+S)*R] holds the layer's
 * C weight channels, R taps each, in ocs_split's [channel][tap] order; channels C..C+S-1 are
 * filled in place with W_codes[n][C+s][:] = W_codes[n][idx_map[C+s]][:].  With the expanded
 * activation codes of ocs_split_quantize, ocs_qlinear (or, after ocs_pack_conv_weights,
 * ocs_qconv) called with C+S plain channels and no gather evaluates the split layer.
 * S = 0 is a no-op.  Device flag: BAD_INDEX (a source index outside [0, C); channel 0 is
 * copied instead). */
ocs_status ocs_dup_weight_columns(int8_t* W_codes, int N, int C, int R, int S, int64_t ldw, const int32_t* idx_map,
                                  int* dev_status, void* stream);

/* ocs_fold_duplicates ------------------------------------------------------------------------
 * The copies of a split channel all multiply the same activation (Eq. 3), so their integer codes
 * can be summed back into the source channel: W_folded[n][i][r] = sum over j with idx_map[j] = i
 * of W_codes[n][j][r].  ocs_qlinear / ocs_qconv on W_folded with C plain channels (S = 0, no
 * gather) give the same int32 accumulators as on W_codes with the index map -- while the codes
 * still carry the finer grid the split bought.  W_codes (device) int8 [N][ldw >= (C+S)*R] in
 * ocs_split's [channel][tap] order; W_folded (device) int8 [N][ld_out >= C*R], may not alias
 * W_codes.  Two copies of k <= 7 bit codes always fit; a sum that leaves [-128, 127] (re-split
 * channels, 8-bit codes) is saturated and sets OCS_DEV_OVERFLOW -- the caller then keeps the
 * gathered form.  Workspace (device, 256-byte aligned): ocs_fold_workspace_bytes(C, S).
 * The paper has no counterpart: it duplicates activation channels at run time (Section 3.5). */
size_t ocs_fold_workspace_bytes(int C, int S);
ocs_status ocs_fold_duplicates(const int8_t* W_codes, int N, int C, int R, int S, int64_t ldw, const int32_t* idx_map,
                               int8_t* W_folded, int64_t ld_out, void* ws, size_t ws_bytes, int* dev_status,
                               void* stream);

/* ocs_act_select_channels --------------------------------------------------------------------
 * Static channel choice for activation OCS (Section 5.3: count, per channel, the sampled values
 * above the 99th percentile and split the channels with the highest counts).
 * P (device) fp32 [rows][ldp >= C]: sampled activations, one row per sample or pixel.
 * t = the `quantile` quantile (0 < quantile <= 1; the paper uses 0.99) of all |a| by nearest rank:
 * the k-th smallest, k = ceil(quantile * rows * C - 1e-9) clamped to [1, rows * C] -- exact, found
 * by a radix select over the bit patterns.  counts[c] = samples of channel c with |a| > t.
 * sel (device, int32 [S], S <= C) = the S channels with the highest counts, highest first, ties to
 * the smaller channel index.  counts (device, int64 [C]) and threshold (device, fp32 [1]) may be
 * NULL.  Workspace (device, 256-byte aligned): ocs_act_select_workspace_bytes(C).  Four passes
 * over P; asynchronous on `stream`.  Device flag: NONFINITE (such samples are left out). */
size_t ocs_act_select_workspace_bytes(int C);
ocs_status ocs_act_select_channels(const float* P, int64_t rows, int C, int64_t ldp, int S, double quantile,
                                   int32_t* sel, int64_t* counts, float* threshold, void* ws, size_t ws_bytes,
                                   int* dev_status, void* stream);

/* ocs_act_split_quantize_static --------------------------------------------------------------
 * Activation side of Eq. 4 for a channel list chosen ahead of time (Section 5.3's static variant;
 * the run-time duplication and scaling of the listed channels that Section 3.5 describes), fused with
 * the quantization: A (device) fp32 [rows][ld_in >= C]; every channel in sel (device, int32 [S],
 * distinct, in [0, C)) is duplicated and both copies carry a * 0.5; codes (device, int8 or the uint8
 * bit pattern) [rows][ld_codes >= C+S], the copy of sel[s] at column C + s; idx_map (device,
 * int32 [C+S]) as in ocs_split.  Grid: alpha_in (device, fp32 [1]) when given -- a threshold
 * profiled ahead of time, values beyond it saturate -- else max |a'| of this batch (one extra pass
 * over A).  *scale (device) = alpha / L.  Workspace: ocs_split_quantize_workspace_bytes(rows, C,
 * 1, S, 1, 1).  Same staging limits as ocs_split_quantize (OCS_ERR_UNSUPPORTED otherwise).
 * Device flags: BAD_INDEX (an entry of sel outside [0, C) or listed twice; outputs unspecified),
 * NONFINITE (dynamic grid: non-finite input; static grid: alpha_in negative or non-finite). */
ocs_status ocs_act_split_quantize_static(const float* A, int rows, int C, int64_t ld_in, int S, const int32_t* sel,
                                         int bits, int is_signed, const float* alpha_in, int8_t* codes,
                                         int64_t ld_codes, int32_t* idx_map, float* scale, void* ws, size_t ws_bytes,
                                         int* dev_status, void* stream);

/* ocs_quantize_noalloc ---------------------------------------------------------------------
 * (No counterpart in the paper: a packaging variant of ocs_quantize.)
 * Same operation, arguments and results as ocs_quantize, minus (ws, ws_bytes).  It is meant for
 * callers that cannot obtain device memory where they need to quantize: code that runs inside
 * another framework's execution callback where cudaMalloc is off limits because it stalls the
 * whole device, a serving process that gave all device memory to its own planner at start-up,
 * or a job so close to the memory limit that an allocation may fail.  Such callers still pass
 * the input and output buffers; what they are spared is the scratch.
 * The scratch (48 KB: running maximum, histogram, candidate scores) is a fixed array inside the
 * library's device image, so every GPU that loads the library carries it until the process
 * exits.  The call allocates nothing and frees nothing.
 * Limits: modes OCS_CLIP_NONE, OCS_CLIP_MSE, OCS_CLIP_KL and OCS_CLIP_ACIQ with n_bins <= 4096
 * and n_candidates <= 1024; anything larger, and OCS_CLIP_MSE_EXACT, returns
 * OCS_ERR_UNSUPPORTED (use ocs_quantize).
 * The first call on each device looks up the array's device address (with that device
 * current) and remembers it; make that first call before starting any stream capture.
 * All calls on a device share the one array, which keeps whatever the previous call left: each
 * call re-clears the parts it needs to start from zero, but two calls whose kernels overlap on
 * the GPU (different streams, no ordering between them) race on it -- order them, or use
 * ocs_quantize with separate workspaces. */
ocs_status ocs_quantize_noalloc(const float* T, int64_t rows, int64_t cols, int64_t ld_in, int bits,
                                int is_signed, ocs_clip_mode mode, int n_candidates, int n_bins,
                                const float* max_abs_in, int8_t* codes, int64_t ld_codes, float* scale,
                                float* alpha, int* dev_status, void* stream);

/* Reads back the search's intermediate results after an MSE-mode ocs_quantize on the same
 * workspace (for tests and reports): hist [n_bins] uint64 and scores [n_candidates] double,
 * both device pointers into ws.  Host call, no GPU work. */
void ocs_quantize_workspace_views(void* ws, int n_bins, int n_candidates, uint64_t** hist,
                                  double** scores);

/* ocs_qlinear -----------------------------------------------------------------------------
 * The split layer of Eq. 3 evaluated on integer codes (Eq. 2 on low-precision MACs):
 *     acc[m][n] = sum_{j < C+S} A[m][idx_map[j]] * Wc[n][j]          (int32, exact)
 *     Y[m][n]   = fmaf((float)acc[m][n], a_scale * w_scale, bias[n])  (bias 0 if NULL)
 * The duplicated activation channels (the run-time channel duplication of Section 3.5)
 * are gathered through idx_map while the operand tiles are staged; an expanded activation
 * tensor is never written.  idx_map[j] must equal j for j < C (as ocs_split produces).
 * A_codes_T (nullable), row stride lda_T bytes: a channel-major copy of the same codes, [C][M]
 * (ocs_transpose_codes makes one); lda_T a multiple of 16, at least M, 16-byte aligned.  With it
 * the K-blocks that hold duplicated channels are fetched by the copy engine, one channel row per
 * contraction index, straight into the operand tile -- the gather costs no thread a load.  Without
 * it the producer warps gather those blocks byte by byte from A_codes.
 * A codes [M][C], row stride lda bytes, uint8 when a_signed = 0 else int8; Wc int8 [N][C+S],
 * row stride ldw bytes, ldw a multiple of 16 and Wc 16-byte aligned; a_scale / w_scale
 * device scalars; Y fp32 [M][N] row stride ldy floats; acc_out (nullable) int32 [M][N] with
 * the same stride.  Limits: (C+S) * 255 * 127 must fit int32.
 * Steps that usually follow a layer can be taken in its epilogue: residual (device, fp32, the
 * shape and row stride of Y, may be NULL) is added to Y with one rounded addition (a block's
 * shortcut connection; it may not alias Y), relu != 0 then stores max(., 0), and max_abs_out (device, fp32 [1], may be NULL) receives max |Y| of
 * the stored output -- the next layer's activation grid (ocs_quantize's max_abs_in).
 * Device flags: BAD_INDEX, TIMEOUT. */
size_t ocs_qlinear_workspace_bytes(int M, int N, int C, int S);
ocs_status ocs_qlinear(const void* A_codes, const void* A_codes_T, int64_t lda_T, int a_signed,
                       const float* a_scale, int M, int C, int64_t lda, const int8_t* W_codes,
                       const float* w_scale, int N, int S, int64_t ldw, const int32_t* idx_map,
                       const float* bias, float* Y, int64_t ldy, int32_t* acc_out,
                       const float* residual, int relu, float* max_abs_out, void* ws, size_t ws_bytes,
                       int* dev_status, void* stream);

/* ocs_transpose_codes: codes_T[c][r] = codes[r][c] for 8-bit codes [rows][cols] (row stride ld
 * bytes) -> [cols][rows] (row stride ld_T bytes).  A pure layout change: the channel-major copy of
 * an activation matrix that ocs_qlinear can gather whole channels from. */
ocs_status ocs_transpose_codes(const void* codes, int64_t rows, int64_t cols, int64_t ld,
                               void* codes_T, int64_t ld_T, void* stream);

/* ocs_selftest_force_gemm_plan (no counterpart in the paper; for tests) ----------------------
 * ocs_qlinear / ocs_qconv choose the output tile width and, for problems with few tiles, how
 * many CTAs share a tile and split its K range (their partial sums are exchanged through
 * distributed shared memory).  The int32 accumulators must not depend on that choice.  This
 * process-wide hook fixes the choice for the following calls (bn in {64, 128, 256}, split_k in
 * {1, 2, 4, 8}; a split that does not fit the problem falls back to a smaller one) so that a test
 * can run one problem under several plans; bn = 0 returns the choice to the planner.  Host call. */
ocs_status ocs_selftest_force_gemm_plan(int bn, int split_k);

/* ocs_pack_conv_weights -------------------------------------------------------------------
 * Reorders quantized conv weights from the split's layout [O][C+S][kh*kw] (row stride
 * ld_src bytes) into the contraction order ocs_qconv consumes: for each output o, first the
 * C original channels of every tap, k = tap*Cp + c, then the S duplicated channels of every
 * tap, k = kh*kw*Cp + tap*S + s.  Cp is the per-tap stride: C, except that a C that is a
 * multiple of 16 but not of 128 is padded up to the next multiple of 128 (zero weights), so
 * that the activation tiles of such layers can be fetched as whole tiles.  Row stride ld_dst
 * bytes (multiple of 16, at least ocs_conv_packed_k); bytes between the last k and ld_dst are
 * set to zero.  A pure permutation (plus zero padding) of Eq. 3's terms.
 * ocs_conv_packed_k (host): the packed contraction length kh*kw*(Cp + S). */
int64_t ocs_conv_packed_k(int C, int S, int kh, int kw);
ocs_status ocs_pack_conv_weights(const int8_t* codes, int O, int C, int S, int kh, int kw,
                                 int64_t ld_src, int8_t* packed, int64_t ld_dst, void* stream);

/* ocs_pack_conv_weights_batch: ocs_pack_conv_weights for up to 64 layers in one launch (the
 * reordering of a whole network's convolutions after ocs_split_quantize_batch).  jobs: HOST array,
 * read before the call returns; fields as the arguments of ocs_pack_conv_weights. */
typedef struct {
  const int8_t* codes;
  int O, C, S, kh, kw;
  int64_t ld_src;
  int8_t* packed;
  int64_t ld_dst;
} ocs_pack_desc;
ocs_status ocs_pack_conv_weights_batch(const ocs_pack_desc* jobs, int n_jobs, void* stream);

/* ocs_qconv -------------------------------------------------------------------------------
 * Convolution form of ocs_qlinear (Section 3.2: a split duplicates a whole 2-D activation
 * channel and all filters connected to it):
 *   acc[(n,oh,ow)][o] = sum_{kh,kw} sum_{j<C+S} X[n][oh*s+kh-p][ow*s+kw-p][idx_map[j]] * W'[o][j][kh][kw]
 * with zeros outside the image, and the same fp32 epilogue.  X codes NHWC [Nb][H][Wd][C]
 * (dense, 16-byte aligned when C is a multiple of 16); W_packed from ocs_pack_conv_weights with row
 * stride ldw bytes; Y fp32 NHWC [Nb][Ho][Wo][O] dense; acc_out (nullable) int32, same shape.
 * residual, relu and max_abs_out as in ocs_qlinear.  A layer whose pixels TMA cannot address (C not a
 * multiple of 16 bytes) is run over its patch matrix, which is built in the workspace.
 * Device flags: BAD_INDEX, TIMEOUT. */
size_t ocs_qconv_workspace_bytes(int Nb, int H, int Wd, int C, int O, int S, int kh, int kw,
                                 int stride, int pad);
ocs_status ocs_qconv(const void* X_codes, int a_signed, const float* a_scale, int Nb, int H,
                     int Wd, int C, const int8_t* W_packed, const float* w_scale, int O, int S,
                     int kh, int kw, int stride, int pad, int64_t ldw, const int32_t* idx_map,
                     const float* bias, float* Y, int32_t* acc_out, const float* residual, int relu,
                     float* max_abs_out, void* ws, size_t ws_bytes, int* dev_status, void* stream);

/* Steps between quantized layers ------------------------------------------------------------
 * The paper runs whole networks through the split and quantized layers (Section 5: ImageNet
 * CNNs; Section 6: a two-layer LSTM language model).  These calls are the float steps between
 * the layers; each output element is produced by single IEEE-rounded fp32 operations in a
 * fixed order, so a network's activations are reproducible bit for bit.  Tensors are dense;
 * images are NHWC.  All pointers device, all calls asynchronous on `stream`.
 *
 * ocs_add_relu: y[i] = a[i] + b[i] (b NULL: y[i] = a[i]), then max(., 0) when relu != 0
 *   (ReLU after a layer; the residual connection of a bottleneck block).  y may equal a.
 *   max_abs_out (device, fp32 [1], may be NULL) receives max |y| of the whole tensor: the next
 *   layer's activation grid (pass it to ocs_quantize as max_abs_in), taken here to save a pass.
 *   A NaN in y does not enter the maximum (ocs_quantize flags non-finite input itself).
 * ocs_maxpool3x3s2: 3x3 window, stride 2, padding 1 (padding never wins);
 *   y [Nb][(H-1)/2+1][(Wd-1)/2+1][C].
 * ocs_global_avgpool: y[n][c] = (sum over (h, w), row-major, sequential) * (1 / (H*Wd)).
 * ocs_nchw_to_nhwc: layout change of the network input.
 * ocs_embedding: out[t][:] = table[ids[t]][:], table [V][E]; an id outside [0, V) reads row 0
 *   and sets OCS_DEV_BAD_INDEX.
 * ocs_lstm_cell (Section 6's LSTM): gates g_ih, g_hh [batch][4*hidden] in the order i, f, g, o,
 *   each already holding its bias; z = g_ih + g_hh; c <- fmaf(sigmoid(z_f), c, sigmoid(z_i) *
 *   tanh(z_g)); h <- sigmoid(z_o) * tanh(c); c [batch][hidden] updated in place, h written.
 *   sigmoid and tanh are fixed routines: e = exp(-|x|) resp. exp(-2|x|) computed as 2^n * P(f ln 2)
 *   with t = x * log2(e), n = rint(t), f = t - n, P the degree-6 Taylor polynomial of exp in
 *   Horner form with fused multiply-adds (x clamped at -87); sigmoid = 1/(1+e) or e/(1+e),
 *   tanh = (1-e)/(1+e) with the sign of x; divisions IEEE. */
ocs_status ocs_add_relu(const float* a, const float* b, int64_t n, int relu, float* y, float* max_abs_out,
                        void* stream);
ocs_status ocs_maxpool3x3s2(const float* x, int Nb, int H, int Wd, int C, float* y, void* stream);
ocs_status ocs_global_avgpool(const float* x, int Nb, int H, int Wd, int C, float* y, void* stream);
ocs_status ocs_nchw_to_nhwc(const float* x, int Nb, int C, int H, int Wd, float* y, void* stream);
ocs_status ocs_embedding(const float* table, const int32_t* ids, int64_t n, int V, int E, float* out,
                         int* dev_status, void* stream);
ocs_status ocs_lstm_cell(const float* g_ih, const float* g_hh, int batch, int hidden, float* c, float* h,
                         void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OCS_H */
