// ocs_quantize: k-bit linear quantization (Eq. 1) with an optional MSE clip-threshold search
// (Section 4.1).
//
// Kernels (each a streaming pass over T in tiles of one row segment of 4096 columns):
//   maxabs_kernel     max|x|, combined with atomicMax on the bits of the non-negative value
//   hist_kernel       histogram of |x| in privatised shared-memory counters, flushed with 64-bit atomics
//   score_kernel      one CTA per candidate threshold: sum_b h[b]*(x_b - Q(x_b))^2 in double
//   kl_score_kernel   one CTA per candidate threshold: KL divergence between the kept part of the histogram
//                     (clipped mass added to its last bin) and its quantized-and-expanded form (Section 4.3)
//   aciq_kernel       Laplace-or-Gauss fit to the histogram and the closed-form threshold (Section 4.2)
//   quantize_kernel   picks the winning threshold (smallest score, ties to the largest threshold), then
//                     code = clamp(rint(x * L/alpha)), round-half-to-even, saturating
#include "common.cuh"

namespace ocs {
namespace {

constexpr int kTileQuads = 4;                     // float4 per thread per tile
constexpr int kTileCols = 256 * 4 * kTileQuads;   // 4096 columns per tile
constexpr int kMaxBins = 4096;
constexpr int kMaxCandidates = 1024;
constexpr int kHistCopies = 2;

struct View {
  const float* T;
  long long rows, cols, ld;
  long long tiles_per_row, tiles;
  bool vec;  // 128-bit loads allowed
};

View make_view(const float* T, int64_t rows, int64_t cols, int64_t ld) {
  View v;
  v.T = T;
  if (ld == cols) {  // dense: one long row
    v.rows = 1; v.cols = rows * cols; v.ld = rows * cols;
    v.vec = aligned(T, 16);
  } else {
    v.rows = rows; v.cols = cols; v.ld = ld;
    v.vec = aligned(T, 16) && (ld % 4 == 0);
  }
  v.tiles_per_row = (v.cols + kTileCols - 1) / kTileCols;
  v.tiles = v.rows * v.tiles_per_row;
  return v;
}

// Grid of a tile-strided kernel: one resident wave at most.
template <typename K>
int grid_for(K kernel, long long tiles, size_t dyn_smem = 0) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, 256, dyn_smem) != cudaSuccess || per_sm < 1)
    per_sm = 4;
  const long long cap = (long long)kNumSMs * per_sm;
  return (int)(tiles < cap ? (tiles > 0 ? tiles : 1) : cap);
}

// A CTA's walk over its tiles (blockIdx.x, blockIdx.x + gridDim.x, ...) without per-tile divisions.
struct TileWalk {
  long long row, seg;     // current tile: row and tile index inside the row
  long long drow, dseg;   // gridDim.x tiles further = drow rows and dseg tiles
  long long left;         // tiles still to visit (including the current one)
  __device__ TileWalk(const View& v) {
    row = blockIdx.x / v.tiles_per_row;
    seg = blockIdx.x - row * v.tiles_per_row;
    drow = gridDim.x / v.tiles_per_row;
    dseg = gridDim.x - drow * v.tiles_per_row;
    left = (long long)blockIdx.x < v.tiles ? (v.tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
  }
  __device__ void next(const View& v) {
    row += drow;
    seg += dseg;
    if (seg >= v.tiles_per_row) { seg -= v.tiles_per_row; ++row; }
    --left;
  }
};

// The thread's kTileQuads quads of the current tile.  x[u] holds quad u, n[u] how many of its four
// values exist (0..4); c[u] is the quad's first column inside the tile.
__device__ __forceinline__ void load_tile(const View& v, const TileWalk& w, float4 x[kTileQuads], int n[kTileQuads]) {
  const long long col0 = w.seg * kTileCols;
  const float* base = v.T + w.row * v.ld + col0;
  const long long rest = v.cols - col0;
  if (v.vec && rest >= kTileCols) {          // a full tile: unconditional 128-bit loads
#pragma unroll
    for (int u = 0; u < kTileQuads; ++u) {
      x[u] = __ldcs(reinterpret_cast<const float4*>(base) + u * 256 + threadIdx.x);
      n[u] = 4;
    }
    return;
  }
  const int nt = (int)(rest < kTileCols ? rest : kTileCols);
#pragma unroll
  for (int u = 0; u < kTileQuads; ++u) {
    const int c = (u * 256 + threadIdx.x) * 4;
    n[u] = max(0, min(4, nt - c));
    x[u] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    if (n[u] == 4 && v.vec) {
      x[u] = __ldcs(reinterpret_cast<const float4*>(base + c));
    } else if (n[u] > 0) {
      x[u].x = __ldcs(base + c);
      if (n[u] > 1) x[u].y = __ldcs(base + c + 1);
      if (n[u] > 2) x[u].z = __ldcs(base + c + 2);
      if (n[u] > 3) x[u].w = __ldcs(base + c + 3);
    }
  }
}

__global__ void __launch_bounds__(256) maxabs_kernel(View v, unsigned int* maxbits) {
  float m = 0.0f;
  for (TileWalk w(v); w.left > 0; w.next(v)) {
    float4 x[kTileQuads];
    int n[kTileQuads];
    load_tile(v, w, x, n);
#pragma unroll
    for (int u = 0; u < kTileQuads; ++u)   // missing values were loaded as 0: they cannot raise the maximum
      m = fmaxf(m, fmaxf(fmaxf(fabsf(x[u].x), fabsf(x[u].y)), fmaxf(fabsf(x[u].z), fabsf(x[u].w))));
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float red[8];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]);
    atomicMax(maxbits, __float_as_uint(m));  // m >= 0: bit order is value order
  }
}

__global__ void __launch_bounds__(256)
hist_kernel(View v, const float* __restrict__ maxp, int n_bins, unsigned long long* __restrict__ hist) {
  extern __shared__ unsigned int sh[];  // kHistCopies * n_bins
  for (int i = threadIdx.x; i < kHistCopies * n_bins; i += 256) sh[i] = 0u;
  __syncthreads();
  const float m = *maxp;
  if (m > 0.0f) {
    const float invw = __fdiv_rn((float)n_bins, m);
    unsigned int* mine = sh + ((threadIdx.x >> 5) % kHistCopies) * n_bins;
    const int last = n_bins - 1;
    auto count = [&](float xv) {
      atomicAdd(&mine[hist_bin(xv, invw, last)], 1u);
    };
    for (TileWalk w(v); w.left > 0; w.next(v)) {
      float4 x[kTileQuads];
      int n[kTileQuads];
      load_tile(v, w, x, n);
#pragma unroll
      for (int u = 0; u < kTileQuads; ++u) {
        if (n[u] == 4) {
          count(x[u].x); count(x[u].y); count(x[u].z); count(x[u].w);
        } else {
          if (n[u] > 0) count(x[u].x);
          if (n[u] > 1) count(x[u].y);
          if (n[u] > 2) count(x[u].z);
        }
      }
    }
  }
  __syncthreads();
  for (int b = threadIdx.x; b < n_bins; b += 256) {
    unsigned int c = 0u;
#pragma unroll
    for (int k = 0; k < kHistCopies; ++k) c += sh[k * n_bins + b];
    if (c) atomicAdd(&hist[b], (unsigned long long)c);
  }
}

// grid = n_candidates, block = 256.  Fixed per-thread bin assignment and a fixed reduction tree:
// the result does not depend on scheduling.
__global__ void __launch_bounds__(256)
score_kernel(const unsigned long long* __restrict__ hist, const float* __restrict__ maxp, int n_bins,
             int n_candidates, int L, int is_signed, double* __restrict__ scores) {
  __shared__ double red[256];
  const int c = blockIdx.x + 1;
  const float m = *maxp;
  double acc = 0.0;
  if (m > 0.0f) {
    const float alpha_c = __double2float_rn(__ddiv_rn(__dmul_rn((double)m, (double)c), (double)n_candidates));
    const double step = __ddiv_rn((double)alpha_c, (double)L);
    const double width = __ddiv_rn((double)m, (double)n_bins);
    const double lo = is_signed ? -(double)L : 0.0, hi = (double)L;
    for (int b = threadIdx.x; b < n_bins; b += 256) {
      const double xb = __dmul_rn(__dadd_rn((double)b, 0.5), width);
      double q = rint(__ddiv_rn(xb, step));
      q = fmin(fmax(q, lo), hi);
      const double e = __dsub_rn(xb, __dmul_rn(q, step));
      acc = __dadd_rn(acc, __dmul_rn(__dmul_rn((double)hist[b], e), e));
    }
  }
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] = __dadd_rn(red[threadIdx.x], red[threadIdx.x + s]);
    __syncthreads();
  }
  if (threadIdx.x == 0) scores[blockIdx.x] = red[0];
}

// Section 4.3, KL divergence search on the histogram of |x| and the candidate list of the MSE search.
// Candidate c keeps the first n_c = ceil(c * n_bins / n_candidates) bins.  P = their counts, the clipped count
// added to the last one (clipped values saturate there), over the total; Q = their counts alone, grouped by the
// quantization level of the bin centre (level = clamp(rint(x_b / step_c), 0, L)) and spread back evenly over each
// level's non-empty bins, over the kept count.  Q can only be zero where P is not in the last kept bin (empty
// itself but receiving clipped mass): that bin then gets kEps of Q's mass and the rest is scaled by 1 - kEps.
// score_c = sum_{P > 0} P ln(P / Q).  Level sums are integers (exact, order-free); the terms are added in a fixed
// per-thread order and a fixed tree.  A candidate that keeps nothing scores +infinity.
constexpr int kMaxLevels = 256;
constexpr double kKlEps = 1e-4;

__global__ void __launch_bounds__(256)
kl_score_kernel(const unsigned long long* __restrict__ hist, const float* __restrict__ maxp, int n_bins,
                int n_candidates, int L, double* __restrict__ scores) {
  __shared__ unsigned long long level_count[kMaxLevels];
  __shared__ int level_bins[kMaxLevels];
  __shared__ unsigned long long red_u[2][8];
  __shared__ double red[256];
  const int c = blockIdx.x + 1;
  const float m = *maxp;
  if (!(m > 0.0f)) {
    if (threadIdx.x == 0) scores[blockIdx.x] = 0.0;
    return;
  }
  const float alpha_c = __double2float_rn(__ddiv_rn(__dmul_rn((double)m, (double)c), (double)n_candidates));
  const double step = __ddiv_rn((double)alpha_c, (double)L);
  const double width = __ddiv_rn((double)m, (double)n_bins);
  int nc = (int)(((long long)c * n_bins + n_candidates - 1) / n_candidates);
  nc = max(1, min(nc, n_bins));
  for (int j = threadIdx.x; j <= L; j += 256) { level_count[j] = 0ull; level_bins[j] = 0; }
  __syncthreads();
  unsigned long long tot = 0ull, kept = 0ull;
  for (int b = threadIdx.x; b < n_bins; b += 256) {
    const unsigned long long h = hist[b];
    tot += h;
    if (b < nc) {
      kept += h;
      const double xb = __dmul_rn(__dadd_rn((double)b, 0.5), width);
      const int lvl = (int)fmin(fmax(rint(__ddiv_rn(xb, step)), 0.0), (double)L);
      if (h) { atomicAdd(&level_count[lvl], h); atomicAdd(&level_bins[lvl], 1); }
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    tot += __shfl_xor_sync(0xffffffffu, tot, o);
    kept += __shfl_xor_sync(0xffffffffu, kept, o);
  }
  if ((threadIdx.x & 31) == 0) { red_u[0][threadIdx.x >> 5] = tot; red_u[1][threadIdx.x >> 5] = kept; }
  __syncthreads();
  tot = 0ull; kept = 0ull;
  for (int w = 0; w < 8; ++w) { tot += red_u[0][w]; kept += red_u[1][w]; }
  if (kept == 0ull) {
    if (threadIdx.x == 0) scores[blockIdx.x] = INFINITY;
    return;
  }
  const unsigned long long clipped = tot - kept;
  const bool smooth = hist[nc - 1] == 0ull && clipped > 0ull;
  double acc = 0.0;
  for (int b = threadIdx.x; b < nc; b += 256) {
    const unsigned long long h = hist[b];
    const unsigned long long pb = h + (b == nc - 1 ? clipped : 0ull);
    if (pb == 0ull) continue;
    const double p = __ddiv_rn((double)pb, (double)tot);
    double q;
    if (h == 0ull) {
      q = kKlEps;
    } else {
      const double xb = __dmul_rn(__dadd_rn((double)b, 0.5), width);
      const int lvl = (int)fmin(fmax(rint(__ddiv_rn(xb, step)), 0.0), (double)L);
      q = __ddiv_rn(__ddiv_rn((double)level_count[lvl], (double)level_bins[lvl]), (double)kept);
      if (smooth) q = __dmul_rn(q, 1.0 - kKlEps);
    }
    acc = __dadd_rn(acc, __dmul_rn(p, log(__ddiv_rn(p, q))));
  }
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int sft = 128; sft > 0; sft >>= 1) {
    if (threadIdx.x < sft) red[threadIdx.x] = __dadd_rn(red[threadIdx.x], red[threadIdx.x + sft]);
    __syncthreads();
  }
  if (threadIdx.x == 0) scores[blockIdx.x] = red[0];
}

// Section 4.2 (ACIQ).  Zero-location Laplace and Gauss densities are fitted to the histogram of |x| through the
// bin centres x_b = (2b + 1) * width / 2: b_fit = mean |x|, s_fit = sqrt(mean x^2), with the sums taken exactly in
// integers (I1 = sum h (2b+1), I2 = sum h (2b+1)^2: order-free).  The density with the larger likelihood at its own
// fit wins (Laplace iff b_fit / s_fit < sqrt(pi / 2e)); alpha = multiplier * scale, capped at max|x|, where the
// multiplier minimises clipping noise + step^2/12 for a grid of 2L intervals (solved on the host: it depends on
// L only).  One CTA.
__global__ void __launch_bounds__(256)
aciq_kernel(const unsigned long long* __restrict__ hist, const float* __restrict__ maxp, int n_bins,
            double mult_laplace, double mult_gauss, float* __restrict__ alpha_sel) {
  __shared__ unsigned long long red_u[3][8];
  const float m = *maxp;
  unsigned long long cnt = 0ull, i1 = 0ull, i2 = 0ull;
  for (int b = threadIdx.x; b < n_bins; b += 256) {
    const unsigned long long h = hist[b], odd = 2ull * (unsigned long long)b + 1ull;
    cnt += h; i1 += h * odd; i2 += h * odd * odd;
  }
  for (int o = 16; o > 0; o >>= 1) {
    cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    i1 += __shfl_xor_sync(0xffffffffu, i1, o);
    i2 += __shfl_xor_sync(0xffffffffu, i2, o);
  }
  if ((threadIdx.x & 31) == 0) { red_u[0][threadIdx.x >> 5] = cnt; red_u[1][threadIdx.x >> 5] = i1; red_u[2][threadIdx.x >> 5] = i2; }
  __syncthreads();
  if (threadIdx.x != 0) return;
  cnt = 0ull; i1 = 0ull; i2 = 0ull;
  for (int w = 0; w < 8; ++w) { cnt += red_u[0][w]; i1 += red_u[1][w]; i2 += red_u[2][w]; }
  if (!(m > 0.0f) || cnt == 0ull) { *alpha_sel = m > 0.0f ? m : 0.0f; return; }
  const double width = __ddiv_rn((double)m, (double)n_bins);
  const double bfit = __dmul_rn(__ddiv_rn((double)i1, __dmul_rn(2.0, (double)cnt)), width);
  const double sfit = __dmul_rn(sqrt(__ddiv_rn((double)i2, __dmul_rn(4.0, (double)cnt))), width);
  const bool laplace = __ddiv_rn(bfit, sfit) < 0.7601734505331404;   // sqrt(pi / (2 e))
  float a = __double2float_rn(laplace ? __dmul_rn(mult_laplace, bfit) : __dmul_rn(mult_gauss, sfit));
  if (!(a < m)) a = m;
  *alpha_sel = a;
}

// The same candidates scored on the elements themselves (no histogram): score_c = sum_i (x_i - Q_c(x_i))^2
// in double.  A CTA stages tiles of kExactTile elements in shared memory (as double); a thread owns up to
// four candidates and one slice of the tile.  Per-CTA partial sums are combined in a fixed order by
// exact_combine_kernel, so the scores do not depend on scheduling.  Bound by the fp64 pipe (one division
// per element and candidate), not by HBM.
constexpr int kExactTile = 2048;
constexpr int kExactMaxGrid = 2 * kNumSMs;
constexpr int kExactOwn = kMaxCandidates / 256;   // candidates per thread at most

__global__ void __launch_bounds__(256)
exact_score_kernel(View v, const float* __restrict__ maxp, int n_candidates, int L, int is_signed,
                   double* __restrict__ partial) {
  __shared__ double xs[kExactTile];
  __shared__ double comb[256];
  const float m = *maxp;
  int slots = 1;                                   // candidate slots per pass: a power of two <= 256
  while (slots < n_candidates && slots < 256) slots <<= 1;
  const int slices = 256 / slots;
  const int my_slot = threadIdx.x % slots, my_slice = threadIdx.x / slots;
  double step[kExactOwn], acc[kExactOwn];
#pragma unroll
  for (int k = 0; k < kExactOwn; ++k) {
    const int c = my_slot + k * slots + 1;
    acc[k] = 0.0;
    step[k] = 0.0;
    if (c <= n_candidates && m > 0.0f) {
      const float alpha_c = __double2float_rn(__ddiv_rn(__dmul_rn((double)m, (double)c), (double)n_candidates));
      step[k] = __ddiv_rn((double)alpha_c, (double)L);
    }
  }
  const double lo = is_signed ? -(double)L : 0.0, hi = (double)L;
  const long long total = v.rows * v.cols;
  const long long n_tiles = (total + kExactTile - 1) / kExactTile;
  for (long long t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    const long long e0 = t * kExactTile;
    const int cnt = (int)min((long long)kExactTile, total - e0);
    for (int i = threadIdx.x; i < cnt; i += 256) {
      const long long e = e0 + i;
      const long long row = e / v.cols;
      xs[i] = (double)__ldcs(v.T + row * v.ld + (e - row * v.cols));
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kExactOwn; ++k) {
      if (step[k] > 0.0) {
        double a = acc[k];
        for (int i = my_slice; i < cnt; i += slices) {   // ascending element order inside the slice
          const double x = xs[i];
          double q = rint(__ddiv_rn(x, step[k]));
          q = fmin(fmax(q, lo), hi);
          const double err = __dsub_rn(x, __dmul_rn(q, step[k]));
          a = __dadd_rn(a, __dmul_rn(err, err));
        }
        acc[k] = a;
      }
    }
    __syncthreads();
  }
  // slices of one candidate are added in slice order
#pragma unroll
  for (int k = 0; k < kExactOwn; ++k) {
    comb[threadIdx.x] = acc[k];
    __syncthreads();
    const int c = my_slot + k * slots + 1;
    if (my_slice == 0 && c <= n_candidates) {
      double a = comb[my_slot];
      for (int sl = 1; sl < slices; ++sl) a = __dadd_rn(a, comb[sl * slots + my_slot]);
      partial[(size_t)blockIdx.x * n_candidates + (c - 1)] = a;
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(256)
exact_combine_kernel(const double* __restrict__ partial, int n_parts, int n_candidates, double* __restrict__ scores) {
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= n_candidates) return;
  double a = 0.0;
  for (int b = 0; b < n_parts; ++b) a = __dadd_rn(a, partial[(size_t)b * n_candidates + c]);
  scores[c] = a;
}

__global__ void __launch_bounds__(256)
quantize_kernel(View v, const float* __restrict__ alpha_p, const double* __restrict__ scores, int n_candidates, int L,
                int is_signed, int8_t* __restrict__ codes, long long ld_codes, int packed_ok,
                float* __restrict__ scale_out, float* __restrict__ alpha_out, int* dev_status) {
  // alpha_p holds max|T|; with scores given the threshold is the search's winner
  float alpha = *alpha_p;
  if (scores && alpha > 0.0f) alpha = pick_alpha(scores, alpha, n_candidates);
  const bool zero = !(alpha > 0.0f);
  const float step = zero ? 0.0f : __fdiv_rn(alpha, (float)L);
  const float inv = zero ? 0.0f : __fdiv_rn((float)L, alpha);
  const float lo = is_signed ? -(float)L : 0.0f, hi = (float)L;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *scale_out = step;
    if (alpha_out) *alpha_out = zero ? 0.0f : alpha;
  }
  bool bad = false;
  for (TileWalk w(v); w.left > 0; w.next(v)) {
    float4 x[kTileQuads];
    int n[kTileQuads];
    load_tile(v, w, x, n);
    // the dense view flattens rows, so its code offset is the flat index
    int8_t* out_tile = codes + w.row * ld_codes + w.seg * kTileCols;
#pragma unroll
    for (int u = 0; u < kTileQuads; ++u) {
      if (!n[u]) continue;
      bad |= !(is_finite(x[u].x) && is_finite(x[u].y) && is_finite(x[u].z) && is_finite(x[u].w));  // missing = 0
      const unsigned int word = pack4(quant_code(x[u].x, inv, lo, hi), quant_code(x[u].y, inv, lo, hi),
                                      quant_code(x[u].z, inv, lo, hi), quant_code(x[u].w, inv, lo, hi));
      int8_t* out = out_tile + (u * 256 + threadIdx.x) * 4;
      if (packed_ok && n[u] == 4) {
        *reinterpret_cast<unsigned int*>(out) = word;
      } else {
        for (int i = 0; i < n[u]; ++i) out[i] = (int8_t)((word >> (8 * i)) & 0xFFu);
      }
    }
  }
  if (bad) flag(dev_status, OCS_DEV_NONFINITE);
}

// Small tensors without a clip search (the per-step activations of a recurrent network, a classifier's
// input): one launch finds max|x| and writes the codes.  The launch is one thread-block cluster of eight CTAs:
// each takes an eighth of the elements, the eight partial maxima are exchanged through distributed shared
// memory (every CTA stores its maximum into every peer, then one cluster barrier), and each CTA quantizes
// its own eighth -- the second read hits the cache, and a launch of latency is saved where latency is all
// there is.
constexpr long long kSmallQuantElems = 65536;
constexpr int kSmallCluster = 8;
constexpr int kSmallThreads = 512;

__global__ void __launch_bounds__(kSmallThreads)
small_quantize_kernel(const float* __restrict__ T, int rows, int cols, long long ld_in, int L, int is_signed,
                      int8_t* __restrict__ codes, long long ld_codes, float* __restrict__ scale_out,
                      float* __restrict__ alpha_out, unsigned int* __restrict__ maxbits, int* dev_status) {
  __shared__ float red[kSmallThreads / 32];
  __shared__ float peer_max[kSmallCluster];
  uint32_t crank, csize;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(csize));
  const int n = rows * cols;
  const int per = (n + (int)csize - 1) / (int)csize;
  const int i0 = (int)crank * per, i1 = min(n, i0 + per);
  const bool dense = ld_in == cols;
  float m = 0.0f;
  bool bad = false;
#pragma unroll 4
  for (int i = i0 + threadIdx.x; i < i1; i += kSmallThreads) {
    const float x = dense ? T[i] : T[(long long)(i / cols) * ld_in + (i % cols)];
    bad |= !is_finite(x);
    m = fmaxf(m, fabsf(x));
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kSmallThreads / 32; ++w) m = fmaxf(m, red[w]);
    // this CTA's maximum into slot `crank` of every CTA of the cluster
    const uint32_t local = (uint32_t)__cvta_generic_to_shared(&peer_max[crank]);
    for (uint32_t dst = 0; dst < csize; ++dst) {
      uint32_t remote;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(dst));
      asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(m) : "memory");
    }
  }
  // all stores of all CTAs are visible after the cluster barrier (release / acquire)
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
  float alpha = 0.0f;
  for (uint32_t k = 0; k < csize; ++k) alpha = fmaxf(alpha, peer_max[k]);
  const bool zero = !(alpha > 0.0f);
  const float step = zero ? 0.0f : __fdiv_rn(alpha, (float)L);
  const float inv = zero ? 0.0f : __fdiv_rn((float)L, alpha);
  const float lo = is_signed ? -(float)L : 0.0f, hi = (float)L;
  if (crank == 0 && threadIdx.x == 0) {
    *scale_out = step;
    if (alpha_out) *alpha_out = zero ? 0.0f : alpha;
    *maxbits = __float_as_uint(alpha);
  }
  const bool dense_out = dense && ld_codes == cols;
#pragma unroll 4
  for (int i = i0 + threadIdx.x; i < i1; i += kSmallThreads) {
    const int r = i / cols, c = i - r * cols;
    const float x = dense ? T[i] : T[(long long)r * ld_in + c];
    const int8_t q = (int8_t)quant_code(x, inv, lo, hi);
    if (dense_out) codes[i] = q;
    else codes[(long long)r * ld_codes + c] = q;
  }
  if (bad) flag(dev_status, OCS_DEV_NONFINITE);
}

struct QuantWs {
  unsigned int* maxbits;       // fp32 bits of max|T|
  float* alpha_sel;            // ACIQ: the chosen threshold (same 256-byte slot as maxbits)
  unsigned long long* hist;
  double* scores;
  double* partial;             // exact scorer only: [kExactMaxGrid][n_candidates]
  size_t total;
};

QuantWs carve_quant_ws(void* ws, int n_bins, int n_candidates) {
  QuantWs w{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    unsigned char* p = ws ? reinterpret_cast<unsigned char*>(ws) + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  };
  w.maxbits = reinterpret_cast<unsigned int*>(take(256));
  w.alpha_sel = w.maxbits ? reinterpret_cast<float*>(w.maxbits) + 16 : nullptr;
  w.hist = reinterpret_cast<unsigned long long*>(take(8 * (size_t)(n_bins > 0 ? n_bins : 1)));
  w.scores = reinterpret_cast<double*>(take(8 * (size_t)(n_candidates > 0 ? n_candidates : 1)));
  if (n_bins == 0)  // the exact scorer's layout
    w.partial = reinterpret_cast<double*>(take(8 * (size_t)kExactMaxGrid * (size_t)(n_candidates > 0 ? n_candidates : 1)));
  w.total = off;
  return w;
}

}  // namespace

namespace {
// alpha / scale that minimises (clipping noise of the fitted density) + step^2 / 12 for a uniform grid of
// n_int steps across [-alpha, alpha] (Section 4.2; step = 2 alpha / n_int, z = 3 n_int^2).
//   Laplace(0, b): noise 2 b^2 exp(-t), t = alpha / b; stationary point t exp(t) = z, i.e. t = W(z): Halley's
//                  iteration on w exp(w) - z.
//   Gauss(0, s):   noise 2 [(1 + t^2) Qf(t) - t phi(t)] s^2; stationary point F(t) = 4 [phi(t) - t Qf(t)] - 2 t / z
//                  = 0 with F' = -4 Qf(t) - 2 / z < 0: Newton steps kept inside a shrinking bracket.
double aciq_multiplier_host(double n_int, bool laplace) {
  const double z = 3.0 * n_int * n_int;
  if (laplace) {
    double w = log(z) - log(log(z) > 1.0 ? log(z) : 1.0);   // first terms of W's expansion for large z
    if (!(w > 0.1)) w = 0.5;
    for (int it = 0; it < 64; ++it) {
      const double ew = exp(w), f = w * ew - z;
      const double wn = w - f / (ew * (w + 1.0) - (w + 2.0) * f / (2.0 * w + 2.0));
      if (fabs(wn - w) <= 4e-16 * fabs(wn)) { w = wn; break; }
      w = wn;
    }
    return w;
  }
  double lo = 0.0, hi = 40.0, t = 2.0;
  const double inv_sqrt_2pi = 0.3989422804014327, inv_sqrt2 = 0.7071067811865476;
  for (int it = 0; it < 200; ++it) {
    const double tail = 0.5 * erfc(t * inv_sqrt2);
    const double f = 4.0 * (inv_sqrt_2pi * exp(-0.5 * t * t) - t * tail) - 2.0 * t / z;
    if (f > 0.0) lo = t; else hi = t;
    double tn = t - f / (-4.0 * tail - 2.0 / z);
    if (!(tn > lo && tn < hi)) tn = 0.5 * (lo + hi);
    if (fabs(tn - t) <= 4e-16 * fabs(tn)) { t = tn; break; }
    t = tn;
  }
  return t;
}
}  // namespace

// The clip search that follows the histogram: fills scores (MSE, KL) or *alpha_sel (ACIQ).
ocs_status launch_clip_search(ocs_clip_mode mode, const unsigned long long* hist, const float* maxp, int n_bins,
                              int n_candidates, int L, int is_signed, double* scores, float* alpha_sel,
                              cudaStream_t stream) {
  if (mode == OCS_CLIP_MSE) {
    LaunchScope ls("score_kernel", stream);
    score_kernel<<<n_candidates, 256, 0, stream>>>(hist, maxp, n_bins, n_candidates, L, is_signed, scores);
    return launch_status();
  }
  if (mode == OCS_CLIP_KL) {
    LaunchScope ls("kl_score_kernel", stream);
    kl_score_kernel<<<n_candidates, 256, 0, stream>>>(hist, maxp, n_bins, n_candidates, L, scores);
    return launch_status();
  }
  if (mode == OCS_CLIP_ACIQ) {
    // the multipliers depend on the code range only: solved once per L on the host
    static double cache[2][256];
    static bool have[256] = {false};
    if (L < 1 || L > 255) return OCS_ERR_INVALID_ARG;
    if (!have[L]) {
      cache[0][L] = aciq_multiplier_host(2.0 * L, true);
      cache[1][L] = aciq_multiplier_host(2.0 * L, false);
      have[L] = true;
    }
    LaunchScope ls("aciq_kernel", stream);
    aciq_kernel<<<1, 256, 0, stream>>>(hist, maxp, n_bins, cache[0][L], cache[1][L], alpha_sel);
    return launch_status();
  }
  return OCS_ERR_INVALID_ARG;
}

}  // namespace ocs

using namespace ocs;

extern "C" size_t ocs_quantize_workspace_bytes(int n_bins, int n_candidates) {
  return carve_quant_ws(nullptr, n_bins, n_candidates).total;
}

extern "C" void ocs_quantize_workspace_views(void* ws, int n_bins, int n_candidates, uint64_t** hist,
                                             double** scores) {
  const QuantWs w = carve_quant_ws(ws, n_bins, n_candidates);
  if (hist) *hist = reinterpret_cast<uint64_t*>(w.hist);
  if (scores) *scores = w.scores;
}

extern "C" ocs_status ocs_quantize(const float* T, int64_t rows, int64_t cols, int64_t ld_in, int bits, int is_signed,
                                   ocs_clip_mode mode, int n_candidates, int n_bins, const float* max_abs_in,
                                   int8_t* codes, int64_t ld_codes, float* scale, float* alpha, void* ws,
                                   size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!T || !codes || !scale) return OCS_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return OCS_ERR_INVALID_ARG;
  if (mode != OCS_CLIP_NONE && mode != OCS_CLIP_MSE && mode != OCS_CLIP_MSE_EXACT && mode != OCS_CLIP_KL &&
      mode != OCS_CLIP_ACIQ)
    return OCS_ERR_INVALID_ARG;
  const bool hist_mode = mode == OCS_CLIP_MSE || mode == OCS_CLIP_KL || mode == OCS_CLIP_ACIQ;
  if (mode == OCS_CLIP_ACIQ) n_candidates = 1;   // no candidate list
  if (hist_mode && (n_candidates < 1 || n_candidates > kMaxCandidates || n_bins < 1 || n_bins > kMaxBins))
    return OCS_ERR_INVALID_ARG;
  if (mode == OCS_CLIP_MSE_EXACT && (n_candidates < 1 || n_candidates > kMaxCandidates)) return OCS_ERR_INVALID_ARG;
  if (mode == OCS_CLIP_MSE_EXACT) n_bins = 0;
  if (rows <= 0 || cols <= 0 || ld_in < cols || ld_codes < cols) return OCS_ERR_SHAPE;
  if (!aligned(T, 4)) return OCS_ERR_SHAPE;
  if (mode == OCS_CLIP_NONE) { n_bins = 1; n_candidates = 1; }
  const QuantWs w = carve_quant_ws(ws, n_bins, n_candidates);
  if (!ws || !aligned(ws, 256) || ws_bytes < w.total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;

  const View v = make_view(T, rows, cols, ld_in);
  const int L = is_signed ? (1 << (bits - 1)) - 1 : (1 << bits) - 1;

  if (mode == OCS_CLIP_NONE && !max_abs_in && rows * cols <= kSmallQuantElems) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kSmallCluster, 1, 1);
    cfg.blockDim = dim3(kSmallThreads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kSmallCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    LaunchScope ls("small_quantize_kernel", stream);
    const int irows = (int)rows, icols = (int)cols;
    const long long ldi = ld_in, ldc = ld_codes;
    if (cudaLaunchKernelEx(&cfg, small_quantize_kernel, T, irows, icols, ldi, L, is_signed, codes, ldc, scale, alpha,
                           w.maxbits, dev_status) != cudaSuccess)
      return OCS_ERR_CUDA;
    return launch_status();
  }
  const float* maxp = max_abs_in;
  if (!maxp) {
    if (cudaMemsetAsync(w.maxbits, 0, 4, stream) != cudaSuccess) return OCS_ERR_CUDA;
    LaunchScope ls("maxabs_kernel", stream);
    maxabs_kernel<<<grid_for(maxabs_kernel, v.tiles), 256, 0, stream>>>(v, w.maxbits);
    if ((st = launch_status()) != OCS_OK) return st;
    maxp = reinterpret_cast<const float*>(w.maxbits);
  }
  const double* scores = nullptr;
  if (hist_mode) {
    if (cudaMemsetAsync(w.hist, 0, 8 * (size_t)n_bins, stream) != cudaSuccess) return OCS_ERR_CUDA;
    {
      const size_t smem = sizeof(unsigned int) * kHistCopies * n_bins;
      LaunchScope ls("hist_kernel", stream);
      hist_kernel<<<grid_for(hist_kernel, v.tiles, smem), 256, smem, stream>>>(v, maxp, n_bins, w.hist);
    }
    if ((st = launch_status()) != OCS_OK) return st;
    if ((st = launch_clip_search(mode, w.hist, maxp, n_bins, n_candidates, L, is_signed ? 1 : 0, w.scores, w.alpha_sel,
                                 stream)) != OCS_OK)
      return st;
    if (mode == OCS_CLIP_ACIQ) maxp = w.alpha_sel;   // the threshold itself; nothing left to pick
    else scores = w.scores;
  } else if (mode == OCS_CLIP_MSE_EXACT) {
    const long long n_tiles = (v.rows * v.cols + kExactTile - 1) / kExactTile;
    const int grid = (int)(n_tiles < kExactMaxGrid ? n_tiles : kExactMaxGrid);
    {
      LaunchScope ls("exact_score_kernel", stream);
      exact_score_kernel<<<grid, 256, 0, stream>>>(v, maxp, n_candidates, L, is_signed, w.partial);
    }
    if ((st = launch_status()) != OCS_OK) return st;
    {
      LaunchScope ls("exact_combine_kernel", stream);
      exact_combine_kernel<<<(n_candidates + 255) / 256, 256, 0, stream>>>(w.partial, grid, n_candidates, w.scores);
    }
    if ((st = launch_status()) != OCS_OK) return st;
    scores = w.scores;
  }
  // the dense view addresses codes by flat index; that is only valid when the codes are dense too
  View vq = v;
  long long ldc = ld_codes;
  if (ld_in == cols && ld_codes != cols) {  // dense input, padded output: keep the 2-D view
    vq.rows = rows; vq.cols = cols; vq.ld = ld_in;
    vq.vec = aligned(T, 16) && (ld_in % 4 == 0);
    vq.tiles_per_row = (cols + kTileCols - 1) / kTileCols;
    vq.tiles = rows * vq.tiles_per_row;
  } else if (ld_in == cols) {
    ldc = rows * cols;
  }
  const int packed_ok = aligned(codes, 4) && (ldc % 4 == 0);
  LaunchScope ls("quantize_kernel", stream);
  quantize_kernel<<<grid_for(quantize_kernel, vq.tiles), 256, 0, stream>>>(vq, maxp, scores, n_candidates, L, is_signed,
                                                                          codes, ldc, packed_ok, scale, alpha,
                                                                          dev_status);
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// ocs_quantize_noalloc: ocs_quantize for callers that cannot hand over a workspace.  The scratch
// (running maximum, histogram, candidate scores) lives in a fixed array that is part of the loaded
// library image on every device; nothing is allocated, now or at load time beyond that image.
namespace ocs {
namespace {
constexpr size_t kStaticScratchBytes = 48 * 1024;   // covers n_bins <= 4096 and n_candidates <= 1024
static __device__ __align__(256) unsigned char g_quantize_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};       // device address of the array, per device
}  // namespace
}  // namespace ocs

extern "C" ocs_status ocs_quantize_noalloc(const float* T, int64_t rows, int64_t cols, int64_t ld_in, int bits,
                                           int is_signed, ocs_clip_mode mode, int n_candidates, int n_bins,
                                           const float* max_abs_in, int8_t* codes, int64_t ld_codes, float* scale,
                                           float* alpha, int* dev_status, void* stream) {
  if (mode == OCS_CLIP_MSE_EXACT) return OCS_ERR_UNSUPPORTED;   // its partial sums need megabytes
  const bool searched = mode == OCS_CLIP_MSE || mode == OCS_CLIP_KL || mode == OCS_CLIP_ACIQ;
  if (mode == OCS_CLIP_ACIQ) n_candidates = 1;
  if (searched && (n_bins > kMaxBins || n_candidates > kMaxCandidates)) return OCS_ERR_UNSUPPORTED;
  const int nb = searched ? n_bins : 1, nc = searched ? n_candidates : 1;
  if (ocs_quantize_workspace_bytes(nb, nc) > kStaticScratchBytes) return OCS_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return OCS_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return OCS_ERR_UNSUPPORTED;
  if (!g_scratch_addr[dev]) {
    // in host code the array's name is only a handle: ask the runtime for its address on this device
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_quantize_scratch) != cudaSuccess || !p) return OCS_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  return ocs_quantize(T, rows, cols, ld_in, bits, is_signed, mode, n_candidates, n_bins, max_abs_in, codes, ld_codes,
                      scale, alpha, g_scratch_addr[dev], kStaticScratchBytes, dev_status, stream);
}
