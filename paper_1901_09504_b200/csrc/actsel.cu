// Static channel choice for activation OCS (Section 5.3): on sampled activations P [rows][C], count per
// channel the samples whose |a| exceeds the q-quantile of all |a| and list the S channels with the
// highest counts.
//
// The quantile is exact (nearest rank): the k-th smallest |a| is found by a three-level radix select
// over the fp32 bit patterns (11 + 11 + 10 bits; for non-negative floats the bit pattern orders like the
// value), each level one streaming pass that counts the digits of the elements matching the prefix fixed
// so far.  A fourth pass counts, per channel, the elements above the threshold; the top-S rule is a rank
// computation (count descending, channel index ascending), so it needs no sort and has one answer.
#include "common.cuh"

namespace ocs {
namespace {

constexpr int kSelThreads = 256;
constexpr int kDigits = 2048;

struct SelState {
  unsigned int prefix;        // bits of the threshold fixed so far (high bits)
  unsigned int pad;
  unsigned long long k;       // 1-based rank still to find among the elements matching the prefix
};

struct SelWs {
  SelState* state;
  unsigned long long* hist;   // [3][kDigits]
  unsigned long long* counts; // [C]
  size_t total;
};

SelWs carve_sel_ws(void* ws, int C) {
  SelWs w{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    unsigned char* p = ws ? reinterpret_cast<unsigned char*>(ws) + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  };
  w.state = reinterpret_cast<SelState*>(take(sizeof(SelState)));
  w.hist = reinterpret_cast<unsigned long long*>(take(8 * 3 * (size_t)kDigits));
  w.counts = reinterpret_cast<unsigned long long*>(take(8 * (size_t)C));
  w.total = off;
  return w;
}

__global__ void sel_init_kernel(SelState* st, unsigned long long k) {
  st->prefix = 0u;
  st->pad = 0u;
  st->k = k;
}

// One level of the select: digit = (key >> shift) & (2^nbits - 1) of every element whose bits above
// shift + nbits equal the prefix.  Rows are walked whole (coalesced, no divisions).
__global__ void __launch_bounds__(kSelThreads)
sel_count_kernel(const float* __restrict__ P, long long rows, int C, long long ldp, int shift, int nbits,
                 const SelState* __restrict__ st, unsigned long long* __restrict__ hist, int* dev_status) {
  __shared__ unsigned int h[kDigits];
  for (int i = threadIdx.x; i < kDigits; i += kSelThreads) h[i] = 0u;
  __syncthreads();
  const unsigned int prefix = st->prefix;
  const int top = shift + nbits;                      // bits at and above `top` must match the prefix
  const unsigned int dmask = (1u << nbits) - 1u;
  bool bad = false;
  unsigned int pending = 0;
  for (long long r = blockIdx.x; r < rows; r += gridDim.x) {
    const float* row = P + r * ldp;
    for (int c = threadIdx.x; c < C; c += kSelThreads) {
      const float x = row[c];
      if (!is_finite(x)) { bad = true; continue; }
      const unsigned int key = __float_as_uint(fabsf(x));
      if (top < 32 && (key >> top) != (prefix >> top)) continue;
      atomicAdd(&h[(key >> shift) & dmask], 1u);
    }
    // a 32-bit shared counter cannot overflow before 2^32 elements per CTA; flush well before that
    pending += (unsigned int)C;
    if (pending > 0x40000000u) {
      __syncthreads();
      for (int i = threadIdx.x; i < kDigits; i += kSelThreads) {
        if (h[i]) atomicAdd(&hist[i], (unsigned long long)h[i]);
        h[i] = 0u;
      }
      __syncthreads();
      pending = 0;
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kDigits; i += kSelThreads)
    if (h[i]) atomicAdd(&hist[i], (unsigned long long)h[i]);
  if (bad) flag(dev_status, OCS_DEV_NONFINITE);
}

// Walks the level's histogram upwards until the cumulative count reaches the wanted rank.
__global__ void sel_pick_kernel(SelState* st, const unsigned long long* __restrict__ hist, int shift, int nbits,
                                float* thr_out, int last) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  unsigned long long k = st->k, below = 0;
  const int n = 1 << nbits;
  int d = 0;
  for (; d < n - 1; ++d) {
    const unsigned long long c = hist[d];
    if (below + c >= k) break;
    below += c;
  }
  st->k = k - below;
  st->prefix |= (unsigned int)d << shift;
  if (last && thr_out) *thr_out = __uint_as_float(st->prefix);
}

__global__ void __launch_bounds__(kSelThreads)
sel_above_kernel(const float* __restrict__ P, long long rows, int C, long long ldp, const SelState* __restrict__ st,
                 unsigned long long* __restrict__ counts) {
  const unsigned int thr = st->prefix;
  for (long long r = blockIdx.x; r < rows; r += gridDim.x) {
    const float* row = P + r * ldp;
    for (int c = threadIdx.x; c < C; c += kSelThreads) {
      const float x = row[c];
      if (is_finite(x) && __float_as_uint(fabsf(x)) > thr) atomicAdd(&counts[c], 1ull);
    }
  }
}

// rank(c) = number of channels that come before c in (count descending, index ascending) order.
__global__ void __launch_bounds__(kSelThreads)
sel_rank_kernel(const unsigned long long* __restrict__ counts, int C, int S, int32_t* __restrict__ sel,
                long long* __restrict__ counts_out) {
  __shared__ unsigned long long tile[kSelThreads];
  const int c = blockIdx.x * kSelThreads + threadIdx.x;
  const unsigned long long mine = c < C ? counts[c] : 0ull;
  int rank = 0;
  for (int base = 0; base < C; base += kSelThreads) {
    const int j = base + threadIdx.x;
    tile[threadIdx.x] = j < C ? counts[j] : 0ull;
    __syncthreads();
    const int lim = min(kSelThreads, C - base);
    for (int t = 0; t < lim; ++t) {
      const unsigned long long o = tile[t];
      rank += (o > mine || (o == mine && base + t < c)) ? 1 : 0;
    }
    __syncthreads();
  }
  if (c < C) {
    if (rank < S) sel[rank] = c;
    if (counts_out) counts_out[c] = (long long)mine;
  }
}

}  // namespace
}  // namespace ocs

using namespace ocs;

extern "C" size_t ocs_act_select_workspace_bytes(int C) {
  if (C <= 0) return 0;
  return carve_sel_ws(nullptr, C).total;
}

extern "C" ocs_status ocs_act_select_channels(const float* P, int64_t rows, int C, int64_t ldp, int S, double quantile,
                                              int32_t* sel, int64_t* counts, float* threshold, void* ws,
                                              size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!P || S < 0 || (S > 0 && !sel)) return OCS_ERR_INVALID_ARG;
  if (!(quantile > 0.0) || !(quantile <= 1.0)) return OCS_ERR_INVALID_ARG;
  if (rows <= 0 || C <= 0 || S > C || ldp < C) return OCS_ERR_SHAPE;
  const SelWs w = carve_sel_ws(ws, C);
  if (!ws || !aligned(ws, 256) || ws_bytes < w.total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const double n = (double)rows * (double)C;
  double kd = ceil(quantile * n - 1e-9);
  if (kd < 1.0) kd = 1.0;
  if (kd > n) kd = n;
  const unsigned long long k = (unsigned long long)kd;

  if (cudaMemsetAsync(w.hist, 0, 8 * 3 * (size_t)kDigits, stream) != cudaSuccess) return OCS_ERR_CUDA;
  if (cudaMemsetAsync(w.counts, 0, 8 * (size_t)C, stream) != cudaSuccess) return OCS_ERR_CUDA;
  {
    LaunchScope ls("sel_init_kernel", stream);
    sel_init_kernel<<<1, 1, 0, stream>>>(w.state, k);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  const int grid = (int)min((long long)rows, (long long)kNumSMs * 8);
  const int shifts[3] = {21, 10, 0};
  const int nbits[3] = {11, 11, 10};
  for (int lvl = 0; lvl < 3; ++lvl) {
    {
      LaunchScope ls("sel_count_kernel", stream);
      sel_count_kernel<<<grid, kSelThreads, 0, stream>>>(P, rows, C, ldp, shifts[lvl], nbits[lvl], w.state,
                                                         w.hist + (size_t)lvl * kDigits, dev_status);
      if ((st = launch_status()) != OCS_OK) return st;
    }
    {
      LaunchScope ls("sel_pick_kernel", stream);
      sel_pick_kernel<<<1, 32, 0, stream>>>(w.state, w.hist + (size_t)lvl * kDigits, shifts[lvl], nbits[lvl], threshold,
                                            lvl == 2);
      if ((st = launch_status()) != OCS_OK) return st;
    }
  }
  {
    LaunchScope ls("sel_above_kernel", stream);
    sel_above_kernel<<<grid, kSelThreads, 0, stream>>>(P, rows, C, ldp, w.state, w.counts);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  {
    LaunchScope ls("sel_rank_kernel", stream);
    sel_rank_kernel<<<(C + kSelThreads - 1) / kSelThreads, kSelThreads, 0, stream>>>(w.counts, C, S, sel,
                                                                                     reinterpret_cast<long long*>(counts));
    if ((st = launch_status()) != OCS_OK) return st;
  }
  return OCS_OK;
}
