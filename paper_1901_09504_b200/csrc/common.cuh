// Shared host/device helpers of the OCS CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <float.h>
#include <math.h>
#include <string.h>
#include <stdint.h>

#include "ocs.h"

namespace ocs {

constexpr int kNumSMs = 148;  // B200: two dies of 74 SMs; grids are sized in multiples of it

// fp32 <-> order-preserving uint32, so that min / max can be combined with integer atomics
__host__ __device__ __forceinline__ uint32_t ord_encode(float f) {
#ifdef __CUDA_ARCH__
  uint32_t b = __float_as_uint(f);
#else
  uint32_t b;
  memcpy(&b, &f, 4);
#endif
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord_decode(uint32_t u) {
  uint32_t b = (u & 0x80000000u) ? (u & 0x7fffffffu) : ~u;
  return __uint_as_float(b);
}

__device__ __forceinline__ bool is_finite(float x) { return fabsf(x) <= FLT_MAX; }

__device__ __forceinline__ void flag(int* dev_status, int bit) {
  if (dev_status) atomicOr(dev_status, bit);
}

inline bool is_finite_host(float x) { return x - x == 0.0f; }

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// true when the current device is compute capability 10.x
inline ocs_status check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return OCS_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return OCS_ERR_CUDA;
  return major == 10 ? OCS_OK : OCS_ERR_UNSUPPORTED;
}

inline ocs_status launch_status() {
  return cudaGetLastError() == cudaSuccess ? OCS_OK : OCS_ERR_CUDA;
}

// Launch accounting (defined in api.cu).  Every kernel launch of the library sits inside one
// LaunchScope: it bumps the process-wide launch counter and, while a trace is active, brackets
// the launch with a pair of CUDA events on the launch stream.
// trace_begin returns the index of the record it opened, or -1 when nothing is recorded (tracing off, or the
// trace is full); trace_end closes exactly that record.
int trace_begin(const char* name, cudaStream_t stream);
void trace_end(int record, cudaStream_t stream);
struct LaunchScope {
  cudaStream_t stream;
  int record;
  LaunchScope(const char* name, cudaStream_t s) : stream(s), record(trace_begin(name, s)) {}
  ~LaunchScope() { trace_end(record, stream); }
};

// The clip search that follows the histogram of |x| (defined in quantize.cu): candidate scores for the MSE and
// KL searches, or the closed-form threshold of ACIQ written to *alpha_sel.
ocs_status launch_clip_search(ocs_clip_mode mode, const unsigned long long* hist, const float* maxp, int n_bins,
                              int n_candidates, int L, int is_signed, double* scores, float* alpha_sel,
                              cudaStream_t stream);

#ifdef __CUDACC__
// The search's winner: smallest score, ties to the largest threshold.  Every CTA of the quantize
// kernel evaluates it (n_candidates doubles) instead of a separate single-thread launch.  Works for
// any one-dimensional block of up to 1024 threads; every thread of the block must call it.
__device__ inline float pick_alpha(const double* __restrict__ scores, float m, int n_candidates) {
  __shared__ double s_best[32];
  __shared__ int c_best[32];
  double bs = INFINITY;
  int bc = 0;
  for (int c = threadIdx.x + 1; c <= n_candidates; c += blockDim.x) {
    const double v = scores[c - 1];
    if (v < bs || (v == bs && c > bc)) { bs = v; bc = c; }
  }
  for (int o = 16; o > 0; o >>= 1) {
    const double v = __shfl_xor_sync(0xffffffffu, bs, o);
    const int c = __shfl_xor_sync(0xffffffffu, bc, o);
    if (c != 0 && (bc == 0 || v < bs || (v == bs && c > bc))) { bs = v; bc = c; }
  }
  if ((threadIdx.x & 31) == 0) { s_best[threadIdx.x >> 5] = bs; c_best[threadIdx.x >> 5] = bc; }
  __syncthreads();
  const int n_warps = (blockDim.x + 31) >> 5;
  bs = s_best[0]; bc = c_best[0];
  for (int w = 1; w < n_warps; ++w) {
    const double v = s_best[w];
    const int c = c_best[w];
    if (c != 0 && (bc == 0 || v < bs || (v == bs && c > bc))) { bs = v; bc = c; }
  }
  return __double2float_rn(__ddiv_rn(__dmul_rn((double)m, (double)bc), (double)n_candidates));
}

// code = clamp(rint(x * inv)): clamping first is the same thing (the bounds are integers).  The rounding is done
// by one addition instead of a conversion instruction: for |t| <= 255, fl(t + 1.5 * 2^23) has unit spacing, so the
// addition rounds t to the nearest integer, ties to even, and the integer sits in the low mantissa bits (two's
// complement for negative t).  Only the low byte of the result is meaningful: that byte is the 8-bit code.
__device__ __forceinline__ int quant_code(float x, float inv, float lo, float hi) {
  return __float_as_int(__fadd_rn(fminf(fmaxf(__fmul_rn(x, inv), lo), hi), 12582912.0f));
}
// Histogram bin of the clip search: min(last, trunc(|x| * invw)).  last is an integer, so clamping the product
// first gives the same bin (and sends NaN and infinity to the last bin instead of out of range).  The truncation
// is one addition rounded toward zero: for 0 <= t < 2^23, fl_rz(t + 2^23) has unit spacing and its bit pattern is
// that of 2^23 plus floor(t) -- no conversion instruction, which runs at a quarter of the addition's rate.
__device__ __forceinline__ int hist_bin(float x, float invw, int last) {
  const float t = fminf(__fmul_rn(fabsf(x), invw), (float)last);
  return __float_as_int(__fadd_rz(t, 8388608.0f)) - 0x4B000000;
}
__device__ __forceinline__ unsigned int pack4(int c0, int c1, int c2, int c3) {
  return __byte_perm(__byte_perm((unsigned)c0, (unsigned)c1, 0x0040), __byte_perm((unsigned)c2, (unsigned)c3, 0x0040),
                     0x5410);
}

#endif  // __CUDACC__

}  // namespace ocs
