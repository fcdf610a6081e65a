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
void trace_begin(const char* name, cudaStream_t stream);
void trace_end(cudaStream_t stream);
struct LaunchScope {
  cudaStream_t stream;
  LaunchScope(const char* name, cudaStream_t s) : stream(s) { trace_begin(name, s); }
  ~LaunchScope() { trace_end(stream); }
};

}  // namespace ocs
