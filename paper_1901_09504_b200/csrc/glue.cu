// Elementwise and pooling steps between the quantized layers of the end-to-end networks
// (ReLU, residual add, pooling, layout change, embedding lookup, LSTM cell).  Every output is
// produced by single IEEE-rounded fp32 operations in a fixed order, so a layer's float output --
// and with it the next layer's activation codes -- is reproducible bit for bit.
#include "common.cuh"

namespace ocs {
namespace {

int ew_grid(long long n, int per_thread) {
  const long long want = (n + 256ll * per_thread - 1) / (256ll * per_thread);
  const long long cap = (long long)kNumSMs * 8;
  return (int)(want < cap ? (want > 0 ? want : 1) : cap);
}

// y = max(x, 0) (relu = 1) applied to a + b (b may be null: plain ReLU / copy)
// max_bits (optional): fp32 bits of max|y| over the whole tensor, combined with atomicMax (the values are
// non-negative, so their bit patterns order like the values); the next layer's activation grid needs it,
// and taking it here saves that layer a pass over the tensor.
template <bool VEC>
__global__ void __launch_bounds__(256)
add_relu_kernel(const float* __restrict__ a, const float* __restrict__ b, long long n, int relu, float* __restrict__ y,
                unsigned int* __restrict__ max_bits) {
  const long long stride = (long long)gridDim.x * 256;
  float m = 0.0f;
  if (VEC) {
    const long long n4 = n >> 2;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n4; i += stride) {
      float4 v = __ldcs(reinterpret_cast<const float4*>(a) + i);
      if (b) {
        const float4 w = __ldcs(reinterpret_cast<const float4*>(b) + i);
        v.x = __fadd_rn(v.x, w.x); v.y = __fadd_rn(v.y, w.y); v.z = __fadd_rn(v.z, w.z); v.w = __fadd_rn(v.w, w.w);
      }
      if (relu) {
        v.x = v.x > 0.0f ? v.x : 0.0f; v.y = v.y > 0.0f ? v.y : 0.0f;
        v.z = v.z > 0.0f ? v.z : 0.0f; v.w = v.w > 0.0f ? v.w : 0.0f;
      }
      m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
      reinterpret_cast<float4*>(y)[i] = v;
    }
    for (long long i = (n4 << 2) + blockIdx.x * 256ll + threadIdx.x; i < n; i += stride) {
      float v = a[i];
      if (b) v = __fadd_rn(v, b[i]);
      v = (relu && !(v > 0.0f)) ? 0.0f : v;
      m = fmaxf(m, fabsf(v));
      y[i] = v;
    }
  } else {
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += stride) {
      float v = a[i];
      if (b) v = __fadd_rn(v, b[i]);
      v = (relu && !(v > 0.0f)) ? 0.0f : v;
      m = fmaxf(m, fabsf(v));
      y[i] = v;
    }
  }
  if (max_bits) {
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m > 0.0f) atomicMax(max_bits, __float_as_uint(m));
  }
}

// 3x3 stride-2 pad-1 max pooling, NHWC; padding never wins.  Thread = one output element.
__global__ void __launch_bounds__(256)
maxpool3x3s2_kernel(const float* __restrict__ x, int Nb, int H, int Wd, int C, int Ho, int Wo, float* __restrict__ y) {
  const long long total = (long long)Nb * Ho * Wo * C;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
    const int c = (int)(i % C);
    long long t = i / C;
    const int ow = (int)(t % Wo); t /= Wo;
    const int oh = (int)(t % Ho);
    const int n = (int)(t / Ho);
    float m = -INFINITY;
#pragma unroll
    for (int dy = 0; dy < 3; ++dy) {
#pragma unroll
      for (int dx = 0; dx < 3; ++dx) {
        const int ih = oh * 2 + dy - 1, iw = ow * 2 + dx - 1;
        if ((unsigned)ih < (unsigned)H && (unsigned)iw < (unsigned)Wd)
          m = fmaxf(m, __ldg(x + (((long long)n * H + ih) * Wd + iw) * C + c));
      }
    }
    y[i] = m;
  }
}

// The same for four channels per thread (C a multiple of 4, 16-byte aligned tensors, fewer than 2^31 quads):
// 128-bit loads, 32-bit index arithmetic.  The comparisons run in the same order, so the results are the same.
__global__ void __launch_bounds__(256)
maxpool3x3s2_vec4_kernel(const float4* __restrict__ x, int Nb, int H, int Wd, int C4, int Ho, int Wo,
                         float4* __restrict__ y) {
  const unsigned total = (unsigned)Nb * Ho * Wo * C4;
  for (unsigned i = blockIdx.x * 256u + threadIdx.x; i < total; i += gridDim.x * 256u) {
    const unsigned pix = i / (unsigned)C4, c = i - pix * (unsigned)C4;
    const unsigned row = pix / (unsigned)Wo, ow = pix - row * (unsigned)Wo;
    const unsigned n = row / (unsigned)Ho, oh = row - n * (unsigned)Ho;
    float4 m = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll
    for (int dy = 0; dy < 3; ++dy) {
#pragma unroll
      for (int dx = 0; dx < 3; ++dx) {
        const int ih = (int)oh * 2 + dy - 1, iw = (int)ow * 2 + dx - 1;
        if ((unsigned)ih < (unsigned)H && (unsigned)iw < (unsigned)Wd) {
          const float4 v = __ldg(x + (((long long)n * H + ih) * Wd + iw) * C4 + c);
          m.x = fmaxf(m.x, v.x); m.y = fmaxf(m.y, v.y); m.z = fmaxf(m.z, v.z); m.w = fmaxf(m.w, v.w);
        }
      }
    }
    y[i] = m;
  }
}

// Global average: sequential fp32 sum over (h, w) row-major, then one multiply by 1/(H*W).
__global__ void __launch_bounds__(256)
global_avgpool_kernel(const float* __restrict__ x, int Nb, int HW, int C, float* __restrict__ y) {
  const float inv = __fdiv_rn(1.0f, (float)HW);
  const long long total = (long long)Nb * C;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
    const int c = (int)(i % C);
    const long long n = i / C;
    const float* p = x + n * HW * (long long)C + c;
    float s = 0.0f;
    for (int k = 0; k < HW; ++k) s = __fadd_rn(s, __ldg(p + (long long)k * C));
    y[i] = __fmul_rn(s, inv);
  }
}

// NCHW -> NHWC for a handful of channels (an image batch): a CTA takes 256 pixels of one image; the C planes are
// read one after the other (coalesced) into shared memory and the 256 * C interleaved values leave as one
// contiguous run.  grid = (ceil(HW / 256), Nb).
constexpr int kFewChannels = 8;
__global__ void __launch_bounds__(256)
nchw_to_nhwc_few_kernel(const float* __restrict__ x, int C, int HW, float* __restrict__ y) {
  __shared__ float tile[256 * kFewChannels];
  const int n = blockIdx.y;
  const int p0 = blockIdx.x * 256;
  const int np = min(256, HW - p0);
  const float* xin = x + (long long)n * C * HW + p0;
  for (int c = 0; c < C; ++c)
    if ((int)threadIdx.x < np) tile[threadIdx.x * C + c] = xin[(long long)c * HW + threadIdx.x];
  __syncthreads();
  float* yout = y + ((long long)n * HW + p0) * C;
  for (int i = threadIdx.x; i < np * C; i += 256) yout[i] = tile[i];
}

// NCHW -> NHWC through a 32 x 33 shared-memory tile over (c, hw) so both sides are coalesced.
__global__ void __launch_bounds__(256)
nchw_to_nhwc_kernel(const float* __restrict__ x, int C, int HW, float* __restrict__ y) {
  __shared__ float tile[32][33];
  const int n = blockIdx.z;
  const int c0 = blockIdx.y * 32, p0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  const float* xin = x + (long long)n * C * HW;
  float* yout = y + (long long)n * C * HW;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int c = c0 + ty + 8 * k, p = p0 + tx;
    if (c < C && p < HW) tile[ty + 8 * k][tx] = xin[(long long)c * HW + p];
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int p = p0 + ty + 8 * k, c = c0 + tx;
    if (c < C && p < HW) yout[(long long)p * C + c] = tile[tx][ty + 8 * k];
  }
}

__global__ void __launch_bounds__(256)
embedding_kernel(const float* __restrict__ table, const int32_t* __restrict__ ids, long long n, int V, int E,
                 float* __restrict__ out, int* dev_status) {
  const long long total = n * E;
  bool bad = false;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
    const long long t = i / E;
    const int e = (int)(i - t * E);
    int id = __ldg(ids + t);
    if ((unsigned)id >= (unsigned)V) { bad = true; id = 0; }
    out[i] = __ldg(table + (long long)id * E + e);
  }
  if (bad) flag(dev_status, OCS_DEV_BAD_INDEX);
}

// exp(x) for x <= 0, clamped at -87: t = x * log2(e), n = rint(t), f = t - n in [-0.5, 0.5],
// 2^f as the degree-6 Taylor polynomial of exp(f ln 2) in Horner form with fused multiply-adds,
// scaled by 2^n.  Each step rounds once; the result is a pure function of the input bits.
__device__ __forceinline__ float exp_nonpos(float x) {
  x = x < -87.0f ? -87.0f : x;
  const float t = __fmul_rn(x, 1.44269504088896341f);
  const float n = rintf(t);
  const float g = __fmul_rn(__fsub_rn(t, n), 0.693147180559945309f);
  float p = __fdiv_rn(1.0f, 720.0f);
  p = __fmaf_rn(p, g, __fdiv_rn(1.0f, 120.0f));
  p = __fmaf_rn(p, g, __fdiv_rn(1.0f, 24.0f));
  p = __fmaf_rn(p, g, __fdiv_rn(1.0f, 6.0f));
  p = __fmaf_rn(p, g, 0.5f);
  p = __fmaf_rn(p, g, 1.0f);
  p = __fmaf_rn(p, g, 1.0f);
  return ldexpf(p, (int)n);
}
__device__ __forceinline__ float sigmoid_d(float x) {
  const float e = exp_nonpos(-fabsf(x));
  const float den = __fadd_rn(1.0f, e);
  return x >= 0.0f ? __fdiv_rn(1.0f, den) : __fdiv_rn(e, den);
}
__device__ __forceinline__ float tanh_d(float x) {
  const float e = exp_nonpos(__fmul_rn(-2.0f, fabsf(x)));
  const float r = __fdiv_rn(__fsub_rn(1.0f, e), __fadd_rn(1.0f, e));
  return x < 0.0f ? -r : r;
}

// gates [batch][4*hidden] in order i, f, g, o; c updated in place, h written.
__global__ void __launch_bounds__(256)
lstm_cell_kernel(const float* __restrict__ g_ih, const float* __restrict__ g_hh, int batch, int hidden,
                 float* __restrict__ c, float* __restrict__ h) {
  const long long total = (long long)batch * hidden;
  for (long long t = blockIdx.x * 256ll + threadIdx.x; t < total; t += (long long)gridDim.x * 256) {
    const long long b = t / hidden;
    const int k = (int)(t - b * hidden);
    const long long base = b * 4 * hidden + k;
    const float zi = __fadd_rn(g_ih[base], g_hh[base]);
    const float zf = __fadd_rn(g_ih[base + hidden], g_hh[base + hidden]);
    const float zg = __fadd_rn(g_ih[base + 2ll * hidden], g_hh[base + 2ll * hidden]);
    const float zo = __fadd_rn(g_ih[base + 3ll * hidden], g_hh[base + 3ll * hidden]);
    const float i = sigmoid_d(zi), f = sigmoid_d(zf), g = tanh_d(zg), o = sigmoid_d(zo);
    const float cn = __fmaf_rn(f, c[t], __fmul_rn(i, g));
    c[t] = cn;
    h[t] = __fmul_rn(o, tanh_d(cn));
  }
}

}  // namespace
}  // namespace ocs

using namespace ocs;

extern "C" ocs_status ocs_add_relu(const float* a, const float* b, int64_t n, int relu, float* y, float* max_abs_out,
                                   void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!a || !y) return OCS_ERR_INVALID_ARG;
  if (n <= 0) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  if (max_abs_out && cudaMemsetAsync(max_abs_out, 0, 4, stream) != cudaSuccess) return OCS_ERR_CUDA;
  unsigned int* mb = reinterpret_cast<unsigned int*>(max_abs_out);
  const bool vec = aligned(a, 16) && aligned(y, 16) && (!b || aligned(b, 16));
  LaunchScope ls("add_relu_kernel", stream);
  if (vec) add_relu_kernel<true><<<ew_grid(n, 8), 256, 0, stream>>>(a, b, n, relu, y, mb);
  else add_relu_kernel<false><<<ew_grid(n, 8), 256, 0, stream>>>(a, b, n, relu, y, mb);
  return launch_status();
}

extern "C" ocs_status ocs_maxpool3x3s2(const float* x, int Nb, int H, int Wd, int C, float* y, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!x || !y) return OCS_ERR_INVALID_ARG;
  if (Nb <= 0 || H <= 0 || Wd <= 0 || C <= 0) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const int Ho = (H - 1) / 2 + 1, Wo = (Wd - 1) / 2 + 1;
  LaunchScope ls("maxpool3x3s2_kernel", stream);
  const long long total = (long long)Nb * Ho * Wo * C;
  if (C % 4 == 0 && total / 4 < 0x7fffffffll && (reinterpret_cast<uintptr_t>(x) & 15) == 0 &&
      (reinterpret_cast<uintptr_t>(y) & 15) == 0)
    maxpool3x3s2_vec4_kernel<<<ew_grid(total / 4, 4), 256, 0, stream>>>(reinterpret_cast<const float4*>(x), Nb, H, Wd, C / 4,
                                                                     Ho, Wo, reinterpret_cast<float4*>(y));
  else
    maxpool3x3s2_kernel<<<ew_grid(total, 4), 256, 0, stream>>>(x, Nb, H, Wd, C, Ho, Wo, y);
  return launch_status();
}

extern "C" ocs_status ocs_global_avgpool(const float* x, int Nb, int H, int Wd, int C, float* y, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!x || !y) return OCS_ERR_INVALID_ARG;
  if (Nb <= 0 || H <= 0 || Wd <= 0 || C <= 0) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  LaunchScope ls("global_avgpool_kernel", stream);
  global_avgpool_kernel<<<ew_grid((long long)Nb * C, 1), 256, 0, stream>>>(x, Nb, H * Wd, C, y);
  return launch_status();
}

extern "C" ocs_status ocs_nchw_to_nhwc(const float* x, int Nb, int C, int H, int Wd, float* y, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!x || !y) return OCS_ERR_INVALID_ARG;
  if (Nb <= 0 || H <= 0 || Wd <= 0 || C <= 0 || Nb > 65535 || (C + 31) / 32 > 65535) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const int HW = H * Wd;
  LaunchScope ls("nchw_to_nhwc_kernel", stream);
  if (C <= kFewChannels && (HW + 255) / 256 <= 0x7fffffff) {
    dim3 grid((HW + 255) / 256, Nb);
    nchw_to_nhwc_few_kernel<<<grid, 256, 0, stream>>>(x, C, HW, y);
  } else {
    dim3 grid((HW + 31) / 32, (C + 31) / 32, Nb);
    nchw_to_nhwc_kernel<<<grid, 256, 0, stream>>>(x, C, HW, y);
  }
  return launch_status();
}

extern "C" ocs_status ocs_embedding(const float* table, const int32_t* ids, int64_t n, int V, int E, float* out,
                                    int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!table || !ids || !out) return OCS_ERR_INVALID_ARG;
  if (n <= 0 || V <= 0 || E <= 0) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  LaunchScope ls("embedding_kernel", stream);
  embedding_kernel<<<ew_grid(n * E, 4), 256, 0, stream>>>(table, ids, n, V, E, out, dev_status);
  return launch_status();
}

extern "C" ocs_status ocs_lstm_cell(const float* g_ih, const float* g_hh, int batch, int hidden, float* c, float* h,
                                    void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!g_ih || !g_hh || !c || !h) return OCS_ERR_INVALID_ARG;
  if (batch <= 0 || hidden <= 0) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  LaunchScope ls("lstm_cell_kernel", stream);
  lstm_cell_kernel<<<ew_grid((long long)batch * hidden, 1), 256, 0, stream>>>(g_ih, g_hh, batch, hidden, c, h);
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// ocs_transpose_codes: channel-major copy of a code matrix, T[c][r] = A[r][c].  A CTA moves a 128 x 128 byte tile:
// a thread loads four 32-bit words -- the same four columns of four consecutive rows --, transposes the 4 x 4 bytes
// in registers (byte permutes) and writes four words into a shared-memory tile laid out like T; the tile's rows
// then leave as whole 128-byte lines.  Reads and writes are both coalesced 32-bit accesses.  A plain byte-by-byte
// form covers matrices whose rows are not 4-byte addressable.
namespace ocs {
namespace {
__global__ void __launch_bounds__(256)
transpose_codes_kernel(const uint8_t* __restrict__ A, long long rows, long long cols, long long ld,
                       uint8_t* __restrict__ T, long long ld_t) {
  __shared__ uint32_t tile[128][33];    // [column of A][four rows of A per word], one word of padding
  const long long tiles_c = (cols + 127) / 128, tiles_r = (rows + 127) / 128;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (long long t = blockIdx.x; t < tiles_c * tiles_r; t += gridDim.x) {
    const long long tr = t / tiles_c, tc = t - tr * tiles_c;
    const long long r0 = tr * 128, c0 = tc * 128;
    __syncthreads();
    // warp w takes row groups w, w + 8, ... (four rows each); lane l takes columns 4l .. 4l + 3
#pragma unroll
    for (int gi = 0; gi < 4; ++gi) {
      const int rg = warp + gi * 8;                         // row group 0..31
      uint32_t w[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const long long r = r0 + rg * 4 + k, c = c0 + lane * 4;
        w[k] = 0u;
        if (r < rows) {
          if (c + 3 < cols) w[k] = __ldg(reinterpret_cast<const uint32_t*>(A + r * ld + c));
          else
            for (int e = 0; e < 4; ++e)
              if (c + e < cols) w[k] |= (uint32_t)__ldg(A + r * ld + c + e) << (8 * e);
        }
      }
      // 4 x 4 byte transpose: out[j] = bytes j of w[0..3]
      const uint32_t a01 = __byte_perm(w[0], w[1], 0x5140), b01 = __byte_perm(w[0], w[1], 0x7362);
      const uint32_t a23 = __byte_perm(w[2], w[3], 0x5140), b23 = __byte_perm(w[2], w[3], 0x7362);
      tile[lane * 4 + 0][rg] = __byte_perm(a01, a23, 0x5410);
      tile[lane * 4 + 1][rg] = __byte_perm(a01, a23, 0x7632);
      tile[lane * 4 + 2][rg] = __byte_perm(b01, b23, 0x5410);
      tile[lane * 4 + 3][rg] = __byte_perm(b01, b23, 0x7632);
    }
    __syncthreads();
    // row c of the tile = 128 consecutive rows of A for one column: one 128-byte line of T per warp instruction
    for (int c = warp; c < 128; c += 8) {
      if (c0 + c >= cols) break;
      const long long r = r0 + lane * 4;
      uint8_t* dst = T + (c0 + c) * ld_t + r;
      const uint32_t v = tile[c][lane];
      if (r + 3 < rows) *reinterpret_cast<uint32_t*>(dst) = v;
      else
        for (int e = 0; e < 4; ++e)
          if (r + e < rows) dst[e] = (uint8_t)(v >> (8 * e));
    }
  }
}

__global__ void __launch_bounds__(256)
transpose_codes_bytes_kernel(const uint8_t* __restrict__ A, long long rows, long long cols, long long ld,
                             uint8_t* __restrict__ T, long long ld_t) {
  __shared__ uint8_t tile[64][65];
  const long long tiles_c = (cols + 63) / 64, tiles_r = (rows + 63) / 64;
  for (long long t = blockIdx.x; t < tiles_c * tiles_r; t += gridDim.x) {
    const long long tr = t / tiles_c, tc = t - tr * tiles_c;
    const long long r0 = tr * 64, c0 = tc * 64;
    __syncthreads();
    for (int i = threadIdx.x; i < 64 * 64; i += 256) {
      const int r = i >> 6, c = i & 63;
      tile[r][c] = (r0 + r < rows && c0 + c < cols) ? __ldg(A + (r0 + r) * ld + c0 + c) : (uint8_t)0;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 64 * 64; i += 256) {
      const int c = i >> 6, r = i & 63;
      if (c0 + c < cols && r0 + r < rows) T[(c0 + c) * ld_t + r0 + r] = tile[r][c];
    }
  }
}
}  // namespace
}  // namespace ocs

extern "C" ocs_status ocs_transpose_codes(const void* codes, int64_t rows, int64_t cols, int64_t ld, void* codes_T,
                                          int64_t ld_T, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!codes || !codes_T) return OCS_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || ld < cols || ld_T < rows) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const bool words = aligned(codes, 4) && aligned(codes_T, 4) && ld % 4 == 0 && ld_T % 4 == 0;
  const long long edge = words ? 128 : 64;
  const long long tiles = ((rows + edge - 1) / edge) * ((cols + edge - 1) / edge);
  const int grid = (int)(tiles < (long long)kNumSMs * 8 ? tiles : (long long)kNumSMs * 8);
  LaunchScope ls("transpose_codes_kernel", stream);
  if (words)
    transpose_codes_kernel<<<grid, 256, 0, stream>>>(reinterpret_cast<const uint8_t*>(codes), rows, cols, ld,
                                                     reinterpret_cast<uint8_t*>(codes_T), ld_T);
  else
    transpose_codes_bytes_kernel<<<grid, 256, 0, stream>>>(reinterpret_cast<const uint8_t*>(codes), rows, cols, ld,
                                                           reinterpret_cast<uint8_t*>(codes_T), ld_T);
  return launch_status();
}
