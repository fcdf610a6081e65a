// ocs_split: weight outlier channel splitting (Section 3.2 Eq. 3, Section 3.3, Section 3.4).
//
// Three kernels:
//   col_minmax_kernel    one streaming pass over W: signed min and max of every column of the
//                        [O][C*R] matrix (threads own columns, rows stream through coalesced),
//                        combined across CTAs with integer atomics on order-preserving bits.
//   split_plan_kernel    the greedy loop of Section 3.4 run on channel extrema only.  Both halves
//                        of a split are monotone in w, so a copy's extrema are the images of its
//                        parent's extrema and the whole loop needs no further pass over W.
//   split_scatter_kernel one streaming pass that writes W' = path(W[:, idx_map[j], :]).
#include "common.cuh"

namespace ocs {
namespace {

constexpr int kPlanThreads = 1024;
constexpr int kPlanSmemSplits = 4096;  // up to this many splits the plan's queues live in shared memory
constexpr int kMaxHalvings = 320;      // 2^-320 * any finite fp32 is zero: deeper plain halvings change nothing

__device__ __forceinline__ float split_keep(float w, float d) { return __fmul_rn(__fsub_rn(w, d), 0.5f); }
__device__ __forceinline__ float split_new(float w, float d) { return __fmul_rn(__fadd_rn(w, d), 0.5f); }

// ------------------------------------------------------------------------------------------------
// K1: per-column signed extrema of a row-major [O][ncols] fp32 matrix.
template <bool VEC>
__global__ void __launch_bounds__(256)
col_minmax_kernel(const float* __restrict__ W, int O, int ncols, int64_t ld, int rows_per_cta,
                  uint32_t* __restrict__ colmin, uint32_t* __restrict__ colmax, int* dev_status) {
  const int col0 = (blockIdx.x * 256 + threadIdx.x) * 4;
  if (col0 >= ncols) return;
  const int r0 = blockIdx.y * rows_per_cta;
  const int r1 = min(O, r0 + rows_per_cta);
  float mn[4], mx[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) { mn[c] = INFINITY; mx[c] = -INFINITY; }
  bool bad = false;
  if (VEC && col0 + 3 < ncols) {
    const float4* p = reinterpret_cast<const float4*>(W + (int64_t)r0 * ld + col0);
    const int64_t stride = ld >> 2;
#pragma unroll 8
    for (int r = r0; r < r1; ++r) {
      const float4 v = __ldcs(p);
      p += stride;
      mn[0] = fminf(mn[0], v.x); mx[0] = fmaxf(mx[0], v.x);
      mn[1] = fminf(mn[1], v.y); mx[1] = fmaxf(mx[1], v.y);
      mn[2] = fminf(mn[2], v.z); mx[2] = fmaxf(mx[2], v.z);
      mn[3] = fminf(mn[3], v.w); mx[3] = fmaxf(mx[3], v.w);
      bad |= !(is_finite(v.x) && is_finite(v.y) && is_finite(v.z) && is_finite(v.w));
    }
  } else {
    for (int r = r0; r < r1; ++r) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (col0 + c < ncols) {
          const float v = __ldcs(W + (int64_t)r * ld + col0 + c);
          mn[c] = fminf(mn[c], v);
          mx[c] = fmaxf(mx[c], v);
          bad |= !is_finite(v);
        }
      }
    }
  }
  if (r1 > r0) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      if (col0 + c < ncols) {
        atomicMin(&colmin[col0 + c], ord_encode(mn[c]));
        atomicMax(&colmax[col0 + c], ord_encode(mx[c]));
      }
    }
  }
  if (bad) flag(dev_status, OCS_DEV_NONFINITE);
}

// ------------------------------------------------------------------------------------------------
// K2: the greedy loop on channel extrema.
//
// A live channel is (expanded index j, min, max).  Its priority is the 64-bit word
// (bits(max(|min|,|max|)) << 32) | (0xFFFFFFFF - j): larger word = larger |w|, ties broken toward the
// smallest current index.  Only the S largest original channels can ever be chosen (before every
// step at least one of them is still untouched and it outranks every other original), so they
// are selected and sorted once; copies created by splits go to a binary heap.

struct PlanArgs {
  const uint32_t* colmin;  // [C*R] order-preserving bits
  const uint32_t* colmax;
  int C, R, S;
  float qa_step;
  int qa_bits;
  float* chmin;  // [C]
  float* chmax;  // [C]
  float* chkey;  // [C]
  int32_t* idx_map;       // [C+S]
  int32_t* split_order;   // [S] or null
  int32_t* depth;         // [C+S]
  unsigned long long* bits;  // [C+S]
  float* max_abs_out;     // [3] or null
  float* qa_step_dev;     // [1] step actually used (read by the scatter kernel)
  // queues for S > kPlanSmemSplits
  unsigned long long* g_sorted;
  float* g_omin;
  float* g_omax;
  unsigned long long* g_hcomp;
  float* g_hmin;
  float* g_hmax;
  int* dev_status;
};

__device__ __forceinline__ unsigned long long make_prio(float key, int j) {
  return ((unsigned long long)__float_as_uint(key) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)j);
}
__device__ __forceinline__ float prio_key(unsigned long long p) { return __uint_as_float((uint32_t)(p >> 32)); }
__device__ __forceinline__ int prio_index(unsigned long long p) { return (int)(0xFFFFFFFFu - (uint32_t)p); }

struct Heap {
  unsigned long long* comp;
  float* mn;
  float* mx;
  int n;
  __device__ void sift_up(int i, unsigned long long c, float a, float b) {
    while (i > 0) {
      const int parent = (i - 1) >> 1;
      const unsigned long long pc = comp[parent];
      if (pc >= c) break;
      comp[i] = pc; mn[i] = mn[parent]; mx[i] = mx[parent];
      i = parent;
    }
    comp[i] = c; mn[i] = a; mx[i] = b;
  }
  __device__ void push(unsigned long long c, float a, float b) { sift_up(n++, c, a, b); }
  __device__ void replace_top(unsigned long long c, float a, float b) {
    int i = 0;
    for (;;) {
      int l = 2 * i + 1;
      if (l >= n) break;
      unsigned long long lc = comp[l];
      if (l + 1 < n) {
        const unsigned long long rc = comp[l + 1];
        if (rc > lc) { lc = rc; ++l; }
      }
      if (lc <= c) break;
      comp[i] = lc; mn[i] = mn[l]; mx[i] = mx[l];
      i = l;
    }
    comp[i] = c; mn[i] = a; mx[i] = b;
  }
};

// One run of the S greedy steps by a single thread.  Returns max|W'| after the last step.
__device__ float greedy_run(const PlanArgs& a, const unsigned long long* sorted, const float* omin,
                            const float* omax, int Sp, Heap heap, float d, float rest_max, bool write) {
  int p = 0;
  heap.n = 0;
  for (int s = 0; s < a.S; ++s) {
    const unsigned long long co = p < Sp ? sorted[p] : 0ull;
    const unsigned long long ch = heap.n > 0 ? heap.comp[0] : 0ull;
    const bool from_heap = !(p < Sp && co >= ch);
    int j, src, dep;
    unsigned long long bt;
    float mn, mx;
    if (!from_heap) {
      j = prio_index(co); src = j; dep = 0; bt = 0ull;
      mn = omin[p]; mx = omax[p];
      ++p;
    } else {
      j = prio_index(ch);
      mn = heap.mn[0]; mx = heap.mx[0];
      if (write) { src = a.idx_map[j]; dep = a.depth[j]; bt = a.bits[j]; } else { src = 0; dep = 0; bt = 0ull; }
    }
    const int jn = a.C + s;
    const float amn = split_keep(mn, d), amx = split_keep(mx, d);
    const float bmn = split_new(mn, d), bmx = split_new(mx, d);
    if (write) {
      if (dep >= 63 && d != 0.0f) flag(a.dev_status, OCS_DEV_DEPTH);
      const unsigned long long nb = dep < 64 ? (bt | (1ull << dep)) : bt;
      a.idx_map[jn] = src;
      if (a.split_order) a.split_order[s] = j;
      a.depth[j] = dep + 1;   // bits[j] unchanged: the kept copy's new step is a 0 bit
      a.depth[jn] = dep + 1;
      a.bits[jn] = nb;
      if (!from_heap) a.bits[j] = 0ull;
    }
    const unsigned long long ca = make_prio(fmaxf(fabsf(amn), fabsf(amx)), j);
    const unsigned long long cb = make_prio(fmaxf(fabsf(bmn), fabsf(bmx)), jn);
    if (from_heap) heap.replace_top(ca, amn, amx); else heap.push(ca, amn, amx);
    heap.push(cb, bmn, bmx);
  }
  float m = rest_max;
  if (p < Sp) m = fmaxf(m, prio_key(sorted[p]));
  // the heap's top has the largest key among the copies
  if (heap.n > 0) m = fmaxf(m, prio_key(heap.comp[0]));
  return m;
}

__global__ void __launch_bounds__(kPlanThreads, 1) split_plan_kernel(PlanArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ unsigned int hist[256];
  __shared__ float red[kPlanThreads / 32];
  __shared__ unsigned long long sh_thresh;
  __shared__ unsigned int sh_count;
  __shared__ float sh_maxw, sh_rest;
  __shared__ int sh_bad;

  const int tid = threadIdx.x;
  const int C = a.C, R = a.R, S = a.S;
  const int Sp = min(S, C);
  int npad = 1;
  while (npad < Sp) npad <<= 1;

  unsigned long long* sorted;
  float *omin, *omax;
  Heap heap;
  if (S <= kPlanSmemSplits) {
    unsigned char* q = smem_raw;
    sorted = reinterpret_cast<unsigned long long*>(q); q += sizeof(unsigned long long) * npad;
    heap.comp = reinterpret_cast<unsigned long long*>(q); q += sizeof(unsigned long long) * 2 * (size_t)S;
    omin = reinterpret_cast<float*>(q); q += sizeof(float) * Sp;
    omax = reinterpret_cast<float*>(q); q += sizeof(float) * Sp;
    heap.mn = reinterpret_cast<float*>(q); q += sizeof(float) * 2 * (size_t)S;
    heap.mx = reinterpret_cast<float*>(q);
  } else {
    sorted = a.g_sorted; omin = a.g_omin; omax = a.g_omax;
    heap.comp = a.g_hcomp; heap.mn = a.g_hmin; heap.mx = a.g_hmax;
  }
  heap.n = 0;

  // ---- phase A: fold the R taps of each channel, priorities, identity part of the outputs
  if (tid == 0) sh_bad = 0;
  float lmax = 0.0f;
  bool bad = false;
  for (int c = tid; c < C; c += kPlanThreads) {
    uint32_t umin = 0xFFFFFFFFu, umax = 0u;
    for (int r = 0; r < R; ++r) {
      umin = min(umin, a.colmin[(size_t)c * R + r]);
      umax = max(umax, a.colmax[(size_t)c * R + r]);
    }
    const float mn = ord_decode(umin), mx = ord_decode(umax);
    const float key = fmaxf(fabsf(mn), fabsf(mx));
    bad |= !is_finite(key);
    a.chmin[c] = mn; a.chmax[c] = mx; a.chkey[c] = key;
    a.idx_map[c] = c; a.depth[c] = 0; a.bits[c] = 0ull;
    lmax = fmaxf(lmax, key);
  }
  for (int o = 16; o > 0; o >>= 1) lmax = fmaxf(lmax, __shfl_xor_sync(0xffffffffu, lmax, o));
  if ((tid & 31) == 0) red[tid >> 5] = lmax;
  __syncthreads();
  if (tid < 32) {
    float v = red[tid];
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (tid == 0) sh_maxw = v;
  }
  if (bad) sh_bad = 1;
  __syncthreads();
  const float maxw = sh_maxw;

  if (S == 0) {
    if (tid == 0) {
      const float step = a.qa_bits >= 2 ? __fdiv_rn(maxw, (float)((1 << (a.qa_bits - 1)) - 1)) : a.qa_step;
      if (a.max_abs_out) { a.max_abs_out[0] = maxw; a.max_abs_out[1] = maxw; a.max_abs_out[2] = step; }
      *a.qa_step_dev = step;
      if (sh_bad) flag(a.dev_status, OCS_DEV_NONFINITE);
    }
    return;
  }

  // ---- phase B: radix select of the Sp-th largest priority word (8 digits of 8 bits, high first)
  unsigned long long prefix = 0ull, mask = 0ull;
  unsigned int remaining = (unsigned int)Sp;
  for (int pass = 7; pass >= 0; --pass) {
    const int shift = pass * 8;
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    for (int c = tid; c < C; c += kPlanThreads) {
      const unsigned long long w = make_prio(a.chkey[c], c);
      if ((w & mask) == prefix) atomicAdd(&hist[(unsigned int)(w >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned int cum = 0u;
      int dsel = 0;
      for (int dgt = 255; dgt >= 0; --dgt) {
        if (cum + hist[dgt] >= remaining) { dsel = dgt; break; }
        cum += hist[dgt];
      }
      sh_thresh = prefix | ((unsigned long long)dsel << shift);
      sh_count = remaining - cum;
    }
    __syncthreads();
    prefix = sh_thresh;
    remaining = sh_count;
    mask |= 255ull << shift;
    __syncthreads();
  }
  const unsigned long long thresh = prefix;  // exactly Sp priority words are >= thresh

  // ---- selection + largest key left outside
  if (tid == 0) sh_count = 0u;
  for (int i = tid; i < npad; i += kPlanThreads) sorted[i] = 0ull;
  __syncthreads();
  float lrest = 0.0f;
  for (int c = tid; c < C; c += kPlanThreads) {
    const float key = a.chkey[c];
    const unsigned long long w = make_prio(key, c);
    if (w >= thresh) {
      const unsigned int pos = atomicAdd(&sh_count, 1u);
      if (pos < (unsigned int)npad) sorted[pos] = w;
    } else {
      lrest = fmaxf(lrest, key);
    }
  }
  for (int o = 16; o > 0; o >>= 1) lrest = fmaxf(lrest, __shfl_xor_sync(0xffffffffu, lrest, o));
  __syncthreads();
  if ((tid & 31) == 0) red[tid >> 5] = lrest;
  __syncthreads();
  if (tid < 32) {
    float v = red[tid];
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (tid == 0) sh_rest = v;
  }
  __syncthreads();

  // ---- phase C: bitonic sort, descending
  for (int k = 2; k <= npad; k <<= 1) {
    for (int jj = k >> 1; jj > 0; jj >>= 1) {
      for (int i = tid; i < npad; i += kPlanThreads) {
        const int ixj = i ^ jj;
        if (ixj > i) {
          const unsigned long long x = sorted[i], y = sorted[ixj];
          const bool desc = (i & k) == 0;
          if (desc ? (x < y) : (x > y)) { sorted[i] = y; sorted[ixj] = x; }
        }
      }
      __syncthreads();
    }
  }
  for (int i = tid; i < Sp; i += kPlanThreads) {
    const int c = prio_index(sorted[i]);
    omin[i] = a.chmin[c];
    omax[i] = a.chmax[c];
  }
  __syncthreads();

  // ---- phase D: the sequential greedy loop
  if (tid == 0) {
    float step = a.qa_step;
    if (a.qa_bits >= 2) {
      const float predicted = greedy_run(a, sorted, omin, omax, Sp, heap, 0.0f, sh_rest, false);
      const int L = (1 << (a.qa_bits - 1)) - 1;
      step = __fdiv_rn(predicted, (float)L);
    }
    const float d = __fmul_rn(step, 0.5f);
    const float maxwp = greedy_run(a, sorted, omin, omax, Sp, heap, d, sh_rest, true);
    if (a.max_abs_out) { a.max_abs_out[0] = maxw; a.max_abs_out[1] = maxwp; a.max_abs_out[2] = step; }
    *a.qa_step_dev = step;
    if (sh_bad) flag(a.dev_status, OCS_DEV_NONFINITE);
  }
}

// ------------------------------------------------------------------------------------------------
// K3: W'[o][j][r] = path_j(W[o][idx_map[j]][r]).  Threads own 4 consecutive output columns.
template <bool VEC>
__global__ void __launch_bounds__(256)
split_scatter_kernel(const float* __restrict__ W, int O, int C, int R, int64_t ld_in, int S,
                     float* __restrict__ Wout, int64_t ld_out, const int32_t* __restrict__ idx_map,
                     const int32_t* __restrict__ depth, const unsigned long long* __restrict__ bits,
                     const float* __restrict__ qa_step_dev, int rows_per_cta) {
  const int ncols_out = (C + S) * R;
  const int e0 = (blockIdx.x * 256 + threadIdx.x) * 4;
  if (e0 >= ncols_out) return;
  const float d = __fmul_rn(*qa_step_dev, 0.5f);
  int src[4], dep[4];
  unsigned long long bt[4];
  int any = 0;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int e = e0 + c;
    if (e < ncols_out) {
      const int j = e / R, r = e - j * R;
      src[c] = idx_map[j] * R + r;
      dep[c] = min(depth[j], d == 0.0f ? kMaxHalvings : 64);
      bt[c] = bits[j];
    } else {
      src[c] = 0; dep[c] = 0; bt[c] = 0ull;
    }
    any |= dep[c];
  }
  const bool full = e0 + 3 < ncols_out;
  const bool identity = VEC && full && (e0 + 3 < C * R);
  const int r0 = blockIdx.y * rows_per_cta;
  const int r1 = min(O, r0 + rows_per_cta);
#pragma unroll 4
  for (int row = r0; row < r1; ++row) {
    float v[4];
    if (identity) {
      const float4 t = __ldcs(reinterpret_cast<const float4*>(W + (int64_t)row * ld_in + e0));
      v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] = (e0 + c < ncols_out) ? __ldg(W + (int64_t)row * ld_in + src[c]) : 0.0f;
    }
    if (any) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float w = v[c];
        for (int i = 0; i < dep[c]; ++i)
          w = (i < 64 && ((bt[c] >> i) & 1ull)) ? split_new(w, d) : split_keep(w, d);
        v[c] = w;
      }
    }
    float* out = Wout + (int64_t)row * ld_out + e0;
    if (VEC && full) {
      __stcs(reinterpret_cast<float4*>(out), make_float4(v[0], v[1], v[2], v[3]));
    } else {
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (e0 + c < ncols_out) out[c] = v[c];
    }
  }
}

struct SplitWs {
  uint32_t* colmin; uint32_t* colmax;
  float* chmin; float* chmax; float* chkey;
  int32_t* depth; unsigned long long* bits;
  float* qa_step_dev;
  unsigned long long* g_sorted; float* g_omin; float* g_omax;
  unsigned long long* g_hcomp; float* g_hmin; float* g_hmax;
  size_t total;
};

SplitWs carve_split_ws(void* ws, int C, int R, int S) {
  SplitWs w{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    unsigned char* p = ws ? reinterpret_cast<unsigned char*>(ws) + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  };
  const size_t ncols = (size_t)C * R;
  w.colmin = reinterpret_cast<uint32_t*>(take(4 * ncols));
  w.colmax = reinterpret_cast<uint32_t*>(take(4 * ncols));
  w.chmin = reinterpret_cast<float*>(take(4 * (size_t)C));
  w.chmax = reinterpret_cast<float*>(take(4 * (size_t)C));
  w.chkey = reinterpret_cast<float*>(take(4 * (size_t)C));
  w.depth = reinterpret_cast<int32_t*>(take(4 * ((size_t)C + S)));
  w.bits = reinterpret_cast<unsigned long long*>(take(8 * ((size_t)C + S)));
  w.qa_step_dev = reinterpret_cast<float*>(take(256));
  if (S > kPlanSmemSplits) {
    size_t npad = 1;
    while (npad < (size_t)(S < C ? S : C)) npad <<= 1;
    w.g_sorted = reinterpret_cast<unsigned long long*>(take(8 * npad));
    w.g_omin = reinterpret_cast<float*>(take(4 * (size_t)S));
    w.g_omax = reinterpret_cast<float*>(take(4 * (size_t)S));
    w.g_hcomp = reinterpret_cast<unsigned long long*>(take(16 * (size_t)S));
    w.g_hmin = reinterpret_cast<float*>(take(8 * (size_t)S));
    w.g_hmax = reinterpret_cast<float*>(take(8 * (size_t)S));
  }
  w.total = off;
  return w;
}

int rows_per_cta_for(int O, int col_blocks) {
  // aim at ~8 CTAs per SM in total, at least 16 rows per CTA so the atomics stay cheap
  const int target_row_chunks = max(1, (kNumSMs * 8 + col_blocks - 1) / col_blocks);
  int rows = (O + target_row_chunks - 1) / target_row_chunks;
  rows = max(rows, 16);
  return min(rows, max(O, 1));
}

}  // namespace
}  // namespace ocs

using namespace ocs;

extern "C" int ocs_num_splits(int C, double ratio) {
  if (C <= 0 || !(ratio > 0.0)) return 0;
  return (int)ceil(ratio * (double)C - 1e-9);
}

extern "C" size_t ocs_split_workspace_bytes(int O, int C, int R, int S) {
  (void)O;
  if (C <= 0 || R <= 0 || S < 0) return 0;
  return carve_split_ws(nullptr, C, R, S).total;
}

extern "C" ocs_status ocs_split(const float* W, int O, int C, int R, int64_t ld_in, int S, float qa_step,
                                int qa_bits, float* W_out, int64_t ld_out, int32_t* idx_map,
                                int32_t* split_order, float* max_abs_out, void* ws, size_t ws_bytes,
                                int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!W || !W_out || !idx_map) return OCS_ERR_INVALID_ARG;
  if (S < 0 || !(qa_step >= 0.0f) || !is_finite_host(qa_step)) return OCS_ERR_INVALID_ARG;
  if (qa_bits != 0 && (qa_bits < 2 || qa_bits > 8)) return OCS_ERR_INVALID_ARG;
  if (O <= 0 || C <= 0 || R <= 0) return OCS_ERR_SHAPE;
  if ((int64_t)C * R >= (1ll << 31) || ((int64_t)C + S) * R >= (1ll << 31)) return OCS_ERR_SHAPE;
  if (ld_in < (int64_t)C * R || ld_out < ((int64_t)C + S) * R) return OCS_ERR_SHAPE;
  if (!aligned(W, 4) || !aligned(W_out, 4)) return OCS_ERR_SHAPE;
  const SplitWs w = carve_split_ws(ws, C, R, S);
  if (!ws || !aligned(ws, 256) || ws_bytes < w.total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;

  const int ncols = C * R;
  if (cudaMemsetAsync(w.colmin, 0xFF, 4 * (size_t)ncols, stream) != cudaSuccess) return OCS_ERR_CUDA;
  if (cudaMemsetAsync(w.colmax, 0x00, 4 * (size_t)ncols, stream) != cudaSuccess) return OCS_ERR_CUDA;

  {
    const int col_blocks = (ncols + 1023) / 1024;
    const int rows = rows_per_cta_for(O, col_blocks);
    dim3 grid(col_blocks, (O + rows - 1) / rows);
    const bool vec = (ld_in % 4 == 0) && aligned(W, 16);
    LaunchScope ls("col_minmax_kernel", stream);
    if (vec)
      col_minmax_kernel<true><<<grid, 256, 0, stream>>>(W, O, ncols, ld_in, rows, w.colmin, w.colmax, dev_status);
    else
      col_minmax_kernel<false><<<grid, 256, 0, stream>>>(W, O, ncols, ld_in, rows, w.colmin, w.colmax, dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  {
    PlanArgs a{};
    a.colmin = w.colmin; a.colmax = w.colmax;
    a.C = C; a.R = R; a.S = S; a.qa_step = qa_step; a.qa_bits = qa_bits;
    a.chmin = w.chmin; a.chmax = w.chmax; a.chkey = w.chkey;
    a.idx_map = idx_map; a.split_order = split_order; a.depth = w.depth; a.bits = w.bits;
    a.max_abs_out = max_abs_out; a.qa_step_dev = w.qa_step_dev;
    a.g_sorted = w.g_sorted; a.g_omin = w.g_omin; a.g_omax = w.g_omax;
    a.g_hcomp = w.g_hcomp; a.g_hmin = w.g_hmin; a.g_hmax = w.g_hmax;
    a.dev_status = dev_status;
    size_t smem = 0;
    if (S <= kPlanSmemSplits && S > 0) {
      const int Sp = S < C ? S : C;
      size_t npad = 1;
      while (npad < (size_t)Sp) npad <<= 1;
      smem = 8 * npad + 16 * (size_t)S + 8 * (size_t)Sp + 16 * (size_t)S;
    }
    static bool attr_set = false;
    if (!attr_set) {
      if (cudaFuncSetAttribute(split_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess)
        return OCS_ERR_CUDA;
      attr_set = true;
    }
    LaunchScope ls("split_plan_kernel", stream);
    split_plan_kernel<<<1, kPlanThreads, smem, stream>>>(a);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  {
    const int ncols_out = (C + S) * R;
    const int col_blocks = (ncols_out + 1023) / 1024;
    const int rows = rows_per_cta_for(O, col_blocks);
    dim3 grid(col_blocks, (O + rows - 1) / rows);
    const bool vec = (ld_in % 4 == 0) && (ld_out % 4 == 0) && aligned(W, 16) && aligned(W_out, 16);
    LaunchScope ls("split_scatter_kernel", stream);
    if (vec)
      split_scatter_kernel<true><<<grid, 256, 0, stream>>>(W, O, C, R, ld_in, S, W_out, ld_out, idx_map, w.depth,
                                                           w.bits, w.qa_step_dev, rows);
    else
      split_scatter_kernel<false><<<grid, 256, 0, stream>>>(W, O, C, R, ld_in, S, W_out, ld_out, idx_map, w.depth,
                                                            w.bits, w.qa_step_dev, rows);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  return OCS_OK;
}
