// ocs_split: weight outlier channel splitting (Section 3.2 Eq. 3, Section 3.3, Section 3.4).
//
// Three kernels:
//   col_minmax_kernel    one streaming pass over W: signed min and max of every column of the
//                        [O][C*R] matrix (threads own columns, rows stream through coalesced),
//                        combined across CTAs with integer atomics on order-preserving bits.
//   split_plan_kernel    the greedy loop of Section 3.4 run on channel extrema only.  Both halves
//                        of a split are monotone in w, so a copy's extrema are the images of its
//                        parent's extrema and the whole loop needs no further pass over W.  The
//                        dependent steps are grouped into rounds whose members are independent.
//   split_rows_kernel    one streaming pass that writes W' = path(W[:, idx_map[j], :]): whole rows staged
//                        in shared memory by bulk copies, duplicated channels gathered there
//   split_scatter_kernel the same pass with plain loads and stores, for shapes the bulk copies
//                        cannot serve (rows longer than the buffers, unaligned rows)
#include <mutex>

#include "common.cuh"

namespace ocs {
namespace {

constexpr int kPlanThreads = 1024;
constexpr int kPlanSmemSplits = 3072;  // up to this many splits the plan's live set lives in shared memory
constexpr int kPlanSmemBytes = 220 * 1024;  // dynamic shared memory the plan kernel may use
constexpr size_t kRowSmemBytes = 226 * 1024;       // shared memory the bulk-copy scatter may use (two row-group buffers)
constexpr int kMaxHalvings = 320;      // 2^-320 * any finite fp32 is zero: deeper plain halvings change nothing

__device__ __forceinline__ float split_keep(float w, float d) { return __fmul_rn(__fsub_rn(w, d), 0.5f); }
__device__ __forceinline__ float split_new(float w, float d) { return __fmul_rn(__fadd_rn(w, d), 0.5f); }

// ------------------------------------------------------------------------------------------------
// Work partition of the two streaming kernels: the matrix is cut into column blocks of 1024
// columns (a thread owns 4 consecutive columns); the (column block, row) pairs are numbered
// column-block-major and every CTA of a grid sized to one resident wave takes one contiguous
// range of them, so all CTAs stream the same number of rows (to within one).
__device__ __forceinline__ void cta_range(long long total, long long* u0, long long* u1, int vb, int vg) {
  *u0 = total * (long long)vb / (long long)vg;
  *u1 = total * ((long long)vb + 1) / (long long)vg;
}

// K1 for a narrow matrix (ncols <= 512): a row needs only ncols/4 threads, so the CTA walks 256 / (ncols/4)
// rows side by side and combines them in shared memory before touching the global extrema.
// (vb, vg): this CTA's index and the number of CTAs working on this matrix -- the block index and grid size of a
// launch for one matrix, or a share of a launch that covers many matrices.
template <bool VEC>
__device__ __forceinline__ void
col_minmax_narrow_body(const float* __restrict__ W, int O, int ncols, int64_t ld, uint32_t* __restrict__ colmin,
                       uint32_t* __restrict__ colmax, int C, int32_t* __restrict__ idx_map,
                       int32_t* __restrict__ depth, unsigned long long* __restrict__ bits, int* dev_status, int vb, int vg) {
  for (int c = vb * 256 + threadIdx.x; c < C; c += vg * 256) {
    idx_map[c] = c; depth[c] = 0; bits[c] = 0ull;
  }
  bool bad = false;
  {
    // narrow matrix: a row needs only ncols/4 threads, so the CTA walks 256 / (ncols/4) rows side by side and
    // combines them in shared memory before touching the global extrema
    __shared__ uint32_t s_min[512], s_max[512];
    for (int i = threadIdx.x; i < ncols; i += 256) { s_min[i] = 0xFFFFFFFFu; s_max[i] = 0u; }
    __syncthreads();
    const int tpr = (ncols + 3) >> 2;
    const int side = 256 / tpr;
    const int lr = threadIdx.x / tpr, col0 = (threadIdx.x - lr * tpr) * 4;
    long long r0, r1;
    cta_range((long long)O, &r0, &r1, vb, vg);
    if (lr < side) {
      float mn[4], mx[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) { mn[c] = INFINITY; mx[c] = -INFINITY; }
      if (VEC && col0 + 3 < ncols) {
        const float4* p = reinterpret_cast<const float4*>(W + (r0 + lr) * ld + col0);
        const int64_t stride = (ld >> 2) * side;
#pragma unroll 8
        for (long long r = r0 + lr; r < r1; r += side) {
          const float4 v = __ldcs(p);
          p += stride;
          mn[0] = fminf(mn[0], v.x); mx[0] = fmaxf(mx[0], v.x);
          mn[1] = fminf(mn[1], v.y); mx[1] = fmaxf(mx[1], v.y);
          mn[2] = fminf(mn[2], v.z); mx[2] = fmaxf(mx[2], v.z);
          mn[3] = fminf(mn[3], v.w); mx[3] = fmaxf(mx[3], v.w);
          bad |= !(is_finite(v.x) && is_finite(v.y) && is_finite(v.z) && is_finite(v.w));
        }
      } else {
        for (long long r = r0 + lr; r < r1; r += side) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (col0 + c < ncols) {
              const float v = __ldcs(W + r * ld + col0 + c);
              mn[c] = fminf(mn[c], v);
              mx[c] = fmaxf(mx[c], v);
              bad |= !is_finite(v);
            }
          }
        }
      }
      if (r0 + lr < r1) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (col0 + c < ncols) {
            atomicMin(&s_min[col0 + c], ord_encode(mn[c]));
            atomicMax(&s_max[col0 + c], ord_encode(mx[c]));
          }
        }
      }
    }
    __syncthreads();
    if (r0 < r1) {
      for (int i = threadIdx.x; i < ncols; i += 256) {
        atomicMin(&colmin[i], s_min[i]);
        atomicMax(&colmax[i], s_max[i]);
      }
    }
    if (bad) flag(dev_status, OCS_DEV_NONFINITE);
  }
}

template <bool VEC>
__global__ void __launch_bounds__(256)
col_minmax_narrow_kernel(const float* __restrict__ W, int O, int ncols, int64_t ld, uint32_t* __restrict__ colmin,
                         uint32_t* __restrict__ colmax, int C, int32_t* __restrict__ idx_map,
                         int32_t* __restrict__ depth, unsigned long long* __restrict__ bits, int* dev_status) {
  col_minmax_narrow_body<VEC>(W, O, ncols, ld, colmin, colmax, C, idx_map, depth, bits, dev_status, blockIdx.x, gridDim.x);
}

// K1: per-column signed extrema of a row-major [O][ncols] fp32 matrix.
template <bool VEC>
__device__ __forceinline__ void
col_minmax_body(const float* __restrict__ W, int O, int ncols, int64_t ld, uint32_t* __restrict__ colmin,
                uint32_t* __restrict__ colmax, int C, int32_t* __restrict__ idx_map, int32_t* __restrict__ depth,
                unsigned long long* __restrict__ bits, int* dev_status, int vb, int vg) {
  // identity part of the plan's outputs: original channel c maps to itself and has no split yet
  for (int c = vb * 256 + threadIdx.x; c < C; c += vg * 256) {
    idx_map[c] = c; depth[c] = 0; bits[c] = 0ull;
  }
  bool bad = false;
  const int col_blocks = (ncols + 1023) / 1024;
  long long u, u1;
  cta_range((long long)col_blocks * O, &u, &u1, vb, vg);
  while (u < u1) {
    const int cb = (int)(u / O);
    const int r0 = (int)(u - (long long)cb * O);
    const int r1 = (int)min((long long)O, r0 + (u1 - u));
    u += r1 - r0;
    const int col0 = (cb * 256 + threadIdx.x) * 4;
    if (col0 >= ncols) continue;
    float mn[4], mx[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) { mn[c] = INFINITY; mx[c] = -INFINITY; }
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

template <bool VEC>
__global__ void __launch_bounds__(256)
col_minmax_kernel(const float* __restrict__ W, int O, int ncols, int64_t ld, uint32_t* __restrict__ colmin,
                  uint32_t* __restrict__ colmax, int C, int32_t* __restrict__ idx_map, int32_t* __restrict__ depth,
                  unsigned long long* __restrict__ bits, int* dev_status) {
  col_minmax_body<VEC>(W, O, ncols, ld, colmin, colmax, C, idx_map, depth, bits, dev_status, blockIdx.x, gridDim.x);
}

// ------------------------------------------------------------------------------------------------
// K2: the greedy loop of Section 3.4 on channel extrema, in rounds.
//
// A live channel is (expanded index j, min, max).  Its priority is the 64-bit word
// (bits(max(|min|,|max|)) << 32) | (0xFFFFFFFF - j): a larger word is a larger |w|, ties broken
// toward the smallest current index -- the order in which the one-at-a-time loop picks channels.
// Only the min(S, C) highest-priority original channels can ever be picked (before every step at
// least one of them is untouched and outranks every other original), so they are selected once
// (radix select) and form the initial live set.
//
// One round: let kmax be the largest live key and B = fl(fl(kmax + d) * 0.5), an upper bound on
// the key of any child of any live channel.  Every live channel whose key is strictly above B is
// picked before any child created from now on, and before every live channel at or below B; so
// the next steps of the one-at-a-time loop are exactly those channels in priority order.  The
// round sorts them (bitonic, shared memory), assigns step numbers base + rank, and performs all
// their splits in parallel.  The top channel itself always joins the batch, so a round makes at
// least one step even when d >= kmax or all keys are zero.  Typical tensors need a handful of
// rounds (each halves the largest key), instead of S dependent steps.

struct PlanArgs {
  const uint32_t* colmin;  // [C*R] order-preserving bits
  const uint32_t* colmax;
  int C, R, S;
  float qa_step;
  int qa_bits;
  float* chmin;  // [C+S] current extrema of the selected originals and of every channel a split creates
  float* chmax;
  float* chkey;  // [C] keys, used when they do not fit in shared memory
  int32_t* idx_map;       // [C+S]  (entries below C are written by the extrema kernel)
  int32_t* split_order;   // [S] or null
  int32_t* depth;         // [C+S]
  unsigned long long* bits;  // [C+S]
  float* max_abs_out;     // [3] or null
  float* qa_step_dev;     // [1] step actually used (read by the scatter kernel)
  int32_t* touched;       // [min(S, C)] original channels that were split at least once
  int* n_touched;         // [1]
  unsigned long long* g_buf;  // sel | live0 | live1 | batch in global memory, used when S > kPlanSmemSplits
  int cap, npad, Sp;      // live capacity Sp + S, sort capacity (power of two >= cap), min(S, C)
  int hist_off, keys_off; // byte offsets in dynamic shared memory: selection histograms; keys (-1: chkey)
  float* curve;           // [S + 1] or null: curve[s] = largest |w| after s plain-halving splits; when given, the
                          // kernel only fills the curve (no index map, no extrema of the copies)
  int* dev_status;
};

constexpr int kSelBins = 2048;    // bins of one selection level
constexpr int kSelCopies = 8;     // private histogram copies (one per four warps)
constexpr int kSelHistBytes = kSelBins * kSelCopies * 4;

__device__ __forceinline__ unsigned long long make_prio(float key, int j) {
  return ((unsigned long long)__float_as_uint(key) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)j);
}
__device__ __forceinline__ float prio_key(unsigned long long p) { return __uint_as_float((uint32_t)(p >> 32)); }
__device__ __forceinline__ int prio_index(unsigned long long p) { return (int)(0xFFFFFFFFu - (uint32_t)p); }

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t > v ? t : v;
  }
  return v;
}

struct PlanShared {
  unsigned long long red[32];
  unsigned long long scan[32];
  unsigned int digit, count;
  int n_batch, n_next;
  int n_touched;
  int bad;
};

// Largest of the threads' words over the whole CTA, returned to every thread.
__device__ unsigned long long block_max_u64(unsigned long long m, unsigned long long* red) {
  m = warp_max_u64(m);
  __syncthreads();  // red may still be read by the previous call
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  return warp_max_u64(red[threadIdx.x & 31]);
}

// Exclusive prefix sum of v over the CTA in thread order (both 32-bit halves of v are summed
// independently as long as neither overflows); *total receives the sum over all threads.
__device__ unsigned long long block_excl_scan(unsigned long long v, unsigned long long* scan,
                                              unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();  // scan may still be read by the previous call
  if (lane == 31) scan[warp] = incl;
  __syncthreads();
  unsigned long long w = scan[lane];
  unsigned long long wincl = w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xffffffffu, wincl, o);
    if (lane >= o) wincl += t;
  }
  *total = __shfl_sync(0xffffffffu, wincl, 31);
  const unsigned long long warp_base = __shfl_sync(0xffffffffu, wincl - w, warp);
  return warp_base + incl - v;
}

// One compare-exchange of a descending bitonic network on a[0..): pair number t of stage (k, jj).
__device__ __forceinline__ void bitonic_pair(unsigned long long* a, int t, int k, int jj) {
  const int i = ((t & ~(jj - 1)) << 1) | (t & (jj - 1));
  const int ixj = i | jj;
  const unsigned long long x = a[i], y = a[ixj];
  const bool desc = (i & k) == 0;
  if (desc ? (x < y) : (x > y)) { a[i] = y; a[ixj] = x; }
}

// Sorts a[0..npad) descending; npad a power of two >= 2.  Every warp owns a contiguous chunk:
// stages whose partners lie inside one chunk need only a warp barrier.  Ends with a CTA barrier.
__device__ void bitonic_sort_desc(unsigned long long* a, int npad) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = max(64, npad / (kPlanThreads / 32));   // elements per warp
  const int warps_used = max(1, npad / chunk);
  const int local_n = min(chunk, npad);
  unsigned long long* mine = a + (size_t)warp * chunk;
  for (int k = 2; k <= npad; k <<= 1) {
    int jj = k >> 1;
    for (; jj >= chunk; jj >>= 1) {                       // partners in different chunks
      for (int t = threadIdx.x; t < (npad >> 1); t += kPlanThreads) bitonic_pair(a, t, k, jj);
      __syncthreads();
    }
    if (warp < warps_used) {
      for (; jj > 0; jj >>= 1) {                          // partners inside this warp's chunk
        for (int t = lane; t < (local_n >> 1); t += 32) {
          const int i = ((t & ~(jj - 1)) << 1) | (t & (jj - 1));
          const int gi = warp * chunk + i;                // the direction depends on the global index
          const unsigned long long x = mine[i], y = mine[i | jj];
          const bool desc = (gi & k) == 0;
          if (desc ? (x < y) : (x > y)) { mine[i] = y; mine[i | jj] = x; }
        }
        __syncwarp();
      }
    }
    if (k >= chunk) __syncthreads();                      // the next cross-chunk stage reads other chunks
  }
  __syncthreads();
}

// Runs the S greedy steps in rounds on the live set `live` (n_live entries).  With write = false
// (plain halving, d = 0) only keys are tracked: both children of key k have key fl(k * 0.5).
// Returns the largest key among the live channels after the last step.
__device__ float greedy_rounds(const PlanArgs& a, PlanShared& sh, unsigned long long* live, unsigned long long* next,
                               unsigned long long* batch, int n_live, float d, bool write) {
  const int tid = threadIdx.x, lane = threadIdx.x & 31;
  const unsigned int lt = (1u << lane) - 1u;
  int base = 0;
  while (base < a.S) {
    unsigned long long m = 0ull;
    for (int i = tid; i < n_live; i += kPlanThreads) m = live[i] > m ? live[i] : m;
    const unsigned long long pmax = block_max_u64(m, sh.red);
    const float bound = __fmul_rn(__fadd_rn(prio_key(pmax), d), 0.5f);
    // Stable partition (positions from prefix sums, not atomics): the selected originals arrive in
    // index order, so a batch of equal keys -- the tie-break case -- comes out already in priority
    // order and the sort below can be skipped.
    int nb = 0, n_keep = 0;
    for (int i0 = 0; i0 < n_live; i0 += kPlanThreads) {   // whole warps iterate together
      const int i = i0 + tid;
      const unsigned long long p = i < n_live ? live[i] : 0ull;
      const bool in_batch = i < n_live && (prio_key(p) > bound || p == pmax);
      const bool in_next = i < n_live && !in_batch;
      const unsigned int mb = __ballot_sync(0xffffffffu, in_batch), mn = __ballot_sync(0xffffffffu, in_next);
      unsigned long long total;
      const unsigned long long mine = lane == 0 ? (((unsigned long long)__popc(mb) << 32) | (unsigned long long)__popc(mn)) : 0ull;
      unsigned long long pre = block_excl_scan(mine, sh.scan, &total);
      pre = __shfl_sync(0xffffffffu, pre, 0);   // lane 0 holds the sum over the warps before this one
      if (in_batch) batch[nb + (int)(pre >> 32) + __popc(mb & lt)] = p;
      if (in_next) next[n_keep + (int)(unsigned int)pre + __popc(mn & lt)] = p;
      nb += (int)(total >> 32);
      n_keep += (int)(unsigned int)total;
    }
    __syncthreads();
    int npad = 1;
    while (npad < nb) npad <<= 1;
    for (int i = nb + tid; i < npad; i += kPlanThreads) batch[i] = 0ull;  // below every real priority word
    __syncthreads();
    bool unsorted = false;
    for (int i = tid + 1; i < nb; i += kPlanThreads) unsorted |= batch[i - 1] < batch[i];
    if (!__syncthreads_or(unsorted)) npad = 1;   // already in descending priority order
    if (npad > 1) bitonic_sort_desc(batch, npad);
    const int take = min(nb, a.S - base);
    // rank i < take performs step base + i; its children go to next[n_keep + 2i, +1]; channels
    // beyond `take` (the last round only) stay live unchanged
    for (int i0 = 0; i0 < nb; i0 += kPlanThreads) {
      const int i = i0 + tid;
      const bool act = i < nb;
      const unsigned long long p = act ? batch[i] : 0ull;
      bool first = false;
      int j = 0;
      if (act && i >= take) next[n_keep + 2 * take + (i - take)] = p;
      if (act && i < take) {
        j = prio_index(p);
        const int s = base + i;
        const int jn = a.C + s;
        if (!write && a.curve) a.curve[s] = prio_key(p);   // the value step s picks is the maximum before it
        unsigned long long ca, cb;
        if (write) {
          const float mn = a.chmin[j], mx = a.chmax[j];
          const float amn = split_keep(mn, d), amx = split_keep(mx, d);
          const float bmn = split_new(mn, d), bmx = split_new(mx, d);
          const int dep = a.depth[j];
          const unsigned long long bt = a.bits[j];
          if (dep >= 63 && d != 0.0f) flag(a.dev_status, OCS_DEV_DEPTH);
          first = dep == 0;   // an original channel's first split
          a.chmin[j] = amn; a.chmax[j] = amx;
          a.chmin[jn] = bmn; a.chmax[jn] = bmx;
          a.idx_map[jn] = a.idx_map[j];
          if (a.split_order) a.split_order[s] = j;
          a.depth[j] = dep + 1;   // bits[j] unchanged: the kept copy's new step is a 0 bit
          a.depth[jn] = dep + 1;
          a.bits[jn] = dep < 64 ? (bt | (1ull << dep)) : bt;
          ca = make_prio(fmaxf(fabsf(amn), fabsf(amx)), j);
          cb = make_prio(fmaxf(fabsf(bmn), fabsf(bmx)), jn);
        } else {
          const float half = __fmul_rn(prio_key(p), 0.5f);
          ca = make_prio(half, j);
          cb = make_prio(half, jn);
        }
        next[n_keep + 2 * i] = ca;
        next[n_keep + 2 * i + 1] = cb;
      }
      const unsigned int mf = __ballot_sync(0xffffffffu, first);
      if (mf) {
        int tb = 0;
        if (lane == 0) tb = atomicAdd(&sh.n_touched, __popc(mf));
        tb = __shfl_sync(0xffffffffu, tb, 0);
        if (first) a.touched[tb + __popc(mf & lt)] = j;
      }
    }
    __syncthreads();
    n_live = n_keep + nb + take;
    base += take;
    unsigned long long* t = live; live = next; next = t;
  }
  unsigned long long m = 0ull;
  for (int i = tid; i < n_live; i += kPlanThreads) m = live[i] > m ? live[i] : m;
  return prio_key(block_max_u64(m, sh.red));
}

__device__ void split_plan_body(const PlanArgs& a, unsigned char* smem_raw) {
  __shared__ PlanShared sh;

  const int tid = threadIdx.x;
  const int C = a.C, R = a.R, S = a.S, Sp = a.Sp;
  unsigned long long* buf = (S <= kPlanSmemSplits) ? reinterpret_cast<unsigned long long*>(smem_raw) : a.g_buf;
  unsigned long long* sel = buf;                 // [Sp]   the selected originals
  unsigned long long* live0 = sel + Sp;          // [cap]
  unsigned long long* live1 = live0 + a.cap;     // [cap]
  unsigned long long* batch = live1 + a.cap;     // [npad]
  // during the selection the space behind sel holds the histograms and (when they fit) the keys
  unsigned int* hist = reinterpret_cast<unsigned int*>(smem_raw + a.hist_off);
  float* keys = a.keys_off >= 0 ? reinterpret_cast<float*>(smem_raw + a.keys_off) : a.chkey;
  const uint32_t* __restrict__ colmin = a.colmin;
  const uint32_t* __restrict__ colmax = a.colmax;

  // ---- phase A: fold the R taps of each channel into its key max(|min|, |max|)
  if (tid == 0) { sh.bad = 0; sh.n_touched = 0; }
  __syncthreads();
  unsigned long long lmax = 0ull;
  bool bad = false;
  for (int c0 = 0; c0 < C; c0 += 8 * kPlanThreads) {
    uint32_t umin[8], umax[8];
    if (R == 1) {
#pragma unroll
      for (int u = 0; u < 8; ++u) {   // sixteen independent loads in flight
        const int c = c0 + u * kPlanThreads + tid;
        umin[u] = c < C ? __ldg(colmin + c) : 0xFFFFFFFFu;
        umax[u] = c < C ? __ldg(colmax + c) : 0u;
      }
    } else {
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c = c0 + u * kPlanThreads + tid;
        umin[u] = 0xFFFFFFFFu; umax[u] = 0u;
        if (c < C) {
          for (int r = 0; r < R; ++r) {
            umin[u] = min(umin[u], __ldg(colmin + (size_t)c * R + r));
            umax[u] = max(umax[u], __ldg(colmax + (size_t)c * R + r));
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int c = c0 + u * kPlanThreads + tid;
      if (c >= C) continue;
      const float key = fmaxf(fabsf(ord_decode(umin[u])), fabsf(ord_decode(umax[u])));
      bad |= !is_finite(key);
      keys[c] = key;
      const unsigned long long kb = (unsigned long long)__float_as_uint(key);
      lmax = kb > lmax ? kb : lmax;
    }
  }
  if (bad) sh.bad = 1;
  const float maxw = __uint_as_float((uint32_t)block_max_u64(lmax, sh.red));

  if (a.curve && S == 0) {
    if (tid == 0) {
      a.curve[0] = maxw;
      if (sh.bad) flag(a.dev_status, OCS_DEV_NONFINITE);
    }
    return;
  }
  if (S == 0) {
    if (tid == 0) {
      const float step = a.qa_bits >= 2 ? __fdiv_rn(maxw, (float)((1 << (a.qa_bits - 1)) - 1)) : a.qa_step;
      if (a.max_abs_out) { a.max_abs_out[0] = maxw; a.max_abs_out[1] = maxw; a.max_abs_out[2] = step; }
      *a.qa_step_dev = step;
      *a.n_touched = 0;
      if (sh.bad) flag(a.dev_status, OCS_DEV_NONFINITE);
    }
    return;
  }

  // ---- phase B: the Sp-th largest key, by a three-level histogram select on the key bits
  // (keys are non-negative floats: their bit patterns order like their values)
  uint32_t prefix = 0u, pmask = 0u;
  unsigned int remaining = (unsigned int)Sp;
  for (int lvl = 0; lvl < 3; ++lvl) {
    const int shift = lvl == 0 ? 21 : (lvl == 1 ? 10 : 0);
    const int nbins = lvl == 2 ? 1024 : 2048;
    for (int i = tid; i < kSelBins * kSelCopies; i += kPlanThreads) hist[i] = 0u;
    __syncthreads();
    unsigned int* copy = hist + ((tid >> 5) & (kSelCopies - 1)) * kSelBins;
    for (int c = tid; c < C; c += kPlanThreads) {
      const uint32_t kb = __float_as_uint(keys[c]);
      if ((kb & pmask) == prefix) atomicAdd(&copy[(kb >> shift) & (uint32_t)(nbins - 1)], 1u);
    }
    __syncthreads();
    // thread t owns bins nbins-1-2t and nbins-2-2t (descending), summed over the copies
    unsigned int hi = 0u, lo = 0u;
    if (2 * tid < nbins) {
      for (int k = 0; k < kSelCopies; ++k) {
        hi += hist[k * kSelBins + nbins - 1 - 2 * tid];
        lo += hist[k * kSelBins + nbins - 2 - 2 * tid];
      }
    }
    unsigned long long total;
    const unsigned int above = (unsigned int)block_excl_scan((unsigned long long)(hi + lo), sh.scan, &total);
    if (above < remaining && remaining <= above + hi + lo) {   // exactly one thread
      if (above + hi >= remaining) { sh.digit = (unsigned int)(nbins - 1 - 2 * tid); sh.count = remaining - above; }
      else { sh.digit = (unsigned int)(nbins - 2 - 2 * tid); sh.count = remaining - above - hi; }
    }
    __syncthreads();
    prefix |= sh.digit << shift;
    pmask |= (uint32_t)(nbins - 1) << shift;
    remaining = sh.count;
    __syncthreads();
  }
  const uint32_t kthr = prefix;          // bit pattern of the Sp-th largest key
  const unsigned int ties_taken = remaining;  // that many channels with exactly this key are selected ...
  const unsigned int n_above = (unsigned int)Sp - ties_taken;   // ... after all channels with a larger key

  // ---- selection: channels with a larger key, then the lowest-index channels with the threshold
  // key.  Threads own contiguous index ranges, so tie ranks follow the channel index.
  const int cpt = ((C + kPlanThreads - 1) / kPlanThreads) | 1;   // odd: conflict-free strided reads
  const int c_begin = min(C, tid * cpt), c_end = min(C, c_begin + cpt);
  unsigned int my_above = 0u, my_ties = 0u;
  for (int c = c_begin; c < c_end; ++c) {
    const uint32_t kb = __float_as_uint(keys[c]);
    my_above += kb > kthr;
    my_ties += kb == kthr;
  }
  unsigned long long total;
  const unsigned long long pre = block_excl_scan(((unsigned long long)my_above << 32) | my_ties, sh.scan, &total);
  unsigned int pos_above = (unsigned int)(pre >> 32), tie_rank = (unsigned int)pre;
  unsigned long long lrest = 0ull;
  for (int c = c_begin; c < c_end; ++c) {
    const float key = keys[c];
    const uint32_t kb = __float_as_uint(key);
    int slot = -1;
    if (kb > kthr) slot = (int)pos_above++;
    else if (kb == kthr && tie_rank++ < ties_taken) slot = (int)(n_above + tie_rank - 1);
    if (slot >= 0) {
      sel[slot] = make_prio(key, c);
    } else {
      lrest = (unsigned long long)kb > lrest ? (unsigned long long)kb : lrest;
    }
  }
  const float rest_max = __uint_as_float((uint32_t)block_max_u64(lrest, sh.red));
  __syncthreads();
  if (a.curve) {
    // range curve only: plain halving on the keys, every step's pick recorded
    for (int i = tid; i < Sp; i += kPlanThreads) live0[i] = sel[i];
    __syncthreads();
    const float last = fmaxf(rest_max, greedy_rounds(a, sh, live0, live1, batch, Sp, 0.0f, false));
    if (tid == 0) {
      a.curve[S] = last;
      if (sh.bad) flag(a.dev_status, OCS_DEV_NONFINITE);
    }
    return;
  }
  // signed extrema of the selected channels (the only originals the greedy steps can touch)
  for (int i = tid; i < Sp; i += kPlanThreads) {
    const int c = prio_index(sel[i]);
    uint32_t umin = 0xFFFFFFFFu, umax = 0u;
    for (int r = 0; r < R; ++r) {
      umin = min(umin, __ldg(colmin + (size_t)c * R + r));
      umax = max(umax, __ldg(colmax + (size_t)c * R + r));
    }
    a.chmin[c] = ord_decode(umin);
    a.chmax[c] = ord_decode(umax);
  }
  __syncthreads();

  // ---- phase C: the greedy steps
  float step = a.qa_step;
  if (a.qa_bits >= 2) {
    // two-pass rule: the grid step is max|W'| of a plain-halving run divided by L
    for (int i = tid; i < Sp; i += kPlanThreads) live0[i] = sel[i];
    __syncthreads();
    const float predicted = fmaxf(rest_max, greedy_rounds(a, sh, live0, live1, batch, Sp, 0.0f, false));
    step = __fdiv_rn(predicted, (float)((1 << (a.qa_bits - 1)) - 1));
    __syncthreads();
  }
  const float d = __fmul_rn(step, 0.5f);
  for (int i = tid; i < Sp; i += kPlanThreads) live0[i] = sel[i];
  __syncthreads();
  const float maxwp = fmaxf(rest_max, greedy_rounds(a, sh, live0, live1, batch, Sp, d, true));
  if (tid == 0) {
    if (a.max_abs_out) { a.max_abs_out[0] = maxw; a.max_abs_out[1] = maxwp; a.max_abs_out[2] = step; }
    *a.qa_step_dev = step;
    *a.n_touched = sh.n_touched;
    if (sh.bad) flag(a.dev_status, OCS_DEV_NONFINITE);
  }
}

__global__ void __launch_bounds__(kPlanThreads, 1) split_plan_kernel(PlanArgs a) {
  extern __shared__ __align__(16) unsigned char plan_smem[];
  split_plan_body(a, plan_smem);
}

// ------------------------------------------------------------------------------------------------
// K3: W'[o][j][r] = path_j(W[o][idx_map[j]][r]).  Threads own 4 consecutive output columns.
template <bool VEC>
__global__ void __launch_bounds__(256)
split_scatter_kernel(const float* __restrict__ W, int O, int C, int R, int64_t ld_in, int S,
                     float* __restrict__ Wout, int64_t ld_out, const int32_t* __restrict__ idx_map,
                     const int32_t* __restrict__ depth, const unsigned long long* __restrict__ bits,
                     const float* __restrict__ qa_step_dev) {
  const int ncols_out = (C + S) * R;
  const int col_blocks = (ncols_out + 1023) / 1024;
  long long u, u1;
  cta_range((long long)col_blocks * O, &u, &u1, blockIdx.x, gridDim.x);
  const float d = __fmul_rn(*qa_step_dev, 0.5f);
  while (u < u1) {
    const int cb = (int)(u / O);
    const int r0 = (int)(u - (long long)cb * O);
    const int r1 = (int)min((long long)O, r0 + (u1 - u));
    u += r1 - r0;
    const int e0 = (cb * 256 + threadIdx.x) * 4;
    if (e0 >= ncols_out) continue;
    const bool full = e0 + 3 < ncols_out;
    if (VEC && full && e0 + 3 < C * R) {
      // four original columns: they move as one 16-byte word; only split channels change value
      int dep[4];
      unsigned long long bt[4];
      int any = 0;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int j = (e0 + c) / R;
        dep[c] = min(depth[j], d == 0.0f ? kMaxHalvings : 64);
        bt[c] = bits[j];
        any |= dep[c];
      }
      const float4* src = reinterpret_cast<const float4*>(W + (int64_t)r0 * ld_in + e0);
      float4* dst = reinterpret_cast<float4*>(Wout + (int64_t)r0 * ld_out + e0);
      const int64_t sstride = ld_in >> 2, dstride = ld_out >> 2;
      if (!any) {
#pragma unroll 8
        for (int row = r0; row < r1; ++row) {
          __stcs(dst, __ldcs(src));
          src += sstride;
          dst += dstride;
        }
      } else {
#pragma unroll 2
        for (int row = r0; row < r1; ++row) {
          const float4 t = __ldcs(src);
          float v[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            float w = v[c];
            for (int i = 0; i < dep[c]; ++i)
              w = (i < 64 && ((bt[c] >> i) & 1ull)) ? split_new(w, d) : split_keep(w, d);
            v[c] = w;
          }
          __stcs(dst, make_float4(v[0], v[1], v[2], v[3]));
          src += sstride;
          dst += dstride;
        }
      }
      continue;
    }
    int src[4], dep[4];
    unsigned long long bt[4];
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
    }
#pragma unroll 4
    for (int row = r0; row < r1; ++row) {
      float v[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] = (e0 + c < ncols_out) ? __ldg(W + (int64_t)row * ld_in + src[c]) : 0.0f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float w = v[c];
        for (int i = 0; i < dep[c]; ++i)
          w = (i < 64 && ((bt[c] >> i) & 1ull)) ? split_new(w, d) : split_keep(w, d);
        v[c] = w;
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
}

// ------------------------------------------------------------------------------------------------
// K3, bulk-copy form.  A group of whole rows is brought into shared memory by the copy engine
// (cp.async.bulk, one copy per row, completion on an mbarrier), laid out with the output's row
// length; threads only compute the 2S channels per row that change -- the S appended copies, read
// from their source channels in shared memory, then the split originals in place -- and the
// finished rows leave by bulk stores.  Every byte of W is read from DRAM once, every byte of W'
// written once, and the duplicated channels are gathered from shared memory, not from global.
// Two row-group buffers alternate: the load of group i+1 and the store of group i-1 overlap the
// (small) compute of group i.  One CTA per SM; row groups are dealt round-robin.
constexpr int kRowThreads = 512;
constexpr int kRowRing = 4;                         // row-group buffers a CTA may cycle through
constexpr long long kRowWaitCycles = 2000000000ll;  // about one second

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ float apply_path(float w, int dep, unsigned long long bt, float d) {
  for (int i = 0; i < dep; ++i) w = (i < 64 && ((bt >> i) & 1ull)) ? split_new(w, d) : split_keep(w, d);
  return w;
}

__device__ __forceinline__ bool row_bar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// What happens to a finished row of W' in shared memory:
//   ROWS_STORE  it is written out as fp32 (ocs_split)
//   ROWS_HIST   its |values| are added to the clip search's histogram, nothing is written
//   ROWS_QUANT  it is quantized and only the codes are written
// The last two serve ocs_split_quantize, which never materialises the fp32 W'.
enum { ROWS_STORE = 0, ROWS_HIST = 1, ROWS_QUANT = 2 };

struct RowsEpilogue {
  const float* maxp;            // max|W'| (device scalar from the plan)
  int n_bins;                   // HIST
  unsigned long long* hist;     // HIST: global histogram [n_bins]
  int hist_copies;              // HIST: private copies of the counters (one per group of warps) behind the row buffers
  const double* scores;         // QUANT: candidate scores (null: no clipping)
  int n_candidates;
  int L;                        // QUANT: code range [-L, L], or [0, L] for unsigned codes
  int is_signed;
  int8_t* codes;                // QUANT: [O][ld_codes]
  long long ld_codes;
  int packed_ok;                // QUANT: 32-bit stores of four codes allowed
  float* scale_out;
  float* alpha_out;
  long long wait_cycles;        // limit of the wait for a row group's copies; 0 = the default (about a second)
  int drop_last_load;           // self-test only: the CTA's last row group is never requested, so its wait runs out
  int n_buf;                    // row-group buffers in the ring (2..kRowRing; 0 means 2)
};

template <int MODE>
__device__ __forceinline__ void
split_rows_body(const float* __restrict__ W, int O, int C, int R, int64_t ld_in, int S, float* __restrict__ Wout,
                int64_t ld_out, const int32_t* __restrict__ idx_map, const int32_t* __restrict__ depth,
                const unsigned long long* __restrict__ bits, const float* __restrict__ qa_step_dev,
                const int32_t* __restrict__ touched, const int* __restrict__ n_touched, int rows_per_group,
                int srow /*floats between rows in shared memory*/, RowsEpilogue ep, int* dev_status,
                unsigned char* row_smem, int vb, int vg) {
  __shared__ __align__(8) unsigned long long bars[kRowRing];
  __shared__ int abort_flag;
  const int n_buf = ep.n_buf >= 2 ? min(ep.n_buf, kRowRing) : 2;
  const size_t buf_floats = (size_t)rows_per_group * srow;
  auto buf_at = [&](int b) { return reinterpret_cast<float*>(row_smem) + (size_t)b * buf_floats; };
  // Row groups requested ahead of the one in work.  A buffer is refilled once its last user is done
  // with it: the threads, as soon as the CTA barrier that ends their group is passed; a bulk store,
  // once it has read the buffer -- so with stores the ring keeps one buffer more out of the loads'
  // way (the newest store may still be reading) whenever it has three or more.
  const int store_lag = (MODE == ROWS_STORE && n_buf >= 3) ? 1 : 0;
  const int ahead = n_buf - 1 - store_lag;
  const int tid = threadIdx.x;
  const int in_cols = C * R;                 // a multiple of 4 (checked by the host)
  const int out_cols = (C + S) * R;
  const int out_bulk = out_cols & ~3;        // floats per row that leave by bulk store
  const int n_groups = (O + rows_per_group - 1) / rows_per_group;
  const int my_groups = vb < n_groups ? (n_groups - 1 - vb) / vg + 1 : 0;
  const float d = __fmul_rn(*qa_step_dev, 0.5f);
  const int nt = *n_touched;
  const int dep_cap = d == 0.0f ? kMaxHalvings : 64;
  const long long wait_limit = ep.wait_cycles > 0 ? ep.wait_cycles : kRowWaitCycles;

  // epilogue state
  unsigned int* hist_sh = reinterpret_cast<unsigned int*>(row_smem + (size_t)n_buf * buf_floats * sizeof(float));
  float invw = 0.0f, q_inv = 0.0f, q_lo = 0.0f, q_hi = 0.0f;
  if (MODE == ROWS_HIST) {
    for (int i = tid; i < ep.hist_copies * ep.n_bins; i += kRowThreads) hist_sh[i] = 0u;
    const float m = *ep.maxp;
    invw = m > 0.0f ? __fdiv_rn((float)ep.n_bins, m) : 0.0f;
  }
  if (MODE == ROWS_QUANT) {
    float alpha = *ep.maxp;
    if (ep.scores && alpha > 0.0f) alpha = pick_alpha(ep.scores, alpha, ep.n_candidates);
    const bool zero = !(alpha > 0.0f);
    const float step = zero ? 0.0f : __fdiv_rn(alpha, (float)ep.L);
    q_inv = zero ? 0.0f : __fdiv_rn((float)ep.L, alpha);
    q_lo = ep.is_signed ? -(float)ep.L : 0.0f; q_hi = (float)ep.L;
    if (vb == 0 && tid == 0) {
      *ep.scale_out = step;
      if (ep.alpha_out) *ep.alpha_out = zero ? 0.0f : alpha;
    }
  }

  if (tid == 0) {
    for (int b = 0; b < kRowRing; ++b)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[b])) : "memory");
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  auto issue_load = [&](int i, int slot) {   // thread 0 only; slot = i mod n_buf
    const int g = vb + i * vg;
    const int r0 = g * rows_per_group;
    const int gn = min(rows_per_group, O - r0);
    const uint32_t bar = smem_addr(&bars[slot]);
    float* dst = buf_at(slot);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)gn * in_cols * 4u)
                 : "memory");
    for (int rl = 0; rl < gn; ++rl) {
      const float* src = W + (int64_t)(r0 + rl) * ld_in;
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
          ::"r"(smem_addr(dst + (size_t)rl * srow)), "l"(src), "r"((uint32_t)in_cols * 4u), "r"(bar)
          : "memory");
    }
  };

  // With one row per group every row needs the same (source, path) items: a thread keeps its
  // share of them in registers instead of re-reading the plan's arrays for every row.
  constexpr int kItems = 8;
  const int tail_items = S * R;
  const int orig_items = nt * R;
  const bool cached = rows_per_group == 1 && tail_items <= kItems * kRowThreads && orig_items <= kItems * kRowThreads;
  int t_src[kItems], t_dep[kItems], o_off[kItems], o_dep[kItems];
  unsigned long long t_bits[kItems];
  if (cached) {
#pragma unroll
    for (int k = 0; k < kItems; ++k) {
      const int e = tid + k * kRowThreads;
      t_src[k] = -1; t_dep[k] = 0; t_bits[k] = 0ull; o_off[k] = -1; o_dep[k] = 0;
      if (e < tail_items) {
        const int sidx = e / R, r = e - sidx * R;
        const int j = C + sidx;
        t_src[k] = __ldg(idx_map + j) * R + r;
        t_dep[k] = min(__ldg(depth + j), dep_cap);
        t_bits[k] = __ldg(bits + j);
      }
      if (e < orig_items) {
        const int t = e / R, r = e - t * R;
        const int j = __ldg(touched + t);
        o_off[k] = j * R + r;
        o_dep[k] = min(__ldg(depth + j), dep_cap);
      }
    }
  }

  // self-test: the last group's copies are never requested (nothing is in flight when its wait gives up)
  const int load_groups = ep.drop_last_load ? my_groups - 1 : my_groups;
  int issued = 0;
  int load_slot = 0;                       // buffer of the next group to request (thread 0)
  if (tid == 0) {
    for (int k = 0; k < ahead && k < load_groups; ++k) {
      issue_load(k, load_slot);
      ++issued;
      load_slot = load_slot + 1 == n_buf ? 0 : load_slot + 1;
    }
  }
  int b = 0;                               // buffer of the group in work, and how often the ring has wrapped
  uint32_t parity = 0;
  for (int i = 0; i < my_groups; ++i) {
    if (tid == 0) {
      // the bulk stores that read the buffer about to be refilled have finished reading it
      if (MODE == ROWS_STORE) {
        if (store_lag) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      }
      if (i + ahead < load_groups) {
        issue_load(i + ahead, load_slot);
        ++issued;
        load_slot = load_slot + 1 == n_buf ? 0 : load_slot + 1;
      }
    }
    {  // bounded wait for this group's rows
      const uint32_t bar = smem_addr(&bars[b]);
      if (!row_bar_try(bar, parity)) {
        const long long t0 = clock64();
        for (uint32_t it = 1;; ++it) {
          if (row_bar_try(bar, parity)) break;
          if ((it & 63u) == 0u && (abort_flag || clock64() - t0 > wait_limit)) { abort_flag = 1; break; }
        }
      }
    }
    __syncthreads();
    if (abort_flag) break;
    const int g = vb + i * vg;
    const int r0 = g * rows_per_group;
    const int gn = min(rows_per_group, O - r0);
    float* rows = buf_at(b);
    if (cached) {
      // appended copies: channel C + s reads its source channel's original values
#pragma unroll
      for (int k = 0; k < kItems; ++k) {
        if (t_src[k] >= 0) {
          const float v = apply_path(rows[t_src[k]], t_dep[k], t_bits[k], d);
          const int col = in_cols + tid + k * kRowThreads;
          rows[col] = v;
          if (MODE == ROWS_STORE && col >= out_bulk) Wout[(int64_t)r0 * ld_out + col] = v;   // the last 1-3 floats of a row
        }
      }
      __syncthreads();
      // split originals, in place: the kept copy takes the (w - d)/2 branch at every level
#pragma unroll
      for (int k = 0; k < kItems; ++k)
        if (o_off[k] >= 0) rows[o_off[k]] = apply_path(rows[o_off[k]], o_dep[k], 0ull, d);
    } else {
      for (int it = tid; it < gn * tail_items; it += kRowThreads) {
        const int rl = it / tail_items, e = it - rl * tail_items;
        const int sidx = e / R, r = e - sidx * R;
        const int j = C + sidx;
        const float v = apply_path(rows[(size_t)rl * srow + (size_t)__ldg(idx_map + j) * R + r],
                                   min(__ldg(depth + j), dep_cap), __ldg(bits + j), d);
        const int col = in_cols + e;
        rows[(size_t)rl * srow + col] = v;
        if (MODE == ROWS_STORE && col >= out_bulk) Wout[(int64_t)(r0 + rl) * ld_out + col] = v;
      }
      __syncthreads();
      for (int it = tid; it < gn * orig_items; it += kRowThreads) {
        const int rl = it / orig_items, e = it - rl * orig_items;
        const int t = e / R, r = e - t * R;
        const int j = __ldg(touched + t);
        float* q = rows + (size_t)rl * srow + (size_t)j * R + r;
        *q = apply_path(*q, min(__ldg(depth + j), dep_cap), 0ull, d);
      }
    }
    // The threads' (generic-proxy) writes into the row buffer are ordered before what the copy engine (async
    // proxy) does with the same bytes next: the bulk store that reads them (ROWS_STORE), and in every mode the
    // bulk load that refills this buffer later.  Each writing thread fences, then the CTA barrier orders the
    // fences before thread 0's next copy.
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (MODE == ROWS_STORE) {
      if (tid == 0 && out_bulk > 0) {
        for (int rl = 0; rl < gn; ++rl) {
          float* dst = Wout + (int64_t)(r0 + rl) * ld_out;
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                       ::"l"(dst), "r"(smem_addr(rows + (size_t)rl * srow)), "r"((uint32_t)out_bulk * 4u)
                       : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    } else {
      // the finished rows are consumed straight from shared memory
      const int quads = out_cols >> 2;
      for (int rl = 0; rl < gn; ++rl) {
        const float* row = rows + (size_t)rl * srow;
        if (MODE == ROWS_HIST) {
          if (invw > 0.0f) {
            unsigned int* mine = hist_sh + ((tid >> 5) % ep.hist_copies) * ep.n_bins;
            const int last = ep.n_bins - 1;
            auto count = [&](float xv) { atomicAdd(&mine[hist_bin(xv, invw, last)], 1u); };
            // A thread's share of the row is loaded first and counted afterwards: the loads are in flight together
            // and the counter updates (which return nothing) follow one another without a dependent load between.
            constexpr int kQ = 6;
            if (quads <= kQ * kRowThreads) {
              float4 v[kQ];
#pragma unroll
              for (int k = 0; k < kQ; ++k) {
                const int q = tid + k * kRowThreads;
                if (q < quads) v[k] = reinterpret_cast<const float4*>(row)[q];
              }
#pragma unroll
              for (int k = 0; k < kQ; ++k) {
                if (tid + k * kRowThreads < quads) { count(v[k].x); count(v[k].y); count(v[k].z); count(v[k].w); }
              }
            } else {
              for (int q = tid; q < quads; q += kRowThreads) {
                const float4 v = reinterpret_cast<const float4*>(row)[q];
                count(v.x); count(v.y); count(v.z); count(v.w);
              }
            }
            if (tid < (out_cols & 3)) count(row[(quads << 2) + tid]);
          }
        } else {
          int8_t* out = ep.codes + (long long)(r0 + rl) * ep.ld_codes;
          for (int q = tid; q < quads; q += kRowThreads) {
            const float4 v = reinterpret_cast<const float4*>(row)[q];
            const unsigned int word = pack4(quant_code(v.x, q_inv, q_lo, q_hi), quant_code(v.y, q_inv, q_lo, q_hi),
                                            quant_code(v.z, q_inv, q_lo, q_hi), quant_code(v.w, q_inv, q_lo, q_hi));
            if (ep.packed_ok) {
              *reinterpret_cast<unsigned int*>(out + 4 * q) = word;
            } else {
#pragma unroll
              for (int k = 0; k < 4; ++k) out[4 * q + k] = (int8_t)((word >> (8 * k)) & 0xFFu);
            }
          }
          if (tid < (out_cols & 3)) out[(quads << 2) + tid] = (int8_t)quant_code(row[(quads << 2) + tid], q_inv, q_lo, q_hi);
        }
      }
      __syncthreads();   // the buffer may be refilled now
    }
    b = b + 1 == n_buf ? 0 : b + 1;
    if (b == 0) parity ^= 1u;
  }
  if (MODE == ROWS_HIST) {
    __syncthreads();
    for (int bin = tid; bin < ep.n_bins; bin += kRowThreads) {
      unsigned int c = 0u;
      for (int k = 0; k < ep.hist_copies; ++k) c += hist_sh[k * ep.n_bins + bin];
      if (c) atomicAdd(&ep.hist[bin], (unsigned long long)c);
    }
  }
  if (tid == 0) {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (abort_flag) {
      flag(dev_status, OCS_DEV_TIMEOUT);
      if (issued > 0)
        for (int k = 0; k < 2000; ++k) __nanosleep(100);   // let copies still in flight land
    }
  }
  __syncthreads();
}

template <int MODE>
__global__ void __launch_bounds__(kRowThreads, 1)
split_rows_kernel(const float* __restrict__ W, int O, int C, int R, int64_t ld_in, int S, float* __restrict__ Wout,
                  int64_t ld_out, const int32_t* __restrict__ idx_map, const int32_t* __restrict__ depth,
                  const unsigned long long* __restrict__ bits, const float* __restrict__ qa_step_dev,
                  const int32_t* __restrict__ touched, const int* __restrict__ n_touched, int rows_per_group,
                  int srow /*floats between rows in shared memory*/, RowsEpilogue ep, int* dev_status) {
  extern __shared__ __align__(128) unsigned char row_smem_dyn[];
  split_rows_body<MODE>(W, O, C, R, ld_in, S, Wout, ld_out, idx_map, depth, bits, qa_step_dev, touched, n_touched,
                        rows_per_group, srow, ep, dev_status, row_smem_dyn, blockIdx.x, gridDim.x);
}

struct SplitWs {
  uint32_t* colmin; uint32_t* colmax;
  float* chmin; float* chmax; float* chkey;
  int32_t* depth; unsigned long long* bits;
  float* qa_step_dev;
  int32_t* touched; int* n_touched;
  unsigned long long* g_buf;
  int cap, npad, Sp;
  size_t plan_words;
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
  w.chmin = reinterpret_cast<float*>(take(4 * ((size_t)C + S)));
  w.chmax = reinterpret_cast<float*>(take(4 * ((size_t)C + S)));
  w.chkey = reinterpret_cast<float*>(take(4 * (size_t)C));
  w.depth = reinterpret_cast<int32_t*>(take(4 * ((size_t)C + S)));
  w.bits = reinterpret_cast<unsigned long long*>(take(8 * ((size_t)C + S)));
  w.qa_step_dev = reinterpret_cast<float*>(take(256));
  w.n_touched = reinterpret_cast<int*>(take(256));
  w.Sp = S < C ? S : C;
  w.touched = reinterpret_cast<int32_t*>(take(4 * (size_t)(w.Sp > 0 ? w.Sp : 1)));
  w.cap = w.Sp + S;
  w.npad = 1;
  while (w.npad < w.cap) w.npad <<= 1;
  w.plan_words = (size_t)w.Sp + 2 * (size_t)w.cap + (size_t)w.npad;
  if (S > kPlanSmemSplits) w.g_buf = reinterpret_cast<unsigned long long*>(take(8 * w.plan_words));
  w.total = off;
  return w;
}

// Rows-per-buffer, row-group count and shared-memory bytes of the row-staged kernels.
struct RowsGeometry {
  long long g;
  int n_groups;
  int n_buf;
  size_t rows_smem;
};
RowsGeometry rows_geometry(int O, size_t row_bytes, size_t hist_bytes) {
  RowsGeometry q{};
  // rows that fit beside the histogram counters (the caller checked that two do)
  const size_t n_fit = (kRowSmemBytes - hist_bytes) / row_bytes;
  q.n_buf = n_fit >= (size_t)kRowRing ? kRowRing : (int)n_fit;
  q.g = (long long)(n_fit / q.n_buf);
  q.g = min(q.g, (long long)max(1, O / (kNumSMs * q.n_buf)));   // every SM should get a ring's worth of groups
  q.g = min(q.g, 64ll);
  q.n_groups = (int)((O + q.g - 1) / q.g);
  q.rows_smem = (size_t)q.n_buf * (size_t)q.g * row_bytes;
  return q;
}

// Grid of a streaming kernel: one resident wave, but no more CTAs than there are 8-row slices.
template <typename K>
int wave_grid(K kernel, long long units) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, 256, 0) != cudaSuccess || per_sm < 1) per_sm = 4;
  const long long cap = (long long)kNumSMs * per_sm;
  const long long want = (units + 7) / 8;
  return (int)(want < cap ? (want > 0 ? want : 1) : cap);
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

namespace ocs {
namespace {

// The part ocs_split and ocs_split_quantize share: channel extrema and the greedy plan.
ocs_status run_split_front(const float* W, int O, int C, int R, int64_t ld_in, int S, float qa_step, int qa_bits,
                           int32_t* idx_map, int32_t* split_order, float* max_abs_out, const SplitWs& w,
                           int* dev_status, cudaStream_t stream, float* curve = nullptr) {
  ocs_status st;
  const int ncols = C * R;
  if (cudaMemsetAsync(w.colmin, 0xFF, 4 * (size_t)ncols, stream) != cudaSuccess) return OCS_ERR_CUDA;
  if (cudaMemsetAsync(w.colmax, 0x00, 4 * (size_t)ncols, stream) != cudaSuccess) return OCS_ERR_CUDA;

  {
    const long long units = (long long)((ncols + 1023) / 1024) * O;
    const bool vec = (ld_in % 4 == 0) && aligned(W, 16);
    LaunchScope ls("col_minmax_kernel", stream);
    if (ncols <= 512 && vec)
      col_minmax_narrow_kernel<true><<<wave_grid(col_minmax_narrow_kernel<true>, units), 256, 0, stream>>>(
          W, O, ncols, ld_in, w.colmin, w.colmax, C, idx_map, w.depth, w.bits, dev_status);
    else if (ncols <= 512)
      col_minmax_narrow_kernel<false><<<wave_grid(col_minmax_narrow_kernel<false>, units), 256, 0, stream>>>(
          W, O, ncols, ld_in, w.colmin, w.colmax, C, idx_map, w.depth, w.bits, dev_status);
    else if (vec)
      col_minmax_kernel<true><<<wave_grid(col_minmax_kernel<true>, units), 256, 0, stream>>>(
          W, O, ncols, ld_in, w.colmin, w.colmax, C, idx_map, w.depth, w.bits, dev_status);
    else
      col_minmax_kernel<false><<<wave_grid(col_minmax_kernel<false>, units), 256, 0, stream>>>(
          W, O, ncols, ld_in, w.colmin, w.colmax, C, idx_map, w.depth, w.bits, dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  {
    PlanArgs a{};
    a.colmin = w.colmin; a.colmax = w.colmax;
    a.C = C; a.R = R; a.S = S; a.qa_step = qa_step; a.qa_bits = qa_bits;
    a.chmin = w.chmin; a.chmax = w.chmax; a.chkey = w.chkey;
    a.idx_map = idx_map; a.split_order = split_order; a.depth = w.depth; a.bits = w.bits;
    a.max_abs_out = max_abs_out; a.qa_step_dev = w.qa_step_dev;
    a.touched = w.touched; a.n_touched = w.n_touched;
    a.g_buf = w.g_buf; a.cap = w.cap; a.npad = w.npad; a.Sp = w.Sp;
    a.curve = curve;
    a.dev_status = dev_status;
    // dynamic shared memory: the plan buffer (when S is small enough) and, overlapping the part of
    // it that the live sets only use after the selection, the selection histograms and the keys
    const size_t plan_bytes = (S <= kPlanSmemSplits) ? 8 * w.plan_words : 0;
    const size_t hist_off = (S <= kPlanSmemSplits) ? align_up(8 * (size_t)w.Sp, 16) : 0;
    const size_t keys_off = hist_off + kSelHistBytes;
    const bool keys_fit = keys_off + 4 * (size_t)C <= (size_t)kPlanSmemBytes;
    a.hist_off = (int)hist_off;
    a.keys_off = keys_fit ? (int)keys_off : -1;
    size_t smem = keys_fit ? keys_off + 4 * (size_t)C : keys_off;
    if (plan_bytes > smem) smem = plan_bytes;
    static bool attr_set = false;
    if (!attr_set) {
      if (cudaFuncSetAttribute(split_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPlanSmemBytes) != cudaSuccess)
        return OCS_ERR_CUDA;
      attr_set = true;
    }
    LaunchScope ls("split_plan_kernel", stream);
    split_plan_kernel<<<1, kPlanThreads, smem, stream>>>(a);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  return OCS_OK;
}

}  // namespace
}  // namespace ocs

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

  if ((st = run_split_front(W, O, C, R, ld_in, S, qa_step, qa_bits, idx_map, split_order, max_abs_out, w, dev_status,
                            stream)) != OCS_OK)
    return st;
  {
    const int ncols_out = (C + S) * R;
    const bool vec = (ld_in % 4 == 0) && (ld_out % 4 == 0) && aligned(W, 16) && aligned(W_out, 16);
    const int srow = (ncols_out + 3) & ~3;
    const size_t row_bytes = 4 * (size_t)srow;
    const bool staged = vec && (C * R) % 4 == 0 && 2 * row_bytes <= kRowSmemBytes;
    LaunchScope ls(staged ? "split_rows_kernel" : "split_scatter_kernel", stream);
    if (staged) {
      const RowsGeometry geo = rows_geometry(O, row_bytes, 0);
      const long long g = geo.g;
      const int n_groups = geo.n_groups;
      RowsEpilogue ep{};
      ep.n_buf = geo.n_buf;
      static bool attr_set = false;
      if (!attr_set) {
        if (cudaFuncSetAttribute(split_rows_kernel<ROWS_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kRowSmemBytes) != cudaSuccess)
          return OCS_ERR_CUDA;
        attr_set = true;
      }
      split_rows_kernel<ROWS_STORE><<<min(n_groups, kNumSMs), kRowThreads, geo.rows_smem, stream>>>(
          W, O, C, R, ld_in, S, W_out, ld_out, idx_map, w.depth, w.bits, w.qa_step_dev, w.touched, w.n_touched, (int)g,
          srow, ep, dev_status);
    } else {
      const long long units = (long long)((ncols_out + 1023) / 1024) * O;
      if (vec)
        split_scatter_kernel<true><<<wave_grid(split_scatter_kernel<true>, units), 256, 0, stream>>>(
            W, O, C, R, ld_in, S, W_out, ld_out, idx_map, w.depth, w.bits, w.qa_step_dev);
      else
        split_scatter_kernel<false><<<wave_grid(split_scatter_kernel<false>, units), 256, 0, stream>>>(
            W, O, C, R, ld_in, S, W_out, ld_out, idx_map, w.depth, w.bits, w.qa_step_dev);
    }
    if ((st = launch_status()) != OCS_OK) return st;
  }
  return OCS_OK;
}

// ------------------------------------------------------------------------------------------------
// ocs_selftest_wait_expiry: makes a bounded device wait run out, on purpose and safely.  The row-staged copy
// kernel runs on W with no splits, but every CTA leaves out the request for its last row group and waits for
// it with a limit of about a millisecond: the wait expires, the CTA sets OCS_DEV_TIMEOUT and returns with no
// copy in flight.  Rows of the dropped groups are left unwritten.  Nothing traps and nothing spins unbounded.
extern "C" ocs_status ocs_selftest_wait_expiry(const float* W, int O, int C, int64_t ld_in, float* W_out, int64_t ld_out,
                                               void* ws, size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!W || !W_out || !dev_status) return OCS_ERR_INVALID_ARG;
  if (O <= 0 || C <= 0 || C % 4 != 0 || ld_in < C || ld_out < C || ld_in % 4 != 0 || ld_out % 4 != 0) return OCS_ERR_SHAPE;
  if (!aligned(W, 16) || !aligned(W_out, 16)) return OCS_ERR_SHAPE;
  const size_t row_bytes = 4 * (size_t)C;
  if (2 * row_bytes > kRowSmemBytes) return OCS_ERR_UNSUPPORTED;
  const SplitWs w = carve_split_ws(ws, C, 1, 0);
  const size_t total = w.total + align_up(4 * (size_t)C, 256);
  if (!ws || !aligned(ws, 256) || ws_bytes < total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  int32_t* idx_map = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(ws) + w.total);
  if ((st = run_split_front(W, O, C, 1, ld_in, 0, 0.0f, 0, idx_map, nullptr, nullptr, w, dev_status, stream)) != OCS_OK)
    return st;
  long long g = (long long)(kRowSmemBytes / 2 / row_bytes);
  g = min(g, (long long)max(1, O / kNumSMs));
  g = min(g, 64ll);
  const int n_groups = (int)((O + g - 1) / g);
  if (cudaFuncSetAttribute(split_rows_kernel<ROWS_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)kRowSmemBytes) != cudaSuccess)
    return OCS_ERR_CUDA;
  RowsEpilogue ep{};
  ep.wait_cycles = 2000000ll;   // about a millisecond
  ep.drop_last_load = 1;
  LaunchScope ls("split_rows_kernel", stream);
  split_rows_kernel<ROWS_STORE><<<min(n_groups, kNumSMs), kRowThreads, 2 * (size_t)g * row_bytes, stream>>>(
      W, O, C, 1, ld_in, 0, W_out, ld_out, idx_map, w.depth, w.bits, w.qa_step_dev, w.touched, w.n_touched, (int)g, C, ep,
      dev_status);
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// ocs_range_curve: curve[s] = max|W'| after s greedy plain-halving splits (Section 3.4), s = 0..S_max: one pass
// over W for the channel extrema, then the plan kernel's rounds on the keys alone.  This is what the knapsack
// allocation's reward is made of.
extern "C" size_t ocs_range_curve_workspace_bytes(int C, int R, int S_max) {
  if (C <= 0 || R <= 0 || S_max < 0) return 0;
  return carve_split_ws(nullptr, C, R, S_max).total + align_up(4 * ((size_t)C + S_max), 256);
}

extern "C" ocs_status ocs_range_curve(const float* W, int O, int C, int R, int64_t ld_in, int S_max, float* curve,
                                      void* ws, size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!W || !curve || S_max < 0) return OCS_ERR_INVALID_ARG;
  if (O <= 0 || C <= 0 || R <= 0) return OCS_ERR_SHAPE;
  if ((int64_t)C * R >= (1ll << 31) || ((int64_t)C + S_max) * R >= (1ll << 31) || ld_in < (int64_t)C * R) return OCS_ERR_SHAPE;
  if (!aligned(W, 4)) return OCS_ERR_SHAPE;
  const SplitWs w = carve_split_ws(ws, C, R, S_max);
  const size_t total = w.total + align_up(4 * ((size_t)C + S_max), 256);
  if (!ws || !aligned(ws, 256) || ws_bytes < total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  // the extrema kernel also writes the identity part of an index map: it goes to scratch here
  int32_t* idx_scratch = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(ws) + w.total);
  return run_split_front(W, O, C, R, ld_in, S_max, 0.0f, 0, idx_scratch, nullptr, nullptr, w, dev_status, stream, curve);
}

// ------------------------------------------------------------------------------------------------
// ocs_split_quantize: split + clip search + quantization without the fp32 W'.
namespace ocs {
namespace {
struct FusedWs {
  SplitWs sp;
  float* mx3;
  unsigned long long* hist;
  double* scores;
  size_t total;
};
FusedWs carve_fused_ws(void* ws, int C, int R, int S, int n_bins, int n_candidates) {
  FusedWs f{};
  f.sp = carve_split_ws(ws, C, R, S);
  size_t off = f.sp.total;
  auto take = [&](size_t bytes) {
    unsigned char* p = ws ? reinterpret_cast<unsigned char*>(ws) + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  };
  f.mx3 = reinterpret_cast<float*>(take(256));
  f.hist = reinterpret_cast<unsigned long long*>(take(8 * (size_t)(n_bins > 0 ? n_bins : 1)));
  f.scores = reinterpret_cast<double*>(take(8 * (size_t)(n_candidates > 0 ? n_candidates : 1)));
  f.total = off;
  return f;
}
}  // namespace
}  // namespace ocs

namespace ocs {
namespace {
// Code pass for short rows under the plain w/2 split (the case of activation matrices: a row is one pixel's
// or one sample's channels).  Staging whole rows in shared memory buys nothing when a row is a few hundred
// bytes, so this form streams.  The warps of a CTA form two groups that walk the CTA's rows independently:
// the main group converts the original columns (a thread owns one group of four columns for every row it
// visits: one 128-bit load, halving counts in registers, one 32-bit store), the tail group the duplicated
// channels (four loads of source columns whose lines the main group has just read).  Keeping the two kinds
// of work in different warps keeps either from waiting on the other's divergent path.  Repeated halving
// keeps the checker's rounding, subnormals included.
__device__ __forceinline__ void
rows_quant_narrow_body(const float* __restrict__ W, int O, int C, int R, long long ld_in, int S,
                       const int32_t* __restrict__ idx_map, const int32_t* __restrict__ depth,
                       const float* __restrict__ maxp, const double* __restrict__ scores, int n_candidates, int L,
                       int is_signed, int8_t* __restrict__ codes, long long ld_codes, int packed_ok, int vec_ok,
                       int tail_warps, float* __restrict__ scale_out, float* __restrict__ alpha_out, int vb, int vg) {
  float alpha = *maxp;
  if (scores && alpha > 0.0f) alpha = pick_alpha(scores, alpha, n_candidates);
  const bool zero = !(alpha > 0.0f);
  const float step = zero ? 0.0f : __fdiv_rn(alpha, (float)L);
  const float inv = zero ? 0.0f : __fdiv_rn((float)L, alpha);
  const float lo = is_signed ? -(float)L : 0.0f, hi = (float)L;
  if (vb == 0 && threadIdx.x == 0) {
    *scale_out = step;
    if (alpha_out) *alpha_out = zero ? 0.0f : alpha;
  }
  const int in_cols = C * R, out_cols = (C + S) * R;
  const int main_threads = 256 - 32 * tail_warps;
  const bool is_tail = (int)threadIdx.x >= main_threads;
  const int t = is_tail ? (int)threadIdx.x - main_threads : (int)threadIdx.x;
  const int group = is_tail ? 32 * tail_warps : main_threads;
  const int first_col = is_tail ? in_cols : 0;
  const int n_quads = ((is_tail ? out_cols - in_cols : in_cols) + 3) >> 2;   // <= group (checked by the host)
  const int side = group / n_quads;
  const int lr = t / n_quads, col0 = first_col + (t - lr * n_quads) * 4;
  if (lr >= side) return;
  const int col_end = is_tail ? out_cols : in_cols;
  int src[4], dep[4];
  bool valid[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int col = col0 + e;
    valid[e] = col < col_end;
    src[e] = 0; dep[e] = 0;
    if (valid[e]) {
      const int ch = col / R, r = col - ch * R;
      dep[e] = min(__ldg(depth + ch), kMaxHalvings);   // further halvings leave (signed) zero
      src[e] = (ch < C ? ch : __ldg(idx_map + ch)) * R + r;
    }
  }
  const bool contiguous = !is_tail && vec_ok && valid[3];
  const bool any_dep = (dep[0] | dep[1] | dep[2] | dep[3]) != 0;
  long long r0, r1;
  cta_range((long long)O, &r0, &r1, vb, vg);
  auto emit = [&](long long r, float (&x)[4]) {
    if (any_dep) {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        for (int d = 0; d < dep[e]; ++d) x[e] = __fmul_rn(x[e], 0.5f);
    }
    const int c0 = quant_code(x[0], inv, lo, hi), c1 = quant_code(x[1], inv, lo, hi);
    const int c2 = quant_code(x[2], inv, lo, hi), c3 = quant_code(x[3], inv, lo, hi);
    int8_t* out = codes + r * ld_codes + col0;
    if (packed_ok && valid[3]) {
      *reinterpret_cast<unsigned int*>(out) = pack4(c0, c1, c2, c3);
    } else {
      if (valid[0]) out[0] = (int8_t)c0;
      if (valid[1]) out[1] = (int8_t)c1;
      if (valid[2]) out[2] = (int8_t)c2;
      if (valid[3]) out[3] = (int8_t)c3;
    }
  };
  if (contiguous) {
    // eight rows' loads in flight per thread before the first is consumed
    constexpr int kBatch = 8;
    const long long stride = (long long)side * ld_in;
    const float* p = W + (r0 + lr) * ld_in + col0;
    for (long long r = r0 + lr; r < r1; r += (long long)kBatch * side, p += kBatch * stride) {
      float4 v[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u)
        v[u] = (r + (long long)u * side < r1) ? __ldcs(reinterpret_cast<const float4*>(p + u * stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        if (r + (long long)u * side < r1) {
          float x[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
          emit(r + (long long)u * side, x);
        }
      }
    }
  } else {
#pragma unroll 2
    for (long long r = r0 + lr; r < r1; r += side) {
      const float* row = W + r * ld_in;
      float x[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) x[e] = valid[e] ? __ldg(row + src[e]) : 0.0f;
      emit(r, x);
    }
  }
}
__global__ void __launch_bounds__(256, 4)
rows_quant_narrow_kernel(const float* __restrict__ W, int O, int C, int R, long long ld_in, int S,
                         const int32_t* __restrict__ idx_map, const int32_t* __restrict__ depth,
                         const float* __restrict__ maxp, const double* __restrict__ scores, int n_candidates, int L,
                         int is_signed, int8_t* __restrict__ codes, long long ld_codes, int packed_ok, int vec_ok,
                         int tail_warps, float* __restrict__ scale_out, float* __restrict__ alpha_out) {
  rows_quant_narrow_body(W, O, C, R, ld_in, S, idx_map, depth, maxp, scores, n_candidates, L, is_signed, codes, ld_codes,
                         packed_ok, vec_ok, tail_warps, scale_out, alpha_out, blockIdx.x, gridDim.x);
}
}  // namespace
}  // namespace ocs

namespace ocs {
namespace {
ocs_status rows_attr_once() {
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(split_rows_kernel<ROWS_HIST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kRowSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(split_rows_kernel<ROWS_QUANT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kRowSmemBytes) != cudaSuccess)
      return OCS_ERR_CUDA;
    attr_set = true;
  }
  return OCS_OK;
}

// The code pass: rows staged in shared memory, split there, quantized and written as packed codes.
ocs_status launch_rows_quant(const float* W, int O, int C, int R, int64_t ld_in, int S, const int32_t* idx_map,
                             const SplitWs& w, RowsEpilogue ep, int8_t* codes, int64_t ld_codes, float* scale,
                             float* alpha, int g, int srow, int n_groups, size_t rows_smem, bool naive, int* dev_status,
                             cudaStream_t stream) {
  ep.codes = codes;
  ep.ld_codes = ld_codes;
  ep.packed_ok = aligned(codes, 4) && (ld_codes % 4 == 0);
  ep.scale_out = scale;
  ep.alpha_out = alpha;
  // short rows, plain halving: the streaming form (both column groups must fit their warps)
  const int main_quads = (C * R + 3) / 4, tail_quads = (S * R + 3) / 4;
  const int tail_warps = S == 0 ? 0 : (12 * tail_quads >= main_quads ? 2 : 1);
  if (naive && (C * R) % 4 == 0 && main_quads <= 256 - 32 * tail_warps && tail_quads <= 32 * tail_warps) {
    const int side = (256 - 32 * tail_warps) / main_quads;
    const int grid = wave_grid(rows_quant_narrow_kernel, ((long long)O + side - 1) / side);   // one resident wave
    const int vec_ok = (ld_in % 4 == 0) && aligned(W, 16);
    LaunchScope ls("split_quantize_kernel", stream);
    rows_quant_narrow_kernel<<<grid, 256, 0, stream>>>(W, O, C, R, ld_in, S, idx_map, w.depth, ep.maxp, ep.scores,
                                                       ep.n_candidates, ep.L, ep.is_signed, codes, ld_codes, ep.packed_ok,
                                                       vec_ok, tail_warps, scale, alpha);
    return launch_status();
  }
  LaunchScope ls("split_quantize_kernel", stream);
  split_rows_kernel<ROWS_QUANT><<<min(n_groups, kNumSMs), kRowThreads, rows_smem, stream>>>(
      W, O, C, R, ld_in, S, nullptr, 0, idx_map, w.depth, w.bits, w.qa_step_dev, w.touched, w.n_touched, g, srow, ep,
      dev_status);
  return launch_status();
}
}  // namespace
}  // namespace ocs

extern "C" size_t ocs_split_quantize_workspace_bytes(int O, int C, int R, int S, int n_bins, int n_candidates) {
  (void)O;
  if (C <= 0 || R <= 0 || S < 0) return 0;
  return carve_fused_ws(nullptr, C, R, S, n_bins, n_candidates).total;
}

extern "C" ocs_status ocs_split_quantize(const float* W, int O, int C, int R, int64_t ld_in, int S, float qa_step,
                                         int qa_bits, int bits, int is_signed, ocs_clip_mode mode, int n_candidates,
                                         int n_bins,
                                         int8_t* codes, int64_t ld_codes, int32_t* idx_map, int32_t* split_order,
                                         float* max_abs_out, float* scale, float* alpha, void* ws, size_t ws_bytes,
                                         int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!W || !codes || !idx_map || !scale) return OCS_ERR_INVALID_ARG;
  if (S < 0 || !(qa_step >= 0.0f) || !is_finite_host(qa_step)) return OCS_ERR_INVALID_ARG;
  if (qa_bits != 0 && (qa_bits < 2 || qa_bits > 8)) return OCS_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return OCS_ERR_INVALID_ARG;
  if (mode != OCS_CLIP_NONE && mode != OCS_CLIP_MSE && mode != OCS_CLIP_KL && mode != OCS_CLIP_ACIQ)
    return OCS_ERR_INVALID_ARG;
  const bool hist_mode = mode != OCS_CLIP_NONE;
  if (mode == OCS_CLIP_ACIQ) n_candidates = 1;
  if (hist_mode && (n_candidates < 1 || n_candidates > 1024 || n_bins < 1 || n_bins > 4096))
    return OCS_ERR_INVALID_ARG;
  if (O <= 0 || C <= 0 || R <= 0) return OCS_ERR_SHAPE;
  if ((int64_t)C * R >= (1ll << 31) || ((int64_t)C + S) * R >= (1ll << 31)) return OCS_ERR_SHAPE;
  const int ncols_out = (C + S) * R;
  if (ld_in < (int64_t)C * R || ld_codes < ncols_out) return OCS_ERR_SHAPE;
  if (mode == OCS_CLIP_NONE) { n_bins = 1; n_candidates = 1; }
  // rows are staged whole in shared memory: they must be 16-byte addressable and fit twice
  const int srow = (ncols_out + 3) & ~3;
  const size_t row_bytes = 4 * (size_t)srow;
  const size_t hist_bytes = hist_mode ? 4 * (size_t)n_bins : 0;
  if (!(ld_in % 4 == 0 && aligned(W, 16) && (C * R) % 4 == 0 && 2 * row_bytes + hist_bytes <= kRowSmemBytes))
    return OCS_ERR_UNSUPPORTED;
  const FusedWs f = carve_fused_ws(ws, C, R, S, n_bins, n_candidates);
  if (!ws || !aligned(ws, 256) || ws_bytes < f.total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const SplitWs& w = f.sp;
  float* mx3 = max_abs_out ? max_abs_out : f.mx3;
  if ((st = run_split_front(W, O, C, R, ld_in, S, qa_step, qa_bits, idx_map, split_order, mx3, w, dev_status, stream)) !=
      OCS_OK)
    return st;

  const RowsGeometry geo = rows_geometry(O, row_bytes, 0);   // the code pass keeps no counters
  const long long g = geo.g;
  const int n_groups = geo.n_groups;
  const size_t rows_smem = geo.rows_smem;
  if ((st = rows_attr_once()) != OCS_OK) return st;
  const int L = is_signed ? (1 << (bits - 1)) - 1 : (1 << bits) - 1;
  RowsEpilogue ep{};
  ep.maxp = mx3 + 1;   // max|W'| as the plan computed it
  ep.n_buf = geo.n_buf;
  ep.L = L;
  ep.is_signed = is_signed ? 1 : 0;
  const double* scores = nullptr;
  if (hist_mode) {
    if (cudaMemsetAsync(f.hist, 0, 8 * (size_t)n_bins, stream) != cudaSuccess) return OCS_ERR_CUDA;
    ep.n_bins = n_bins;
    ep.hist = f.hist;
    // four counter copies when a full ring of rows fits beside them, else two or one
    int copies = 4;
    while (copies > 1 && (kRowSmemBytes - copies * hist_bytes) / row_bytes < (size_t)kRowRing) copies >>= 1;
    const RowsGeometry gh = rows_geometry(O, row_bytes, copies * hist_bytes);
    ep.hist_copies = copies;
    ep.n_buf = gh.n_buf;
    {
      LaunchScope ls("split_hist_kernel", stream);
      split_rows_kernel<ROWS_HIST><<<min(gh.n_groups, kNumSMs), kRowThreads, gh.rows_smem + copies * hist_bytes, stream>>>(
          W, O, C, R, ld_in, S, nullptr, 0, idx_map, w.depth, w.bits, w.qa_step_dev, w.touched, w.n_touched, (int)gh.g,
          srow, ep, dev_status);
    }
    ep.n_buf = geo.n_buf;
    if ((st = launch_status()) != OCS_OK) return st;
    if ((st = launch_clip_search(mode, f.hist, ep.maxp, n_bins, n_candidates, L, is_signed ? 1 : 0, f.scores,
                                 f.mx3 + 8, stream)) != OCS_OK)
      return st;
    if (mode == OCS_CLIP_ACIQ) ep.maxp = f.mx3 + 8;   // the closed-form threshold replaces max|W'|
    else scores = f.scores;
  }
  ep.scores = scores;
  ep.n_candidates = n_candidates;
  return launch_rows_quant(W, O, C, R, ld_in, S, idx_map, w, ep, codes, ld_codes, scale, alpha, (int)g, srow, n_groups,
                           rows_smem, qa_step == 0.0f && qa_bits == 0, dev_status, stream);
}

// ------------------------------------------------------------------------------------------------
// ocs_split_quantize_batch: ocs_split_quantize (plain halving, no clip search) for many layers in five launches
// instead of five per layer: one extrema pass, one plan launch with a CTA per layer, one code pass each for
// the short-row and the row-staged layers.  A network's layers are small next to the GPU (ResNet-50: 97 MiB of
// weights in 54 layers); launched one by one their kernels are latency-bound, together they stream at memory rate.
// The per-layer kernels' bodies are reused: a CTA of a batched launch looks up its layer and its position among
// that layer's CTAs.
namespace ocs {
namespace {
constexpr int kMaxBatch = 64;

struct BatchLayer {
  const float* W;
  int O, C, R, S;
  uint32_t* colmin; uint32_t* colmax;
  float* chmin; float* chmax; float* chkey;
  int32_t* depth; unsigned long long* bits;
  float* qa_step_dev; int32_t* touched; int* n_touched; unsigned long long* g_buf;
  int cap, npad, Sp, hist_off, keys_off;
  int32_t* idx_map; float* mx3;
  int8_t* codes; long long ld_codes; float* scale;
  int mm_blk0, mm_blks, mm_narrow, vec;            // extrema pass: first CTA, CTAs, kernel form, 128-bit loads
  int cp_kind, cp_blk0, cp_blks;                   // code pass: 0 = short rows, 1 = row-staged; first CTA, CTAs
  int tail_warps, packed_ok, rows_per_group, srow, n_buf; // code pass geometry
};
struct BatchTable {
  int n, L, is_signed, pad;
  BatchLayer l[kMaxBatch];
};

__global__ void __launch_bounds__(256)
batch_minmax_kernel(const __grid_constant__ BatchTable t, int* dev_status) {
  int li = 0;
  while (li + 1 < t.n && (int)blockIdx.x >= t.l[li + 1].mm_blk0) ++li;
  const BatchLayer& y = t.l[li];
  const int vb = (int)blockIdx.x - y.mm_blk0, vg = y.mm_blks;
  const int ncols = y.C * y.R;
  if (y.mm_narrow) {
    if (y.vec) col_minmax_narrow_body<true>(y.W, y.O, ncols, ncols, y.colmin, y.colmax, y.C, y.idx_map, y.depth, y.bits, dev_status, vb, vg);
    else col_minmax_narrow_body<false>(y.W, y.O, ncols, ncols, y.colmin, y.colmax, y.C, y.idx_map, y.depth, y.bits, dev_status, vb, vg);
  } else {
    if (y.vec) col_minmax_body<true>(y.W, y.O, ncols, ncols, y.colmin, y.colmax, y.C, y.idx_map, y.depth, y.bits, dev_status, vb, vg);
    else col_minmax_body<false>(y.W, y.O, ncols, ncols, y.colmin, y.colmax, y.C, y.idx_map, y.depth, y.bits, dev_status, vb, vg);
  }
}

__global__ void __launch_bounds__(kPlanThreads, 1)
batch_plan_kernel(const __grid_constant__ BatchTable t, int* dev_status) {
  extern __shared__ __align__(16) unsigned char plan_smem_b[];
  const BatchLayer& y = t.l[blockIdx.x];
  PlanArgs a{};
  a.colmin = y.colmin; a.colmax = y.colmax;
  a.C = y.C; a.R = y.R; a.S = y.S; a.qa_step = 0.0f; a.qa_bits = 0;
  a.chmin = y.chmin; a.chmax = y.chmax; a.chkey = y.chkey;
  a.idx_map = y.idx_map; a.split_order = nullptr; a.depth = y.depth; a.bits = y.bits;
  a.max_abs_out = y.mx3; a.qa_step_dev = y.qa_step_dev;
  a.touched = y.touched; a.n_touched = y.n_touched;
  a.g_buf = y.g_buf; a.cap = y.cap; a.npad = y.npad; a.Sp = y.Sp;
  a.hist_off = y.hist_off; a.keys_off = y.keys_off;
  a.curve = nullptr;
  a.dev_status = dev_status;
  split_plan_body(a, plan_smem_b);
}

// the layer of kind `kind` that CTA b of a code-pass launch belongs to (the launches of the two kinds number
// their CTAs separately)
__device__ __forceinline__ int code_layer(const BatchTable& t, int b, int kind) {
  int li = -1;
  for (int i = 0; i < t.n; ++i)
    if (t.l[i].cp_kind == kind && b >= t.l[i].cp_blk0) li = i;
  return li;
}

__global__ void __launch_bounds__(256, 4)
batch_narrow_code_kernel(const __grid_constant__ BatchTable t) {
  const BatchLayer& y = t.l[code_layer(t, (int)blockIdx.x, 0)];
  rows_quant_narrow_body(y.W, y.O, y.C, y.R, (long long)y.C * y.R, y.S, y.idx_map, y.depth, y.mx3 + 1, nullptr, 1, t.L,
                         t.is_signed, y.codes, y.ld_codes, y.packed_ok, y.vec, y.tail_warps, y.scale, nullptr,
                         (int)blockIdx.x - y.cp_blk0, y.cp_blks);
}

__global__ void __launch_bounds__(kRowThreads, 1)
batch_staged_code_kernel(const __grid_constant__ BatchTable t, int* dev_status) {
  extern __shared__ __align__(128) unsigned char row_smem_b[];
  const BatchLayer& y = t.l[code_layer(t, (int)blockIdx.x, 1)];
  RowsEpilogue ep{};
  ep.maxp = y.mx3 + 1;
  ep.L = t.L;
  ep.is_signed = t.is_signed;
  ep.scores = nullptr;
  ep.n_candidates = 1;
  ep.codes = y.codes;
  ep.ld_codes = y.ld_codes;
  ep.packed_ok = y.packed_ok;
  ep.scale_out = y.scale;
  ep.alpha_out = nullptr;
  ep.n_buf = y.n_buf;
  split_rows_body<ROWS_QUANT>(y.W, y.O, y.C, y.R, (int64_t)y.C * y.R, y.S, nullptr, 0, y.idx_map, y.depth, y.bits,
                              y.qa_step_dev, y.touched, y.n_touched, y.rows_per_group, y.srow, ep, dev_status, row_smem_b,
                              (int)blockIdx.x - y.cp_blk0, y.cp_blks);
}

// Table and workspace layout of a batch; false if a layer cannot go through the fused path.
struct BatchPlan {
  BatchTable t;
  int mm_grid, narrow_grid, staged_grid;
  size_t plan_smem, staged_smem;
  size_t colmin_bytes;   // all layers' column minima are one region (one memset), then all maxima
  size_t total;
};

bool plan_batch(const ocs_layer_desc* layers, int n, int bits, int is_signed, void* ws, BatchPlan* bp, ocs_status* why) {
  *why = OCS_OK;
  if (n < 1 || n > kMaxBatch) { *why = OCS_ERR_UNSUPPORTED; return false; }
  BatchTable& t = bp->t;
  memset(&t, 0, sizeof(t));
  t.n = n;
  t.L = is_signed ? (1 << (bits - 1)) - 1 : (1 << bits) - 1;
  t.is_signed = is_signed ? 1 : 0;
  size_t cm = 0;
  for (int i = 0; i < n; ++i) cm += align_up(4 * (size_t)layers[i].C * layers[i].R, 256);
  bp->colmin_bytes = cm;
  size_t off_min = 0, off = 2 * cm;
  auto at = [&](size_t o) { return ws ? reinterpret_cast<unsigned char*>(ws) + o : nullptr; };
  auto take = [&](size_t bytes) { unsigned char* q = at(off); off += align_up(bytes, 256); return q; };
  int mm_blk = 0, nb = 0, sb = 0;
  bp->plan_smem = 0; bp->staged_smem = 0;
  for (int i = 0; i < n; ++i) {
    const ocs_layer_desc& d = layers[i];
    BatchLayer& y = t.l[i];
    if (!d.W || !d.codes || !d.idx_map || !d.scale) { *why = OCS_ERR_INVALID_ARG; return false; }
    if (d.O <= 0 || d.C <= 0 || d.R <= 0 || d.S < 0) { *why = OCS_ERR_SHAPE; return false; }
    const long long ncols = (long long)d.C * d.R, ncols_out = ((long long)d.C + d.S) * d.R;
    if (ncols_out >= (1ll << 31) || d.ld_codes < ncols_out) { *why = OCS_ERR_SHAPE; return false; }
    const int srow = (int)((ncols_out + 3) & ~3ll);
    const size_t row_bytes = 4 * (size_t)srow;
    if (!(aligned(d.W, 16) && ncols % 4 == 0 && 2 * row_bytes <= kRowSmemBytes)) { *why = OCS_ERR_UNSUPPORTED; return false; }
    y.W = d.W; y.O = d.O; y.C = d.C; y.R = d.R; y.S = d.S;
    y.colmin = reinterpret_cast<uint32_t*>(at(off_min));
    y.colmax = reinterpret_cast<uint32_t*>(at(cm + off_min));
    off_min += align_up(4 * (size_t)ncols, 256);
    const size_t CS = (size_t)d.C + d.S;
    y.chmin = reinterpret_cast<float*>(take(4 * CS));
    y.chmax = reinterpret_cast<float*>(take(4 * CS));
    y.chkey = reinterpret_cast<float*>(take(4 * (size_t)d.C));
    y.depth = reinterpret_cast<int32_t*>(take(4 * CS));
    y.bits = reinterpret_cast<unsigned long long*>(take(8 * CS));
    y.qa_step_dev = reinterpret_cast<float*>(take(256));
    y.n_touched = reinterpret_cast<int*>(take(256));
    y.Sp = d.S < d.C ? d.S : d.C;
    y.touched = reinterpret_cast<int32_t*>(take(4 * (size_t)(y.Sp > 0 ? y.Sp : 1)));
    y.cap = y.Sp + d.S;
    y.npad = 1;
    while (y.npad < y.cap) y.npad <<= 1;
    const size_t plan_words = (size_t)y.Sp + 2 * (size_t)y.cap + (size_t)y.npad;
    y.g_buf = d.S > kPlanSmemSplits ? reinterpret_cast<unsigned long long*>(take(8 * plan_words)) : nullptr;
    y.mx3 = d.max_abs3 ? d.max_abs3 : reinterpret_cast<float*>(take(256));
    y.idx_map = d.idx_map; y.codes = d.codes; y.ld_codes = d.ld_codes; y.scale = d.scale;
    // plan kernel's shared memory, as in the single-layer call
    const size_t plan_bytes = (d.S <= kPlanSmemSplits) ? 8 * plan_words : 0;
    const size_t hist_off = (d.S <= kPlanSmemSplits) ? align_up(8 * (size_t)y.Sp, 16) : 0;
    const size_t keys_off = hist_off + kSelHistBytes;
    const bool keys_fit = keys_off + 4 * (size_t)d.C <= (size_t)kPlanSmemBytes;
    y.hist_off = (int)hist_off;
    y.keys_off = keys_fit ? (int)keys_off : -1;
    size_t smem = keys_fit ? keys_off + 4 * (size_t)d.C : keys_off;
    if (plan_bytes > smem) smem = plan_bytes;
    if (smem > bp->plan_smem) bp->plan_smem = smem;
    // extrema pass: CTAs in proportion to the (column block, row) units, eight rows per CTA at least
    const long long units = ((ncols + 1023) / 1024) * d.O;
    long long want = (units + 7) / 8;
    if (want < 1) want = 1;
    if (want > 4 * kNumSMs) want = 4 * kNumSMs;
    y.mm_blk0 = mm_blk; y.mm_blks = (int)want; mm_blk += (int)want;
    y.mm_narrow = ncols <= 512;
    y.vec = 1;
    // code pass: the same choice of form and geometry as the single-layer call
    y.packed_ok = aligned(d.codes, 4) && (d.ld_codes % 4 == 0);
    const int main_quads = (int)((ncols + 3) / 4), tail_quads = (d.S * d.R + 3) / 4;
    const int tail_warps = d.S == 0 ? 0 : (12 * tail_quads >= main_quads ? 2 : 1);
    y.tail_warps = tail_warps;
    y.srow = srow;
    if (main_quads <= 256 - 32 * tail_warps && tail_quads <= 32 * tail_warps) {
      const int side = (256 - 32 * tail_warps) / main_quads;
      long long g = (((long long)d.O + side - 1) / side + 7) / 8;
      if (g < 1) g = 1;
      if (g > 2 * kNumSMs) g = 2 * kNumSMs;
      y.cp_kind = 0; y.cp_blk0 = nb; y.cp_blks = (int)g; nb += (int)g;
    } else {
      const RowsGeometry geo = rows_geometry(d.O, row_bytes, 0);
      y.rows_per_group = (int)geo.g;
      y.n_buf = geo.n_buf;
      int g = geo.n_groups < kNumSMs / 4 ? geo.n_groups : kNumSMs / 4;   // a layer takes a quarter of the SMs at most
      if (g < 1) g = 1;
      y.cp_kind = 1; y.cp_blk0 = sb; y.cp_blks = g; sb += g;
      if (geo.rows_smem > bp->staged_smem) bp->staged_smem = geo.rows_smem;
    }
  }
  bp->mm_grid = mm_blk; bp->narrow_grid = nb; bp->staged_grid = sb;
  bp->total = off;
  return true;
}
}  // namespace
}  // namespace ocs

extern "C" size_t ocs_split_quantize_batch_workspace_bytes(const ocs_layer_desc* layers, int n_layers) {
  BatchPlan bp;
  ocs_status why;
  if (!layers || !plan_batch(layers, n_layers, 8, 1, nullptr, &bp, &why)) return 0;
  return bp.total;
}

extern "C" ocs_status ocs_split_quantize_batch(const ocs_layer_desc* layers, int n_layers, int bits, int is_signed,
                                               void* ws, size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!layers) return OCS_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return OCS_ERR_INVALID_ARG;
  if (!ws || !aligned(ws, 256)) return OCS_ERR_WORKSPACE;
  static BatchPlan bp;                 // 14 KB: kept off the stack (calls are serialised by the mutex below)
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  ocs_status why;
  if (!plan_batch(layers, n_layers, bits, is_signed, ws, &bp, &why)) return why;
  if (ws_bytes < bp.total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(batch_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPlanSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(batch_staged_code_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRowSmemBytes) != cudaSuccess)
      return OCS_ERR_CUDA;
    attr_set = true;
  }
  if (cudaMemsetAsync(ws, 0xFF, bp.colmin_bytes, stream) != cudaSuccess) return OCS_ERR_CUDA;
  if (cudaMemsetAsync(reinterpret_cast<unsigned char*>(ws) + bp.colmin_bytes, 0x00, bp.colmin_bytes, stream) != cudaSuccess)
    return OCS_ERR_CUDA;
  {
    LaunchScope ls("batch_minmax_kernel", stream);
    batch_minmax_kernel<<<bp.mm_grid, 256, 0, stream>>>(bp.t, dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  {
    LaunchScope ls("batch_plan_kernel", stream);
    batch_plan_kernel<<<n_layers, kPlanThreads, bp.plan_smem, stream>>>(bp.t, dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  if (bp.narrow_grid > 0) {
    LaunchScope ls("batch_narrow_code_kernel", stream);
    batch_narrow_code_kernel<<<bp.narrow_grid, 256, 0, stream>>>(bp.t);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  if (bp.staged_grid > 0) {
    LaunchScope ls("batch_staged_code_kernel", stream);
    batch_staged_code_kernel<<<bp.staged_grid, kRowThreads, bp.staged_smem, stream>>>(bp.t, dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  return OCS_OK;
}

// ------------------------------------------------------------------------------------------------
// ocs_act_split_quantize_static: Eq. 4 for a channel list fixed ahead of time (Section 5.3).  The
// list is turned into the plan arrays the row-staged kernel reads (every listed channel: one split,
// both copies halved), then the code pass runs as in ocs_split_quantize.
namespace ocs {
namespace {
constexpr int kStaticPlanThreads = 1024;

__global__ void __launch_bounds__(kStaticPlanThreads)
static_plan_kernel(const int32_t* __restrict__ sel, int C, int S, const uint32_t* __restrict__ colmin,
                   const uint32_t* __restrict__ colmax, const float* __restrict__ alpha_in, int32_t* idx_map,
                   int32_t* depth, unsigned long long* bits, float* qa_step_dev, int32_t* touched, int* n_touched,
                   float* mx3, int* dev_status) {
  __shared__ float s_m0[32], s_m1[32];
  const int tid = threadIdx.x;
  for (int j = tid; j < C + S; j += kStaticPlanThreads) {
    idx_map[j] = j < C ? j : 0;
    depth[j] = j < C ? 0 : 1;
    bits[j] = 0ull;
  }
  __syncthreads();
  bool bad = false;
  for (int sidx = tid; sidx < S; sidx += kStaticPlanThreads) {
    int c = sel[sidx];
    if ((unsigned)c >= (unsigned)C) { bad = true; c = 0; }
    if (atomicAdd(&depth[c], 1) != 0) bad = true;   // listed twice
    touched[sidx] = c;
    idx_map[C + sidx] = c;
  }
  if (bad) flag(dev_status, OCS_DEV_BAD_INDEX);
  __syncthreads();
  float m0 = 0.0f, m1 = 0.0f;
  if (colmax) {
    for (int c = tid; c < C; c += kStaticPlanThreads) {
      const uint32_t lo = colmin[c], hi = colmax[c];
      if (lo > hi) continue;                          // no finite sample seen in this column
      const float m = fmaxf(fabsf(ord_decode(lo)), fabsf(ord_decode(hi)));
      m0 = fmaxf(m0, m);
      m1 = fmaxf(m1, depth[c] > 0 ? __fmul_rn(m, 0.5f) : m);
    }
    for (int o = 16; o > 0; o >>= 1) {
      m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
      m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
    }
    if ((tid & 31) == 0) { s_m0[tid >> 5] = m0; s_m1[tid >> 5] = m1; }
    __syncthreads();
  }
  if (tid == 0) {
    if (colmax) {
      for (int w = 1; w < kStaticPlanThreads / 32; ++w) { m0 = fmaxf(m0, s_m0[w]); m1 = fmaxf(m1, s_m1[w]); }
    } else {
      m1 = *alpha_in;
      if (!(m1 >= 0.0f) || !is_finite(m1)) { flag(dev_status, OCS_DEV_NONFINITE); m1 = 0.0f; }
    }
    mx3[0] = m0; mx3[1] = m1; mx3[2] = 0.0f;
    *qa_step_dev = 0.0f;
    *n_touched = S;
  }
}
}  // namespace
}  // namespace ocs

extern "C" ocs_status ocs_act_split_quantize_static(const float* A, int rows, int C, int64_t ld_in, int S,
                                                    const int32_t* sel, int bits, int is_signed, const float* alpha_in,
                                                    int8_t* codes, int64_t ld_codes, int32_t* idx_map, float* scale,
                                                    void* ws, size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!A || !codes || !idx_map || !scale || S < 0 || (S > 0 && !sel)) return OCS_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return OCS_ERR_INVALID_ARG;
  if (rows <= 0 || C <= 0 || S > C) return OCS_ERR_SHAPE;
  const int ncols_out = C + S;
  if (ld_in < C || ld_codes < ncols_out) return OCS_ERR_SHAPE;
  const int srow = (ncols_out + 3) & ~3;
  const size_t row_bytes = 4 * (size_t)srow;
  if (!(ld_in % 4 == 0 && aligned(A, 16) && C % 4 == 0 && 2 * row_bytes <= kRowSmemBytes)) return OCS_ERR_UNSUPPORTED;
  const FusedWs f = carve_fused_ws(ws, C, 1, S, 1, 1);
  if (!ws || !aligned(ws, 256) || ws_bytes < f.total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const SplitWs& w = f.sp;
  if (!alpha_in) {
    // dynamic grid: channel extrema of this batch (the kernel also flags non-finite input)
    if (cudaMemsetAsync(w.colmin, 0xFF, 4 * (size_t)C, stream) != cudaSuccess) return OCS_ERR_CUDA;
    if (cudaMemsetAsync(w.colmax, 0x00, 4 * (size_t)C, stream) != cudaSuccess) return OCS_ERR_CUDA;
    const long long units = (long long)((C + 1023) / 1024) * rows;
    LaunchScope ls("col_minmax_kernel", stream);
    if (C <= 512)
      col_minmax_narrow_kernel<true><<<wave_grid(col_minmax_narrow_kernel<true>, units), 256, 0, stream>>>(
          A, rows, C, ld_in, w.colmin, w.colmax, C, idx_map, w.depth, w.bits, dev_status);
    else
      col_minmax_kernel<true><<<wave_grid(col_minmax_kernel<true>, units), 256, 0, stream>>>(
          A, rows, C, ld_in, w.colmin, w.colmax, C, idx_map, w.depth, w.bits, dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  {
    LaunchScope ls("static_plan_kernel", stream);
    static_plan_kernel<<<1, kStaticPlanThreads, 0, stream>>>(sel, C, S, alpha_in ? nullptr : w.colmin,
                                                             alpha_in ? nullptr : w.colmax, alpha_in, idx_map, w.depth,
                                                             w.bits, w.qa_step_dev, w.touched, w.n_touched, f.mx3,
                                                             dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  const RowsGeometry geo = rows_geometry(rows, row_bytes, 0);
  if ((st = rows_attr_once()) != OCS_OK) return st;
  RowsEpilogue ep{};
  ep.maxp = f.mx3 + 1;
  ep.n_buf = geo.n_buf;
  ep.L = is_signed ? (1 << (bits - 1)) - 1 : (1 << bits) - 1;
  ep.is_signed = is_signed ? 1 : 0;
  ep.scores = nullptr;
  ep.n_candidates = 1;
  return launch_rows_quant(A, rows, C, 1, ld_in, S, idx_map, w, ep, codes, ld_codes, scale, nullptr, (int)geo.g, srow,
                           geo.n_groups, geo.rows_smem, true, dev_status, stream);
}

// ------------------------------------------------------------------------------------------------
// ocs_dup_weight_columns: the weight side of activation OCS (Eq. 4): the duplicated channels'
// weight columns are plain copies, Wc[n][C + s][:] = Wc[n][idx_map[C + s]][:] (R taps per channel).
namespace ocs {
namespace {
__global__ void __launch_bounds__(256)
dup_columns_kernel(int8_t* __restrict__ Wc, int N, int C, int R, int S, long long ldw,
                   const int32_t* __restrict__ idx_map, int* dev_status) {
  const long long per_row = (long long)S * R;
  const long long total = (long long)N * per_row;
  bool bad = false;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
    const long long n = i / per_row;
    const int rem = (int)(i - n * per_row);
    const int sidx = rem / R;
    const int r = rem - sidx * R;
    int src = __ldg(idx_map + C + sidx);
    if ((unsigned)src >= (unsigned)C) { bad = true; src = 0; }
    Wc[n * ldw + (long long)(C + sidx) * R + r] = Wc[n * ldw + (long long)src * R + r];
  }
  if (bad) flag(dev_status, OCS_DEV_BAD_INDEX);
}
}  // namespace
}  // namespace ocs

extern "C" ocs_status ocs_dup_weight_columns(int8_t* W_codes, int N, int C, int R, int S, int64_t ldw,
                                             const int32_t* idx_map, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!W_codes || !idx_map || S < 0) return OCS_ERR_INVALID_ARG;
  if (N <= 0 || C <= 0 || R <= 0 || ldw < ((int64_t)C + S) * R) return OCS_ERR_SHAPE;
  if (S == 0) return OCS_OK;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const long long total = (long long)N * S * R;
  const int grid = (int)min((total + 255) / 256, (long long)kNumSMs * 8);
  LaunchScope ls("dup_columns_kernel", stream);
  dup_columns_kernel<<<grid, 256, 0, stream>>>(W_codes, N, C, R, S, ldw, idx_map, dev_status);
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// ocs_fold_duplicates: the copies of a split channel all multiply the same activation, so their
// integer codes can be summed back into the source channel (Eq. 3 read right to left):
// Wf[n][i][r] = sum over j with idx_map[j] = i of Wc[n][j][r].  The layer on Wf needs no gather and
// gives the same int32 accumulators.  Per-source lists of the appended copies are built with one
// atomic exchange per copy; integer sums do not depend on the list order.
namespace ocs {
namespace {
__global__ void __launch_bounds__(256)
fold_lists_kernel(const int32_t* __restrict__ idx_map, int C, int S, int32_t* head, int32_t* next, int* dev_status) {
  const int sidx = blockIdx.x * 256 + threadIdx.x;
  if (sidx >= S) return;
  int c = __ldg(idx_map + C + sidx);
  if ((unsigned)c >= (unsigned)C) { flag(dev_status, OCS_DEV_BAD_INDEX); c = 0; }
  next[sidx] = atomicExch(&head[c], sidx);
}

__global__ void __launch_bounds__(256)
fold_kernel(const int8_t* __restrict__ Wc, int N, int C, int R, long long ldw, const int32_t* __restrict__ head,
            const int32_t* __restrict__ next, int8_t* __restrict__ Wf, long long ld_out, int* dev_status) {
  const int cols = C * R;
  bool over = false;
  for (int n = blockIdx.y; n < N; n += gridDim.y) {
    const int8_t* src = Wc + (long long)n * ldw;
    int8_t* dst = Wf + (long long)n * ld_out;
    for (int e = blockIdx.x * 256 + threadIdx.x; e < cols; e += gridDim.x * 256) {
      const int c = e / R, r = e - c * R;
      int sum = src[e];
      for (int sidx = __ldg(head + c); sidx >= 0; sidx = __ldg(next + sidx)) sum += src[(long long)(C + sidx) * R + r];
      if (sum > 127) { sum = 127; over = true; }
      if (sum < -128) { sum = -128; over = true; }
      dst[e] = (int8_t)sum;
    }
  }
  if (over) flag(dev_status, OCS_DEV_OVERFLOW);
}
}  // namespace
}  // namespace ocs

extern "C" size_t ocs_fold_workspace_bytes(int C, int S) {
  if (C <= 0 || S < 0) return 0;
  return align_up(4 * (size_t)C, 256) + align_up(4 * (size_t)(S > 0 ? S : 1), 256);
}

extern "C" ocs_status ocs_fold_duplicates(const int8_t* W_codes, int N, int C, int R, int S, int64_t ldw,
                                          const int32_t* idx_map, int8_t* W_folded, int64_t ld_out, void* ws,
                                          size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!W_codes || !W_folded || !idx_map || S < 0) return OCS_ERR_INVALID_ARG;
  if (N <= 0 || C <= 0 || R <= 0) return OCS_ERR_SHAPE;
  if ((int64_t)C * R >= (1ll << 31) || ldw < ((int64_t)C + S) * R || ld_out < (int64_t)C * R) return OCS_ERR_SHAPE;
  if (!ws || !aligned(ws, 256) || ws_bytes < ocs_fold_workspace_bytes(C, S)) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  int32_t* head = reinterpret_cast<int32_t*>(ws);
  int32_t* next = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(ws) + align_up(4 * (size_t)C, 256));
  if (cudaMemsetAsync(head, 0xFF, 4 * (size_t)C, stream) != cudaSuccess) return OCS_ERR_CUDA;   // -1 = empty list
  if (S > 0) {
    LaunchScope ls("fold_lists_kernel", stream);
    fold_lists_kernel<<<(S + 255) / 256, 256, 0, stream>>>(idx_map, C, S, head, next, dev_status);
    if ((st = launch_status()) != OCS_OK) return st;
  }
  const int cols = C * R;
  const int gx = min((cols + 255) / 256, 64);
  const int gy = min(N, max(1, kNumSMs * 8 / gx));
  LaunchScope ls("fold_kernel", stream);
  fold_kernel<<<dim3(gx, gy), 256, 0, stream>>>(W_codes, N, C, R, ldw, head, next, W_folded, ld_out, dev_status);
  return launch_status();
}
