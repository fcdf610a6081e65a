// ocs_qlinear / ocs_qconv: the split layer of Eq. 3 on integer codes, as one tcgen05 int8 GEMM /
// implicit-GEMM convolution (Section 3.2, Section 3.5).
//
//   acc[m][n] = sum_k Aexp[m][k] * Wc[n][k]      int8/uint8 x int8 -> int32 in tensor memory
//   Y[m][n]   = fmaf((float)acc, a_scale*w_scale, bias[n])
// A convolution whose pixels TMA cannot address runs as the same GEMM over a patch matrix built first.
//
// The expanded activation operand Aexp (activations with the duplicated channels appended) is never
// written to global memory: K-blocks that hold only original channels are fetched by TMA straight
// from the unexpanded tensor, and K-blocks that hold duplicated channels (or that the TMA alignment
// rules cannot serve) are assembled in shared memory by four producer warps that read the source
// channels through idx_map and store them in the 128-byte-swizzled layout the tensor core reads.
//
// A work item = one 128 x BN output tile.  The grid is persistent: one CTA per SM, grouped in thread-block
// clusters of CL = 1, 2, 4 or 8 CTAs; a cluster walks its share of the tiles and its CTAs split the tile's
// K-blocks among themselves (CTA r takes blocks r, r + CL, ...), so that short-and-wide problems still fill the
// GPU.  The CL partial accumulators of a tile are summed through distributed shared memory: every CTA sends
// the rows another CTA owns straight into that CTA's shared memory (st.async, counted as transaction bytes on
// the owner's barrier), barriers in shared memory pace the exchange, and each CTA finishes 128 / CL rows of the
// tile (integer sums: exact in any order).
// No second launch, no global scratch, and the only waits are on CTAs the hardware co-schedules.  Warp roles:
//   warp 0      TMA producer (weights always, activations when the block is TMA-able); its ring of
//               stages runs on across tiles
//   warp 1      allocates tensor memory (two accumulators), issues tcgen05.mma, commits to barriers
//   warps 2..5  gather producers: assemble the A tiles of the K-blocks that hold duplicated channels -- or, when
//               the caller supplies a channel-major copy of the activations, warp 2 alone requests each
//               duplicated channel as one row of that copy by TMA (an MN-major operand tile)
//   warps 6..13 epilogue of tile i while the main loop of tile i+1 runs: tcgen05.ld, transposition through
//               shared memory for full-sector stores, int32 -> fp32, fmaf (optionally ReLU and max |Y|);
//               the two warps of a tensor-memory lane quadrant take alternate 16-column pieces
// The K-blocks whose A tile is assembled ("tail" blocks) come last in a CTA's K order and use three
// dedicated A buffers, so the gather warps start at kernel begin and run ahead of the TMA-fed main
// loop.
// Every mbarrier wait is bounded by a clock limit; on expiry the CTA sets OCS_DEV_TIMEOUT, lets its
// outstanding copies land, frees its tensor memory and returns.
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace ocs {
namespace {

constexpr int BM = 128;        // UMMA M
constexpr int BK = 128;        // bytes (= int8 elements) per K-block: one 128-byte swizzle span
constexpr int UMMA_K = 32;     // K of one tcgen05.mma.kind::i8
constexpr int kGemmThreads = 448;    // TMA warp, MMA warp, 4 gather warps, 8 epilogue warps
constexpr int kEpiWarps = 8;
constexpr int kEpiCols = 16;         // accumulator columns an epilogue warp moves at a time
constexpr int kGatherThreads = 128;
constexpr long long kWaitCycles = 2000000000ll;  // about one second
// A waiting thread sleeps inside mbarrier.try_wait until the phase completes or about this many nanoseconds
// pass, instead of spinning on the issue slots the epilogue warps of the same SM partition need.
constexpr uint32_t kSuspendHintNs = 2000u;
constexpr uint32_t kExchangeHintNs = 100u;   // the exchange of partial sums sits on the critical path: short naps

enum { MODE_LINEAR = 0, MODE_CONV = 1 };

struct GemmParams {
  int mode;
  int M, N, Ktot;   // Ktot = number of valid contraction indices
  int C, S, R;
  int Cp;            // contraction indices one filter tap occupies: C, or C padded to a K-block (see conv_tap_stride)
  const uint8_t* A;  // linear: [M][lda] ; conv: NHWC codes
  long long lda;
  int a_signed;
  const int32_t* idx_map;
  int a_vec16;       // 16-byte loads of A allowed (alignment)
  int tail_T;        // the tail K-blocks are fetched by TMA from the channel-major copy of A (linear layers)
  // convolution geometry
  int Nb, H, Wd, Ho, Wo, kh, kw, stride, pad;
  int bw, bh, bn;               // output-pixel box of one M tile: bw*bh*bn <= 128
  int tiles_w, tiles_h, tiles_n;
  // k-blocks
  int num_kb;
  int kb_tma_a;      // K-blocks [0, kb_tma_a) get their A tile by TMA
  int split_k;       // = cluster size: CTAs that share one output tile, each taking every split_k-th K-block
  // work items of the persistent grid: output tiles (M tile, N tile), dealt to the clusters
  int m_tiles, n_tiles, total_items;
  // epilogue
  const float* a_scale;
  const float* w_scale;
  const float* bias;
  float* Y;
  long long ldy;
  int32_t* acc_out;
  const float* residual;        // optional fp32 tensor of Y's shape and stride, added before the ReLU
  int relu;                     // max(., 0) applied to Y
  unsigned int* max_bits;       // fp32 bits of max |Y| over the whole output (optional)
  long long out_rows;           // rows of Y
  int a_box_bytes;              // bytes one TMA load of A delivers
  int* dev_status;
};

// ------------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the CTA is aborting (this wait or another one ran out of time).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kExchangeHintNs)
      : "memory");
  return ok != 0;
}
// The same bounded wait for barriers that peer CTAs of the cluster arrive on.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_cluster() { asm volatile("fence.proxy.async.shared::cluster;" ::: "memory"); }

// Thread-block cluster: rank and size, a peer CTA's view of one of our shared-memory addresses,
// stores and barrier arrivals into a peer's shared memory, cluster-wide barrier.
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_size() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t peer_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_local_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void mbar_arrive_peer(uint32_t addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at the same shared-memory offset in every CTA of the mask.
__device__ __forceinline__ void umma_commit_multicast(uint32_t bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(cta_mask) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives lane (base + t)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t v[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// (float)acc with round-to-nearest-even, without the conversion unit (which is slow on this part and sits
// on the epilogue's critical path): u = acc + 2^31 is split into two 16-bit halves, each placed by one byte
// permute into the mantissa of 1.5 * 2^23, where it is exact; subtracting the offsets gives hi = floor(acc /
// 65536) and lo exactly, and one fused multiply-add rounds the exact sum hi * 65536 + lo once -- the same
// result as cvt.rn.f32.s32 for every int32.
__device__ __forceinline__ float int_to_float_rn(int acc) {
  const uint32_t u = (uint32_t)acc ^ 0x80000000u;
  const float fh = __fsub_rn(__uint_as_float(__byte_perm(u, 0x4B400000u, 0x7632)), 12615680.0f);   // 1.5*2^23 + 2^15
  const float fl = __fsub_rn(__uint_as_float(__byte_perm(u, 0x4B400000u, 0x7610)), 12582912.0f);
  return fmaf(fh, 65536.0f, fl);
}

// Two fp32 values in one 64-bit register, and the packed arithmetic on them (each half rounds on its own,
// exactly as the scalar instruction would).
__device__ __forceinline__ unsigned long long pack_f32x2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ unsigned long long sub_f32x2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
// int_to_float_rn for two accumulators at once (the same five steps, the floating-point ones packed).
__device__ __forceinline__ unsigned long long int2_to_float2_rn(int acc0, int acc1) {
  const uint32_t u0 = (uint32_t)acc0 ^ 0x80000000u, u1 = (uint32_t)acc1 ^ 0x80000000u;
  const unsigned long long hi = pack_f32x2(__uint_as_float(__byte_perm(u0, 0x4B400000u, 0x7632)),
                                           __uint_as_float(__byte_perm(u1, 0x4B400000u, 0x7632)));
  const unsigned long long lo = pack_f32x2(__uint_as_float(__byte_perm(u0, 0x4B400000u, 0x7610)),
                                           __uint_as_float(__byte_perm(u1, 0x4B400000u, 0x7610)));
  const unsigned long long fh = sub_f32x2(hi, pack_f32x2(12615680.0f, 12615680.0f));   // 1.5*2^23 + 2^15
  const unsigned long long fl = sub_f32x2(lo, pack_f32x2(12582912.0f, 12582912.0f));
  return fma_f32x2(fh, pack_f32x2(65536.0f, 65536.0f), fl);
}

// 32 lanes x 16 consecutive 32-bit columns
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t v[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, groups of
// 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFFu);        // start address
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset: next 8-row group
  d |= (uint64_t)1 << 46;                         // descriptor version
  d |= (uint64_t)2 << 61;                         // SWIZZLE_128B
  return d;
}
__host__ __device__ constexpr uint32_t instr_desc_i8(int n, int a_signed) {
  return (2u << 4)                         // accumulator S32
         | ((uint32_t)(a_signed ? 1 : 0) << 7)   // A: uint8 / int8
         | (1u << 10)                      // B: int8
         | ((uint32_t)(n >> 3) << 17)      // N
         | ((uint32_t)(BM >> 4) << 24);    // M
}

// ------------------------------------------------------------------------------------------------
// Row r of M tile `mt` -> what it reads and where it writes.
struct RowInfo {
  long long out_row;   // linear: m ; conv: output pixel index (n*Ho+oh)*Wo+ow ; -1 = padding row
  int n, ih0, iw0;     // conv: image and top-left input coordinate of the receptive field
};

// Where row r of an M tile sits inside the tile's box of output pixels: the same for every tile, so a thread that
// keeps its row works it out once.
struct RowPos {
  int wl, hl, nl;
};
__device__ __forceinline__ RowPos row_pos(const GemmParams& p, int r) {
  RowPos rp;
  rp.wl = r; rp.hl = 0; rp.nl = 0;
  if (p.mode == MODE_LINEAR) return rp;
  const int t = r / p.bw;
  rp.wl = r - t * p.bw;
  rp.nl = t / p.bh;
  rp.hl = t - rp.nl * p.bh;
  return rp;
}

__device__ __forceinline__ RowInfo row_info_at(const GemmParams& p, int mt, const RowPos& rp) {
  RowInfo ri;
  ri.n = 0; ri.ih0 = 0; ri.iw0 = 0;
  if (p.mode == MODE_LINEAR) {
    const long long m = (long long)mt * BM + rp.wl;
    ri.out_row = m < p.M ? m : -1;
    return ri;
  }
  const int t = mt / p.tiles_w;
  const int tw = mt - t * p.tiles_w;
  const int tn = t / p.tiles_h;
  const int th = t - tn * p.tiles_h;
  const int wl = rp.wl, hl = rp.hl, nl = rp.nl;
  const int ow = tw * p.bw + wl, oh = th * p.bh + hl, n = tn * p.bn + nl;
  if (nl >= p.bn || ow >= p.Wo || oh >= p.Ho || n >= p.Nb) { ri.out_row = -1; return ri; }
  ri.out_row = ((long long)n * p.Ho + oh) * p.Wo + ow;
  ri.n = n; ri.ih0 = oh * p.stride - p.pad; ri.iw0 = ow * p.stride - p.pad;
  return ri;
}
__device__ __forceinline__ RowInfo row_info(const GemmParams& p, int mt, int r) {
  return row_info_at(p, mt, row_pos(p, r));
}

// Where contraction index k of a K-block reads from, relative to the row's base address (linear:
// the row of A; convolution: the top-left pixel of the output pixel's receptive field).
struct KSrc {
  int off;   // byte offset from the row base; negative: this k contributes zero
  int dydx;  // convolution: dy | dx << 8 of the filter tap (for the image-border test)
};

__device__ __forceinline__ int checked_src(const GemmParams& p, int j, bool* bad) {
  int c = __ldg(p.idx_map + j);
  if ((unsigned)c >= (unsigned)p.C) { *bad = true; c = 0; }
  return c;
}

__device__ __forceinline__ KSrc k_source(const GemmParams& p, int k, bool* bad) {
  KSrc e;
  e.off = -1; e.dydx = 0;
  if (k >= p.Ktot) return e;
  if (p.mode == MODE_LINEAR) {
    e.off = k < p.C ? k : checked_src(p, k, bad);
    return e;
  }
  // convolution: contraction order is [tap][c < C] then [tap][s < S]
  const int KO = p.R * p.Cp;
  int tap, c;
  if (k < KO) {
    tap = k / p.Cp; c = k - tap * p.Cp;
    if (c >= p.C) return e;   // padding between taps
  } else {
    const int kd = k - KO; tap = kd / p.S; c = checked_src(p, p.C + (kd - tap * p.S), bad);
  }
  const int dy = tap / p.kw, dx = tap - dy * p.kw;
  e.off = (dy * p.Wd + dx) * p.C + c;
  e.dydx = dy | (dx << 8);
  return e;
}

// One operand byte, loaded only when `ok` (a predicated load: no branch, and no memory transaction for an index
// that contributes zero).
__device__ __forceinline__ uint32_t ldg_u8_if(const uint8_t* addr, bool ok) {
  uint32_t v;
  // not volatile: a read-only load, free to be scheduled early and side by side with its fifteen siblings
  asm("{\n\t.reg .pred p;\n\t"
      "setp.ne.u32 p, %2, 0;\n\t"
      "mov.u32 %0, 0;\n\t"
      "@p ld.global.nc.u8 %0, [%1];\n\t}"
      : "=r"(v) : "l"(addr), "r"((uint32_t)ok));
  return v;
}

// The operand bytes of one tile row for the 16 contraction indices whose sources are tab[0..16).
// The 16 loads are independent (predicated, not branched) and in flight together; indices that contribute zero
// (K padding, a tap outside the image) issue no load.
// n = how many of the 16 indices lie below the last contraction index (the K padding comes last): groups of four
// indices beyond it are skipped altogether -- with a handful of duplicated channels most of a chunk is padding.
__device__ __forceinline__ uint4 gather_chunk(const GemmParams& p, const RowInfo& ri, const uint8_t* base,
                                              const KSrc* __restrict__ tab, int n) {
  uint32_t w[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    w[q] = 0u;
    if (4 * q < n) {
      uint32_t b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const KSrc e = tab[4 * q + i];
        bool ok = ri.out_row >= 0 && e.off >= 0;
        if (p.mode == MODE_CONV) {
          const int ih = ri.ih0 + (e.dydx & 255), iw = ri.iw0 + (e.dydx >> 8);
          ok = ok && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.Wd;
        }
        b[i] = ldg_u8_if(base + (ok ? e.off : 0), ok);
      }
      w[q] = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
    }
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// A 16-byte chunk that is one aligned run of original channels (no duplicate, one filter tap).
__device__ __forceinline__ uint4 direct_chunk(const GemmParams& p, const RowInfo& ri, int k0) {
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  if (ri.out_row < 0) return zero;
  if (p.mode == MODE_LINEAR) return __ldg(reinterpret_cast<const uint4*>(p.A + ri.out_row * p.lda + k0));
  const int tap = k0 / p.Cp, c0 = k0 - tap * p.Cp;
  const int ih = ri.ih0 + tap / p.kw, iw = ri.iw0 + tap % p.kw;
  if (c0 < p.C && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.Wd)
    return __ldg(reinterpret_cast<const uint4*>(p.A + (((long long)ri.n * p.H + ih) * p.Wd + iw) * p.C + c0));
  return zero;
}

constexpr int kTailBufs = 3;   // A tiles assembled by the gather warps (shared across the cluster)

template <int BN>
struct SmemLayout {
  static constexpr int kABytes = BM * BK;
  static constexpr int kBBytes = BN * BK;
  static constexpr int kStageBytes = kABytes + kBBytes;
  // ring depth: shallower when the tail buffers are needed
  static constexpr int kStagesNoTail = (BN == 256) ? 4 : (BN == 192 ? 4 : (BN == 128 ? 6 : 8));
  static constexpr int kStagesTail = (BN == 256) ? 3 : (BN == 192 ? 3 : (BN == 128 ? 4 : 6));
  static constexpr int kMaxStages = kStagesNoTail;
  static constexpr int kTileBytes =
      (kStagesNoTail * kStageBytes > kStagesTail * kStageBytes + kTailBufs * kABytes)
          ? kStagesNoTail * kStageBytes : kStagesTail * kStageBytes + kTailBufs * kABytes;
  static constexpr int kCtrlBytes = 1024;               // barriers, tensor-memory slot, flags
  static constexpr int kRowTableBytes = 2 * BM * 24;    // RowInfo per tile row, two tiles
  static constexpr int kSrcTableBytes = 2 * BK * 8;     // KSrc per contraction index, two gathered K-blocks
  // epilogue staging: per epilogue warp a 32 x 32 tile of 32-bit words, rows padded to 36 words (16-byte
  // aligned, conflict-free for 128-bit accesses by quarter warps), and the 32 output-row numbers
  static constexpr int kEpiRowWords = kEpiCols + 4;
  static constexpr int kEpiWarpBytes = 32 * kEpiRowWords * 4 + 128 * 4;   // + the bias of the warp's pieces of a tile
  static constexpr int kEpiBytes = kEpiWarps * kEpiWarpBytes;
  static constexpr int kDynBytes =
      kTileBytes + 1024 /*alignment slack*/ + kCtrlBytes + kRowTableBytes + kSrcTableBytes + kEpiBytes;
  static_assert(kDynBytes <= 227 * 1024, "more dynamic shared memory than a CTA can have");
  // exchange buffer of a K split: CL slots of (BN / 4) chunk columns of (128 / CL + 1) cells of 16 bytes
  static constexpr int kExchangeBytes = (BN / 4) * 16 * (BM + 8);   // CL * (128 / CL + 1) <= 136 for CL <= 8
  static_assert(kExchangeBytes <= kStagesTail * kStageBytes, "the ring must hold the partial sums of one tile");
};

// One work item of a CTA: an output tile, and this CTA's share of its K-blocks.
struct WorkItem {
  int mt, nt;
  int my_kb, n_tma, n_tail;   // K-blocks of the share: first those with a TMA-fed A tile, then the tail
};

// Item j of this CTA's cluster (tiles are dealt round-robin to the clusters of the grid; CTA `crank` of the
// cluster takes K-blocks crank, crank + CL, ... of every tile).
__device__ __forceinline__ bool work_item(const GemmParams& p, int j, uint32_t crank, uint32_t CL, WorkItem* w) {
  // total_items fits an int, and so does every index a CTA looks at before it finds the end (32-bit divisions)
  const unsigned idx = blockIdx.x + (unsigned)j * gridDim.x;
  if (idx >= (unsigned)p.total_items) return false;
  w->mt = (int)(idx / (unsigned)p.n_tiles);
  w->nt = (int)(idx - (unsigned)w->mt * (unsigned)p.n_tiles);
  const int kz = (int)crank, sk = (int)CL;
  w->my_kb = p.num_kb > kz ? (p.num_kb - kz + sk - 1) / sk : 0;
  w->n_tma = p.kb_tma_a > kz ? min(w->my_kb, (p.kb_tma_a - kz + sk - 1) / sk) : 0;
  w->n_tail = w->my_kb - w->n_tma;
  return true;
}

__device__ __forceinline__ void fence_acq_rel_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
// 16 bytes into a (peer) CTA's shared memory, asynchronously: the store counts 16 bytes toward the transaction
// count of the barrier `mbar` in the destination CTA, which is how the receiver learns that the data is there.
__device__ __forceinline__ void st_async_v4(uint32_t addr, uint4 v, uint32_t mbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(mbar) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
ocs_gemm_kernel(const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmA,
                const __grid_constant__ CUtensorMap tmAT, const GemmParams p) {
  using L = SmemLayout<BN>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* tiles = smem_dyn + (base - raw);
  unsigned char* ctrl = tiles + L::kTileBytes;
  // barriers: full[kMaxStages], empty[kMaxStages], gfull[kTailBufs], gempty[kTailBufs], acc_full[2], acc_empty[2],
  // xready, xfull, xdone (exchange of the K slices' partial tiles)
  uint64_t* bars = reinterpret_cast<uint64_t*>(ctrl);
  constexpr int kNumBars = 2 * L::kMaxStages + 2 * kTailBufs + 4 + 3;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 8 * kNumBars + 8);
  RowInfo* rows = reinterpret_cast<RowInfo*>(ctrl + L::kCtrlBytes);
  KSrc* ksrc = reinterpret_cast<KSrc*>(ctrl + L::kCtrlBytes + L::kRowTableBytes);
  unsigned char* epi_stage = ctrl + L::kCtrlBytes + L::kRowTableBytes + L::kSrcTableBytes;
  auto full_bar = [&](int s) { return smem_u32(bars + s); };
  auto empty_bar = [&](int s) { return smem_u32(bars + L::kMaxStages + s); };
  auto gfull_bar = [&](int g) { return smem_u32(bars + 2 * L::kMaxStages + g); };
  auto gempty_bar = [&](int g) { return smem_u32(bars + 2 * L::kMaxStages + kTailBufs + g); };
  auto accfull_bar = [&](int a) { return smem_u32(bars + 2 * L::kMaxStages + 2 * kTailBufs + a); };
  auto accempty_bar = [&](int a) { return smem_u32(bars + 2 * L::kMaxStages + 2 * kTailBufs + 2 + a); };
  const uint32_t xready_bar = smem_u32(bars + 2 * L::kMaxStages + 2 * kTailBufs + 4);
  const uint32_t xfull_bar = xready_bar + 8, xdone_bar = xready_bar + 16;
  const int stages = p.num_kb > p.kb_tma_a ? L::kStagesTail : L::kStagesNoTail;
  const uint32_t tail_base = base + stages * L::kStageBytes;   // kTailBufs A tiles (only with tail blocks)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // The CTAs of a cluster work on the same output tile and split its K-blocks.
  const uint32_t crank = cluster_rank(), CL = cluster_size();

  // The TMA producer is thread 0.  (Requesting the first ring of operand tiles before the set-up barriers, to
  // overlap the set-up with the first bytes' way from DRAM, was measured: the whole CTA then waits for that thread's
  // cold code, and the fc6 GEMM takes 4 us longer.)
  int prod_j = 0, prod_i = 0, prod_it = 0;   // producer position: work item, K-block inside it, ring slot counter
  bool prod_ok = true;
  WorkItem prod_w;
  int prod_w_j = -1;                         // the work item prod_w describes (-1: none yet)
  auto produce = [&]() {                     // thread 0 only: issue the K-blocks of all of this CTA's work items
    while (prod_ok) {
      if (prod_w_j != prod_j) {              // look the tile up once, not once per K-block
        if (!work_item(p, prod_j, crank, CL, &prod_w)) break;
        prod_w_j = prod_j;
      }
      const WorkItem& w = prod_w;
      if (prod_i >= w.my_kb) {
        ++prod_j; prod_i = 0;
        continue;
      }
      if (CL > 1 && prod_i == 0 && prod_j > 0) {
        // the ring doubles as the exchange buffer of the previous tile's partial sums: wait until this CTA
        // has summed them, then hand the memory back to the copy engine
        if (!mbar_wait(xdone_bar, (uint32_t)(prod_j - 1) & 1u, abort_flag)) { prod_ok = false; break; }
        fence_proxy_async_smem();
      }
      const int i = prod_i, it = prod_it;
      const int kb = (int)crank + i * (int)CL;
      const int s = it % stages;
      const uint32_t par = ((it / stages) & 1) ^ 1;
      if (!mbar_wait(empty_bar(s), par, abort_flag)) { prod_ok = false; break; }
      const uint32_t a_dst = base + s * L::kStageBytes;
      const uint32_t b_dst = a_dst + L::kABytes;
      const bool a_tma = i < w.n_tma;
      mbar_arrive_expect_tx(full_bar(s), L::kBBytes + (a_tma ? p.a_box_bytes : 0));
      tma_load_2d(b_dst, &tmB, full_bar(s), kb * BK, w.nt * BN);
      if (a_tma) {
        if (p.mode == MODE_LINEAR) {
          tma_load_2d(a_dst, &tmA, full_bar(s), kb * BK, w.mt * BM);
        } else {
          const int k0 = kb * BK;
          const int tap = k0 / p.Cp, c0 = k0 - tap * p.Cp;
          const int tw = w.mt % p.tiles_w, th = (w.mt / p.tiles_w) % p.tiles_h, tn = w.mt / (p.tiles_w * p.tiles_h);
          tma_load_4d(a_dst, &tmA, full_bar(s), c0, tw * p.bw * p.stride + tap % p.kw - p.pad,
                      th * p.bh * p.stride + tap / p.kw - p.pad, tn * p.bn);
        }
      }
      ++prod_i; ++prod_it;
    }
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int g = 0; g < kTailBufs; ++g) {
      mbar_init(gfull_bar(g), p.tail_T ? 1 : kGatherThreads / 32);   // every gather warp, or the one that issues copies
      mbar_init(gempty_bar(g), 1);                    // the MMA issuer
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accfull_bar(a), 1);    // the MMA issuer's commit
      mbar_init(accempty_bar(a), kEpiWarps);   // every epilogue warp
    }
    mbar_init(xready_bar, CL);               // every CTA of the cluster: "my ring may be written"
    mbar_init(xfull_bar, 1);                 // this CTA's own announcement of the bytes it expects; the partial rows
                                             // then arrive as asynchronous stores that count against it
    mbar_init(xdone_bar, kEpiWarps);         // this CTA's epilogue warps: "the exchange buffer has been read"
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmB);
    if (p.kb_tma_a > 0) prefetch_tmap(&tmA);
    if (p.tail_T) prefetch_tmap(&tmAT);
  }
  constexpr uint32_t kTmemCols = 2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512);   // a power of two
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);   // two accumulators: the epilogue of one tile
  tc_fence_before();                                        // overlaps the main loop of the next
  __syncthreads();
  cluster_sync_all();   // no peer touches our barriers or our ring before they are set up
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      produce();
      if (*abort_flag && prod_it > 0) {
        // give copies that are still in flight time to land before the CTA's shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(100);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_i8(BN, p.a_signed);
      const uint32_t idesc_mn = idesc | (1u << 15);   // A operand stored MN-major (a tail tile made of channel rows)
      WorkItem w;
      int total_tail = 0;   // tail tiles this CTA consumes over all its items
      for (int j = 0; work_item(p, j, crank, CL, &w); ++j) total_tail += w.n_tail;
      int it = 0, tt = 0;
      bool ok = true;
      for (int j = 0; ok && work_item(p, j, crank, CL, &w); ++j) {
        const int acc = j & 1;
        // the epilogue has drained this accumulator (two tiles ago)
        if (!mbar_wait(accempty_bar(acc), (((uint32_t)j >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int i = 0; i < w.my_kb; ++i, ++it) {
          const int s = it % stages;
          const uint32_t par = (it / stages) & 1;
          if (!mbar_wait(full_bar(s), par, abort_flag)) { ok = false; break; }
          uint32_t a_addr = base + s * L::kStageBytes;
          const uint32_t b_addr = a_addr + L::kABytes;
          const bool tail = i >= w.n_tma;   // the A tile is assembled by the gather warps
          if (tail) {
            if (!mbar_wait(gfull_bar(tt % kTailBufs), (uint32_t)(tt / kTailBufs) & 1u, abort_flag)) { ok = false; break; }
            a_addr = tail_base + (tt % kTailBufs) * L::kABytes;
          }
          tc_fence_after();
          if (tail && p.tail_T) {
            // the tile holds one 128-byte row per contraction index (MN-major): 32 indices = 4 KB per instruction
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              umma_i8(d_tmem, smem_desc_sw128(a_addr + k * UMMA_K * 128), smem_desc_sw128(b_addr + k * UMMA_K), idesc_mn,
                      (i > 0 || k > 0) ? 1u : 0u);
            }
          } else {
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              umma_i8(d_tmem, smem_desc_sw128(a_addr + k * UMMA_K), smem_desc_sw128(b_addr + k * UMMA_K), idesc,
                      (i > 0 || k > 0) ? 1u : 0u);
            }
          }
          umma_commit(empty_bar(s));  // frees the stage when these MMAs have read it
          if (tail) {
            // ... and the tail buffer, if it is filled again
            if (tt + kTailBufs < total_tail) umma_commit(gempty_bar(tt % kTailBufs));
            ++tt;
          }
        }
        if (ok) umma_commit(accfull_bar(acc));
      }
    }
  } else if (warp < 6) {
    // ---------------------------------------------------------------- gather producers
    // The four warps assemble every tail tile of this CTA: 128 rows x 8 chunks of 16 bytes, dealt so that
    // neighbouring threads work on the same rows (one pixel's channels share cache lines).  The tail buffers
    // are separate from the TMA ring, so the gather runs ahead of the TMA-fed main loop (also across tiles).
    const int gt = threadIdx.x - 64;   // 0..127
    bool bad = false;
    bool ok = true;
    int tt = 0;          // tail tiles assembled so far
    if (p.tail_T) {
      // Linear layer with a channel-major copy of the activations: contraction index k of a tail block is channel
      // idx_map[k], and that channel's values for the tile's 128 rows are 128 contiguous bytes of the copy.  One
      // warp asks the copy engine for them, one row per index; the tile is MN-major (row k = index k).  No thread
      // touches an activation byte.
      if (warp == 2) {
        int buf_kb[kTailBufs];
        for (int g = 0; g < kTailBufs; ++g) buf_kb[g] = -1;
        WorkItem w;
        for (int j = 0; ok && work_item(p, j, crank, CL, &w); ++j) {
          for (int t = 0; t < w.n_tail; ++t, ++tt) {
            const int kb = (int)crank + (w.n_tma + t) * (int)CL;
            const int g = tt % kTailBufs;
            if (tt >= kTailBufs && !mbar_wait(gempty_bar(g), (uint32_t)(tt / kTailBufs - 1) & 1u, abort_flag)) {
              ok = false;
              break;
            }
            const int n_valid = min(BK, p.Ktot - kb * BK);
            const uint32_t tile_local = tail_base + g * L::kABytes;
            if (n_valid < BK && buf_kb[g] != kb) {   // rows past the last contraction index: zero
              for (int r = n_valid + lane; r < BK; r += 32)
#pragma unroll
                for (int c = 0; c < 8; ++c) st_local_v4(tile_local + r * 128 + c * 16, make_uint4(0u, 0u, 0u, 0u));
            }
            buf_kb[g] = kb;
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive_expect_tx(gfull_bar(g), (uint32_t)n_valid * 128u);
            __syncwarp();
            for (int k = lane; k < n_valid; k += 32) {
              const int kk = kb * BK + k;
              const int ch = kk < p.C ? kk : checked_src(p, kk, &bad);
              tma_load_2d(tile_local + k * 128, &tmAT, gfull_bar(g), w.mt * BM, ch);
            }
          }
        }
        if (*abort_flag && tt > 0)
          for (int i = 0; i < 2000; ++i) __nanosleep(100);   // copies still in flight land before the CTA leaves
      }
      if (bad) flag(p.dev_status, OCS_DEV_BAD_INDEX);
      ok = false;   // nothing left for the byte gather below
    }
    const RowPos gather_pos = row_pos(p, gt);   // this thread's row of every tile's row table
    int n_tiles_done = 0;
    int table_kb[2] = {-1, -1};   // which K-block each of the two source tables describes
    int buf_kb[kTailBufs];        // which K-block each tail buffer held last
    for (int g = 0; g < kTailBufs; ++g) buf_kb[g] = -1;
    WorkItem w;
    for (int j = 0; ok && work_item(p, j, crank, CL, &w); ++j) {
      if (w.n_tail == 0) continue;
      // row table of this tile (two tables alternate, so the previous tile's may still be in use)
      RowInfo* trow = rows + (n_tiles_done & 1) * BM;
      ++n_tiles_done;
      trow[gt] = row_info_at(p, w.mt, gather_pos);
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int t = 0; t < w.n_tail; ++t, ++tt) {
        const int kb = (int)crank + (w.n_tma + t) * (int)CL;
        const int g = tt % kTailBufs;
        if (tt >= kTailBufs && !mbar_wait(gempty_bar(g), (uint32_t)(tt / kTailBufs - 1) & 1u, abort_flag)) {
          ok = false;
          break;
        }
        // Chunks of 16 original channels inside one tap move as one 16-byte load; chunks past the
        // last contraction index are zero; the rest goes through the block's source table, which
        // is kept while the same K-block recurs (every tile of a layer has the same tail blocks).
        const int direct_chunks = p.a_vec16 ? min(8, max(0, (p.R * p.Cp - kb * BK) >> 4)) : 0;
        const int valid_chunks = min(8, (p.Ktot - kb * BK + 15) >> 4);
        const KSrc* tab = ksrc + (t & 1) * BK;
        if (direct_chunks < valid_chunks && table_kb[t & 1] != kb) {  // uniform over the gather threads
          asm volatile("bar.sync 1, 128;" ::: "memory");  // nobody still reads the table being replaced
          ksrc[(t & 1) * BK + gt] = k_source(p, kb * BK + gt, &bad);
          asm volatile("bar.sync 1, 128;" ::: "memory");
          table_kb[t & 1] = kb;
        }
        const uint32_t tile_local = tail_base + g * L::kABytes;
        // (row, chunk) pairs with data, dealt evenly over the threads
        const int n_valid = BM * valid_chunks;
#pragma unroll 2
        for (int it = gt; it < n_valid; it += kGatherThreads) {
          const int r = it / valid_chunks, c = it - r * valid_chunks;
          const RowInfo ri = trow[r];
          uint4 v;
          if (ri.out_row < 0) {
            v = make_uint4(0u, 0u, 0u, 0u);   // padding row
          } else if (c < direct_chunks) {
            v = direct_chunk(p, ri, kb * BK + c * 16);
          } else {
            const uint8_t* rbase;
            if (p.mode == MODE_LINEAR) rbase = p.A + ri.out_row * p.lda;
            else rbase = p.A + (((long long)ri.n * p.H + ri.ih0) * p.Wd + ri.iw0) * p.C;
            v = gather_chunk(p, ri, rbase, tab + c * 16, p.Ktot - (kb * BK + c * 16));
          }
          st_local_v4(tile_local + r * 128 + ((c ^ (r & 7)) << 4), v);
        }
        // the K padding: zero, unless this buffer's last occupant was the same K-block (every tile of a layer
        // has the same tail blocks, so the chunks that hold data are overwritten and the padding stays zero)
        const int zero_chunks = 8 - valid_chunks;
        if (buf_kb[g] != kb) {
          for (int it = gt; it < BM * zero_chunks; it += kGatherThreads) {
            const int r = it / zero_chunks, c = valid_chunks + (it - r * zero_chunks);
            st_local_v4(tile_local + r * 128 + ((c ^ (r & 7)) << 4), make_uint4(0u, 0u, 0u, 0u));
          }
          buf_kb[g] = kb;
        }
        // make the generic-proxy stores visible to the tensor cores that read them
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(gfull_bar(g));
      }
    }
    if (bad) flag(p.dev_status, OCS_DEV_BAD_INDEX);
  } else {
    // ---------------------------------------------------------------- epilogue (tcgen05.ld -> global)
    // warp w may read tensor-memory lanes 32*(w%4) .. +31
    const int q = warp & 3;
    const float sc = __fmul_rn(__ldg(p.a_scale), __ldg(p.w_scale));
    const bool direct = CL == 1;
    const RowPos my_pos = row_pos(p, q * 32 + lane);
    WorkItem w;
    bool ok = true;
    for (int j = 0; ok && work_item(p, j, crank, CL, &w); ++j) {
      const int acc = j & 1;
      const RowInfo ri = row_info_at(p, w.mt, my_pos);
      const int nt = w.nt;
      const int ew = warp - 6, half = ew >> 2;
      if (p.residual && direct && ri.out_row >= 0) {
        // the shortcut tensor's part of this tile is asked into L2 while the main loop still runs
        const float* rrow = p.residual + ri.out_row * p.ldy + (long long)nt * BN;
        const int n_left = p.N - nt * BN;
        for (int c = (warp >= 10 ? 32 : 0); c < BN && c < n_left; c += 64)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(rrow + c));
      }
      // The bias of this warp's pieces of the tile (piece k = columns half*16 + 32k .. +15): lane l asks for four
      // values of piece l/4 now, before the wait for the accumulator, and parks them in shared memory afterwards, so
      // that the pieces read them from there instead of waiting for global memory once each.
      float4 bias_mine = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      if (direct && p.bias) {
        const int col = half * kEpiCols + 2 * kEpiCols * (lane >> 2) + (lane & 3) * 4;   // inside the tile
        const int n = nt * BN + col;
        if (col < BN) {
          if (n + 3 < p.N && ((reinterpret_cast<uintptr_t>(p.bias) & 15) == 0)) {
            bias_mine = __ldg(reinterpret_cast<const float4*>(p.bias + n));
          } else {
            if (n < p.N) bias_mine.x = __ldg(p.bias + n);
            if (n + 1 < p.N) bias_mine.y = __ldg(p.bias + n + 1);
            if (n + 2 < p.N) bias_mine.z = __ldg(p.bias + n + 2);
            if (n + 3 < p.N) bias_mine.w = __ldg(p.bias + n + 3);
          }
        }
      }
      // K split: a thread of the summing step below keeps one 4-column group for all the rows it finishes (256
      // threads step over the row-major quads of the tile's part in strides that are multiples of a row), so its
      // bias is fetched here, while the main loop runs, instead of from a cold cache at the end of the tile
      constexpr bool kBiasOnce = 256 % (BN / 4) == 0;
      float4 bias_split = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      if (!direct && kBiasOnce && p.bias && (reinterpret_cast<uintptr_t>(p.bias) & 15) == 0 && (nt + 1) * BN <= p.N)
        bias_split = __ldg(reinterpret_cast<const float4*>(p.bias + nt * BN + ((threadIdx.x - 6 * 32) % (BN / 4)) * 4));
      if (!mbar_wait(accfull_bar(acc), ((uint32_t)j >> 1) & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      if (!direct) {
        // ------------------------------------------------------------ K split over the cluster: exchange and sum
        // CTA r of the cluster finishes rows [r * RP, (r + 1) * RP) of the tile.  The exchange buffer is the TMA
        // ring of the owning CTA (idle now: the producer does not start the next tile before the sum is done):
        // slot s holds sender s's partial sums of the owner's rows, [RP][BN] int32.
        const int RP = BM / (int)CL;
        const uint32_t xparity = (uint32_t)j & 1u;
        // (1) this CTA's tensor cores are done with its ring: it announces the bytes it is about to receive (the
        // rows it owns, from every CTA of the cluster including itself) and tells every CTA that it may be written
        const uint32_t cell_stride = (uint32_t)(RP + 1) * 16u;                 // bytes from one chunk to the next
        const uint32_t slot_bytes = (uint32_t)(BN / 4) * cell_stride;
        if (ew == 0 && lane == 0) {
          mbar_arrive_expect_tx(xfull_bar, CL * (uint32_t)(RP * BN) * 4u);
          for (uint32_t dst = 0; dst < CL; ++dst) mbar_arrive_peer(peer_addr(xready_bar, dst));
        }
        // (2) ... and this CTA writes into the others' once they have said the same
        if (!mbar_wait_cluster(xready_bar, xparity, abort_flag)) { ok = false; break; }
        // (3) a lane holds one row of the accumulator, 32 columns at a time.  The exchange buffer is laid out in
        // 16-byte cells [sender][4-column chunk][row of the owner] (+1 cell of padding per chunk): the lanes of a
        // warp, which hold consecutive rows, store consecutive cells, and the owner later reads consecutive chunks
        // of one row without bank conflicts.  The stores are asynchronous and count against the owner's barrier.
        {
          const int m = q * 32 + lane;
          const uint32_t owner = (uint32_t)(m / RP);
          const uint32_t cell0 = base + crank * slot_bytes + (uint32_t)(m - (int)owner * RP) * 16u;
          const uint32_t dst_cell0 = peer_addr(cell0, owner);
          const uint32_t dst_bar = peer_addr(xfull_bar, owner);
          for (int c0 = half * 32; c0 < BN; c0 += 64) {
            uint32_t v[32];
            __syncwarp();
            tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + c0), v);
#pragma unroll
            for (int jj = 0; jj < 32; jj += 4)
              st_async_v4(dst_cell0 + (uint32_t)((c0 + jj) >> 2) * cell_stride, make_uint4(v[jj], v[jj + 1], v[jj + 2], v[jj + 3]),
                          dst_bar);
          }
        }
        // the accumulator has been read out: hand it back to the MMA issuer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(accempty_bar(acc));
        // (4) all partial sums of this CTA's rows are in place
        if (!mbar_wait_cluster(xfull_bar, xparity, abort_flag)) { ok = false; break; }
        // (5) sum the CL slots and finish the rows: a thread takes four consecutive columns
        {
          const int et = threadIdx.x - 6 * 32;                    // 0..255
          const int n_lim = min(BN, p.N - nt * BN);
          const bool vec = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.Y) & 15) == 0) && (p.ldy % 4 == 0) &&
                           (!p.acc_out || (reinterpret_cast<uintptr_t>(p.acc_out) & 15) == 0) &&
                           (!p.residual || (reinterpret_cast<uintptr_t>(p.residual) & 15) == 0);
          // This code runs once per tile and its instructions come straight from L2: on a 40 us kernel every
          // instruction of it costs about as much as 16 cycles, so the common case (a whole tile of a linear
          // layer, aligned output, no shortcut tensor, no copy of the accumulators) has its own short loop.
          constexpr int kQuads = BN / 4;                          // 4-column groups per tile row
          const int total = RP * kQuads;
          const unsigned char* ring = tiles;                      // the exchange buffer: this CTA's ring
          float fmx = 0.0f;
          const bool lean = vec && p.mode == MODE_LINEAR && n_lim == BN && !p.residual && !p.acc_out &&
                            (!p.bias || (reinterpret_cast<uintptr_t>(p.bias) & 15) == 0) &&
                            (long long)(w.mt + 1) * BM <= p.M;
          if (lean) {
            const float* bias_n = p.bias ? p.bias + nt * BN : nullptr;
            float* ybase = p.Y + ((long long)w.mt * BM + (long long)crank * RP) * p.ldy + (long long)nt * BN;
            for (int g = et; g < total; g += 256) {
              const int rl = g / kQuads, c = (g - rl * kQuads) * 4;
              const unsigned char* src = ring + (uint32_t)(c >> 2) * cell_stride + (uint32_t)rl * 16u;
              int4 a = *reinterpret_cast<const int4*>(src);
              for (uint32_t sl = 1; sl < CL; ++sl) {
                const int4 v = *reinterpret_cast<const int4*>(src + sl * slot_bytes);
                a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
              }
              float4 b4 = bias_split;   // zero without a bias
              if (!kBiasOnce && bias_n) b4 = __ldg(reinterpret_cast<const float4*>(bias_n + c));
              // cvt.rn.f32.s32: the same value as the conversion of the direct epilogue, in one instruction
              float4 f = make_float4(fmaf(__int2float_rn(a.x), sc, b4.x), fmaf(__int2float_rn(a.y), sc, b4.y),
                                     fmaf(__int2float_rn(a.z), sc, b4.z), fmaf(__int2float_rn(a.w), sc, b4.w));
              if (p.relu) { f.x = fmaxf(f.x, 0.0f); f.y = fmaxf(f.y, 0.0f); f.z = fmaxf(f.z, 0.0f); f.w = fmaxf(f.w, 0.0f); }
              fmx = fmaxf(fmx, fmaxf(fmaxf(fabsf(f.x), fabsf(f.y)), fmaxf(fabsf(f.z), fabsf(f.w))));
              *reinterpret_cast<float4*>(ybase + (long long)rl * p.ldy + c) = f;
            }
          } else {
            for (int g = et; g < total; g += 256) {
              const int rl = g / kQuads, cc = g - rl * kQuads, c = cc * 4;
              if (c >= n_lim) continue;
              const long long orow = row_info(p, w.mt, (int)crank * RP + rl).out_row;
              if (orow < 0) continue;
              const unsigned char* src = ring + (uint32_t)cc * cell_stride + (uint32_t)rl * 16u;
              int4 a = *reinterpret_cast<const int4*>(src);
              for (uint32_t sl = 1; sl < CL; ++sl) {
                const int4 v = *reinterpret_cast<const int4*>(src + sl * slot_bytes);
                a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
              }
              const int n = nt * BN + c;
              const int av[4] = {a.x, a.y, a.z, a.w};
              float f[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const bool in = c + e < n_lim;
                f[e] = fmaf(__int2float_rn(av[e]), sc, (p.bias && in) ? __ldg(p.bias + n + e) : 0.0f);
                if (p.residual && in) f[e] = __fadd_rn(f[e], p.residual[orow * p.ldy + n + e]);
                if (p.relu) f[e] = f[e] > 0.0f ? f[e] : 0.0f;
                if (in) fmx = fmaxf(fmx, fabsf(f[e]));
              }
              float* y = p.Y + orow * p.ldy + n;
              if (vec) {
                *reinterpret_cast<float4*>(y) = make_float4(f[0], f[1], f[2], f[3]);
                if (p.acc_out) *reinterpret_cast<int4*>(p.acc_out + orow * p.ldy + n) = a;
              } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  if (c + e < n_lim) {
                    y[e] = f[e];
                    if (p.acc_out) p.acc_out[orow * p.ldy + n + e] = av[e];
                  }
                }
              }
            }
          }
          if (p.max_bits) {
            for (int o = 16; o > 0; o >>= 1) fmx = fmaxf(fmx, __shfl_xor_sync(0xffffffffu, fmx, o));
            if (lane == 0 && fmx > 0.0f) atomicMax(p.max_bits, __float_as_uint(fmx));
          }
        }
        // (6) the ring may be refilled
        __syncwarp();
        if (lane == 0) mbar_arrive(xdone_bar);
        continue;
      }
      // ------------------------------------------------------------ one CTA per tile: straight to the output
      // Each lane holds one row of a 32 x 16 piece of the accumulator; written out that way a store
      // instruction would touch 32 rows with 16 bytes each.  The piece goes through shared memory instead, so
      // that four neighbouring lanes write 64 contiguous bytes of one row (lane -> row i*8 + (qd&1)*4 + qd/2
      // with qd = lane/4, words (lane%4)*4 .. +3; the row order keeps the shared-memory reads conflict-free).
      // The two epilogue warps that share a tensor-memory lane quadrant take alternate pieces.
      uint32_t* st_words = reinterpret_cast<uint32_t*>(epi_stage + (size_t)ew * L::kEpiWarpBytes);
      float* st_bias = reinterpret_cast<float*>(st_words + 32 * L::kEpiRowWords);   // [piece][16]
      __syncwarp();   // the previous tile's pieces have read their bias
      *reinterpret_cast<float4*>(st_bias + lane * 4) = bias_mine;   // read after the piece loop's first __syncwarp
      const int qd = lane >> 2, sub = (qd & 1) * 4 + (qd >> 1), cq = (lane & 3) * 4;
      // the four rows this lane writes, the same for every piece of the tile
      long long orow[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) orow[i] = __shfl_sync(0xffffffffu, ri.out_row, i * 8 + sub);
      // ... and where their part of the tile starts in Y (for the common case below)
      float* yrow[4];
      bool rok[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        rok[i] = orow[i] >= 0;
        yrow[i] = p.Y + (rok[i] ? orow[i] : 0) * p.ldy + (long long)nt * BN + cq;
      }
      uint32_t* dst0 = reinterpret_cast<uint32_t*>(p.Y);
      const long long ldd = p.ldy;
      const bool base_vec = ((reinterpret_cast<uintptr_t>(dst0) & 15) == 0) && (ldd % 4 == 0);
      const bool acc_vec = p.acc_out && ((reinterpret_cast<uintptr_t>(p.acc_out) & 15) == 0) && (p.ldy % 4 == 0);
      // the shortcut tensor is read with 128-bit loads only when it is itself 16-byte aligned (a view that
      // starts a few floats into a buffer takes the scalar loads)
      const bool res_vec = p.residual && ((reinterpret_cast<uintptr_t>(p.residual) & 15) == 0) && (p.ldy % 4 == 0);
      float tile_max = 0.0f;
      const bool want_max = p.max_bits != nullptr;
      // a warp whose 32 rows are all padding (a short M tile) has nothing to write
      const bool warp_has_rows = __any_sync(0xffffffffu, ri.out_row >= 0);
      for (int c0 = half * kEpiCols; warp_has_rows && c0 < BN; c0 += 2 * kEpiCols) {
        const int n0 = nt * BN + c0;
        if (n0 >= p.N) break;  // warp-uniform
        const bool full = n0 + kEpiCols <= p.N;   // warp-uniform
        // the shortcut values of the piece (common case below): asked for first, so that their way from L2 -- where
        // the tile's part of the shortcut tensor was prefetched -- overlaps the accumulator's way through shared memory
        float4 r4[4];
        if (p.residual && full && base_vec && res_vec && !p.acc_out) {
#pragma unroll
          for (int i = 0; i < 4; ++i)
            r4[i] = rok[i] ? __ldcs(reinterpret_cast<const float4*>(p.residual + (yrow[i] - p.Y) + c0))
                           : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
        uint32_t v[kEpiCols];
        __syncwarp();
        // this lane's four columns of every row it writes: their bias (zero without one, and past column N)
        const float4 bq = *reinterpret_cast<const float4*>(st_bias + (c0 >> 5) * kEpiCols + cq);
        const float b4[4] = {bq.x, bq.y, bq.z, bq.w};
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + c0), v);
        // raw accumulators -> shared memory, one row per lane
        uint32_t* mine = st_words + lane * L::kEpiRowWords;
#pragma unroll
        for (int jj = 0; jj < kEpiCols; jj += 4)
          *reinterpret_cast<uint4*>(mine + jj) = make_uint4(v[jj], v[jj + 1], v[jj + 2], v[jj + 3]);
        __syncwarp();
        const bool vec0 = full && base_vec, vec1 = full && acc_vec;
        uint4 a[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          a[i] = *reinterpret_cast<const uint4*>(st_words + (i * 8 + sub) * L::kEpiRowWords + cq);
        if (vec0 && !p.acc_out && (!p.residual || res_vec)) {
          // the common case, without per-element tests: whole piece inside N, 16-byte aligned output (and
          // shortcut tensor), scale, bias, shortcut, ReLU and the maximum; the floating-point steps work on pairs
          const unsigned long long sc2 = pack_f32x2(sc, sc);
          const unsigned long long b01 = pack_f32x2(b4[0], b4[1]), b23 = pack_f32x2(b4[2], b4[3]);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float f0, f1, f2, f3;
            unpack_f32x2(fma_f32x2(int2_to_float2_rn((int)a[i].x, (int)a[i].y), sc2, b01), f0, f1);
            unpack_f32x2(fma_f32x2(int2_to_float2_rn((int)a[i].z, (int)a[i].w), sc2, b23), f2, f3);
            if (p.residual) {   // one more rounded addition per output
              f0 = __fadd_rn(f0, r4[i].x); f1 = __fadd_rn(f1, r4[i].y); f2 = __fadd_rn(f2, r4[i].z); f3 = __fadd_rn(f3, r4[i].w);
            }
            if (p.relu) {
              f0 = f0 > 0.0f ? f0 : 0.0f; f1 = f1 > 0.0f ? f1 : 0.0f;
              f2 = f2 > 0.0f ? f2 : 0.0f; f3 = f3 > 0.0f ? f3 : 0.0f;
            }
            if (rok[i]) {
              if (want_max) tile_max = fmaxf(tile_max, fmaxf(fmaxf(fabsf(f0), fabsf(f1)), fmaxf(fabsf(f2), fabsf(f3))));
              *reinterpret_cast<float4*>(yrow[i] + c0) = make_float4(f0, f1, f2, f3);
            }
          }
          continue;
        }
        uint4 o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float f0 = fmaf(int_to_float_rn((int)a[i].x), sc, b4[0]), f1 = fmaf(int_to_float_rn((int)a[i].y), sc, b4[1]);
          float f2 = fmaf(int_to_float_rn((int)a[i].z), sc, b4[2]), f3 = fmaf(int_to_float_rn((int)a[i].w), sc, b4[3]);
          if (p.residual && orow[i] >= 0) {   // the block's shortcut: one more rounded addition per output
            const float* rr = p.residual + orow[i] * p.ldy + n0 + cq;
            if (full && res_vec) {
              const float4 r4 = __ldcs(reinterpret_cast<const float4*>(rr));
              f0 = __fadd_rn(f0, r4.x); f1 = __fadd_rn(f1, r4.y); f2 = __fadd_rn(f2, r4.z); f3 = __fadd_rn(f3, r4.w);
            } else {
              if (n0 + cq + 0 < p.N) f0 = __fadd_rn(f0, rr[0]);
              if (n0 + cq + 1 < p.N) f1 = __fadd_rn(f1, rr[1]);
              if (n0 + cq + 2 < p.N) f2 = __fadd_rn(f2, rr[2]);
              if (n0 + cq + 3 < p.N) f3 = __fadd_rn(f3, rr[3]);
            }
          }
          if (p.relu) {
            f0 = f0 > 0.0f ? f0 : 0.0f; f1 = f1 > 0.0f ? f1 : 0.0f;
            f2 = f2 > 0.0f ? f2 : 0.0f; f3 = f3 > 0.0f ? f3 : 0.0f;
          }
          if (want_max) {   // padding rows and columns past N are not part of the output
            float rm;
            if (full) {
              rm = fmaxf(fmaxf(fabsf(f0), fabsf(f1)), fmaxf(fabsf(f2), fabsf(f3)));
            } else {
              rm = n0 + cq + 0 < p.N ? fabsf(f0) : 0.0f;
              if (n0 + cq + 1 < p.N) rm = fmaxf(rm, fabsf(f1));
              if (n0 + cq + 2 < p.N) rm = fmaxf(rm, fabsf(f2));
              if (n0 + cq + 3 < p.N) rm = fmaxf(rm, fabsf(f3));
            }
            tile_max = fmaxf(tile_max, orow[i] >= 0 ? rm : 0.0f);
          }
          o[i] = make_uint4(__float_as_uint(f0), __float_as_uint(f1), __float_as_uint(f2), __float_as_uint(f3));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (orow[i] < 0) continue;
          uint32_t* d = dst0 + orow[i] * ldd + n0 + cq;
          if (vec0) {
            *reinterpret_cast<uint4*>(d) = o[i];
          } else {
            if (n0 + cq + 0 < p.N) d[0] = o[i].x;
            if (n0 + cq + 1 < p.N) d[1] = o[i].y;
            if (n0 + cq + 2 < p.N) d[2] = o[i].z;
            if (n0 + cq + 3 < p.N) d[3] = o[i].w;
          }
        }
        if (p.acc_out) {
          // the caller's copy of the accumulators
          uint32_t* rbase = reinterpret_cast<uint32_t*>(p.acc_out);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (orow[i] < 0) continue;
            uint32_t* d = rbase + orow[i] * p.ldy + n0 + cq;
            if (vec1) {
              __stcg(reinterpret_cast<uint4*>(d), a[i]);
            } else {
              if (n0 + cq + 0 < p.N) d[0] = a[i].x;
              if (n0 + cq + 1 < p.N) d[1] = a[i].y;
              if (n0 + cq + 2 < p.N) d[2] = a[i].z;
              if (n0 + cq + 3 < p.N) d[3] = a[i].w;
            }
          }
        }
      }
      if (want_max) {
        for (int o = 16; o > 0; o >>= 1) tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, o));
        if (lane == 0 && tile_max > 0.0f) atomicMax(p.max_bits, __float_as_uint(tile_max));
      }
      // the accumulator has been read out: hand it back to the MMA issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(accempty_bar(acc));
    }
    tc_fence_before();
  }

  __syncthreads();
  cluster_sync_all();   // no CTA leaves while a peer may still store into it or arrive on its barriers
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag) flag(p.dev_status, OCS_DEV_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// elem_strides (nullable): traversal stride per dimension; a box extent of N * stride then delivers N elements
bool encode_u8(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
               const cuuint32_t* box, const cuuint32_t* elem_strides = nullptr) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  if (elem_strides)
    for (int i = 0; i < rank; ++i) estr[i] = elem_strides[i];
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct GemmPlan {
  int BN;
  int split_k;   // = cluster size: CTAs that share an output tile and split its K-blocks
  int m_tiles, n_tiles;
};

// CTAs that can be resident at once for cluster sizes 1, 2, 4, 8 with one CTA per SM (B200: 148 SMs;
// a cluster must fit inside one GPC, so larger clusters leave SMs unused).
constexpr int kClusterSizes[4] = {1, 2, 4, 8};
constexpr int kClusterCapacity[4] = {148, 148, 132, 120};

// Self-test override (ocs_selftest_force_gemm_plan): tile width and K split taken as given where they are
// valid for the problem.
int g_force_bn = 0, g_force_sk = 0;

// Tile width and K split by a small time model (microseconds), fitted to measurements on this part: an SM takes
// in about 105 GB/s of operand tiles, all SMs together about 9.5 TB/s from L2 (the activation tile of a K-block is
// re-read from L2 by every N tile), DRAM delivers about 6.3 TB/s, a 128 x 256 x 128 block of int8 MMAs takes about
// 0.27 us, the epilogue writes a tile at about 22 GB/s per SM (it overlaps the next tile's main loop, so a tile
// costs the longer of the two), and every tile costs about 1.5 us of hand-offs.  A K split adds the exchange of
// the partial tiles; K is split only so far that all clusters are resident at once.  n_tail = K-blocks whose A
// tile is assembled by threads or fetched as channel rows, tail_k = contraction indices in them.
GemmPlan choose_plan(int m_tiles, int N, int num_kb, int n_tail, int tail_k, bool conv, bool tail_by_tma) {
  if (g_force_bn) {
    const int BN = g_force_bn;
    const int n_tiles = (N + BN - 1) / BN;
    int ci = 0;
    while (ci < 3 && kClusterSizes[ci + 1] <= g_force_sk) ++ci;
    while (ci > 0 && ((long long)m_tiles * n_tiles * kClusterSizes[ci] > kClusterCapacity[ci] || kClusterSizes[ci] > num_kb)) --ci;
    return GemmPlan{BN, kClusterSizes[ci], m_tiles, n_tiles};
  }
  GemmPlan best{64, 1, m_tiles, (N + 63) / 64};
  double best_cost = 1e300;
  const int bns[4] = {256, 192, 128, 64};
  const double kSmIngest = 105e3, kL2Total = 9.5e6, kDram = 6.3e6, kEpilogue = 22e3;   // bytes per microsecond
  const double gather_us = tail_by_tma ? 0.0 : (conv ? 4.0 : 16.0);  // per assembled K-block full of data
  const double K = (double)num_kb * BK, Mrows = (double)m_tiles * BM;
  const double dram_us = ((double)N * K + Mrows * K + 4.0 * Mrows * N) / kDram;
  for (int bi = 0; bi < 4; ++bi) {
    const int BN = bns[bi];
    if (BN > 64 && N <= BN / 2) continue;  // tile mostly empty
    const int n_tiles = (N + BN - 1) / BN;
    const long long tiles = (long long)m_tiles * n_tiles;
    const double block_bytes = (double)(BM + BN) * BK;
    double block_us = block_bytes / kSmIngest;                       // one K-block: operand intake or the MMAs
    if (0.27 * BN / 256.0 > block_us) block_us = 0.27 * BN / 256.0;
    const double epi_us = (double)BM * ((double)N / n_tiles) * 4.0 / kEpilogue;
    for (int ci = 0; ci < 4; ++ci) {
      const int sk = kClusterSizes[ci];
      if (sk > 1 && (tiles * sk > kClusterCapacity[ci] || num_kb < 4 * sk)) continue;   // one resident wave, >= 4 blocks each
      const long long waves = (tiles * sk + kClusterCapacity[ci] - 1) / kClusterCapacity[ci];
      const int cta_blocks = (num_kb + sk - 1) / sk;
      const int tail_blocks = (n_tail + sk - 1) / sk;
      // the most loaded CTA assembles tail_blocks K-blocks per tile, of which at most tail_k indices hold data
      const int cta_k = tail_k < tail_blocks * BK ? tail_k : tail_blocks * BK;
      const double gather = tail_blocks > 0 ? 0.5 + (cta_k / 128.0) * gather_us : 0.0;
      double tile_us = cta_blocks * block_us;
      if (sk == 1 && epi_us > tile_us) tile_us = epi_us;
      if (gather > tile_us) tile_us = gather;
      double body = (double)waves * (tile_us + 1.5);
      const double total_bytes = (double)tiles * num_kb * block_bytes;
      if (total_bytes / kL2Total > body) body = total_bytes / kL2Total;
      if (dram_us > body) body = dram_us;
      double cost = 5.0 + body + (sk == 1 ? epi_us : 3.0 + 6.0 * BN / 256.0);   // start-up; last epilogue or exchange
      cost *= 1.0 + 0.002 * ci + 0.001 * bi;                             // ties: fewer slices, wider tile
      if (cost < best_cost) {
        best_cost = cost;
        best = GemmPlan{BN, sk, m_tiles, n_tiles};
      }
    }
  }
  return best;
}

// The K split needs no global scratch (kept for the workspace queries' layout).
size_t splitk_ws_bound(long long, int, long long) { return 0; }

template <int BN>
ocs_status launch_gemm(const CUtensorMap& tmB, const CUtensorMap& tmA, const CUtensorMap& tmAT, const GemmParams& p,
                       const GemmPlan& plan, cudaStream_t stream) {
  using L = SmemLayout<BN>;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(ocs_gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynBytes) != cudaSuccess)
      return OCS_ERR_CUDA;
    attr_set = true;
  }
  // persistent grid: as many clusters as fit on the device at once (or fewer, if there is less work)
  int ci = 0;
  while (ci < 3 && kClusterSizes[ci] != plan.split_k) ++ci;
  const long long slots = kClusterCapacity[ci] / plan.split_k;
  const long long n_clusters = p.total_items < slots ? p.total_items : slots;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)n_clusters, plan.split_k, 1);
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = L::kDynBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = plan.split_k; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  LaunchScope ls(p.mode == MODE_CONV ? "ocs_gemm_kernel(conv)" : "ocs_gemm_kernel(linear)", stream);
  if (cudaLaunchKernelEx(&cfg, ocs_gemm_kernel<BN>, tmB, tmA, tmAT, p) != cudaSuccess) return OCS_ERR_CUDA;
  return launch_status();
}

ocs_status run_gemm(GemmParams& p, const int8_t* W_codes, long long ldw, long long out_rows, int m_tiles, bool tma_a_ok,
                    const CUtensorMap* tmA_in, void* ws, size_t ws_bytes, cudaStream_t stream,
                    const CUtensorMap* tmAT_in = nullptr) {
  p.num_kb = (p.Ktot + BK - 1) / BK;
  if (!tma_a_ok) p.kb_tma_a = 0;
  p.tail_T = tmAT_in != nullptr && p.num_kb > p.kb_tma_a;
  const GemmPlan plan = choose_plan(m_tiles, p.N, p.num_kb, p.num_kb - p.kb_tma_a, p.Ktot - p.kb_tma_a * BK,
                                    p.mode == MODE_CONV, p.tail_T != 0);
  p.split_k = plan.split_k;
  p.m_tiles = plan.m_tiles;
  p.n_tiles = plan.n_tiles;
  p.total_items = (int)((long long)plan.m_tiles * plan.n_tiles);

  CUtensorMap tmB;
  {
    const cuuint64_t dims[2] = {(cuuint64_t)p.Ktot, (cuuint64_t)p.N};
    const cuuint64_t strides[1] = {(cuuint64_t)ldw};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)plan.BN};
    if (!encode_u8(&tmB, W_codes, 2, dims, strides, box)) return OCS_ERR_CUDA;
  }
  CUtensorMap tmA = tmB;  // a valid map even when unused
  if (p.kb_tma_a > 0) tmA = *tmA_in;
  CUtensorMap tmAT = tmB;
  if (p.tail_T) tmAT = *tmAT_in;

  p.out_rows = out_rows;
  (void)ws; (void)ws_bytes;   // the K split exchanges its partial sums through shared memory: no global scratch
  switch (plan.BN) {
    case 256: return launch_gemm<256>(tmB, tmA, tmAT, p, plan, stream);
    case 192: return launch_gemm<192>(tmB, tmA, tmAT, p, plan, stream);
    case 128: return launch_gemm<128>(tmB, tmA, tmAT, p, plan, stream);
    default: return launch_gemm<64>(tmB, tmA, tmAT, p, plan, stream);
  }
}

// M-tile box for the convolution: the (bw, bh, bn) with bw*bh*bn <= 128 that needs the fewest tiles.
void choose_conv_box(int Wo, int Ho, int Nb, int* bw_o, int* bh_o, int* bn_o) {
  long long best_tiles = -1;
  int bbw = 1, bbh = 1, bbn = 1;
  for (int bw = 1; bw <= Wo && bw <= BM; ++bw) {
    for (int bh = 1; bh <= Ho && bw * bh <= BM; ++bh) {
      int bn = BM / (bw * bh);
      if (bn > Nb) bn = Nb;
      if (bn > 256) bn = 256;
      const long long tiles = (long long)((Wo + bw - 1) / bw) * ((Ho + bh - 1) / bh) * ((Nb + bn - 1) / bn);
      if (best_tiles < 0 || tiles < best_tiles || (tiles == best_tiles && bw > bbw)) {
        best_tiles = tiles; bbw = bw; bbh = bh; bbn = bn;
      }
    }
  }
  *bw_o = bbw; *bh_o = bbh; *bn_o = bbn;
}

// Contraction indices one filter tap occupies in the packed weights: C, except that a channel count
// that is a multiple of 16 but not of the K-block is padded up to the K-block, so that every K-block
// lies inside one tap and its activation tile can come by TMA (the padding multiplies zero weights
// with zero-filled out-of-range channels).
int conv_tap_stride(int C) { return (C % 16 == 0 && C % BK != 0) ? (C + BK - 1) / BK * BK : C; }

// (vb, vg): this CTA's index and the number of CTAs working on this layer (a whole launch, or a share of one)
__device__ __forceinline__ void pack_conv_body(const int8_t* __restrict__ src, int O, int C, int Cp, int S, int R,
                                               long long ld_src, int8_t* __restrict__ dst, long long ld_dst, int vb, int vg) {
  const long long total = (long long)O * ld_dst;
  const int KO = R * Cp, Kt = KO + R * S;
  for (long long i = vb * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)vg * blockDim.x) {
    const long long o = i / ld_dst;
    const int k = (int)(i - o * ld_dst);
    int8_t v = 0;
    if (k < Kt) {
      int tap, j;
      if (k < KO) { tap = k / Cp; j = k - tap * Cp; }
      else { const int kd = k - KO; tap = kd / S; j = C + (kd - tap * S); }
      if (k >= KO || j < C) v = src[o * ld_src + (long long)j * R + tap];
    }
    dst[i] = v;
  }
}

__global__ void pack_conv_kernel(const int8_t* __restrict__ src, int O, int C, int Cp, int S, int R, long long ld_src,
                                 int8_t* __restrict__ dst, long long ld_dst) {
  pack_conv_body(src, O, C, Cp, S, R, ld_src, dst, ld_dst, blockIdx.x, gridDim.x);
}

// The same reordering for many layers in one launch: a CTA looks up its layer and its place among that layer's CTAs.
constexpr int kMaxPackBatch = 64;
struct PackJob {
  const int8_t* src; int8_t* dst;
  long long ld_src, ld_dst;
  int O, C, Cp, S, R, blk0, blks, pad;
};
struct PackTable {
  int n, pad[3];
  PackJob j[kMaxPackBatch];
};
__global__ void __launch_bounds__(256) batch_pack_kernel(const __grid_constant__ PackTable t) {
  int li = 0;
  while (li + 1 < t.n && (int)blockIdx.x >= t.j[li + 1].blk0) ++li;
  const PackJob& y = t.j[li];
  pack_conv_body(y.src, y.O, y.C, y.Cp, y.S, y.R, y.ld_src, y.dst, y.ld_dst, (int)blockIdx.x - y.blk0, y.blks);
}


// A convolution whose pixels TMA cannot address (a channel count that is not a multiple of 16 bytes, such
// as a network's first layer) is run as a plain GEMM over its patch matrix: row m = output pixel
// (n, oh, ow), column k = packed contraction index ([tap][c < C] then [tap][s < S], the order of the packed
// weights), out-of-image taps zero.  Building it costs one pass of coalesced 32-bit stores; every byte of
// the main loop then arrives by TMA instead of by byte gathers.  The duplicated channels are columns of
// the matrix like any other, read through idx_map here.
constexpr int kPatchMaxK = 4096;   // source table in shared memory: 8 bytes per contraction index

// One CTA builds the patch rows of `tw` neighbouring output pixels of one output row: the kh input rows they
// touch are staged in shared memory once (zero where the image ends), so every input byte is read from global
// memory once per CTA instead of once per tap, and the gather runs on shared memory.
__global__ void __launch_bounds__(256)
conv_patches_kernel(GemmParams p, uint8_t* __restrict__ P, long long ldp, int tw, int seg_per_row, long long n_units,
                    int span_bytes) {
  extern __shared__ unsigned char patch_smem[];
  KSrc* tab = reinterpret_cast<KSrc*>(patch_smem);                  // [ldp]: off = dy * span + dx * C + c
  uint8_t* img = patch_smem + (size_t)ldp * sizeof(KSrc);           // [kh][span_bytes]
  bool bad = false;
  for (int k = threadIdx.x; k < (int)ldp; k += 256) {
    KSrc e = k_source(p, k, &bad);
    if (e.off >= 0) {
      const int dy = e.dydx & 255, dx = e.dydx >> 8;
      const int c = e.off - (dy * p.Wd + dx) * p.C;
      e.off = dy * span_bytes + dx * p.C + c;
    }
    tab[k] = e;
  }
  if (bad) flag(p.dev_status, OCS_DEV_BAD_INDEX);
  const int words_per_row = (int)(ldp >> 2);
  for (long long u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int seg = (int)(u % seg_per_row);
    const long long rest = u / seg_per_row;
    const int oh = (int)(rest % p.Ho), n = (int)(rest / p.Ho);
    const int ow0 = seg * tw, cnt = min(tw, p.Wo - ow0);
    const int ih0 = oh * p.stride - p.pad, iw0 = ow0 * p.stride - p.pad;
    __syncthreads();   // the previous unit's gather is done (and the table is complete)
    // bytes [lo, hi) of a staged row lie inside the image
    const int lo = max(0, -iw0) * p.C, hi = min(span_bytes, (p.Wd - iw0) * p.C);
    for (int dy = 0; dy < p.kh; ++dy) {
      const int ih = ih0 + dy;
      const bool row_ok = (unsigned)ih < (unsigned)p.H;
      const uint8_t* src = p.A + (((long long)n * p.H + ih) * p.Wd + iw0) * p.C;
      uint8_t* dst = img + dy * span_bytes;
      for (int bx = threadIdx.x; bx < span_bytes; bx += 256)
        dst[bx] = (row_ok && bx >= lo && bx < hi) ? __ldg(src + bx) : (uint8_t)0;
    }
    __syncthreads();
    const long long m0 = ((long long)n * p.Ho + oh) * p.Wo + ow0;
    if (words_per_row <= 256) {
      // a thread keeps one group of four contraction indices (their offsets in registers) and walks the pixels
      const int side = 256 / words_per_row;
      const int lp = threadIdx.x / words_per_row, kq = threadIdx.x - lp * words_per_row;
      if (lp < side) {
        int off[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) off[e] = tab[kq * 4 + e].off;
        const int step = p.stride * p.C;
        uint8_t* dst = P + (m0 + lp) * ldp + kq * 4;
        const uint8_t* base = img + lp * step;
        for (int px = lp; px < cnt; px += side, base += side * step, dst += side * ldp) {
          uint32_t word = 0;
#pragma unroll
          for (int e = 0; e < 4; ++e) word |= (off[e] >= 0 ? (uint32_t)base[off[e]] : 0u) << (8 * e);
          *reinterpret_cast<uint32_t*>(dst) = word;
        }
      }
    } else {
      for (int i = threadIdx.x; i < cnt * words_per_row; i += 256) {
        const int px = i / words_per_row, kq = i - px * words_per_row;
        const uint8_t* base = img + px * p.stride * p.C;
        uint32_t word = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int off = tab[kq * 4 + e].off;
          word |= (off >= 0 ? (uint32_t)base[off] : 0u) << (8 * e);
        }
        *reinterpret_cast<uint32_t*>(P + (m0 + px) * ldp + kq * 4) = word;
      }
    }
  }
}

}  // namespace
}  // namespace ocs

using namespace ocs;

extern "C" size_t ocs_qlinear_workspace_bytes(int M, int N, int C, int S) {
  if (M <= 0 || N <= 0 || C <= 0 || S < 0) return 256;
  const int m_tiles = (M + BM - 1) / BM;
  return 256 + align_up(splitk_ws_bound(M, N, m_tiles), 256);
}

extern "C" ocs_status ocs_qlinear(const void* A_codes, const void* A_codes_T, int64_t lda_T, int a_signed, const float* a_scale,
                                  int M, int C, int64_t lda, const int8_t* W_codes, const float* w_scale, int N, int S,
                                  int64_t ldw,
                                  const int32_t* idx_map, const float* bias, float* Y, int64_t ldy, int32_t* acc_out,
                                  const float* residual, int relu, float* max_abs_out, void* ws, size_t ws_bytes,
                                  int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!A_codes || !a_scale || !W_codes || !w_scale || !idx_map || !Y) return OCS_ERR_INVALID_ARG;
  if (S < 0) return OCS_ERR_INVALID_ARG;
  if (M <= 0 || C <= 0 || N <= 0) return OCS_ERR_SHAPE;
  const long long Ktot = (long long)C + S;
  if (lda < C || ldw < Ktot || ldy < N) return OCS_ERR_SHAPE;
  if (ldw % 16 != 0 || !aligned(W_codes, 16) || !aligned(Y, 4)) return OCS_ERR_SHAPE;
  if (A_codes_T && (lda_T < M || lda_T % 16 != 0 || !aligned(A_codes_T, 16))) return OCS_ERR_SHAPE;
  if ((residual && !aligned(residual, 4)) || (acc_out && !aligned(acc_out, 4)) || (bias && !aligned(bias, 4)))
    return OCS_ERR_SHAPE;
  if (Ktot * 255ll * 127ll > 2147483647ll) return OCS_ERR_UNSUPPORTED;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;

  GemmParams p{};
  p.mode = MODE_LINEAR;
  p.M = M; p.N = N; p.Ktot = (int)Ktot; p.C = C; p.Cp = C; p.S = S; p.R = 1;
  p.A = reinterpret_cast<const uint8_t*>(A_codes); p.lda = lda; p.a_signed = a_signed ? 1 : 0;
  p.idx_map = idx_map;
  p.a_vec16 = (lda % 16 == 0) && aligned(A_codes, 16);
  p.a_scale = a_scale; p.w_scale = w_scale; p.bias = bias; p.Y = Y; p.ldy = ldy; p.acc_out = acc_out;
  p.dev_status = dev_status;
  p.relu = relu ? 1 : 0;
  p.residual = residual;
  p.max_bits = reinterpret_cast<unsigned int*>(max_abs_out);
  if (max_abs_out && cudaMemsetAsync(max_abs_out, 0, 4, stream) != cudaSuccess) return OCS_ERR_CUDA;
  const int m_tiles = (M + BM - 1) / BM;
  // K-blocks made of original channels only; without duplicates the last, partial block is TMA-fed too (the
  // tensor map zero-fills past C)
  p.kb_tma_a = S == 0 ? (C + BK - 1) / BK : C / BK;
  p.a_box_bytes = BM * BK;
  CUtensorMap tmA;
  bool tma_ok = p.a_vec16 && p.kb_tma_a > 0;
  if (tma_ok) {
    const cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)lda};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BM};
    if (!encode_u8(&tmA, A_codes, 2, dims, strides, box)) return OCS_ERR_CUDA;
  }
  // the channel-major copy, if the caller has one: [C][lda_T], one channel's values for all rows contiguous
  CUtensorMap tmAT;
  if (A_codes_T) {
    const cuuint64_t dims[2] = {(cuuint64_t)M, (cuuint64_t)C};
    const cuuint64_t strides[1] = {(cuuint64_t)lda_T};
    const cuuint32_t box[2] = {(cuuint32_t)BM, 1u};
    if (!encode_u8(&tmAT, A_codes_T, 2, dims, strides, box)) return OCS_ERR_CUDA;
  }
  return run_gemm(p, W_codes, ldw, M, m_tiles, tma_ok, &tmA, ws, ws_bytes, stream, A_codes_T ? &tmAT : nullptr);
}

extern "C" int64_t ocs_conv_packed_k(int C, int S, int kh, int kw) {
  if (C <= 0 || S < 0 || kh <= 0 || kw <= 0) return 0;
  return (int64_t)kh * kw * ((int64_t)conv_tap_stride(C) + S);
}

extern "C" ocs_status ocs_pack_conv_weights(const int8_t* codes, int O, int C, int S, int kh, int kw, int64_t ld_src,
                                            int8_t* packed, int64_t ld_dst, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!codes || !packed || S < 0) return OCS_ERR_INVALID_ARG;
  if (O <= 0 || C <= 0 || kh <= 0 || kw <= 0) return OCS_ERR_SHAPE;
  const long long Ksrc = (long long)kh * kw * ((long long)C + S);
  const long long Kt = (long long)kh * kw * ((long long)conv_tap_stride(C) + S);
  if (ld_src < Ksrc || ld_dst < Kt || ld_dst % 16 != 0 || Kt >= (1ll << 31)) return OCS_ERR_SHAPE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  const long long total = (long long)O * ld_dst;
  const int grid = (int)((total + 255) / 256 < kNumSMs * 8 ? (total + 255) / 256 : kNumSMs * 8);
  LaunchScope ls("pack_conv_kernel", stream);
  pack_conv_kernel<<<grid, 256, 0, stream>>>(codes, O, C, conv_tap_stride(C), S, kh * kw, ld_src, packed, ld_dst);
  return launch_status();
}

extern "C" ocs_status ocs_pack_conv_weights_batch(const ocs_pack_desc* jobs, int n_jobs, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!jobs || n_jobs < 1) return OCS_ERR_INVALID_ARG;
  if (n_jobs > kMaxPackBatch) return OCS_ERR_UNSUPPORTED;
  static PackTable t;                  // 5 KB, kept off the stack; calls are serialised
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  t.n = n_jobs;
  int blk = 0;
  for (int i = 0; i < n_jobs; ++i) {
    const ocs_pack_desc& d = jobs[i];
    if (!d.codes || !d.packed || d.S < 0) return OCS_ERR_INVALID_ARG;
    if (d.O <= 0 || d.C <= 0 || d.kh <= 0 || d.kw <= 0) return OCS_ERR_SHAPE;
    const long long Ksrc = (long long)d.kh * d.kw * ((long long)d.C + d.S);
    const long long Kt = (long long)d.kh * d.kw * ((long long)conv_tap_stride(d.C) + d.S);
    if (d.ld_src < Ksrc || d.ld_dst < Kt || d.ld_dst % 16 != 0 || Kt >= (1ll << 31)) return OCS_ERR_SHAPE;
    PackJob& y = t.j[i];
    y.src = d.codes; y.dst = d.packed; y.ld_src = d.ld_src; y.ld_dst = d.ld_dst;
    y.O = d.O; y.C = d.C; y.Cp = conv_tap_stride(d.C); y.S = d.S; y.R = d.kh * d.kw;
    const long long total = (long long)d.O * d.ld_dst;
    long long want = (total + 256 * 16 - 1) / (256 * 16);     // sixteen bytes per thread
    if (want < 1) want = 1;
    if (want > kNumSMs) want = kNumSMs;
    y.blk0 = blk; y.blks = (int)want; blk += (int)want;
  }
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  LaunchScope ls("batch_pack_kernel", stream);
  batch_pack_kernel<<<blk, 256, 0, stream>>>(t);
  return launch_status();
}

namespace {
struct ConvGeom {
  int Ho, Wo, bw, bh, bn, tiles_w, tiles_h, tiles_n;
  long long m_tiles, out_rows;
};
bool conv_geom(int Nb, int H, int Wd, int kh, int kw, int stride, int pad, ConvGeom* g) {

  g->Ho = (H + 2 * pad - kh) / stride + 1;
  g->Wo = (Wd + 2 * pad - kw) / stride + 1;
  if (g->Ho <= 0 || g->Wo <= 0) return false;
  choose_conv_box(g->Wo, g->Ho, Nb, &g->bw, &g->bh, &g->bn);
  g->tiles_w = (g->Wo + g->bw - 1) / g->bw;
  g->tiles_h = (g->Ho + g->bh - 1) / g->bh;
  g->tiles_n = (Nb + g->bn - 1) / g->bn;
  g->m_tiles = (long long)g->tiles_w * g->tiles_h * g->tiles_n;
  g->out_rows = (long long)Nb * g->Ho * g->Wo;
  return true;
}
bool conv_tma_shape_ok(const ConvGeom& g, int C, int stride) {
  return (conv_tap_stride(C) % BK == 0) && stride <= 8 && g.bw * stride <= 256 && g.bh * stride <= 256;
}
// Bytes of the patch matrix for layers TMA cannot address (0 when TMA can, or when the matrix would be
// unreasonably wide or large: those layers keep the in-kernel gather).
size_t patch_matrix_bytes(const ConvGeom& g, int C, int S, int kh, int kw, int stride) {
  if (conv_tma_shape_ok(g, C, stride)) return 0;
  const long long Kt = (long long)kh * kw * ((long long)C + S);
  const long long ldp = (Kt + 15) / 16 * 16;
  if (ldp > kPatchMaxK || g.out_rows * ldp > (8ll << 30)) return 0;
  return align_up((size_t)(g.out_rows * ldp), 256);
}
}  // namespace

extern "C" size_t ocs_qconv_workspace_bytes(int Nb, int H, int Wd, int C, int O, int S, int kh, int kw, int stride,
                                            int pad) {
  ConvGeom g;
  if (Nb <= 0 || H <= 0 || Wd <= 0 || C <= 0 || S < 0 || O <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0 ||
      !conv_geom(Nb, H, Wd, kh, kw, stride, pad, &g))
    return 256;
  size_t bytes = 256 + align_up(splitk_ws_bound(g.out_rows, O, (g.out_rows + BM - 1) / BM), 256) +
                 align_up(splitk_ws_bound(g.out_rows, O, g.m_tiles), 256);
  bytes += patch_matrix_bytes(g, C, S, kh, kw, stride);
  return bytes;
}

extern "C" ocs_status ocs_qconv(const void* X_codes, int a_signed, const float* a_scale, int Nb, int H, int Wd, int C,
                                const int8_t* W_packed, const float* w_scale, int O, int S, int kh, int kw, int stride,
                                int pad, int64_t ldw, const int32_t* idx_map, const float* bias, float* Y,
                                int32_t* acc_out, const float* residual, int relu, float* max_abs_out, void* ws,
                                size_t ws_bytes, int* dev_status, void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!X_codes || !a_scale || !W_packed || !w_scale || !idx_map || !Y) return OCS_ERR_INVALID_ARG;
  if (S < 0) return OCS_ERR_INVALID_ARG;
  if (Nb <= 0 || H <= 0 || Wd <= 0 || C <= 0 || O <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
    return OCS_ERR_SHAPE;
  const int Cp = conv_tap_stride(C);
  const long long Ktot = (long long)kh * kw * ((long long)Cp + S);   // packed contraction length (ocs_conv_packed_k)
  if (ldw < Ktot || ldw % 16 != 0 || !aligned(W_packed, 16) || !aligned(Y, 4)) return OCS_ERR_SHAPE;
  if ((residual && !aligned(residual, 4)) || (acc_out && !aligned(acc_out, 4)) || (bias && !aligned(bias, 4)))
    return OCS_ERR_SHAPE;
  if (Ktot * 255ll * 127ll > 2147483647ll) return OCS_ERR_UNSUPPORTED;
  ConvGeom g;
  if (!conv_geom(Nb, H, Wd, kh, kw, stride, pad, &g)) return OCS_ERR_SHAPE;
  if (g.m_tiles >= (1ll << 31) || g.out_rows * (long long)O >= (1ll << 40)) return OCS_ERR_UNSUPPORTED;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;

  GemmParams p{};
  p.mode = MODE_CONV;
  p.M = (int)(g.out_rows < (1ll << 31) ? g.out_rows : 0x7fffffff);
  p.N = O; p.Ktot = (int)Ktot; p.C = C; p.Cp = Cp; p.S = S; p.R = kh * kw;
  p.A = reinterpret_cast<const uint8_t*>(X_codes); p.lda = C; p.a_signed = a_signed ? 1 : 0;
  p.idx_map = idx_map;
  p.a_vec16 = (C % 16 == 0) && aligned(X_codes, 16);
  p.Nb = Nb; p.H = H; p.Wd = Wd; p.Ho = g.Ho; p.Wo = g.Wo; p.kh = kh; p.kw = kw; p.stride = stride; p.pad = pad;
  p.bw = g.bw; p.bh = g.bh; p.bn = g.bn; p.tiles_w = g.tiles_w; p.tiles_h = g.tiles_h; p.tiles_n = g.tiles_n;
  p.a_scale = a_scale; p.w_scale = w_scale; p.bias = bias; p.Y = Y; p.ldy = O; p.acc_out = acc_out;
  p.dev_status = dev_status;
  p.relu = relu ? 1 : 0;
  p.residual = residual;
  p.max_bits = reinterpret_cast<unsigned int*>(max_abs_out);
  if (max_abs_out && cudaMemsetAsync(max_abs_out, 0, 4, stream) != cudaSuccess) return OCS_ERR_CUDA;

  // TMA serves the K-blocks of original channels: each lies inside one tap (the per-tap stride Cp is a
  // multiple of the K-block; channels past C read as zero); a strided convolution walks the image
  // with the tensor map's traversal stride
  CUtensorMap tmA;
  bool tma_ok = conv_tma_shape_ok(g, C, stride) && aligned(X_codes, 16);
  // layers TMA cannot address: build the patch matrix (if the caller's workspace has room for it) and run
  // the plain GEMM on it
  const size_t patch_bytes = patch_matrix_bytes(g, C, S, kh, kw, stride);
  if (patch_bytes > 0 && ws && aligned(ws, 256)) {
    const size_t gemm_ws = 256 + align_up(splitk_ws_bound(g.out_rows, O, (g.out_rows + BM - 1) / BM), 256);
    if (ws_bytes >= gemm_ws + patch_bytes) {
      const long long ldp = (Ktot + 15) / 16 * 16;
      uint8_t* P = reinterpret_cast<uint8_t*>(ws) + gemm_ws;
      {
        // output pixels per CTA: as many of one output row as keep the staged input rows within 40 KB
        int tw = g.Wo;
        auto span = [&](int t) { return ((t - 1) * stride + kw) * C; };
        while (tw > 1 && (size_t)kh * span(tw) > 40 * 1024) tw = (tw + 1) / 2;
        const int seg_per_row = (g.Wo + tw - 1) / tw;
        const long long n_units = (long long)Nb * g.Ho * seg_per_row;
        const size_t smem = (size_t)ldp * sizeof(KSrc) + (size_t)kh * span(tw);
        static bool attr_set = false;
        if (!attr_set) {
          if (cudaFuncSetAttribute(conv_patches_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024) != cudaSuccess)
            return OCS_ERR_CUDA;
          attr_set = true;
        }
        const int grid = (int)min(n_units, (long long)kNumSMs * 8);
        LaunchScope ls("conv_patches_kernel", stream);
        conv_patches_kernel<<<grid, 256, smem, stream>>>(p, P, ldp, tw, seg_per_row, n_units, span(tw));
        if ((st = launch_status()) != OCS_OK) return st;
      }
      GemmParams q = p;
      q.mode = MODE_LINEAR;
      q.C = (int)Ktot; q.Cp = (int)Ktot; q.S = 0; q.R = 1;
      q.A = P; q.lda = ldp; q.a_vec16 = 1;
      q.kb_tma_a = (int)((Ktot + BK - 1) / BK);
      q.a_box_bytes = BM * BK;
      const cuuint64_t dims[2] = {(cuuint64_t)Ktot, (cuuint64_t)g.out_rows};
      const cuuint64_t strides[1] = {(cuuint64_t)ldp};
      const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BM};
      if (!encode_u8(&tmA, P, 2, dims, strides, box)) return OCS_ERR_CUDA;
      return run_gemm(q, W_packed, ldw, g.out_rows, (int)((g.out_rows + BM - 1) / BM), true, &tmA, ws, gemm_ws, stream);
    }
  }
  p.kb_tma_a = tma_ok ? (kh * kw * Cp) / BK : 0;
  p.a_box_bytes = g.bw * g.bh * g.bn * BK;
  if (tma_ok) {
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)Wd, (cuuint64_t)H, (cuuint64_t)Nb};
    const cuuint64_t strides[3] = {(cuuint64_t)C, (cuuint64_t)C * Wd, (cuuint64_t)C * Wd * H};
    const cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)(g.bw * stride), (cuuint32_t)(g.bh * stride), (cuuint32_t)g.bn};
    const cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    if (!encode_u8(&tmA, X_codes, 4, dims, strides, box, estr)) return OCS_ERR_CUDA;
  }
  return run_gemm(p, W_packed, ldw, g.out_rows, (int)g.m_tiles, tma_ok, &tmA, ws, ws_bytes, stream);
}

// Self-test hook: the next ocs_qlinear / ocs_qconv calls of this process use the given tile width (64, 128, 256)
// and K split (1, 2, 4, 8; the cluster size) instead of the planner's choice, wherever the values are valid for
// the problem; bn = 0 gives the choice back to the planner.
extern "C" ocs_status ocs_selftest_force_gemm_plan(int bn, int split_k) {
  if (bn != 0 && bn != 64 && bn != 128 && bn != 192 && bn != 256) return OCS_ERR_INVALID_ARG;
  if (split_k < 0 || split_k > 8) return OCS_ERR_INVALID_ARG;
  g_force_bn = bn; g_force_sk = split_k;
  return OCS_OK;
}
