// Tensor-core path of LPConvolution / LPInnerProduct (paper Sec. 2) for sm_100a.
//
// The layer is an exact integer GEMM  acc[m][n] = sum_k A[m][k] * B[n][k]  with
//   A = activations (implicit im2col of the NHWC planes for a convolution, [B][K] rows for an
//       inner product), B = weights [N][K] (K ordered tap-major, channel-minor).
// Operands of more than 8 bits live as two byte planes (q = 256*hi + lo, hi signed, lo
// unsigned); the product of two such numbers is four int8 products
//   q_a*q_b = 2^16 hi_a*hi_b + 2^8 (hi_a*lo_b + lo_a*hi_b) + lo_a*lo_b
// each accumulated exactly in int32 by tcgen05.mma kind::i8 into its own TMEM accumulator
// (the two middle terms share one) and recombined in int64 in the epilogue.  8-bit operands
// take a single product.
//
// One persistent CTA per SM walks over output tiles (128 rows x BN columns):
//   warp 0     : TMA producer (im2col / tiled loads into a ring of shared-memory stages)
//   warp 1     : TMEM allocation and the single MMA-issuing thread
//   warps 2-5  : epilogue (tcgen05.ld -> int64 recombination -> bias, ReLU, requantize with
//                saturation, zero / saturation counters, byte-plane stores; or range / split-K)
// Every device-side wait is bounded; on expiry the kernel flags ADAPTION_ERR_TIMEOUT in the
// caller's stats word, drains what it has in flight, frees its TMEM and returns.
#include <cuda.h>

#include <cstdlib>
#include <cstring>

#include "common.cuh"

namespace adaption {

int num_sms();

namespace {

constexpr int kBM = 128;
constexpr int kMaxStages = 8;
constexpr int kMaxAccBufs = 4;
constexpr int kThreads = 192;
constexpr int kMaxBN = 256;
// int32 accumulators: the shared middle accumulator takes two products of magnitude
// <= 128*255 per k, so a reduction of up to 32768 stays below 2^31.
constexpr int64_t kMaxKPerAccumulation = 32768;

struct TcParams {
  int M, N;
  int tiles_m, tiles_n, splits, total_tiles;
  int num_kb, kb_per_split;
  int BN, BK, ksteps;
  uint32_t sbo, layout_type;
  int stages;
  uint32_t a_bytes, b_bytes, stage_bytes;
  int acc_bufs;
  uint32_t tmem_cols;
  int is_conv, OH, OW, S, cblks, w_pitch, stride_h, stride_w, pad_h, pad_w;
  const int16_t* bias;
  int bias_shift;
  RequantParams rq;
  int mode;
  int8_t* y_hi;
  uint8_t* y_lo;
  int16_t* y_q16;
  long long y_stride;
  long long* ws;
  long long ws_ld;
  adaption_stats* stats;
  unsigned long long timeout_ns;
};

struct Ctrl {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long tmem_full[kMaxAccBufs];
  unsigned long long tmem_empty[kMaxAccBufs];
  unsigned long long drain;
  uint32_t tmem_base;
  volatile uint32_t abort;
  long long bias64[4][kMaxBN];
};

// ---------------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c,
                                                int w, int h, int n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// Operand descriptors are passed as 32-bit halves: the high word (group stride, version, swizzle)
// is the same for every operand tile of a launch, the low word is the shared-memory address in
// 16-byte units, so stepping along K or to another plane is one 32-bit add.
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                       uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      ".reg .b64 da, db;\n"
      "setp.ne.b32 p, %5, 0;\n"
      "mov.b64 da, {%1, %3};\n"
      "mov.b64 db, {%2, %3};\n"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p;\n"
      "}\n" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile whose rows are BK bytes long and
// swizzled with a span of BK bytes: eight-row groups are `sbo` bytes apart; the two 16-byte
// halves of one 32-byte k-step are adjacent (leading offset 1).
// High word: group stride / 16 in bits 0-13, descriptor version 1 in bit 14, swizzle in bits 29-31.
__device__ __forceinline__ uint32_t smem_desc_hi(uint32_t sbo, uint32_t layout_type) {
  return ((sbo >> 4) & 0x3FFFu) | (1u << 14) | (layout_type << 29);
}
// Low word: start address / 16 in bits 0-13, leading offset 1 in bits 16-29.
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr) {
  return ((saddr >> 4) & 0x3FFFu) | (1u << 16);
}

// Instruction descriptor: int32 accumulate, 8-bit operands with independent signedness,
// both K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t make_idesc(bool a_signed, bool b_signed, int bn) {
  return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | ((b_signed ? 1u : 0u) << 10) |
         ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// Bounded wait on an mbarrier phase.  Returns false once the time limit is hit (or another
// role already gave up); the caller then leaves its loop.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, Ctrl* ctrl, const TcParams& p) {
  const unsigned long long t0 = global_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 127u) == 0) {
      if (ctrl->abort) return false;
      if (global_ns() - t0 > p.timeout_ns) {
        ctrl->abort = 1;
        atomicExch(&p.stats->status, (int)ADAPTION_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, Ctrl* ctrl, const TcParams& p) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow(bar, parity, ctrl, p);
}

struct TileCoord {
  int m0, n0, kb_begin, kb_end;
};
__device__ __forceinline__ TileCoord decode_tile(int t, const TcParams& p) {
  TileCoord tc;
  const int tn = t % p.tiles_n;
  const int rest = t / p.tiles_n;
  const int split = rest % p.splits;
  const int tm = rest / p.splits;
  tc.m0 = tm * kBM;
  tc.n0 = tn * p.BN;
  tc.kb_begin = split * p.kb_per_split;
  tc.kb_end = min(p.num_kb, tc.kb_begin + p.kb_per_split);
  return tc;
}

template <int NACC>
__device__ __forceinline__ long long combine(int32_t a0, int32_t a1, int32_t a2) {
  if (NACC == 3) return (long long)a0 * 65536ll + (long long)a1 * 256ll + (long long)a2;
  if (NACC == 2) return (long long)a0 * 256ll + (long long)a1;
  return (long long)a0;
}

// Requantization of one pre-activation value for the common case of a rounding right shift
// (shift >= 1): v / 2^shift rounded half away from zero, saturated to [qmin, qmax].  The shifted
// value is narrowed to 32 bits with saturation first, so clamping and counting are 32-bit work.
// With ReLU the value is non-negative and the lower bound cannot be crossed.
template <bool RELU, bool COUNT_ALL>
__device__ __forceinline__ int32_t requant_shift_right(long long v, long long half, int shift, int32_t qmin,
                                                       int32_t qmax, bool counted, Counts& c) {
  if (RELU) v = v < 0 ? 0ll : v;
  long long t = v + half;
  if (!RELU) t += (v >> 63);
  const long long r = t >> shift;
  const int32_t r32 = (int32_t)r;
  const int32_t rh = (int32_t)(r >> 32);
  const int32_t rs = (rh == (r32 >> 31)) ? r32 : (rh < 0 ? (int32_t)0x80000000 : 0x7fffffff);
  const int32_t q = min(max(rs, qmin), qmax);
  if (COUNT_ALL) {
    c.sat_pos += (rs > qmax);
    if (!RELU) c.sat_neg += (rs < qmin);
    c.zeros += (q == 0);
  } else {
    c.sat_pos += (counted && rs > qmax);
    if (!RELU) c.sat_neg += (counted && rs < qmin);
    c.zeros += (counted && q == 0);
  }
  return q;
}

// Sixteen consecutive output columns of one row: recombine, add bias, requantize, pack into
// byte planes (and the optional int16 copy) and store 16 bytes per plane.
template <int NACC, bool RELU>
__device__ __forceinline__ void requant_store16(const int32_t* a0, const int32_t* a1, const int32_t* a2,
                                                const long long* bias64, const TcParams& p, bool row_ok,
                                                int m, int col, Counts& cnt) {
  int32_t q[16];
  const int nvalid = row_ok ? min(max(p.N - col, 0), 16) : 0;
  if (p.rq.shift > 0) {
    const long long half = 1ll << (p.rq.shift - 1);
    if (nvalid == 16) {
#pragma unroll
      for (int j = 0; j < 16; ++j)
        q[j] = requant_shift_right<RELU, true>(
            combine<NACC>(a0[j], NACC >= 2 ? a1[j] : 0, NACC == 3 ? a2[j] : 0) + bias64[j], half, p.rq.shift,
            p.rq.qmin, p.rq.qmax, true, cnt);
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j)
        q[j] = requant_shift_right<RELU, false>(
            combine<NACC>(a0[j], NACC >= 2 ? a1[j] : 0, NACC == 3 ? a2[j] : 0) + bias64[j], half, p.rq.shift,
            p.rq.qmin, p.rq.qmax, j < nvalid, cnt);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      q[j] = requant_value(combine<NACC>(a0[j], NACC >= 2 ? a1[j] : 0, NACC == 3 ? a2[j] : 0) + bias64[j],
                           p.rq, j < nvalid, cnt);
  }
  if (row_ok && col < p.y_stride) {
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) w[j] = __byte_perm((uint32_t)q[2 * j], (uint32_t)q[2 * j + 1], 0x5410);
    const size_t off = (size_t)m * (size_t)p.y_stride + (size_t)col;
    *reinterpret_cast<uint4*>(p.y_lo + off) =
        make_uint4(__byte_perm(w[0], w[1], 0x6420), __byte_perm(w[2], w[3], 0x6420),
                   __byte_perm(w[4], w[5], 0x6420), __byte_perm(w[6], w[7], 0x6420));
    if (p.rq.out_planes == 2)
      *reinterpret_cast<uint4*>(p.y_hi + off) =
          make_uint4(__byte_perm(w[0], w[1], 0x7531), __byte_perm(w[2], w[3], 0x7531),
                     __byte_perm(w[4], w[5], 0x7531), __byte_perm(w[6], w[7], 0x7531));
    if (p.y_q16 != nullptr) {
      uint4* dst = reinterpret_cast<uint4*>(p.y_q16 + off);
      dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
      dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
  }
}

// ---------------------------------------------------------------------------------- kernel
template <int NAX, int NBW>
__global__ void __launch_bounds__(kThreads, 1)
lp_gemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
               const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
               const TcParams p) {
  constexpr int NACC = NAX + NBW - 1;
  extern __shared__ uint8_t smem_raw[];
  __shared__ Ctrl ctrl;

  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctrl.full[s]), 1);
      mbar_init(smem_u32(&ctrl.empty[s]), 1);
    }
    for (int b = 0; b < p.acc_bufs; ++b) {
      mbar_init(smem_u32(&ctrl.tmem_full[b]), 1);
      mbar_init(smem_u32(&ctrl.tmem_empty[b]), 4);
    }
    mbar_init(smem_u32(&ctrl.drain), 1);
    ctrl.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctrl.tmem_base), p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0, ph = 0;
      int s = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x) {
        const TileCoord tc = decode_tile(t, p);
        int img = 0, base_h = 0, base_w = 0;
        int tap = 0, cb = 0, r = 0, sx = 0;       // position of kb in the (tap, channel block) order
        if (p.is_conv) {
          const int ow = tc.m0 % p.OW;
          const int rest = tc.m0 / p.OW;
          const int oh = rest % p.OH;
          img = rest / p.OH;
          base_w = ow * p.stride_w - p.pad_w;
          base_h = oh * p.stride_h - p.pad_h;
          tap = tc.kb_begin / p.cblks;
          cb = tc.kb_begin - tap * p.cblks;
          r = tap / p.S;
          sx = tap - r * p.S;
        }
        for (int kb = tc.kb_begin; kb < tc.kb_end; ++kb, ++it) {
          if (!wait_bar(smem_u32(&ctrl.empty[s]), ph ^ 1u, &ctrl, p)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctrl.full[s]);
          mbar_expect_tx(full, p.stage_bytes);
          const uint32_t sa = ring + (uint32_t)s * p.stage_bytes;
          const uint32_t sb = sa + NAX * p.a_bytes;
          if (p.is_conv) {
            tma_load_im2col(sa, &map_a0, full, cb * p.BK, base_w, base_h, img, (uint16_t)sx, (uint16_t)r);
            if (NAX == 2)
              tma_load_im2col(sa + p.a_bytes, &map_a1, full, cb * p.BK, base_w, base_h, img, (uint16_t)sx,
                              (uint16_t)r);
            const int kcol = tap * p.w_pitch + cb * p.BK;
            tma_load_2d(sb, &map_b0, full, kcol, tc.n0);
            if (NBW == 2) tma_load_2d(sb + p.b_bytes, &map_b1, full, kcol, tc.n0);
            if (++cb == p.cblks) {
              cb = 0;
              ++tap;
              if (++sx == p.S) { sx = 0; ++r; }
            }
          } else {
            const int kcol = kb * p.BK;
            tma_load_2d(sa, &map_a0, full, kcol, tc.m0);
            if (NAX == 2) tma_load_2d(sa + p.a_bytes, &map_a1, full, kcol, tc.m0);
            tma_load_2d(sb, &map_b0, full, kcol, tc.n0);
            if (NBW == 2) tma_load_2d(sb + p.b_bytes, &map_b1, full, kcol, tc.n0);
          }
          if (++s == p.stages) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok || ctrl.abort) {
        // gave up: let the copies already issued land before the CTA releases its shared memory
        const uint32_t n = it < (uint32_t)p.stages ? it : (uint32_t)p.stages;
        for (uint32_t j = it - n; j < it; ++j) {
          const int sj = (int)(j % (uint32_t)p.stages);
          const uint32_t pj = (j / (uint32_t)p.stages) & 1u;
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(smem_u32(&ctrl.full[sj]), pj) && global_ns() - t0 < 50000000ull) {
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t id_ss = make_idesc(true, true, p.BN);
      const uint32_t id_su = make_idesc(true, false, p.BN);
      const uint32_t id_us = make_idesc(false, true, p.BN);
      const uint32_t id_uu = make_idesc(false, false, p.BN);
      const uint32_t dhi = smem_desc_hi(p.sbo, p.layout_type);
      const uint32_t ring_lo = smem_desc_lo(ring);
      const uint32_t stage_u = p.stage_bytes >> 4, a_u = p.a_bytes >> 4, b_u = p.b_bytes >> 4;
      uint32_t it = 0, tile_iter = 0, ph = 0;
      int s = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x, ++tile_iter) {
        const TileCoord tc = decode_tile(t, p);
        const uint32_t buf = tile_iter % (uint32_t)p.acc_bufs;
        const uint32_t bph = (tile_iter / (uint32_t)p.acc_bufs) & 1u;
        if (!wait_bar(smem_u32(&ctrl.tmem_empty[buf]), bph ^ 1u, &ctrl, p)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d0 = tmem_base + buf * (uint32_t)(NACC * p.BN);
        const uint32_t d1 = d0 + (uint32_t)p.BN, d2 = d0 + 2u * (uint32_t)p.BN;
        for (int kb = tc.kb_begin; kb < tc.kb_end; ++kb, ++it) {
          if (!wait_bar(smem_u32(&ctrl.full[s]), ph, &ctrl, p)) { ok = false; break; }
          tc_fence_after();
          // low descriptor words of the operand planes of this stage (16-byte units)
          const uint32_t a0 = ring_lo + (uint32_t)s * stage_u;
          const uint32_t a1 = a0 + a_u;
          const uint32_t b0 = a0 + NAX * a_u;
          const uint32_t b1 = b0 + b_u;
          uint32_t acc = kb > tc.kb_begin ? 1u : 0u;
          for (uint32_t ks = 0; ks < 2u * (uint32_t)p.ksteps; ks += 2u, acc = 1u) {   // 32 bytes per k-step
            if (NAX == 2 && NBW == 2) {
              mma_i8(d0, a0 + ks, b0 + ks, dhi, id_ss, acc);          // hi*hi   weight 2^16
              mma_i8(d1, a0 + ks, b1 + ks, dhi, id_su, acc);          // hi*lo   weight 2^8
              mma_i8(d1, a1 + ks, b0 + ks, dhi, id_us, 1u);           // lo*hi   weight 2^8
              mma_i8(d2, a1 + ks, b1 + ks, dhi, id_uu, acc);          // lo*lo   weight 1
            } else if (NAX == 2 && NBW == 1) {
              mma_i8(d0, a0 + ks, b0 + ks, dhi, id_ss, acc);          // hi*w    weight 2^8
              mma_i8(d1, a1 + ks, b0 + ks, dhi, id_us, acc);          // lo*w    weight 1
            } else if (NAX == 1 && NBW == 2) {
              mma_i8(d0, a0 + ks, b0 + ks, dhi, id_ss, acc);          // x*hi    weight 2^8
              mma_i8(d1, a0 + ks, b1 + ks, dhi, id_su, acc);          // x*lo    weight 1
            } else {
              mma_i8(d0, a0 + ks, b0 + ks, dhi, id_ss, acc);
            }
          }
          tc_commit(smem_u32(&ctrl.empty[s]));                // stage reusable once these MMAs retire
          if (++s == p.stages) { s = 0; ph ^= 1u; }
        }
        if (ok) tc_commit(smem_u32(&ctrl.tmem_full[buf]));    // accumulators of this tile complete
      }
      if (!ok || ctrl.abort) {
        // make sure no MMA still reads shared memory or writes TMEM when the CTA tears down
        tc_commit(smem_u32(&ctrl.drain));
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&ctrl.drain), 0) && global_ns() - t0 < 50000000ull) {
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;          // TMEM lanes 32*quarter .. 32*quarter+31
    const int ew = warp - 2;               // private bias staging slot
    long long* bias64 = ctrl.bias64[ew];
    uint32_t tile_iter = 0;
    Counts cnt;
    long long vmax = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x, ++tile_iter) {
      const TileCoord tc = decode_tile(t, p);
      const uint32_t buf = tile_iter % (uint32_t)p.acc_bufs;
      const uint32_t bph = (tile_iter / (uint32_t)p.acc_bufs) & 1u;
      __syncwarp();
      for (int c = lane; c < p.BN; c += 32) {
        const int n = tc.n0 + c;
        long long b = 0;
        if (p.bias != nullptr && n < p.N && p.splits == 1) b = (long long)p.bias[n] * (1ll << p.bias_shift);
        bias64[c] = b;
      }
      __syncwarp();
      bool w = wait_bar(smem_u32(&ctrl.tmem_full[buf]), bph, &ctrl, p);
      w = __all_sync(0xffffffffu, w);
      if (!w) { ok = false; break; }
      tc_fence_after();
      const int m = tc.m0 + quarter * 32 + lane;
      const bool row_ok = m < p.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * (uint32_t)(NACC * p.BN);
      for (int c0 = 0; c0 < p.BN; c0 += 32) {
        int32_t a0[32], a1[32], a2[32];
        tmem_ld32(taddr + c0, a0);
        if (NACC >= 2) tmem_ld32(taddr + p.BN + c0, a1);
        if (NACC == 3) tmem_ld32(taddr + 2 * p.BN + c0, a2);
        tmem_ld_wait();
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          const int col = tc.n0 + c0 + 16 * g;
          if (p.splits > 1) {
            // partial sums of this K range go to the int64 workspace
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const long long v = combine<NACC>(a0[16 * g + j], NACC >= 2 ? a1[16 * g + j] : 0,
                                                NACC == 3 ? a2[16 * g + j] : 0);
              if (row_ok && col + j < p.N && v != 0)
                atomicAdd((unsigned long long*)(p.ws + (long long)m * p.ws_ld + col + j),
                          (unsigned long long)v);
            }
          } else if (p.mode == ADAPTION_MODE_RANGE) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              long long v = combine<NACC>(a0[16 * g + j], NACC >= 2 ? a1[16 * g + j] : 0,
                                          NACC == 3 ? a2[16 * g + j] : 0) +
                            bias64[c0 + 16 * g + j];
              if (p.rq.relu && v < 0) v = 0;
              v = v < 0 ? -v : v;
              if (row_ok && col + j < p.N) vmax = v > vmax ? v : vmax;
            }
          } else if (p.rq.relu) {
            requant_store16<NACC, true>(a0 + 16 * g, a1 + 16 * g, a2 + 16 * g, bias64 + c0 + 16 * g, p, row_ok, m,
                                        col, cnt);
          } else {
            requant_store16<NACC, false>(a0 + 16 * g, a1 + 16 * g, a2 + 16 * g, bias64 + c0 + 16 * g, p, row_ok,
                                         m, col, cnt);
          }
        }
      }
      // accumulators of this buffer are in registers / memory: hand the buffer back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl.tmem_empty[buf]));
    }
    if (p.splits == 1) {
      if (p.mode == ADAPTION_MODE_RANGE)
        flush_max_warp(vmax, p.stats);
      else
        flush_counts_warp(cnt, p.stats);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// ---------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

bool load_driver_entry_points() {
  if (g_encode_tiled != nullptr && g_encode_im2col != nullptr) return true;
  void* f1 = nullptr;
  void* f2 = nullptr;
  cudaDriverEntryPointQueryResult q1, q2;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f1, cudaEnableDefault, &q1) != cudaSuccess ||
      q1 != cudaDriverEntryPointSuccess || f1 == nullptr)
    return false;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f2, cudaEnableDefault, &q2) != cudaSuccess ||
      q2 != cudaDriverEntryPointSuccess || f2 == nullptr)
    return false;
  g_encode_tiled = reinterpret_cast<EncodeTiledFn>(f1);
  g_encode_im2col = reinterpret_cast<EncodeIm2colFn>(f2);
  return true;
}

struct TcConfig {
  bool ok = false;
  int BN = 0, BK = 0;
  CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE;
  uint32_t layout_type = 0;
  int nax = 1, nbw = 1, nacc = 1;
  int stages = 0;
  uint32_t a_bytes = 0, b_bytes = 0, stage_bytes = 0;
  int acc_bufs = 1;
  uint32_t tmem_cols = 32;
  int num_kb = 0, splits = 1, kb_per_split = 0;
  int tiles_m = 0, tiles_n = 0;
  int cblks = 1;
  size_t smem_bytes = 0;
  size_t workspace_bytes = 0;
};

int env_int(const char* name, int dflt) {
  const char* v = std::getenv(name);
  if (v == nullptr || *v == 0) return dflt;
  return std::atoi(v);
}

TcConfig make_config(const GemmProblem& g) {
  TcConfig c;
  if (g.M <= 0 || g.N <= 0 || g.M > (int64_t)1 << 30 || g.N > (int64_t)1 << 24) return c;
  c.nax = g.x.fmt.n_bits > 8 ? 2 : 1;
  c.nbw = g.w.fmt.n_bits > 8 ? 2 : 1;
  c.nacc = c.nax + c.nbw - 1;
  int64_t k_padded;
  if (g.is_conv) {
    const int64_t cs = g.x.c_stride;
    if (cs != g.w.c_stride || cs % 32 != 0 || cs > 65536) return c;
    c.BK = cs % 128 == 0 ? 128 : (cs % 64 == 0 ? 64 : 32);
    c.cblks = (int)(cs / c.BK);
    c.num_kb = g.cs.R * g.cs.S * c.cblks;
    k_padded = (int64_t)g.cs.R * g.cs.S * cs;
    // im2col traversal limits of the tensor map (two spatial dimensions: 8-bit signed corners)
    const int lo_w = -g.cs.pad_w, lo_h = -g.cs.pad_h;
    const int up_w = g.cs.pad_w - (g.cs.S - 1), up_h = g.cs.pad_h - (g.cs.R - 1);
    if (lo_w < -128 || lo_h < -128 || up_w < -128 || up_h < -128 || up_w > 127 || up_h > 127) return c;
    if (g.cs.stride_h > 8 || g.cs.stride_w > 8 || g.cs.R > 255 || g.cs.S > 255) return c;
    // tensors below 128 KiB stay on the direct kernel (tiny problems gain nothing here)
    if ((int64_t)g.cs.N * g.cs.H * g.cs.W * cs < 131072) return c;
    if (k_padded > (int64_t)1 << 30) return c;
  } else {
    if (g.K < 32) return c;
    c.BK = g.K >= 128 ? 128 : (g.K >= 64 ? 64 : 32);
    c.num_kb = (int)((g.K + c.BK - 1) / c.BK);
    k_padded = g.K;
    if (g.K > (int64_t)1 << 30) return c;
  }
  c.swizzle = c.BK == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : (c.BK == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  c.layout_type = c.BK == 128 ? 2u : (c.BK == 64 ? 4u : 6u);
  c.BN = g.N <= 32 ? 32 : (g.N <= 64 ? 64 : 128);
  c.tiles_m = (int)((g.M + kBM - 1) / kBM);
  c.tiles_n = (int)((g.N + c.BN - 1) / c.BN);
  c.a_bytes = (uint32_t)(kBM * c.BK);
  c.b_bytes = (uint32_t)(c.BN * c.BK);
  c.stage_bytes = c.nax * c.a_bytes + c.nbw * c.b_bytes;
  const size_t budget = 232448 - sizeof(Ctrl) - 2048;
  c.stages = (int)((budget - 1024) / c.stage_bytes);
  if (c.stages > kMaxStages) c.stages = kMaxStages;
  if (c.stages < 2) return c;
  c.smem_bytes = (size_t)c.stages * c.stage_bytes + 1024;
  c.acc_bufs = 512 / (c.nacc * c.BN);
  if (c.acc_bufs > kMaxAccBufs) c.acc_bufs = kMaxAccBufs;
  if (c.acc_bufs < 1) return c;
  uint32_t cols = (uint32_t)(c.acc_bufs * c.nacc * c.BN);
  c.tmem_cols = 32;
  while (c.tmem_cols < cols) c.tmem_cols <<= 1;
  // split the reduction when one accumulation would exceed the int32-safe length, or when
  // there are too few output tiles to fill the machine and the reduction is long
  const int max_kb_per_acc = (int)(kMaxKPerAccumulation / c.BK);
  int splits = (c.num_kb + max_kb_per_acc - 1) / max_kb_per_acc;
  const int tiles = c.tiles_m * c.tiles_n;
  const int sms = num_sms();
  if (tiles * 2 <= sms && c.num_kb >= 16) {
    int want = sms / tiles;
    int cap = c.num_kb / 8;
    if (want > cap) want = cap;
    if (want > splits) splits = want;
  }
  const int forced = env_int("ADAPTION_TC_SPLITS", 0);
  if (forced > 0) splits = forced > splits ? forced : splits;
  if (splits > c.num_kb) splits = c.num_kb;
  if (splits < 1) splits = 1;
  c.kb_per_split = (c.num_kb + splits - 1) / splits;
  c.splits = (c.num_kb + c.kb_per_split - 1) / c.kb_per_split;
  if ((int64_t)c.kb_per_split * c.BK > kMaxKPerAccumulation) return c;
  if ((int64_t)tiles * c.splits > (int64_t)1 << 30) return c;
  c.workspace_bytes = c.splits > 1 ? (size_t)g.M * (size_t)g.N * sizeof(long long) : 0;
  c.ok = true;
  return c;
}

bool encode_tiled_2d(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
                     uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz) {
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_im2col_nhwc(CUtensorMap* map, const void* base, const adaption_conv_shape& s, int64_t c_stride,
                        uint32_t channels_per_pixel, CUtensorMapSwizzle swz) {
  cuuint64_t dims[4] = {(cuuint64_t)c_stride, (cuuint64_t)s.W, (cuuint64_t)s.H, (cuuint64_t)s.N};
  cuuint64_t strides[3] = {(cuuint64_t)c_stride, (cuuint64_t)c_stride * s.W,
                           (cuuint64_t)c_stride * s.W * s.H};
  int lower[2] = {-s.pad_w, -s.pad_h};
  int upper[2] = {s.pad_w - (s.S - 1), s.pad_h - (s.R - 1)};
  cuuint32_t estr[4] = {1, (cuuint32_t)s.stride_w, (cuuint32_t)s.stride_h, 1};
  return g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides,
                         lower, upper, channels_per_pixel, (cuuint32_t)kBM, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NAX, int NBW>
int launch_kernel(const CUtensorMap* maps, const TcParams& p, int grid, size_t smem, cudaStream_t stream) {
  static bool attr_set = false;
  static size_t attr_size = 0;
  if (!attr_set || smem > attr_size) {
    if (cudaFuncSetAttribute(lp_gemm_kernel<NAX, NBW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return ADAPTION_ERR_CUDA;
    attr_set = true;
    attr_size = smem;
  }
  lp_gemm_kernel<NAX, NBW><<<grid, kThreads, smem, stream>>>(maps[0], maps[1], maps[2], maps[3], p);
  return cuda_status(cudaGetLastError());
}

}  // namespace

bool tensor_path_supported(const GemmProblem& g) { return make_config(g).ok; }

size_t tensor_path_workspace(const GemmProblem& g) { return make_config(g).workspace_bytes; }

int launch_tensor(const GemmProblem& g) {
  const TcConfig c = make_config(g);
  if (!c.ok) return ADAPTION_ERR_UNSUPPORTED;
  if (!load_driver_entry_points()) return ADAPTION_ERR_CUDA;

  // plane 0 is the high byte plane when there are two, else the single plane
  const void* xa[2] = {c.nax == 2 ? g.x.hi : g.x.lo, g.x.lo};
  const void* wb[2] = {c.nbw == 2 ? g.w.hi : g.w.lo, g.w.lo};
  CUtensorMap maps[4];
  std::memset(maps, 0, sizeof(maps));
  for (int i = 0; i < 2; ++i) {
    bool ok;
    if (g.is_conv)
      ok = encode_im2col_nhwc(&maps[i], xa[i], g.cs, g.x.c_stride, (uint32_t)c.BK, c.swizzle);
    else
      ok = encode_tiled_2d(&maps[i], xa[i], (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.x.c_stride,
                           (uint32_t)c.BK, (uint32_t)kBM, c.swizzle);
    if (!ok) return ADAPTION_ERR_CUDA;
    const uint64_t wk = g.is_conv ? (uint64_t)g.cs.R * g.cs.S * g.w.c_stride : (uint64_t)g.K;
    const uint64_t wpitch = g.is_conv ? wk : (uint64_t)g.w.c_stride;
    if (!encode_tiled_2d(&maps[2 + i], wb[i], wk, (uint64_t)g.N, wpitch, (uint32_t)c.BK, (uint32_t)c.BN,
                         c.swizzle))
      return ADAPTION_ERR_CUDA;
  }

  TcParams p;
  std::memset(&p, 0, sizeof(p));
  p.M = (int)g.M; p.N = (int)g.N;
  p.tiles_m = c.tiles_m; p.tiles_n = c.tiles_n; p.splits = c.splits;
  p.total_tiles = c.tiles_m * c.tiles_n * c.splits;
  p.num_kb = c.num_kb; p.kb_per_split = c.kb_per_split;
  p.BN = c.BN; p.BK = c.BK; p.ksteps = c.BK / 32;
  p.sbo = (uint32_t)(8 * c.BK); p.layout_type = c.layout_type;
  p.stages = c.stages; p.a_bytes = c.a_bytes; p.b_bytes = c.b_bytes; p.stage_bytes = c.stage_bytes;
  p.acc_bufs = c.acc_bufs; p.tmem_cols = c.tmem_cols;
  p.is_conv = g.is_conv ? 1 : 0;
  if (g.is_conv) {
    p.OH = g.OH; p.OW = g.OW; p.S = g.cs.S; p.cblks = c.cblks; p.w_pitch = (int)g.w.c_stride;
    p.stride_h = g.cs.stride_h; p.stride_w = g.cs.stride_w; p.pad_h = g.cs.pad_h; p.pad_w = g.cs.pad_w;
  }
  p.bias = g.bias; p.bias_shift = g.bias_shift;
  p.mode = g.mode;
  if (g.mode == ADAPTION_MODE_REQUANT) {
    p.rq = make_requant(g.acc_frac_bits, g.y.fmt, g.relu);
    p.y_hi = (int8_t*)g.y.hi; p.y_lo = (uint8_t*)g.y.lo; p.y_q16 = g.y.q16; p.y_stride = g.y.c_stride;
  } else {
    p.rq = RequantParams{0, g.relu ? 1 : 0, 0, 0, 1};
  }
  p.ws = (long long*)g.workspace; p.ws_ld = g.N;
  p.stats = g.stats;
  p.timeout_ns = 2000000000ull;

  if (c.splits > 1) {
    if (cudaMemsetAsync(g.workspace, 0, c.workspace_bytes, g.stream) != cudaSuccess) return ADAPTION_ERR_CUDA;
  }
  int grid = p.total_tiles < num_sms() ? p.total_tiles : num_sms();
  int rc;
  if (c.nax == 2 && c.nbw == 2) rc = launch_kernel<2, 2>(maps, p, grid, c.smem_bytes, g.stream);
  else if (c.nax == 2) rc = launch_kernel<2, 1>(maps, p, grid, c.smem_bytes, g.stream);
  else if (c.nbw == 2) rc = launch_kernel<1, 2>(maps, p, grid, c.smem_bytes, g.stream);
  else rc = launch_kernel<1, 1>(maps, p, grid, c.smem_bytes, g.stream);
  if (rc != ADAPTION_OK) return rc;
  if (c.splits > 1) return launch_finalize((const int64_t*)g.workspace, g.N, g);
  return ADAPTION_OK;
}

}  // namespace adaption
