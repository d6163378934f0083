// Tensor-core path of LPConvolution / LPInnerProduct (paper Sec. 2) for sm_100a.
//
// The layer is an exact integer GEMM  acc[m][n] = sum_k A[m][k] * B[n][k]  with
//   A = activations (implicit im2col of the NHWC planes for a convolution, [B][K] rows for an
//       inner product), B = weights [N][K] (K ordered tap-major, channel-minor).
// Operands of more than 8 bits live as two byte planes (q = 256*hi + lo, hi signed, lo
// unsigned); the product of two such numbers is four int8 products
//   q_a*q_b = 2^16 hi_a*hi_b + 2^8 (hi_a*lo_b + lo_a*hi_b) + lo_a*lo_b
// each accumulated exactly in int32 by tcgen05.mma kind::i8 into its own TMEM accumulator
// (the two middle terms share one) and recombined exactly in the epilogue.  8-bit operands
// take a single product.
//
// One persistent CTA per SM walks over output tiles (128 rows x BN columns):
//   warps 0-2  : TMA producers, spread over the operand planes (im2col / tiled loads into a ring
//                of shared-memory stages; a single warp issues bulk-tensor copies too slowly)
//   warp  3    : MMA issue; also owns the TMEM allocation
//   warps 4-19 : epilogue (tcgen05.ld -> 64-bit recombination -> bias, ReLU, requantize with
//                saturation, zero / saturation counters; byte planes staged in shared memory and
//                written by bulk-tensor stores; or range / split-K)
// Every device-side wait is bounded; on expiry the kernel flags ADAPTION_ERR_TIMEOUT in the
// caller's stats word, drains what it has in flight, frees its TMEM and returns.
#include <cuda.h>

#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace adaption {

int num_sms();

namespace {

constexpr int kBM = 128;
constexpr int kMaxStages = 12;
constexpr int kMaxAccBufs = 4;
constexpr int kEpiWarps = 16;                // four per TMEM lane quarter, each takes a quarter of the columns
constexpr int kProducerWarps = 3;            // spread over the operand planes: TMA issue is slow per warp
// One MMA-issuing warp (a second one, alternating stages, measured no faster).
constexpr int kMmaWarps = 1;
constexpr int kMmaWarp = kProducerWarps;
constexpr int kFirstEpiWarp = kProducerWarps + kMmaWarps;
constexpr int kThreads = 32 * (kFirstEpiWarp + kEpiWarps);
// int32 accumulators: the shared middle accumulator takes two products of magnitude
// <= 128*255 per k, so a reduction of up to 32768 stays below 2^31.
constexpr int64_t kMaxKPerAccumulation = 32768;
// epilogue variants (a template parameter of the kernel): generic 64-bit, the 32-bit fast path of
// ReLU layers, generic with stochastic rounding
constexpr int kEpiGeneric = 0, kEpiFast = 1, kEpiStochastic = 2;

struct TcParams {
  int M, N;
  int tile_m;                 // rows per tile: 128, or 256 for a CTA pair
  int tiles_m, tiles_n, splits, total_tiles;
  int num_kb, kb_per_split;
  int BN, BK, ksteps;
  uint32_t sbo, layout_type;
  int stages;
  uint32_t a_bytes, b_bytes, stage_bytes;
  // a stage holds `kps` consecutive k-blocks of `kb_bytes` each (short k-blocks are grouped so
  // that the per-stage hand-shake is amortised over enough MMAs)
  int kps;
  uint32_t kb_bytes;
  // weights resident in shared memory (one column tile, short reduction): the ring then holds
  // only activation planes and all weight k-blocks are loaded once per CTA at this offset
  int b_resident;
  uint32_t b_res_off;
  int acc_bufs;
  // Three accumulators of 128 columns leave one quarter of TMEM free: the high accumulator then
  // alternates between the first and the last quarter from tile to tile (the other two stay put),
  // and the epilogue hands the low and middle accumulators back before it reads the high one, so
  // that the next tile's MMAs start while this tile's high accumulator is still being read.
  int split_hh;
  // With the split release: the last two k-blocks of a tile are issued product by product (all low
  // products, then the middle ones, then the high ones) with a completion signal after each group,
  // so that the epilogue pulls the low and the middle accumulator into registers while the
  // remaining MMAs of the tile still run, and the next tile's MMAs can follow almost at once.
  int tail_stagger;
  uint32_t tmem_cols;
  int is_conv, OH, OW, S, cblks, w_pitch, stride_h, stride_w, pad_h, pad_w;
  const int16_t* bias;
  int bias_shift;
  RequantParams rq;
  StochasticParams st;         // stochastic rounding in the requantization (generic epilogue only)
  int mode;
  int8_t* y_hi;
  uint8_t* y_lo;
  int16_t* y_q16;
  long long y_stride;
  long long* ws;
  long long ws_ld;
  adaption_stats* stats;
  unsigned long long timeout_ns;
  // test aid (adaption_debug_set "stall_at"): every producer warp stops, with nothing in flight for
  // that stage, before its stage number `stall_at` (counted per CTA from 0); -1 = never.  The waits
  // of the other roles then run out and the kernel reports ADAPTION_ERR_TIMEOUT.
  int stall_at;
  // epilogue variants chosen on the host
  int fast_relu;              // launch the FAST kernel variant (paired 16-bit epilogue)
  int pool_w;                 // store max(row 2j, row 2j+1) of the tile: half of a 2x2 max-pool (staged only)
  int epi_groups;             // 1, or 2: the epilogue warps form two groups that take alternate tiles
  int staged;                 // outputs leave through shared memory and bulk-tensor stores
  int stage_bufs;             // staging buffers per epilogue group: 1, or 2 used in turn (narrow tiles)
  uint32_t stage_off;         // offset of the staging planes from the ring base
  uint32_t const_off;         // offset of the per-column epilogue constants (8 bytes per column and group)
};

// Optional per-role time stamps of CTA 0 (development builds only: -DADAPTION_TIMELINE).
#ifdef ADAPTION_TIMELINE
__device__ long long g_timeline[8192];
#define TL_STAMP(role, tile, slot)                                                        \
  do {                                                                                    \
    if (blockIdx.x == 0 && (tile) < 32u) g_timeline[((role) * 32 + (tile)) * 8 + (slot)] = clock64(); \
  } while (0)
#else
#define TL_STAMP(role, tile, slot) do { } while (0)
#endif

struct Ctrl {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long tmem_full[kMaxAccBufs];
  unsigned long long tmem_empty[kMaxAccBufs];
  unsigned long long part_full[2];   // staggered tail: low accumulator complete, middle accumulator complete
  unsigned long long drain;     // the issuing warp's last commit before an early exit
  unsigned long long b_ready;   // resident weights have landed
  uint32_t tmem_base;
  volatile uint32_t abort;
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
// The same test, but the hardware may keep the thread suspended for up to `hint_ns` while the phase
// is incomplete (it resumes as soon as the phase completes): far fewer polling instructions.
__device__ __forceinline__ bool mbar_try_wait_suspend(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
// True in exactly one lane of a converged warp.  Code guarded by it still has its operands computed
// warp-uniformly outside the guard, which lets the compiler keep them in uniform registers (the
// tensor-core and bulk-copy instructions take uniform-register operands).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n"
      ".reg .pred P;\n"
      "elect.sync _|P, 0xffffffff;\n"
      "selp.u32 %0, 1, 0, P;\n"
      "}\n"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// PAIR: the copy lands in this CTA's shared memory but reports its bytes to an mbarrier that may
// live in the other CTA of the pair (the leader's "full" barrier).
template <bool PAIR>
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y) {
  if (PAIR)
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
  else
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c,
                                                int w, int h, int n, uint16_t off_w, uint16_t off_h) {
  if (PAIR)
    asm volatile(
        "cp.async.bulk.tensor.4d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
  else
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  if (PAIR)
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
                 "r"(ncols)
                 : "memory");
  else
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
                 "r"(ncols)
                 : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void tmem_relinquish() {
  if (PAIR)
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  else
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
template <bool PAIR>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  if (PAIR)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
  else
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}
// ---- CTA-pair plumbing
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// Arrive on `bar` once every MMA issued so far by this thread has retired.  PAIR: the arrival is
// delivered to the barrier at the same offset in both CTAs of the pair.
template <bool PAIR>
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  if (PAIR)
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
            bar),
        "h"((uint16_t)3)
        : "memory");
  else
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
// Operand descriptors are passed as 32-bit halves: the high word (group stride, version, swizzle)
// is the same for every operand tile of a launch, the low word is the shared-memory address in
// 16-byte units, so stepping along K or to another plane is one 32-bit add.
// PAIR: one instruction computes a 256-row tile across the two CTAs of the pair: each CTA supplies
// its own 128 rows of A and half of the B rows, and receives its 128 rows of the result in its TMEM.
template <bool PAIR>
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                       uint32_t idesc, uint32_t accumulate) {
  if (PAIR)
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        ".reg .b64 da, db;\n"
        "setp.ne.b32 p, %5, 0;\n"
        "mov.b64 da, {%1, %3};\n"
        "mov.b64 db, {%2, %3};\n"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p;\n"
        "}\n" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
        : "memory");
  else
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
// sixteen consecutive columns: the first eight into `lo`, the next eight into `hi`
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int32_t (&lo)[8], int32_t (&hi)[8]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(lo[0]), "=r"(lo[1]), "=r"(lo[2]), "=r"(lo[3]), "=r"(lo[4]), "=r"(lo[5]), "=r"(lo[6]), "=r"(lo[7]),
        "=r"(hi[0]), "=r"(hi[1]), "=r"(hi[2]), "=r"(hi[3]), "=r"(hi[4]), "=r"(hi[5]), "=r"(hi[6]), "=r"(hi[7])
      : "r"(taddr)
      : "memory");
}
// thirty-two consecutive columns in one instruction (a TMEM load costs about the same latency
// whatever its width, so the widest form that the register budget allows drains fastest)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void pin_after_wait32(int32_t (&r)[32]) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                 "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]),
                 "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]),
                 "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// Placed after tcgen05.wait::ld: ties the loaded registers to that point so that no use of them can
// be scheduled before the wait (the load fills them asynchronously).
__device__ __forceinline__ void pin_after_wait(int32_t (&r)[8]) {
  asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7])
               :
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


// One 32-byte k-step of a tile, issued as a single instruction sequence so that the issuing thread
// spends as few instructions per MMA as possible (its instruction stream, not the tensor pipe, is
// what limits the mainloop otherwise).  Operand descriptors: low words a0/a1/b0/b1, shared high
// word dhi.  acc = 0 overwrites the accumulators (first k-step of a tile).
#define ADAPTION_MMA_KSTEP_2X2(CG)                                                              \
  asm volatile(                                                                                 \
      "{\n"                                                                                     \
      ".reg .pred p, q;\n"                                                                      \
      ".reg .b64 da0, da1, db0, db1;\n"                                                         \
      "setp.ne.b32 p, %12, 0;\n"                                                                \
      "setp.eq.b32 q, %7, %7;\n"                                                                \
      "mov.b64 da0, {%3, %7};\n"                                                                \
      "mov.b64 da1, {%4, %7};\n"                                                                \
      "mov.b64 db0, {%5, %7};\n"                                                                \
      "mov.b64 db1, {%6, %7};\n"                                                                \
      "tcgen05.mma.cta_group::" CG ".kind::i8 [%0], da0, db0, %8, p;\n"                         \
      "tcgen05.mma.cta_group::" CG ".kind::i8 [%1], da0, db1, %9, p;\n"                         \
      "tcgen05.mma.cta_group::" CG ".kind::i8 [%1], da1, db0, %10, q;\n"                        \
      "tcgen05.mma.cta_group::" CG ".kind::i8 [%2], da1, db1, %11, p;\n"                        \
      "}\n" ::"r"(d0),                                                                          \
      "r"(d1), "r"(d2), "r"(a0), "r"(a1), "r"(b0), "r"(b1), "r"(dhi), "r"(id_ss), "r"(id_su),  \
      "r"(id_us), "r"(id_uu), "r"(acc)                                                          \
      : "memory")

template <bool PAIR>
__device__ __forceinline__ void mma_kstep_2x2(uint32_t d0, uint32_t d1, uint32_t d2, uint32_t a0, uint32_t a1,
                                              uint32_t b0, uint32_t b1, uint32_t dhi, uint32_t id_ss,
                                              uint32_t id_su, uint32_t id_us, uint32_t id_uu, uint32_t acc) {
  // hi*hi -> d0 (weight 2^16); hi*lo and lo*hi -> d1 (weight 2^8); lo*lo -> d2 (weight 1)
  if (PAIR)
    ADAPTION_MMA_KSTEP_2X2("2");
  else
    ADAPTION_MMA_KSTEP_2X2("1");
}
#undef ADAPTION_MMA_KSTEP_2X2

template <int NAX, int NBW, bool PAIR>
__device__ __forceinline__ void mma_kstep(uint32_t d0, uint32_t d1, uint32_t d2, uint32_t a0, uint32_t a1,
                                          uint32_t b0, uint32_t b1, uint32_t dhi, uint32_t id_ss, uint32_t id_su,
                                          uint32_t id_us, uint32_t id_uu, uint32_t acc) {
  if (NAX == 2 && NBW == 2) {
    mma_kstep_2x2<PAIR>(d0, d1, d2, a0, a1, b0, b1, dhi, id_ss, id_su, id_us, id_uu, acc);
  } else if (NAX == 2 && NBW == 1) {
    mma_i8<PAIR>(d0, a0, b0, dhi, id_ss, acc);          // hi*w    weight 2^8
    mma_i8<PAIR>(d1, a1, b0, dhi, id_us, acc);          // lo*w    weight 1
  } else if (NAX == 1 && NBW == 2) {
    mma_i8<PAIR>(d0, a0, b0, dhi, id_ss, acc);          // x*hi    weight 2^8
    mma_i8<PAIR>(d1, a0, b1, dhi, id_su, acc);          // x*lo    weight 1
  } else {
    mma_i8<PAIR>(d0, a0, b0, dhi, id_ss, acc);
  }
}

// Instruction descriptor: int32 accumulate, 8-bit operands with independent signedness,
// both K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t make_idesc(bool a_signed, bool b_signed, int bn, int m) {
  return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | ((b_signed ? 1u : 0u) << 10) |
         ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Bounded wait on an mbarrier phase.  Returns false once the time limit is hit (or another
// role already gave up); the caller then leaves its loop.
// `relaxed` waiters (producers, epilogue) let the hardware suspend them while the phase is
// incomplete, so that their polling neither takes issue slots from the MMA-issuing thread, whose
// instruction stream is the critical path, nor burns power during the long mainloops.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, Ctrl* ctrl, const TcParams& p,
                                       bool relaxed) {
  const unsigned long long t0 = global_ns();
  uint32_t spins = 0;
  while (!(relaxed ? mbar_try_wait_suspend(bar, parity, 1000u) : mbar_try_wait(bar, parity))) {
    if (relaxed || (++spins & 127u) == 0) {
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
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, Ctrl* ctrl, const TcParams& p,
                                         bool relaxed = true) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow(bar, parity, ctrl, p, relaxed);
}

// The same bounded wait without a function call, for waits that sit between TMEM loads whose
// results are live in registers (a call there would make the compiler save and restore them).
__device__ __forceinline__ bool wait_bar_inline(uint32_t bar, uint32_t parity, Ctrl* ctrl, const TcParams& p) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  while (!mbar_try_wait_suspend(bar, parity, 1000u)) {
    if (ctrl->abort) return false;
    if (global_ns() - t0 > p.timeout_ns) {
      ctrl->abort = 1;
      atomicExch(&p.stats->status, (int)ADAPTION_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
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
  tc.m0 = tm * p.tile_m;
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


// Fast requantization for ReLU layers with a rounding right shift 9 <= shift <= 31, in 32-bit
// arithmetic.  Wanted: floor((v + C) / 2^shift) with v = 2^16 hh + 2^8 mid + ll and the per-column
// constant C = bias * 2^bias_shift + 2^(shift-1) (ReLU maps negative values to zero, so rounding
// half away from zero is this floor).  With C = 2^16 Ch + Cl, 0 <= Cl < 2^16:
//   T = mid + floor((ll + Cl) / 2^8),  H = hh + Ch,   v + C = 2^8 (2^8 H + T) + (a remainder below 2^8)
// and because shift >= 8 the remainder cannot change the floor:
//   shift >= 16:  floor((H + floor(T / 2^8)) / 2^(shift-16))
//   shift <  16:  H * 2^(16-shift) + floor(T / 2^(shift-8))
// The host checks from the reduction length that none of these 32-bit quantities can overflow
// (otherwise the layer takes the generic 64-bit epilogue).
__device__ __forceinline__ int32_t mad_lo(int32_t a, int32_t b, int32_t c) {
  int32_t d;
  asm("mad.lo.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// two 32-bit values -> two 16-bit values saturated to [-32768, 32767]; `lo` lands in the low half
__device__ __forceinline__ uint32_t pack_sat_s16x2(int32_t hi, int32_t lo) {
  uint32_t d;
  asm("cvt.pack.sat.s16.s32 %0, %1, %2;" : "=r"(d) : "r"(hi), "r"(lo));
  return d;
}
__device__ __forceinline__ uint32_t max_s16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.s16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t min_s16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("min.s16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// Fast path, accumulator by accumulator over thirty-two columns of one row.  With T and H as derived
// above, `t` holds T (with a mixed 16 x 8-bit layer hh is absent and H = Ch) or, with 8-bit
// operands on both sides, the single accumulator (the whole sum: one 32-bit add, any shift >= 0);
// `h` holds hh.  Outputs are handled as pairs of 16-bit lanes (saturating pack, ReLU, upper bound,
// zero count).  Saturation is only detected here (some lane reached the bound); the exact count of
// that group of eight is then redone from the 32-bit results, which is rare.  Every group of eight
// columns is either entirely real or entirely padding (N is a multiple of 8).
template <int NACC, bool WIDE>
__device__ __forceinline__ int32_t fast_result(int32_t t, int32_t h, int shift) {
  if (NACC == 1) return t >> shift;
  if (WIDE) return (h + (t >> 8)) >> (shift - 16);
  return mad_lo(h, 1 << (16 - shift), t >> (shift - 8));
}
// sixteen of the thirty-two columns (`half` = 0 or 1) -> eight packed words; `t` and `h` hold T and H
// (or, with a single accumulator, t holds the sum plus its constant)
template <int NACC, bool WIDE>
__device__ __forceinline__ void fast_outputs16(const int32_t (&t)[32], const int32_t (&h)[32], int half, int shift,
                                               int32_t qmax, bool row_ok, int col, int N, Counts& cnt,
                                               uint32_t (&w)[8]) {
  const uint32_t qmax2 = (uint32_t)qmax * 0x00010001u;
  const int32_t bound = qmax == 32767 ? 32767 : qmax + 1;      // a lane that reached this may have been clipped
#pragma unroll
  for (int g = 0; g < 2; ++g) {
    const int base = 16 * half + 8 * g;
    const bool counted = row_ok && col + base < N;
    uint32_t top = 0, nonzero = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int k = base + 2 * j;
      const int32_t r0 = fast_result<NACC, WIDE>(t[k], h[k], shift);
      const int32_t r1 = fast_result<NACC, WIDE>(t[k + 1], h[k + 1], shift);
      uint32_t v = max_s16x2(pack_sat_s16x2(r1, r0), 0u);
      top = max_s16x2(top, v);
      if (qmax != 32767) v = min_s16x2(v, qmax2);
      nonzero += min_s16x2(v, 0x00010001u);
      w[4 * g + j] = v;
    }
    if (counted) cnt.zeros += 8u - (nonzero & 0xffffu) - (nonzero >> 16);
    if (counted && ((int32_t)(top & 0xffffu) >= bound || (int32_t)(top >> 16) >= bound)) {
#pragma unroll
      for (int j = 0; j < 8; ++j) cnt.sat_pos += (fast_result<NACC, WIDE>(t[base + j], h[base + j], shift) > qmax);
    }
  }
}

// One group of accumulators for eight consecutive columns of one row.
template <int NACC>
struct Acc8 {
  int32_t a[3][8];
};
// sixteen columns as two groups of eight, one load instruction per accumulator
template <int NACC>
__device__ __forceinline__ void load_acc16(uint32_t taddr, uint32_t first_off, int bn, Acc8<NACC>& x, Acc8<NACC>& y) {
  tmem_ld16(taddr + first_off, x.a[0], y.a[0]);
  if (NACC >= 2) tmem_ld16(taddr + (uint32_t)bn, x.a[1], y.a[1]);
  if (NACC == 3) tmem_ld16(taddr + 2u * (uint32_t)bn, x.a[2], y.a[2]);
}
template <int NACC>
__device__ __forceinline__ void pin_acc8(Acc8<NACC>& x) {
  pin_after_wait(x.a[0]);
  if (NACC >= 2) pin_after_wait(x.a[1]);
  if (NACC == 3) pin_after_wait(x.a[2]);
}
template <int NACC>
__device__ __forceinline__ long long acc_value(const Acc8<NACC>& x, int j) {
  return combine<NACC>(x.a[0][j], NACC >= 2 ? x.a[1][j] : 0, NACC == 3 ? x.a[2][j] : 0);
}

// Draws of the eight consecutive elements i0 .. i0 + 7 (two or three generator blocks).
__device__ __forceinline__ void philox_draws8(uint64_t i0, uint32_t k0, uint32_t k1, uint32_t (&R)[8]) {
  const uint64_t b0 = i0 >> 2;
  const uint32_t off = (uint32_t)i0 & 3u;
  const Philox4 a = philox4x32_10((uint32_t)b0, (uint32_t)(b0 >> 32), 0u, 0u, k0, k1);
  const Philox4 b = philox4x32_10((uint32_t)(b0 + 1), (uint32_t)((b0 + 1) >> 32), 0u, 0u, k0, k1);
  if (off == 0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) { R[j] = a.w[j]; R[4 + j] = b.w[j]; }
    return;
  }
  const Philox4 c = philox4x32_10((uint32_t)(b0 + 2), (uint32_t)((b0 + 2) >> 32), 0u, 0u, k0, k1);
  const uint32_t w[12] = {a.w[0], a.w[1], a.w[2], a.w[3], b.w[0], b.w[1], b.w[2], b.w[3], c.w[0], c.w[1], c.w[2], c.w[3]};
#pragma unroll
  for (int j = 0; j < 8; ++j) R[j] = off == 1 ? w[j + 1] : (off == 2 ? w[j + 2] : w[j + 3]);
}

template <int NACC, bool RELU, bool STOCH>
__device__ __forceinline__ void requant8(const Acc8<NACC>& x, const long long* c64, const TcParams& p, bool row_ok,
                                         int m, int col, Counts& cnt, uint32_t* w) {
  const int nvalid = row_ok ? min(max(p.N - col, 0), 8) : 0;
  int32_t q[8];
  if (STOCH && p.rq.shift > 0) {
    // stochastic rounding: element index = row-major index over the real M x N outputs
    uint32_t R[8];
    if (nvalid > 0) philox_draws8((uint64_t)m * (uint64_t)p.N + (uint64_t)col, p.st.key0, p.st.key1, R);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      q[j] = j < nvalid ? requant_value_stochastic(acc_value<NACC>(x, j) + c64[j], p.rq, R[j], true, cnt)
                        : requant_value(0, p.rq, false, cnt);
  } else if (p.rq.shift > 0) {
    const long long half = 1ll << (p.rq.shift - 1);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      q[j] = requant_shift_right<RELU, false>(acc_value<NACC>(x, j) + c64[j], half, p.rq.shift, p.rq.qmin, p.rq.qmax,
                                              j < nvalid, cnt);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) q[j] = requant_value(acc_value<NACC>(x, j) + c64[j], p.rq, j < nvalid, cnt);
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) w[j] = __byte_perm((uint32_t)q[2 * j], (uint32_t)q[2 * j + 1], 0x5410);
}

// What the epilogue does with eight accumulator columns of one row in the modes that store nothing:
// split-K partial sums go to the int64 workspace, the range mode keeps the largest magnitude.
template <int NACC>
__device__ __forceinline__ void partial_or_range8(const Acc8<NACC>& x, const long long* c64, const TcParams& p,
                                                  bool row_ok, int m, int col, long long& vmax) {
  if (p.splits > 1) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const long long v = acc_value<NACC>(x, j);
      if (row_ok && col + j < p.N && v != 0)
        atomicAdd((unsigned long long*)(p.ws + (long long)m * p.ws_ld + col + j), (unsigned long long)v);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      long long v = acc_value<NACC>(x, j) + c64[j];
      if (p.rq.relu && v < 0) v = 0;
      v = v < 0 ? -v : v;
      if (row_ok && col + j < p.N) vmax = v > vmax ? v : vmax;
    }
  }
}

// byte planes of sixteen packed outputs: four low bytes / four high bytes per word
__device__ __forceinline__ uint4 plane_lo(const uint32_t* w) {
  return make_uint4(__byte_perm(w[0], w[1], 0x6420), __byte_perm(w[2], w[3], 0x6420),
                    __byte_perm(w[4], w[5], 0x6420), __byte_perm(w[6], w[7], 0x6420));
}
__device__ __forceinline__ uint4 plane_hi(const uint32_t* w) {
  return make_uint4(__byte_perm(w[0], w[1], 0x7531), __byte_perm(w[2], w[3], 0x7531),
                    __byte_perm(w[4], w[5], 0x7531), __byte_perm(w[6], w[7], 0x7531));
}

// Direct stores of sixteen outputs of one row (16 bytes per plane; optional int16 copy).
__device__ __forceinline__ void store16_global(const uint32_t* w, const TcParams& p, bool row_ok, int m,
                                               int col) {
  if (row_ok && col < p.y_stride) {
    const size_t off = (size_t)m * (size_t)p.y_stride + (size_t)col;
    *reinterpret_cast<uint4*>(p.y_lo + off) = plane_lo(w);
    if (p.rq.out_planes == 2) *reinterpret_cast<uint4*>(p.y_hi + off) = plane_hi(w);
    if (p.y_q16 != nullptr) {
      uint4* dst = reinterpret_cast<uint4*>(p.y_q16 + off);
      dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
      dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
  }
}

// Staged stores: the tile's byte planes are assembled in shared memory (rows of BN bytes, 16-byte
// chunks swizzled the way the bulk-tensor store expects for that row length, which also keeps the
// 16-byte writes of a quarter warp on distinct banks) and leave as one bulk-tensor store per plane.
// (Rows longer than the 128-byte swizzle span are kept as sub-planes of 128 columns, one store each.)
__device__ __forceinline__ uint32_t staged_offset(int row, int chunk, int bn) {
  const int sub = chunk >> 3;
  const int w = bn < 128 ? bn : 128;                       // row length of a (sub-)plane
  uint32_t off = (uint32_t)row * (uint32_t)w + (uint32_t)(chunk & 7) * 16u;
  off ^= ((off >> 7) & (uint32_t)((w >> 4) - 1) & 7u) << 4;
  return off + (uint32_t)sub * (uint32_t)(kBM * 128);
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map),
               "r"(src), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// the bulk stores committed so far have read their shared-memory source
// ... all but the most recent group have (two staging buffers in turn)
__device__ __forceinline__ void bulk_wait_read_all_but_one() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_read_all() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
// ... and have completed
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_shared() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Barriers among the warps of one epilogue group only (barrier 0 belongs to __syncthreads; group g
// uses barriers 1 + 2g and 2 + 2g).
__device__ __forceinline__ void epi_bar_sync(int group, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(1 + 2 * group), "r"(threads) : "memory");
}
// ... that also returns the conjunction of every thread's predicate
__device__ __forceinline__ bool epi_bar_all(int group, int threads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n"
      ".reg .pred p, q;\n"
      "setp.ne.b32 p, %1, 0;\n"
      "bar.red.and.pred q, %2, %3, p;\n"
      "selp.u32 %0, 1, 0, q;\n"
      "}\n"
      : "=r"(r)
      : "r"((uint32_t)pred), "r"(2 + 2 * group), "r"(threads)
      : "memory");
  return r != 0;
}

// An epilogue warp hands accumulator columns back to the issuing warp (of the leader CTA in a pair).
template <bool PAIR>
__device__ __forceinline__ void release_accumulators(unsigned long long* bar_ptr, int lane) {
  tc_fence_before();
  __syncwarp();
  if (lane == 0) {
    const uint32_t bar = smem_u32(bar_ptr);
    if (PAIR)
      mbar_arrive_cluster(mapa_rank(bar, 0));
    else
      mbar_arrive(bar);
  }
}

// ---------------------------------------------------------------------------------- kernel
// GROUPED: stages hold several k-blocks and / or the weights are resident in shared memory (short
// reductions); the plain variant keeps the issue loops free of that bookkeeping.
// FAST: ReLU layer in requantizing mode whose shift lies in [9, 31] ([0, 31] with 8-bit operands
// on both sides), N a multiple of 8, no split-K,
// magnitudes within the 32-bit bounds of the fast epilogue: it then contains only that path.
// 20 warps: one block per SM, 96 registers per thread.
template <int NAX, int NBW, bool PAIR, bool GROUPED, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
lp_gemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
               const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
               const __grid_constant__ CUtensorMap map_y_hi, const __grid_constant__ CUtensorMap map_y_lo,
               const TcParams p) {
  constexpr int NACC = NAX + NBW - 1;
  constexpr bool FAST = EPI == kEpiFast;
  constexpr bool STOCH = EPI == kEpiStochastic;
  extern __shared__ uint8_t smem_raw[];
  __shared__ Ctrl ctrl;

  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform for the compiler too
  const int lane = threadIdx.x & 31;
  // PAIR: two CTAs (a cluster of two) share every tile of 256 rows.  Rank 0 is the leader: it owns
  // the "full" and "tmem_empty" barriers that are in use and issues the MMAs for both.
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  // rows of B this CTA stages per k-block, and where they start inside the tile's columns
  const int b_rows = PAIR ? p.BN / 2 : p.BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctrl.full[s]), 1);
      mbar_init(smem_u32(&ctrl.empty[s]), 1);
    }
    for (int b = 0; b < kMaxAccBufs; ++b) {
      mbar_init(smem_u32(&ctrl.tmem_full[b]), 1);
      mbar_init(smem_u32(&ctrl.tmem_empty[b]), (uint32_t)((PAIR ? 2 : 1) * (kEpiWarps / p.epi_groups)));
    }
    mbar_init(smem_u32(&ctrl.part_full[0]), 1);
    mbar_init(smem_u32(&ctrl.part_full[1]), 1);
    mbar_init(smem_u32(&ctrl.drain), 1);
    mbar_init(smem_u32(&ctrl.b_ready), 1);
    ctrl.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    tmem_alloc<PAIR>(smem_u32(&ctrl.tmem_base), p.tmem_cols);
    tmem_relinquish<PAIR>();
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();      // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = ctrl.tmem_base;
  // Everything above touched only this block's shared and tensor memory.  From here on global memory
  // is read (operands) and written (outputs, counters): wait for the previous kernel of the stream.
  pdl_wait();
  pdl_launch_dependents();

  if (warp < kProducerWarps) {
    // ------------------------------------------------------------------ TMA producers
    // Operand planes are numbered A planes first, then B planes.  Every producer warp walks the same
    // sequence of stages and issues only the copies of its own planes (warp w takes planes w and
    // w + 3), so the copies of a stage are in flight side by side.
    constexpr int NPLANES = NAX + NBW;
    // (whole warp in uniform control flow; one elected lane issues the copies)
    // Planes that are streamed through the ring: all of them, or only the activation planes when
    // the weights are resident.  With fewer streamed planes than producer warps, several warps
    // share a plane and take turns stage by stage.
    const bool b_res = GROUPED && p.b_resident;
    const int nact = b_res ? NAX : NPLANES;
    const int kps = GROUPED ? p.kps : 1;
    const int nsub = nact >= kProducerWarps ? 1 : kProducerWarps / nact;   // warps per streamed plane
    const int act_plane = nact >= kProducerWarps ? warp : warp % nact;
    const int sub = nact >= kProducerWarps ? 0 : warp / nact;
    const bool two_planes = act_plane + kProducerWarps < nact;             // this warp also owns a second plane
    {
      const bool is_a = act_plane < NAX;
      const int plane = is_a ? act_plane : act_plane - NAX;
      const CUtensorMap* my_map = is_a ? (plane == 0 ? &map_a0 : &map_a1) : (plane == 0 ? &map_b0 : &map_b1);
      const uint32_t my_off = is_a ? (uint32_t)plane * p.a_bytes : NAX * p.a_bytes + (uint32_t)plane * p.b_bytes;
      // the second plane, if any, is the last B plane (plane index 3 of 4)
      const CUtensorMap* my_map2 = &map_b1;
      const uint32_t my_off2 = NAX * p.a_bytes + (uint32_t)(NBW - 1) * p.b_bytes;
      uint32_t it = 0, ph = 0;
      int s = 0;
      bool ok = true;
      if (b_res && warp == kProducerWarps - 1) {
        // the whole weight matrix of this (single) column tile, one copy per k-block and plane,
        // all reporting to one barrier
        // (in a pair each CTA fetches its own half of the weight rows; the bytes of both are counted
        // on the leader's barrier, which the leader arms for both)
        if (elect_one()) {
          uint32_t bar = smem_u32(&ctrl.b_ready);
          if (rank == 0) mbar_expect_tx(bar, (PAIR ? 2u : 1u) * (uint32_t)p.num_kb * NBW * p.b_bytes);
          if (PAIR) bar = mapa_rank(bar, 0);
          for (int kb = 0; kb < p.num_kb; ++kb) {
            const int kcol = p.is_conv ? (kb / p.cblks) * p.w_pitch + (kb % p.cblks) * p.BK : kb * p.BK;
            for (int bplane = 0; bplane < NBW; ++bplane) {
              const uint32_t dst =
                  ring + p.b_res_off + (uint32_t)kb * (NBW * p.b_bytes) + (uint32_t)bplane * p.b_bytes;
              tma_load_2d<PAIR>(dst, bplane == 0 ? &map_b0 : &map_b1, bar, kcol, (int)rank * b_rows);
            }
          }
        }
        __syncwarp();
      }
      const bool in_tile_loop = sub < nsub;
      bool stalled = false;
      for (int t = worker; t < p.total_tiles && ok && in_tile_loop && !stalled; t += workers) {
        const TileCoord tc = decode_tile(t, p);
        const int m_begin = tc.m0 + (int)rank * kBM;        // first of the 128 rows this CTA stages
        const int n_begin = tc.n0 + (int)rank * b_rows;     // first weight row this CTA stages
        int img = 0, base_h = 0, base_w = 0;
        int tap = 0, cb = 0, r = 0, sx = 0;       // position of kb in the (tap, channel block) order
        if (lane == 0 && warp == 0) TL_STAMP(0, (uint32_t)((t - worker) / workers), 0);
        if (p.is_conv) {
          const int ow = m_begin % p.OW;
          const int rest = m_begin / p.OW;
          const int oh = rest % p.OH;
          img = rest / p.OH;
          base_w = ow * p.stride_w - p.pad_w;
          base_h = oh * p.stride_h - p.pad_h;
          tap = tc.kb_begin / p.cblks;
          cb = tc.kb_begin - tap * p.cblks;
          r = tap / p.S;
          sx = tap - r * p.S;
        }
        for (int kb = tc.kb_begin; kb < tc.kb_end; kb += kps, ++it) {
          if (it == (uint32_t)p.stall_at) { stalled = true; break; }
          const int nkb = GROUPED ? min(kps, tc.kb_end - kb) : 1;      // k-blocks in this stage
          const bool my_turn = (s % nsub) == sub;     // ring slots have fixed owners
          uint32_t full = 0, dst = 0;
          if (my_turn) {                                  // this warp's turn for its plane
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&ctrl.empty[s]), ph ^ 1u, &ctrl, p));
            if (!ok) break;
            // bytes are reported to the leader's barrier; the leader arms it for both CTAs' copies
            full = smem_u32(&ctrl.full[s]);
            if (PAIR) full = mapa_rank(full, 0);
            dst = ring + (uint32_t)s * p.stage_bytes;
            if (act_plane == 0 && rank == 0 && elect_one())
              mbar_expect_tx(smem_u32(&ctrl.full[s]), (PAIR ? 2u : 1u) * (uint32_t)nkb * p.kb_bytes);
          }
          for (int j = 0; j < nkb; ++j) {
            if (my_turn && elect_one()) {
              if (p.is_conv) {
                if (is_a)
                  tma_load_im2col<PAIR>(dst + my_off, my_map, full, cb * p.BK, base_w, base_h, img, (uint16_t)sx,
                                        (uint16_t)r);
                else
                  tma_load_2d<PAIR>(dst + my_off, my_map, full, tap * p.w_pitch + cb * p.BK, n_begin);
                if (two_planes)
                  tma_load_2d<PAIR>(dst + my_off2, my_map2, full, tap * p.w_pitch + cb * p.BK, n_begin);
              } else {
                tma_load_2d<PAIR>(dst + my_off, my_map, full, (kb + j) * p.BK, is_a ? m_begin : n_begin);
                if (two_planes) tma_load_2d<PAIR>(dst + my_off2, my_map2, full, (kb + j) * p.BK, n_begin);
              }
            }
            dst += p.kb_bytes;
            if (p.is_conv) {
              if (++cb == p.cblks) {
                cb = 0;
                ++tap;
                if (++sx == p.S) { sx = 0; ++r; }
              }
            }
          }
          if (++s == p.stages) { s = 0; ph ^= 1u; }
        }
      }
      const bool is_b_loader = b_res && warp == kProducerWarps - 1;
      if (ctrl.abort && lane == 0 && is_b_loader) {
        // another role gave up: let the resident-weight copies land before the CTA exits (the
        // follower of a pair cannot see the leader's barrier: it waits a fixed time)
        const unsigned long long t0 = global_ns();
        if (PAIR && rank != 0) {
          while (global_ns() - t0 < 2000000ull) {
          }
        } else {
          while (!mbar_try_wait(smem_u32(&ctrl.b_ready), 0) && global_ns() - t0 < 50000000ull) {
          }
        }
      }
      if ((!ok || ctrl.abort) && lane == 0) {
        // gave up: let the copies already issued land before the CTA releases its shared memory.
        // (In a pair the bytes are counted on the leader's barriers, so the follower just waits.)
        const uint32_t n = it < (uint32_t)p.stages ? it : (uint32_t)p.stages;
        for (uint32_t j = it - n; j < it; ++j) {
          const int sj = (int)(j % (uint32_t)p.stages);
          const uint32_t pj = (j / (uint32_t)p.stages) & 1u;
          const unsigned long long t0 = global_ns();
          if (PAIR && rank != 0) {
            while (global_ns() - t0 < 2000000ull) {
            }
            break;
          }
          while (!mbar_try_wait(smem_u32(&ctrl.full[sj]), pj) && global_ns() - t0 < 50000000ull) {
          }
        }
      }
    }
    __syncwarp();
  } else if (warp < kFirstEpiWarp) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    // The warp walks the stages in uniform control flow; one elected lane issues.
    if (rank == 0) {
      const int tile_rows = PAIR ? 2 * kBM : kBM;
      const uint32_t id_ss = make_idesc(true, true, p.BN, tile_rows);
      const uint32_t id_su = make_idesc(true, false, p.BN, tile_rows);
      const uint32_t id_us = make_idesc(false, true, p.BN, tile_rows);
      const uint32_t id_uu = make_idesc(false, false, p.BN, tile_rows);
      const uint32_t dhi = smem_desc_hi(p.sbo, p.layout_type);
      const uint32_t ring_lo = smem_desc_lo(ring);
      const uint32_t stage_u = p.stage_bytes >> 4, a_u = p.a_bytes >> 4, b_u = p.b_bytes >> 4;
      const uint32_t kb_u = p.kb_bytes >> 4;
      const uint32_t off_a1 = a_u, off_b0 = NAX * a_u;
      const int ksteps = p.ksteps;
      const uint32_t full_bar0 = smem_u32(&ctrl.full[0]), empty_bar0 = smem_u32(&ctrl.empty[0]);
      uint32_t tile_iter = 0, ph = 0;
      uint32_t a0 = ring_lo, full_bar = full_bar0, empty_bar = empty_bar0;
      int s = 0;
      bool ok = true;
      const bool b_res = GROUPED && p.b_resident;
      const int kps = GROUPED ? p.kps : 1;
      const uint32_t bres_lo = smem_desc_lo(ring + p.b_res_off), bres_u = NBW * b_u;
      if (b_res) {
        ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&ctrl.b_ready), 0u, &ctrl, p, false));
        tc_fence_after();
      }
      for (int t = worker; t < p.total_tiles && ok; t += workers, ++tile_iter) {
        const TileCoord tc = decode_tile(t, p);
        const uint32_t buf = tile_iter % (uint32_t)p.acc_bufs;
        const uint32_t bph = (tile_iter / (uint32_t)p.acc_bufs) & 1u;
        if (lane == 0) TL_STAMP(1, tile_iter, 0);
        ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&ctrl.tmem_empty[buf]), bph ^ 1u, &ctrl, p, false));
        // split release: barrier 0 above covers the middle and low accumulators, barriers 1 and 2
        // the two places of the high one
        const uint32_t hh_sel = (NACC == 3 && p.split_hh) ? (tile_iter & 1u) : 0u;
        if (ok && NACC == 3 && p.split_hh)
          ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&ctrl.tmem_empty[1u + hh_sel]), ((tile_iter >> 1) & 1u) ^ 1u,
                                                &ctrl, p, false));
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) TL_STAMP(1, tile_iter, 1);
        // accumulator columns of this tile: the set's three (or fewer) consecutive groups of BN
        // columns, except that with the split release the first (high) one may sit in the last quarter
        const uint32_t dset = tmem_base + buf * (uint32_t)(NACC * p.BN);
        const uint32_t d0 = dset + hh_sel * (uint32_t)(3 * p.BN);
        const uint32_t d1 = dset + (uint32_t)p.BN, d2 = dset + 2u * (uint32_t)p.BN;
        uint32_t bres = bres_lo + (uint32_t)tc.kb_begin * bres_u;   // resident weights of this k-block
        const bool stagger = !GROUPED && NAX == 2 && NBW == 2 && p.tail_stagger != 0;
        const int kb_main_end = stagger ? tc.kb_end - 2 : tc.kb_end;
        for (int kb = tc.kb_begin; kb < kb_main_end; kb += kps) {
          const int nkb = GROUPED ? min(kps, tc.kb_end - kb) : 1;
          {
#ifdef ADAPTION_TIMELINE
          const long long tw0 = clock64();
#endif
          ok = __all_sync(0xffffffffu, wait_bar(full_bar, ph, &ctrl, p, false));
#ifdef ADAPTION_TIMELINE
          if (lane == 0 && blockIdx.x == 0 && tile_iter < 32u)
            g_timeline[(1 * 32 + tile_iter) * 8 + 3] += clock64() - tw0;   // time waiting for data
#endif
          if (!ok) break;
          tc_fence_after();
          const uint32_t acc = kb == tc.kb_begin ? 0u : 1u;
          if (elect_one()) {
            // a0 / ak: low descriptor word of the first A plane of a k-block; the other planes and
            // the k-steps are fixed offsets (16-byte units) from it (weights: in the stage or
            // resident).  The first k-block is straight-line code; grouped stages loop over the rest.
            {
              const uint32_t b0 = b_res ? bres : a0 + off_b0;
              mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, a0, a0 + off_a1, b0, b0 + b_u, dhi, id_ss, id_su, id_us,
                                        id_uu, acc);
              if (ksteps > 1)
                mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, a0 + 2u, a0 + off_a1 + 2u, b0 + 2u, b0 + b_u + 2u, dhi,
                                          id_ss, id_su, id_us, id_uu, 1u);
              if (ksteps > 2) {
                mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, a0 + 4u, a0 + off_a1 + 4u, b0 + 4u, b0 + b_u + 4u, dhi,
                                          id_ss, id_su, id_us, id_uu, 1u);
                mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, a0 + 6u, a0 + off_a1 + 6u, b0 + 6u, b0 + b_u + 6u, dhi,
                                          id_ss, id_su, id_us, id_uu, 1u);
              }
            }
            if (GROUPED && nkb > 1) {
              uint32_t ak = a0 + kb_u, bk = bres + bres_u;
              for (int j = 1; j < nkb; ++j, ak += kb_u, bk += bres_u) {
                const uint32_t b0 = b_res ? bk : ak + off_b0;
                mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, ak, ak + off_a1, b0, b0 + b_u, dhi, id_ss, id_su, id_us,
                                          id_uu, 1u);
                if (ksteps > 1)
                  mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, ak + 2u, ak + off_a1 + 2u, b0 + 2u, b0 + b_u + 2u, dhi,
                                            id_ss, id_su, id_us, id_uu, 1u);
                if (ksteps > 2) {
                  mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, ak + 4u, ak + off_a1 + 4u, b0 + 4u, b0 + b_u + 4u, dhi,
                                            id_ss, id_su, id_us, id_uu, 1u);
                  mma_kstep<NAX, NBW, PAIR>(d0, d1, d2, ak + 6u, ak + off_a1 + 6u, b0 + 6u, b0 + b_u + 6u, dhi,
                                            id_ss, id_su, id_us, id_uu, 1u);
                }
              }
            }
            tc_commit<PAIR>(empty_bar);                        // stage reusable once these MMAs retire
          }
          }
          if (GROUPED) bres += (uint32_t)nkb * bres_u;
          a0 += stage_u;
          full_bar += 8u;
          empty_bar += 8u;
          if (++s == p.stages) {
            s = 0;
            ph ^= 1u;
            a0 = ring_lo;
            full_bar = full_bar0;
            empty_bar = empty_bar0;
          }
        }
        if (ok && stagger) {
          // The two last k-blocks together, product by product.  (Integer accumulation: the order of
          // the MMAs does not matter.)  Both stages are handed back at the end.
          uint32_t st_a[2], st_full[2], st_empty[2], st_ph[2];
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            st_a[j] = a0; st_full[j] = full_bar; st_empty[j] = empty_bar; st_ph[j] = ph;
            a0 += stage_u;
            full_bar += 8u;
            empty_bar += 8u;
            if (++s == p.stages) {
              s = 0;
              ph ^= 1u;
              a0 = ring_lo;
              full_bar = full_bar0;
              empty_bar = empty_bar0;
            }
          }
          ok = __all_sync(0xffffffffu, wait_bar(st_full[0], st_ph[0], &ctrl, p, false));
          if (ok) ok = __all_sync(0xffffffffu, wait_bar(st_full[1], st_ph[1], &ctrl, p, false));
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {
            const uint32_t off_b1 = off_b0 + b_u;
#pragma unroll
            for (int j = 0; j < 2; ++j)
              for (int ks = 0; ks < ksteps; ++ks)                     // lo * lo
                mma_i8<PAIR>(d2, st_a[j] + off_a1 + 2u * ks, st_a[j] + off_b1 + 2u * ks, dhi, id_uu, 1u);
            tc_commit<PAIR>(smem_u32(&ctrl.part_full[0]));
#pragma unroll
            for (int j = 0; j < 2; ++j)
              for (int ks = 0; ks < ksteps; ++ks) {                   // hi * lo and lo * hi
                mma_i8<PAIR>(d1, st_a[j] + 2u * ks, st_a[j] + off_b1 + 2u * ks, dhi, id_su, 1u);
                mma_i8<PAIR>(d1, st_a[j] + off_a1 + 2u * ks, st_a[j] + off_b0 + 2u * ks, dhi, id_us, 1u);
              }
            tc_commit<PAIR>(smem_u32(&ctrl.part_full[1]));
#pragma unroll
            for (int j = 0; j < 2; ++j)
              for (int ks = 0; ks < ksteps; ++ks)                     // hi * hi
                mma_i8<PAIR>(d0, st_a[j] + 2u * ks, st_a[j] + off_b0 + 2u * ks, dhi, id_ss, 1u);
            tc_commit<PAIR>(st_empty[0]);
            tc_commit<PAIR>(st_empty[1]);
          }
        }
        if (ok && elect_one()) tc_commit<PAIR>(smem_u32(&ctrl.tmem_full[buf]));   // tile complete
        __syncwarp();
        if (lane == 0) TL_STAMP(1, tile_iter, 2);
      }
      if ((!ok || ctrl.abort) && lane == 0) {
        // make sure no MMA still reads shared memory or writes TMEM when the CTAs tear down
        tc_commit<PAIR>(smem_u32(&ctrl.drain));
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&ctrl.drain), 0) && global_ns() - t0 < 50000000ull) {
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;          // TMEM lanes 32*quarter .. 32*quarter+31
    // With two accumulator sets and narrow tiles the warps form two groups that take alternate
    // tiles (and accumulator sets), so that one group's TMEM loads overlap the other's arithmetic;
    // each group has its own barriers, constants and staging planes.
    const int groups = p.epi_groups;
    const int gwarps = kEpiWarps / groups, gthreads = 32 * gwarps;
    const int group = (warp - kFirstEpiWarp) / gwarps;
    const int ew = (warp - kFirstEpiWarp) - group * gwarps;      // warp index within its group
    // the warps of a lane quarter split the columns of the tile
    const int cols_per_warp = max(16, p.BN / (gwarps / 4));
    const int col_begin = min(p.BN, (ew >> 2) * cols_per_warp);
    const int col_end = min(p.BN, col_begin + cols_per_warp);
    const int row = quarter * 32 + lane;   // row of the tile (and of this CTA's staging planes)
    const int planes_bytes = kBM * p.BN * p.rq.out_planes;
    const uint32_t stage_group = ring + p.stage_off + (uint32_t)(group * planes_bytes * p.stage_bufs);
    uint32_t stage_lo = stage_group;
    uint32_t stage_hi = stage_lo + (uint32_t)(kBM * p.BN);
    uint32_t stage_turn = 0;
    // per-column epilogue constants of the current tile, one array per group, behind the staging planes
    long long* colconst = reinterpret_cast<long long*>(smem_raw + (ring - smem_u32(smem_raw)) + p.const_off) +
                          group * p.BN;
    const bool store_leader = ew == 0 && lane == 0;
    uint32_t tile_iter = (uint32_t)group;
    Counts cnt;
    long long vmax = 0;
    bool ok = true;
    int const_n0 = -1;          // first column of the tile whose constants are staged
    for (int t = worker + group * workers; t < p.total_tiles; t += groups * workers, tile_iter += (uint32_t)groups) {
      const TileCoord tc = decode_tile(t, p);
      const uint32_t buf = tile_iter % (uint32_t)p.acc_bufs;
      const uint32_t bph = (tile_iter / (uint32_t)p.acc_bufs) & 1u;
      // per-column constants of this tile (the last barrier of the previous tile separates these
      // writes from its readers): bias aligned to the accumulator, plus the rounding half on the
      // fast path.  Kept when the tile covers the same columns as the previous one.
      if (tc.n0 != const_n0) {
        for (int c = 32 * ew + lane; c < p.BN; c += gthreads) {
          const int n = tc.n0 + c;
          long long b = 0;
          if (p.bias != nullptr && n < p.N && p.splits == 1) b = (long long)p.bias[n] * (1ll << p.bias_shift);
          if (FAST) {
            // two arrays of BN 32-bit words: C mod 2^16 and C div 2^16 (a single accumulator takes all
            // of C from the first), read four columns per load
            const long long C = b + (p.rq.shift > 0 ? 1ll << (p.rq.shift - 1) : 0ll);
            int* cw = reinterpret_cast<int*>(colconst);
            cw[c] = NACC == 1 ? (int)C : (int)(C & 0xffff);
            cw[p.BN + c] = (int)(C >> 16);
          } else {
            colconst[c] = b;
          }
        }
        const_n0 = tc.n0;
      }
      // the previous tile's bulk stores must have read the staging planes before they are reused
      // (with two buffers in turn: the store from two tiles ago)
      if (p.stage_bufs == 2) {
        stage_lo = stage_group + stage_turn * (uint32_t)planes_bytes;
        stage_hi = stage_lo + (uint32_t)(kBM * p.BN);
        stage_turn ^= 1u;
        if (p.staged && store_leader) bulk_wait_read_all_but_one();
      } else if (p.staged && store_leader) {
        bulk_wait_read_all();
      }
      if (lane == 0 && (ew & 3) == 0) TL_STAMP(2 + (ew >> 2), tile_iter, 0);
      // (staggered tail: the first thing to wait for is the low accumulator)
      const bool stagger = FAST && NACC == 3 && p.tail_stagger != 0;
      bool w = wait_bar(smem_u32(stagger ? &ctrl.part_full[0] : &ctrl.tmem_full[buf]), bph, &ctrl, p);
      // one decision for all epilogue warps (they meet at barriers below), which also publishes the
      // constants and the free staging planes
      w = epi_bar_all(group, gthreads, w);
      if (lane == 0 && (ew & 3) == 0) TL_STAMP(2 + (ew >> 2), tile_iter, 1);
      if (!w) { ok = false; break; }
      tc_fence_after();
      const int m = tc.m0 + (int)rank * kBM + row;
      const bool row_ok = m < p.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * (uint32_t)(NACC * p.BN);
      // where this tile's high accumulator lives, and the barrier that hands it back
      const bool split = NACC == 3 && p.split_hh != 0;
      const uint32_t hh_sel = split ? (tile_iter & 1u) : 0u;
      const uint32_t hh_off = hh_sel * (uint32_t)(3 * p.BN);
      unsigned long long* const bar_rest = &ctrl.tmem_empty[buf];
      unsigned long long* const bar_hh = split ? &ctrl.tmem_empty[1u + hh_sel] : bar_rest;
      // Sixteen columns per step.  The accumulators are handed back to the issuing warp as soon as
      // the last step's values are in registers, before the arithmetic on them.
      const bool storing = FAST || (p.splits == 1 && p.mode == ADAPTION_MODE_REQUANT);
      bool released = false;
      bool tile_ok = true;        // a later wait of this tile gave up: finish the tile, then leave together
      // Fast path with thirty-two columns per warp step: one TMEM load per accumulator, the low and
      // middle accumulators first (they fold into T), the high one last; the accumulators go back
      // to the issuing warp as soon as the last load has landed.
      // (the host launches the FAST kernels only where every warp owns a multiple of 32 columns)
      if (FAST) {
        if (col_begin >= col_end) {          // a warp without columns only hands the accumulators back
          release_accumulators<PAIR>(bar_rest, lane);
          if (split) release_accumulators<PAIR>(bar_hh, lane);
          released = true;
        }
        for (int c0 = col_begin; c0 < col_end; c0 += 32) {
          int32_t t[32], h[32];
          const int4* cl4 = reinterpret_cast<const int4*>(reinterpret_cast<const int*>(colconst) + c0);
          const int4* ch4 = reinterpret_cast<const int4*>(reinterpret_cast<const int*>(colconst) + p.BN + c0);
          if (NACC == 3) {
            tmem_ld32(taddr + (uint32_t)(c0 + 2 * p.BN), t);       // ll
            if (!stagger) tmem_ld32(taddr + (uint32_t)(c0 + p.BN), h);   // mid
          } else if (NACC == 2) {
            tmem_ld32(taddr + (uint32_t)(c0 + p.BN), t);           // weight 1
            tmem_ld32(taddr + (uint32_t)c0, h);                    // weight 2^8
          } else {
            tmem_ld32(taddr + (uint32_t)c0, t);
          }
          tmem_ld_wait();
          pin_after_wait32(t);
          if (NACC >= 2 && !stagger) pin_after_wait32(h);
          if (NACC == 3 && stagger) {
            // fold the constant into the low accumulator while the middle one completes, then fetch it
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int4 c = cl4[j];
              t[4 * j + 0] = (t[4 * j + 0] + c.x) >> 8;
              t[4 * j + 1] = (t[4 * j + 1] + c.y) >> 8;
              t[4 * j + 2] = (t[4 * j + 2] + c.z) >> 8;
              t[4 * j + 3] = (t[4 * j + 3] + c.w) >> 8;
            }
            tile_ok = wait_bar_inline(smem_u32(&ctrl.part_full[1]), bph, &ctrl, p) && tile_ok;
            tc_fence_after();
            tmem_ld32(taddr + (uint32_t)(c0 + p.BN), h);           // mid
            tmem_ld_wait();
            pin_after_wait32(h);
#pragma unroll
            for (int j = 0; j < 32; ++j) t[j] += h[j];             // T
          }
          // the low and middle accumulators are in registers: with the split release they go back now
          if (split && c0 + 32 >= col_end) {
            release_accumulators<PAIR>(bar_rest, lane);
            if (lane == 0 && (ew & 3) == 0) TL_STAMP(2 + (ew >> 2), tile_iter, 3);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (NACC == 3 && stagger) break;
            const int4 c = cl4[j];
            if (NACC >= 2) {                                       // T = mid + floor((ll + Cl) / 2^8)
              t[4 * j + 0] = h[4 * j + 0] + ((t[4 * j + 0] + c.x) >> 8);
              t[4 * j + 1] = h[4 * j + 1] + ((t[4 * j + 1] + c.y) >> 8);
              t[4 * j + 2] = h[4 * j + 2] + ((t[4 * j + 2] + c.z) >> 8);
              t[4 * j + 3] = h[4 * j + 3] + ((t[4 * j + 3] + c.w) >> 8);
            } else {
              t[4 * j + 0] += c.x; t[4 * j + 1] += c.y; t[4 * j + 2] += c.z; t[4 * j + 3] += c.w;
            }
          }
          if (NACC == 3) {
            if (stagger) {
              tile_ok = wait_bar_inline(smem_u32(&ctrl.tmem_full[buf]), bph, &ctrl, p) && tile_ok;
              tc_fence_after();
            }
            tmem_ld32(taddr + hh_off + (uint32_t)c0, h);           // hh
            tmem_ld_wait();
            pin_after_wait32(h);
          }
          if (c0 + 32 >= col_end) {
            release_accumulators<PAIR>(bar_hh, lane);
            if (lane == 0 && (ew & 3) == 0) TL_STAMP(2 + (ew >> 2), tile_iter, 4);
            released = true;
          }
          if (NACC >= 2) {                                         // H = hh + Ch
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int4 c = ch4[j];
              if (NACC == 3) {
                h[4 * j + 0] += c.x; h[4 * j + 1] += c.y; h[4 * j + 2] += c.z; h[4 * j + 3] += c.w;
              } else {
                h[4 * j + 0] = c.x; h[4 * j + 1] = c.y; h[4 * j + 2] = c.z; h[4 * j + 3] = c.w;
              }
            }
          }
          const int col = tc.n0 + c0;
          const bool wide = NACC == 1 || p.rq.shift >= 16;
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t wq[8];
            if (wide)
              fast_outputs16<NACC, true>(t, h, half, p.rq.shift, p.rq.qmax, row_ok, col, p.N, cnt, wq);
            else
              fast_outputs16<NACC, false>(t, h, half, p.rq.shift, p.rq.qmax, row_ok, col, p.N, cnt, wq);
            const int chunk = (c0 >> 4) + half;
            if (p.staged && p.pool_w) {
#pragma unroll
              for (int j = 0; j < 8; ++j) wq[j] = max_s16x2(wq[j], __shfl_xor_sync(0xffffffffu, wq[j], 1));
              if ((lane & 1) == 0) {
                const uint32_t off = staged_offset(row >> 1, chunk, p.BN);
                st_shared_v4(stage_lo + off, plane_lo(wq));
                if (p.rq.out_planes == 2) st_shared_v4(stage_hi + off, plane_hi(wq));
              }
            } else if (p.staged) {
              const uint32_t off = staged_offset(row, chunk, p.BN);
              st_shared_v4(stage_lo + off, plane_lo(wq));
              if (p.rq.out_planes == 2) st_shared_v4(stage_hi + off, plane_hi(wq));
            } else {
              store16_global(wq, p, row_ok, m, col + 16 * half);
            }
          }
        }
      }
      for (int c0 = col_begin; !FAST && (c0 < col_end || !released); c0 += 16) {
        const bool have = c0 < col_end;
        Acc8<NACC> xa, xb;
        if (have) {
          load_acc16<NACC>(taddr + c0, hh_off, p.BN, xa, xb);
          tmem_ld_wait();
          pin_acc8<NACC>(xa);
          pin_acc8<NACC>(xb);
        }
        if (c0 + 16 >= col_end) {
          release_accumulators<PAIR>(bar_rest, lane);
          if (split) release_accumulators<PAIR>(bar_hh, lane);
          released = true;
        }
        if (!have) break;
        const int col = tc.n0 + c0;
        const long long* bcol = colconst + c0;
        if (!storing) {
          partial_or_range8<NACC>(xa, bcol, p, row_ok, m, col, vmax);
          partial_or_range8<NACC>(xb, bcol + 8, p, row_ok, m, col + 8, vmax);
        } else {
          uint32_t wq[8];
          if (p.rq.relu) {
            requant8<NACC, true, STOCH>(xa, bcol, p, row_ok, m, col, cnt, wq);
            requant8<NACC, true, STOCH>(xb, bcol + 8, p, row_ok, m, col + 8, cnt, wq + 4);
          } else {
            requant8<NACC, false, STOCH>(xa, bcol, p, row_ok, m, col, cnt, wq);
            requant8<NACC, false, STOCH>(xb, bcol + 8, p, row_ok, m, col + 8, cnt, wq + 4);
          }
          if (p.staged && p.pool_w) {
            // Horizontal half of a 2x2 max-pool: rows 2j and 2j+1 of the tile are neighbouring
            // pixels of one image row (even width, tiles start at even rows) and sit in neighbouring
            // lanes; the maximum of the packed 16-bit values is stored once, as row j.
#pragma unroll
            for (int j = 0; j < 8; ++j) wq[j] = max_s16x2(wq[j], __shfl_xor_sync(0xffffffffu, wq[j], 1));
            if ((lane & 1) == 0) {
              const uint32_t off = staged_offset(row >> 1, c0 >> 4, p.BN);
              st_shared_v4(stage_lo + off, plane_lo(wq));
              if (p.rq.out_planes == 2) st_shared_v4(stage_hi + off, plane_hi(wq));
            }
          } else if (p.staged) {
            const uint32_t off = staged_offset(row, c0 >> 4, p.BN);
            st_shared_v4(stage_lo + off, plane_lo(wq));
            if (p.rq.out_planes == 2) st_shared_v4(stage_hi + off, plane_hi(wq));
          } else {
            store16_global(wq, p, row_ok, m, col);
          }
        }
      }
      // staged planes complete -> one bulk-tensor store per plane (rows beyond M and columns beyond
      // the channel pitch are clipped by the tensor map); the barrier also ends this tile's reads
      // of the per-column constants
      if (p.staged) fence_async_shared();
      if (stagger) {
        // the same barrier also carries the verdict on this tile's later waits, so that all warps
        // of the group leave together if one of them gave up
        if (!epi_bar_all(group, gthreads, tile_ok)) { ok = false; break; }
      } else {
        epi_bar_sync(group, gthreads);
      }
      if (p.staged && store_leader) {
        const int m_first = (tc.m0 + (int)rank * kBM) >> (p.pool_w ? 1 : 0);     // row of the stored tensor
        for (int sub = 0; sub * 128 < p.BN; ++sub) {
          const uint32_t so = (uint32_t)sub * (uint32_t)(kBM * 128);
          tma_store_2d(&map_y_lo, stage_lo + so, tc.n0 + sub * 128, m_first);
          if (p.rq.out_planes == 2) tma_store_2d(&map_y_hi, stage_hi + so, tc.n0 + sub * 128, m_first);
        }
        bulk_commit();
      }
      if (lane == 0 && (ew & 3) == 0) TL_STAMP(2 + (ew >> 2), tile_iter, 2);
    }
    (void)ok;
    if (p.staged && store_leader) bulk_wait_all();
    if (p.splits == 1) {
      if (p.mode == ADAPTION_MODE_RANGE)
        flush_max_warp(vmax, p.stats);
      else
        flush_counts_warp(cnt, p.stats);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();      // neither CTA leaves (or frees TMEM) while the other may still signal it
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc<PAIR>(tmem_base, p.tmem_cols);
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
std::once_flag g_encode_once;

// The two tensor-map encoders of the driver, looked up once per process (they are the same for
// every device).
bool load_driver_entry_points() {
  std::call_once(g_encode_once, [] {
    void* f1 = nullptr;
    void* f2 = nullptr;
    cudaDriverEntryPointQueryResult q1, q2;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f1, cudaEnableDefault, &q1) != cudaSuccess ||
        q1 != cudaDriverEntryPointSuccess || f1 == nullptr)
      return;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f2, cudaEnableDefault, &q2) != cudaSuccess ||
        q2 != cudaDriverEntryPointSuccess || f2 == nullptr)
      return;
    g_encode_im2col = reinterpret_cast<EncodeIm2colFn>(f2);
    g_encode_tiled = reinterpret_cast<EncodeTiledFn>(f1);
  });
  return g_encode_tiled != nullptr && g_encode_im2col != nullptr;
}

struct TcConfig {
  bool ok = false;
  int BN = 0, BK = 0;
  CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE;
  uint32_t layout_type = 0;
  int nax = 1, nbw = 1, nacc = 1;
  int stages = 0;
  uint32_t a_bytes = 0, b_bytes = 0, stage_bytes = 0;
  int a_rows = kBM;            // rows of the activation tile that are staged
  int acc_bufs = 1;
  uint32_t tmem_cols = 32;
  int num_kb = 0, splits = 1, kb_per_split = 0;
  int tiles_m = 0, tiles_n = 0;
  int cblks = 1;
  bool b_resident = false;
  uint32_t b_res_bytes = 0;
  int kps = 1;
  uint32_t kb_bytes = 0;
  bool pair = false;           // two CTAs per 256-row tile (cta_group::2)
  int tile_m = kBM;
  int epi_groups = 1;
  bool staged = false;         // outputs staged in shared memory and written by bulk-tensor stores
  uint32_t stage_out_bytes = 0, stage_off = 0, const_bytes = 0;
  int stage_bufs = 1;
  size_t smem_bytes = 0;
  size_t workspace_bytes = 0;
};

// Test and experiment overrides of the tile heuristics, set through adaption_debug_set (never read
// from the environment, so the layer calls themselves do no string work).  Each holds its
// default until set; the setter is the only writer.
enum Knob { kSplits, kPair, kFast, kStaged, kStages, kBK, kBN, kKps, kBres, kWide, kEpiGroups, kTimeoutUs, kStallAt,
            kSplitHh, kPdl, kStagger, kStageBufs, kNumKnobs };
const char* const kKnobNames[kNumKnobs] = {"splits", "pair", "fast", "staged", "stages", "bk", "bn", "kps", "bres",
                                           "wide", "epigroups", "timeout_us", "stall_at", "split_hh", "pdl", "stagger", "stage_bufs"};
const int kKnobDefaults[kNumKnobs] = {0, -1, 1, 1, 0, 0, 0, 0, 1, 1, 2, 0, -1, 1, 1, 1, 2};
std::atomic<int> g_knobs[kNumKnobs] = {{0}, {-1}, {1}, {1}, {0}, {0}, {0}, {0}, {1}, {1}, {2}, {0}, {-1}, {1}, {1}, {1}, {2}};
inline int knob(Knob k) { return g_knobs[k].load(std::memory_order_relaxed); }

TcConfig make_config_impl(const GemmProblem& g, bool allow_wide);

// 256-column tiles only exist as CTA pairs: if the wide attempt does not end up paired (the
// reduction gets split, say), the ordinary configuration is taken.
TcConfig make_config(const GemmProblem& g) {
  TcConfig c = make_config_impl(g, true);
  if (c.BN == 256 && !(c.ok && c.pair)) c = make_config_impl(g, false);
  return c;
}

TcConfig make_config_impl(const GemmProblem& g, bool allow_wide) {
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
    const int forced_bk = knob(kBK);   // experiment knob: narrower K-blocks
    if ((forced_bk == 32 || forced_bk == 64) && forced_bk < c.BK) c.BK = forced_bk;
    c.num_kb = (int)((g.K + c.BK - 1) / c.BK);
    k_padded = g.K;
    if (g.K > (int64_t)1 << 30) return c;
  }
  c.swizzle = c.BK == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : (c.BK == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  c.layout_type = c.BK == 128 ? 2u : (c.BK == 64 ? 4u : 6u);
  c.BN = g.N <= 32 ? 32 : (g.N <= 64 ? 64 : 128);
  const int forced_bn = knob(kBN);    // experiment knob: narrower tiles
  if ((forced_bn == 32 || forced_bn == 64) && forced_bn < c.BN) c.BN = forced_bn;
  // Single-pass (8-bit) layers with many output channels take 256-column pair tiles: one int32
  // accumulator per tile leaves room for two sets of 256 columns, and a 256 x 256 tile halves the
  // operand bytes per MMA cycle, which is what limits the int8 rate (see make_config's pair notes).
  const bool wide = allow_wide && c.nacc == 1 && c.BK == 128 && g.N >= 256 && c.num_kb >= 9 && g.M >= 1024 &&
                    (num_sms() % 2) == 0 && forced_bn == 0 && knob(kPair) != 0 &&
                    knob(kWide) != 0;
  if (wide) c.BN = 256;
  c.tiles_m = (int)((g.M + kBM - 1) / kBM);
  c.tiles_n = (int)((g.N + c.BN - 1) / c.BN);
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
  const int forced = knob(kSplits);
  if (forced > 0) splits = forced > splits ? forced : splits;
  if (splits > c.num_kb) splits = c.num_kb;
  if (splits < 1) splits = 1;
  c.kb_per_split = (c.num_kb + splits - 1) / splits;
  c.splits = (c.num_kb + c.kb_per_split - 1) / c.kb_per_split;
  if ((int64_t)c.kb_per_split * c.BK > kMaxKPerAccumulation) return c;
  if ((int64_t)tiles * c.splits > (int64_t)1 << 30) return c;
  c.workspace_bytes = c.splits > 1 ? (size_t)g.M * (size_t)g.N * sizeof(long long) : 0;
  // Large unsplit problems run as CTA pairs: 256-row tiles, each CTA stages its own 128 rows of A
  // and only half of the weight rows, which cuts the bytes (and TMA rows) per MAC by a quarter.
  const int pair_env = knob(kPair);
  // (measured: pairs win from K = 1152 bytes per plane row on; 256 x 64 pair tiles with two
  // accumulator sets were tried for medium reductions and lost to these once the epilogue hands the
  // accumulators back early)
  const bool pair_ok = c.splits == 1 && g.M >= 1024 && (sms % 2) == 0;
  c.pair = pair_ok && c.BN >= 128 && c.BK == 128 && c.num_kb >= 9;
  // 64-channel convolutions with at most 64 output channels (64-byte k-blocks, one 64-column tile):
  // as a pair each CTA stages half of the weight rows and the MMAs find half of their B operand in
  // the peer's shared memory; with one filter row of taps per stage this measured 0.43 ms against
  // 0.53 ms for 64 x 224 x 224 x 64 -> 64 with the weights resident in a single CTA.
  // (16-bit operands only: with one int8 product per k-step the single CTA with resident weights
  // stays ahead, 0.65 ms against 0.79 ms for the same layer at 8 bits and batch 128)
  const bool narrow_pair = pair_ok && g.is_conv && c.nacc == 3 && c.BK == 64 && c.BN == 64 && c.num_kb >= 9 &&
                           c.num_kb % 3 == 0;
  if (narrow_pair) c.pair = true;
  if (pair_env == 0) c.pair = false;
  if (pair_env == 1 && c.splits == 1 && (sms % 2) == 0) c.pair = true;
  if (c.pair) {
    c.tile_m = 2 * kBM;
    c.tiles_m = (int)((g.M + c.tile_m - 1) / c.tile_m);
  }
  // Inner products on a small batch: only the rows that exist are staged (the MMA still covers 128
  // rows; the rest reads whatever follows in the stage and lands in accumulator rows nobody stores).
  // Smaller stages mean a deeper ring, i.e. more weight bytes in flight per SM, which is what bounds
  // these weight-streaming layers.
  c.a_rows = (!g.is_conv && !c.pair && g.M <= 64) ? 64 : kBM;
  c.a_bytes = (uint32_t)(c.a_rows * c.BK);
  c.b_bytes = (uint32_t)((c.pair ? c.BN / 2 : c.BN) * c.BK);
  // Output staging: one plane of 128 rows x BN bytes per output byte plane.  Needs a tensor map over
  // the output planes (pitch a multiple of 16 bytes and at least one tile wide) and no int16 copy.
  const int out_planes = g.y.fmt.n_bits > 8 ? 2 : 1;
  c.staged = g.mode == ADAPTION_MODE_REQUANT && c.splits == 1 && g.y.q16 == nullptr && g.y.lo != nullptr &&
             g.y.c_stride >= c.BN && g.y.c_stride % 16 == 0 && knob(kStaged) != 0;
  // two epilogue groups when two tiles can be in flight in TMEM and their constants fit the halves
  // of the per-column array
  c.epi_groups = (c.acc_bufs >= 2 && c.acc_bufs % 2 == 0 && c.BN <= 64 &&
                  knob(kEpiGroups) == 2) ? 2 : 1;
  c.stage_out_bytes = c.staged ? (uint32_t)(kBM * c.BN * out_planes * c.epi_groups) : 0u;
  // dynamic shared memory: everything up to the per-block limit except the control block
  c.const_bytes = (uint32_t)(c.BN * c.epi_groups * sizeof(long long));
  const size_t budget = 232448 - sizeof(Ctrl) - 256 - c.stage_out_bytes - c.const_bytes;
  // group short k-blocks so that a stage carries roughly 768 tensor-pipe cycles of work or more
  {
    const int products = c.nax * c.nbw;
    const int cyc_per_kb = (c.BK / 32) * products * (c.BN >= 128 ? c.BN / 2 : 48);
    int kps = (768 + cyc_per_kb - 1) / cyc_per_kb;
    if (kps > 4) kps = 4;
    const int kps_env = knob(kKps);
    if (narrow_pair && c.pair) kps = 3;
    if (kps_env >= 1 && kps_env <= 4) kps = kps_env;
    if (kps > c.kb_per_split) kps = c.kb_per_split;
    if (kps < 1) kps = 1;
    c.kps = kps;
  }
  c.kb_bytes = c.nax * c.a_bytes + c.nbw * c.b_bytes;
  // One column tile and a short reduction: keep every weight k-block resident in shared memory and
  // stream only the activation planes (fewer bulk copies per k-block for the 64-channel and
  // 3-channel layers).  Only if at least three activation stages still fit.
  const size_t res_bytes = (size_t)c.num_kb * c.nbw * c.b_bytes;
  if (c.tiles_n == 1 && c.splits == 1 && c.tiles_m >= 4 * sms && (!c.pair || knob(kBres) != 2) &&
      res_bytes + 3 * (size_t)c.kps * c.nax * c.a_bytes + 1024 <= budget && knob(kBres) != 0) {
    c.b_resident = true;
    c.b_res_bytes = (uint32_t)res_bytes;
    c.kb_bytes = c.nax * c.a_bytes;
  }
  c.stage_bytes = (uint32_t)c.kps * c.kb_bytes;
  c.stages = (int)((budget - 1024 - c.b_res_bytes) / c.stage_bytes);
  if (c.staged && c.stages < 3) {
    // not enough room for a useful ring beside the staging planes: store directly instead
    c.stages = (int)((budget + c.stage_out_bytes - 1024 - c.b_res_bytes) / c.stage_bytes);
    c.staged = false;
    c.stage_out_bytes = 0;
    c.stage_bufs = 1;
  }
  if (c.stages > kMaxStages) c.stages = kMaxStages;
  // Narrow tiles with two epilogue groups: a second staging buffer per group, so that a group does
  // not wait for its previous tile's bulk store to have read shared memory - where the ring keeps at
  // least four stages beside it (short reductions with small stages, e.g. a packed first layer).
  if (c.staged && c.epi_groups == 2 && c.BN <= 64 && knob(kStageBufs) != 1) {
    const size_t extra = c.stage_out_bytes;
    const size_t used = (size_t)c.stages * c.stage_bytes + c.b_res_bytes + 1024;
    size_t slack = budget > used ? budget - used : 0;
    int stages = c.stages;
    while (slack < extra && stages > 4) {
      --stages;
      slack += c.stage_bytes;
    }
    if (slack >= extra) {
      c.stages = stages;
      c.stage_bufs = 2;
      c.stage_out_bytes = (uint32_t)(2 * extra);
    }
  }
  const int stage_cap = knob(kStages);   // experiment knob: shallower ring
  if (stage_cap >= 2 && stage_cap < c.stages) c.stages = stage_cap;
  if (c.stages < 2) return c;
  c.stage_off = (uint32_t)(((size_t)c.stages * c.stage_bytes + c.b_res_bytes + 1023) & ~(size_t)1023);
  c.smem_bytes = (size_t)c.stage_off + 1024 + c.stage_out_bytes + c.const_bytes;
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

template <int NAX, int NBW, bool PAIR, bool GROUPED, int EPI>
int launch_kernel(const CUtensorMap* maps, const TcParams& p, int grid, size_t smem, cudaStream_t stream) {
  // The dynamic shared-memory limit is a per-device attribute of the kernel: remember, per device
  // ordinal, the largest size it has been raised to (a racing thread at worst sets it once more).
  constexpr int kMaxDevices = 64;
  static std::atomic<size_t> attr_size[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ADAPTION_ERR_CUDA;
  const bool cached = dev >= 0 && dev < kMaxDevices;
  if (!cached || smem > attr_size[dev].load(std::memory_order_acquire)) {
    const cudaError_t ae = cudaFuncSetAttribute(lp_gemm_kernel<NAX, NBW, PAIR, GROUPED, EPI>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (ae != cudaSuccess) return cuda_failure(ae, "lp_gemm_kernel shared-memory attribute");
    if (cached) {
      size_t seen = attr_size[dev].load(std::memory_order_relaxed);
      while (seen < smem && !attr_size[dev].compare_exchange_weak(seen, smem, std::memory_order_release)) {
      }
    }
  }
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  unsigned n_attr = 0;
  if (PAIR) {
    attr[n_attr].id = cudaLaunchAttributeClusterDimension;
    attr[n_attr].val.clusterDim.x = 2;
    attr[n_attr].val.clusterDim.y = 1;
    attr[n_attr].val.clusterDim.z = 1;
    ++n_attr;
  }
  if (knob(kPdl) != 0) {
    // the kernel waits for its predecessor itself (pdl_wait) before it touches global memory
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
  }
  cfg.attrs = n_attr ? attr : nullptr;
  cfg.numAttrs = n_attr;
  const cudaError_t le =
      cudaLaunchKernelEx(&cfg, lp_gemm_kernel<NAX, NBW, PAIR, GROUPED, EPI>, maps[0], maps[1], maps[2], maps[3], maps[4],
                         maps[5], p);
  if (le != cudaSuccess) {
    (void)cudaGetLastError();
    return cuda_failure(le, "lp_gemm_kernel launch");
  }
  return cuda_status(cudaGetLastError(), "after lp_gemm_kernel launch");
}

template <int NAX, int NBW, bool PAIR, bool GROUPED>
int launch_epi(const CUtensorMap* maps, const TcParams& p, int grid, size_t smem, cudaStream_t stream) {
  if (p.fast_relu != 0) return launch_kernel<NAX, NBW, PAIR, GROUPED, kEpiFast>(maps, p, grid, smem, stream);
  if (p.st.enabled != 0) return launch_kernel<NAX, NBW, PAIR, GROUPED, kEpiStochastic>(maps, p, grid, smem, stream);
  return launch_kernel<NAX, NBW, PAIR, GROUPED, kEpiGeneric>(maps, p, grid, smem, stream);
}

template <int NAX, int NBW>
int launch_either(bool pair, const CUtensorMap* maps, const TcParams& p, int grid, size_t smem,
                  cudaStream_t stream) {
  const bool grouped = p.kps > 1 || p.b_resident != 0;
  if (pair)
    return grouped ? launch_epi<NAX, NBW, true, true>(maps, p, grid, smem, stream)
                   : launch_epi<NAX, NBW, true, false>(maps, p, grid, smem, stream);
  return grouped ? launch_epi<NAX, NBW, false, true>(maps, p, grid, smem, stream)
                 : launch_epi<NAX, NBW, false, false>(maps, p, grid, smem, stream);
}


// ---------------------------------------------------------------------------------- peak probe
// Issue-rate probe for the roofline denominator: every SM (or SM pair) runs back-to-back
// tcgen05.mma kind::i8 instructions on operand tiles that stay resident in shared memory (no
// loads), so the time per instruction is the tensor pipe's own.
template <bool PAIR>
__global__ void __launch_bounds__(128, 1)
i8_peak_kernel(int bn, int iters, int commit_every, unsigned long long* out_cycles, int* out_status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ unsigned long long done_bar;
  __shared__ unsigned long long side_bar;      // target of the optional intermediate commits
  __shared__ uint32_t tmem_slot;
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  // A: 128 rows x 128 bytes, B: up to 256 rows x 128 bytes, filled with a fixed byte pattern
  uint32_t* words = reinterpret_cast<uint32_t*>(smem_raw + (ring - smem_u32(smem_raw)));
  for (int i = threadIdx.x; i < (16384 + 32768) / 4; i += blockDim.x) words[i] = 0x9E3779B9u * (uint32_t)(i + 1);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&done_bar), 1);
    mbar_init(smem_u32(&side_bar), (1u << 20) - 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if ((threadIdx.x >> 5) == 0) {
    tmem_alloc<PAIR>(smem_u32(&tmem_slot), 512);
    tmem_relinquish<PAIR>();
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  if (threadIdx.x == 0 && rank == 0) {
    const uint32_t idesc = make_idesc(true, true, bn, PAIR ? 256 : 128);
    const uint32_t dhi = smem_desc_hi(1024, 2);
    const uint32_t a_lo = smem_desc_lo(ring), b_lo = smem_desc_lo(ring + 16384);
    const long long t0 = clock64();
    for (int i = 0; i < iters; ++i) {
#pragma unroll
      for (uint32_t ks = 0; ks < 8; ks += 2) mma_i8<PAIR>(tmem_base, a_lo + ks, b_lo + ks, dhi, idesc, 1u);
      // optional: an intermediate commit every `commit_every` groups of four instructions, as a
      // pipelined mainloop issues when it hands a shared-memory stage back
      if (commit_every > 0 && (i + 1) % commit_every == 0) tc_commit<PAIR>(smem_u32(&side_bar));
    }
    tc_commit<PAIR>(smem_u32(&done_bar));
    const unsigned long long w0 = global_ns();
    bool ok = true;
    while (!mbar_try_wait(smem_u32(&done_bar), 0)) {
      if (global_ns() - w0 > 2000000000ull) { ok = false; break; }
    }
    const long long t1 = clock64();
    if (!ok) atomicExch(out_status, (int)ADAPTION_ERR_TIMEOUT);
    out_cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();
  if ((threadIdx.x >> 5) == 0) {
    tc_fence_after();
    tmem_dealloc<PAIR>(tmem_base, 512);
  }
}

template <bool PAIR>
int launch_peak(int bn, int iters, int commit_every, unsigned long long* d_cycles, int* d_status, int grid,
                cudaStream_t stream) {
  const size_t smem = 16384 + 32768 + 1024;
  if (cudaFuncSetAttribute(i8_peak_kernel<PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return ADAPTION_ERR_CUDA;
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  if (PAIR) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  if (cudaLaunchKernelEx(&cfg, i8_peak_kernel<PAIR>, bn, iters, commit_every, d_cycles, d_status) != cudaSuccess) {
    (void)cudaGetLastError();
    return ADAPTION_ERR_CUDA;
  }
  return ADAPTION_OK;
}

}  // namespace

int probe_i8_peak(int bn, int pair, int iters, int commit_every, unsigned long long* d_cycles, int* d_status,
                  cudaStream_t stream) {
  const int sms = num_sms();
  const int grid = pair ? (sms / 2) * 2 : sms;
  return pair ? launch_peak<true>(bn, iters, commit_every, d_cycles, d_status, grid, stream)
              : launch_peak<false>(bn, iters, commit_every, d_cycles, d_status, grid, stream);
}

namespace {

}  // namespace

#ifdef ADAPTION_TIMELINE
extern "C" __attribute__((visibility("default"))) int adaption_debug_timeline_reset() {
  static long long zeros[8192];
  return cudaMemcpyToSymbol(g_timeline, zeros, sizeof(zeros)) == cudaSuccess ? 0 : 6;
}
extern "C" __attribute__((visibility("default"))) int adaption_debug_timeline(long long* h_out, int n) {
  return cudaMemcpyFromSymbol(h_out, g_timeline, sizeof(long long) * (size_t)n) == cudaSuccess ? 0 : 6;
}
#endif

bool pdl_enabled() { return knob(kPdl) != 0; }

int debug_set(const char* name, int value) {
  if (name == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if (std::strcmp(name, "reset") == 0) {
    for (int k = 0; k < kNumKnobs; ++k) g_knobs[k].store(kKnobDefaults[k], std::memory_order_relaxed);
    return ADAPTION_OK;
  }
  for (int k = 0; k < kNumKnobs; ++k)
    if (std::strcmp(name, kKnobNames[k]) == 0) {
      g_knobs[k].store(value, std::memory_order_relaxed);
      return ADAPTION_OK;
    }
  return ADAPTION_ERR_INVALID_ARG;
}

bool tensor_path_supported(const GemmProblem& g) { return make_config(g).ok; }

// The horizontal half of a 2x2 max-pool can ride on the staged stores of a requantizing layer.
bool tensor_path_can_pool(const GemmProblem& g) {
  const TcConfig c = make_config(g);
  return c.ok && c.staged && g.M % 2 == 0;
}

size_t tensor_path_workspace(const GemmProblem& g) { return make_config(g).workspace_bytes; }

int launch_tensor(const GemmProblem& g) {
  const TcConfig c = make_config(g);
  if (!c.ok) return ADAPTION_ERR_UNSUPPORTED;
  if (!load_driver_entry_points()) return ADAPTION_ERR_CUDA;

  // plane 0 is the high byte plane when there are two, else the single plane
  const void* xa[2] = {c.nax == 2 ? g.x.hi : g.x.lo, g.x.lo};
  const void* wb[2] = {c.nbw == 2 ? g.w.hi : g.w.lo, g.w.lo};
  CUtensorMap maps[6];   // activation planes, weight planes, output planes (hi, lo)
  std::memset(maps, 0, sizeof(maps));
  for (int i = 0; i < 2; ++i) {
    bool ok;
    if (g.is_conv)
      ok = encode_im2col_nhwc(&maps[i], xa[i], g.cs, g.x.c_stride, (uint32_t)c.BK, c.swizzle);
    else
      ok = encode_tiled_2d(&maps[i], xa[i], (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.x.c_stride,
                           (uint32_t)c.BK, (uint32_t)c.a_rows, c.swizzle);
    if (!ok) return ADAPTION_ERR_CUDA;
    const uint64_t wk = g.is_conv ? (uint64_t)g.cs.R * g.cs.S * g.w.c_stride : (uint64_t)g.K;
    const uint64_t wpitch = g.is_conv ? wk : (uint64_t)g.w.c_stride;
    if (!encode_tiled_2d(&maps[2 + i], wb[i], wk, (uint64_t)g.N, wpitch, (uint32_t)c.BK,
                         (uint32_t)(c.pair ? c.BN / 2 : c.BN), c.swizzle))
      return ADAPTION_ERR_CUDA;
  }

  if (c.staged) {
    const int ybox = c.BN < 128 ? c.BN : 128;       // wider tiles leave as several stores of 128 columns
    const CUtensorMapSwizzle yswz = ybox == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                                : (ybox == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    const void* planes[2] = {g.y.hi, g.y.lo};
    for (int i = 0; i < 2; ++i) {
      if (planes[i] == nullptr) continue;      // single-plane outputs have no high plane
      if (!encode_tiled_2d(&maps[4 + i], planes[i], (uint64_t)g.y.c_stride, (uint64_t)(g.pool_w ? g.M / 2 : g.M),
                           (uint64_t)g.y.c_stride, (uint32_t)ybox, (uint32_t)(g.pool_w ? kBM / 2 : kBM), yswz))
        return ADAPTION_ERR_CUDA;
    }
  }

  TcParams p;
  std::memset(&p, 0, sizeof(p));
  p.M = (int)g.M; p.N = (int)g.N; p.tile_m = c.tile_m;
  p.tiles_m = c.tiles_m; p.tiles_n = c.tiles_n; p.splits = c.splits;
  p.total_tiles = c.tiles_m * c.tiles_n * c.splits;
  p.num_kb = c.num_kb; p.kb_per_split = c.kb_per_split;
  p.BN = c.BN; p.BK = c.BK; p.ksteps = c.BK / 32;
  p.sbo = (uint32_t)(8 * c.BK); p.layout_type = c.layout_type;
  p.stages = c.stages; p.a_bytes = c.a_bytes; p.b_bytes = c.b_bytes; p.stage_bytes = c.stage_bytes;
  p.kps = c.kps; p.kb_bytes = c.kb_bytes;
  p.b_resident = c.b_resident ? 1 : 0;
  p.b_res_off = (uint32_t)c.stages * c.stage_bytes;
  p.acc_bufs = c.acc_bufs; p.tmem_cols = c.tmem_cols;
  p.split_hh = (c.nacc == 3 && c.acc_bufs == 1 && 4 * c.BN <= 512 && knob(kSplitHh) != 0) ? 1 : 0;
  if (p.split_hh) p.tmem_cols = 512;
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
  if (g.pool_w && !(c.staged && g.M % 2 == 0)) return ADAPTION_ERR_UNSUPPORTED;
  p.pool_w = g.pool_w ? 1 : 0;
  p.epi_groups = c.epi_groups;
  p.staged = c.staged ? 1 : 0;
  p.stage_bufs = c.stage_bufs;
  p.stage_off = c.stage_off;
  p.const_off = c.stage_off + c.stage_out_bytes;
  const bool single = c.nacc == 1;
  // (its epilogue takes 32 columns per warp step: tiles of 64 columns need the two warp groups,
  // tiles of 32 columns take the generic epilogue)
  const int cols_per_epi_warp = c.BN / (kEpiWarps / c.epi_groups / 4);
  // stochastic rounding happens where the value is requantized: in this kernel's epilogue, or in the
  // finalize kernel when the reduction is split
  p.st = g.stochastic;
  if (g.mode != ADAPTION_MODE_REQUANT || c.splits > 1) p.st.enabled = 0;
  if (g.mode == ADAPTION_MODE_REQUANT && c.splits == 1 && g.relu && !g.stochastic.enabled &&
      p.rq.shift >= (single ? 0 : 9) &&
      p.rq.shift <= 31 && g.N % 8 == 0 && cols_per_epi_warp >= 32 && cols_per_epi_warp % 32 == 0 &&
      knob(kFast) != 0) {
    // 32-bit bounds of the fast epilogue (see fast_result): with a reduction of kred bytes per plane row
    // |hh| <= kred 2^14, |mid| <= kred 65280, |ll| <= kred 65025, and |C| < 2^(15 + bias_shift) + 2^(shift-1)
    const long long kred = (long long)c.num_kb * c.BK;
    const long long cmax = (g.bias != nullptr ? (1ll << (15 + g.bias_shift)) : 0ll) +
                           (p.rq.shift > 0 ? 1ll << (p.rq.shift - 1) : 0ll);
    const long long hmax = kred * 16384 + (cmax >> 16) + 1;
    const long long tmax = kred * 65280 + ((kred * 65025 + 65535) >> 8) + 1;
    const long long lim = 1ll << 31;
    bool ok32 = kred * 65025 + 65535 < lim && tmax < lim && hmax + (tmax >> 8) + 1 < lim;
    if (p.rq.shift < 16 && !single)
      ok32 = ok32 && (hmax << (16 - p.rq.shift)) + (tmax >> (p.rq.shift - 8)) + 1 < lim;
    // single accumulator: s8 x s8 products only, the constant added in full
    if (single) ok32 = kred * 16384 + cmax < lim;
    p.fast_relu = ok32 ? 1 : 0;
  }
  const bool grouped_kernel = c.kps > 1 || c.b_resident;
  p.tail_stagger = (p.split_hh && p.fast_relu && !grouped_kernel && c.kb_per_split >= 3 && c.stages >= 3 &&
                    c.nax == 2 && c.nbw == 2 && knob(kStagger) != 0) ? 1 : 0;
  p.ws = (long long*)g.workspace; p.ws_ld = g.N;
  p.stats = g.stats;
  p.timeout_ns = knob(kTimeoutUs) > 0 ? 1000ull * (unsigned long long)knob(kTimeoutUs) : 2000000000ull;
  p.stall_at = knob(kStallAt);

  if (c.splits > 1) {
    const cudaError_t me = cudaMemsetAsync(g.workspace, 0, c.workspace_bytes, g.stream);
    if (me != cudaSuccess) return cuda_failure(me, "split-K workspace memset");
  }
  int grid;
  if (c.pair) {
    const int pairs = num_sms() / 2;
    grid = 2 * (p.total_tiles < pairs ? p.total_tiles : pairs);
  } else {
    grid = p.total_tiles < num_sms() ? p.total_tiles : num_sms();
  }
  int rc;
  if (c.nax == 2 && c.nbw == 2) rc = launch_either<2, 2>(c.pair, maps, p, grid, c.smem_bytes, g.stream);
  else if (c.nax == 2) rc = launch_either<2, 1>(c.pair, maps, p, grid, c.smem_bytes, g.stream);
  else if (c.nbw == 2) rc = launch_either<1, 2>(c.pair, maps, p, grid, c.smem_bytes, g.stream);
  else rc = launch_either<1, 1>(c.pair, maps, p, grid, c.smem_bytes, g.stream);
  if (rc != ADAPTION_OK) return rc;
  if (c.splits > 1) return launch_finalize((const int64_t*)g.workspace, g.N, g);
  return ADAPTION_OK;
}

}  // namespace adaption
