// Shared device/host helpers of the CUDA path (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "adaption.h"

namespace adaption {

// Parameters of the requantizer applied to a pre-activation value v given in units of
// 2^-F (paper Sec. 2.1: the activation is quantized to the layer's format, ReLU follows;
// rounding is to nearest with ties away from zero, then saturation).
struct RequantParams {
  int32_t shift;     // F - f_out; > 0: rounding right shift, <= 0: exact left shift by -shift
  int32_t relu;      // clamp negatives to zero first
  int32_t qmin;      // -2^(n_out-1)
  int32_t qmax;      //  2^(n_out-1)-1
  int32_t out_planes;  // 2: hi/lo byte planes (n_out > 8), 1: single signed byte plane
};

struct Counts {
  uint32_t zeros = 0, sat_pos = 0, sat_neg = 0;
};

// Seed of a layer whose rounding_scheme is stochastic (paper Sec. 2, Sec. 2.4); enabled = 0 means
// deterministic rounding.
struct StochasticParams {
  int32_t enabled;
  uint32_t key0, key1;
};

struct Philox4 {
  uint32_t w[4];
};

// Philox4x32 with ten rounds, from its published definition: per round two 32x32 -> 64-bit
// products with fixed multipliers, the high halves mixed with the other counter words and the
// key, the key bumped by the Weyl constants between rounds.
__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  Philox4 o;
  o.w[0] = c0; o.w[1] = c1; o.w[2] = c2; o.w[3] = c3;
  return o;
}

// The 32-bit draw of element `i` (row-major index over the real elements of a tensor): word i & 3 of
// Philox4x32-10 with counter (i >> 2 as two 32-bit words, 0, 0) and the caller's seed as key.
__device__ __forceinline__ uint32_t philox_draw(uint64_t i, uint32_t k0, uint32_t k1) {
  const Philox4 b = philox4x32_10((uint32_t)(i >> 2), (uint32_t)(i >> 34), 0u, 0u, k0, k1);
  const uint32_t w = (uint32_t)i & 3u;
  return w == 0 ? b.w[0] : (w == 1 ? b.w[1] : (w == 2 ? b.w[2] : b.w[3]));
}

// v / 2^shift rounded half away from zero, saturated.  For shift > 0 and negative v the
// identity -((-v + h) >> s) == (v + h - 1) >> s (h = 2^(s-1), arithmetic shift) is used.
__device__ __forceinline__ int32_t requant_value(int64_t v, const RequantParams& rq, bool counted,
                                                 Counts& c) {
  if (rq.relu && v < 0) v = 0;
  int64_t r;
  if (rq.shift > 0) {
    const int64_t half = (int64_t)1 << (rq.shift - 1);
    r = (v + half + (v >> 63)) >> rq.shift;
  } else {
    // Exact left shift by at most 15 bits.  Any |v| above 2^16 already lies outside every output
    // range (at most 16 bits) after the shift, so clipping v there first keeps the stored value and
    // the saturation decision while the product stays far inside 64 bits (accumulators can reach
    // 2^61 for the longest reductions).
    const int64_t lim = (int64_t)1 << 16;
    const int64_t vc = v > lim ? lim : (v < -lim ? -lim : v);
    r = vc * ((int64_t)1 << (-rq.shift));
  }
  if (r > (int64_t)rq.qmax) {
    r = rq.qmax;
    c.sat_pos += counted;
  } else if (r < (int64_t)rq.qmin) {
    r = rq.qmin;
    c.sat_neg += counted;
  }
  c.zeros += (counted && r == 0);
  return (int32_t)r;
}

// The same with stochastic rounding (Sec. 2.4) for shift > 0: v / 2^shift = q + rem / 2^shift with
// q = floor(v / 2^shift); the result is q + 1 iff draw < T, T = rem * 2^(32 - shift), so that the
// expectation is the unrounded value and rem = 0 never moves.  shift <= 32 (the formats allow at most 30).
__device__ __forceinline__ int32_t requant_value_stochastic(int64_t v, const RequantParams& rq, uint32_t draw,
                                                            bool counted, Counts& c) {
  if (rq.shift <= 0) return requant_value(v, rq, counted, c);
  if (rq.relu && v < 0) v = 0;
  const int64_t q = v >> rq.shift;
  const uint64_t rem = (uint64_t)(v - (q << rq.shift));
  const uint32_t T = (uint32_t)(rem << (32 - rq.shift));
  int64_t r = q + (draw < T ? 1 : 0);
  if (r > (int64_t)rq.qmax) {
    r = rq.qmax;
    c.sat_pos += counted;
  } else if (r < (int64_t)rq.qmin) {
    r = rq.qmin;
    c.sat_neg += counted;
  }
  c.zeros += (counted && r == 0);
  return (int32_t)r;
}

__device__ __forceinline__ uint32_t warp_sum(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ int64_t warp_max_i64(int64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    int64_t t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t > v ? t : v;
  }
  return v;
}

// One atomic per warp and counter; lanes must all call.
__device__ __forceinline__ void flush_counts_warp(const Counts& c, adaption_stats* stats) {
  uint32_t z = warp_sum(c.zeros), p = warp_sum(c.sat_pos), n = warp_sum(c.sat_neg);
  if ((threadIdx.x & 31) == 0 && stats != nullptr) {
    if (z) atomicAdd((unsigned long long*)&stats->zeros, (unsigned long long)z);
    if (p) atomicAdd((unsigned long long*)&stats->sat_pos, (unsigned long long)p);
    if (n) atomicAdd((unsigned long long*)&stats->sat_neg, (unsigned long long)n);
  }
}

__device__ __forceinline__ void flush_max_warp(int64_t m, adaption_stats* stats) {
  m = warp_max_i64(m);
  if ((threadIdx.x & 31) == 0 && m > 0) atomicMax((long long*)&stats->max_abs_acc, (long long)m);
}

// canonical integer of element i from the stored planes
__device__ __forceinline__ int32_t load_q(const int8_t* hi, const uint8_t* lo, size_t i) {
  if (hi != nullptr) return ((int32_t)hi[i]) * 256 + (int32_t)lo[i];
  return (int32_t)((const int8_t*)lo)[i];
}

__device__ __forceinline__ void store_q(int8_t* hi, uint8_t* lo, int16_t* q16, size_t i, int32_t q) {
  if (hi != nullptr) {
    hi[i] = (int8_t)(q >> 8);
    lo[i] = (uint8_t)(q & 255);
  } else {
    lo[i] = (uint8_t)(q & 255);
  }
  if (q16 != nullptr) q16[i] = (int16_t)q;
}

inline RequantParams make_requant(int32_t acc_frac_bits, adaption_qfmt out, int32_t relu) {
  RequantParams rq;
  rq.shift = acc_frac_bits - out.frac_bits;
  rq.relu = relu ? 1 : 0;
  rq.qmin = -(1 << (out.n_bits - 1));
  rq.qmax = (1 << (out.n_bits - 1)) - 1;
  rq.out_planes = out.n_bits > 8 ? 2 : 1;
  return rq;
}

inline bool fmt_ok(adaption_qfmt f) {
  return f.n_bits >= 1 && f.n_bits <= 16 && f.frac_bits >= 0 && f.frac_bits <= f.n_bits - 1;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// a fixed-point tensor as an input operand: planes present and aligned
int check_qtensor_in(const adaption_qtensor& t, int64_t inner);
// ... as an output: planes (or at least q16) present
int check_qtensor_out(const adaption_qtensor& t, int64_t inner);

// CUDA runtime failure -> ADAPTION_ERR_CUDA; with ADAPTION_LOG set in the environment the runtime's
// message goes to stderr.
int cuda_failure(cudaError_t e, const char* where);
inline int cuda_status(cudaError_t e, const char* where = "") {
  return e == cudaSuccess ? ADAPTION_OK : cuda_failure(e, where);
}

// ---- programmatic dependent launch ---------------------------------------------------------
// A kernel launched with the stream-serialization attribute may start while its predecessor in the
// stream is still running (its blocks take the SMs the predecessor's blocks leave), which hides the
// launch latency between the many short kernels of a forward pass.  Such a kernel must not touch
// global memory before pdl_wait(), which returns once the predecessor has completed and its writes
// are visible; pdl_launch_dependents() lets the scheduler launch the successor as soon as resources
// free up.  Both are no-ops in kernels launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// First statement of every kernel launched through launch_after_predecessor: wait for the
// predecessor, and only then let the successor be scheduled.  (The other order - announcing the
// successor before this kernel has itself synchronised with its predecessor - was tried: a chain of
// three short kernels then once let the third read what the second had only partly written.)
__device__ __forceinline__ void pdl_prologue() {
  pdl_wait();
  pdl_launch_dependents();
}

bool pdl_enabled();      // process-wide switch (adaption_debug_set "pdl")

// Launch of a kernel whose first statement is pdl_prologue().
template <typename... KArgs, typename... Args>
inline cudaError_t launch_after_predecessor(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream,
                                            Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  if (pdl_enabled()) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- launches implemented in the other translation units ---------------------------------
struct GemmProblem {
  // logical GEMM: rows M (pixels or batch), columns N (output channels), reduction over K
  int64_t M = 0, N = 0, K = 0;   // K: real reduction length (no padding)
  bool is_conv = false;
  adaption_conv_shape cs{};      // valid when is_conv
  int32_t OH = 0, OW = 0;
  adaption_qtensor x{}, w{}, y{};
  const int16_t* bias = nullptr;
  int32_t bias_shift = 0;        // F - bias_frac_bits
  int32_t acc_frac_bits = 0;     // F = f_x + f_w
  int32_t relu = 0, mode = 0;
  adaption_stats* stats = nullptr;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  cudaStream_t stream = nullptr;
  // Tensor-core path only: y receives max(row 2j, row 2j+1) of the layer's output as its row j (the
  // horizontal half of a 2x2 max-pool; y then has M / 2 rows).  Counters still refer to all M rows.
  bool pool_w = false;
  // rounding_scheme STOCHASTIC for the requantization of this layer (REQUANT mode only)
  StochasticParams stochastic{0, 0u, 0u};
};

int launch_direct(const GemmProblem& p);
bool tensor_path_supported(const GemmProblem& p);
size_t tensor_path_workspace(const GemmProblem& p);
int launch_tensor(const GemmProblem& p);
bool tensor_path_can_pool(const GemmProblem& p);   // whether launch_tensor takes `p` with pool_w set
// Convolutions with at most 4 input channels whose taps fit one 32-byte row: gather the taps into
// packed planes in the workspace and run the layer as an inner product on the tensor-core path.
bool pack_taps_applicable(const GemmProblem& p);
size_t pack_taps_workspace(const GemmProblem& p);
int launch_pack_taps(const GemmProblem& p);
bool pack_taps_can_pool(const GemmProblem& p);
// bias/ReLU/requantize (or range) of an int64 accumulator matrix acc[M][ld] -> y
int launch_finalize(const int64_t* acc, int64_t ld, const GemmProblem& p);

}  // namespace adaption
