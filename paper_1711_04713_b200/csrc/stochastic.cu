// Stochastic rounding in the quantizer (paper Sec. 2.4: a stochastically rounded value is one of
// the two nearest fixed-point values and has the unrounded value as its expectation).
//
// For y = x * 2^f = floor(y) + frac the result is floor(y) + 1 with probability T / 2^32,
// T = floor(frac * 2^32), else floor(y); then ReLU (if asked) and saturation as in the
// deterministic quantizer (NaN -> 0, +-Inf saturate).  Both parts of y are exact in double
// precision because x is fp32.  The draw of element i (index in the logical [outer][inner] order)
// is word i & 3 of Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with counter
// (i >> 2 as two 32-bit words, 0, 0) and the caller's 64-bit seed as key; the value moves up iff
// draw < T.  A counter-based generator makes the result a pure function of (seed, index), so it
// does not depend on the launch shape.
#include "common.cuh"

namespace adaption {

int num_sms();

namespace {

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

struct Out {
  int8_t* hi;
  uint8_t* lo;
  int16_t* q16;
};

// One thread per group of four stored channels of one row (padding channels receive zeros and
// are neither drawn for nor counted).
__global__ void __launch_bounds__(256) quantize_stochastic_kernel(const float* __restrict__ x, size_t outer,
                                                                  int64_t inner, int64_t c_stride, Out out,
                                                                  int32_t frac_bits,
                                                                  const adaption_qfmt* __restrict__ d_fmt, int relu,
                                                                  int32_t qmin, int32_t qmax, uint32_t key0,
                                                                  uint32_t key1, adaption_stats* __restrict__ stats) {
  if (d_fmt != nullptr) frac_bits = d_fmt->frac_bits;
  const double scale = __longlong_as_double((long long)(1023 + frac_bits) << 52);   // 2^frac_bits
  Counts c;
  const int64_t groups_per_row = c_stride / 4;
  const size_t total = outer * (size_t)groups_per_row;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += nthreads) {
    const size_t row = g / groups_per_row;
    const int64_t c0 = (int64_t)(g - row * groups_per_row) * 4;
    unsigned long long have_block = ~0ull;
    Philox4 rnd{};
    int32_t q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const bool real = c0 + u < inner;
      int32_t r = 0;
      if (real) {
        const unsigned long long i = (unsigned long long)row * (unsigned long long)inner + (unsigned long long)(c0 + u);
        const unsigned long long blk = i >> 2;
        if (blk != have_block) {
          rnd = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u, key0, key1);
          have_block = blk;
        }
        const uint32_t sel = (uint32_t)(i & 3ull);
        const uint32_t draw = sel == 0 ? rnd.w[0] : (sel == 1 ? rnd.w[1] : (sel == 2 ? rnd.w[2] : rnd.w[3]));
        const float xv = __ldg(x + i);
        double y = (xv != xv) ? 0.0 : (double)xv * scale;
        // far outside the range only saturation matters: clamp so that the integer parts stay small
        y = fmin(fmax(y, (double)qmin - 2.0), (double)qmax + 2.0);
        const double fl = floor(y);
        const uint32_t T = (uint32_t)(unsigned long long)((y - fl) * 4294967296.0);
        r = (int32_t)fl + (draw < T ? 1 : 0);
        if (relu) r = max(r, 0);
      }
      const int32_t qq = min(max(r, qmin), qmax);
      c.sat_pos += (real && r > qmax);
      c.sat_neg += (real && r < qmin);
      c.zeros += (real && qq == 0);
      q[u] = qq;
    }
    const size_t e0 = g * 4;
#pragma unroll
    for (int u = 0; u < 4; ++u) store_q(out.hi, out.lo, out.q16, e0 + u, q[u]);
  }
  if (stats != nullptr) flush_counts_warp(c, stats);
}

}  // namespace

int quantize_stochastic_impl(const float* d_x, size_t outer, size_t inner, const adaption_qtensor& out,
                             const adaption_qfmt* d_fmt, int32_t relu, uint64_t seed, adaption_stats* d_stats,
                             cudaStream_t stream) {
  int rc = check_qtensor_out(out, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  if (outer == 0 || inner == 0) return ADAPTION_OK;
  if (d_x == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_x) & 3u) != 0) return ADAPTION_ERR_ALIGNMENT;
  const int32_t qmin = -(1 << (out.fmt.n_bits - 1)), qmax = (1 << (out.fmt.n_bits - 1)) - 1;
  Out o;
  o.hi = out.fmt.n_bits > 8 ? static_cast<int8_t*>(out.hi) : nullptr;
  o.lo = static_cast<uint8_t*>(out.lo);
  o.q16 = out.q16;
  const size_t groups = outer * (size_t)(out.c_stride / 4);
  size_t want = (groups + 255) / 256;
  const size_t cap = (size_t)num_sms() * 8;
  const int grid = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
  quantize_stochastic_kernel<<<grid, 256, 0, stream>>>(d_x, outer, (int64_t)inner, out.c_stride, o,
                                                        out.fmt.frac_bits, d_fmt, relu ? 1 : 0, qmin, qmax,
                                                        (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32), d_stats);
  return cuda_status(cudaGetLastError(), "quantize_stochastic_kernel launch");
}

}  // namespace adaption
