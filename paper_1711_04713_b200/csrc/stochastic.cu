// Stochastic rounding in the quantizer (paper Sec. 2.4: a stochastically rounded value is one of
// the two nearest fixed-point values and has the unrounded value as its expectation).
//
// For y = x * 2^f = floor(y) + frac the result is floor(y) + 1 with probability T / 2^32,
// T = floor(frac * 2^32), else floor(y); then ReLU (if asked) and saturation as in the
// deterministic quantizer (NaN -> 0, +-Inf saturate).  y * 2^32 is exact in double precision
// because x is fp32, and floor(y * 2^32) = floor(y) * 2^32 + T.  The draw of element i (index in the logical [outer][inner] order)
// is word i & 3 of Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with counter
// (i >> 2 as two 32-bit words, 0, 0) and the caller's 64-bit seed as key; the value moves up iff
// draw < T.  A counter-based generator makes the result a pure function of (seed, index), so it
// does not depend on the launch shape.
#include "common.cuh"

namespace adaption {

int num_sms();

namespace {

// floor(y) plus one where the draw falls below T = floor(frac(y) 2^32), y = x 2^f, from
// single-precision and 32-bit integer steps only; every step is exact:
//   y = x * 2^f never rounds (f >= 0; an overflow gives +-Inf, which the clamp to a little outside
//   the output range absorbs: beyond it only saturation matters; NaN counts as 0);
//   a = |y| < 2^16, fa = a - floor(a) is exact (a multiple of ulp(a) below 1, or a itself) and so is
//   t = fa 2^32 < 2^32;
//   y >= 0: floor(y) = floor(a), T = floor(t);
//   y <  0: floor(y) = -floor(a) - [fa > 0], frac = 1 - fa, T = 2^32 - ceil(t) (0 when fa = 0),
//           which is 0 - ceil(t) in 32-bit arithmetic.
__device__ __forceinline__ int32_t stochastic_round(float x, float scale, float y_lo, float y_hi, uint32_t draw) {
  const float y = (x != x) ? 0.0f : fminf(fmaxf(x * scale, y_lo), y_hi);
  const float a = fabsf(y);
  const float fl = floorf(a);
  const float t = (a - fl) * 4294967296.0f;
  const int32_t ia = __float2int_rz(fl);
  if (y >= 0.0f) return ia + (draw < __float2uint_rd(t) ? 1 : 0);
  const uint32_t up = __float2uint_ru(t);
  return -ia - (up != 0u ? 1 : 0) + (draw < 0u - up ? 1 : 0);
}

struct Out {
  uint4* hi;      // sixteen bytes per group of sixteen stored channels
  uint4* lo;
  uint4* q16;     // two vectors per group
  int planes;
};

// One thread per group of sixteen stored channels of one row (padding channels receive zeros and
// are neither drawn for nor counted).
__global__ void __launch_bounds__(256) quantize_stochastic_kernel(const float* __restrict__ x, size_t outer,
                                                                  int64_t inner, int64_t c_stride, Out out,
                                                                  int32_t frac_bits,
                                                                  const adaption_qfmt* __restrict__ d_fmt, int relu,
                                                                  int32_t qmin, int32_t qmax, uint32_t key0,
                                                                  uint32_t key1, adaption_stats* __restrict__ stats) {
  if (d_fmt != nullptr) frac_bits = d_fmt->frac_bits;
  const float scale = __int_as_float((127 + frac_bits) << 23);   // 2^frac_bits
  const float y_lo = (float)qmin - 2.0f, y_hi = (float)qmax + 2.0f;
  Counts c;
  const int64_t groups_per_row = c_stride / 16;
  const size_t total = outer * (size_t)groups_per_row;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += nthreads) {
    const size_t row = g / groups_per_row;
    const int64_t c0 = (int64_t)(g - row * groups_per_row) * 16;
    const int nreal = (int)min((int64_t)16, max((int64_t)0, inner - c0));
    const unsigned long long i0 = (unsigned long long)row * (unsigned long long)inner + (unsigned long long)c0;
    unsigned long long have_block = ~0ull;
    Philox4 rnd{};
    uint32_t lo[4], hi[4], h16[8];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      int32_t q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = 4 * w + u;
        const bool real = e < nreal;
        int32_t r = 0;
        if (real) {
          const unsigned long long i = i0 + (unsigned long long)e;
          const unsigned long long blk = i >> 2;
          if (blk != have_block) {
            rnd = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u, key0, key1);
            have_block = blk;
          }
          const uint32_t sel = (uint32_t)(i & 3ull);
          const uint32_t draw = sel == 0 ? rnd.w[0] : (sel == 1 ? rnd.w[1] : (sel == 2 ? rnd.w[2] : rnd.w[3]));
          r = stochastic_round(__ldg(x + i), scale, y_lo, y_hi, draw);
          if (relu) r = max(r, 0);
        }
        const int32_t qq = min(max(r, qmin), qmax);
        c.sat_pos += (real && r > qmax);
        c.sat_neg += (real && r < qmin);
        c.zeros += (real && qq == 0);
        q[u] = qq;
      }
      lo[w] = (uint32_t)(q[0] & 255) | ((uint32_t)(q[1] & 255) << 8) | ((uint32_t)(q[2] & 255) << 16) |
              ((uint32_t)(q[3] & 255) << 24);
      hi[w] = (uint32_t)((q[0] >> 8) & 255) | ((uint32_t)((q[1] >> 8) & 255) << 8) |
              ((uint32_t)((q[2] >> 8) & 255) << 16) | ((uint32_t)((q[3] >> 8) & 255) << 24);
      h16[2 * w] = (uint32_t)(q[0] & 0xffff) | ((uint32_t)(q[1] & 0xffff) << 16);
      h16[2 * w + 1] = (uint32_t)(q[2] & 0xffff) | ((uint32_t)(q[3] & 0xffff) << 16);
    }
    out.lo[g] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    if (out.planes == 2) out.hi[g] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    if (out.q16 != nullptr) {
      out.q16[2 * g] = make_uint4(h16[0], h16[1], h16[2], h16[3]);
      out.q16[2 * g + 1] = make_uint4(h16[4], h16[5], h16[6], h16[7]);
    }
  }
  if (stats != nullptr) flush_counts_warp(c, stats);
}

// Dense rows (inner == c_stride, 16-byte aligned input): the tensor is one flat array; a thread
// takes one float4 = the four elements of one generator block, and writes one 4-byte word per plane.
__global__ void __launch_bounds__(256) quantize_stochastic_flat_kernel(const float4* __restrict__ x, size_t n4,
                                                                       uint32_t* __restrict__ out_hi,
                                                                       uint32_t* __restrict__ out_lo,
                                                                       uint2* __restrict__ out_q16, int32_t frac_bits,
                                                                       const adaption_qfmt* __restrict__ d_fmt,
                                                                       int relu, int32_t qmin, int32_t qmax,
                                                                       uint32_t key0, uint32_t key1,
                                                                       adaption_stats* __restrict__ stats) {
  if (d_fmt != nullptr) frac_bits = d_fmt->frac_bits;
  const float scale = __int_as_float((127 + frac_bits) << 23);   // 2^frac_bits
  const float y_lo = (float)qmin - 2.0f, y_hi = (float)qmax + 2.0f;
  Counts c;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += nthreads) {
    const float4 v = __ldcs(x + i);
    const Philox4 rnd = philox4x32_10((uint32_t)i, (uint32_t)((unsigned long long)i >> 32), 0u, 0u, key0, key1);
    const float xs[4] = {v.x, v.y, v.z, v.w};
    int32_t q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      int32_t r = stochastic_round(xs[u], scale, y_lo, y_hi, rnd.w[u]);
      if (relu) r = max(r, 0);
      q[u] = min(max(r, qmin), qmax);
      c.sat_pos += (r > qmax);
      c.sat_neg += (r < qmin);
      c.zeros += (q[u] == 0);
    }
    out_lo[i] = (uint32_t)(q[0] & 255) | ((uint32_t)(q[1] & 255) << 8) | ((uint32_t)(q[2] & 255) << 16) |
                ((uint32_t)(q[3] & 255) << 24);
    if (out_hi != nullptr)
      out_hi[i] = (uint32_t)((q[0] >> 8) & 255) | ((uint32_t)((q[1] >> 8) & 255) << 8) |
                  ((uint32_t)((q[2] >> 8) & 255) << 16) | ((uint32_t)((q[3] >> 8) & 255) << 24);
    if (out_q16 != nullptr)
      out_q16[i] = make_uint2((uint32_t)(q[0] & 0xffff) | ((uint32_t)(q[1] & 0xffff) << 16),
                              (uint32_t)(q[2] & 0xffff) | ((uint32_t)(q[3] & 0xffff) << 16));
  }
  if (stats != nullptr) flush_counts_warp(c, stats);
}

// Format change of a stored fixed-point tensor with stochastic rounding: v / 2^s = floor + rem / 2^s
// moves up with probability rem / 2^s, taken as T = rem * 2^(32 - s) against the element's draw
// (s = f_in - f_out <= 15, so T is exact); s <= 0 is an exact left shift.  Sixteen stored channels
// per thread, as above.
__global__ void __launch_bounds__(256) requant_stochastic_kernel(const uint4* __restrict__ in_hi,
                                                                 const uint4* __restrict__ in_lo, int64_t in_stride,
                                                                 size_t outer, int64_t inner, int64_t c_stride,
                                                                 Out out, int32_t in_frac_bits, int32_t out_frac_bits,
                                                                 const adaption_qfmt* __restrict__ d_fmt, int relu,
                                                                 int32_t qmin, int32_t qmax, uint32_t key0,
                                                                 uint32_t key1, adaption_stats* __restrict__ stats) {
  if (d_fmt != nullptr) out_frac_bits = d_fmt->frac_bits;
  const int shift = in_frac_bits - out_frac_bits;
  Counts c;
  const int64_t groups_per_row = c_stride / 16, in_groups = in_stride / 16;
  const size_t total = outer * (size_t)groups_per_row;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += nthreads) {
    const size_t row = g / groups_per_row;
    const int64_t gc = (int64_t)(g - row * groups_per_row);
    const int64_t c0 = gc * 16;
    const int nreal = (int)min((int64_t)16, max((int64_t)0, inner - c0));
    uint4 l = make_uint4(0, 0, 0, 0), h = make_uint4(0, 0, 0, 0);
    if (gc < in_groups) {
      l = __ldcs(in_lo + row * (size_t)in_groups + (size_t)gc);
      if (in_hi != nullptr) h = __ldcs(in_hi + row * (size_t)in_groups + (size_t)gc);
    }
    const uint32_t lw[4] = {l.x, l.y, l.z, l.w}, hw[4] = {h.x, h.y, h.z, h.w};
    const unsigned long long i0 = (unsigned long long)row * (unsigned long long)inner + (unsigned long long)c0;
    unsigned long long have_block = ~0ull;
    Philox4 rnd{};
    uint32_t lo[4], hi[4], h16[8];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      int32_t q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = 4 * w + u;
        const bool real = e < nreal;
        int32_t r = 0;
        if (real) {
          const int32_t l8 = (lw[w] >> (8 * u)) & 255;
          int32_t v = in_hi != nullptr ? ((int32_t)(int8_t)((hw[w] >> (8 * u)) & 255)) * 256 + l8
                                       : (int32_t)(int8_t)l8;
          if (relu) v = max(v, 0);
          if (shift > 0) {
            const unsigned long long i = i0 + (unsigned long long)e;
            const unsigned long long blk = i >> 2;
            if (blk != have_block) {
              rnd = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u, key0, key1);
              have_block = blk;
            }
            const uint32_t sel = (uint32_t)(i & 3ull);
            const uint32_t draw = sel == 0 ? rnd.w[0] : (sel == 1 ? rnd.w[1] : (sel == 2 ? rnd.w[2] : rnd.w[3]));
            const int32_t fl = v >> shift;                                   // floor
            const uint32_t T = (uint32_t)(v - fl * (1 << shift)) << (32 - shift);   // remainder, scaled to 32 bits
            r = fl + (draw < T ? 1 : 0);
          } else {
            r = v * (1 << (-shift));
          }
        }
        const int32_t qq = min(max(r, qmin), qmax);
        c.sat_pos += (real && r > qmax);
        c.sat_neg += (real && r < qmin);
        c.zeros += (real && qq == 0);
        q[u] = qq;
      }
      lo[w] = (uint32_t)(q[0] & 255) | ((uint32_t)(q[1] & 255) << 8) | ((uint32_t)(q[2] & 255) << 16) |
              ((uint32_t)(q[3] & 255) << 24);
      hi[w] = (uint32_t)((q[0] >> 8) & 255) | ((uint32_t)((q[1] >> 8) & 255) << 8) |
              ((uint32_t)((q[2] >> 8) & 255) << 16) | ((uint32_t)((q[3] >> 8) & 255) << 24);
      h16[2 * w] = (uint32_t)(q[0] & 0xffff) | ((uint32_t)(q[1] & 0xffff) << 16);
      h16[2 * w + 1] = (uint32_t)(q[2] & 0xffff) | ((uint32_t)(q[3] & 0xffff) << 16);
    }
    out.lo[g] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    if (out.planes == 2) out.hi[g] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    if (out.q16 != nullptr) {
      out.q16[2 * g] = make_uint4(h16[0], h16[1], h16[2], h16[3]);
      out.q16[2 * g + 1] = make_uint4(h16[4], h16[5], h16[6], h16[7]);
    }
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
  o.planes = out.fmt.n_bits > 8 ? 2 : 1;
  o.hi = o.planes == 2 ? static_cast<uint4*>(out.hi) : nullptr;
  o.lo = static_cast<uint4*>(out.lo);
  o.q16 = reinterpret_cast<uint4*>(out.q16);
  const bool flat = (int64_t)inner == out.c_stride && aligned16(d_x);
  const size_t groups = flat ? outer * inner / 4 : outer * (size_t)(out.c_stride / 16);
  size_t want = (groups + 255) / 256;
  const size_t cap = (size_t)num_sms() * 8;
  const int grid = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
  if (flat) {
    quantize_stochastic_flat_kernel<<<grid, 256, 0, stream>>>(
        reinterpret_cast<const float4*>(d_x), groups, reinterpret_cast<uint32_t*>(o.hi),
        reinterpret_cast<uint32_t*>(o.lo), reinterpret_cast<uint2*>(o.q16), out.fmt.frac_bits, d_fmt, relu ? 1 : 0,
        qmin, qmax, (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32), d_stats);
    return cuda_status(cudaGetLastError(), "quantize_stochastic_flat_kernel launch");
  }
  quantize_stochastic_kernel<<<grid, 256, 0, stream>>>(d_x, outer, (int64_t)inner, out.c_stride, o,
                                                        out.fmt.frac_bits, d_fmt, relu ? 1 : 0, qmin, qmax,
                                                        (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32), d_stats);
  return cuda_status(cudaGetLastError(), "quantize_stochastic_kernel launch");
}

int requant_stochastic_impl(const adaption_qtensor& in, size_t outer, size_t inner, int32_t relu,
                            const adaption_qtensor& out, const adaption_qfmt* d_fmt, uint64_t seed,
                            adaption_stats* d_stats, cudaStream_t stream) {
  int rc = check_qtensor_in(in, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  rc = check_qtensor_out(out, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  if (outer == 0 || inner == 0) return ADAPTION_OK;
  const int32_t qmin = -(1 << (out.fmt.n_bits - 1)), qmax = (1 << (out.fmt.n_bits - 1)) - 1;
  Out o;
  o.planes = out.fmt.n_bits > 8 ? 2 : 1;
  o.hi = o.planes == 2 ? static_cast<uint4*>(out.hi) : nullptr;
  o.lo = static_cast<uint4*>(out.lo);
  o.q16 = reinterpret_cast<uint4*>(out.q16);
  const size_t groups = outer * (size_t)(out.c_stride / 16);
  size_t want = (groups + 255) / 256;
  const size_t cap = (size_t)num_sms() * 8;
  const int grid = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
  requant_stochastic_kernel<<<grid, 256, 0, stream>>>(
      in.fmt.n_bits > 8 ? static_cast<const uint4*>(in.hi) : nullptr, static_cast<const uint4*>(in.lo), in.c_stride,
      outer, (int64_t)inner, out.c_stride, o, in.fmt.frac_bits, out.fmt.frac_bits, d_fmt, relu ? 1 : 0, qmin, qmax,
      (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32), d_stats);
  return cuda_status(cudaGetLastError(), "requant_stochastic_kernel launch");
}

}  // namespace adaption
