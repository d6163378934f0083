// HBM-bound kernels: dynamic-range measurement, the fp32 -> fixed-point quantizer (LPAct with an
// fp32 input is the same kernel with the ReLU flag), fixed-point format conversion, 2x2 max-pool.
// All of them are coalesced streaming kernels sized to a multiple of the SM count.
#include <atomic>

#include "common.cuh"

namespace adaption {

// SM count of the current device, cached per device ordinal (each entry is written once with the
// same value by whichever thread gets there first, so a relaxed atomic is all it needs).
int num_sms() {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cache[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  const bool cached = dev >= 0 && dev < kMaxDevices;
  int n = cached ? cache[dev].load(std::memory_order_relaxed) : 0;
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    if (cached) cache[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

static inline int stream_grid(size_t work_items, int threads, int blocks_per_sm) {
  size_t want = (work_items + threads - 1) / threads;
  size_t cap = (size_t)num_sms() * blocks_per_sm;
  if (want < 1) want = 1;
  return (int)(want < cap ? want : cap);
}

// ------------------------------------------------------------------------------------------
// Dynamic range (paper Sec. 2.1, Sec. 2.3): max |x|, NaN ignored.  Non-negative floats order
// like their bit patterns, so the cross-block reduction is an integer atomicMax.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) range_max_abs_kernel(const float* __restrict__ x, size_t numel,
                                                            size_t head, size_t n4,
                                                            float* __restrict__ d_max_abs) {
  pdl_prologue();
  float m = 0.0f;
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  // unaligned head and tail as scalars
  if (tid < head) m = fmaxf(m, fabsf(x[tid]));
  const size_t tail_begin = head + n4 * 4;
  if (tail_begin + tid < numel) m = fmaxf(m, fabsf(x[tail_begin + tid]));
  const float4* __restrict__ x4 = reinterpret_cast<const float4*>(x + head);
  size_t i = tid;
  for (; i + 3 * nthreads < n4; i += 4 * nthreads) {
    float4 a = __ldg(x4 + i), b = __ldg(x4 + i + nthreads), c = __ldg(x4 + i + 2 * nthreads),
           d = __ldg(x4 + i + 3 * nthreads);
    m = fmaxf(m, fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w))));
    m = fmaxf(m, fmaxf(fmaxf(fabsf(b.x), fabsf(b.y)), fmaxf(fabsf(b.z), fabsf(b.w))));
    m = fmaxf(m, fmaxf(fmaxf(fabsf(c.x), fabsf(c.y)), fmaxf(fabsf(c.z), fabsf(c.w))));
    m = fmaxf(m, fmaxf(fmaxf(fabsf(d.x), fabsf(d.y)), fmaxf(fabsf(d.z), fabsf(d.w))));
  }
  for (; i < n4; i += nthreads) {
    float4 a = __ldg(x4 + i);
    m = fmaxf(m, fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w))));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float wmax[8];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    float b = wmax[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) b = fmaxf(b, wmax[w]);
    if (b > 0.0f) atomicMax(reinterpret_cast<int*>(d_max_abs), __float_as_int(b));
  }
}

// Decimal point from the maximum (Sec. 2.3): smallest m in [0, n-1] with max < 2^m.  For
// max >= 1 with binary exponent e (max in [2^e, 2^(e+1))) that is e+1; Inf has e = 128.
__global__ void choose_fmt_kernel(const float* __restrict__ d_max_abs, int32_t n_bits,
                                  adaption_qfmt* __restrict__ d_fmt) {
  pdl_prologue();
  const int bits = __float_as_int(*d_max_abs) & 0x7fffffff;
  const int e = (bits >> 23) - 127;
  int m = e >= 0 ? e + 1 : 0;
  if (m > n_bits - 1) m = n_bits - 1;
  d_fmt->n_bits = n_bits;
  d_fmt->frac_bits = n_bits - 1 - m;
}

// ------------------------------------------------------------------------------------------
// Quantizer (paper Sec. 2): q = saturate(round_half_away(x * 2^f)).  x * 2^f is exact in fp32;
// the tie rule is applied on the exact fractional part (trunc + exact remainder), never on a
// rounded sum.
// ------------------------------------------------------------------------------------------
// `scale2` is 2^(f+1): z = trunc(2 * x * 2^f) is taken with the saturating float->int conversion
// (NaN -> 0, +-Inf and anything beyond int32 -> INT_MAX / INT_MIN), and the nearest integer with
// ties away from zero is sign(z) * ((|z| + 1) >> 1): for 2y = n + e, 0 <= e < 1,
// floor(y + 1/2) = floor((n + 1) / 2 + e / 2) = (n + 1) >> 1 because (n + 1) / 2 is an integer or a
// half-integer and e / 2 < 1/2.  Only integer work follows the one conversion.
__device__ __forceinline__ int32_t quantize_f32(float x, float scale2, int relu, int32_t qmin,
                                                int32_t qmax, bool counted, Counts& c) {
  int32_t z = __float2int_rz(x * scale2);
  if (relu) z = max(z, 0);
  const uint32_t a = (uint32_t)(z < 0 ? -(long long)z : (long long)z);   // |z| up to 2^31
  const int32_t mag = (int32_t)((a + 1u) >> 1);                          // <= 2^30
  const int32_t r = z < 0 ? -mag : mag;
  const int32_t q = min(max(r, qmin), qmax);
  c.sat_pos += (counted && r > qmax);
  c.sat_neg += (counted && r < qmin);
  c.zeros += (counted && q == 0);
  return q;
}

// Four elements at once for the dense kernel; the counters are derived per group (clipping is
// detected by OR-ing r ^ q and only then counted exactly).
__device__ __forceinline__ void quantize_f32x4(const float4 v, float scale2, int relu, int32_t qmin,
                                               int32_t qmax, Counts& c, int32_t (&q)[4]) {
  const float x[4] = {v.x, v.y, v.z, v.w};
  int32_t r[4], clipped = 0, nonzero = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    int32_t z = __float2int_rz(x[k] * scale2);
    if (relu) z = max(z, 0);
    const uint32_t a = (uint32_t)(z < 0 ? -(long long)z : (long long)z);
    const int32_t mag = (int32_t)((a + 1u) >> 1);
    r[k] = z < 0 ? -mag : mag;
    q[k] = min(max(r[k], qmin), qmax);
    clipped |= r[k] ^ q[k];
    nonzero += min(abs(q[k]), 1);
  }
  c.zeros += 4 - nonzero;
  if (clipped != 0) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      c.sat_pos += (r[k] > qmax);
      c.sat_neg += (r[k] < qmin);
    }
  }
}

// 2^(frac_bits + 1), the scale quantize_f32 expects
__device__ __forceinline__ float scale_of(int32_t frac_bits) {
  return __int_as_float((128 + frac_bits) << 23);
}

struct QuantOut {
  uint32_t* hi;   // words of 4 bytes
  uint32_t* lo;
  uint2* q16;     // 4 int16
  int32_t planes;
};

__device__ __forceinline__ void store4(const QuantOut& o, size_t word, int32_t q0, int32_t q1,
                                       int32_t q2, int32_t q3) {
  const uint32_t lo = (uint32_t)(q0 & 255) | ((uint32_t)(q1 & 255) << 8) |
                      ((uint32_t)(q2 & 255) << 16) | ((uint32_t)(q3 & 255) << 24);
  __stcs(o.lo + word, lo);                    // streaming stores: the planes are read much later
  if (o.planes == 2) {
    const uint32_t hi = (uint32_t)((q0 >> 8) & 255) | ((uint32_t)((q1 >> 8) & 255) << 8) |
                        ((uint32_t)((q2 >> 8) & 255) << 16) | ((uint32_t)((q3 >> 8) & 255) << 24);
    __stcs(o.hi + word, hi);
  }
  if (o.q16 != nullptr) {
    uint2 v;
    v.x = (uint32_t)(q0 & 0xffff) | ((uint32_t)(q1 & 0xffff) << 16);
    v.y = (uint32_t)(q2 & 0xffff) | ((uint32_t)(q3 & 0xffff) << 16);
    o.q16[word] = v;
  }
}

// Dense rows (inner == c_stride): the tensor is one flat array; one float4 in, one 4-byte word
// per plane out, four independent groups in flight per thread.
__global__ void __launch_bounds__(256) quantize_flat_kernel(const float4* __restrict__ x, size_t n4,
                                                            QuantOut out, int32_t frac_bits,
                                                            const adaption_qfmt* __restrict__ d_fmt,
                                                            int relu, int32_t qmin, int32_t qmax,
                                                            adaption_stats* __restrict__ stats) {
  pdl_prologue();
  if (d_fmt != nullptr) frac_bits = d_fmt->frac_bits;
  const float scale = scale_of(frac_bits);
  Counts c;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * nthreads < n4; i += 4 * nthreads) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = __ldcs(x + i + u * nthreads);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      int32_t q[4];
      quantize_f32x4(v[u], scale, relu, qmin, qmax, c, q);
      store4(out, i + u * nthreads, q[0], q[1], q[2], q[3]);
    }
  }
  for (; i < n4; i += nthreads) {
    int32_t q[4];
    quantize_f32x4(__ldcs(x + i), scale, relu, qmin, qmax, c, q);
    store4(out, i, q[0], q[1], q[2], q[3]);
  }
  if (stats != nullptr) flush_counts_warp(c, stats);
}

// Rows with channel padding (inner < c_stride) or unaligned input: one thread per group of sixteen
// stored channels (one 16-byte vector per plane); padding channels receive zeros and are not
// counted.
__global__ void __launch_bounds__(256) quantize_rows_kernel(const float* __restrict__ x, size_t outer,
                                                            int64_t inner, int64_t c_stride,
                                                            QuantOut out, int32_t frac_bits,
                                                            const adaption_qfmt* __restrict__ d_fmt,
                                                            int relu, int32_t qmin, int32_t qmax,
                                                            adaption_stats* __restrict__ stats) {
  pdl_prologue();
  if (d_fmt != nullptr) frac_bits = d_fmt->frac_bits;
  const float scale = scale_of(frac_bits);
  Counts c;
  const int64_t groups_per_row = c_stride / 16;
  const size_t total = outer * (size_t)groups_per_row;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  const bool small = total <= 0xffffffffull;      // 32-bit division whenever the group index fits
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += nthreads) {
    const size_t row = small ? (size_t)((uint32_t)g / (uint32_t)groups_per_row) : g / groups_per_row;
    const int64_t c0 = (int64_t)(g - row * groups_per_row) * 16;
    const float* __restrict__ src = x + row * (size_t)inner + c0;
    const int nreal = (int)min((int64_t)16, max((int64_t)0, inner - c0));
    uint32_t lo[4], hi[4], h16[8];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      if (4 * w >= nreal) {               // only padding from here on: zeros, nothing to compute
        lo[w] = hi[w] = h16[2 * w] = h16[2 * w + 1] = 0u;
        continue;
      }
      int32_t q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool real = 4 * w + u < nreal;
        const float v = real ? __ldg(src + 4 * w + u) : 0.0f;
        q[u] = quantize_f32(v, scale, relu, qmin, qmax, real, c);
      }
      lo[w] = (uint32_t)(q[0] & 255) | ((uint32_t)(q[1] & 255) << 8) | ((uint32_t)(q[2] & 255) << 16) |
              ((uint32_t)(q[3] & 255) << 24);
      hi[w] = (uint32_t)((q[0] >> 8) & 255) | ((uint32_t)((q[1] >> 8) & 255) << 8) |
              ((uint32_t)((q[2] >> 8) & 255) << 16) | ((uint32_t)((q[3] >> 8) & 255) << 24);
      h16[2 * w] = (uint32_t)(q[0] & 0xffff) | ((uint32_t)(q[1] & 0xffff) << 16);
      h16[2 * w + 1] = (uint32_t)(q[2] & 0xffff) | ((uint32_t)(q[3] & 0xffff) << 16);
    }
    reinterpret_cast<uint4*>(out.lo)[g] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    if (out.planes == 2) reinterpret_cast<uint4*>(out.hi)[g] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    if (out.q16 != nullptr) {
      uint4* d = reinterpret_cast<uint4*>(out.q16) + 2 * g;
      d[0] = make_uint4(h16[0], h16[1], h16[2], h16[3]);
      d[1] = make_uint4(h16[4], h16[5], h16[6], h16[7]);
    }
  }
  if (stats != nullptr) flush_counts_warp(c, stats);
}

// Requantization of a stored value (|v| <= 2^15, |shift| <= 15): everything fits in 32 bits.
__device__ __forceinline__ int32_t requant_small(int32_t v, const RequantParams& rq, bool counted, Counts& c) {
  if (rq.relu) v = max(v, 0);
  int32_t r;
  if (rq.shift > 0) {
    const int32_t mag = (abs(v) + (1 << (rq.shift - 1))) >> rq.shift;
    r = v < 0 ? -mag : mag;
  } else {
    r = v * (1 << (-rq.shift));
  }
  const int32_t q = min(max(r, rq.qmin), rq.qmax);
  c.sat_pos += (counted && r > rq.qmax);
  c.sat_neg += (counted && r < rq.qmin);
  c.zeros += (counted && q == 0);
  return q;
}

// Format conversion of a stored fixed-point tensor (LPAct on quantized values): optional ReLU,
// rounding shift from f_in to f_out, saturation to the output width.
__global__ void __launch_bounds__(256) requant_rows_kernel(const uint32_t* __restrict__ in_hi,
                                                           const uint32_t* __restrict__ in_lo,
                                                           int64_t in_stride, size_t outer,
                                                           int64_t inner, int64_t c_stride, QuantOut out,
                                                           int32_t in_frac_bits, int32_t out_frac_bits,
                                                           const adaption_qfmt* __restrict__ d_fmt,
                                                           RequantParams rq,
                                                           adaption_stats* __restrict__ stats) {
  if (d_fmt != nullptr) out_frac_bits = d_fmt->frac_bits;
  rq.shift = in_frac_bits - out_frac_bits;
  Counts c;
  const int64_t groups_per_row = c_stride / 4;
  const size_t total = outer * (size_t)groups_per_row;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += nthreads) {
    const size_t row = g / groups_per_row;
    const int64_t c0 = (int64_t)(g - row * groups_per_row) * 4;
    uint32_t wlo = 0, whi = 0;
    if (c0 < in_stride) {
      const size_t word = (row * (size_t)in_stride + (size_t)c0) / 4;
      wlo = __ldg(in_lo + word);
      if (in_hi != nullptr) whi = __ldg(in_hi + word);
    }
    int32_t q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int32_t l = (wlo >> (8 * u)) & 255;
      int32_t v;
      if (in_hi != nullptr)
        v = ((int32_t)(int8_t)((whi >> (8 * u)) & 255)) * 256 + l;
      else
        v = (int32_t)(int8_t)l;
      const bool real = c0 + u < inner;
      q[u] = requant_small(real ? v : 0, rq, real, c);
    }
    store4(out, g, q[0], q[1], q[2], q[3]);
  }
  if (stats != nullptr) flush_counts_warp(c, stats);
}

// Dense rows on both sides (pitch == inner extent, no int16 copy): the tensor is one flat array,
// sixteen elements (one 16-byte vector per plane) per thread and step, no index arithmetic.
// The kernel has to stay below about ten integer instructions per element to run at memory speed
// (4 bytes of traffic per element), so bytes are gathered and scattered with byte permutes, the
// rounding shift is v + h - (v < 0) >> s (equal to the half-away-from-zero form: for v < 0,
// -((-v + h) >> s) = ceil((v - h) / 2^s) = floor((v + h - 1) / 2^s) with 2 h = 2^s), zeros are counted
// on the packed output bytes and saturations only where a clamp changed something.
__device__ __forceinline__ uint32_t byte_perm(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// element b of a word pair: hi * 256 + lo with the sign of the high byte (or of the only byte)
// replicated upwards (selector nibbles with bit 3 set copy the sign of the byte they name)
template <bool TWO_PLANES_IN>
__device__ __forceinline__ int32_t stored_value(uint32_t lw, uint32_t hw, int b) {
  return TWO_PLANES_IN ? (int32_t)byte_perm(lw, hw, 0xCC40u + 0x1111u * b)
                       : (int32_t)byte_perm(lw, 0u, 0x8880u + 0x1111u * b);
}

__device__ __forceinline__ int32_t requant_unclamped(int32_t v, const RequantParams& rq, int32_t half) {
  if (rq.relu) v = max(v, 0);
  return rq.shift > 0 ? (v + half + (v >> 31)) >> rq.shift : v * (1 << (-rq.shift));
}

template <bool TWO_PLANES_IN>
__device__ __forceinline__ void requant_word(uint32_t lw, uint32_t hw, const RequantParams& rq, int32_t half,
                                             Counts& c, uint32_t& out_lo, uint32_t& out_hi) {
  int32_t q[4], clipped = 0;
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const int32_t r = requant_unclamped(stored_value<TWO_PLANES_IN>(lw, hw, b), rq, half);
    q[b] = min(max(r, rq.qmin), rq.qmax);
    clipped |= r ^ q[b];
  }
  if (clipped != 0) {             // rare: count exactly
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int32_t r = requant_unclamped(stored_value<TWO_PLANES_IN>(lw, hw, b), rq, half);
      c.sat_pos += (r > rq.qmax);
      c.sat_neg += (r < rq.qmin);
    }
  }
  const uint32_t p01 = byte_perm((uint32_t)q[0], (uint32_t)q[1], 0x5410u);   // two int16
  const uint32_t p23 = byte_perm((uint32_t)q[2], (uint32_t)q[3], 0x5410u);
  out_lo = byte_perm(p01, p23, 0x6420u);
  out_hi = byte_perm(p01, p23, 0x7531u);
  // zero elements: both bytes zero.  A byte of ((x & 0x7f7f7f7f) + 0x7f7f7f7f) | x has its top
  // bit clear exactly where the byte of x is zero (no carry crosses a byte).
  const uint32_t x = rq.out_planes == 2 ? (out_lo | out_hi) : out_lo;
  const uint32_t nz = (((x & 0x7f7f7f7fu) + 0x7f7f7f7fu) | x) & 0x80808080u;
  c.zeros += 4 - __popc(nz);
}

template <bool TWO_PLANES_IN>
__global__ void __launch_bounds__(256) requant_flat_kernel(const uint4* __restrict__ in_hi,
                                                           const uint4* __restrict__ in_lo, size_t n16,
                                                           uint4* __restrict__ out_hi, uint4* __restrict__ out_lo,
                                                           int32_t in_frac_bits, int32_t out_frac_bits,
                                                           const adaption_qfmt* __restrict__ d_fmt,
                                                           RequantParams rq, adaption_stats* __restrict__ stats) {
  if (d_fmt != nullptr) out_frac_bits = d_fmt->frac_bits;
  rq.shift = in_frac_bits - out_frac_bits;
  const int32_t half = rq.shift > 0 ? 1 << (rq.shift - 1) : 0;
  Counts c;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  auto one = [&](size_t at, const uint4 lo, const uint4 hi) {
    const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w}, hw[4] = {hi.x, hi.y, hi.z, hi.w};
    uint32_t olo[4], ohi[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) requant_word<TWO_PLANES_IN>(lw[w], hw[w], rq, half, c, olo[w], ohi[w]);
    __stcs(out_lo + at, make_uint4(olo[0], olo[1], olo[2], olo[3]));
    if (rq.out_planes == 2) __stcs(out_hi + at, make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]));
  };
  for (; i + nthreads < n16; i += 2 * nthreads) {      // two vectors per plane in flight
    const uint4 lo0 = __ldcs(in_lo + i), lo1 = __ldcs(in_lo + i + nthreads);
    uint4 hi0 = make_uint4(0, 0, 0, 0), hi1 = hi0;
    if (TWO_PLANES_IN) {
      hi0 = __ldcs(in_hi + i);
      hi1 = __ldcs(in_hi + i + nthreads);
    }
    one(i, lo0, hi0);
    one(i + nthreads, lo1, hi1);
  }
  for (; i < n16; i += nthreads)
    one(i, __ldcs(in_lo + i), TWO_PLANES_IN ? __ldcs(in_hi + i) : make_uint4(0, 0, 0, 0));
  if (stats != nullptr) flush_counts_warp(c, stats);
}

// ------------------------------------------------------------------------------------------
// 2x2 / stride 2 max-pool on stored integers; 16 channels (one 16-byte vector per plane) per
// thread.  Exact on the quantized values because the quantizer is monotone.
// ------------------------------------------------------------------------------------------
// Sixteen values at once, four per 32-bit word, without unpacking the byte planes: a candidate
// 256*qh + ql beats the current 256*ph + pl iff qh > ph (signed bytes) or qh == ph and ql > pl
// (unsigned bytes); the per-byte comparison masks then select whole bytes in both planes.
__device__ __forceinline__ void max16(uint4& bh, uint4& bl, const uint4& h, const uint4& l, bool two) {
  uint32_t* ph = reinterpret_cast<uint32_t*>(&bh);
  uint32_t* pl = reinterpret_cast<uint32_t*>(&bl);
  const uint32_t* qh = reinterpret_cast<const uint32_t*>(&h);
  const uint32_t* ql = reinterpret_cast<const uint32_t*>(&l);
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    if (two) {
      const uint32_t m = __vcmpgts4(qh[w], ph[w]) | (__vcmpeq4(qh[w], ph[w]) & __vcmpgtu4(ql[w], pl[w]));
      ph[w] = (qh[w] & m) | (ph[w] & ~m);
      pl[w] = (ql[w] & m) | (pl[w] & ~m);
    } else {
      pl[w] = __vmaxs4(pl[w], ql[w]);       // one plane of signed bytes
    }
  }
}

// IDX: 32-bit index arithmetic (three divisions per output vector) whenever the tensors allow it.
template <typename IDX>
__global__ void __launch_bounds__(256) maxpool2x2_kernel(const uint4* __restrict__ in_hi,
                                                         const uint4* __restrict__ in_lo,
                                                         uint4* __restrict__ out_hi,
                                                         uint4* __restrict__ out_lo,
                                                         int16_t* __restrict__ out_q16, int N, int H,
                                                         int W, int kw, int64_t in_vecs64, int64_t out_vecs64) {
  pdl_prologue();
  // in_vecs / out_vecs: 16-byte vectors per pixel (c_stride / 16).  kw = 2: 2x2 windows; kw = 1: the
  // input is already the horizontal maximum of pixel pairs (W columns), only rows are paired.
  // H is even, so output row r = n * OH + oh (counted over the batch) pairs input rows 2r, 2r + 1.
  const IDX in_vecs = (IDX)in_vecs64, out_vecs = (IDX)out_vecs64;
  const IDX OW = (IDX)(W / kw);
  const IDX vecs = in_vecs < out_vecs ? in_vecs : out_vecs;
  const IDX total = (IDX)N * (IDX)(H / 2) * OW * out_vecs;
  const IDX nthreads = (IDX)gridDim.x * (IDX)blockDim.x;
  const bool two = in_hi != nullptr;
  for (IDX t = (IDX)blockIdx.x * (IDX)blockDim.x + (IDX)threadIdx.x; t < total; t += nthreads) {
    const IDX q = t / out_vecs;
    const IDX v = t - q * out_vecs;
    const IDX r = q / OW;
    const IDX ow = q - r * OW;
    uint4 bh = make_uint4(0, 0, 0, 0), bl = make_uint4(0, 0, 0, 0);
    if (v < vecs) {
      const IDX p00 = ((IDX)2 * r * (IDX)W + (IDX)kw * ow) * in_vecs + v;
      const IDX offs[4] = {p00, p00 + (IDX)W * in_vecs, p00 + in_vecs, p00 + (IDX)W * in_vecs + in_vecs};
      const int ncand = 2 * kw;          // the two rows first, then (2x2 only) their right neighbours
      uint4 h[4], l[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (k < ncand) {
          l[k] = __ldg(in_lo + offs[k]);
          h[k] = two ? __ldg(in_hi + offs[k]) : make_uint4(0, 0, 0, 0);
        }
      }
      bh = h[0];
      bl = l[0];
#pragma unroll
      for (int k = 1; k < 4; ++k)
        if (k < ncand) max16(bh, bl, h[k], l[k], two);
    }
    out_lo[t] = bl;
    if (two) out_hi[t] = bh;
    if (out_q16 != nullptr) {
      const uint32_t* ph = reinterpret_cast<const uint32_t*>(&bh);
      const uint32_t* pl = reinterpret_cast<const uint32_t*>(&bl);
      int16_t* dst = out_q16 + (size_t)t * 16;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int32_t l8 = (pl[e / 4] >> (8 * (e % 4))) & 255;
        dst[e] = two ? (int16_t)(((int32_t)(int8_t)((ph[e / 4] >> (8 * (e % 4))) & 255)) * 256 + l8)
                     : (int16_t)(int8_t)l8;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
int check_qtensor_in(const adaption_qtensor& t, int64_t inner) {
  if (!fmt_ok(t.fmt)) return ADAPTION_ERR_INVALID_ARG;
  if (t.lo == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if (t.fmt.n_bits > 8 && t.hi == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if (t.c_stride < inner || (t.c_stride % 16) != 0) return ADAPTION_ERR_INVALID_ARG;
  if (!aligned16(t.lo) || !aligned16(t.hi)) return ADAPTION_ERR_ALIGNMENT;
  return ADAPTION_OK;
}

int check_qtensor_out(const adaption_qtensor& t, int64_t inner) {
  int rc = check_qtensor_in(t, inner);
  if (rc != ADAPTION_OK) return rc;
  if (t.q16 != nullptr && !aligned16(t.q16)) return ADAPTION_ERR_ALIGNMENT;
  return ADAPTION_OK;
}

static QuantOut quant_out_of(const adaption_qtensor& t) {
  QuantOut o;
  o.planes = t.fmt.n_bits > 8 ? 2 : 1;
  o.hi = o.planes == 2 ? reinterpret_cast<uint32_t*>(t.hi) : nullptr;
  o.lo = reinterpret_cast<uint32_t*>(t.lo);
  o.q16 = reinterpret_cast<uint2*>(t.q16);
  return o;
}

int quantize_impl(const float* d_x, size_t outer, size_t inner, const adaption_qtensor& out,
                  const adaption_qfmt* d_fmt, int32_t relu, int32_t rounding, adaption_stats* d_stats,
                  cudaStream_t stream) {
  if (rounding == ADAPTION_ROUND_STOCHASTIC) return ADAPTION_ERR_UNSUPPORTED;
  if (rounding != ADAPTION_ROUND_DETERMINISTIC) return ADAPTION_ERR_INVALID_ARG;
  int rc = check_qtensor_out(out, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  if (outer == 0 || inner == 0) return ADAPTION_OK;
  if (d_x == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_x) & 3u) != 0) return ADAPTION_ERR_ALIGNMENT;
  const int32_t qmin = -(1 << (out.fmt.n_bits - 1)), qmax = (1 << (out.fmt.n_bits - 1)) - 1;
  const QuantOut qo = quant_out_of(out);
  if ((int64_t)inner == out.c_stride && aligned16(d_x)) {
    const size_t n4 = outer * inner / 4;
    const int grid = stream_grid((n4 + 3) / 4, 256, 8);
    launch_after_predecessor(quantize_flat_kernel, dim3(grid), dim3(256), stream, reinterpret_cast<const float4*>(d_x), n4, qo,
                                                   out.fmt.frac_bits, d_fmt, relu, qmin, qmax, d_stats);
  } else {
    const size_t groups = outer * (size_t)(out.c_stride / 16);
    const int grid = stream_grid(groups, 256, 8);
    launch_after_predecessor(quantize_rows_kernel, dim3(grid), dim3(256), stream, d_x, outer, (int64_t)inner, out.c_stride, qo,
                                                   out.fmt.frac_bits, d_fmt, relu, qmin, qmax, d_stats);
  }
  return cuda_status(cudaGetLastError());
}

// ------------------------------------------------------------------------------------------
// Several dense tensors in one launch (the weights and biases of a whole network, quantized anew
// in every forward pass): the tensors are cut into chunks of 1024 float4, numbered across the
// batch; a block walks the chunks with the grid's stride and looks up the tensor a chunk belongs
// to in the launch parameters (first_chunk is the running sum).  Per element the work is that of
// quantize_flat_kernel.
constexpr int kBatchItems = 40;
constexpr int kBatchChunk4 = 1024;      // float4 per chunk: four per thread of a 256-thread block

struct BatchItem {
  const float4* x;
  uint32_t* hi;
  uint32_t* lo;
  uint2* q16;
  const adaption_qfmt* d_fmt;
  unsigned long long n4;            // float4 in this tensor
  unsigned long long first_chunk;   // chunks of the tensors before it
  int32_t frac_bits, qmin, qmax, planes;
};

struct BatchArgs {
  BatchItem item[kBatchItems];
  unsigned long long total_chunks;
  int32_t n;
};

__global__ void __launch_bounds__(256) quantize_batch_kernel(const __grid_constant__ BatchArgs a) {
  pdl_prologue();
  Counts unused;
  // Chunks come in increasing order, so the search for a chunk's tensor only moves forward; the
  // tensor's fields are copied to registers when it changes, not once per chunk (they sit in an
  // array of the kernel's parameters, which a varying index can only reach through loads).
  int t = -1;
  const float4* x = nullptr;
  QuantOut o{};
  unsigned long long n4 = 0, first = 0;
  float scale = 1.0f;
  int32_t qmin = 0, qmax = 0;
  for (unsigned long long chunk = blockIdx.x; chunk < a.total_chunks; chunk += gridDim.x) {
    int nt = t < 0 ? 0 : t;
    while (nt + 1 < a.n && a.item[nt + 1].first_chunk <= chunk) ++nt;
    if (nt != t) {
      t = nt;
      const BatchItem& it = a.item[t];
      x = it.x;
      o.hi = it.hi; o.lo = it.lo; o.q16 = it.q16; o.planes = it.planes;
      n4 = it.n4;
      first = it.first_chunk;
      scale = scale_of(it.d_fmt != nullptr ? it.d_fmt->frac_bits : it.frac_bits);
      qmin = it.qmin;
      qmax = it.qmax;
    }
    const unsigned long long base = (chunk - first) * kBatchChunk4 + threadIdx.x;
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const unsigned long long i = base + u * 256;
      v[u] = i < n4 ? __ldcs(x + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const unsigned long long i = base + u * 256;
      if (i < n4) {
        int32_t q[4];
        quantize_f32x4(v[u], scale, 0, qmin, qmax, unused, q);
        store4(o, (size_t)i, q[0], q[1], q[2], q[3]);
      }
    }
  }
}

int quantize_batch_impl(const adaption_quantize_item* h_items, int32_t n_items, cudaStream_t stream) {
  if (n_items < 0 || (n_items > 0 && h_items == nullptr)) return ADAPTION_ERR_INVALID_ARG;
  // validate everything before the first launch
  for (int32_t k = 0; k < n_items; ++k) {
    const adaption_quantize_item& h = h_items[k];
    if (h.outer < 0 || h.inner < 0) return ADAPTION_ERR_INVALID_ARG;
    int rc = check_qtensor_out(h.q, h.inner);
    if (rc != ADAPTION_OK) return rc;
    if (h.outer == 0 || h.inner == 0) continue;
    if (h.d_x == nullptr) return ADAPTION_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(h.d_x) & 3u) != 0) return ADAPTION_ERR_ALIGNMENT;
  }
  BatchArgs args;
  args.n = 0;
  args.total_chunks = 0;
  auto flush = [&]() -> int {
    if (args.n == 0) return ADAPTION_OK;
    const int grid = stream_grid((size_t)args.total_chunks, 1, 8);
    launch_after_predecessor(quantize_batch_kernel, dim3(grid), dim3(256), stream, args);
    args.n = 0;
    args.total_chunks = 0;
    return cuda_status(cudaGetLastError());
  };
  for (int32_t k = 0; k < n_items; ++k) {
    const adaption_quantize_item& h = h_items[k];
    if (h.outer == 0 || h.inner == 0) continue;
    const bool dense = h.inner == h.q.c_stride && aligned16(h.d_x);
    if (!dense) {               // padded rows: the row kernel, on its own
      int rc = quantize_impl(h.d_x, (size_t)h.outer, (size_t)h.inner, h.q, h.d_fmt, 0,
                             ADAPTION_ROUND_DETERMINISTIC, nullptr, stream);
      if (rc != ADAPTION_OK) return rc;
      continue;
    }
    BatchItem& it = args.item[args.n];
    const QuantOut qo = quant_out_of(h.q);
    it.x = reinterpret_cast<const float4*>(h.d_x);
    it.hi = qo.hi; it.lo = qo.lo; it.q16 = qo.q16; it.planes = qo.planes;
    it.d_fmt = h.d_fmt;
    it.n4 = (unsigned long long)h.outer * (unsigned long long)h.inner / 4;   // c_stride is a multiple of 16
    it.first_chunk = args.total_chunks;
    it.frac_bits = h.q.fmt.frac_bits;
    it.qmin = -(1 << (h.q.fmt.n_bits - 1));
    it.qmax = (1 << (h.q.fmt.n_bits - 1)) - 1;
    args.total_chunks += (it.n4 + kBatchChunk4 - 1) / kBatchChunk4;
    if (++args.n == kBatchItems) {
      int rc = flush();
      if (rc != ADAPTION_OK) return rc;
    }
  }
  return flush();
}

int requant_impl(const adaption_qtensor& in, size_t outer, size_t inner, int32_t relu,
                 const adaption_qtensor& out, const adaption_qfmt* d_fmt, int32_t rounding,
                 adaption_stats* d_stats, cudaStream_t stream) {
  if (rounding == ADAPTION_ROUND_STOCHASTIC) return ADAPTION_ERR_UNSUPPORTED;
  if (rounding != ADAPTION_ROUND_DETERMINISTIC) return ADAPTION_ERR_INVALID_ARG;
  int rc = check_qtensor_in(in, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  rc = check_qtensor_out(out, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  if (outer == 0 || inner == 0) return ADAPTION_OK;
  RequantParams rq = make_requant(in.fmt.frac_bits, out.fmt, relu);
  if ((int64_t)inner == in.c_stride && in.c_stride == out.c_stride && out.q16 == nullptr) {
    const size_t n16 = outer * inner / 16;
    const int grid = stream_grid((n16 + 1) / 2, 256, 8);
    if (in.fmt.n_bits > 8)
      requant_flat_kernel<true><<<grid, 256, 0, stream>>>(
          reinterpret_cast<const uint4*>(in.hi), reinterpret_cast<const uint4*>(in.lo), n16,
          reinterpret_cast<uint4*>(out.hi), reinterpret_cast<uint4*>(out.lo), in.fmt.frac_bits,
          out.fmt.frac_bits, d_fmt, rq, d_stats);
    else
      requant_flat_kernel<false><<<grid, 256, 0, stream>>>(
          nullptr, reinterpret_cast<const uint4*>(in.lo), n16, reinterpret_cast<uint4*>(out.hi),
          reinterpret_cast<uint4*>(out.lo), in.fmt.frac_bits, out.fmt.frac_bits, d_fmt, rq, d_stats);
    return cuda_status(cudaGetLastError());
  }
  const size_t groups = outer * (size_t)(out.c_stride / 4);
  const int grid = stream_grid(groups, 256, 8);
  requant_rows_kernel<<<grid, 256, 0, stream>>>(
      in.fmt.n_bits > 8 ? reinterpret_cast<const uint32_t*>(in.hi) : nullptr,
      reinterpret_cast<const uint32_t*>(in.lo), in.c_stride, outer, (int64_t)inner, out.c_stride,
      quant_out_of(out), in.fmt.frac_bits, out.fmt.frac_bits, d_fmt, rq, d_stats);
  return cuda_status(cudaGetLastError());
}

int measure_range_impl(const float* d_x, size_t numel, int32_t n_bits, float* d_max_abs,
                       adaption_qfmt* d_fmt_out, cudaStream_t stream) {
  if (n_bits < 1 || n_bits > 16 || d_max_abs == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if (numel > 0 && d_x == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_x) & 3u) != 0 || (reinterpret_cast<uintptr_t>(d_max_abs) & 3u) != 0)
    return ADAPTION_ERR_ALIGNMENT;
  if (numel > 0) {
    size_t head = ((16 - (reinterpret_cast<uintptr_t>(d_x) & 15u)) & 15u) / 4;
    if (head > numel) head = numel;
    const size_t n4 = (numel - head) / 4;
    int grid = stream_grid((n4 + 3) / 4 + 4, 256, 8);
    launch_after_predecessor(range_max_abs_kernel, dim3(grid), dim3(256), stream, d_x, numel, head, n4, d_max_abs);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return ADAPTION_ERR_CUDA;
  }
  if (d_fmt_out != nullptr)
    launch_after_predecessor(choose_fmt_kernel, dim3(1), dim3(1), stream, (const float*)d_max_abs, n_bits, d_fmt_out);
  return cuda_status(cudaGetLastError());
}

// half_pooled: x already holds the horizontal maxima (N x H x W/2 pixels); only rows are paired.
int maxpool_impl(const adaption_qtensor& x, int32_t N, int32_t H, int32_t W, int32_t C,
                 const adaption_qtensor& y, cudaStream_t stream, bool half_pooled) {
  if (N < 0 || H < 0 || W < 0 || C < 0 || (H & 1) || (W & 1)) return ADAPTION_ERR_INVALID_ARG;
  int rc = check_qtensor_in(x, C);
  if (rc != ADAPTION_OK) return rc;
  rc = check_qtensor_out(y, C);
  if (rc != ADAPTION_OK) return rc;
  if (x.fmt.n_bits != y.fmt.n_bits || x.fmt.frac_bits != y.fmt.frac_bits) return ADAPTION_ERR_INVALID_ARG;
  const size_t total = (size_t)N * (H / 2) * (W / 2) * (size_t)(y.c_stride / 16);
  if (total == 0) return ADAPTION_OK;
  const bool two = x.fmt.n_bits > 8;
  const int grid = stream_grid(total, 256, 8);
  const uint4* xh = two ? reinterpret_cast<const uint4*>(x.hi) : nullptr;
  const uint4* xl = reinterpret_cast<const uint4*>(x.lo);
  uint4* yh = two ? reinterpret_cast<uint4*>(y.hi) : nullptr;
  uint4* yl = reinterpret_cast<uint4*>(y.lo);
  const int Win = half_pooled ? W / 2 : W, kw = half_pooled ? 1 : 2;
  const int64_t in_vecs = x.c_stride / 16, out_vecs = y.c_stride / 16;
  // 32-bit indices while every input vector index and the loop counter plus one grid stride fit
  const unsigned long long in_total = (unsigned long long)N * H * Win * (unsigned long long)in_vecs;
  const unsigned long long limit = (1ull << 32) - (unsigned long long)grid * 256ull;
  if (in_total < limit && (unsigned long long)total < limit)
    launch_after_predecessor(maxpool2x2_kernel<uint32_t>, dim3(grid), dim3(256), stream, xh, xl, yh, yl, y.q16, N, H, Win, kw,
                             in_vecs, out_vecs);
  else
    launch_after_predecessor(maxpool2x2_kernel<unsigned long long>, dim3(grid), dim3(256), stream, xh, xl, yh, yl, y.q16, N, H, Win, kw, in_vecs,
                                                                    out_vecs);
  return cuda_status(cudaGetLastError());
}

}  // namespace adaption
