// Statistics behind the thresholded integer-bit allocation (paper Sec. 2.3: with the total width
// fixed, give bits of the integer part to the fraction while the share of values that can no
// longer be represented stays within a user threshold) and the width statistic of quantized
// tensors (Sec. 2.2: how many 16-bit weights fit 4 or 8 bits).
//
// Both are one streaming pass that sorts every element into ADAPTION_HIST_BINS bins:
//   fp32 tensor:      bin b = integer bits |x| needs, b = 0 for |x| < 1, else floor(log2|x|) + 1,
//                     read from the binary exponent; 16 and more (and +-Inf) share the top bin,
//                     NaN is skipped
//   fixed-point tensor: bin w = two's complement width of q, smallest w >= 1 with
//                     -2^(w-1) <= q < 2^(w-1)
// Every thread counts into a private histogram in shared memory (bin-major, so that the lanes of a
// warp touch distinct banks and nothing is atomic); a block ends with one reduction over its
// threads and one global atomic per non-empty bin.  HBM bound: 4 (resp. 2 or 1) bytes per element.
#include "common.cuh"

namespace adaption {

int num_sms();

namespace {

constexpr int kBins = ADAPTION_HIST_BINS;
constexpr int kWarps = 8;

__device__ __forceinline__ int bits_of_f32(float x, bool& valid) {
  const uint32_t u = __float_as_uint(x) & 0x7fffffffu;
  valid = u <= 0x7f800000u;                    // not NaN
  const int e = (int)(u >> 23) - 127;          // |x| in [2^e, 2^(e+1)); Inf: e = 128
  const int b = e >= 0 ? e + 1 : 0;
  return b < kBins - 1 ? b : kBins - 1;
}

__device__ __forceinline__ int width_of_q(int32_t q) {
  const uint32_t mag = (uint32_t)(q >= 0 ? q : -q - 1);      // q >= 0: q < 2^(w-1); q < 0: -q-1 < 2^(w-1)
  return 33 - __clz((int)mag);                               // bit length of mag, plus the sign bit
}

constexpr int kThreadsHist = 32 * kWarps;

// private counters: hist[bin][thread]
struct PrivateHist {
  uint32_t c[kBins][kThreadsHist];
};

__device__ __forceinline__ void hist_clear(PrivateHist& h) {
#pragma unroll
  for (int b = 0; b < kBins; ++b) h.c[b][threadIdx.x] = 0u;
}

__device__ __forceinline__ void block_flush(PrivateHist& h, unsigned long long* d_hist) {
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int b = warp; b < kBins; b += kWarps) {
    unsigned long long s = 0;
    for (int t = lane; t < kThreadsHist; t += 32) s += h.c[b][t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0 && s) atomicAdd(d_hist + b, s);
  }
}

__device__ __forceinline__ void count_f32(PrivateHist& h, float x) {
  bool valid;
  const int b = bits_of_f32(x, valid);
  if (valid) h.c[b][threadIdx.x] += 1u;
}

// head: elements before the first 16-byte boundary, then n4 float4, then the tail
__global__ void __launch_bounds__(kThreadsHist) bit_histogram_kernel(const float* __restrict__ x, size_t numel,
                                                                     size_t head, size_t n4,
                                                                     unsigned long long* __restrict__ d_hist) {
  __shared__ PrivateHist h;
  hist_clear(h);
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const float4* __restrict__ x4 = reinterpret_cast<const float4*>(x + head);
  size_t i = tid;
  for (; i + nthreads < n4; i += 2 * nthreads) {
    const float4 a = __ldcs(x4 + i), b = __ldcs(x4 + i + nthreads);
    count_f32(h, a.x); count_f32(h, a.y); count_f32(h, a.z); count_f32(h, a.w);
    count_f32(h, b.x); count_f32(h, b.y); count_f32(h, b.z); count_f32(h, b.w);
  }
  for (; i < n4; i += nthreads) {
    const float4 a = __ldcs(x4 + i);
    count_f32(h, a.x); count_f32(h, a.y); count_f32(h, a.z); count_f32(h, a.w);
  }
  const size_t tail0 = head + 4 * n4;
  for (size_t j = tid; j < head + (numel - tail0); j += nthreads)
    count_f32(h, x[j < head ? j : tail0 + (j - head)]);
  block_flush(h, d_hist);
}

// sixteen stored elements (one 16-byte vector per plane) per thread and step
__global__ void __launch_bounds__(kThreadsHist) width_histogram_kernel(const uint4* __restrict__ hi,
                                                                       const uint4* __restrict__ lo, size_t outer,
                                                                       int64_t inner, int64_t c_stride,
                                                                       unsigned long long* __restrict__ d_hist) {
  __shared__ PrivateHist h;
  hist_clear(h);
  const int64_t groups_per_row = c_stride / 16;
  const size_t total = outer * (size_t)groups_per_row;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += nthreads) {
    const int64_t c0 = (int64_t)(g % (size_t)groups_per_row) * 16;
    const int nreal = (int)min((int64_t)16, max((int64_t)0, inner - c0));     // padding channels are not counted
    const uint4 l = __ldcs(lo + g);
    const uint4 u = hi != nullptr ? __ldcs(hi + g) : make_uint4(0, 0, 0, 0);
    const uint32_t lw[4] = {l.x, l.y, l.z, l.w}, hw[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const int32_t l8 = (lw[e >> 2] >> (8 * (e & 3))) & 255;
      const int32_t q = hi != nullptr ? ((int32_t)(int8_t)((hw[e >> 2] >> (8 * (e & 3))) & 255)) * 256 + l8
                                      : (int32_t)(int8_t)l8;
      if (e < nreal) h.c[width_of_q(q)][threadIdx.x] += 1u;
    }
  }
  block_flush(h, d_hist);
}

int grid_for(size_t items) {
  size_t want = (items + 32 * kWarps - 1) / (32 * kWarps);
  const size_t cap = (size_t)num_sms() * 8;
  if (want < 1) want = 1;
  return (int)(want < cap ? want : cap);
}

}  // namespace

int bit_histogram_impl(const float* d_x, size_t numel, uint64_t* d_hist, cudaStream_t stream) {
  if (d_hist == nullptr || (numel > 0 && d_x == nullptr)) return ADAPTION_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_x) & 3u) != 0 || (reinterpret_cast<uintptr_t>(d_hist) & 7u) != 0)
    return ADAPTION_ERR_ALIGNMENT;
  if (numel == 0) return ADAPTION_OK;
  size_t head = ((16 - (reinterpret_cast<uintptr_t>(d_x) & 15u)) & 15u) / 4;
  if (head > numel) head = numel;
  const size_t n4 = (numel - head) / 4;
  bit_histogram_kernel<<<grid_for(n4 / 2 + 64), 32 * kWarps, 0, stream>>>(
      d_x, numel, head, n4, reinterpret_cast<unsigned long long*>(d_hist));
  return cuda_status(cudaGetLastError(), "bit_histogram_kernel launch");
}

int width_histogram_impl(const adaption_qtensor& x, size_t outer, size_t inner, uint64_t* d_hist,
                         cudaStream_t stream) {
  if (d_hist == nullptr) return ADAPTION_ERR_INVALID_ARG;
  const int rc = check_qtensor_in(x, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  if ((reinterpret_cast<uintptr_t>(d_hist) & 7u) != 0) return ADAPTION_ERR_ALIGNMENT;
  if (outer == 0 || inner == 0) return ADAPTION_OK;
  width_histogram_kernel<<<grid_for(outer * (size_t)(x.c_stride / 16)), 32 * kWarps, 0, stream>>>(
      x.fmt.n_bits > 8 ? static_cast<const uint4*>(x.hi) : nullptr, static_cast<const uint4*>(x.lo), outer,
      (int64_t)inner, x.c_stride, reinterpret_cast<unsigned long long*>(d_hist));
  return cuda_status(cudaGetLastError(), "width_histogram_kernel launch");
}

// Host: the allocation itself.  Starts with all n - 1 non-sign bits in the integer part and moves
// bits to the fraction while the values that would no longer fit stay within threshold * total.
int choose_frac_bits_from_hist(const uint64_t* h_hist, int32_t n_bits, double threshold, adaption_qfmt* h_out) {
  if (h_hist == nullptr || h_out == nullptr || n_bits < 1 || n_bits > 16 || !(threshold >= 0.0) || threshold > 1.0)
    return ADAPTION_ERR_INVALID_ARG;
  // (counts are compared in double precision: exact below 2^53 elements)
  uint64_t total = 0;
  for (int b = 0; b < kBins; ++b) total += h_hist[b];
  const double allowed = threshold * (double)total;
  int m = n_bits - 1;
  while (m > 0) {
    uint64_t lost = 0;                          // values that need more than m - 1 integer bits
    for (int b = m; b < kBins; ++b) lost += h_hist[b];
    if ((double)lost > allowed) break;
    --m;
  }
  h_out->n_bits = n_bits;
  h_out->frac_bits = n_bits - 1 - m;
  return ADAPTION_OK;
}

// Host: the same allocation for a tensor already stored with `frac_bits` fractional bits, from the
// histogram of its two's complement widths: q keeps its value with m integer bits iff its width is
// at most m + frac_bits + 1.
int choose_frac_bits_from_widths(const uint64_t* h_hist, int32_t frac_bits, int32_t n_bits, double threshold,
                                 adaption_qfmt* h_out) {
  if (h_hist == nullptr || frac_bits < 0 || frac_bits > 15) return ADAPTION_ERR_INVALID_ARG;
  uint64_t need[kBins];                 // need[b]: values that need b integer bits
  for (int b = 0; b < kBins; ++b) need[b] = 0;
  for (int w = 0; w < kBins; ++w) {
    int b = w - 1 - frac_bits;
    if (b < 0) b = 0;
    need[b] += h_hist[w];
  }
  return choose_frac_bits_from_hist(need, n_bits, threshold, h_out);
}

}  // namespace adaption
