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
// Lanes of a warp that hit the same bin are grouped with a match instruction and one of them adds
// the group's size to the warp's private histogram in shared memory (no atomics there); a block
// ends with one global atomic per non-empty bin.  HBM bound: 4 (resp. 2 or 1) bytes per element.
#include "common.cuh"

namespace adaption {

int num_sms();

namespace {

constexpr int kBins = ADAPTION_HIST_BINS;
constexpr int kWarps = 8;

__device__ __forceinline__ void warp_bin_add(uint32_t* hist, int bin, bool valid) {
  const unsigned active = __ballot_sync(0xffffffffu, valid);
  if (!valid) return;
  const unsigned peers = __match_any_sync(active, bin);
  if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) hist[bin] += (uint32_t)__popc(peers);
}

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

__device__ __forceinline__ void block_flush(uint32_t (*wh)[kBins], unsigned long long* d_hist) {
  __syncthreads();
  if (threadIdx.x < kBins) {
    unsigned long long s = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) s += wh[w][threadIdx.x];
    if (s) atomicAdd(d_hist + threadIdx.x, s);
  }
}

__global__ void __launch_bounds__(32 * kWarps) bit_histogram_kernel(const float* __restrict__ x, size_t numel,
                                                                    unsigned long long* __restrict__ d_hist) {
  __shared__ uint32_t wh[kWarps][kBins];
  for (int i = threadIdx.x; i < kWarps * kBins; i += blockDim.x) (&wh[0][0])[i] = 0u;
  __syncthreads();
  uint32_t* mine = wh[threadIdx.x >> 5];
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  // whole warps walk the array together (the match needs converged lanes); the tail is masked
  const size_t rounds = (numel + nthreads - 1) / nthreads;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (size_t r = 0; r < rounds; ++r, i += nthreads) {
    bool valid = false;
    int b = 0;
    if (i < numel) b = bits_of_f32(__ldcs(x + i), valid);
    warp_bin_add(mine, b, valid);
    __syncwarp();
  }
  block_flush(wh, d_hist);
}

__global__ void __launch_bounds__(32 * kWarps) width_histogram_kernel(const int8_t* __restrict__ hi,
                                                                      const uint8_t* __restrict__ lo, size_t outer,
                                                                      int64_t inner, int64_t c_stride,
                                                                      unsigned long long* __restrict__ d_hist) {
  __shared__ uint32_t wh[kWarps][kBins];
  for (int i = threadIdx.x; i < kWarps * kBins; i += blockDim.x) (&wh[0][0])[i] = 0u;
  __syncthreads();
  uint32_t* mine = wh[threadIdx.x >> 5];
  const size_t total = outer * (size_t)c_stride;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  const size_t rounds = (total + nthreads - 1) / nthreads;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (size_t r = 0; r < rounds; ++r, i += nthreads) {
    bool valid = false;
    int w = 0;
    if (i < total && (int64_t)(i % (size_t)c_stride) < inner) {     // padding channels are not counted
      valid = true;
      w = width_of_q(load_q(hi, lo, i));
    }
    warp_bin_add(mine, w, valid);
    __syncwarp();
  }
  block_flush(wh, d_hist);
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
  bit_histogram_kernel<<<grid_for(numel), 32 * kWarps, 0, stream>>>(
      d_x, numel, reinterpret_cast<unsigned long long*>(d_hist));
  return cuda_status(cudaGetLastError(), "bit_histogram_kernel launch");
}

int width_histogram_impl(const adaption_qtensor& x, size_t outer, size_t inner, uint64_t* d_hist,
                         cudaStream_t stream) {
  if (d_hist == nullptr) return ADAPTION_ERR_INVALID_ARG;
  const int rc = check_qtensor_in(x, (int64_t)inner);
  if (rc != ADAPTION_OK) return rc;
  if ((reinterpret_cast<uintptr_t>(d_hist) & 7u) != 0) return ADAPTION_ERR_ALIGNMENT;
  if (outer == 0 || inner == 0) return ADAPTION_OK;
  width_histogram_kernel<<<grid_for(outer * (size_t)x.c_stride), 32 * kWarps, 0, stream>>>(
      x.fmt.n_bits > 8 ? static_cast<const int8_t*>(x.hi) : nullptr, static_cast<const uint8_t*>(x.lo), outer,
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

}  // namespace adaption
