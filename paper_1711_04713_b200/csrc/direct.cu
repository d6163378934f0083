// Plain integer kernels for LPConvolution / LPInnerProduct (paper Sec. 2): one thread per output
// element, exact int64 accumulation, any shape.  They serve shapes the tensor-core path does not
// take (channel pitch not a multiple of 32, reductions beyond its int32-safe length) and the
// forced ADAPTION_ALGO_DIRECT mode.  Also the shared finalize kernel that turns an int64
// accumulator matrix (split-K workspace) into the requantized output.
#include "common.cuh"

namespace adaption {

int num_sms();

struct DirectParams {
  int64_t M, N, K;              // K: reduction length for the inner product
  int is_conv;
  int H, W, C, R, S, OH, OW, pad_h, pad_w, stride_h, stride_w;
  const int8_t* x_hi; const uint8_t* x_lo; int64_t x_stride;
  const int8_t* w_hi; const uint8_t* w_lo; int64_t w_stride;
  const int16_t* bias; int32_t bias_shift;
  int8_t* y_hi; uint8_t* y_lo; int16_t* y_q16; int64_t y_stride;
  RequantParams rq;
  StochasticParams st;
  int mode;
  adaption_stats* stats;
};

__device__ __forceinline__ int64_t dot_row(const int8_t* __restrict__ ah, const uint8_t* __restrict__ al,
                                           const int8_t* __restrict__ bh, const uint8_t* __restrict__ bl,
                                           int64_t len, int64_t acc) {
  for (int64_t i = 0; i < len; ++i) {
    const int32_t a = load_q(ah, al, (size_t)i);
    const int32_t b = load_q(bh, bl, (size_t)i);
    acc += (int64_t)a * (int64_t)b;
  }
  return acc;
}

__global__ void __launch_bounds__(256) direct_kernel(DirectParams p) {
  pdl_prologue();
  const int64_t cols = p.mode == ADAPTION_MODE_RANGE ? p.N : p.y_stride;
  const size_t total = (size_t)p.M * (size_t)cols;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  Counts c;
  int64_t vmax = 0;
  for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += nthreads) {
    const int64_t m = (int64_t)(t / (size_t)cols);
    const int64_t n = (int64_t)(t % (size_t)cols);
    const bool real = n < p.N;
    int64_t acc = 0;
    if (real) {
      if (p.is_conv) {
        const int ow = (int)(m % p.OW);
        const int oh = (int)((m / p.OW) % p.OH);
        const int64_t img = m / ((int64_t)p.OW * p.OH);
        for (int r = 0; r < p.R; ++r) {
          const int ih = oh * p.stride_h + r - p.pad_h;
          if (ih < 0 || ih >= p.H) continue;
          for (int s = 0; s < p.S; ++s) {
            const int iw = ow * p.stride_w + s - p.pad_w;
            if (iw < 0 || iw >= p.W) continue;
            const size_t xo = (((size_t)img * p.H + ih) * p.W + iw) * (size_t)p.x_stride;
            const size_t wo = (((size_t)n * p.R + r) * p.S + s) * (size_t)p.w_stride;
            acc = dot_row(p.x_hi ? p.x_hi + xo : nullptr, p.x_lo + xo, p.w_hi ? p.w_hi + wo : nullptr,
                          p.w_lo + wo, p.C, acc);
          }
        }
      } else {
        const size_t xo = (size_t)m * (size_t)p.x_stride, wo = (size_t)n * (size_t)p.w_stride;
        acc = dot_row(p.x_hi ? p.x_hi + xo : nullptr, p.x_lo + xo, p.w_hi ? p.w_hi + wo : nullptr,
                      p.w_lo + wo, p.K, acc);
      }
      if (p.bias != nullptr) acc += (int64_t)p.bias[n] * ((int64_t)1 << p.bias_shift);
    }
    if (p.mode == ADAPTION_MODE_RANGE) {
      if (p.rq.relu && acc < 0) acc = 0;
      const int64_t a = acc < 0 ? -acc : acc;
      vmax = a > vmax ? a : vmax;
    } else {
      const int32_t q = (p.st.enabled && real)
                            ? requant_value_stochastic(acc, p.rq, philox_draw((uint64_t)m * (uint64_t)p.N + (uint64_t)n,
                                                                              p.st.key0, p.st.key1), real, c)
                            : requant_value(acc, p.rq, real, c);
      store_q(p.rq.out_planes == 2 ? p.y_hi : nullptr, p.y_lo, p.y_q16,
              (size_t)m * (size_t)p.y_stride + (size_t)n, q);
    }
  }
  if (p.mode == ADAPTION_MODE_RANGE)
    flush_max_warp(vmax, p.stats);
  else
    flush_counts_warp(c, p.stats);
}

struct FinalizeParams {
  const int64_t* acc; int64_t ld;
  int64_t M, N;
  const int16_t* bias; int32_t bias_shift;
  uint32_t* y_hi; uint32_t* y_lo; uint2* y_q16; int64_t y_stride;
  RequantParams rq;
  StochasticParams st;
  int mode;
  adaption_stats* stats;
};

// one thread per four consecutive output columns
__global__ void __launch_bounds__(256) finalize_kernel(FinalizeParams p) {
  pdl_prologue();
  const int64_t groups_per_row = (p.mode == ADAPTION_MODE_RANGE ? (p.N + 3) / 4 : p.y_stride / 4);
  const size_t total = (size_t)p.M * (size_t)groups_per_row;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  Counts c;
  int64_t vmax = 0;
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += nthreads) {
    const int64_t m = (int64_t)(g / (size_t)groups_per_row);
    const int64_t n0 = (int64_t)(g % (size_t)groups_per_row) * 4;
    int32_t q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t n = n0 + u;
      const bool real = n < p.N;
      int64_t v = 0;
      if (real) {
        v = p.acc[(size_t)m * (size_t)p.ld + (size_t)n];
        if (p.bias != nullptr) v += (int64_t)p.bias[n] * ((int64_t)1 << p.bias_shift);
      }
      if (p.mode == ADAPTION_MODE_RANGE) {
        if (p.rq.relu && v < 0) v = 0;
        const int64_t a = v < 0 ? -v : v;
        vmax = a > vmax ? a : vmax;
        q[u] = 0;
      } else {
        q[u] = (p.st.enabled && real)
                   ? requant_value_stochastic(v, p.rq, philox_draw((uint64_t)m * (uint64_t)p.N + (uint64_t)n,
                                                                   p.st.key0, p.st.key1), real, c)
                   : requant_value(v, p.rq, real, c);
      }
    }
    if (p.mode != ADAPTION_MODE_RANGE) {
      const size_t word = ((size_t)m * (size_t)p.y_stride + (size_t)n0) / 4;
      p.y_lo[word] = (uint32_t)(q[0] & 255) | ((uint32_t)(q[1] & 255) << 8) |
                     ((uint32_t)(q[2] & 255) << 16) | ((uint32_t)(q[3] & 255) << 24);
      if (p.rq.out_planes == 2)
        p.y_hi[word] = (uint32_t)((q[0] >> 8) & 255) | ((uint32_t)((q[1] >> 8) & 255) << 8) |
                       ((uint32_t)((q[2] >> 8) & 255) << 16) | ((uint32_t)((q[3] >> 8) & 255) << 24);
      if (p.y_q16 != nullptr) {
        uint2 v;
        v.x = (uint32_t)(q[0] & 0xffff) | ((uint32_t)(q[1] & 0xffff) << 16);
        v.y = (uint32_t)(q[2] & 0xffff) | ((uint32_t)(q[3] & 0xffff) << 16);
        p.y_q16[word] = v;
      }
    }
  }
  if (p.mode == ADAPTION_MODE_RANGE)
    flush_max_warp(vmax, p.stats);
  else
    flush_counts_warp(c, p.stats);
}

static int grid_for(size_t items) {
  size_t want = (items + 255) / 256;
  size_t cap = (size_t)num_sms() * 8;
  if (want < 1) want = 1;
  return (int)(want < cap ? want : cap);
}

int launch_direct(const GemmProblem& g) {
  DirectParams p{};
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.is_conv = g.is_conv ? 1 : 0;
  if (g.is_conv) {
    p.H = g.cs.H; p.W = g.cs.W; p.C = g.cs.C; p.R = g.cs.R; p.S = g.cs.S;
    p.OH = g.OH; p.OW = g.OW; p.pad_h = g.cs.pad_h; p.pad_w = g.cs.pad_w;
    p.stride_h = g.cs.stride_h; p.stride_w = g.cs.stride_w;
  }
  p.x_hi = g.x.fmt.n_bits > 8 ? (const int8_t*)g.x.hi : nullptr;
  p.x_lo = (const uint8_t*)g.x.lo; p.x_stride = g.x.c_stride;
  p.w_hi = g.w.fmt.n_bits > 8 ? (const int8_t*)g.w.hi : nullptr;
  p.w_lo = (const uint8_t*)g.w.lo; p.w_stride = g.w.c_stride;
  p.bias = g.bias; p.bias_shift = g.bias_shift;
  p.mode = g.mode; p.stats = g.stats;
  p.st = g.stochastic;
  if (g.mode == ADAPTION_MODE_REQUANT) {
    p.rq = make_requant(g.acc_frac_bits, g.y.fmt, g.relu);
    p.y_hi = (int8_t*)g.y.hi; p.y_lo = (uint8_t*)g.y.lo; p.y_q16 = g.y.q16; p.y_stride = g.y.c_stride;
  } else {
    p.rq = RequantParams{0, g.relu ? 1 : 0, 0, 0, 1};
  }
  const size_t items = (size_t)g.M * (size_t)(g.mode == ADAPTION_MODE_RANGE ? g.N : g.y.c_stride);
  if (items == 0) return ADAPTION_OK;
  launch_after_predecessor(direct_kernel, dim3(grid_for(items)), dim3(256), g.stream, p);
  return cuda_status(cudaGetLastError());
}

int launch_finalize(const int64_t* acc, int64_t ld, const GemmProblem& g) {
  FinalizeParams p{};
  p.acc = acc; p.ld = ld; p.M = g.M; p.N = g.N;
  p.bias = g.bias; p.bias_shift = g.bias_shift;
  p.mode = g.mode; p.stats = g.stats;
  p.st = g.stochastic;
  if (g.mode == ADAPTION_MODE_REQUANT) {
    p.rq = make_requant(g.acc_frac_bits, g.y.fmt, g.relu);
    p.y_hi = (uint32_t*)g.y.hi; p.y_lo = (uint32_t*)g.y.lo; p.y_q16 = (uint2*)g.y.q16;
    p.y_stride = g.y.c_stride;
  } else {
    p.rq = RequantParams{0, g.relu ? 1 : 0, 0, 0, 1};
  }
  const size_t items =
      (size_t)g.M * (size_t)(g.mode == ADAPTION_MODE_RANGE ? (g.N + 3) / 4 : g.y.c_stride / 4);
  if (items == 0) return ADAPTION_OK;
  launch_after_predecessor(finalize_kernel, dim3(grid_for(items)), dim3(256), g.stream, p);
  return cuda_status(cudaGetLastError());
}

}  // namespace adaption
