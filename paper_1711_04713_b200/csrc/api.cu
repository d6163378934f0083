// extern "C" entry points: argument validation and dispatch.  See include/adaption.h.
#include <cstdio>
#include <cstdlib>

#include "common.cuh"

namespace adaption {
int cuda_failure(cudaError_t e, const char* where) {
  if (std::getenv("ADAPTION_LOG") != nullptr)
    std::fprintf(stderr, "adaption: CUDA error at %s: %s\n", where, cudaGetErrorString(e));
  return ADAPTION_ERR_CUDA;
}

int quantize_impl(const float*, size_t, size_t, const adaption_qtensor&, const adaption_qfmt*, int32_t,
                  int32_t, adaption_stats*, cudaStream_t);
int quantize_batch_impl(const adaption_quantize_item*, int32_t, cudaStream_t);
int requant_impl(const adaption_qtensor&, size_t, size_t, int32_t, const adaption_qtensor&,
                 const adaption_qfmt*, int32_t, adaption_stats*, cudaStream_t);
int measure_range_impl(const float*, size_t, int32_t, float*, adaption_qfmt*, cudaStream_t);
int maxpool_impl(const adaption_qtensor&, int32_t, int32_t, int32_t, int32_t, const adaption_qtensor&,
                 cudaStream_t, bool half_pooled = false);

int quantize_stochastic_impl(const float*, size_t, size_t, const adaption_qtensor&, const adaption_qfmt*, int32_t,
                             uint64_t, adaption_stats*, cudaStream_t);
int requant_stochastic_impl(const adaption_qtensor&, size_t, size_t, int32_t, const adaption_qtensor&,
                            const adaption_qfmt*, uint64_t, adaption_stats*, cudaStream_t);
int bit_histogram_impl(const float*, size_t, uint64_t*, cudaStream_t);
int width_histogram_impl(const adaption_qtensor&, size_t, size_t, uint64_t*, cudaStream_t);
int choose_frac_bits_from_hist(const uint64_t*, int32_t, double, adaption_qfmt*);
int choose_frac_bits_from_widths(const uint64_t*, int32_t, int32_t, double, adaption_qfmt*);

int probe_i8_peak(int bn, int pair, int iters, int commit_every, unsigned long long* d_cycles, int* d_status,
                  cudaStream_t stream);
int num_sms();
int debug_set(const char* name, int value);

// Longest reduction the direct kernels and the int64 workspace can take without overflow:
// |q_x * q_w| <= 2^30, so 2^31 terms still leave a sign bit and headroom for the bias.
static const int64_t kMaxReduction = (int64_t)1 << 31;

static int build_conv_problem(const adaption_conv_shape* s, const adaption_qtensor& x,
                              const adaption_qtensor& w, const int16_t* bias, int32_t bias_frac_bits,
                              int32_t relu, int32_t mode, const adaption_qtensor& y,
                              adaption_stats* stats, void* ws, size_t ws_bytes, void* stream,
                              GemmProblem& g) {
  if (s == nullptr) return ADAPTION_ERR_INVALID_ARG;
  if (s->N < 0 || s->H <= 0 || s->W <= 0 || s->C <= 0 || s->K <= 0 || s->R <= 0 || s->S <= 0 ||
      s->pad_h < 0 || s->pad_w < 0 || s->stride_h <= 0 || s->stride_w <= 0)
    return ADAPTION_ERR_INVALID_ARG;
  if (s->H + 2 * s->pad_h < s->R || s->W + 2 * s->pad_w < s->S) return ADAPTION_ERR_INVALID_ARG;
  if (mode != ADAPTION_MODE_REQUANT && mode != ADAPTION_MODE_RANGE) return ADAPTION_ERR_INVALID_ARG;
  int rc = check_qtensor_in(x, s->C);
  if (rc != ADAPTION_OK) return rc;
  rc = check_qtensor_in(w, s->C);
  if (rc != ADAPTION_OK) return rc;
  if (x.c_stride != w.c_stride) return ADAPTION_ERR_INVALID_ARG;
  g.is_conv = true;
  g.cs = *s;
  g.OH = (s->H + 2 * s->pad_h - s->R) / s->stride_h + 1;
  g.OW = (s->W + 2 * s->pad_w - s->S) / s->stride_w + 1;
  g.M = (int64_t)s->N * g.OH * g.OW;
  g.N = s->K;
  g.K = (int64_t)s->R * s->S * s->C;
  if (g.K >= kMaxReduction) return ADAPTION_ERR_K_TOO_LARGE;
  g.x = x; g.w = w; g.y = y;
  g.acc_frac_bits = x.fmt.frac_bits + w.fmt.frac_bits;
  g.bias = bias;
  if (bias != nullptr) {
    if (bias_frac_bits < 0 || bias_frac_bits > g.acc_frac_bits) return ADAPTION_ERR_INVALID_ARG;
    g.bias_shift = g.acc_frac_bits - bias_frac_bits;
  }
  g.relu = relu ? 1 : 0;
  g.mode = mode;
  if (stats == nullptr) return ADAPTION_ERR_INVALID_ARG;
  g.stats = stats;
  if (mode == ADAPTION_MODE_REQUANT) {
    rc = check_qtensor_out(y, g.N);
    if (rc != ADAPTION_OK) return rc;
  }
  g.workspace = ws;
  g.workspace_bytes = ws_bytes;
  g.stream = reinterpret_cast<cudaStream_t>(stream);
  return ADAPTION_OK;
}

static int build_ip_problem(int64_t B, int64_t K, int64_t O, const adaption_qtensor& x,
                            const adaption_qtensor& w, const int16_t* bias, int32_t bias_frac_bits,
                            int32_t relu, int32_t mode, const adaption_qtensor& y, adaption_stats* stats,
                            void* ws, size_t ws_bytes, void* stream, GemmProblem& g) {
  if (B < 0 || K <= 0 || O <= 0) return ADAPTION_ERR_INVALID_ARG;
  if (mode != ADAPTION_MODE_REQUANT && mode != ADAPTION_MODE_RANGE) return ADAPTION_ERR_INVALID_ARG;
  if (K >= kMaxReduction) return ADAPTION_ERR_K_TOO_LARGE;
  int rc = check_qtensor_in(x, K);
  if (rc != ADAPTION_OK) return rc;
  rc = check_qtensor_in(w, K);
  if (rc != ADAPTION_OK) return rc;
  g.is_conv = false;
  g.M = B; g.N = O; g.K = K;
  g.x = x; g.w = w; g.y = y;
  g.acc_frac_bits = x.fmt.frac_bits + w.fmt.frac_bits;
  g.bias = bias;
  if (bias != nullptr) {
    if (bias_frac_bits < 0 || bias_frac_bits > g.acc_frac_bits) return ADAPTION_ERR_INVALID_ARG;
    g.bias_shift = g.acc_frac_bits - bias_frac_bits;
  }
  g.relu = relu ? 1 : 0;
  g.mode = mode;
  if (stats == nullptr) return ADAPTION_ERR_INVALID_ARG;
  g.stats = stats;
  if (mode == ADAPTION_MODE_REQUANT) {
    rc = check_qtensor_out(y, O);
    if (rc != ADAPTION_OK) return rc;
  }
  g.workspace = ws;
  g.workspace_bytes = ws_bytes;
  g.stream = reinterpret_cast<cudaStream_t>(stream);
  return ADAPTION_OK;
}

static int dispatch(const GemmProblem& g, int32_t algo) {
  if (algo != ADAPTION_ALGO_AUTO && algo != ADAPTION_ALGO_TENSOR && algo != ADAPTION_ALGO_DIRECT)
    return ADAPTION_ERR_INVALID_ARG;
  if (g.M == 0) return ADAPTION_OK;
  if (algo != ADAPTION_ALGO_DIRECT && pack_taps_applicable(g)) {
    const size_t need = pack_taps_workspace(g);
    if (g.workspace == nullptr || g.workspace_bytes < need) return ADAPTION_ERR_WORKSPACE;
    if (!aligned16(g.workspace)) return ADAPTION_ERR_ALIGNMENT;
    return launch_pack_taps(g);
  }
  const bool tensor_ok = tensor_path_supported(g);
  if (algo == ADAPTION_ALGO_TENSOR && !tensor_ok) return ADAPTION_ERR_UNSUPPORTED;
  if (algo != ADAPTION_ALGO_DIRECT && tensor_ok) {
    const size_t need = tensor_path_workspace(g);
    if (need > 0) {
      if (g.workspace == nullptr || g.workspace_bytes < need) return ADAPTION_ERR_WORKSPACE;
      if (!aligned16(g.workspace)) return ADAPTION_ERR_ALIGNMENT;
    }
    return launch_tensor(g);
  }
  return launch_direct(g);
}

// ---- LPConvolution followed by the 2x2 max-pool of its output -------------------------------
// The convolution's own output goes to temporary planes in the workspace (behind whatever the
// convolution itself needs there): only its horizontal pair maxima when the tensor-core path can
// store those (half the bytes), else all of it; a pooling pass then writes y.
struct ConvPoolPlan {
  bool fused = false;        // the layer kernel stores horizontal maxima
  size_t conv_ws = 0;        // bytes the convolution needs at the start of the workspace
  size_t plane = 0;          // bytes of one temporary plane
  size_t total = 0;
};

static ConvPoolPlan plan_conv_pool(GemmProblem g, int32_t algo) {
  ConvPoolPlan pl;
  const int planes = g.y.fmt.n_bits > 8 ? 2 : 1;
  // a stand-in output of the right shape decides whether the staged (pool-capable) stores apply
  g.y.lo = reinterpret_cast<void*>(uintptr_t(256));
  g.y.hi = planes == 2 ? reinterpret_cast<void*>(uintptr_t(256)) : nullptr;
  g.y.q16 = nullptr;
  const bool packs = algo != ADAPTION_ALGO_DIRECT && pack_taps_applicable(g);
  if (algo != ADAPTION_ALGO_DIRECT) {
    if (packs) {
      pl.conv_ws = pack_taps_workspace(g);
      pl.fused = pack_taps_can_pool(g);
    } else if (tensor_path_supported(g)) {
      pl.conv_ws = tensor_path_workspace(g);
      pl.fused = tensor_path_can_pool(g);
    }
  }
  pl.conv_ws = (pl.conv_ws + 255) & ~(size_t)255;
  const size_t rows = pl.fused ? (size_t)g.M / 2 : (size_t)g.M;
  pl.plane = (rows * (size_t)g.y.c_stride + 255) & ~(size_t)255;
  pl.total = pl.conv_ws + (size_t)planes * pl.plane;
  return pl;
}

}  // namespace adaption

using namespace adaption;

extern "C" {

int adaption_measure_range(const float* d_x, size_t numel, int32_t n_bits, float* d_max_abs,
                           adaption_qfmt* d_fmt_out, void* stream) {
  return measure_range_impl(d_x, numel, n_bits, d_max_abs, d_fmt_out, reinterpret_cast<cudaStream_t>(stream));
}

int adaption_quantize(const float* d_x, size_t outer, size_t inner, adaption_qtensor out,
                      const adaption_qfmt* d_fmt, int32_t rounding, adaption_stats* d_stats,
                      void* stream) {
  return quantize_impl(d_x, outer, inner, out, d_fmt, 0, rounding, d_stats,
                       reinterpret_cast<cudaStream_t>(stream));
}

int adaption_quantize_batch(const adaption_quantize_item* h_items, int32_t n_items, void* stream) {
  return quantize_batch_impl(h_items, n_items, reinterpret_cast<cudaStream_t>(stream));
}

int adaption_quantize_stochastic(const float* d_x, size_t outer, size_t inner, adaption_qtensor out,
                                 const adaption_qfmt* d_fmt, int32_t relu, uint64_t seed,
                                 adaption_stats* d_stats, void* stream) {
  return quantize_stochastic_impl(d_x, outer, inner, out, d_fmt, relu, seed, d_stats,
                                  reinterpret_cast<cudaStream_t>(stream));
}

int adaption_lp_act_stochastic(const float* d_x_f32, const adaption_qtensor* h_x_q, size_t outer, size_t inner,
                               int32_t relu, adaption_qtensor out, const adaption_qfmt* d_fmt, uint64_t seed,
                               adaption_stats* d_stats, void* stream) {
  if ((d_x_f32 == nullptr) == (h_x_q == nullptr)) {
    if (outer == 0 || inner == 0) return ADAPTION_OK;
    return ADAPTION_ERR_INVALID_ARG;
  }
  if (d_x_f32 != nullptr)
    return quantize_stochastic_impl(d_x_f32, outer, inner, out, d_fmt, relu, seed, d_stats,
                                    reinterpret_cast<cudaStream_t>(stream));
  return requant_stochastic_impl(*h_x_q, outer, inner, relu, out, d_fmt, seed, d_stats,
                                 reinterpret_cast<cudaStream_t>(stream));
}

int adaption_bit_histogram(const float* d_x, size_t numel, uint64_t* d_hist, void* stream) {
  return bit_histogram_impl(d_x, numel, d_hist, reinterpret_cast<cudaStream_t>(stream));
}

int adaption_width_histogram(adaption_qtensor x, size_t outer, size_t inner, uint64_t* d_hist, void* stream) {
  return width_histogram_impl(x, outer, inner, d_hist, reinterpret_cast<cudaStream_t>(stream));
}

int adaption_choose_frac_bits_from_hist(const uint64_t* h_hist, int32_t n_bits, double threshold,
                                        adaption_qfmt* h_out) {
  return choose_frac_bits_from_hist(h_hist, n_bits, threshold, h_out);
}

int adaption_choose_frac_bits_from_widths(const uint64_t* h_hist, int32_t frac_bits, int32_t n_bits,
                                          double threshold, adaption_qfmt* h_out) {
  return choose_frac_bits_from_widths(h_hist, frac_bits, n_bits, threshold, h_out);
}

int adaption_lp_act(const float* d_x_f32, const adaption_qtensor* h_x_q, size_t outer, size_t inner,
                    int32_t relu, adaption_qtensor out, const adaption_qfmt* d_fmt, int32_t rounding,
                    adaption_stats* d_stats, void* stream) {
  if ((d_x_f32 == nullptr) == (h_x_q == nullptr)) {
    if (outer == 0 || inner == 0) return ADAPTION_OK;
    return ADAPTION_ERR_INVALID_ARG;
  }
  if (d_x_f32 != nullptr)
    return quantize_impl(d_x_f32, outer, inner, out, d_fmt, relu ? 1 : 0, rounding, d_stats,
                         reinterpret_cast<cudaStream_t>(stream));
  return requant_impl(*h_x_q, outer, inner, relu ? 1 : 0, out, d_fmt, rounding, d_stats,
                      reinterpret_cast<cudaStream_t>(stream));
}

size_t adaption_lp_conv_workspace_bytes(const adaption_conv_shape* h_shape, adaption_qfmt fx,
                                        adaption_qfmt fw, int64_t c_stride, int32_t algo) {
  if (h_shape == nullptr || algo == ADAPTION_ALGO_DIRECT) return 0;
  GemmProblem g;
  adaption_qtensor x{}, w{}, y{};
  x.fmt = fx; w.fmt = fw; x.c_stride = w.c_stride = c_stride;
  // only shapes and formats matter for the query; give the checks non-null aligned planes
  x.lo = w.lo = x.hi = w.hi = reinterpret_cast<void*>(uintptr_t(256));
  adaption_stats* fake_stats = reinterpret_cast<adaption_stats*>(uintptr_t(256));
  if (build_conv_problem(h_shape, x, w, nullptr, 0, 0, ADAPTION_MODE_RANGE, y, fake_stats, nullptr, 0,
                         nullptr, g) != ADAPTION_OK)
    return 0;
  if (pack_taps_applicable(g)) return pack_taps_workspace(g);
  return tensor_path_supported(g) ? tensor_path_workspace(g) : 0;
}

int adaption_lp_conv_fwd(const adaption_conv_shape* h_shape, adaption_qtensor x, adaption_qtensor w,
                         const int16_t* d_bias_q, int32_t bias_frac_bits, int32_t relu, int32_t mode,
                         int32_t algo, adaption_qtensor y, adaption_stats* d_stats, void* d_workspace,
                         size_t workspace_bytes, void* stream) {
  GemmProblem g;
  int rc = build_conv_problem(h_shape, x, w, d_bias_q, bias_frac_bits, relu, mode, y, d_stats,
                              d_workspace, workspace_bytes, stream, g);
  if (rc != ADAPTION_OK) return rc;
  return dispatch(g, algo);
}

int adaption_lp_conv_fwd_stochastic(const adaption_conv_shape* h_shape, adaption_qtensor x, adaption_qtensor w,
                                    const int16_t* d_bias_q, int32_t bias_frac_bits, int32_t relu, int32_t algo,
                                    adaption_qtensor y, uint64_t seed, adaption_stats* d_stats, void* d_workspace,
                                    size_t workspace_bytes, void* stream) {
  GemmProblem g;
  int rc = build_conv_problem(h_shape, x, w, d_bias_q, bias_frac_bits, relu, ADAPTION_MODE_REQUANT, y, d_stats,
                              d_workspace, workspace_bytes, stream, g);
  if (rc != ADAPTION_OK) return rc;
  g.stochastic = StochasticParams{1, (uint32_t)seed, (uint32_t)(seed >> 32)};
  return dispatch(g, algo);
}

size_t adaption_lp_conv_pool_workspace_bytes(const adaption_conv_shape* h_shape, adaption_qfmt fx, adaption_qfmt fw,
                                             adaption_qfmt fy, int64_t c_stride, int64_t y_c_stride, int32_t algo) {
  if (h_shape == nullptr) return 0;
  GemmProblem g;
  adaption_qtensor x{}, w{}, y{};
  x.fmt = fx; w.fmt = fw; y.fmt = fy;
  x.c_stride = w.c_stride = c_stride;
  y.c_stride = y_c_stride;
  x.lo = w.lo = x.hi = w.hi = y.lo = reinterpret_cast<void*>(uintptr_t(256));
  y.hi = fy.n_bits > 8 ? reinterpret_cast<void*>(uintptr_t(256)) : nullptr;
  adaption_stats* fake_stats = reinterpret_cast<adaption_stats*>(uintptr_t(256));
  if (build_conv_problem(h_shape, x, w, nullptr, 0, 0, ADAPTION_MODE_REQUANT, y, fake_stats, nullptr, 0, nullptr,
                         g) != ADAPTION_OK)
    return 0;
  return plan_conv_pool(g, algo).total;
}

int adaption_lp_conv_pool_fwd(const adaption_conv_shape* h_shape, adaption_qtensor x, adaption_qtensor w,
                              const int16_t* d_bias_q, int32_t bias_frac_bits, int32_t relu, int32_t algo,
                              int32_t phases, adaption_qtensor y, adaption_stats* d_stats, void* d_workspace,
                              size_t workspace_bytes, void* stream) {
  GemmProblem g;
  int rc = build_conv_problem(h_shape, x, w, d_bias_q, bias_frac_bits, relu, ADAPTION_MODE_REQUANT, y, d_stats,
                              d_workspace, workspace_bytes, stream, g);
  if (rc != ADAPTION_OK) return rc;
  if (phases < 1 || phases > (ADAPTION_PHASE_CONV | ADAPTION_PHASE_POOL)) return ADAPTION_ERR_INVALID_ARG;
  if (algo != ADAPTION_ALGO_AUTO && algo != ADAPTION_ALGO_TENSOR && algo != ADAPTION_ALGO_DIRECT)
    return ADAPTION_ERR_INVALID_ARG;
  if ((g.OH & 1) || (g.OW & 1)) return ADAPTION_ERR_INVALID_ARG;      // 2x2 windows need even sizes
  if (g.M == 0) return ADAPTION_OK;
  const ConvPoolPlan pl = plan_conv_pool(g, algo);
  if (d_workspace == nullptr || workspace_bytes < pl.total) return ADAPTION_ERR_WORKSPACE;
  if (!aligned16(d_workspace)) return ADAPTION_ERR_ALIGNMENT;
  // temporary planes for the convolution's own (or half-pooled) output
  uint8_t* ws = static_cast<uint8_t*>(d_workspace);
  adaption_qtensor t = y;
  t.q16 = nullptr;
  t.lo = ws + pl.conv_ws;
  t.hi = y.fmt.n_bits > 8 ? ws + pl.conv_ws + pl.plane : nullptr;
  g.y = t;
  g.workspace = ws;
  g.workspace_bytes = pl.conv_ws;
  g.pool_w = pl.fused;
  if (phases & ADAPTION_PHASE_CONV) {
    rc = dispatch(g, algo);
    if (rc != ADAPTION_OK) return rc;
  }
  if (!(phases & ADAPTION_PHASE_POOL)) return ADAPTION_OK;
  return maxpool_impl(t, h_shape->N, g.OH, g.OW, h_shape->K, y, reinterpret_cast<cudaStream_t>(stream), pl.fused);
}

size_t adaption_lp_ip_workspace_bytes(int64_t B, int64_t K, int64_t O, adaption_qfmt fx,
                                      adaption_qfmt fw, int32_t algo) {
  if (algo == ADAPTION_ALGO_DIRECT) return 0;
  GemmProblem g;
  adaption_qtensor x{}, w{}, y{};
  x.fmt = fx; w.fmt = fw;
  x.c_stride = w.c_stride = (K + 15) / 16 * 16;
  x.lo = w.lo = x.hi = w.hi = reinterpret_cast<void*>(uintptr_t(256));
  adaption_stats* fake_stats = reinterpret_cast<adaption_stats*>(uintptr_t(256));
  if (build_ip_problem(B, K, O, x, w, nullptr, 0, 0, ADAPTION_MODE_RANGE, y, fake_stats, nullptr, 0,
                       nullptr, g) != ADAPTION_OK)
    return 0;
  return tensor_path_supported(g) ? tensor_path_workspace(g) : 0;
}

int adaption_lp_ip_fwd(int64_t B, int64_t K, int64_t O, adaption_qtensor x, adaption_qtensor w,
                       const int16_t* d_bias_q, int32_t bias_frac_bits, int32_t relu, int32_t mode,
                       int32_t algo, adaption_qtensor y, adaption_stats* d_stats, void* d_workspace,
                       size_t workspace_bytes, void* stream) {
  GemmProblem g;
  int rc = build_ip_problem(B, K, O, x, w, d_bias_q, bias_frac_bits, relu, mode, y, d_stats, d_workspace,
                            workspace_bytes, stream, g);
  if (rc != ADAPTION_OK) return rc;
  return dispatch(g, algo);
}

int adaption_lp_ip_fwd_stochastic(int64_t B, int64_t K, int64_t O, adaption_qtensor x, adaption_qtensor w,
                                  const int16_t* d_bias_q, int32_t bias_frac_bits, int32_t relu, int32_t algo,
                                  adaption_qtensor y, uint64_t seed, adaption_stats* d_stats, void* d_workspace,
                                  size_t workspace_bytes, void* stream) {
  GemmProblem g;
  int rc = build_ip_problem(B, K, O, x, w, d_bias_q, bias_frac_bits, relu, ADAPTION_MODE_REQUANT, y, d_stats,
                            d_workspace, workspace_bytes, stream, g);
  if (rc != ADAPTION_OK) return rc;
  g.stochastic = StochasticParams{1, (uint32_t)seed, (uint32_t)(seed >> 32)};
  return dispatch(g, algo);
}

int adaption_maxpool2x2(adaption_qtensor x, int32_t N, int32_t H, int32_t W, int32_t C,
                        adaption_qtensor y, void* stream) {
  return maxpool_impl(x, N, H, W, C, y, reinterpret_cast<cudaStream_t>(stream));
}

int adaption_choose_frac_bits_from_acc(int64_t max_abs_acc, int32_t acc_frac_bits, int32_t n_bits,
                                       adaption_qfmt* h_out) {
  if (h_out == nullptr || n_bits < 1 || n_bits > 16 || max_abs_acc < 0 || acc_frac_bits < 0)
    return ADAPTION_ERR_INVALID_ARG;
  // smallest m in [0, n-1] with max_abs_acc < 2^(m + acc_frac_bits)
  int bitlen = 0;
  while (bitlen < 63 && (max_abs_acc >> bitlen) != 0) ++bitlen;
  int m = bitlen - acc_frac_bits;
  if (m < 0) m = 0;
  if (m > n_bits - 1) m = n_bits - 1;
  h_out->n_bits = n_bits;
  h_out->frac_bits = n_bits - 1 - m;
  return ADAPTION_OK;
}

int adaption_probe_i8_peak(int32_t bn, int32_t pair, int32_t iters, int32_t commit_every, uint64_t* d_cycles,
                           int32_t* d_status, void* stream) {
  if ((bn != 64 && bn != 128 && bn != 256) || iters < 1 || iters > (1 << 19) || commit_every < 0 ||
      d_cycles == nullptr ||
      d_status == nullptr)
    return ADAPTION_ERR_INVALID_ARG;
  return probe_i8_peak(bn, pair ? 1 : 0, iters, commit_every, reinterpret_cast<unsigned long long*>(d_cycles), d_status,
                       reinterpret_cast<cudaStream_t>(stream));
}

int adaption_debug_set(const char* h_name, int32_t value) { return debug_set(h_name, value); }

const char* adaption_status_string(int status) {
  switch (status) {
    case ADAPTION_OK: return "ok";
    case ADAPTION_ERR_INVALID_ARG: return "invalid argument";
    case ADAPTION_ERR_UNSUPPORTED: return "unsupported";
    case ADAPTION_ERR_ALIGNMENT: return "misaligned pointer";
    case ADAPTION_ERR_WORKSPACE: return "workspace missing or too small";
    case ADAPTION_ERR_K_TOO_LARGE: return "reduction too long";
    case ADAPTION_ERR_CUDA: return "CUDA error";
    case ADAPTION_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

}  // extern "C"
