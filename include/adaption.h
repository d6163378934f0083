/*
 * adaption.h - C ABI of the B200 (sm_100a) forward path of the low-precision layers of
 * ADaPTION (arXiv 1711.04713): LPConvolution, LPInnerProduct, LPAct, the quantizer they
 * share and the dynamic-range measurement that fixes each layer's decimal point.
 *
 * Fixed point (Sec. 2 of the paper, "QBD.AD"): a value is stored as a signed integer q of
 * n_bits = BD + AD bits (BD counts the sign bit) and stands for q * 2^-frac_bits,
 * frac_bits = AD.  q lies in [-2^(n_bits-1), 2^(n_bits-1)-1].  1 <= n_bits <= 16 and
 * 0 <= frac_bits <= n_bits-1.
 *
 * Storage of a fixed-point tensor in device memory ("planes"): rows of `inner` elements with
 * a pitch of c_stride elements (c_stride >= inner, a multiple of 16; the padding holds zeros).
 *   n_bits >  8 : two byte planes, hi = q >> 8 (signed) and lo = q & 255 (unsigned),
 *                 so that q = 256*hi + lo;
 *   n_bits <= 8 : one plane, `lo`, holding q itself as a signed byte; hi is NULL.
 * An optional int16 copy q16 (same pitch) can be requested on outputs.
 * Activations are NHWC (rows = pixels, inner = channels); convolution weights are
 * [K][R][S][C] (rows = K*R*S, inner = C); inner-product operands are [B][K] and [O][K].
 *
 * General rules.  Every pointer is a DEVICE pointer unless its name starts with h_.  The
 * caller owns every buffer; the library allocates nothing.  All work is enqueued on the
 * given CUDA stream (a cudaStream_t passed as void*; NULL = default stream) and returns
 * without synchronising.  Every function returns an ADAPTION_* status; argument errors are
 * found on the host before anything is launched.  Plane and workspace pointers must be
 * 16-byte aligned.  Counters in adaption_stats accumulate: the caller zeroes them.
 */
#ifndef ADAPTION_H
#define ADAPTION_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* exported symbols of the shared library */
#if defined(__GNUC__)
#define ADAPTION_API __attribute__((visibility("default")))
#else
#define ADAPTION_API
#endif

enum {
  ADAPTION_OK = 0,
  ADAPTION_ERR_INVALID_ARG = 1,
  ADAPTION_ERR_UNSUPPORTED = 2,
  ADAPTION_ERR_ALIGNMENT = 3,
  ADAPTION_ERR_WORKSPACE = 4,
  ADAPTION_ERR_K_TOO_LARGE = 5,
  ADAPTION_ERR_CUDA = 6,
  ADAPTION_ERR_TIMEOUT = 7
};

/* rounding_scheme of the paper (Sec. 2, Sec. 2.4).  Deterministic = round to nearest, ties
 * away from zero.  Stochastic rounding needs a seed and therefore has entry points of its own
 * (adaption_quantize_stochastic, adaption_lp_act_stochastic); the calls that take a `rounding`
 * argument but no seed answer ADAPTION_ERR_UNSUPPORTED for ADAPTION_ROUND_STOCHASTIC. */
enum { ADAPTION_ROUND_DETERMINISTIC = 0, ADAPTION_ROUND_STOCHASTIC = 1 };

/* Bins of the bit-occupancy histograms (Sec. 2.2, 2.3): 0..15 bits, and 16 or more. */
#define ADAPTION_HIST_BINS 17

/* What a layer call does with its pre-activation values v (accumulator + bias, after ReLU if
 * asked): REQUANT rounds them to the output format and stores them; RANGE only records
 * max|v| in stats.max_abs_acc (the per-layer range measurement of Sec. 2.1 / 2.3). */
enum { ADAPTION_MODE_REQUANT = 0, ADAPTION_MODE_RANGE = 1 };

/* Kernel choice for the layer calls.  AUTO takes the tensor-core path whenever the shape
 * allows it; DIRECT forces the plain integer kernel, TENSOR fails with
 * ADAPTION_ERR_UNSUPPORTED where the tensor-core path cannot run. */
enum { ADAPTION_ALGO_AUTO = 0, ADAPTION_ALGO_TENSOR = 1, ADAPTION_ALGO_DIRECT = 2 };

typedef struct adaption_qfmt {
  int32_t n_bits;    /* BD + AD */
  int32_t frac_bits; /* AD */
} adaption_qfmt;

typedef struct adaption_qtensor {
  void* hi;          /* int8 plane q >> 8, NULL when n_bits <= 8 */
  void* lo;          /* uint8 plane q & 255 (n_bits > 8) or int8 plane q (n_bits <= 8) */
  int16_t* q16;      /* optional int16 copy (outputs only), may be NULL */
  adaption_qfmt fmt;
  int64_t c_stride;  /* row pitch in elements, multiple of 16, >= inner extent */
} adaption_qtensor;

typedef struct adaption_stats {
  uint64_t zeros;       /* stored outputs equal to 0 (Sec. 3.1: sparsity = zeros / total) */
  uint64_t sat_pos;     /* values clipped at the top of the output range */
  uint64_t sat_neg;     /* values clipped at the bottom */
  int64_t max_abs_acc;  /* RANGE mode: max |v| in units of 2^-(f_x + f_w) */
  int32_t status;       /* 0, or ADAPTION_ERR_TIMEOUT if a device-side wait gave up */
  int32_t reserved;
} adaption_stats;

typedef struct adaption_conv_shape {
  int32_t N, H, W, C; /* input NHWC */
  int32_t K;          /* output channels */
  int32_t R, S;       /* filter height, width */
  int32_t pad_h, pad_w;
  int32_t stride_h, stride_w;
} adaption_conv_shape;

/* Sec. 2.1 / 2.3 (dynamic range -> decimal point).  Folds max|x| of x[0..numel) into
 * *d_max_abs (the caller sets it to 0 before the first tensor of a group; NaN is ignored),
 * then writes to *d_fmt_out the format with n_bits total bits whose integer part is the
 * smallest that holds the maximum: m = min{m in [0, n_bits-1] : max < 2^m},
 * frac_bits = n_bits-1-m.  d_fmt_out may be NULL.  numel may be 0. */
ADAPTION_API int adaption_measure_range(const float* d_x, size_t numel, int32_t n_bits, float* d_max_abs,
                           adaption_qfmt* d_fmt_out, void* stream);

/* Sec. 2 (the quantizer of the LP layers).  x is fp32 [outer][inner] dense; out receives
 * q = saturate(round(x * 2^frac_bits)).  If d_fmt is not NULL the fractional bits are read
 * on the device from d_fmt->frac_bits (as written by adaption_measure_range) instead of
 * out.fmt.frac_bits; n_bits always comes from out.fmt.  NaN -> 0, +-Inf saturate.
 * d_stats (may be NULL) accumulates zeros and saturations over the outer*inner real elements. */
ADAPTION_API int adaption_quantize(const float* d_x, size_t outer, size_t inner, adaption_qtensor out,
                      const adaption_qfmt* d_fmt, int32_t rounding, adaption_stats* d_stats,
                      void* stream);

/* Sec. 2.1 (weights and biases are quantized anew in every forward pass): adaption_quantize with
 * deterministic rounding and no counters for n_items tensors at once.  h_items is a HOST array,
 * read before the call returns; each item means what the arguments of the same names mean to
 * adaption_quantize (d_fmt may be NULL).  Dense tensors (inner == q.c_stride, d_x 16-byte aligned)
 * share one kernel launch per 40 items; the others are quantized by launches of their own.  All
 * items are validated before anything is launched; the tensors must not overlap. */
typedef struct adaption_quantize_item {
  const float* d_x;
  int64_t outer, inner;
  adaption_qtensor q;
  const adaption_qfmt* d_fmt;
} adaption_quantize_item;
ADAPTION_API int adaption_quantize_batch(const adaption_quantize_item* h_items, int32_t n_items, void* stream);

/* Sec. 2.4 (rounding_scheme STOCHASTIC).  As adaption_quantize (with the ReLU option of
 * adaption_lp_act), but x * 2^frac_bits = floor + frac is rounded up with probability
 * floor(frac * 2^32) / 2^32 and down otherwise, so that the expectation is the unrounded value and
 * a value already on the grid never moves.  The draw of element i (row-major index over the
 * outer*inner real elements) is word i & 3 of Philox4x32-10 with counter (i >> 2, 0, 0) and key
 * `seed`: the result is a pure function of (x, format, seed), whatever the launch shape.
 * adaption_quantize / adaption_lp_act themselves return ADAPTION_ERR_UNSUPPORTED for
 * ADAPTION_ROUND_STOCHASTIC because they carry no seed. */
ADAPTION_API int adaption_quantize_stochastic(const float* d_x, size_t outer, size_t inner, adaption_qtensor out,
                                 const adaption_qfmt* d_fmt, int32_t relu, uint64_t seed,
                                 adaption_stats* d_stats, void* stream);

/* Sec. 2.1 + 2.4 (LPAct with rounding_scheme STOCHASTIC).  As adaption_lp_act.  fp32 input:
 * adaption_quantize_stochastic.  Fixed-point input (format change f_in -> f_out, s = f_in - f_out):
 * for s > 0 the stored integer v (after ReLU) gives v / 2^s = floor + rem / 2^s and moves up with
 * probability rem / 2^s (threshold rem * 2^(32 - s) against the same per-element draw); for
 * s <= 0 the shift is exact and nothing is drawn. */
ADAPTION_API int adaption_lp_act_stochastic(const float* d_x_f32, const adaption_qtensor* h_x_q, size_t outer,
                               size_t inner, int32_t relu, adaption_qtensor out, const adaption_qfmt* d_fmt,
                               uint64_t seed, adaption_stats* d_stats, void* stream);

/* Sec. 2.3 (iterative, thresholded allocation of the integer bits).  Adds to d_hist[0..17) (device,
 * uint64, caller zeroes it before the first tensor of a group) the number of elements of
 * x[0..numel) that need b integer bits: b = 0 for |x| < 1, else floor(log2 |x|) + 1; bin 16 also
 * takes everything larger and +-Inf; NaN is skipped. */
ADAPTION_API int adaption_bit_histogram(const float* d_x, size_t numel, uint64_t* d_hist, void* stream);

/* Sec. 2.2 (how many quantized values fit fewer bits).  Adds to d_hist[w] the number of real
 * elements of the fixed-point tensor x ([outer][inner], pitch x.c_stride) whose two's complement
 * width is w: the smallest w >= 1 with -2^(w-1) <= q < 2^(w-1). */
ADAPTION_API int adaption_width_histogram(adaption_qtensor x, size_t outer, size_t inner, uint64_t* d_hist,
                             void* stream);

/* Host helper for adaption_bit_histogram.  Starts with all n_bits - 1 non-sign bits in the integer
 * part and moves bits to the fraction while the values that would be lost (those needing more
 * integer bits) number at most threshold * total; threshold in [0, 1], 0 gives the format of
 * adaption_measure_range.  h_hist is a host copy of the 17 bins. */
ADAPTION_API int adaption_choose_frac_bits_from_hist(const uint64_t* h_hist, int32_t n_bits, double threshold,
                                        adaption_qfmt* h_out);

/* The same allocation for a tensor that is already stored with frac_bits fractional bits (e.g. a
 * layer output quantized with the max-based format, so that nothing was clipped), from the
 * histogram of adaption_width_histogram: a value keeps its bits with m integer bits iff its width
 * is at most m + frac_bits + 1. */
ADAPTION_API int adaption_choose_frac_bits_from_widths(const uint64_t* h_hist, int32_t frac_bits, int32_t n_bits,
                                          double threshold, adaption_qfmt* h_out);

/* Sec. 2.1 (LPAct: the activation quantizer, followed by ReLU when relu != 0).  Exactly one
 * of d_x_f32 (fp32 [outer][inner]) and h_x_q (host pointer to the descriptor of a fixed-point
 * tensor, whose format is converted) is given.  Otherwise as adaption_quantize. */
ADAPTION_API int adaption_lp_act(const float* d_x_f32, const adaption_qtensor* h_x_q, size_t outer,
                    size_t inner, int32_t relu, adaption_qtensor out, const adaption_qfmt* d_fmt,
                    int32_t rounding, adaption_stats* d_stats, void* stream);

/* Sec. 2 (LPConvolution forward).  y[n,oh,ow,k] = requant(relu(sum_{r,s,c} x[n, oh*stride_h
 * + r - pad_h, ow*stride_w + s - pad_w, c] * w[k,r,s,c] + bias[k])), taps outside the image
 * contribute 0, the sum is exact.  x and w must share c_stride.  bias_q (int16 [K], may be
 * NULL) has bias_frac_bits <= x.fmt.frac_bits + w.fmt.frac_bits.  In RANGE mode y is ignored.
 * The workspace query returns the bytes the call needs (possibly 0); the workspace contents
 * need no initialisation.  (Layers with at most 4 input channels whose R*S*C taps fit 32 bytes,
 * e.g. the first 3x3 layer of an RGB network, gather their taps into packed planes there: 64 bytes
 * per output pixel.)  d_stats must not be NULL. */
ADAPTION_API size_t adaption_lp_conv_workspace_bytes(const adaption_conv_shape* h_shape, adaption_qfmt fx,
                                        adaption_qfmt fw, int64_t c_stride, int32_t algo);
ADAPTION_API int adaption_lp_conv_fwd(const adaption_conv_shape* h_shape, adaption_qtensor x,
                         adaption_qtensor w, const int16_t* d_bias_q, int32_t bias_frac_bits,
                         int32_t relu, int32_t mode, int32_t algo, adaption_qtensor y,
                         adaption_stats* d_stats, void* d_workspace, size_t workspace_bytes,
                         void* stream);

/* Sec. 2 (rounding_scheme is a parameter of every LP layer) + Sec. 2.4: the layer calls with
 * stochastic rounding in the fused requantization.  As adaption_lp_conv_fwd / adaption_lp_ip_fwd in
 * ADAPTION_MODE_REQUANT (same workspace queries), except for the rounding of the pre-activation value
 * v (accumulator + bias, after ReLU), an integer in units of 2^-F with F = x.fmt.frac_bits +
 * w.fmt.frac_bits: with s = F - y.fmt.frac_bits > 0, v / 2^s = q + rem / 2^s (q = floor, 0 <= rem <
 * 2^s) becomes q + 1 with probability rem / 2^s and q otherwise, so that the expectation is the
 * unrounded value and a value on the output grid never moves; for s <= 0 the shift is exact.  The
 * draw of output element i (row-major index over the real [M][K] outputs, M = N*OH*OW pixels or B
 * rows) is word i & 3 of Philox4x32-10 with counter (i >> 2, 0, 0) and key `seed`, and the value
 * moves up iff draw < rem * 2^(32 - s): a pure function of (operands, formats, seed), whatever
 * kernel or tile shape runs the layer.  Saturation and counters as in the deterministic calls. */
ADAPTION_API int adaption_lp_conv_fwd_stochastic(const adaption_conv_shape* h_shape, adaption_qtensor x,
                                    adaption_qtensor w, const int16_t* d_bias_q, int32_t bias_frac_bits,
                                    int32_t relu, int32_t algo, adaption_qtensor y, uint64_t seed,
                                    adaption_stats* d_stats, void* d_workspace, size_t workspace_bytes,
                                    void* stream);
ADAPTION_API int adaption_lp_ip_fwd_stochastic(int64_t B, int64_t K, int64_t O, adaption_qtensor x,
                                  adaption_qtensor w, const int16_t* d_bias_q, int32_t bias_frac_bits,
                                  int32_t relu, int32_t algo, adaption_qtensor y, uint64_t seed,
                                  adaption_stats* d_stats, void* d_workspace, size_t workspace_bytes,
                                  void* stream);

/* Sec. 2 + Table 1 "Pooling" (LPConvolution followed by the 2x2 / stride-2 max-pool of its output,
 * as in VGG16 and Giga1Net).  y is the pooled tensor [N, OH/2, OW/2, K] in the layer's output format;
 * OH and OW must be even.  The result equals adaption_lp_conv_fwd followed by adaption_maxpool2x2
 * (the quantizer is monotone, so pooling the stored integers is exact); d_stats counts the
 * convolution's own outputs, before pooling.  Requantizing mode only.  The convolution's output
 * lives in the workspace: where the tensor-core path can, only the maxima of horizontal pixel
 * pairs are stored there (half the bytes written and read back), otherwise all of it.
 * phases: ADAPTION_PHASE_CONV | ADAPTION_PHASE_POOL runs the whole layer pair; the two phases may
 * also be issued by two calls with otherwise identical arguments (convolution first, same stream
 * order, workspace untouched in between), e.g. to time them apart.
 * y_c_stride in the query is the pitch of y. */
#define ADAPTION_PHASE_CONV 1
#define ADAPTION_PHASE_POOL 2
ADAPTION_API size_t adaption_lp_conv_pool_workspace_bytes(const adaption_conv_shape* h_shape, adaption_qfmt fx,
                                             adaption_qfmt fw, adaption_qfmt fy, int64_t c_stride,
                                             int64_t y_c_stride, int32_t algo);
ADAPTION_API int adaption_lp_conv_pool_fwd(const adaption_conv_shape* h_shape, adaption_qtensor x,
                              adaption_qtensor w, const int16_t* d_bias_q, int32_t bias_frac_bits,
                              int32_t relu, int32_t algo, int32_t phases, adaption_qtensor y,
                              adaption_stats* d_stats, void* d_workspace, size_t workspace_bytes,
                              void* stream);

/* Sec. 2 (LPInnerProduct forward).  y[b,o] = requant(relu(sum_k x[b,k] * w[o,k] + bias[o])).
 * x is [B][K], w is [O][K], y is [B][O]. */
ADAPTION_API size_t adaption_lp_ip_workspace_bytes(int64_t B, int64_t K, int64_t O, adaption_qfmt fx,
                                      adaption_qfmt fw, int32_t algo);
ADAPTION_API int adaption_lp_ip_fwd(int64_t B, int64_t K, int64_t O, adaption_qtensor x, adaption_qtensor w,
                       const int16_t* d_bias_q, int32_t bias_frac_bits, int32_t relu,
                       int32_t mode, int32_t algo, adaption_qtensor y, adaption_stats* d_stats,
                       void* d_workspace, size_t workspace_bytes, void* stream);

/* No counterpart in the paper: a convenience for callers that cannot allocate device memory.
 * Same operation, arguments, results and status codes as adaption_lp_ip_fwd, but the split-K
 * workspace is not passed in: it is a fixed array of ADAPTION_STATIC_WORKSPACE_BYTES inside the
 * library image (every GPU that loads the library carries it until the process exits).  It is
 * meant for code that must not call cudaMalloc where it runs: plug-ins handed a fixed memory
 * arena by their host application, or real-time loops in which an allocation would stall or
 * synchronise the device.  The call itself allocates and frees nothing.
 *   - Limit: if the shape needs more workspace than the array holds (the amount
 *     adaption_lp_ip_workspace_bytes reports, i.e. 8 bytes per output element when the reduction
 *     is split), the call returns ADAPTION_ERR_WORKSPACE and launches nothing; use
 *     adaption_lp_ip_fwd with your own buffer for such shapes.
 *   - The first call on each device looks the array's device address up (one runtime query with
 *     that device current; a failure is reported as ADAPTION_ERR_CUDA).  That query may be the
 *     moment the CUDA runtime loads the library's device code on that device, array included, so
 *     "allocates nothing" describes every call after the first.  Make that first call before any
 *     stream capture begins.  The address is cached per device for the life of the process: do
 *     not use this entry point on a device after cudaDeviceReset.
 *   - Shapes that need no workspace (an unsplit reduction, or ADAPTION_ALGO_DIRECT) never touch
 *     the array.
 *   - All calls on a device share the one array and it keeps the previous call's contents; each
 *     call clears the part it uses before accumulating.  Two calls whose GPU work can overlap
 *     (different streams, or different host threads on the same device) race on it: run them on
 *     one stream or order them yourself. */
#define ADAPTION_STATIC_WORKSPACE_BYTES (4u << 20)
ADAPTION_API int adaption_lp_ip_fwd_static_ws(int64_t B, int64_t K, int64_t O, adaption_qtensor x,
                                              adaption_qtensor w, const int16_t* d_bias_q,
                                              int32_t bias_frac_bits, int32_t relu, int32_t mode,
                                              int32_t algo, adaption_qtensor y, adaption_stats* d_stats,
                                              void* stream);

/* The 2x2, stride-2 max pooling that sits between the low-precision layers of the networks
 * the paper studies (VGG16; Table 1, "Pooling").  Works on the stored integers, same format
 * in and out; H and W even.  x is [N][H][W][C], y is [N][H/2][W/2][C]. */
ADAPTION_API int adaption_maxpool2x2(adaption_qtensor x, int32_t N, int32_t H, int32_t W, int32_t C,
                        adaption_qtensor y, void* stream);

/* Host helper for RANGE mode (Sec. 2.3): the format with n_bits whose integer part is the
 * smallest that holds max_abs_acc * 2^-acc_frac_bits. */
ADAPTION_API int adaption_choose_frac_bits_from_acc(int64_t max_abs_acc, int32_t acc_frac_bits,
                                       int32_t n_bits, adaption_qfmt* h_out);

/* Measurement aid for the roofline of the layer calls (no counterpart in the paper): every SM
 * (pair != 0: every pair of SMs working on 256-row tiles) issues 4*iters back-to-back int8
 * tensor-core instructions of shape 128 (256) x bn x 32 on operands resident in shared memory.
 * d_cycles receives, per launched block (one per SM; at least 148 entries), the SM clock cycles
 * the issuing block needed (entries of non-issuing blocks are left untouched); *d_status is set to
 * ADAPTION_ERR_TIMEOUT if a wait gave up.  bn is 64, 128 or 256.  commit_every > 0 adds a
 * completion signal (tcgen05.commit) after every commit_every groups of four instructions, as a
 * pipelined mainloop issues them; 0 issues none.  Asynchronous on `stream`. */
ADAPTION_API int adaption_probe_i8_peak(int32_t bn, int32_t pair, int32_t iters, int32_t commit_every,
                                        uint64_t* d_cycles, int32_t* d_status, void* stream);

/* Test and experiment aid (no counterpart in the paper; not meant for production callers).  Sets one
 * process-wide override of the tensor-core path's tile heuristics, so that tests can drive the same
 * layer through its alternative code paths and compare the bits.  h_name is a host string:
 *   "splits" n     at least n splits of the reduction            (default 0: heuristic)
 *   "pair" 0|1     forbid / force CTA pairs                       (default -1: heuristic)
 *   "fast" 0       generic 64-bit epilogue instead of the 32-bit one        (default 1)
 *   "staged" 0     direct stores instead of shared-memory staging           (default 1)
 *   "stages" n     cap the depth of the shared-memory ring                  (default 0: none)
 *   "bk" 32|64, "bn" 32|64, "kps" 1..4, "bres" 0, "wide" 0, "epigroups" 1   narrower tiles etc.
 *   "split_hh" 0   three 128-column accumulators are handed back together            (default 1)
 *   "stagger" 0    the last k-blocks of a tile are issued like the others                 (default 1)
 *   "stage_bufs" 1 one output staging buffer per epilogue group even where two would fit (default 2)
 *   "pdl" 0        layer kernels are launched without programmatic stream serialization (default 1)
 *   "timeout_us" t limit of every device-side wait in microseconds (default 0: two seconds)
 *   "stall_at" i   the copy-issuing warps of every block stop before their i-th stage with nothing
 *                  in flight for it, so that the waits of the other warps run out: the kernel then
 *                  sets stats.status = ADAPTION_ERR_TIMEOUT, drains and returns (default -1: never)
 *   "reset"        every override back to its default (value ignored)
 * Returns ADAPTION_ERR_INVALID_ARG for an unknown name.  Calls already enqueued are not affected;
 * do not change overrides while another host thread is inside a layer call. */
ADAPTION_API int adaption_debug_set(const char* h_name, int32_t value);

ADAPTION_API const char* adaption_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* ADAPTION_H */
