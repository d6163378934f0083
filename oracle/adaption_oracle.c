/*
 * CPU oracle for the forward pass of ADaPTION's low-precision layers
 * (arXiv 1711.04713, Sec. 2 "Low-precision add-on for Caffe", Sec. 2.1, Sec. 2.3).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, direct
 * restatement of what the layers compute, kept independent of the CUDA path:
 * it shares no code, header, table or helper with it.  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Everything is written as the definition: direct loops, canonical integers
 * q (real value q * 2^-f), int64 accumulators, no blocking, no plane tricks.
 * OpenMP pragmas only distribute independent (image, output-row) iterations;
 * they change no arithmetic and no order of any sum that matters (integer
 * sums are exact in any order anyway).
 *
 * Notation (Sec. 2): n = total bits = BD + AD, f = AD = fractional bits,
 * BD includes the sign bit, so q lies in [-2^(n-1), 2^(n-1)-1].
 *
 * Readings fixed here where the paper is silent:
 *   - deterministic rounding (Sec. 2, rounding_scheme) = round to nearest,
 *     ties away from zero; then saturate (two's-complement asymmetric range);
 *   - NaN quantizes to 0, +-Inf saturate; the range measurement ignores NaN;
 *   - integer bits m (excluding sign) from a maximum M: the smallest m in
 *     [0, n-1] with M < 2^m, f = n-1-m  (Sec. 2.3, zero-loss case of the
 *     iterative scheme: "check against the maximum number present");
 *   - accumulation is exact (int64); bias is a fixed-point number aligned to
 *     the accumulator by an exact left shift; ReLU, then one rounding to the
 *     output format (Sec. 2.1: LPAct quantizes, ReLU follows; the two
 *     commute because rounding is monotone and maps 0 to 0);
 *   - sparsity counter = stored outputs equal to zero (Sec. 3.1: zeros
 *     divided by total elements); saturation counters = elements whose
 *     rounded value fell outside the representable range.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* counters[0] = zeros, [1] = positive saturations, [2] = negative saturations */

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static int64_t q_min(int n_bits) { return -((int64_t)1 << (n_bits - 1)); }
static int64_t q_max(int n_bits) { return ((int64_t)1 << (n_bits - 1)) - 1; }

/* Sec. 2: quantize one fp32 value to signed fixed point with n bits, f fractional
 * bits, deterministic rounding (ties away from zero), saturation.
 * x * 2^f is exact in double; for a float x, |y| + 0.5 is exact in double
 * whenever it can influence floor(). */
static int64_t quantize_one(float x, int n_bits, int f, int relu, uint64_t* counters) {
  int64_t lo = q_min(n_bits), hi = q_max(n_bits);
  int64_t q;
  if (isnan(x)) {
    q = 0;
  } else {
    double y = ldexp((double)x, f);
    if (relu && y < 0.0) y = 0.0;
    double r = (y >= 0.0) ? floor(y + 0.5) : -floor(-y + 0.5);
    if (r > (double)hi) {
      q = hi;
      if (counters) counters[1]++;
    } else if (r < (double)lo) {
      q = lo;
      if (counters) counters[2]++;
    } else {
      q = (int64_t)r;
    }
  }
  if (counters && q == 0) counters[0]++;
  return q;
}

void oracle_quantize(const float* x, size_t numel, int n_bits, int f, int relu,
                     int16_t* q, uint64_t* counters /* [3], accumulated */) {
  for (size_t i = 0; i < numel; ++i)
    q[i] = (int16_t)quantize_one(x[i], n_bits, f, relu, counters);
}

/* Value represented by q: q * 2^-f (exact in double). */
void oracle_dequantize(const int16_t* q, size_t numel, int f, double* out) {
  for (size_t i = 0; i < numel; ++i) out[i] = ldexp((double)q[i], -f);
}

/* Byte planes of the canonical integer: q = 256 * hi + lo with hi signed
 * (floor division) and lo in [0, 255]. */
void oracle_split_planes(const int16_t* q, size_t numel, int8_t* hi, uint8_t* lo) {
  for (size_t i = 0; i < numel; ++i) {
    int v = q[i];
    int l = ((v % 256) + 256) % 256;
    hi[i] = (int8_t)((v - l) / 256);
    lo[i] = (uint8_t)l;
  }
}

/* Sec. 2.1 / 2.3: dynamic range of a tensor = max |x| (NaN ignored). */
float oracle_max_abs(const float* x, size_t numel) {
  float m = 0.0f;
  for (size_t i = 0; i < numel; ++i) {
    float a = fabsf(x[i]);
    if (!isnan(a) && a > m) m = a;
  }
  return m;
}

/* Sec. 2.3: integer bits (sign excluded) needed so that max_abs < 2^m,
 * clamped to [0, n-1]; the caller gets f = n-1-m. */
int oracle_int_bits_from_max(float max_abs, int n_bits) {
  int m = 0;
  if (isinf(max_abs)) return n_bits - 1;
  /* smallest m >= 0 with max_abs < 2^m, by direct search (no logarithm) */
  while (m < n_bits - 1 && !((double)max_abs < ldexp(1.0, m))) ++m;
  return m;
}

/* Same rule on an accumulator-domain maximum A >= 0 with F fractional bits:
 * smallest m in [0, n-1] with A * 2^-F < 2^m, i.e. A < 2^(m+F). */
int oracle_int_bits_from_acc(int64_t max_abs_acc, int acc_frac_bits, int n_bits) {
  int m = 0;
  while (m < n_bits - 1) {
    int sh = m + acc_frac_bits;
    /* A < 2^sh ?  (sh may exceed 62: then always true for int64 A) */
    if (sh >= 63 || max_abs_acc < ((int64_t)1 << sh)) break;
    ++m;
  }
  return m;
}

/* Sec. 2: LPConvolution "operates the same way as its high-precision
 * counterpart" on quantized values: a direct convolution (cross-correlation,
 * as in Caffe) with zero padding.  x: [N][H][W][C], w: [K][R][S][C],
 * acc: [N][OH][OW][K], all dense.  Seven loops, int64 sums. */
void oracle_conv_acc(const int16_t* x, const int16_t* w, int N, int H, int W, int C, int K,
                     int R, int S, int pad_h, int pad_w, int stride_h, int stride_w,
                     int64_t* acc) {
  int OH = (H + 2 * pad_h - R) / stride_h + 1;
  int OW = (W + 2 * pad_w - S) / stride_w + 1;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int oh = 0; oh < OH; ++oh)
      for (int ow = 0; ow < OW; ++ow)
        for (int k = 0; k < K; ++k) {
          int64_t sum = 0;
          for (int r = 0; r < R; ++r)
            for (int s = 0; s < S; ++s) {
              int ih = oh * stride_h + r - pad_h;
              int iw = ow * stride_w + s - pad_w;
              if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue; /* zero padding */
              const int16_t* xp = x + (((size_t)n * H + ih) * W + iw) * C;
              const int16_t* wp = w + (((size_t)k * R + r) * S + s) * C;
              for (int c = 0; c < C; ++c) sum += (int64_t)xp[c] * (int64_t)wp[c];
            }
          acc[(((size_t)n * OH + oh) * OW + ow) * K + k] = sum;
        }
}

/* One output position of the convolution (for spot checks at sizes where the
 * full loop nest would take too long). */
int64_t oracle_conv_acc_at(const int16_t* x, const int16_t* w, int N, int H, int W, int C,
                           int K, int R, int S, int pad_h, int pad_w, int stride_h,
                           int stride_w, int n, int oh, int ow, int k) {
  (void)N;
  (void)K;
  int64_t sum = 0;
  for (int r = 0; r < R; ++r)
    for (int s = 0; s < S; ++s) {
      int ih = oh * stride_h + r - pad_h;
      int iw = ow * stride_w + s - pad_w;
      if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
      const int16_t* xp = x + (((size_t)n * H + ih) * W + iw) * C;
      const int16_t* wp = w + (((size_t)k * R + r) * S + s) * C;
      for (int c = 0; c < C; ++c) sum += (int64_t)xp[c] * (int64_t)wp[c];
    }
  return sum;
}

/* Sec. 2: LPInnerProduct on quantized values.  x: [B][K], w: [O][K], acc: [B][O]. */
void oracle_ip_acc(const int16_t* x, const int16_t* w, int64_t B, int64_t K, int64_t O,
                   int64_t* acc) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t b = 0; b < B; ++b)
    for (int64_t o = 0; o < O; ++o) {
      int64_t sum = 0;
      for (int64_t k = 0; k < K; ++k) sum += (int64_t)x[b * K + k] * (int64_t)w[o * K + k];
      acc[b * O + o] = sum;
    }
}

/* Round v / 2^s to the nearest integer, ties away from zero (s > 0);
 * exact left shift for s <= 0.  Where v * 2^-s does not fit 64 bits the result is
 * INT64_MAX / INT64_MIN: the callers saturate to at most 16 bits right after, so the
 * stored value and the saturation count are those of the exact product. */
static int64_t shift_round(int64_t v, int s) {
  if (s <= 0) {
    int64_t lim = INT64_MAX >> (-s);
    if (v > lim) return INT64_MAX;
    if (v < -lim) return INT64_MIN;
    return v * ((int64_t)1 << (-s));
  }
  int64_t a = v < 0 ? -v : v;
  int64_t r = (a + ((int64_t)1 << (s - 1))) >> s;
  return v < 0 ? -r : r;
}

int64_t oracle_shift_round(int64_t v, int s) { return shift_round(v, s); }

/* Bias, ReLU, requantization of an accumulator tensor acc[outer][channels]
 * whose unit is 2^-acc_frac_bits  (Sec. 2.1: weights, biases and activations
 * are quantized; the quantized activation feeds ReLU).
 *   v = acc + (bias_q << (acc_frac_bits - bias_frac_bits))
 *   v = max(v, 0) if relu
 *   y = saturate_n( round_half_away( v / 2^(acc_frac_bits - out_frac_bits) ) )
 * bias_q may be NULL.  y is int16; counters as in oracle_quantize. */
void oracle_epilogue(const int64_t* acc, size_t outer, size_t channels, const int16_t* bias_q,
                     int bias_frac_bits, int acc_frac_bits, int relu, int out_n_bits,
                     int out_frac_bits, int16_t* y, uint64_t* counters) {
  int64_t lo = q_min(out_n_bits), hi = q_max(out_n_bits);
  int s = acc_frac_bits - out_frac_bits;
  for (size_t i = 0; i < outer; ++i)
    for (size_t c = 0; c < channels; ++c) {
      int64_t v = acc[i * channels + c];
      if (bias_q) v += (int64_t)bias_q[c] * ((int64_t)1 << (acc_frac_bits - bias_frac_bits));
      if (relu && v < 0) v = 0;
      int64_t r = shift_round(v, s);
      if (r > hi) {
        r = hi;
        if (counters) counters[1]++;
      } else if (r < lo) {
        r = lo;
        if (counters) counters[2]++;
      }
      if (counters && r == 0) counters[0]++;
      y[i * channels + c] = (int16_t)r;
    }
}

/* Dynamic range of what the requantizer will see (Sec. 2.1: range of the
 * activations measured on a batch): max |v| after bias and optional ReLU,
 * in accumulator units. */
int64_t oracle_epilogue_range(const int64_t* acc, size_t outer, size_t channels,
                              const int16_t* bias_q, int bias_frac_bits, int acc_frac_bits,
                              int relu) {
  int64_t m = 0;
  for (size_t i = 0; i < outer; ++i)
    for (size_t c = 0; c < channels; ++c) {
      int64_t v = acc[i * channels + c];
      if (bias_q) v += (int64_t)bias_q[c] * ((int64_t)1 << (acc_frac_bits - bias_frac_bits));
      if (relu && v < 0) v = 0;
      int64_t a = v < 0 ? -v : v;
      if (a > m) m = a;
    }
  return m;
}

/* LPAct on an already quantized tensor: change of format f_in -> f_out with
 * optional ReLU (Sec. 2.1). */
void oracle_requantize(const int16_t* xq, size_t numel, int in_frac_bits, int relu,
                       int out_n_bits, int out_frac_bits, int16_t* y, uint64_t* counters) {
  int64_t lo = q_min(out_n_bits), hi = q_max(out_n_bits);
  int s = in_frac_bits - out_frac_bits;
  for (size_t i = 0; i < numel; ++i) {
    int64_t v = xq[i];
    if (relu && v < 0) v = 0;
    int64_t r = shift_round(v, s);
    if (r > hi) {
      r = hi;
      if (counters) counters[1]++;
    } else if (r < lo) {
      r = lo;
      if (counters) counters[2]++;
    }
    if (counters && r == 0) counters[0]++;
    y[i] = (int16_t)r;
  }
}

/* 2x2 max pooling, stride 2, on quantized values (the pooling layers between
 * the low-precision layers; VGG16 and Table 1 "Pooling").  x: [N][H][W][C],
 * H and W even, y: [N][H/2][W/2][C]. */
void oracle_maxpool2x2(const int16_t* x, int N, int H, int W, int C, int16_t* y) {
  int OH = H / 2, OW = W / 2;
  for (int n = 0; n < N; ++n)
    for (int oh = 0; oh < OH; ++oh)
      for (int ow = 0; ow < OW; ++ow)
        for (int c = 0; c < C; ++c) {
          int16_t m = x[(((size_t)n * H + 2 * oh) * W + 2 * ow) * C + c];
          for (int dh = 0; dh < 2; ++dh)
            for (int dw = 0; dw < 2; ++dw) {
              int16_t v = x[(((size_t)n * H + 2 * oh + dh) * W + 2 * ow + dw) * C + c];
              if (v > m) m = v;
            }
          y[(((size_t)n * OH + oh) * OW + ow) * C + c] = m;
        }
}
