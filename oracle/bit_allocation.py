"""CPU oracle for the thresholded integer-bit allocation (test infrastructure, not the product).

Paper Sec. 2.3: with the total number of bits n fixed, reduce the bits of the integer part step by
step, count how many weights / activations can then no longer be represented, and accept the
reduction while the lost percentage stays within a user-defined threshold (usually below 1 %).
Sec. 2.2 reads the same statistic off the quantized weights ("~90 % can be represented with
4 bits, ~99 % with 8 bits").

Readings (the paper gives no formulas):
B1  A value x needs  b(x) = 0 integer bits if |x| < 1, else floor(log2 |x|) + 1  (the sign bit is
    not counted; this is the m of the max-based rule: x is representable with m integer bits iff
    |x| < 2^m).  NaN is skipped, +-Inf counts in the top bin.
B2  The histogram has ADAPTION_HIST_BINS = 17 bins: bin b counts the values with b(x) = b for
    b < 16, bin 16 everything that needs 16 bits or more.
B3  A value is "lost" with m integer bits iff b(x) > m.  The allocation starts from all n - 1
    non-sign bits in the integer part and gives bits to the fraction while
    lost(m - 1) <= threshold * (number of counted values); threshold = 0 reproduces the max-based
    rule of the range measurement.
B4  For a quantized tensor (canonical integers q) the statistic of Sec. 2.2 is the two's
    complement width: q fits w bits iff -2^(w-1) <= q < 2^(w-1).
Plain numpy, fp64 / integers only; shares no code with the CUDA path.
"""
from __future__ import annotations

import math

import numpy as np

HIST_BINS = 17


def integer_bits_needed(x) -> np.ndarray:
    """b(x) per element (reading B1), -1 for NaN.  Taken from the binary exponent, no logarithm."""
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    out = np.zeros(x.shape, dtype=np.int64)
    a = np.abs(x)
    big = a >= 1.0
    fin = np.isfinite(a)
    _, e = np.frexp(np.where(big & fin, a, 1.0))      # a = mant * 2^e, 0.5 <= mant < 1  =>  2^(e-1) <= a < 2^e
    out[big & fin] = e[big & fin]
    out[np.isinf(a)] = 1 << 20
    out[np.isnan(a)] = -1
    return out


def bit_histogram(x) -> np.ndarray:
    """Reading B2."""
    b = integer_bits_needed(x)
    b = b[b >= 0]
    h = np.zeros(HIST_BINS, dtype=np.uint64)
    for v in np.minimum(b, HIST_BINS - 1):
        h[int(v)] += np.uint64(1)
    return h


def choose_int_bits(hist, n_bits: int, threshold: float) -> int:
    """Reading B3, in the paper's order: start with every non-sign bit in the integer part and move
    bits to the fraction while the share of lost values stays within the threshold."""
    hist = [int(v) for v in hist]
    total = sum(hist)

    def lost(m: int) -> int:
        return sum(hist[b] for b in range(len(hist)) if b > m)

    m = n_bits - 1
    while m > 0 and lost(m - 1) <= threshold * total:
        m -= 1
    return m


def choose_frac_bits(hist, n_bits: int, threshold: float) -> int:
    return n_bits - 1 - choose_int_bits(hist, n_bits, threshold)


def width_histogram(q) -> np.ndarray:
    """Histogram over w = 1..16 of the two's complement widths of a quantized tensor (bin 0 stays 0)."""
    return np.bincount(twos_complement_width(q), minlength=HIST_BINS).astype(np.uint64)


def choose_int_bits_from_widths(width_hist, frac_bits: int, n_bits: int, threshold: float) -> int:
    """Reading B3 for a tensor already stored with ``frac_bits`` fractional bits (the layer output
    quantized with the max-based format, so that nothing was clipped): q keeps its value with m
    integer bits iff its width is at most m + frac_bits + 1.  Same order as the paper: start with
    all n - 1 non-sign bits in the integer part, give bits away while the loss stays within the
    threshold."""
    hist = [int(v) for v in width_hist]
    total = sum(hist)

    def lost(m: int) -> int:
        return sum(hist[w] for w in range(len(hist)) if w > m + frac_bits + 1)

    m = n_bits - 1
    while m > 0 and lost(m - 1) <= threshold * total:
        m -= 1
    return m


def twos_complement_width(q) -> np.ndarray:
    """Reading B4: smallest w >= 1 with -2^(w-1) <= q < 2^(w-1)."""
    q = np.asarray(q, dtype=np.int64).reshape(-1)
    mag = np.where(q >= 0, q, -q - 1)          # q >= 0: q < 2^(w-1);  q < 0: -q - 1 < 2^(w-1)
    _, e = np.frexp(mag.astype(np.float64))    # exact below 2^53: mag in [2^(e-1), 2^e), e = 0 for 0
    return e.astype(np.int64) + 1              # bit length of mag, plus the sign bit
