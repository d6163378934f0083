"""CPU oracle for stochastic rounding (test infrastructure, not the product).

Paper Sec. 2.4: a stochastically rounded value is one of the two nearest fixed-point values,
drawn so that its expectation is the unrounded value.  The paper fixes neither the random
number generator nor how a draw is compared with the fraction, so both are fixed here
(readings S1-S3) and the CUDA path follows them bit for bit:

S1  The real value y = x * 2^f is split as y = floor(y) + frac, 0 <= frac < 1, exactly.  The
    result is floor(y) + 1 with probability T / 2^32, T = floor(frac * 2^32), else floor(y); then
    it is saturated like the deterministic quantizer (NaN -> 0, +-Inf saturate).  A value already
    on the grid never moves.  (floor(y) and T are computed from |y|, whose integer and fractional
    parts are both exact in fp64 because x is fp32; for y < 0 the fraction 1 - frac(|y|) need not
    be representable, so T is formed in integers: see ``floor_and_threshold``.)
S2  The draw for element i (index in the logical [outer][inner] order, padding excluded) is the
    32-bit word  R_i = Philox4x32-10(counter = (i >> 2, 0, 0) as (lo32, hi32, 0, 0),
    key = (seed lo32, seed hi32))[i & 3]  and the value moves up iff R_i < T.
S3  Philox4x32-10 is the counter-based generator of Salmon, Moraes, Dror and Shaw, "Parallel
    random numbers: as easy as 1, 2, 3" (SC'11), written out below from its definition: ten
    rounds of two 32x32 -> 64-bit multiplications with the constants 0xD2511F53 and 0xCD9E8D57,
    the key bumped by 0x9E3779B9 and 0xBB67AE85 between rounds.

Plain numpy, vectorised over elements; no code is shared with the CUDA path.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(counter, key):
    """counter: four arrays (or scalars) of 32-bit words, key: two 32-bit words -> four arrays of
    32-bit words.  Definition: Salmon et al. 2011, Sec. 3.3 (Philox-4x32 with 10 rounds)."""
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & _MASK for c in counter)
    k0 = np.uint64(key[0]) & _MASK
    k1 = np.uint64(key[1]) & _MASK
    for rnd in range(10):
        if rnd > 0:                       # key schedule: bumped before every round but the first
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0                     # 32 x 32 -> 64 bit products (operands below 2^32)
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK, lo1, (hi0 ^ c3 ^ k1) & _MASK, lo0
    return c0, c1, c2, c3


def draws(n: int, seed: int) -> np.ndarray:
    """R_i for i in [0, n): reading S2."""
    i = np.arange(n, dtype=np.uint64)
    blk = i >> np.uint64(2)
    out = philox4x32_10((blk & _MASK, blk >> _S32, np.zeros_like(blk), np.zeros_like(blk)),
                        (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    words = np.stack(out, axis=1)                       # [n, 4]
    return words[np.arange(n), (i & np.uint64(3)).astype(np.int64)].astype(np.uint64)


def floor_and_threshold(y):
    """Reading S1 for finite fp64 values y that carry at most 24 significant bits (an fp32 value
    times a power of two): returns (floor(y) as int64, T = floor((y - floor(y)) * 2^32) as uint64),
    both exact.  With a = |y| = ia + fa (integer and fractional part, both exact in fp64) and
    U = fa * 2^32 (exact: a power-of-two scaling):
        y >= 0            : floor = ia,       T = floor(U)
        y <  0, fa == 0   : floor = -ia,      T = 0
        y <  0, fa >  0   : floor = -ia - 1,  frac = 1 - fa,  T = floor(2^32 - U) = 2^32 - ceil(U)
    The last line is taken in integers; 1 - fa itself can need more than 53 bits (fa = 2^-60)."""
    y = np.asarray(y, dtype=np.float64)
    a = np.abs(y)
    ia = np.floor(a)
    fa = a - ia                                         # exact
    U = fa * 4294967296.0                               # exact, 0 <= U < 2^32
    neg = (y < 0) & (fa > 0)
    lo = np.where(y < 0, -ia, ia).astype(np.int64) - neg.astype(np.int64)
    T_pos = np.floor(U).astype(np.uint64)
    T_neg = np.uint64(1 << 32) - np.ceil(U).astype(np.uint64)
    return lo, np.where(neg, T_neg, T_pos)


def quantize_stochastic(x, n_bits: int, frac_bits: int, seed: int, relu: bool = False):
    """Stochastically rounded canonical integers (int16) of a fp32 tensor, with counters
    (zeros, sat_pos, sat_neg) like the deterministic quantizer.  Readings S1-S2."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    flat = x.reshape(-1).astype(np.float64)
    qmin, qmax = -(1 << (n_bits - 1)), (1 << (n_bits - 1)) - 1
    y = flat * float(2.0 ** frac_bits)                  # exact: power-of-two scaling of an fp32 value
    nan = np.isnan(y)
    y = np.where(nan, 0.0, y)
    # far outside the range the fraction is irrelevant: clamp first so that floor() stays finite
    y = np.clip(y, float(qmin) - 2.0, float(qmax) + 2.0)
    lo, T = floor_and_threshold(y)
    R = draws(flat.size, seed)
    r = lo + (R < T).astype(np.int64)
    if relu:
        r = np.maximum(r, 0)
    sat_pos = int((r > qmax).sum())
    sat_neg = int((r < qmin).sum())
    q = np.clip(r, qmin, qmax)
    zeros = int((q == 0).sum())
    return q.astype(np.int16).reshape(x.shape), (zeros, sat_pos, sat_neg)


def requantize_stochastic(xq, in_frac_bits: int, relu: bool, out_n_bits: int, out_frac_bits: int, seed: int):
    """LPAct on an already quantized tensor with stochastic rounding: format change f_in -> f_out.
    The stored integer v (after the optional ReLU) stands for v * 2^-f_in; with s = f_in - f_out > 0
    the exact quotient v / 2^s = floor + rem / 2^s moves up with probability rem / 2^s, taken as
    T = rem * 2^(32 - s) against the same 32-bit draw as in S2 (exact: s <= 15); s <= 0 is an exact
    left shift.  Saturation and counters as in the deterministic requantizer."""
    q = np.ascontiguousarray(xq, dtype=np.int16)
    v = q.reshape(-1).astype(np.int64)
    if relu:
        v = np.maximum(v, 0)
    s = in_frac_bits - out_frac_bits
    qmin, qmax = -(1 << (out_n_bits - 1)), (1 << (out_n_bits - 1)) - 1
    if s > 0:
        lo = v >> s                                   # floor division by 2^s (arithmetic shift)
        rem = v - (lo << s)                           # 0 <= rem < 2^s
        T = (rem << (32 - s)).astype(np.uint64)
        r = lo + (draws(v.size, seed) < T).astype(np.int64)
    else:
        r = v << (-s)
    sat_pos = int((r > qmax).sum())
    sat_neg = int((r < qmin).sum())
    y = np.clip(r, qmin, qmax)
    return y.astype(np.int16).reshape(q.shape), (int((y == 0).sum()), sat_pos, sat_neg)


def epilogue_stochastic(acc, bias_q, bias_frac_bits: int, acc_frac_bits: int, relu: bool, out_n_bits: int,
                        out_frac_bits: int, seed: int):
    """Epilogue of an LP layer whose rounding_scheme is STOCHASTIC (paper Sec. 2: a per-layer
    parameter; Sec. 2.4): bias, ReLU, then the pre-activation value v (an integer in units of
    2^-acc_frac_bits) is brought to the output format by one of its two neighbouring codes.
    Readings (the paper gives no formula), in line with S1-S2 above:
    E1  s = acc_frac_bits - out_frac_bits.  For s > 0, v / 2^s = q + rem / 2^s with q = floor(v / 2^s)
        and 0 <= rem < 2^s, all integers; the result is q + 1 with probability T / 2^32,
        T = rem * 2^(32 - s) (exact: s <= 30 because both operand formats have at most 15
        fractional bits), else q.  rem = 0 never moves.  For s <= 0 the left shift is exact.
    E2  The draw of the output with row-major index i over acc's [outer][channels] elements is the
        word R_i of reading S2 (same generator, same key = seed); the value moves up iff R_i < T.
    E3  Saturation and the three counters as in the deterministic epilogue, after the rounding.
    acc: int64 array [..., channels]; returns (int16 array, (zeros, sat_pos, sat_neg))."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    ch = acc.shape[-1]
    v = acc.reshape(-1, ch).copy()
    if bias_q is not None:
        b = np.asarray(bias_q, dtype=np.int64).reshape(1, ch)
        v = v + b * np.int64(1 << (acc_frac_bits - bias_frac_bits))
    if relu:
        v = np.maximum(v, 0)
    v = v.reshape(-1)
    s = acc_frac_bits - out_frac_bits
    qmin, qmax = -(1 << (out_n_bits - 1)), (1 << (out_n_bits - 1)) - 1
    if s > 0:
        assert s <= 32
        q = v >> s                                    # floor (arithmetic shift)
        rem = v - (q << s)                            # 0 <= rem < 2^s
        T = rem.astype(np.uint64) << np.uint64(32 - s)
        r = q + (draws(v.size, seed) < T).astype(np.int64)
    else:
        lim = np.int64(1) << np.int64(40)             # beyond any output range after the shift
        r = np.clip(v, -lim, lim) << np.int64(-s)
    sat_pos = int((r > qmax).sum())
    sat_neg = int((r < qmin).sum())
    y = np.clip(r, qmin, qmax)
    return y.astype(np.int16).reshape(acc.shape), (int((y == 0).sum()), sat_pos, sat_neg)
