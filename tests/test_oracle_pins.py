"""Pins for the CPU oracle against things other than itself.

Hand-worked values for the formats the paper names, invariants, brute force
over all codes, exact decimal arithmetic from the standard library, and
double-precision library convolutions / matrix products (exact for these
magnitudes).  None of these re-use the oracle's own formulae.
"""
import os
from decimal import ROUND_HALF_UP, Decimal
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import reference as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


# ---------------------------------------------------------------- quantizer (Sec. 2)
def test_handworked_qmf_values():
    for n, f, x, q, sat in _read_rows("qmf_handworked.txt"):
        n, f, q, sat = int(n), int(f), int(q), int(sat)
        got, cnt = orc.quantize(np.array([float(x)], dtype=np.float32), n, f)
        assert int(got[0]) == q, (n, f, x, int(got[0]), q)
        assert cnt.sat_pos == (1 if sat > 0 else 0), (n, f, x)
        assert cnt.sat_neg == (1 if sat < 0 else 0), (n, f, x)
        assert cnt.zeros == (1 if q == 0 else 0)


def _nearest_code_bruteforce(x: float, n: int, f: int) -> int:
    """Nearest representable value by exhaustive search over all 2^n codes, in exact
    rational arithmetic; ties go to the larger magnitude; outside the range the nearest
    code is the end of the range."""
    xv = Fraction(x)
    best, best_d = None, None
    for q in range(-(1 << (n - 1)), 1 << (n - 1)):
        d = abs(xv - Fraction(q, 1 << f))
        if best is None or d < best_d or (d == best_d and abs(q) > abs(best)):
            best, best_d = q, d
    return best


def test_quantizer_is_nearest_code_bruteforce_n4():
    # every fp32 value on a fine grid across and beyond the range of Q1.3 ... Q4.0
    for f in range(0, 4):
        step = 2.0 ** -(f + 3)
        xs = np.arange(-80, 81, dtype=np.float64) * step * (2.0 ** f) / 4 + 0.0
        xs = np.concatenate([xs, np.arange(-80, 81) * step]).astype(np.float32)
        got, _ = orc.quantize(xs, 4, f)
        for x, g in zip(xs, got):
            assert int(g) == _nearest_code_bruteforce(float(x), 4, f), (f, float(x))


def test_quantizer_against_decimal_half_up_random():
    rng = np.random.default_rng(1)
    for n, f in [(16, 15), (16, 8), (16, 2), (12, 9), (8, 4), (5, 0)]:
        xs = (rng.standard_normal(4000) * 2.0 ** (n - 1 - f) * 0.6).astype(np.float32)
        # add exact ties
        ties = ((rng.integers(-(1 << (n - 1)), 1 << (n - 1), 200) + 0.5) * 2.0 ** -f).astype(np.float32)
        xs = np.concatenate([xs, ties])
        got, cnt = orc.quantize(xs, n, f)
        lo, hi = -(1 << (n - 1)), (1 << (n - 1)) - 1
        sp = sn = z = 0
        for x, g in zip(xs, got):
            r = int((Decimal(float(x)) * (1 << f)).quantize(Decimal(1), rounding=ROUND_HALF_UP))
            sp += r > hi
            sn += r < lo
            r = min(max(r, lo), hi)
            z += r == 0
            assert int(g) == r, (n, f, float(x))
        assert (cnt.sat_pos, cnt.sat_neg, cnt.zeros) == (sp, sn, z)


def test_quantizer_invariants_exhaustive_16bit():
    n = 16
    for f in (15, 8, 0):
        q_all = np.arange(-32768, 32768, dtype=np.int64)
        x = (q_all * 2.0 ** -f).astype(np.float32)          # exact: 16-bit integers scaled
        q, cnt = orc.quantize(x, n, f)
        assert np.array_equal(q.astype(np.int64), q_all)    # idempotence on representable values
        assert cnt.sat_pos == 0 and cnt.sat_neg == 0 and cnt.zeros == 1
        assert np.array_equal(orc.dequantize(q, f), q_all * 2.0 ** -f)


def test_quantizer_monotone_bounded_symmetric_error():
    rng = np.random.default_rng(2)
    n, f = 12, 7
    xs = np.sort((rng.standard_normal(20000) * 12).astype(np.float32))
    q, _ = orc.quantize(xs, n, f)
    qi = q.astype(np.int64)
    assert np.all(np.diff(qi) >= 0)
    assert qi.min() >= -(1 << (n - 1)) and qi.max() <= (1 << (n - 1)) - 1
    inside = (xs.astype(np.float64) * 2 ** f < (1 << (n - 1)) - 0.5) & (xs.astype(np.float64) * 2 ** f > -(1 << (n - 1)) - 0.5)
    err = np.abs(orc.dequantize(q, f) - xs.astype(np.float64))
    assert np.all(err[inside] <= 2.0 ** -(f + 1))
    # odd symmetry away from the asymmetric end of the range
    qn, _ = orc.quantize(-xs, n, f)
    keep = np.abs(qi) < (1 << (n - 1)) - 1
    assert np.array_equal(qn.astype(np.int64)[keep], -qi[keep])


def test_quantizer_special_values():
    x = np.array([np.nan, np.inf, -np.inf, -0.0, 1e-45, -1e-45, 3e38, -3e38], dtype=np.float32)
    q, cnt = orc.quantize(x, 16, 8)
    assert q.tolist() == [0, 32767, -32768, 0, 0, 0, 32767, -32768]
    assert (cnt.sat_pos, cnt.sat_neg, cnt.zeros) == (2, 2, 4)


def test_relu_commutes_with_quantizer():
    rng = np.random.default_rng(3)
    xs = (rng.standard_normal(5000) * 3).astype(np.float32)
    a, ca = orc.quantize(xs, 16, 10, relu=True)
    b, _ = orc.quantize(xs, 16, 10, relu=False)
    assert np.array_equal(a, np.maximum(b, 0))
    assert ca.zeros == int(np.sum(np.maximum(b, 0) == 0))
    c, _ = orc.quantize(np.maximum(xs, 0), 16, 10)
    assert np.array_equal(a, c)


def test_coarser_format_creates_zeros():
    # Sec. 3.1: quantization raises the number of zero activations
    rng = np.random.default_rng(4)
    xs = np.abs(rng.standard_normal(10000)).astype(np.float32)
    zeros = [orc.quantize(xs, 16, f)[1].zeros for f in (14, 8, 4, 2, 0)]
    assert zeros == sorted(zeros) and zeros[-1] > zeros[0]
    assert orc.quantize(np.array([0.1], np.float32), 16, 2)[0][0] == 0


# ---------------------------------------------------------------- planes
def test_plane_split_handworked_and_exhaustive():
    q = np.array([-1, -32768, 32767, -255, 300, 0, 255, 256, -256, -257], dtype=np.int16)
    hi, lo = orc.split_planes(q)
    assert hi.tolist() == [-1, -128, 127, -1, 1, 0, 0, 1, -1, -2]
    assert lo.tolist() == [255, 0, 255, 1, 44, 0, 255, 0, 0, 255]
    q_all = np.arange(-32768, 32768, dtype=np.int16)
    hi, lo = orc.split_planes(q_all)
    assert np.array_equal(256 * hi.astype(np.int64) + lo.astype(np.int64), q_all.astype(np.int64))


# ---------------------------------------------------------------- range rule (Sec. 2.3)
@pytest.mark.parametrize("M,n,m", [(0.0, 16, 0), (0.99, 16, 0), (1.0, 16, 1), (1.5, 16, 1),
                                   (2.0, 16, 2), (127.9, 16, 7), (128.0, 16, 8), (300.0, 8, 7),
                                   (1e-30, 16, 0), (float("inf"), 16, 15), (40000.0, 16, 15),
                                   (16383.9, 16, 14), (16384.0, 16, 15), (3.0, 1, 0)])
def test_range_rule_handworked(M, n, m):
    assert orc.int_bits_from_max(M, n) == m


def test_range_from_tensor_and_paper_formats():
    # Sec. 3.1: weights "very small and centered around zero" fit with 1-2 integer bits
    x = np.array([0.02, -0.6, 0.3, np.nan], dtype=np.float32)
    M, m, f = orc.measure_range(x, 16)
    assert abs(M - 0.6) < 1e-7 and (m, f) == (0, 15)        # Q1.15
    M, m, f = orc.measure_range(np.array([1.7, -0.2], np.float32), 16)
    assert (m, f) == (1, 14)                                  # Q2.14
    M, m, f = orc.measure_range(np.array([-5000.0, 20.0], np.float32), 16)
    assert (m, f) == (13, 2)                                  # Q14.2
    M, m, f = orc.measure_range(np.array([100.0], np.float32), 16)
    assert (m, f) == (7, 8)                                   # Q8.8


def test_range_rule_guarantees_representable_up_to_one_lsb():
    rng = np.random.default_rng(5)
    for _ in range(200):
        n = int(rng.integers(2, 17))
        x = (rng.standard_normal(64) * 10.0 ** rng.uniform(-3, 3)).astype(np.float32)
        M, m, f = orc.measure_range(x, n)
        q, cnt = orc.quantize(x, n, f)
        if m < n - 1 or M < 2.0 ** (n - 1):
            assert cnt.sat_neg == 0
            assert np.all(np.abs(orc.dequantize(q, f) - x.astype(np.float64)) <= 2.0 ** -f)
            if m > 0:
                assert M >= 2.0 ** (m - 1)                    # m is the smallest that fits


def test_range_accumulator_form_matches_float_form():
    for F in (0, 5, 20, 29):
        for A in [0, 1, (1 << F) - 1, 1 << F, (1 << F) + 1, 3 << F, (1 << (F + 6)) - 1, 1 << (F + 6),
                  1 << (F + 20)]:
            want = orc.int_bits_from_max(float(Fraction(A, 1 << F)), 16) if A < (1 << 52) else None
            got = orc.int_bits_from_acc(A, F, 16)
            exact = 0
            while exact < 15 and not (Fraction(A, 1 << F) < (1 << exact)):
                exact += 1
            assert got == exact
            if want is not None and A < (1 << 24):
                assert got == want


# ---------------------------------------------------------------- accumulation (Sec. 2)
def test_handworked_dot_product():
    kv, shifts = {}, []
    for row in _read_rows("dot_product_handworked.txt"):
        if row[0] == "shift":
            shifts.append(tuple(int(t) for t in row[1:]))
        else:
            kv[row[0]] = [int(t) for t in row[1:]]
    xq, _ = orc.quantize(np.array([[0.5, 0.25]], np.float32), 16, 15)
    wq, _ = orc.quantize(np.array([[1.0, -0.5]], np.float32), 16, 14)
    bq, _ = orc.quantize(np.array([0.1], np.float32), 16, 14)
    assert xq.ravel().tolist() == kv["x_q"] and wq.ravel().tolist() == kv["w_q"]
    assert bq.tolist() == kv["bias_q"]
    acc = orc.ip_acc(xq, wq)
    assert acc.ravel().tolist() == kv["acc"]
    y, _ = orc.epilogue(acc, bq, 14, 29, False, 16, 15)
    assert y.ravel().tolist() == kv["y_q"]
    assert orc.epilogue_range(acc, bq, 14, 29, False) == kv["v"][0]
    assert orc.epilogue_range(acc, None, 0, 29, False) == kv["acc"][0]
    for v, s, r in shifts:
        assert orc.shift_round(v, s) == r


def _torch_conv_double(xq, fx, wq, fw, pad, stride):
    """Library convolution (double) of the dequantized operands; exact because every product
    is < 2^30 and every sum < 2^53."""
    x = torch.from_numpy(xq.astype(np.float64) * 2.0 ** -fx).permute(0, 3, 1, 2)
    w = torch.from_numpy(wq.astype(np.float64) * 2.0 ** -fw).permute(0, 3, 1, 2)
    y = torch.nn.functional.conv2d(x, w, None, stride=stride, padding=pad)
    return y.permute(0, 2, 3, 1).numpy()


@pytest.mark.parametrize("shape", [
    # N, H, W, C, K, R, S, pad, stride
    (2, 7, 6, 5, 4, 3, 3, 1, 1), (1, 9, 9, 3, 7, 5, 5, 0, 1), (2, 8, 10, 4, 3, 3, 3, 1, 2),
    (1, 5, 5, 2, 2, 1, 1, 0, 1), (3, 6, 6, 1, 5, 3, 2, 0, 1), (1, 11, 7, 6, 2, 3, 3, 2, 2),
])
def test_conv_equals_double_precision_library_conv(shape):
    N, H, W, C, K, R, S, pad, stride = shape
    rng = np.random.default_rng(sum(shape))
    xq = rng.integers(-32768, 32768, (N, H, W, C)).astype(np.int16)
    wq = rng.integers(-32768, 32768, (K, R, S, C)).astype(np.int16)
    fx, fw = 9, 14
    acc = orc.conv_acc(xq, wq, (pad, pad), (stride, stride))
    ref = _torch_conv_double(xq, fx, wq, fw, pad, stride) * 2.0 ** (fx + fw)
    assert acc.shape == ref.shape
    assert np.array_equal(acc.astype(np.float64), ref)
    # spot-check entry point
    n, oh, ow, k = N - 1, acc.shape[1] // 2, acc.shape[2] - 1, K - 1
    assert orc.conv_acc_at(xq, wq, (pad, pad), (stride, stride), n, oh, ow, k) == acc[n, oh, ow, k]


def test_ip_equals_integer_matmul():
    rng = np.random.default_rng(7)
    xq = rng.integers(-32768, 32768, (5, 37)).astype(np.int16)
    wq = rng.integers(-32768, 32768, (11, 37)).astype(np.int16)
    acc = orc.ip_acc(xq, wq)
    assert np.array_equal(acc, xq.astype(np.int64) @ wq.astype(np.int64).T)


def test_structural_special_cases():
    rng = np.random.default_rng(8)
    xq = rng.integers(-2000, 2000, (2, 6, 5, 4)).astype(np.int16)
    # 1x1 convolution is an inner product over pixels
    w1 = rng.integers(-300, 300, (3, 1, 1, 4)).astype(np.int16)
    a = orc.conv_acc(xq, w1)
    b = orc.ip_acc(xq.reshape(-1, 4), w1.reshape(3, 4)).reshape(2, 6, 5, 3)
    assert np.array_equal(a, b)
    # inner product is a convolution over a 1x1 image
    c = orc.conv_acc(xq.reshape(2, 1, 1, -1), rng.integers(-9, 9, (7, 1, 1, 120)).astype(np.int16))
    assert c.shape == (2, 1, 1, 7)
    # centre-tap delta kernel reproduces the input channel
    wd = np.zeros((4, 3, 3, 4), dtype=np.int16)
    for k in range(4):
        wd[k, 1, 1, k] = 1
    assert np.array_equal(orc.conv_acc(xq, wd, (1, 1)), xq.astype(np.int64))
    # off-centre delta shifts: tap (r=0, s=1) reads the pixel one row above (cross-correlation)
    ws = np.zeros((1, 3, 3, 4), dtype=np.int16)
    ws[0, 0, 1, 2] = 1
    sh = orc.conv_acc(xq, ws, (1, 1))[..., 0]
    assert np.array_equal(sh[:, 1:, :], xq[:, :-1, :, 2]) and np.all(sh[:, 0, :] == 0)
    # all-ones kernel on an all-ones image counts the taps inside the image: 4 / 6 / 9
    ones = np.ones((1, 5, 5, 1), dtype=np.int16)
    box = orc.conv_acc(ones, np.ones((1, 3, 3, 1), dtype=np.int16), (1, 1))[0, :, :, 0]
    assert box[0, 0] == 4 and box[0, 2] == 6 and box[2, 2] == 9 and box[4, 4] == 4
    # batch independence, linearity in x, output-channel permutation
    w = rng.integers(-500, 500, (6, 3, 3, 4)).astype(np.int16)
    full = orc.conv_acc(xq, w, (1, 1))
    assert np.array_equal(full[1:], orc.conv_acc(xq[1:], w, (1, 1)))
    assert np.array_equal(orc.conv_acc((2 * xq).astype(np.int16), w, (1, 1)), 2 * full)
    perm = np.array([3, 0, 5, 1, 2, 4])
    assert np.array_equal(orc.conv_acc(xq, w[perm], (1, 1)), full[..., perm])


# ---------------------------------------------------------------- epilogue (Sec. 2.1)
def test_epilogue_against_decimal_arithmetic():
    rng = np.random.default_rng(9)
    acc = rng.integers(-(1 << 40), 1 << 40, (50, 6)).astype(np.int64)
    acc[0, :] = [0, 1 << 13, -(1 << 13), (1 << 13) - 1, 3 << 13, -(3 << 13)]   # exact ties at s = 14
    bq = rng.integers(-32768, 32768, 6).astype(np.int16)
    for relu in (False, True):
        for (F, fb, n_out, f_out) in [(29, 14, 16, 15), (29, 14, 16, 3), (20, 20, 8, 2), (10, 4, 16, 12),
                                      (30, 15, 4, 0)]:
            y, cnt = orc.epilogue(acc, bq, fb, F, relu, n_out, f_out)
            lo, hi = -(1 << (n_out - 1)), (1 << (n_out - 1)) - 1
            sp = sn = z = 0
            vmax = 0
            for i in range(acc.shape[0]):
                for c in range(6):
                    v = int(acc[i, c]) + int(bq[c]) * (1 << (F - fb))
                    if relu:
                        v = max(v, 0)
                    vmax = max(vmax, abs(v))
                    r = int((Decimal(v) / Decimal(2) ** (F - f_out)).quantize(Decimal(1), rounding=ROUND_HALF_UP))
                    sp += r > hi
                    sn += r < lo
                    r = min(max(r, lo), hi)
                    z += r == 0
                    assert int(y[i, c]) == r
            assert (cnt.sat_pos, cnt.sat_neg, cnt.zeros) == (sp, sn, z)
            assert orc.epilogue_range(acc, bq, fb, F, relu) == vmax


def test_layer_equals_float_layer_then_quantize():
    """Brute-force float-vs-fixed: the fixed-point layer output equals the quantizer applied to
    the real-valued (double) layer on the dequantized operands, and so stays within half an
    output LSB of it."""
    rng = np.random.default_rng(10)
    x = np.maximum(rng.standard_normal((2, 6, 6, 8)), 0).astype(np.float32)
    w = (rng.standard_normal((5, 3, 3, 8)) * 0.15).astype(np.float32)
    b = (rng.standard_normal(5) * 0.01).astype(np.float32)
    fx = orc.measure_range(x, 16)[2]
    xq, _ = orc.quantize(x, 16, fx)
    wq, fw = orc.quantize_param(w, 16)
    bq, _ = orc.quantize(b, 16, fw)
    acc = orc.conv_acc(xq, wq, (1, 1))
    res = orc.lp_layer(acc, fx, fw, bq, fw, True, 16)
    real = _torch_conv_double(xq, fx, wq, fw, 1, 1) + bq.astype(np.float64) * 2.0 ** -fw
    real = np.maximum(real, 0)
    assert real.max() < 2.0 ** (15 - res.frac_bits)
    if res.frac_bits < 15:
        assert real.max() >= 2.0 ** (14 - res.frac_bits)     # decimal point as far left as the range allows
    yq, _ = orc.quantize(real.astype(np.float32), 16, res.frac_bits)
    # real is not an fp32 number in general: compare through exact decimal rounding instead
    for v, got in zip(real.ravel(), res.y.ravel()):
        r = int((Decimal(float(v)) * (1 << res.frac_bits)).quantize(Decimal(1), rounding=ROUND_HALF_UP))
        assert int(got) == min(r, 32767)
    assert np.all(np.abs(orc.dequantize(res.y, res.frac_bits) - real) <= 2.0 ** -res.frac_bits)
    del yq


def test_epilogue_left_shift_of_huge_accumulators():
    """Requantizing to MORE fractional bits than the accumulator has (an exact left shift) with
    accumulators as large as the longest admitted reductions produce: v * 2^15 no longer fits 64
    bits, the result is still the saturated exact product.  Hand-worked: with F = 0 and Q1.15 out,
    1 -> 32768 saturates to 32767, -1 -> -32768 exactly, anything larger in magnitude saturates."""
    acc = np.array([[2 ** 50, -(2 ** 50), 2 ** 62, -(2 ** 62), 1, -1, 0]], dtype=np.int64)
    y, cnt = orc.epilogue(acc, None, 0, 0, False, 16, 15)
    assert y.tolist() == [[32767, -32768, 32767, -32768, 32767, -32768, 0]]
    assert (cnt.zeros, cnt.sat_pos, cnt.sat_neg) == (1, 3, 2)
    y, cnt = orc.epilogue(acc, None, 0, 0, True, 16, 15)
    assert y.tolist() == [[32767, 0, 32767, 0, 32767, 0, 0]]
    assert (cnt.zeros, cnt.sat_pos, cnt.sat_neg) == (4, 3, 0)
    assert orc.shift_round(3, -2) == 12 and orc.shift_round(-3, -2) == -12
    assert orc.shift_round(2 ** 47, -15) == 2 ** 62 and orc.shift_round(-(2 ** 47), -15) == -(2 ** 62)


def test_requantize_format_change():
    q = np.array([5, -5, 6, -6, 3, 4, -4, 32767, -32768, 0], dtype=np.int16)
    y, cnt = orc.requantize(q, 10, False, 16, 9)          # one bit coarser
    assert y.tolist() == [3, -3, 3, -3, 2, 2, -2, 16384, -16384, 0]
    y, cnt = orc.requantize(q, 10, True, 16, 12)          # two bits finer: saturates the ends
    assert y.tolist() == [20, 0, 24, 0, 12, 16, 0, 32767, 0, 0]
    assert (cnt.sat_pos, cnt.sat_neg, cnt.zeros) == (1, 0, 5)
    y, _ = orc.requantize(q, 10, False, 8, 3)
    assert y.tolist()[:7] == [0, 0, 0, 0, 0, 0, 0] and y.tolist()[7:9] == [127, -128]


# ---------------------------------------------------------------- pooling
def test_maxpool_commutes_with_quantizer():
    rng = np.random.default_rng(11)
    x = (rng.standard_normal((2, 6, 8, 3)) * 2).astype(np.float32)
    q, _ = orc.quantize(x, 16, 9)
    pooled_real = x.reshape(2, 3, 2, 4, 2, 3).max(axis=(2, 4))
    want, _ = orc.quantize(pooled_real, 16, 9)
    assert np.array_equal(orc.maxpool2x2(q), want)
    # negative-only window: maximum is the least negative value, not zero
    neg = -np.arange(1, 17, dtype=np.int16).reshape(1, 4, 4, 1)
    assert orc.maxpool2x2(neg).ravel().tolist() == [-1, -3, -9, -11]


# ---------------------------------------------------------------- network driver
def test_network_driver_lenet_shapes_and_formats():
    from paper_1711_04713_b200 import workloads as wl
    specs = wl.lenet_specs()
    params = wl.make_params(specs, seed=0)
    x = wl.lenet_input(2, seed=0)
    rec = orc.run_network(params, x, (16, 15), 16)
    shapes = [r["y"].shape for r in rec]
    assert shapes == [(2, 28, 28, 1), (2, 24, 24, 20), (2, 12, 12, 20), (2, 8, 8, 50), (2, 4, 4, 50),
                      (2, 500), (2, 10)]
    for r in rec:
        if r["type"] in ("conv", "ip"):
            assert 0 <= r["frac_bits"] <= 15
            assert r["counters"].sat_neg == 0
            # the decimal point chosen from the batch range leaves at most the one-LSB edge case
            assert r["counters"].sat_pos <= 1
    # running again with the formats fixed reproduces the calibrated run
    fixed = [r["frac_bits"] for r in rec if r["type"] in ("conv", "ip")]
    rec2 = orc.run_network(params, x, (16, 15), 16, fixed_formats=fixed)
    for a, b in zip(rec, rec2):
        assert np.array_equal(a["y"], b["y"])


# ---------------------------------------------------------------- thresholded bit allocation (Sec. 2.3)
def test_bit_allocation_handworked():
    from oracle import bit_allocation as ba
    for row in _read_rows("bit_allocation_handworked.txt"):
        if row[0] == "bits":
            assert int(ba.integer_bits_needed(np.array([float(row[1])]))[0]) == int(row[2]), row
        elif row[0] == "walloc":
            n, f, thr = int(row[1]), int(row[2]), float(row[3])
            hist = [int(v) for v in row[4:4 + ba.HIST_BINS]]
            assert ba.choose_int_bits_from_widths(hist, f, n, thr) == int(row[4 + ba.HIST_BINS]), row
        else:
            n, thr = int(row[1]), float(row[2])
            hist = [int(v) for v in row[3:3 + ba.HIST_BINS]]
            assert ba.choose_int_bits(hist, n, thr) == int(row[3 + ba.HIST_BINS]), row


def test_bit_histogram_against_exact_integer_definition():
    """b(x) = smallest m >= 0 with |x| < 2^m, checked with exact rationals; the histogram is its
    count; threshold 0 reproduces the max-based rule of the range measurement."""
    from oracle import bit_allocation as ba
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(4000) * np.exp(rng.uniform(-3, 9, 4000))).astype(np.float32)
    x[:8] = [0.0, -0.0, 1.0, -1.0, 2.0 ** 15, -(2.0 ** 16), 65535.9, 1e30]
    want = []
    for v in x.tolist():
        fv, m = abs(Fraction(v)), 0
        while fv >= Fraction(2) ** m:
            m += 1
        want.append(m)
    got = ba.integer_bits_needed(x)
    assert got.tolist() == want
    hist = ba.bit_histogram(x)
    assert int(hist.sum()) == x.size
    for b in range(ba.HIST_BINS - 1):
        assert int(hist[b]) == sum(1 for m in want if m == b)
    assert int(hist[-1]) == sum(1 for m in want if m >= ba.HIST_BINS - 1)
    for n in (4, 8, 16):
        assert ba.choose_int_bits(hist, n, 0.0) == orc.measure_range(x, n)[1]
    # specials: NaN skipped, Inf in the top bin
    h2 = ba.bit_histogram(np.array([np.nan, np.inf, -np.inf, 0.5], dtype=np.float32))
    assert int(h2.sum()) == 3 and int(h2[-1]) == 2 and int(h2[0]) == 1


def test_bit_allocation_is_monotone_and_bounds_the_loss():
    from oracle import bit_allocation as ba
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(20000) * 40).astype(np.float32)
    hist = ba.bit_histogram(x)
    prev = None
    for thr in (0.0, 1e-4, 1e-3, 1e-2, 0.05, 0.3, 1.0):
        m = ba.choose_int_bits(hist, 16, thr)
        lost = int((ba.integer_bits_needed(x) > m).sum())
        assert lost <= thr * x.size                      # the accepted loss is within the threshold
        if m > 0:                                        # and one bit fewer would exceed it
            assert int((ba.integer_bits_needed(x) > m - 1).sum()) > thr * x.size
        assert prev is None or m <= prev                 # a larger threshold never needs more bits
        prev = m
    # the lost values are exactly those the quantizer saturates (up to the half-LSB edge)
    m = ba.choose_int_bits(hist, 16, 0.01)
    _, cnt = orc.quantize(x, 16, 15 - m)
    assert cnt.sat_pos + cnt.sat_neg >= int((ba.integer_bits_needed(x) > m).sum())


def test_twos_complement_width():
    from oracle import bit_allocation as ba
    q = np.array([0, -1, 1, -2, 2, 7, 8, -8, -9, 127, 128, -128, -129, 32767, -32768])
    assert ba.twos_complement_width(q).tolist() == [1, 1, 2, 2, 3, 4, 5, 4, 5, 8, 9, 8, 9, 16, 16]


def _fits(q: int, f: int, m: int) -> bool:
    """Whether the real value q * 2^-f is a code of the format with m integer bits and f fractional
    bits (plus sign): -2^m <= value <= 2^m - 2^-f.  Exact rationals, from the format's definition."""
    v = Fraction(q, 1 << f)
    return -(Fraction(2) ** m) <= v <= Fraction(2) ** m - Fraction(1, 1 << f)


def _allocate(lost_with, total: int, n_bits: int, thr: float) -> int:
    """Sec. 2.3 as stated: start with every non-sign bit in the integer part, take one away while the
    values that would no longer be representable number at most thr * total."""
    m = n_bits - 1
    while m > 0 and lost_with(m - 1) <= thr * total:
        m -= 1
    return m


def test_width_allocation_against_exact_rational_definition():
    """choose_int_bits_from_widths on the histogram of a stored tensor == the allocation done value by
    value with exact rationals on the real values q * 2^-f; a larger threshold never needs more bits;
    the accepted loss is within the threshold and one bit fewer would exceed it."""
    from oracle import bit_allocation as ba
    rng = np.random.default_rng(5)
    for n, f in [(16, 8), (16, 2), (12, 9), (8, 3), (8, 0), (4, 1)]:
        qmin, qmax = -(1 << (n - 1)), (1 << (n - 1)) - 1
        q = np.clip(np.round(rng.standard_normal(700) * 2.0 ** rng.uniform(0, n - 1, 700)), qmin, qmax).astype(np.int64)
        q[:6] = [qmin, qmax, 0, -1, 1 << f if (1 << f) <= qmax else 1, -(1 << f) if -(1 << f) >= qmin else -1]
        hist = ba.width_histogram(q)
        assert int(hist.sum()) == q.size and int(hist[0]) == 0
        prev = None
        for thr in (0.0, 0.003, 0.02, 0.1, 0.4, 1.0):
            want = _allocate(lambda m: sum(1 for v in q.tolist() if not _fits(v, f, m)), q.size, n, thr)
            got = ba.choose_int_bits_from_widths(hist, f, n, thr)
            assert got == want, (n, f, thr)
            lost = sum(1 for v in q.tolist() if not _fits(v, f, got))
            assert lost <= thr * q.size
            if got > 0:
                assert sum(1 for v in q.tolist() if not _fits(v, f, got - 1)) > thr * q.size
            assert prev is None or got <= prev
            prev = got
    # a value that does not fit is exactly one the requantizer to (n, n-1-m) saturates
    q = rng.integers(-32768, 32768, 3000).astype(np.int16)
    m = ba.choose_int_bits_from_widths(ba.width_histogram(q), 9, 16, 0.6)
    f_new = 15 - m
    assert f_new > 9                                     # bits moved to the fraction: an exact left shift
    _, cnt = orc.requantize(q, 9, False, 16, f_new)
    assert cnt.sat_pos + cnt.sat_neg == sum(1 for v in q.tolist() if not _fits(int(v), 9, m))


def _restated_threshold_network(layers, x, n, thr):
    """The thresholded workflow of Sec. 2.1 / 2.3 on a tiny stack, restated from the definitions in
    exact rational / integer arithmetic with plain loops (nothing of the oracle is called):
    formats of fp32 tensors from how many values need more integer bits than offered; a layer output
    first stored with the format its maximum needs, then, if the threshold lets integer bits go,
    stored again from the exact sums with the finer format."""
    qmin, qmax = -(1 << (n - 1)), (1 << (n - 1)) - 1

    def rnd(v: Fraction) -> int:                        # nearest integer, ties away from zero
        a = abs(v)
        r = int(a + Fraction(1, 2))                     # floor(a + 1/2)
        return r if v >= 0 else -r

    def fmt_real(vals):                                 # fractional bits for real values
        vals = [abs(Fraction(float(v))) for v in vals]
        m = _allocate(lambda mm: sum(1 for v in vals if v >= Fraction(2) ** mm), len(vals), n, thr)
        return n - 1 - m

    def quant(vals, f):
        return [min(max(rnd(Fraction(float(v)) * (1 << f)), qmin), qmax) for v in vals]

    out = []
    fx = fmt_real(x.reshape(-1))
    a = np.array(quant(x.reshape(-1), fx), dtype=np.int64).reshape(x.shape)
    out.append((fx, a.copy()))
    for L in layers:
        if L["type"] == "pool":
            N, H, W, C = a.shape
            p = np.zeros((N, H // 2, W // 2, C), dtype=np.int64)
            for idx in np.ndindex(*p.shape):
                nn, i, j, c = idx
                p[idx] = max(a[nn, 2 * i, 2 * j, c], a[nn, 2 * i + 1, 2 * j, c], a[nn, 2 * i, 2 * j + 1, c],
                             a[nn, 2 * i + 1, 2 * j + 1, c])
            a = p
            out.append((fx, a.copy()))
            continue
        fw = fmt_real(L["w"].reshape(-1))
        w = np.array(quant(L["w"].reshape(-1), fw), dtype=np.int64).reshape(L["w"].shape)
        b = quant(L["b"], fw)
        F = fx + fw
        if L["type"] == "conv":
            N, H, W, C = a.shape
            K, R, S, _ = w.shape
            pad = L["pad"]
            OH, OW = H + 2 * pad - R + 1, W + 2 * pad - S + 1
            v = np.zeros((N, OH, OW, K), dtype=object)
            for nn, i, j, k in np.ndindex(N, OH, OW, K):
                t = 0
                for r in range(R):
                    for s_ in range(S):
                        ih, iw = i + r - pad, j + s_ - pad
                        if 0 <= ih < H and 0 <= iw < W:
                            for c in range(C):
                                t += int(a[nn, ih, iw, c]) * int(w[k, r, s_, c])
                v[nn, i, j, k] = t + (b[k] << fx)
        else:
            flat = a.reshape(a.shape[0], -1)
            v = np.zeros((flat.shape[0], w.shape[0]), dtype=object)
            for i, o in np.ndindex(*v.shape):
                v[i, o] = sum(int(p) * int(q) for p, q in zip(flat[i], w[o])) + (b[o] << fx)
        if L["relu"]:
            for idx in np.ndindex(*v.shape):
                v[idx] = max(v[idx], 0)
        vals = [Fraction(int(t), 1 << F) for t in v.reshape(-1)]
        top = max(abs(t) for t in vals)
        m0 = 0
        while m0 < n - 1 and top >= Fraction(2) ** m0:
            m0 += 1
        f0 = n - 1 - m0
        y0 = [min(max(rnd(t * (1 << f0)), qmin), qmax) for t in vals]
        m = _allocate(lambda mm: sum(1 for q in y0 if not _fits(q, f0, mm)), len(y0), n, thr)
        f1 = n - 1 - m
        y = y0 if f1 == f0 else [min(max(rnd(t * (1 << f1)), qmin), qmax) for t in vals]
        a = np.array(y, dtype=np.int64).reshape(v.shape)
        fx = f1
        out.append((fx, a.copy(), fw, w, f0))
    return out


def _check_thresholded_network(n_bits, thr) -> int:
    """run_network(threshold > 0) on a tiny conv / pool / inner-product stack: every decimal point
    and every stored integer equals the from-definition restatement above.  Returns how many layer
    outputs gave integer bits away."""
    rng = np.random.default_rng(n_bits * 7 + int(thr * 1000))
    # heavy-tailed values so that a threshold really moves decimal points
    def heavy(shape, scale):
        return (rng.standard_normal(shape) * np.exp(rng.uniform(-2.0, 2.0, shape)) * scale).astype(np.float32)
    layers = [
        {"type": "conv", "w": heavy((3, 3, 3, 2), 0.4), "b": heavy((3,), 0.05), "pad": 1, "stride": 1, "relu": True},
        {"type": "pool"},
        {"type": "ip", "w": heavy((5, 2 * 2 * 3), 0.5), "b": heavy((5,), 0.05), "relu": True},
        {"type": "ip", "w": heavy((4, 5), 0.8), "b": heavy((4,), 0.05), "relu": False},
    ]
    x = heavy((2, 4, 4, 2), 1.5)
    rec = orc.run_network(layers, x, None, n_bits, threshold=thr)
    want = _restated_threshold_network(layers, x, n_bits, thr)
    assert len(rec) == len(want)
    moved = 0
    for r, wnt in zip(rec, want):
        assert r["frac_bits"] == wnt[0], r["type"]
        assert np.array_equal(r["y"].astype(np.int64), wnt[1]), r["type"]
        if r["type"] in ("conv", "ip"):
            assert r["w_frac_bits"] == wnt[2]
            assert np.array_equal(r["wq"].astype(np.int64), wnt[3])
            moved += int(wnt[4] != wnt[0])
    base = orc.run_network(layers, x, None, n_bits)
    assert all(r["frac_bits"] >= b["frac_bits"] for r, b in zip(rec[:1], base[:1]))
    return moved


def test_thresholded_network_driver_against_restatement():
    moved = [_check_thresholded_network(n, t) for n, t in [(8, 0.1), (8, 0.02), (16, 0.05), (6, 0.25)]]
    assert sum(moved) > 0          # not vacuous: somewhere a layer output gives integer bits away


# ---------------------------------------------------------------- stochastic rounding (Sec. 2.4)
def test_stochastic_floor_and_threshold_exact():
    """floor(y) and T = floor(frac(y) * 2^32) against exact rationals, on the values where a
    double-precision y - floor(y) is not exact: tiny negative y (frac = 1 - 2^-k), the largest
    fractions below one, both signs, grid values, and random fp32 values over many binades."""
    from oracle import stochastic as st
    f32 = lambda v: float(np.float32(v))
    ys = [0.0, 1.0, -1.0, 0.5, -0.5, 2.0 ** -60, -(2.0 ** -60), f32(-1e-30), f32(1e-30), -(2.0 ** -33), 2.0 ** -33,
          -(2.0 ** -32), 2.0 ** -32, -(2.0 ** -31), 1 - 2.0 ** -24, -(1 - 2.0 ** -24), 7 + (1 - 2.0 ** -21),
          -7 - (1 - 2.0 ** -21), -(2.0 ** -149), 2.0 ** -149, 32766.998046875, -32768.998046875,
          f32(0.1) * 2.0 ** 15, -f32(0.1) * 2.0 ** 15, 3.0 + 2.0 ** -20, -3.0 - 2.0 ** -20]
    rng = np.random.default_rng(12)
    xs = (rng.standard_normal(3000) * np.exp(rng.uniform(-40, 10, 3000))).astype(np.float32)
    ys += [float(v) * 2.0 ** 9 for v in xs if abs(float(v) * 2.0 ** 9) < 2.0 ** 40]
    lo, T = st.floor_and_threshold(np.array(ys, dtype=np.float64))
    for y, l, t in zip(ys, lo.tolist(), T.tolist()):
        fy = Fraction(y)
        fl = fy.numerator // fy.denominator            # floor of the exact value
        frac = fy - fl
        assert l == fl, y
        assert t == (frac * (1 << 32)).numerator // (frac * (1 << 32)).denominator, y
        assert 0 <= t < (1 << 32)
    # the cases the text names
    lo, T = st.floor_and_threshold(np.array([-(2.0 ** -60), 1 - 2.0 ** -24, -(1 - 2.0 ** -24), 5.0, -5.0]))
    assert lo.tolist() == [-1, 0, -1, 5, -5]
    assert T.tolist() == [(1 << 32) - 1, (1 << 32) - 256, 256, 0, 0]
    # and through the quantizer: a tiny negative value goes to 0 unless the draw is exactly 2^32 - 1,
    # a tiny positive one stays 0 (T = 0: no draw is below it)
    q, _ = st.quantize_stochastic(np.array([-1e-30, 1e-30, -(2.0 ** -140)], dtype=np.float32), 16, 8, seed=5)
    assert q.tolist() == [0, 0, 0]


def test_philox_known_answers():
    from oracle import stochastic as st
    for row in _read_rows("philox4x32_10_kat.txt"):
        w = [int(v, 16) for v in row]
        out = st.philox4x32_10(w[0:4], w[4:6])
        assert [int(v) for v in out] == w[6:10]


def test_philox_draws_layout_and_uniformity():
    from oracle import stochastic as st
    r = st.draws(10, seed=(7 << 32) | 5)
    for i in range(10):                                  # element i uses word i & 3 of block i >> 2
        blk = st.philox4x32_10((i >> 2, 0, 0, 0), (5, 7))
        assert int(r[i]) == int(blk[i & 3])
    big = st.draws(1 << 18, seed=123).astype(np.float64) / 2.0 ** 32
    assert abs(big.mean() - 0.5) < 4e-3 and abs(big.var() - 1.0 / 12.0) < 2e-3
    assert not np.array_equal(st.draws(64, 1), st.draws(64, 2))


def test_stochastic_rounding_support_and_expectation():
    """Sec. 2.4: the result is one of the two nearest fixed-point values and its expectation is the
    unrounded value; values on the grid never move; saturation and specials as the deterministic rule."""
    from oracle import stochastic as st
    n, f = 16, 8
    xs = np.array([0.3, -0.3, 1.0 / 512, -1.0 / 512, 3.14159, -2.71828, 100.123], dtype=np.float32)
    reps = 20000
    x = np.tile(xs, reps)
    q, _ = st.quantize_stochastic(x, n, f, seed=99)
    q = q.reshape(reps, xs.size).astype(np.float64)
    y = xs.astype(np.float64) * 2.0 ** f
    assert np.all((q == np.floor(y)) | (q == np.floor(y) + 1))
    se = np.sqrt(0.25 / reps)
    assert np.all(np.abs(q.mean(axis=0) - y) < 5 * se)
    grid = (np.arange(-300, 300, dtype=np.float32) / 2.0 ** f)
    qg, _ = st.quantize_stochastic(grid, n, f, seed=1)
    assert np.array_equal(qg, np.arange(-300, 300).astype(np.int16))
    sp = np.array([np.nan, np.inf, -np.inf, 1e9, -1e9, 127.999, -0.0], dtype=np.float32)
    qs, (z, sp_, sn) = st.quantize_stochastic(sp, 16, 8, seed=3)
    assert qs.tolist()[:5] == [0, 32767, -32768, 32767, -32768] and qs[6] == 0
    assert qs[5] == 32767 and sp_ in (2, 3) and sn == 2    # 127.999 * 2^8 stays or saturates by one step
    # the deterministic quantizer's result is always one of the two candidates as well
    xr = (np.random.default_rng(4).standard_normal(5000) * 3).astype(np.float32)
    qd, _ = orc.quantize(xr, 16, 10)
    qs2, _ = st.quantize_stochastic(xr, 16, 10, seed=8)
    assert np.all(np.abs(qd.astype(np.int64) - qs2.astype(np.int64)) <= 1)


def test_stochastic_requantization_support_expectation_and_exact_cases():
    """Format change of stored integers with stochastic rounding: one of the two neighbours of
    v / 2^s, mean equal to it, exact when v is a multiple of 2^s or when the shift is to the left,
    and never further than one step from the deterministic requantizer."""
    from oracle import stochastic as st
    vals = np.array([5, -5, 1, -1, 1023, -1023, 12345, -12345, 7, 64], dtype=np.int16)
    reps = 20000
    y, _ = st.requantize_stochastic(np.tile(vals, reps), 10, False, 16, 4, seed=11)      # s = 6
    y = y.reshape(reps, vals.size).astype(np.float64)
    exact = vals.astype(np.float64) / 64.0
    assert np.all((y == np.floor(exact)) | (y == np.floor(exact) + 1))
    assert np.all(np.abs(y.mean(axis=0) - exact) < 5 * np.sqrt(0.25 / reps))
    assert np.all(y[:, 9] == 1.0)                                                         # 64 / 64 exactly
    up, _ = st.requantize_stochastic(vals, 4, False, 16, 6, seed=1)                       # left shift by 2
    assert np.array_equal(up[:6], vals[:6] * 4) and up[6] == 32767 and up[7] == -32768     # 12345 * 4 saturates
    rng = np.random.default_rng(2)
    q = rng.integers(-32768, 32768, 5000).astype(np.int16)
    for relu in (False, True):
        ys, (z, sp, sn) = st.requantize_stochastic(q, 12, relu, 8, 3, seed=5)            # s = 9, saturating
        yd, cd = orc.requantize(q, 12, relu, 8, 3)
        assert np.all(np.abs(ys.astype(np.int64) - yd.astype(np.int64)) <= 1)
        assert z == int((ys == 0).sum()) and sn == (0 if relu else sn)
        assert abs(sp - cd.sat_pos) <= int((np.abs(q.astype(np.int64) - 127 * 512) < 512).sum()) + 1


def test_stochastic_epilogue_handworked_support_expectation_and_exact_cases():
    """The fused layer epilogue with stochastic rounding (Sec. 2 rounding_scheme, Sec. 2.4):
    hand-worked outcomes from the generator's own draws, support on the two neighbours, unbiased
    mean, values on the grid never move, exact left shifts, bias / ReLU / saturation / counters as
    in the deterministic epilogue, and agreement with the (separately pinned) format change of a
    stored tensor where the two coincide."""
    from oracle import stochastic as st
    # hand-worked: four outputs in one row, s = 3, bias 1 * 2^2 added to every accumulator
    seed = 2024
    R = [int(v) for v in st.draws(4, seed)]                   # pinned by the known-answer vectors
    acc = np.array([[5, -5, 16, 1]], dtype=np.int64)          # + 4 -> 9, -1, 20, 5
    y, cnt = st.epilogue_stochastic(acc, np.array([1, 1, 1, 1], dtype=np.int16), 1, 3, False, 16, 0, seed)
    want = []
    for v, r in zip([9, -1, 20, 5], R):
        fl = Fraction(v, 8).numerator // Fraction(v, 8).denominator
        frac = Fraction(v, 8) - fl
        want.append(fl + (1 if r < int(frac * (1 << 32)) else 0))
    assert y.tolist() == [want]
    assert all(t in pair for t, pair in zip(want, [(1, 2), (-1, 0), (2, 3), (0, 1)]))
    assert cnt[0] == sum(1 for t in want if t == 0)
    # support and expectation over many draws, positive and negative values, with ReLU and without
    vals = np.array([5, -5, 1, -1, 1023, -1023, 123457, -123457, 7, 64], dtype=np.int64)
    reps = 20000
    y, _ = st.epilogue_stochastic(np.tile(vals, (reps, 1)), None, 0, 20, False, 16, 14, seed=11)   # s = 6
    y = y.astype(np.float64)
    exact = vals.astype(np.float64) / 64.0
    assert np.all((y == np.floor(exact)) | (y == np.floor(exact) + 1))
    assert np.all(np.abs(y.mean(axis=0) - exact) < 5 * np.sqrt(0.25 / reps))
    assert np.all(y[:, 9] == 1.0)                             # 64 / 64: on the grid
    yr, _ = st.epilogue_stochastic(np.tile(vals, (200, 1)), None, 0, 20, True, 16, 14, seed=12)
    assert np.all(yr[:, [1, 3, 5, 7]] == 0)                   # ReLU before rounding: negatives are exactly 0
    # grid values never move; left shifts are exact; huge accumulators saturate
    grid = (np.arange(-300, 300, dtype=np.int64) * 32).reshape(1, -1)
    yg, _ = st.epilogue_stochastic(grid, None, 0, 5, False, 16, 0, seed=3)
    assert np.array_equal(yg.reshape(-1), np.arange(-300, 300))
    up, c = st.epilogue_stochastic(np.array([[3, -3, 2 ** 50, -(2 ** 50), 0]], dtype=np.int64), None, 0, 2, False,
                                   16, 4, seed=4)
    assert up.tolist() == [[12, -12, 32767, -32768, 0]] and c == (1, 1, 1)
    # same rule as the stored-tensor format change where both apply (16-bit values, no bias)
    rng = np.random.default_rng(6)
    q = rng.integers(-32768, 32768, (37, 24)).astype(np.int16)
    for relu in (False, True):
        a, ca = st.epilogue_stochastic(q.astype(np.int64), None, 0, 12, relu, 8, 3, seed=77)
        b, cb = st.requantize_stochastic(q, 12, relu, 8, 3, seed=77)
        assert np.array_equal(a, b) and ca == cb
    # never further than one step from the deterministic epilogue, equal where rem = 0
    accr = rng.integers(-(2 ** 34), 2 ** 34, (50, 16)).astype(np.int64)
    bq = rng.integers(-32768, 32768, 16).astype(np.int16)
    ys, _ = st.epilogue_stochastic(accr, bq, 15, 28, True, 16, 9, seed=8)
    yd, _ = orc.epilogue(accr, bq, 15, 28, True, 16, 9)
    assert np.all(np.abs(ys.astype(np.int64) - yd.astype(np.int64)) <= 1)
