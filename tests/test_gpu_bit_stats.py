"""GPU parity of the bit-occupancy histograms (paper Sec. 2.2, 2.3) and of the stochastic quantizer
(Sec. 2.4) against the CPU oracle, bit-exact, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import bit_allocation as ba
from oracle import reference as orc
from oracle import stochastic as st
from paper_1711_04713_b200 import binding as B
from tests.util import dev, from_qtensor, q16_of, stats_tuple, to_qtensor

pytestmark = pytest.mark.gpu


def _spread(rng, n):
    """Values over many binades, with zeros, exact powers of two and specials."""
    x = (rng.standard_normal(n) * np.exp(rng.uniform(-4, 12, n))).astype(np.float32)
    k = min(n, 12)
    x[:k] = np.array([0.0, -0.0, 1.0, -1.0, 0.99999994, 2.0, 32768.0, -65536.0, 1e30, np.inf, -np.inf,
                      np.nan], dtype=np.float32)[:k]
    return x


@pytest.mark.parametrize("numel", [0, 1, 31, 33, 1000, 4099, (1 << 20) + 3, 148 * 256 * 8 + 5])
def test_bit_histogram_sizes(numel):
    x = _spread(np.random.default_rng(numel), numel)
    hist = B.new_hist()
    B.adaption_bit_histogram(dev(x) if numel else torch.empty(0, device="cuda"), hist)
    want = ba.bit_histogram(x)
    assert hist.cpu().numpy().astype(np.uint64).tolist() == want.tolist()


def test_bit_histogram_accumulates_and_drives_the_allocation():
    rng = np.random.default_rng(7)
    a, b = _spread(rng, 50000), (rng.standard_normal(70001) * 3).astype(np.float32)
    hist = B.new_hist()
    B.adaption_bit_histogram(dev(a), hist)
    B.adaption_bit_histogram(dev(b)[1:], hist)                     # 4-byte aligned, not 16
    want = ba.bit_histogram(a) + ba.bit_histogram(b[1:])
    got = hist.cpu().numpy().astype(np.uint64)
    assert got.tolist() == want.tolist()
    for n_bits in (16, 8, 4):
        for thr in (0.0, 0.001, 0.01, 0.1):
            f = B.adaption_choose_frac_bits_from_hist(got.tolist(), n_bits, thr)
            assert f == ba.choose_frac_bits(want, n_bits, thr)
    # threshold 0 on one tensor is the range measurement's format
    h1 = B.new_hist()
    B.adaption_bit_histogram(dev(b), h1)
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    B.adaption_measure_range(dev(b), 16, mx, fmt)
    assert B.adaption_choose_frac_bits_from_hist(h1.cpu().tolist(), 16, 0.0) == int(fmt.cpu()[1])


@pytest.mark.parametrize("n_bits", [16, 12, 8, 4])
@pytest.mark.parametrize("shape", [(1000, 64), (37, 3), (129, 20), (4097, 16)])
def test_width_histogram(n_bits, shape):
    rng = np.random.default_rng(n_bits + shape[0])
    # mostly small magnitudes, like quantized weights, plus the extremes of the format
    q = np.clip(np.round(rng.standard_normal(shape) * 2.0 ** rng.uniform(0, n_bits - 1, shape)),
                -(1 << (n_bits - 1)), (1 << (n_bits - 1)) - 1).astype(np.int16)
    q.flat[:2] = [-(1 << (n_bits - 1)), (1 << (n_bits - 1)) - 1]
    x = to_qtensor(q, n_bits, 0)
    hist = B.new_hist()
    B.adaption_width_histogram(x, hist)
    w = ba.twos_complement_width(q)
    want = np.bincount(w, minlength=ba.HIST_BINS)
    assert hist.cpu().numpy().tolist() == want.tolist()
    assert int(hist.sum()) == q.size                                   # padding channels are not counted


@pytest.mark.parametrize("n_bits,frac_bits", [(16, 15), (16, 8), (16, 2), (12, 9), (8, 4), (4, 1)])
@pytest.mark.parametrize("shape", [(1000, 64), (37, 3), (129, 20), (5, 16), (3, 100)])
@pytest.mark.parametrize("relu", [False, True])
def test_quantize_stochastic_matches_oracle(n_bits, frac_bits, shape, relu):
    rng = np.random.default_rng(n_bits * 100 + frac_bits + shape[0])
    x = (rng.standard_normal(shape) * 2.0 ** (n_bits - 2 - frac_bits)).astype(np.float32)
    g = 2.0 ** -frac_bits                                 # one grid step
    special = [np.nan, np.inf, -np.inf, 0.0, -0.0, g, -g, 3 * g, -3 * g, g / 2, -g / 2, g * 2.0 ** -20,
               -g * 2.0 ** -20, g * (1 - 2.0 ** -24), -g * (1 - 2.0 ** -24), g * (1 + 2.0 ** -23),
               -g * (1 + 2.0 ** -23), 1e-30, -1e-30, 3e38, -3e38, 5.5 * g, -5.5 * g, 2.0 ** (n_bits - 1) * g,
               -2.0 ** (n_bits - 1) * g - g / 4]
    x.flat[:len(special)] = np.array(special, dtype=np.float32)
    seed = (0x9E3779B97F4A7C15 * (shape[0] + 1)) & 0xFFFFFFFFFFFFFFFF
    want, (z, sp, sn) = st.quantize_stochastic(x, n_bits, frac_bits, seed, relu)
    out = B.QTensor.empty(shape[0], shape[1], n_bits, frac_bits, None, with_q16=True)
    stats = B.new_stats()
    B.adaption_quantize_stochastic(dev(x), shape[0], shape[1], out, seed, relu, None, stats)
    got = from_qtensor(out)
    assert np.array_equal(got, want)
    assert np.array_equal(q16_of(out), want)
    assert out.padding_is_zero()
    assert stats_tuple(stats) == (z, sp, sn)


def test_quantize_stochastic_properties_at_size():
    """At a size the oracle still finishes quickly: parity, then the properties Sec. 2.4 states: each
    result is one of the two neighbours of x * 2^f, the mean error vanishes, another seed gives
    another draw, the same seed the same bits, and the device-side format is honoured."""
    n, f = 16, 10
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((1 << 21) + 3) * 4).astype(np.float32)
    xd = dev(x)
    out = B.QTensor.empty(1, x.size, n, f, B.pad_to(x.size, 16))
    B.adaption_quantize_stochastic(xd, 1, x.size, out, 1234)
    got = from_qtensor(out).reshape(-1)
    want, _ = st.quantize_stochastic(x, n, f, 1234)
    assert np.array_equal(got, want)
    y = x.astype(np.float64) * 2.0 ** f
    assert np.all((got == np.floor(y)) | (got == np.floor(y) + 1))
    assert abs(float((got - y).mean())) < 5 * 0.5 / np.sqrt(x.size)
    out2 = B.QTensor.empty(1, x.size, n, f, B.pad_to(x.size, 16))
    B.adaption_quantize_stochastic(xd, 1, x.size, out2, 1235)
    assert not np.array_equal(from_qtensor(out2).reshape(-1), got)
    fmt = torch.tensor([n, f], dtype=torch.int32, device="cuda")
    out3 = B.QTensor.empty(1, x.size, n, 0, B.pad_to(x.size, 16))
    B.adaption_quantize_stochastic(xd, 1, x.size, out3, 1234, False, fmt)
    assert np.array_equal(from_qtensor(out3).reshape(-1), got)
    # the deterministic entry points carry no seed and say so
    with pytest.raises(B.AdaptionError) as e:
        B.adaption_quantize(xd, 1, x.size, out, None, B.ROUND_STOCHASTIC)
    assert e.value.status == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("n_in,f_in,n_out,f_out,relu", [
    (16, 12, 16, 6, False), (16, 12, 8, 3, True), (16, 10, 16, 10, False), (16, 4, 16, 9, True),
    (8, 6, 8, 2, False), (12, 8, 4, 1, True), (8, 3, 16, 0, False)])
@pytest.mark.parametrize("shape", [(1000, 64), (37, 3), (129, 20)])
def test_lp_act_stochastic_format_change(n_in, f_in, n_out, f_out, relu, shape):
    rng = np.random.default_rng(n_in + f_in + n_out + shape[0])
    q = rng.integers(-(1 << (n_in - 1)), 1 << (n_in - 1), shape).astype(np.int16)
    q.flat[:3] = [-(1 << (n_in - 1)), (1 << (n_in - 1)) - 1, 0]
    seed = 0xC0FFEE00 + shape[1]
    want, (z, sp, sn) = st.requantize_stochastic(q, f_in, relu, n_out, f_out, seed)
    xin = to_qtensor(q, n_in, f_in)
    out = B.QTensor.empty(shape[0], shape[1], n_out, f_out, None, with_q16=True)
    stats = B.new_stats()
    B.adaption_lp_act_stochastic(None, xin, shape[0], shape[1], relu, out, seed, None, stats)
    assert np.array_equal(from_qtensor(out), want)
    assert np.array_equal(q16_of(out), want)
    assert out.padding_is_zero()
    assert stats_tuple(stats) == (z, sp, sn)


def test_lp_act_stochastic_fp32_is_the_stochastic_quantizer_with_relu():
    x = (np.random.default_rng(9).standard_normal((300, 48)) * 3).astype(np.float32)
    want, _ = st.quantize_stochastic(x, 16, 9, 77, relu=True)
    out = B.QTensor.empty(300, 48, 16, 9)
    B.adaption_lp_act_stochastic(dev(x), None, 300, 48, True, out, 77)
    assert np.array_equal(from_qtensor(out), want)
