"""GPU parity of the streaming kernels (range, quantizer, LPAct, max-pool) against the CPU oracle,
bit-exact, through the C ABI."""
import os

import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_1711_04713_b200 import binding as B
from tests.util import dev, from_qtensor, q16_of, stats_tuple, to_qtensor

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _range_gpu(x: torch.Tensor, n_bits: int):
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    B.adaption_measure_range(x, n_bits, mx, fmt)
    return float(mx.cpu()[0]), fmt.cpu().tolist()


@pytest.mark.parametrize("numel", [0, 1, 3, 5, 1000, 4099, (1 << 20) + 3, 148 * 256 * 16 + 7])
def test_range_sizes(numel):
    rng = np.random.default_rng(numel)
    x = (rng.standard_normal(numel) * 10.0 ** rng.uniform(-2, 2)).astype(np.float32)
    for n_bits in (16, 8, 4):
        M, fmt = _range_gpu(dev(x), n_bits)
        Mo, m, f = orc.measure_range(x, n_bits)
        assert M == Mo and fmt == [n_bits, f]


def test_range_unaligned_nan_inf_and_accumulation():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(10007).astype(np.float32)
    x[17] = np.nan
    x[5000] = -77.25
    d = dev(x)
    for off in (0, 1, 2, 3):
        M, fmt = _range_gpu(d[off:], 16)
        Mo, m, f = orc.measure_range(x[off:], 16)
        assert M == Mo == 77.25 and fmt == [16, f] and f == 8
    # two tensors share one range
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    B.adaption_measure_range(d[:100], 16, mx, fmt)
    small = float(mx.cpu()[0])
    B.adaption_measure_range(d, 16, mx, fmt)
    assert small < 77.25 and float(mx.cpu()[0]) == 77.25
    x[3] = np.inf
    M, fmt = _range_gpu(dev(x), 12)
    assert M == float("inf") and fmt == [12, 0]
    # exact powers of two sit on the boundary of the rule
    for val, f in [(1.0, 14), (0.99999994, 15), (128.0, 7), (127.99999, 8), (65536.0, 0)]:
        M, fmt = _range_gpu(dev(np.array([val], np.float32)), 16)
        assert fmt == [16, f] == [16, orc.measure_range(np.array([val], np.float32), 16)[2]]


def test_quantizer_handworked_values_on_gpu():
    for line in open(os.path.join(GOLDEN, "qmf_handworked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        n, f, x, q, sat = line.split()
        n, f, q, sat = int(n), int(f), int(q), int(sat)
        xs = np.zeros(16, dtype=np.float32)
        xs[0] = float(x)
        out = B.QTensor.empty(1, 16, n, f)
        st = B.new_stats()
        B.adaption_quantize(dev(xs), 1, 16, out, None, B.ROUND_DETERMINISTIC, st)
        got = from_qtensor(out)[0]
        z, sp, sn = stats_tuple(st)
        assert int(got[0]) == q and np.all(got[1:] == 0), (line, got[:2])
        assert (sp, sn) == (int(sat > 0), int(sat < 0))
        assert z == 15 + int(q == 0)


@pytest.mark.parametrize("n_bits,frac_bits", [(16, 15), (16, 8), (16, 2), (12, 9), (8, 4), (8, 7), (4, 1), (1, 0)])
@pytest.mark.parametrize("shape", [(1000, 64), (37, 3), (129, 20), (5, 16), (3, 100)])
def test_quantize_matches_oracle(n_bits, frac_bits, shape):
    outer, inner = shape
    rng = np.random.default_rng(n_bits * 100 + frac_bits + outer)
    x = (rng.standard_normal(shape) * 2.0 ** (n_bits - 1 - frac_bits) * 0.7).astype(np.float32)
    ties = (rng.integers(-(1 << n_bits), 1 << n_bits, shape) + 0.5) * 2.0 ** -frac_bits
    x = np.where(rng.random(shape) < 0.1, ties, x).astype(np.float32)
    x.ravel()[::97] = 0.0
    cs = B.pad_to(inner, 32 if inner in (3, 20) else 16)
    out = B.QTensor.empty(outer, inner, n_bits, frac_bits, cs, with_q16=True)
    out.lo.fill_(0xAB)
    if out.hi is not None:
        out.hi.fill_(0x5C)
    st = B.new_stats()
    B.adaption_quantize(dev(x), outer, inner, out, None, B.ROUND_DETERMINISTIC, st)
    want, cnt = orc.quantize(x, n_bits, frac_bits)
    assert np.array_equal(from_qtensor(out), want)
    assert np.array_equal(q16_of(out), want)
    assert out.padding_is_zero()
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    # dequantized view within one output LSB of the input wherever nothing saturated
    ok = (want > -(1 << (n_bits - 1))) & (want < (1 << (n_bits - 1)) - 1)
    err = np.abs(want.astype(np.float64) * 2.0 ** -frac_bits - x.astype(np.float64))
    assert np.all(err[ok] <= 2.0 ** -frac_bits)


def test_quantize_large_flat_with_device_format_and_specials():
    rng = np.random.default_rng(5)
    outer, inner = 4096, 256          # one million elements: many blocks, grid-stride and tail paths
    x = (rng.standard_normal((outer, inner)) * 3).astype(np.float32)
    x[0, :8] = [np.nan, np.inf, -np.inf, -0.0, 1e-45, -1e-45, 3e38, -3e38]
    d = dev(x)
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    finite = dev(np.where(np.isfinite(x), x, 0).astype(np.float32))
    B.adaption_measure_range(finite, 16, mx, fmt)
    f = int(fmt.cpu()[1])
    assert f == orc.measure_range(np.where(np.isfinite(x), x, 0).astype(np.float32), 16)[2]
    out = B.QTensor.empty(outer, inner, 16, 0)        # host-side frac_bits deliberately wrong
    st = B.new_stats()
    B.adaption_quantize(d, outer, inner, out, fmt, B.ROUND_DETERMINISTIC, st)
    want, cnt = orc.quantize(x, 16, f)
    assert np.array_equal(from_qtensor(out), want)
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)


@pytest.mark.parametrize("n_bits,frac_bits", [(16, 10), (8, 3)])
def test_lp_act_fp32_relu(n_bits, frac_bits):
    rng = np.random.default_rng(6)
    x = (rng.standard_normal((300, 48)) * 4).astype(np.float32)
    out = B.QTensor.empty(300, 48, n_bits, frac_bits)
    st = B.new_stats()
    B.adaption_lp_act(dev(x), None, 300, 48, True, out, None, B.ROUND_DETERMINISTIC, st)
    want, cnt = orc.quantize(x, n_bits, frac_bits, relu=True)
    assert np.array_equal(from_qtensor(out), want)
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    # quantize-then-ReLU (the paper's order) gives the same tensor
    plain, _ = orc.quantize(x, n_bits, frac_bits)
    assert np.array_equal(want, np.maximum(plain, 0))


@pytest.mark.parametrize("n_in,f_in,n_out,f_out,relu", [
    (16, 10, 16, 9, False), (16, 10, 16, 12, True), (16, 10, 8, 3, False), (8, 4, 16, 12, True),
    (8, 4, 8, 1, False), (16, 15, 4, 2, True), (12, 6, 16, 6, False)])
def test_lp_act_format_change(n_in, f_in, n_out, f_out, relu):
    rng = np.random.default_rng(n_in + f_in + n_out + f_out)
    q = rng.integers(-(1 << (n_in - 1)), 1 << (n_in - 1), (77, 40)).astype(np.int16)
    q[0, :4] = [-(1 << (n_in - 1)), (1 << (n_in - 1)) - 1, 0, -1]
    xin = to_qtensor(q, n_in, f_in, 48)
    out = B.QTensor.empty(77, 40, n_out, f_out, 64, with_q16=True)
    out.lo.fill_(0x77)
    st = B.new_stats()
    B.adaption_lp_act(None, xin, 77, 40, relu, out, None, B.ROUND_DETERMINISTIC, st)
    want, cnt = orc.requantize(q, f_in, relu, n_out, f_out)
    assert np.array_equal(from_qtensor(out), want)
    assert np.array_equal(q16_of(out), want)
    assert out.padding_is_zero()
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)


@pytest.mark.parametrize("n_in,f_in,n_out,f_out,relu", [
    (16, 15, 16, 0, False), (16, 15, 16, 14, False), (16, 10, 16, 9, True), (16, 10, 8, 3, False),
    (16, 3, 16, 12, False), (16, 0, 16, 15, True), (16, 8, 5, 2, False), (16, 7, 16, 7, False),
    (8, 4, 16, 12, True), (8, 7, 8, 0, False), (8, 0, 16, 15, False), (8, 3, 4, 1, True)])
def test_lp_act_format_change_dense_every_input_value(n_in, f_in, n_out, f_out, relu):
    """Dense tensors (pitch == extent, planes only) take the flat kernel: every representable
    input value, in a tensor long enough for the paired and the tail loop, a full-size grid
    included."""
    lo, hi = -(1 << (n_in - 1)), 1 << (n_in - 1)
    vals = np.arange(lo, hi, dtype=np.int64)
    reps = 65536 // vals.size
    for rows_mult in (1, 37):
        q = np.tile(vals, reps * rows_mult + 1)[: (65536 * rows_mult // 48 + 1) * 48]
        q = q.reshape(-1, 48).astype(np.int16)
        xin = to_qtensor(q, n_in, f_in, 48)
        out = B.QTensor.empty(q.shape[0], 48, n_out, f_out, 48)
        out.lo.fill_(0x77)
        st = B.new_stats()
        B.adaption_lp_act(None, xin, q.shape[0], 48, relu, out, None, B.ROUND_DETERMINISTIC, st)
        want, cnt = orc.requantize(q, f_in, relu, n_out, f_out)
        assert np.array_equal(from_qtensor(out), want)
        assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)


@pytest.mark.parametrize("n_bits", [16, 8])
@pytest.mark.parametrize("shape", [(2, 6, 8, 3), (1, 4, 4, 64), (3, 10, 6, 20), (2, 2, 2, 130)])
def test_maxpool(n_bits, shape):
    N, H, W, Cc = shape
    rng = np.random.default_rng(sum(shape) + n_bits)
    q = rng.integers(-(1 << (n_bits - 1)), 1 << (n_bits - 1), shape).astype(np.int16)
    q[0, :2, :2, 0] = -np.arange(1, 5).reshape(2, 2)          # all-negative window
    cs = B.pad_to(Cc, 32)
    xin = to_qtensor(q.reshape(-1, Cc), n_bits, 5, cs)
    out = B.QTensor.empty(N * (H // 2) * (W // 2), Cc, n_bits, 5, cs, with_q16=True)
    out.lo.fill_(0x11)
    B.adaption_maxpool2x2(xin, N, H, W, Cc, out)
    want = orc.maxpool2x2(q).reshape(-1, Cc)
    assert np.array_equal(from_qtensor(out), want)
    assert np.array_equal(q16_of(out), want)
    assert out.padding_is_zero()


def test_empty_inputs_are_no_ops():
    out = B.QTensor.empty(4, 16, 16, 3)
    out.lo.fill_(9)
    B.adaption_quantize(torch.empty(0, device="cuda"), 0, 16, out)
    torch.cuda.synchronize()
    assert int(out.lo[0]) == 9


def test_quantize_batch_matches_oracle():
    """Many tensors in one call: mixed sizes (below, at and above a 1024-vector chunk), 16- and 8-bit
    outputs, with and without the int16 copy, host- and device-side formats, padded rows, an empty
    tensor, and more dense tensors than one launch carries; every element against the oracle."""
    rng = np.random.default_rng(77)
    shapes = [(64, 64), (1, 16), (4096, 16), (4097, 16), (300, 1024), (3, 48), (27, 3), (1, 1000), (0, 16), (1, 64)]
    shapes += [(rng.integers(1, 40), 16 * int(rng.integers(1, 9))) for _ in range(45)]
    entries, checks, keep = [], [], []
    for k, (outer, inner) in enumerate(shapes):
        outer, inner = int(outer), int(inner)
        n_bits = 8 if k % 3 == 1 else 16
        frac_bits = n_bits - 1 - (k % 3)
        x = (rng.standard_normal((outer, inner)) * 2.0 ** (k % 3) * 0.6).astype(np.float32)
        if x.size:
            x.ravel()[0] = np.nan
            x.ravel()[-1] = np.inf
        cs = B.pad_to(inner, 16)
        use_dev_fmt = k % 4 == 2
        out = B.QTensor.empty(max(outer, 1), inner, n_bits, 0 if use_dev_fmt else frac_bits, cs,
                              with_q16=(k % 2 == 0))
        out.lo.fill_(0xAB)
        if outer == 0:                                     # an empty tensor leaves its output alone
            entries.append((None, 0, inner, out, None))
            continue
        fmt = torch.tensor([n_bits, frac_bits], dtype=torch.int32, device="cuda") if use_dev_fmt else None
        xd = dev(x)
        keep.append((xd, fmt))
        entries.append((xd, outer, inner, out, fmt))
        checks.append((x, out, n_bits, frac_bits))
    items = B.quantize_items(entries)
    B.adaption_quantize_batch(items)
    torch.cuda.synchronize()
    for x, out, n_bits, frac_bits in checks:
        want, _ = orc.quantize(x, n_bits, frac_bits)
        assert np.array_equal(from_qtensor(out), want), x.shape
        if out.q16 is not None:
            assert np.array_equal(q16_of(out), want)
        assert out.padding_is_zero()
    B.adaption_quantize_batch(items, 0)                   # nothing to do
    # one bad item: nothing is launched, the others stay untouched
    checks[0][1].lo.fill_(0x11)
    bad = B.QTensor.empty(4, 16, 16, 3, 16)
    bad.n_bits = 17
    with pytest.raises(B.AdaptionError):
        B.adaption_quantize_batch(B.quantize_items(entries[:1] + [(keep[0][0], 4, 16, bad, None)]))
    torch.cuda.synchronize()
    assert int(checks[0][1].lo.min()) == 0x11 and int(checks[0][1].lo.max()) == 0x11
