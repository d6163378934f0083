"""GPU parity of LPConvolution / LPInnerProduct (both kernels: plain integer and tensor core)
against the CPU oracle, bit-exact, through the C ABI.  Shapes span several 128-row tiles and
ragged tails in M, N and K."""
import os

import numpy as np
import pytest
import torch

from oracle import reference as orc
from oracle import stochastic as orc_st
from paper_1711_04713_b200 import binding as B
from tests.util import Guards, dev, from_qtensor, q16_of, stats_tuple, to_qtensor

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _default_overrides():
    """Every test starts from and leaves behind the library's default heuristics."""
    B.adaption_debug_set("reset")
    yield
    B.adaption_debug_set("reset")


def _rand_q(rng, shape, n_bits, zero_frac=0.0):
    q = rng.integers(-(1 << (n_bits - 1)), 1 << (n_bits - 1), shape).astype(np.int16)
    if zero_frac > 0:
        q[rng.random(shape) < zero_frac] = 0
    return q


def _pick_f_out(acc, bq, fb, F, relu, n_out):
    A = orc.epilogue_range(acc, bq, fb, F, relu)
    return A, n_out - 1 - orc.int_bits_from_acc(A, F, n_out)


def run_conv_case(rng, N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu, algo, with_bias=True,
                  extreme=False, f_out=None, with_q16=True, mag_bits=None, fmts=None, cs=None, ws_offset=0,
                  stochastic_seed=None):
    """`with_q16=False` leaves out the optional int16 copy of the output, which lets the tensor-core
    kernel stage its byte planes in shared memory and write them with bulk-tensor stores.
    `mag_bits` limits operand magnitudes (small accumulators -> short requantization shifts)."""
    cs = B.pad_to(Cin, 32) if cs is None else cs
    xq = _rand_q(rng, (N, H, W, Cin), nx if mag_bits is None else min(nx, mag_bits[0]), 0.4)
    wq = _rand_q(rng, (K, R, R, Cin), nw if mag_bits is None else min(nw, mag_bits[1]))
    if extreme:   # drive every byte plane to its extremes
        xq[:] = np.where(rng.random(xq.shape) < 0.5, -(1 << (nx - 1)), (1 << (nx - 1)) - 1)
        wq[:] = np.where(rng.random(wq.shape) < 0.5, -(1 << (nw - 1)), (1 << (nw - 1)) - 1)
    fx, fw = (nx - 3, nw - 1) if fmts is None else fmts
    bq = _rand_q(rng, (K,), nw) if with_bias else None
    acc = orc.conv_acc(xq, wq, (pad, pad), (stride, stride))
    F = fx + fw
    A, f_auto = _pick_f_out(acc, bq, fw, F, relu, n_out)
    f_out = f_auto if f_out is None else f_out
    want, cnt = orc.epilogue(acc, bq, fw, F, relu, n_out, f_out)
    if stochastic_seed is not None:
        want, c3 = orc_st.epilogue_stochastic(acc, bq, fw, F, relu, n_out, f_out, stochastic_seed)
        cnt = orc.Counters(*c3)
    OH, OW = acc.shape[1], acc.shape[2]

    x = to_qtensor(xq.reshape(-1, Cin), nx, fx, cs)
    w = to_qtensor(wq.reshape(-1, Cin), nw, fw, cs)
    ycs = B.pad_to(K, 32)
    guards = Guards()         # canaries around the output planes and the workspace
    y = guards.qtensor(N * OH * OW, K, n_out, f_out, ycs, with_q16=with_q16)
    shp = B.conv_shape(N, H, W, Cin, K, R, R, pad, stride)
    bias_dev = dev(bq) if with_bias else None
    need = B.adaption_lp_conv_workspace_bytes(shp, x.fmt(), w.fmt(), cs, algo)
    ws = guards.alloc(max(need, 16) + ws_offset)[ws_offset:] if need else None
    st = B.new_stats()
    B.adaption_lp_conv_fwd(shp, x, w, bias_dev, fw, relu, B.MODE_RANGE, algo, None, st, ws)
    s = B.read_stats(st)
    assert s.status == 0
    assert int(s.max_abs_acc) == A
    assert B.adaption_choose_frac_bits_from_acc(A, F, n_out) == f_auto
    st = B.new_stats()
    if stochastic_seed is not None:
        B.adaption_lp_conv_fwd_stochastic(shp, x, w, bias_dev, fw, relu, algo, y, stochastic_seed, st, ws)
    else:
        B.adaption_lp_conv_fwd(shp, x, w, bias_dev, fw, relu, B.MODE_REQUANT, algo, y, st, ws)
    s = B.read_stats(st)
    assert s.status == 0
    got = from_qtensor(y).reshape(want.shape)
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}: got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}"
    if with_q16:
        assert np.array_equal(q16_of(y).reshape(want.shape), want)
    assert y.padding_is_zero()
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    guards.check()
    return cnt


def run_ip_case(rng, Bsz, K, O, nx, nw, n_out, relu, algo, with_bias=True, f_out=None, with_q16=True,
                stochastic_seed=None):
    xq = _rand_q(rng, (Bsz, K), nx, 0.4)
    wq = _rand_q(rng, (O, K), nw)
    fx, fw = nx - 2, nw - 1
    bq = _rand_q(rng, (O,), nw) if with_bias else None
    acc = orc.ip_acc(xq, wq)
    F = fx + fw
    A, f_auto = _pick_f_out(acc, bq, fw, F, relu, n_out)
    f_out = f_auto if f_out is None else f_out
    want, cnt = orc.epilogue(acc, bq, fw, F, relu, n_out, f_out)
    if stochastic_seed is not None:
        want, c3 = orc_st.epilogue_stochastic(acc, bq, fw, F, relu, n_out, f_out, stochastic_seed)
        cnt = orc.Counters(*c3)
    x = to_qtensor(xq, nx, fx)
    w = to_qtensor(wq, nw, fw)
    guards = Guards()
    y = guards.qtensor(Bsz, O, n_out, f_out, None, with_q16=with_q16)
    bias_dev = dev(bq) if with_bias else None
    need = B.adaption_lp_ip_workspace_bytes(Bsz, K, O, x.fmt(), w.fmt(), algo)
    ws = guards.alloc(max(need, 16)) if need else None
    st = B.new_stats()
    B.adaption_lp_ip_fwd(Bsz, K, O, x, w, bias_dev, fw, relu, B.MODE_RANGE, algo, None, st, ws)
    s = B.read_stats(st)
    assert s.status == 0 and int(s.max_abs_acc) == A
    st = B.new_stats()
    if stochastic_seed is not None:
        B.adaption_lp_ip_fwd_stochastic(Bsz, K, O, x, w, bias_dev, fw, relu, algo, y, stochastic_seed, st, ws)
    else:
        B.adaption_lp_ip_fwd(Bsz, K, O, x, w, bias_dev, fw, relu, B.MODE_REQUANT, algo, y, st, ws)
    s = B.read_stats(st)
    assert s.status == 0
    got = from_qtensor(y)
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}"
    if with_q16:
        assert np.array_equal(q16_of(y), want)
    assert y.padding_is_zero()
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    guards.check()
    return need


# ------------------------------------------------------------------ plain integer kernels
@pytest.mark.parametrize("case", [
    # N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu
    (2, 7, 6, 5, 4, 3, 1, 1, 16, 16, 16, True), (1, 9, 9, 3, 7, 5, 0, 1, 16, 16, 16, False),
    (2, 8, 10, 4, 3, 3, 1, 2, 8, 8, 8, True), (1, 5, 5, 20, 50, 5, 0, 1, 16, 16, 16, True),
    (1, 6, 6, 9, 5, 1, 0, 1, 16, 8, 12, False), (2, 6, 6, 16, 8, 3, 2, 1, 4, 4, 4, True),
    (1, 8, 8, 33, 17, 3, 1, 1, 12, 16, 8, True),
])
def test_conv_direct(case):
    N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu = case
    run_conv_case(np.random.default_rng(sum(case)), N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu,
                  B.ALGO_DIRECT)


@pytest.mark.parametrize("case", [(8, 800, 500, 16, 16, 16, True), (8, 500, 10, 16, 16, 16, False),
                                  (3, 17, 5, 8, 8, 8, True), (5, 64, 33, 16, 8, 16, False),
                                  (1, 1, 1, 16, 16, 16, False)])
def test_ip_direct(case):
    Bsz, K, O, nx, nw, n_out, relu = case
    run_ip_case(np.random.default_rng(sum(case)), Bsz, K, O, nx, nw, n_out, relu, B.ALGO_DIRECT)


def test_direct_without_bias_and_fixed_saturating_format():
    rng = np.random.default_rng(3)
    run_conv_case(rng, 1, 6, 6, 8, 6, 3, 1, 1, 16, 16, 16, False, B.ALGO_DIRECT, with_bias=False)
    # a format with too few integer bits saturates on both sides; counters must agree
    run_ip_case(rng, 6, 40, 12, 16, 16, 16, False, B.ALGO_DIRECT, f_out=15)
    run_ip_case(rng, 6, 40, 12, 16, 16, 8, True, B.ALGO_DIRECT, f_out=7)


# ------------------------------------------------------------------ tensor-core kernels
TC_CONV = [
    # N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu      (N*H*W*pitch >= 128 KiB)
    (6, 20, 20, 64, 96, 3, 1, 1, 16, 16, 16, True),      # BK=64, ragged N tile, 18.75 M tiles
    (2, 24, 24, 128, 128, 3, 1, 1, 16, 16, 16, True),    # BK=128
    (2, 30, 30, 256, 64, 3, 1, 1, 16, 16, 16, False),    # two channel blocks per tap, BN=64
    (8, 28, 28, 20, 50, 5, 0, 1, 16, 16, 16, True),      # valid 5x5, pitch 32 (BK=32), ragged N
    (8, 32, 32, 3, 64, 3, 1, 1, 16, 16, 16, True),       # first-layer shape: 3 channels padded to 32
    (4, 33, 31, 64, 130, 3, 1, 2, 16, 16, 16, True),     # stride 2, odd sizes, N spills into 2nd tile
    (2, 40, 40, 64, 32, 1, 0, 1, 16, 16, 16, False),     # 1x1
    (2, 24, 24, 128, 128, 3, 1, 1, 8, 8, 8, True),       # single int8 pass
    (2, 24, 24, 128, 72, 3, 1, 1, 4, 4, 4, True),        # 4-bit operands in the int8 pass
    (2, 24, 24, 128, 128, 3, 1, 1, 16, 8, 16, True),     # 16-bit activations x 8-bit weights
    (2, 24, 24, 128, 128, 3, 1, 1, 8, 16, 12, False),    # 8-bit activations x 16-bit weights
    (2, 24, 24, 128, 128, 3, 1, 1, 12, 12, 12, True),    # 12-bit operands in planes
    (1, 64, 64, 32, 16, 3, 1, 1, 16, 16, 8, True),       # 16-bit in, 8-bit out, BN=32
    (5, 30, 30, 64, 64, 3, 1, 1, 16, 16, 16, True),      # 64 -> 64 channels: CTA pair on 64-byte k-blocks, M tail
    (4, 24, 24, 64, 48, 5, 2, 1, 16, 16, 16, False),     # same family without the paired rule (25 taps), signed
]


@pytest.fixture(params=["single", "pair"])
def cta_mode(request, _default_overrides):
    """Run a tensor-core case with one CTA per 128-row tile and with CTA pairs on 256-row tiles
    (cross-path identity: both must give the oracle's bits)."""
    B.adaption_debug_set("pair", 1 if request.param == "pair" else 0)
    return request.param


@pytest.mark.parametrize("case", TC_CONV)
def test_conv_tensor(case, cta_mode):
    N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu = case
    run_conv_case(np.random.default_rng(sum(case)), N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu,
                  B.ALGO_TENSOR)


@pytest.mark.parametrize("case", TC_CONV)
def test_conv_tensor_staged_stores(case, cta_mode):
    """Same cases without the int16 copy: byte planes leave through shared memory and bulk-tensor
    stores, ReLU layers with shifts of 9 and more take the paired 16-bit epilogue."""
    N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu = case
    run_conv_case(np.random.default_rng(sum(case) + 1), N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu,
                  B.ALGO_TENSOR, with_q16=False)


@pytest.mark.parametrize("shift", [2, 8, 9, 12, 15, 16, 17, 22])
@pytest.mark.parametrize("n_out", [16, 8])
def test_fast_epilogue_shifts_and_saturation(shift, n_out, cta_mode):
    """ReLU layers across the requantization shifts on both sides of the fast epilogue's limits
    (9 <= shift: 32-bit path, its two forms split at 16), with outputs that saturate: operands of
    reduced magnitude so that short shifts still give in-range values."""
    nx = nw = 16
    fmts = (4, 8) if shift <= 12 else ((8, 12) if shift <= 17 else (13, 15))
    f_out = sum(fmts) - shift
    if not 0 <= f_out <= n_out - 1:
        pytest.skip("shift not reachable with this output width")
    mag = (min(16, (shift + 8) // 2), min(16, (shift + 7) // 2))   # accumulators of about 2^(shift + 8)
    cnt = run_conv_case(np.random.default_rng(100 + shift), 2, 24, 24, 128, 128, 3, 1, 1, nx, nw, n_out, True,
                        B.ALGO_TENSOR, f_out=f_out, with_q16=False, mag_bits=mag, fmts=fmts)
    assert cnt.zeros > 0
    if n_out == 8:
        assert cnt.sat_pos > 0   # the case does exercise saturation


@pytest.mark.parametrize("shift", [0, 1, 3, 6, 8, 9, 11, 14])
@pytest.mark.parametrize("n_out", [8, 5])
@pytest.mark.parametrize("K,Cin", [(128, 128), (256, 512)])
def test_single_pass_fast_epilogue_every_shift(shift, n_out, K, Cin, cta_mode):
    """8-bit operands on both sides give one accumulator: ReLU layers take the 32-bit epilogue at
    every non-negative shift (128- and 256-column tiles); magnitudes chosen so that outputs span
    the range and some saturate."""
    fmts = (shift // 2, shift - shift // 2)
    f_out = 0
    bits = 3 if shift <= 3 else (5 if shift <= 8 else 8)
    cnt = run_conv_case(np.random.default_rng(300 + shift + K), 2, 24, 24, Cin, K, 3, 1, 1, 8, 8, n_out, True,
                        B.ALGO_TENSOR, f_out=f_out, with_q16=False, mag_bits=(bits, bits), fmts=fmts)
    assert cnt.zeros > 0
    if n_out == 5:
        assert cnt.sat_pos > 0   # the case does exercise saturation


def test_epilogue_variants_agree():
    """Cross-path identity: the generic 64-bit epilogue with direct stores, the staged stores and the
    fast paired path all give the oracle's bits on the same case."""
    case = (2, 24, 24, 128, 128, 3, 1, 1, 16, 16, 16, True)
    for fast, staged in ((0, 0), (0, 1), (1, 0), (1, 1)):
        B.adaption_debug_set("fast", fast)
        B.adaption_debug_set("staged", staged)
        run_conv_case(np.random.default_rng(5), *case, B.ALGO_TENSOR, with_q16=False, mag_bits=(10, 10))


FEW_CHANNELS = [
    # N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu, channel pitch
    (8, 32, 32, 3, 64, 3, 1, 1, 16, 16, 16, True, 16),    # RGB 3x3 (27 taps x channels), pitch 16
    (8, 28, 28, 1, 20, 5, 0, 1, 16, 16, 16, True, 16),    # one channel, 5x5 valid (25 taps)
    (3, 41, 37, 2, 72, 4, 2, 2, 16, 16, 16, False, 32),   # two channels, 4x4, stride 2, pad 2, ragged N
    (4, 30, 30, 4, 128, 2, 0, 1, 8, 8, 8, True, 16),      # four channels, 2x2, single int8 pass
    (2, 40, 24, 3, 40, 3, 1, 1, 16, 8, 12, True, 48),     # mixed widths, pitch 48
    (16, 9, 9, 4, 16, 1, 0, 1, 12, 12, 12, False, 16),    # 1x1, M just above the threshold
]


@pytest.mark.parametrize("case", FEW_CHANNELS)
@pytest.mark.parametrize("with_q16", [True, False])
def test_conv_few_channels_packed_taps(case, with_q16):
    """Layers with at most 4 input channels whose taps fit 32 bytes run as a packed inner product
    (taps gathered into the workspace): image borders, strides, every channel count, both stores."""
    N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu, cs = case
    run_conv_case(np.random.default_rng(sum(case)), N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu,
                  B.ALGO_AUTO, with_q16=with_q16, cs=cs)
    shp = B.conv_shape(N, H, W, Cin, K, R, R, pad, stride)
    OH = (H + 2 * pad - R) // stride + 1
    OW = (W + 2 * pad - R) // stride + 1
    need = B.adaption_lp_conv_workspace_bytes(shp, B.adaption_qfmt(nx, 0), B.adaption_qfmt(nw, 0), cs, B.ALGO_AUTO)
    assert need >= N * OH * OW * 32 * ((nx > 8) + 1)      # the packed planes are in the workspace


@pytest.mark.parametrize("case", [
    (20, 56, 56, 128, 128, 3, 1, 1, 16, 16, 16, True),     # 245 pair tiles / 490 single tiles of 128 columns
    (9, 56, 56, 128, 200, 3, 1, 1, 16, 16, 16, False),     # generic epilogue, two column tiles, ragged N
    (40, 28, 28, 256, 128, 3, 1, 1, 16, 16, 12, True),     # 18 k-blocks, 12-bit outputs
])
@pytest.mark.parametrize("split_hh", [1, 0])
def test_conv_many_tiles_per_cta(case, split_hh, cta_mode):
    """More tiles than CTAs, so that every persistent CTA walks several tiles: the accumulator sets
    (and, for three 128-column accumulators, the alternating place of the high one) rotate."""
    B.adaption_debug_set("split_hh", split_hh)
    run_conv_case(np.random.default_rng(sum(case)), *case, B.ALGO_TENSOR, with_q16=False)


def test_conv_tensor_extreme_operands(cta_mode):
    # every operand at +-full scale: largest possible partial sums in all three accumulators
    run_conv_case(np.random.default_rng(1), 1, 32, 32, 256, 128, 3, 1, 1, 16, 16, 16, False, B.ALGO_TENSOR,
                  extreme=True)
    run_conv_case(np.random.default_rng(2), 1, 32, 32, 256, 128, 3, 1, 1, 8, 8, 8, False, B.ALGO_TENSOR,
                  extreme=True)


TC_IP = [(8, 800, 500, 16, 16, 16, True), (70, 1000, 260, 16, 16, 16, False), (200, 4096, 100, 16, 16, 16, True),
         (130, 256, 128, 8, 8, 8, True), (64, 1184, 96, 16, 8, 16, True), (3, 64, 10, 16, 16, 16, False),
         (256, 512, 512, 12, 12, 12, True)]


@pytest.mark.parametrize("case", TC_IP)
def test_ip_tensor(case, cta_mode):
    Bsz, K, O, nx, nw, n_out, relu = case
    run_ip_case(np.random.default_rng(sum(case)), Bsz, K, O, nx, nw, n_out, relu, B.ALGO_TENSOR)


@pytest.mark.parametrize("case", [FEW_CHANNELS[0], FEW_CHANNELS[3]])
def test_conv_few_channels_workspace_on_a_16_byte_boundary(case):
    """A workspace that is only 16-byte aligned (all the interface asks for) serves the packed rows
    and the bulk-tensor loads that read them."""
    N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu, cs = case
    run_conv_case(np.random.default_rng(sum(case) + 7), N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu,
                  B.ALGO_AUTO, with_q16=False, cs=cs, ws_offset=16)


WIDE_CONV = [
    # single-pass layers with 256 and more output channels: 256-column pair tiles
    (2, 24, 24, 128, 256, 3, 1, 1, 8, 8, 8, True),        # one column tile, 5 row tiles (ragged)
    (3, 28, 28, 256, 512, 3, 1, 1, 8, 8, 8, True),        # two column tiles, two channel blocks per tap
    (2, 24, 24, 128, 320, 3, 1, 1, 8, 8, 8, False),       # ragged N (320 = 256 + 64), signed outputs
    (2, 24, 24, 128, 256, 3, 1, 1, 8, 8, 16, True),       # 8-bit operands, 16-bit outputs (two planes)
    (2, 24, 24, 128, 264, 3, 1, 1, 4, 4, 4, True),        # 4-bit, N = 264
]


@pytest.mark.parametrize("case", WIDE_CONV)
@pytest.mark.parametrize("with_q16", [False, True])
@pytest.mark.parametrize("wide", [1, 0])
def test_conv_single_pass_wide_tiles(case, with_q16, wide):
    B.adaption_debug_set("wide", wide)
    run_conv_case(np.random.default_rng(sum(case)), *case, B.ALGO_TENSOR, with_q16=with_q16)


def test_ip_single_pass_wide_tiles():
    run_ip_case(np.random.default_rng(77), 1100, 1152, 384, 8, 8, 8, True, B.ALGO_TENSOR, with_q16=False)
    run_ip_case(np.random.default_rng(78), 2048, 2304, 256, 8, 8, 8, False, B.ALGO_TENSOR, with_q16=True)


@pytest.mark.parametrize("groups", [1, 2])
@pytest.mark.parametrize("with_q16", [False, True])
def test_epilogue_groups_agree(groups, with_q16):
    """Narrow tiles (two accumulator sets in TMEM): one group of epilogue warps, or two groups taking
    alternate tiles, give the same bits; odd and even tile counts per CTA, ReLU and signed outputs."""
    B.adaption_debug_set("epigroups", groups)
    for case in [(5, 40, 40, 64, 64, 3, 1, 1, 16, 16, 16, True),       # 63 tiles of 128 x 64
                 (2, 30, 30, 256, 48, 3, 1, 1, 16, 16, 16, False),     # signed outputs, ragged N
                 (37, 64, 64, 32, 32, 3, 1, 1, 16, 16, 8, True),       # BN = 32, more tiles than CTAs
                 (37, 64, 64, 3, 64, 3, 1, 1, 16, 16, 16, True)]:      # packed taps, K = 32, 1184 tiles
        run_conv_case(np.random.default_rng(sum(case)), *case, B.ALGO_AUTO, with_q16=with_q16)


@pytest.mark.parametrize("case", TC_IP)
def test_ip_tensor_staged_stores(case, cta_mode):
    Bsz, K, O, nx, nw, n_out, relu = case
    run_ip_case(np.random.default_rng(sum(case) + 1), Bsz, K, O, nx, nw, n_out, relu, B.ALGO_TENSOR, with_q16=False)


def test_ip_tensor_split_k_paths():
    # long reduction with few output tiles: the library splits K and needs its workspace
    need = run_ip_case(np.random.default_rng(11), 64, 25088, 256, 16, 16, 16, True, B.ALGO_TENSOR)
    assert need == 64 * 256 * 8
    # forcing other split factors gives the same bits
    for splits in (3, 7):
        B.adaption_debug_set("splits", splits)
        need = run_ip_case(np.random.default_rng(12), 40, 2048, 200, 16, 16, 16, False, B.ALGO_TENSOR)
        assert need == 40 * 200 * 8
        run_conv_case(np.random.default_rng(13), 2, 24, 24, 128, 128, 3, 1, 1, 16, 16, 16, True,
                      B.ALGO_TENSOR)


def test_workspace_too_small_is_rejected():
    rng = np.random.default_rng(14)
    xq, wq = _rand_q(rng, (64, 25088), 16), _rand_q(rng, (256, 25088), 16)
    x, w = to_qtensor(xq, 16, 10), to_qtensor(wq, 16, 15)
    y = B.QTensor.empty(64, 256, 16, 5)
    st = B.new_stats()
    with pytest.raises(B.AdaptionError) as e:
        B.adaption_lp_ip_fwd(64, 25088, 256, x, w, None, 0, True, B.MODE_REQUANT, B.ALGO_TENSOR, y, st,
                             torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.ERR_WORKSPACE


def test_eight_bit_data_through_plane_path_equals_single_pass():
    """Cross-path identity: 8-bit values stored as 16-bit planes (hi = sign extension) go through
    the four-product path and must give the bits of the single int8 pass."""
    rng = np.random.default_rng(15)
    N, H, W, Cin, K = 4, 24, 24, 64, 64
    xq, wq = _rand_q(rng, (N, H, W, Cin), 8, 0.3), _rand_q(rng, (K, 3, 3, Cin), 8)
    shp = B.conv_shape(N, H, W, Cin, K, 3, 3, 1, 1)
    outs = []
    for nb in (8, 16):
        x, w = to_qtensor(xq.reshape(-1, Cin), nb, 4, 64), to_qtensor(wq.reshape(-1, Cin), nb, 7, 64)
        y = B.QTensor.empty(N * H * W, K, 16, 6, 64)
        st = B.new_stats()
        B.adaption_lp_conv_fwd(shp, x, w, None, 0, True, B.MODE_REQUANT, B.ALGO_TENSOR, y, st, None)
        outs.append((from_qtensor(y), stats_tuple(st)))
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]
    want, _ = orc.epilogue(orc.conv_acc(xq, wq, (1, 1)), None, 0, 11, True, 16, 6)
    assert np.array_equal(outs[0][0].reshape(want.shape), want)


def test_one_by_one_conv_equals_inner_product_on_gpu():
    rng = np.random.default_rng(16)
    N, H, W, Cin, K = 2, 40, 40, 64, 48
    xq, wq = _rand_q(rng, (N, H, W, Cin), 16, 0.3), _rand_q(rng, (K, 1, 1, Cin), 16)
    x, w = to_qtensor(xq.reshape(-1, Cin), 16, 9, 64), to_qtensor(wq.reshape(-1, Cin), 16, 14, 64)
    st = B.new_stats()
    y1 = B.QTensor.empty(N * H * W, K, 16, 4, 64)
    B.adaption_lp_conv_fwd(B.conv_shape(N, H, W, Cin, K, 1, 1, 0, 1), x, w, None, 0, False, B.MODE_REQUANT,
                           B.ALGO_TENSOR, y1, st, None)
    y2 = B.QTensor.empty(N * H * W, K, 16, 4, 64)
    B.adaption_lp_ip_fwd(N * H * W, Cin, K, x, w, None, 0, False, B.MODE_REQUANT, B.ALGO_TENSOR, y2, st, None)
    assert np.array_equal(from_qtensor(y1), from_qtensor(y2))


def test_auto_falls_back_to_direct_for_small_or_odd_pitch():
    rng = np.random.default_rng(17)
    # pitch 48 is not a multiple of 32 and the tensor is tiny: AUTO must still be exact
    run_conv_case(rng, 1, 6, 6, 8, 6, 3, 1, 1, 16, 16, 16, True, B.ALGO_AUTO)
    run_ip_case(rng, 4, 20, 6, 16, 16, 16, True, B.ALGO_AUTO)
    xq, wq = _rand_q(rng, (1, 4, 4, 8), 16), _rand_q(rng, (4, 3, 3, 8), 16)
    x, w = to_qtensor(xq.reshape(-1, 8), 16, 9, 32), to_qtensor(wq.reshape(-1, 8), 16, 9, 32)
    with pytest.raises(B.AdaptionError) as e:
        B.adaption_lp_conv_fwd(B.conv_shape(1, 4, 4, 8, 4, 3, 3, 1, 1), x, w, None, 0, False, B.MODE_RANGE,
                               B.ALGO_TENSOR, None, B.new_stats(), None)
    assert e.value.status == B.ERR_UNSUPPORTED


# ------------------------------------------------------------------ convolution + 2x2 max-pool
POOL_CONV = [
    # N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu
    (2, 24, 24, 128, 128, 3, 1, 1, 16, 16, 16, True),     # pair tiles, fused horizontal maxima
    (6, 20, 20, 64, 96, 3, 1, 1, 16, 16, 16, True),       # BK = 64, ragged N tile and M tail
    (2, 30, 30, 256, 64, 3, 1, 1, 16, 16, 16, False),     # signed outputs (generic epilogue), BN = 64
    (8, 32, 32, 3, 64, 3, 1, 1, 16, 16, 16, True),        # packed taps
    (2, 24, 24, 128, 256, 3, 1, 1, 8, 8, 8, True),        # single pass, 256-column tiles
    (1, 64, 64, 32, 16, 3, 1, 1, 16, 16, 8, True),        # BN = 32 > output pitch 16: direct stores, full temp
    (2, 12, 12, 20, 50, 5, 2, 1, 16, 16, 16, True),       # plain integer kernel (odd pitch), full temp
    (3, 44, 44, 128, 128, 3, 1, 2, 16, 16, 16, True),     # stride 2: 22 x 22 outputs, M = 1452 (ragged last tile)
    (1, 36, 20, 256, 128, 3, 1, 1, 16, 16, 12, True),     # H != W, 12-bit outputs, one image
    (5, 16, 16, 128, 128, 1, 0, 1, 16, 16, 16, True),     # 1x1 filter
    (4, 32, 32, 64, 64, 3, 1, 1, 16, 16, 16, True),       # 64 -> 64 channels: CTA pair, 64-column tiles, two epilogue groups
    (3, 26, 30, 64, 40, 3, 1, 1, 16, 16, 16, True),       # same with a ragged M tail and 40 channels
]


@pytest.mark.parametrize("case", POOL_CONV)
@pytest.mark.parametrize("with_q16", [False, True])
def test_conv_with_fused_pool(case, with_q16):
    """adaption_lp_conv_pool_fwd equals convolution, epilogue and 2x2 max-pool of the oracle; its
    counters are those of the convolution's own output."""
    N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu = case
    rng = np.random.default_rng(sum(case))
    cs = B.pad_to(Cin, 32) if Cin != 20 else 48
    xq = _rand_q(rng, (N, H, W, Cin), nx, 0.4)
    wq = _rand_q(rng, (K, R, R, Cin), nw)
    bq = _rand_q(rng, (K,), nw)
    fx, fw = nx - 3, nw - 1
    acc = orc.conv_acc(xq, wq, (pad, pad), (stride, stride))
    F = fx + fw
    _, f_out = _pick_f_out(acc, bq, fw, F, relu, n_out)
    conv_y, cnt = orc.epilogue(acc, bq, fw, F, relu, n_out, f_out)
    want = orc.maxpool2x2(conv_y)
    OH, OW = acc.shape[1], acc.shape[2]
    x = to_qtensor(xq.reshape(-1, Cin), nx, fx, cs)
    w = to_qtensor(wq.reshape(-1, Cin), nw, fw, cs)
    guards = Guards()
    y = guards.qtensor(N * (OH // 2) * (OW // 2), K, n_out, f_out, B.pad_to(K, 16), with_q16=with_q16)
    shp = B.conv_shape(N, H, W, Cin, K, R, R, pad, stride)
    need = B.adaption_lp_conv_pool_workspace_bytes(shp, x.fmt(), w.fmt(), y.fmt(), cs, y.c_stride, B.ALGO_AUTO)
    assert need > 0
    ws = guards.alloc(need)
    st = B.new_stats()
    B.adaption_lp_conv_pool_fwd(shp, x, w, dev(bq), fw, relu, B.ALGO_AUTO, y, st, ws)
    assert B.read_stats(st).status == 0
    assert np.array_equal(from_qtensor(y).reshape(want.shape), want)
    if with_q16:
        assert np.array_equal(q16_of(y).reshape(want.shape), want)
    assert y.padding_is_zero()
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    with pytest.raises(B.AdaptionError):                      # too small a workspace is refused
        B.adaption_lp_conv_pool_fwd(shp, x, w, dev(bq), fw, relu, B.ALGO_AUTO, y, st, ws[:need - 256])
    # the two phases issued by separate calls give the same tensor and count the outputs once
    y.lo.fill_(0x3C)
    st2 = B.new_stats()
    B.adaption_lp_conv_pool_fwd(shp, x, w, dev(bq), fw, relu, B.ALGO_AUTO, y, st2, ws, B.PHASE_CONV)
    B.adaption_lp_conv_pool_fwd(shp, x, w, dev(bq), fw, relu, B.ALGO_AUTO, y, st2, ws, B.PHASE_POOL)
    assert np.array_equal(from_qtensor(y).reshape(want.shape), want)
    assert stats_tuple(st2) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    for bad_phases in (0, 4):
        with pytest.raises(B.AdaptionError):
            B.adaption_lp_conv_pool_fwd(shp, x, w, dev(bq), fw, relu, B.ALGO_AUTO, y, st2, ws, bad_phases)
    guards.check()


# ------------------------------------------------------------------ stochastic rounding in the layer epilogue
STOCHASTIC_CONV = [
    # N, H, W, Cin, K, R, pad, stride, nx, nw, n_out, relu
    (2, 24, 24, 128, 128, 3, 1, 1, 16, 16, 16, True),     # 128-column tiles (pair or single)
    (6, 20, 20, 64, 96, 3, 1, 1, 16, 16, 16, False),      # signed outputs, ragged N tile, M tail
    (4, 33, 31, 64, 130, 3, 1, 2, 16, 16, 12, True),      # N = 130: element indices misaligned to the generator's blocks
    (2, 30, 30, 256, 61, 3, 1, 1, 16, 16, 16, True),      # odd N: every row starts at another word of a block
    (2, 24, 24, 128, 128, 3, 1, 1, 8, 8, 8, True),        # single int8 pass
    (2, 24, 24, 128, 256, 3, 1, 1, 8, 8, 8, True),        # 256-column tiles
    (8, 32, 32, 3, 64, 3, 1, 1, 16, 16, 16, True),        # packed first-layer taps
    (2, 12, 12, 20, 50, 5, 2, 1, 16, 16, 16, True),       # plain integer kernel (odd pitch)
]


@pytest.mark.parametrize("case", STOCHASTIC_CONV)
@pytest.mark.parametrize("with_q16", [False, True])
def test_conv_stochastic_rounding(case, with_q16, cta_mode):
    """rounding_scheme STOCHASTIC in the fused requantization: every kernel and tile shape gives the
    oracle's bits for the same seed (the draw depends on the output's index only)."""
    seed = 0xC0FFEE123456789 + sum(case)
    cs = 48 if case[3] == 20 else None
    cnt = run_conv_case(np.random.default_rng(sum(case) + 3), *case, B.ALGO_AUTO, with_q16=with_q16, cs=cs,
                        stochastic_seed=seed)
    assert cnt.zeros > 0


@pytest.mark.parametrize("shift_case", [(13, 15, 12), (4, 8, 12), (2, 3, 9), (0, 0, 0)])
def test_conv_stochastic_rounding_across_shifts(shift_case):
    """Long and short right shifts, an exact left shift (more fractional bits out than in) and shift 0."""
    fx, fw, f_out = shift_case
    run_conv_case(np.random.default_rng(sum(shift_case)), 2, 24, 24, 128, 128, 3, 1, 1, 16, 16, 16, True,
                  B.ALGO_TENSOR, f_out=f_out, with_q16=False, mag_bits=(6, 6), fmts=(fx, fw), stochastic_seed=99)


@pytest.mark.parametrize("case", [(70, 1000, 260, 16, 16, 16, False), (64, 25088, 250, 16, 16, 16, True),
                                  (130, 256, 128, 8, 8, 8, True), (5, 64, 33, 16, 8, 16, False)])
@pytest.mark.parametrize("algo", [B.ALGO_AUTO, B.ALGO_DIRECT])
def test_ip_stochastic_rounding(case, algo):
    """Inner products, including a split reduction (the finalize kernel rounds) and the plain kernel."""
    if algo == B.ALGO_DIRECT and case[1] > 2000:
        pytest.skip("the plain kernel takes too long on the long reduction")
    run_ip_case(np.random.default_rng(sum(case) + 9), *case, algo, stochastic_seed=0xFEEDFACE + case[0])


def test_stochastic_layer_statistics():
    """Sec. 2.4 at the level of a layer: another seed gives other bits, the same seed the same; every
    output is one of the two neighbours of the unrounded value; the mean error over a large layer
    vanishes where the deterministic tie rule does not matter."""
    rng = np.random.default_rng(4)
    N, H, W, Cin, K = 2, 24, 24, 128, 128
    xq, wq = _rand_q(rng, (N, H, W, Cin), 12, 0.4), _rand_q(rng, (K, 3, 3, Cin), 12)
    x, w = to_qtensor(xq.reshape(-1, Cin), 16, 9, Cin), to_qtensor(wq.reshape(-1, Cin), 16, 11, Cin)
    shp = B.conv_shape(N, H, W, Cin, K, 3, 3, 1, 1)
    acc = orc.conv_acc(xq, wq, (1, 1))
    outs = []
    for seed in (1, 1, 2):
        y = B.QTensor.empty(N * H * W, K, 16, 2, K)
        B.adaption_lp_conv_fwd_stochastic(shp, x, w, None, 0, False, B.ALGO_TENSOR, y, seed, B.new_stats(), None)
        outs.append(from_qtensor(y).reshape(acc.shape).astype(np.float64))
    assert np.array_equal(outs[0], outs[1]) and not np.array_equal(outs[0], outs[2])
    exact = acc.astype(np.float64) / 2.0 ** 18
    assert np.all((outs[0] == np.floor(exact)) | (outs[0] == np.floor(exact) + 1))
    assert abs(float((outs[0] - exact).mean())) < 5 * 0.5 / np.sqrt(exact.size)


# ------------------------------------------------------------------ robustness of the boundary
@pytest.mark.parametrize("mode", ["single", "pair"])
@pytest.mark.parametrize("stall_at", [0, 5])
def test_device_side_wait_runs_out_and_the_next_call_is_exact(mode, stall_at):
    """Failure detection without a fault: the copy-issuing warps are told to stop before one of their
    stages (nothing is in flight for it), the waits of the other warps run out after a few
    milliseconds, the kernel flags ADAPTION_ERR_TIMEOUT in the caller's stats word, drains, frees its
    tensor memory and returns.  The context stays usable: the same call without the stall gives the
    oracle's bits."""
    case = (4, 16, 16, 128, 128, 3, 1, 1, 16, 16, 16, True)       # four tiles of 256 rows / eight of 128
    N, H, W, Cin, K = case[:5]
    rng = np.random.default_rng(21)
    xq, wq = _rand_q(rng, (N, H, W, Cin), 16, 0.4), _rand_q(rng, (K, 3, 3, Cin), 16)
    x, w = to_qtensor(xq.reshape(-1, Cin), 16, 13, Cin), to_qtensor(wq.reshape(-1, Cin), 16, 15, Cin)
    shp = B.conv_shape(N, H, W, Cin, K, 3, 3, 1, 1)
    y = B.QTensor.empty(N * H * W, K, 16, 5, K)
    B.adaption_debug_set("pair", 1 if mode == "pair" else 0)
    B.adaption_debug_set("timeout_us", 3000)
    B.adaption_debug_set("stall_at", stall_at)
    st = B.new_stats()
    B.adaption_lp_conv_fwd(shp, x, w, None, 0, True, B.MODE_REQUANT, B.ALGO_TENSOR, y, st, None)
    torch.cuda.synchronize()                                   # the kernel returned by itself
    assert B.read_stats(st).status == B.ERR_TIMEOUT
    assert B.status_string(B.read_stats(st).status) == "device-side wait timed out"
    B.adaption_debug_set("stall_at", -1)
    B.adaption_debug_set("timeout_us", 0)
    run_conv_case(np.random.default_rng(22), *case, B.ALGO_TENSOR, with_q16=False)


def test_left_shift_of_accumulators_beyond_2_to_the_48():
    """An inner product long enough for |acc| = 2^48 (262144 products of -32768 * -32768) requantized
    to MORE fractional bits than the accumulator has: the exact product acc * 2^15 does not fit 64 bits
    and must still saturate (both kernels)."""
    Bsz, K, O = 2, 1 << 18, 3
    xq = np.full((Bsz, K), -32768, dtype=np.int16)
    xq[1, :] = 32767
    wq = np.full((O, K), -32768, dtype=np.int16)
    wq[2, :] = 0
    wq[2, 0] = 1
    want, cnt = orc.epilogue(orc.ip_acc(xq, wq), None, 0, 0, False, 16, 15)
    assert want.tolist() == [[32767, 32767, -32768], [-32768, -32768, 32767]]
    x, w = to_qtensor(xq, 16, 0), to_qtensor(wq, 16, 0)
    for algo in (B.ALGO_DIRECT, B.ALGO_TENSOR):
        need = B.adaption_lp_ip_workspace_bytes(Bsz, K, O, x.fmt(), w.fmt(), algo)
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda") if need else None
        y = B.QTensor.empty(Bsz, O, 16, 15)
        st = B.new_stats()
        B.adaption_lp_ip_fwd(Bsz, K, O, x, w, None, 0, False, B.MODE_REQUANT, algo, y, st, ws)
        assert np.array_equal(from_qtensor(y), want)
        assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)


def test_layer_calls_from_two_host_threads():
    """The library keeps no per-call state: two host threads, each with its own stream and buffers,
    run different layers at the same time and both get the oracle's bits."""
    import threading
    errors = []

    def work(seed, case):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                for rep in range(3):
                    run_conv_case(np.random.default_rng(seed + rep), *case, B.ALGO_TENSOR, with_q16=False)
        except Exception as exc:                              # noqa: BLE001 - reported to the main thread
            errors.append(exc)

    t1 = threading.Thread(target=work, args=(31, (2, 24, 24, 128, 128, 3, 1, 1, 16, 16, 16, True)))
    t2 = threading.Thread(target=work, args=(41, (5, 30, 30, 64, 64, 3, 1, 1, 16, 16, 16, True)))
    t1.start(); t2.start(); t1.join(); t2.join()
    assert not errors, errors
