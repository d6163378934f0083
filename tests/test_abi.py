"""CPU-side checks of the boundary: the library builds, loads without a GPU, exports every symbol
the header declares, and rejects bad arguments on the host before any launch."""
import ctypes
import os
import re

import pytest

from paper_1711_04713_b200 import binding as B
from paper_1711_04713_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.load()


def test_header_symbols_are_exported(lib):
    text = open(os.path.join(ROOT, "include", "adaption.h")).read()
    declared = sorted(set(re.findall(r"ADAPTION_API\s+[\w\s\*]+?\b(adaption_\w+)\s*\(", text)))
    assert declared == sorted(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_header():
    assert ctypes.sizeof(B.adaption_qfmt) == 8
    assert ctypes.sizeof(B.adaption_qtensor) == 40
    assert ctypes.sizeof(B.adaption_stats) == 40
    assert ctypes.sizeof(B.adaption_conv_shape) == 44
    assert ctypes.sizeof(B.adaption_quantize_item) == 72


def test_status_strings(lib):
    assert B.status_string(B.OK) == "ok"
    assert "timed out" in B.status_string(B.ERR_TIMEOUT)
    assert B.status_string(99) == "unknown status"


def test_choose_frac_bits_host_helper(lib):
    # max 0.375 * 2^29 needs no integer bit; 2^29 (= 1.0) needs one
    assert B.adaption_choose_frac_bits_from_acc(201326592, 29, 16) == 15
    assert B.adaption_choose_frac_bits_from_acc(1 << 29, 29, 16) == 14
    assert B.adaption_choose_frac_bits_from_acc((1 << 29) - 1, 29, 16) == 15
    assert B.adaption_choose_frac_bits_from_acc(0, 10, 8) == 7
    assert B.adaption_choose_frac_bits_from_acc(1 << 60, 10, 8) == 0
    with pytest.raises(B.AdaptionError):
        B.adaption_choose_frac_bits_from_acc(-1, 10, 8)


def test_host_side_argument_errors_need_no_gpu(lib):
    fake = 4096  # never dereferenced: every call below must fail validation first
    bad_fmt = B.adaption_qtensor(fake, fake, None, B.adaption_qfmt(17, 3), 16)
    assert lib.adaption_quantize(fake, 4, 16, bad_fmt, None, 0, None, None) == B.ERR_INVALID_ARG
    good = B.adaption_qtensor(fake, fake, None, B.adaption_qfmt(16, 3), 16)
    assert lib.adaption_quantize(fake, 4, 16, good, None, B.ROUND_STOCHASTIC, None, None) == B.ERR_UNSUPPORTED
    assert lib.adaption_quantize(fake, 4, 17, good, None, 0, None, None) == B.ERR_INVALID_ARG  # inner > pitch
    odd = B.adaption_qtensor(fake + 8, fake, None, B.adaption_qfmt(16, 3), 16)
    assert lib.adaption_quantize(fake, 4, 16, odd, None, 0, None, None) == B.ERR_ALIGNMENT
    assert lib.adaption_measure_range(fake, 10, 0, fake, None, None) == B.ERR_INVALID_ARG
    shp = B.conv_shape(1, 8, 8, 16, 16, 3, 3, 1, 1)
    assert lib.adaption_lp_conv_fwd(ctypes.byref(shp), good, good, None, 0, 1, 0, 0, good, None, None, 0,
                                    None) == B.ERR_INVALID_ARG      # stats missing
    shp0 = B.conv_shape(1, 8, 8, 16, 16, 3, 3, 1, 0)
    assert lib.adaption_lp_conv_fwd(ctypes.byref(shp0), good, good, None, 0, 1, 0, 0, good, fake, None, 0,
                                    None) == B.ERR_INVALID_ARG      # stride 0
    assert lib.adaption_lp_ip_fwd(4, 1 << 31, 8, good, good, None, 0, 0, 0, 0, good, fake, None, 0,
                                  None) == B.ERR_K_TOO_LARGE
    assert lib.adaption_maxpool2x2(good, 1, 3, 4, 16, good, None) == B.ERR_INVALID_ARG  # odd H
    # zero-sized work is accepted without touching memory
    assert lib.adaption_quantize(None, 0, 16, good, None, 0, None, None) == B.OK
    items = (B.adaption_quantize_item * 2)()
    items[0].d_x, items[0].outer, items[0].inner, items[0].q = None, 0, 16, good
    items[1].d_x, items[1].outer, items[1].inner, items[1].q = fake, 4, 16, bad_fmt
    assert lib.adaption_quantize_batch(items, 1, None) == B.OK              # only the empty tensor
    assert lib.adaption_quantize_batch(items, 2, None) == B.ERR_INVALID_ARG  # validated before any launch
    assert lib.adaption_quantize_batch(None, 1, None) == B.ERR_INVALID_ARG
    assert lib.adaption_quantize_batch(None, 0, None) == B.OK


def test_workspace_queries(lib):
    f16 = B.adaption_qfmt(16, 10)
    # direct algorithm never needs a workspace
    assert B.adaption_lp_ip_workspace_bytes(64, 25088, 4096, f16, f16, B.ALGO_DIRECT) == 0
    shp = B.conv_shape(1, 8, 8, 24, 16, 3, 3, 1, 1)   # pitch 48 is not a multiple of 32 -> direct kernel
    assert B.adaption_lp_conv_workspace_bytes(shp, f16, f16, 48) == 0


def test_threshold_allocation_host_helper_matches_oracle(lib):
    """adaption_choose_frac_bits_from_hist is host logic: compare it with the oracle's allocation on
    the hand-worked rows and on random histograms, thresholds included that sit exactly on a count."""
    import numpy as np

    from oracle import bit_allocation as ba

    golden = os.path.join(ROOT, "tests", "golden", "bit_allocation_handworked.txt")
    for line in open(golden):
        row = line.split()
        if row and row[0] == "alloc":
            n, thr = int(row[1]), float(row[2])
            hist = [int(v) for v in row[3:3 + ba.HIST_BINS]]
            assert B.adaption_choose_frac_bits_from_hist(hist, n, thr) == n - 1 - int(row[3 + ba.HIST_BINS]), row
    rng = np.random.default_rng(0)
    for _ in range(300):
        hist = (rng.integers(0, 1000, ba.HIST_BINS) * (rng.random(ba.HIST_BINS) < 0.5)).tolist()
        n = int(rng.integers(1, 17))
        total = sum(hist)
        tail = sum(hist[int(rng.integers(0, ba.HIST_BINS)):])
        for thr in (0.0, 0.01, float(rng.random()) * 0.2, (tail / total) if total else 0.0, 1.0):
            assert B.adaption_choose_frac_bits_from_hist(hist, n, thr) == ba.choose_frac_bits(hist, n, thr)
    for _ in range(200):
        hist = [0] + (rng.integers(0, 500, ba.HIST_BINS - 1) * (rng.random(ba.HIST_BINS - 1) < 0.6)).tolist()
        n, f = int(rng.integers(2, 17)), int(rng.integers(0, 16))
        for thr in (0.0, 0.01, 0.1):
            want = n - 1 - ba.choose_int_bits_from_widths(hist, f, n, thr)
            assert B.adaption_choose_frac_bits_from_widths(hist, f, n, thr) == want
    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(B.AdaptionError):
            B.adaption_choose_frac_bits_from_hist([0] * ba.HIST_BINS, 16, bad)
    with pytest.raises(B.AdaptionError):
        B.adaption_choose_frac_bits_from_hist([0] * ba.HIST_BINS, 17, 0.0)
