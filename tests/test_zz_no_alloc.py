"""The allocation-free inner product (adaption_lp_ip_fwd_static_ws).

Some users of this library cannot call cudaMalloc at the point where they run a layer: a plug-in
that was handed a fixed memory arena by its host application, or a latency-critical loop in which an
allocation would stall the device.  For them the library carries its own split-K scratch.  This file
checks, through the C ABI, that the entry point gives exactly the bits of the regular entry point
(which takes a caller-allocated workspace), on two calls in a row with different data - the second
call finds the first call's partial sums in the shared scratch and must not be disturbed by them -
and that a shape beyond the built-in scratch is refused cleanly.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_1711_04713_b200 import binding as B
from tests.util import dev, from_qtensor, stats_tuple, to_qtensor

pytestmark = pytest.mark.gpu


def _case(seed, Bsz, K, O, relu):
    rng = np.random.default_rng(seed)
    xq = rng.integers(-32768, 32768, (Bsz, K)).astype(np.int16)
    xq[rng.random(xq.shape) < 0.4] = 0
    wq = rng.integers(-32768, 32768, (O, K)).astype(np.int16)
    bq = rng.integers(-32768, 32768, (O,)).astype(np.int16)
    return to_qtensor(xq, 16, 12), to_qtensor(wq, 16, 15), dev(bq), (xq, wq, bq)


def _run_both(seed, Bsz, K, O, relu, f_out, uses_scratch=True):
    x, w, bias, host = _case(seed, Bsz, K, O, relu)
    need = B.adaption_lp_ip_workspace_bytes(Bsz, K, O, x.fmt(), w.fmt(), B.ALGO_TENSOR)
    if uses_scratch:
        assert 0 < need <= B.STATIC_WORKSPACE_BYTES      # the split-K (scratch-using) path is exercised
    else:
        assert need == 0                                 # an unsplit reduction: the array is not touched
    ws_bytes = max(need, 16)
    # regular entry point, caller-owned workspace
    y_ref = B.QTensor.empty(Bsz, O, 16, f_out, None, with_q16=True)
    st_ref = B.new_stats()
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    B.adaption_lp_ip_fwd(Bsz, K, O, x, w, bias, 15, relu, B.MODE_REQUANT, B.ALGO_TENSOR, y_ref, st_ref, ws)
    rg_ref = B.new_stats()
    B.adaption_lp_ip_fwd(Bsz, K, O, x, w, bias, 15, relu, B.MODE_RANGE, B.ALGO_TENSOR, None, rg_ref, ws)
    # allocation-free entry point: every buffer it is given exists already
    y = B.QTensor.empty(Bsz, O, 16, f_out, None, with_q16=True)
    y.lo.fill_(0x5A)
    st, rg = B.new_stats(), B.new_stats()
    torch.cuda.synchronize()
    B.adaption_lp_ip_fwd_static_ws(Bsz, K, O, x, w, bias, 15, relu, B.MODE_REQUANT, B.ALGO_TENSOR, y, st)
    B.adaption_lp_ip_fwd_static_ws(Bsz, K, O, x, w, bias, 15, relu, B.MODE_RANGE, B.ALGO_TENSOR, None, rg)
    torch.cuda.synchronize()
    assert B.read_stats(st).status == 0 and B.read_stats(rg).status == 0
    assert np.array_equal(from_qtensor(y), from_qtensor(y_ref))          # bit-exact, like every parity test
    assert torch.equal(y.q16, y_ref.q16)
    assert stats_tuple(st) == stats_tuple(st_ref)
    assert int(B.read_stats(rg).max_abs_acc) == int(B.read_stats(rg_ref).max_abs_acc) > 0
    # and against the CPU oracle directly, not only through the regular entry point
    xq, wq, bq = host
    want, cnt = orc.epilogue(orc.ip_acc(xq, wq), bq, 15, 27, relu, 16, f_out)
    assert np.array_equal(from_qtensor(y), want)
    assert stats_tuple(st) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    return from_qtensor(y)


def test_static_workspace_matches_regular_entry_point_twice_in_a_row():
    first = _run_both(1, 64, 25088, 256, True, 2)        # FC6-like: long reduction, two output tiles
    second = _run_both(2, 48, 8192, 200, False, 3)       # other shape and data on the same scratch
    assert first.shape == (64, 256) and second.shape == (48, 200)
    assert first.any() and second.any()


def test_shapes_without_scratch_and_calls_on_another_stream():
    """A reduction short enough to stay unsplit needs no scratch (the entry point then passes none on);
    and the entry point honours the caller's stream like every other call."""
    _run_both(3, 256, 512, 384, True, 4, uses_scratch=False)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        out = _run_both(4, 64, 25088, 256, True, 2)
    side.synchronize()
    torch.cuda.current_stream().wait_stream(side)
    assert out.any()


def test_shape_beyond_the_built_in_scratch_is_refused():
    Bsz, K, O = 640, 4096, 1024
    x = B.QTensor.empty(Bsz, K, 16, 12)
    w = B.QTensor.empty(O, K, 16, 15)
    y = B.QTensor.empty(Bsz, O, 16, 3)
    y.lo.fill_(7)
    need = B.adaption_lp_ip_workspace_bytes(Bsz, K, O, x.fmt(), w.fmt(), B.ALGO_TENSOR)
    assert need > B.STATIC_WORKSPACE_BYTES
    with pytest.raises(B.AdaptionError) as e:
        B.adaption_lp_ip_fwd_static_ws(Bsz, K, O, x, w, None, 0, True, B.MODE_REQUANT, B.ALGO_TENSOR, y,
                                       B.new_stats())
    assert e.value.status == B.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert int(y.lo[0]) == 7                              # nothing was launched
