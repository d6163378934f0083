"""Thin ctypes binding of the C ABI in include/adaption.h (argument marshalling only).

Every function here has the name of the C entry point it calls.  Device memory comes from
torch tensors (``QTensor`` wraps the byte planes of one fixed-point tensor); all arithmetic runs
in the CUDA library.  Importing this module never builds or falls back to anything: if the
shared library is missing, ``load()`` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

from . import build as _build

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE = 1, 2, 3, 4
ERR_K_TOO_LARGE, ERR_CUDA, ERR_TIMEOUT = 5, 6, 7
ROUND_DETERMINISTIC, ROUND_STOCHASTIC = 0, 1
MODE_REQUANT, MODE_RANGE = 0, 1
ALGO_AUTO, ALGO_TENSOR, ALGO_DIRECT = 0, 1, 2
PHASE_CONV, PHASE_POOL = 1, 2


class adaption_qfmt(C.Structure):
    _fields_ = [("n_bits", C.c_int32), ("frac_bits", C.c_int32)]


class adaption_qtensor(C.Structure):
    _fields_ = [("hi", C.c_void_p), ("lo", C.c_void_p), ("q16", C.c_void_p),
                ("fmt", adaption_qfmt), ("c_stride", C.c_int64)]


class adaption_quantize_item(C.Structure):
    _fields_ = [("d_x", C.c_void_p), ("outer", C.c_int64), ("inner", C.c_int64), ("q", adaption_qtensor),
                ("d_fmt", C.c_void_p)]


class adaption_stats(C.Structure):
    _fields_ = [("zeros", C.c_uint64), ("sat_pos", C.c_uint64), ("sat_neg", C.c_uint64),
                ("max_abs_acc", C.c_int64), ("status", C.c_int32), ("reserved", C.c_int32)]


class adaption_conv_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("N", "H", "W", "C", "K", "R", "S", "pad_h", "pad_w",
                                          "stride_h", "stride_w")]


STATS_BYTES = C.sizeof(adaption_stats)
EXPORTS = [
    "adaption_measure_range", "adaption_quantize", "adaption_lp_act",
    "adaption_lp_conv_workspace_bytes", "adaption_lp_conv_fwd", "adaption_lp_ip_workspace_bytes",
    "adaption_lp_ip_fwd", "adaption_lp_ip_fwd_static_ws", "adaption_maxpool2x2", "adaption_choose_frac_bits_from_acc",
    "adaption_probe_i8_peak", "adaption_status_string",
    "adaption_quantize_stochastic", "adaption_bit_histogram", "adaption_width_histogram",
    "adaption_choose_frac_bits_from_hist", "adaption_choose_frac_bits_from_widths",
    "adaption_lp_act_stochastic", "adaption_lp_conv_pool_workspace_bytes", "adaption_lp_conv_pool_fwd",
    "adaption_quantize_batch", "adaption_debug_set", "adaption_lp_conv_fwd_stochastic",
    "adaption_lp_ip_fwd_stochastic",
]
HIST_BINS = 17

_lib = None


class AdaptionError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def load(path: str | None = None):
    """Load lib/libadaption.so (built in-tree by build.build_library).  Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"CUDA library not built: {path} is missing "
                           "(run `python -m paper_1711_04713_b200.build`)")
    lib = C.CDLL(path)
    P, I32, I64, SZ = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    lib.adaption_measure_range.argtypes = [P, SZ, I32, P, P, P]
    lib.adaption_quantize.argtypes = [P, SZ, SZ, adaption_qtensor, P, I32, P, P]
    lib.adaption_lp_act.argtypes = [P, C.POINTER(adaption_qtensor), SZ, SZ, I32, adaption_qtensor, P, I32, P, P]
    lib.adaption_lp_conv_workspace_bytes.argtypes = [C.POINTER(adaption_conv_shape), adaption_qfmt,
                                                     adaption_qfmt, I64, I32]
    lib.adaption_lp_conv_workspace_bytes.restype = SZ
    lib.adaption_lp_conv_fwd.argtypes = [C.POINTER(adaption_conv_shape), adaption_qtensor, adaption_qtensor,
                                         P, I32, I32, I32, I32, adaption_qtensor, P, P, SZ, P]
    lib.adaption_quantize_batch.argtypes = [C.POINTER(adaption_quantize_item), I32, P]
    lib.adaption_lp_conv_fwd_stochastic.argtypes = [C.POINTER(adaption_conv_shape), adaption_qtensor,
                                                    adaption_qtensor, P, I32, I32, I32, adaption_qtensor,
                                                    C.c_uint64, P, P, SZ, P]
    lib.adaption_lp_ip_fwd_stochastic.argtypes = [I64, I64, I64, adaption_qtensor, adaption_qtensor, P, I32, I32,
                                                  I32, adaption_qtensor, C.c_uint64, P, P, SZ, P]
    lib.adaption_lp_conv_pool_workspace_bytes.argtypes = [C.POINTER(adaption_conv_shape), adaption_qfmt,
                                                          adaption_qfmt, adaption_qfmt, I64, I64, I32]
    lib.adaption_lp_conv_pool_workspace_bytes.restype = SZ
    lib.adaption_lp_conv_pool_fwd.argtypes = [C.POINTER(adaption_conv_shape), adaption_qtensor, adaption_qtensor,
                                              P, I32, I32, I32, I32, adaption_qtensor, P, P, SZ, P]
    lib.adaption_lp_ip_workspace_bytes.argtypes = [I64, I64, I64, adaption_qfmt, adaption_qfmt, I32]
    lib.adaption_lp_ip_workspace_bytes.restype = SZ
    lib.adaption_lp_ip_fwd.argtypes = [I64, I64, I64, adaption_qtensor, adaption_qtensor, P, I32, I32, I32,
                                       I32, adaption_qtensor, P, P, SZ, P]
    lib.adaption_lp_ip_fwd_static_ws.argtypes = [I64, I64, I64, adaption_qtensor, adaption_qtensor, P, I32, I32,
                                                 I32, I32, adaption_qtensor, P, P]
    lib.adaption_maxpool2x2.argtypes = [adaption_qtensor, I32, I32, I32, I32, adaption_qtensor, P]
    lib.adaption_choose_frac_bits_from_acc.argtypes = [I64, I32, I32, C.POINTER(adaption_qfmt)]
    lib.adaption_probe_i8_peak.argtypes = [I32, I32, I32, I32, P, P, P]
    lib.adaption_quantize_stochastic.argtypes = [P, SZ, SZ, adaption_qtensor, P, I32, C.c_uint64, P, P]
    lib.adaption_lp_act_stochastic.argtypes = [P, C.POINTER(adaption_qtensor), SZ, SZ, I32, adaption_qtensor, P,
                                               C.c_uint64, P, P]
    lib.adaption_bit_histogram.argtypes = [P, SZ, P, P]
    lib.adaption_width_histogram.argtypes = [adaption_qtensor, SZ, SZ, P, P]
    lib.adaption_choose_frac_bits_from_hist.argtypes = [C.POINTER(C.c_uint64), I32, C.c_double,
                                                        C.POINTER(adaption_qfmt)]
    lib.adaption_choose_frac_bits_from_widths.argtypes = [C.POINTER(C.c_uint64), I32, I32, C.c_double,
                                                          C.POINTER(adaption_qfmt)]
    lib.adaption_debug_set.argtypes = [C.c_char_p, C.c_int32]
    lib.adaption_status_string.argtypes = [C.c_int]
    lib.adaption_status_string.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("adaption_lp_conv_workspace_bytes", "adaption_lp_ip_workspace_bytes",
                        "adaption_lp_conv_pool_workspace_bytes", "adaption_status_string"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def adaption_debug_set(name: str, value: int = 0):
    """Test / experiment override of the tensor-core path's heuristics (see the header)."""
    _check(load().adaption_debug_set(name.encode(), int(value)), f"adaption_debug_set({name})")


def status_string(status: int) -> str:
    return load().adaption_status_string(int(status)).decode()


def _check(rc: int, where: str):
    if rc != OK:
        raise AdaptionError(rc, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def pad_to(n: int, mult: int) -> int:
    return (n + mult - 1) // mult * mult


@dataclass
class QTensor:
    """Byte planes of a fixed-point tensor on the device: logical shape (outer, inner), row pitch
    ``c_stride``.  ``lo``/``hi`` are uint8/int8 torch tensors of outer*c_stride bytes."""
    outer: int
    inner: int
    c_stride: int
    n_bits: int
    frac_bits: int
    lo: torch.Tensor
    hi: torch.Tensor | None = None
    q16: torch.Tensor | None = None

    @staticmethod
    def empty(outer: int, inner: int, n_bits: int, frac_bits: int = 0, c_stride: int | None = None,
              with_q16: bool = False, device="cuda") -> "QTensor":
        cs = pad_to(inner, 16) if c_stride is None else c_stride
        lo = torch.empty(outer * cs, dtype=torch.uint8, device=device)
        hi = torch.empty(outer * cs, dtype=torch.int8, device=device) if n_bits > 8 else None
        q16 = torch.empty(outer * cs, dtype=torch.int16, device=device) if with_q16 else None
        return QTensor(outer, inner, cs, n_bits, frac_bits, lo, hi, q16)

    def c_struct(self) -> adaption_qtensor:
        return adaption_qtensor(_ptr(self.hi), _ptr(self.lo), _ptr(self.q16),
                                adaption_qfmt(self.n_bits, self.frac_bits), self.c_stride)

    def fmt(self) -> adaption_qfmt:
        return adaption_qfmt(self.n_bits, self.frac_bits)

    def to_int16(self) -> torch.Tensor:
        """Canonical integers as an (outer, inner) int16 CPU tensor (view/convert only)."""
        lo = self.lo.view(self.outer, self.c_stride)[:, :self.inner].cpu()
        if self.hi is None:
            return lo.view(torch.int8).to(torch.int16)
        hi = self.hi.view(self.outer, self.c_stride)[:, :self.inner].cpu()
        return hi.to(torch.int16) * 256 + lo.to(torch.int16)

    def padding_is_zero(self) -> bool:
        if self.c_stride == self.inner:
            return True
        ok = bool((self.lo.view(self.outer, self.c_stride)[:, self.inner:] == 0).all())
        if self.hi is not None:
            ok = ok and bool((self.hi.view(self.outer, self.c_stride)[:, self.inner:] == 0).all())
        return ok

    def reshaped(self, outer: int, inner: int, c_stride: int | None = None) -> "QTensor":
        """Same bytes seen with another row structure (e.g. NHWC activations flattened per image)."""
        cs = inner if c_stride is None else c_stride
        assert outer * cs == self.outer * self.c_stride
        return QTensor(outer, inner, cs, self.n_bits, self.frac_bits, self.lo, self.hi, self.q16)


def new_stats(device="cuda") -> torch.Tensor:
    """Zeroed device-resident adaption_stats (as raw bytes)."""
    return torch.zeros(STATS_BYTES, dtype=torch.uint8, device=device)


def read_stats(stats: torch.Tensor) -> adaption_stats:
    raw = bytes(stats.cpu().numpy().tobytes())
    return adaption_stats.from_buffer_copy(raw)


# --------------------------------------------------------------------------- entry points
def adaption_measure_range(x: torch.Tensor, n_bits: int, d_max_abs: torch.Tensor,
                           d_fmt_out: torch.Tensor | None):
    """x: fp32 CUDA tensor (contiguous); d_max_abs: 1 fp32; d_fmt_out: 2 int32 (n_bits, frac_bits)."""
    _check(load().adaption_measure_range(_ptr(x), x.numel(), n_bits, _ptr(d_max_abs), _ptr(d_fmt_out),
                                         _stream()), "adaption_measure_range")


def adaption_quantize(x: torch.Tensor, outer: int, inner: int, out: QTensor,
                      d_fmt: torch.Tensor | None = None, rounding: int = ROUND_DETERMINISTIC,
                      d_stats: torch.Tensor | None = None):
    _check(load().adaption_quantize(_ptr(x), outer, inner, out.c_struct(), _ptr(d_fmt), rounding,
                                    _ptr(d_stats), _stream()), "adaption_quantize")


def quantize_items(entries) -> "C.Array":
    """Host array of adaption_quantize_item from (x, outer, inner, out, d_fmt or None) tuples."""
    arr = (adaption_quantize_item * len(entries))()
    for it, (x, outer, inner, out, d_fmt) in zip(arr, entries):
        it.d_x, it.outer, it.inner, it.q, it.d_fmt = _ptr(x), outer, inner, out.c_struct(), _ptr(d_fmt)
    return arr


def adaption_quantize_batch(items, n_items: int | None = None):
    """``items``: a ctypes array from quantize_items() (the tensors it names must stay alive)."""
    n = len(items) if n_items is None else n_items
    _check(load().adaption_quantize_batch(items, n, _stream()), "adaption_quantize_batch")


def adaption_quantize_stochastic(x: torch.Tensor, outer: int, inner: int, out: QTensor, seed: int,
                                 relu: bool = False, d_fmt: torch.Tensor | None = None,
                                 d_stats: torch.Tensor | None = None):
    _check(load().adaption_quantize_stochastic(_ptr(x), outer, inner, out.c_struct(), _ptr(d_fmt), int(relu),
                                               seed & 0xFFFFFFFFFFFFFFFF, _ptr(d_stats), _stream()),
           "adaption_quantize_stochastic")


def adaption_lp_act_stochastic(x_f32: torch.Tensor | None, x_q: QTensor | None, outer: int, inner: int, relu: bool,
                               out: QTensor, seed: int, d_fmt: torch.Tensor | None = None,
                               d_stats: torch.Tensor | None = None):
    xq = None if x_q is None else C.byref(x_q.c_struct())
    _check(load().adaption_lp_act_stochastic(_ptr(x_f32), xq, outer, inner, int(relu), out.c_struct(), _ptr(d_fmt),
                                             seed & 0xFFFFFFFFFFFFFFFF, _ptr(d_stats), _stream()),
           "adaption_lp_act_stochastic")


def new_hist(device="cuda") -> torch.Tensor:
    """Zeroed device histogram of HIST_BINS 64-bit counters (int64 storage, values are counts)."""
    return torch.zeros(HIST_BINS, dtype=torch.int64, device=device)


def adaption_bit_histogram(x: torch.Tensor, d_hist: torch.Tensor):
    _check(load().adaption_bit_histogram(_ptr(x), x.numel(), _ptr(d_hist), _stream()), "adaption_bit_histogram")


def adaption_width_histogram(x: QTensor, d_hist: torch.Tensor):
    _check(load().adaption_width_histogram(x.c_struct(), x.outer, x.inner, _ptr(d_hist), _stream()),
           "adaption_width_histogram")


def adaption_choose_frac_bits_from_hist(hist, n_bits: int, threshold: float) -> int:
    """hist: HIST_BINS counts on the host (sequence or CPU tensor)."""
    arr = (C.c_uint64 * HIST_BINS)(*[int(v) for v in hist])
    out = adaption_qfmt()
    _check(load().adaption_choose_frac_bits_from_hist(arr, n_bits, float(threshold), C.byref(out)),
           "adaption_choose_frac_bits_from_hist")
    return int(out.frac_bits)


def adaption_choose_frac_bits_from_widths(hist, frac_bits: int, n_bits: int, threshold: float) -> int:
    """hist: HIST_BINS width counts on the host of a tensor stored with ``frac_bits`` fractional bits."""
    arr = (C.c_uint64 * HIST_BINS)(*[int(v) for v in hist])
    out = adaption_qfmt()
    _check(load().adaption_choose_frac_bits_from_widths(arr, frac_bits, n_bits, float(threshold), C.byref(out)),
           "adaption_choose_frac_bits_from_widths")
    return int(out.frac_bits)


def adaption_lp_act(x_f32: torch.Tensor | None, x_q: QTensor | None, outer: int, inner: int, relu: bool,
                    out: QTensor, d_fmt: torch.Tensor | None = None, rounding: int = ROUND_DETERMINISTIC,
                    d_stats: torch.Tensor | None = None):
    xq = None if x_q is None else C.byref(x_q.c_struct())
    _check(load().adaption_lp_act(_ptr(x_f32), xq, outer, inner, int(relu), out.c_struct(), _ptr(d_fmt),
                                  rounding, _ptr(d_stats), _stream()), "adaption_lp_act")


def conv_shape(N, H, W, Cin, K, R, S, pad, stride) -> adaption_conv_shape:
    return adaption_conv_shape(N, H, W, Cin, K, R, S, pad, pad, stride, stride)


def adaption_lp_conv_workspace_bytes(shape: adaption_conv_shape, fx: adaption_qfmt, fw: adaption_qfmt,
                                     c_stride: int, algo: int = ALGO_AUTO) -> int:
    return int(load().adaption_lp_conv_workspace_bytes(C.byref(shape), fx, fw, c_stride, algo))


def adaption_lp_conv_fwd(shape: adaption_conv_shape, x: QTensor, w: QTensor, bias_q: torch.Tensor | None,
                         bias_frac_bits: int, relu: bool, mode: int, algo: int, y: QTensor | None,
                         d_stats: torch.Tensor, workspace: torch.Tensor | None = None):
    ys = y.c_struct() if y is not None else adaption_qtensor()
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().adaption_lp_conv_fwd(C.byref(shape), x.c_struct(), w.c_struct(), _ptr(bias_q),
                                       bias_frac_bits, int(relu), mode, algo, ys, _ptr(d_stats),
                                       _ptr(workspace), wsb, _stream()), "adaption_lp_conv_fwd")


def adaption_lp_conv_fwd_stochastic(shape: adaption_conv_shape, x: QTensor, w: QTensor, bias_q: torch.Tensor | None,
                                    bias_frac_bits: int, relu: bool, algo: int, y: QTensor, seed: int,
                                    d_stats: torch.Tensor, workspace: torch.Tensor | None = None):
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().adaption_lp_conv_fwd_stochastic(C.byref(shape), x.c_struct(), w.c_struct(), _ptr(bias_q),
                                                  bias_frac_bits, int(relu), algo, y.c_struct(),
                                                  seed & 0xFFFFFFFFFFFFFFFF, _ptr(d_stats), _ptr(workspace), wsb,
                                                  _stream()), "adaption_lp_conv_fwd_stochastic")


def adaption_lp_ip_fwd_stochastic(B: int, K: int, O: int, x: QTensor, w: QTensor, bias_q: torch.Tensor | None,
                                  bias_frac_bits: int, relu: bool, algo: int, y: QTensor, seed: int,
                                  d_stats: torch.Tensor, workspace: torch.Tensor | None = None):
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().adaption_lp_ip_fwd_stochastic(B, K, O, x.c_struct(), w.c_struct(), _ptr(bias_q), bias_frac_bits,
                                                int(relu), algo, y.c_struct(), seed & 0xFFFFFFFFFFFFFFFF,
                                                _ptr(d_stats), _ptr(workspace), wsb, _stream()),
           "adaption_lp_ip_fwd_stochastic")


def adaption_lp_conv_pool_workspace_bytes(shape: adaption_conv_shape, fx: adaption_qfmt, fw: adaption_qfmt,
                                          fy: adaption_qfmt, c_stride: int, y_c_stride: int,
                                          algo: int = ALGO_AUTO) -> int:
    return int(load().adaption_lp_conv_pool_workspace_bytes(C.byref(shape), fx, fw, fy, c_stride, y_c_stride, algo))


def adaption_lp_conv_pool_fwd(shape: adaption_conv_shape, x: QTensor, w: QTensor, bias_q: torch.Tensor | None,
                              bias_frac_bits: int, relu: bool, algo: int, y: QTensor, d_stats: torch.Tensor,
                              workspace: torch.Tensor | None, phases: int = 3):
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().adaption_lp_conv_pool_fwd(C.byref(shape), x.c_struct(), w.c_struct(), _ptr(bias_q), bias_frac_bits,
                                            int(relu), algo, phases, y.c_struct(), _ptr(d_stats), _ptr(workspace),
                                            wsb, _stream()), "adaption_lp_conv_pool_fwd")


def adaption_lp_ip_workspace_bytes(B: int, K: int, O: int, fx: adaption_qfmt, fw: adaption_qfmt,
                                   algo: int = ALGO_AUTO) -> int:
    return int(load().adaption_lp_ip_workspace_bytes(B, K, O, fx, fw, algo))


def adaption_lp_ip_fwd(B: int, K: int, O: int, x: QTensor, w: QTensor, bias_q: torch.Tensor | None,
                       bias_frac_bits: int, relu: bool, mode: int, algo: int, y: QTensor | None,
                       d_stats: torch.Tensor, workspace: torch.Tensor | None = None):
    ys = y.c_struct() if y is not None else adaption_qtensor()
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().adaption_lp_ip_fwd(B, K, O, x.c_struct(), w.c_struct(), _ptr(bias_q), bias_frac_bits,
                                     int(relu), mode, algo, ys, _ptr(d_stats), _ptr(workspace), wsb,
                                     _stream()), "adaption_lp_ip_fwd")


STATIC_WORKSPACE_BYTES = 4 << 20


def adaption_lp_ip_fwd_static_ws(B: int, K: int, O: int, x: QTensor, w: QTensor, bias_q: torch.Tensor | None,
                                 bias_frac_bits: int, relu: bool, mode: int, algo: int, y: QTensor | None,
                                 d_stats: torch.Tensor):
    """adaption_lp_ip_fwd without a workspace argument: the library's built-in scratch array is used.
    For callers that must not allocate; shapes whose workspace exceeds STATIC_WORKSPACE_BYTES raise
    AdaptionError(ERR_WORKSPACE).  Calls that may overlap on the GPU must be ordered by the caller."""
    ys = y.c_struct() if y is not None else adaption_qtensor()
    _check(load().adaption_lp_ip_fwd_static_ws(B, K, O, x.c_struct(), w.c_struct(), _ptr(bias_q),
                                               bias_frac_bits, int(relu), mode, algo, ys, _ptr(d_stats),
                                               _stream()), "adaption_lp_ip_fwd_static_ws")


def adaption_maxpool2x2(x: QTensor, N: int, H: int, W: int, Cc: int, y: QTensor):
    _check(load().adaption_maxpool2x2(x.c_struct(), N, H, W, Cc, y.c_struct(), _stream()),
           "adaption_maxpool2x2")


def adaption_probe_i8_peak(bn: int, pair: bool, iters: int, d_cycles: torch.Tensor, d_status: torch.Tensor,
                           commit_every: int = 0):
    """d_cycles: int64 CUDA tensor with one entry per SM; d_status: one int32."""
    _check(load().adaption_probe_i8_peak(bn, int(pair), iters, commit_every, _ptr(d_cycles), _ptr(d_status), _stream()),
           "adaption_probe_i8_peak")


def adaption_choose_frac_bits_from_acc(max_abs_acc: int, acc_frac_bits: int, n_bits: int) -> int:
    out = adaption_qfmt()
    _check(load().adaption_choose_frac_bits_from_acc(max_abs_acc, acc_frac_bits, n_bits, C.byref(out)),
           "adaption_choose_frac_bits_from_acc")
    return int(out.frac_bits)
