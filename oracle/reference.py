"""Python face of the CPU oracle (test infrastructure, not the product).

Loads ``adaption_oracle.c`` (compiled on demand with gcc) through ctypes and
offers numpy-level functions plus a small network driver.  It is a slow,
plain restatement of the forward pass of the low-precision layers of
arXiv 1711.04713 (Sec. 2, 2.1, 2.3) and shares nothing with the CUDA path.
Only tests, the smoke check and the benchmark's CPU-baseline leg use it.

Conventions: a fixed-point tensor is a numpy int16 array of canonical integers
``q`` plus a format ``(n_bits, frac_bits)``; its real value is ``q * 2**-frac_bits``.
Activations are NHWC, convolution weights [K][R][S][C], inner-product weights [O][K].
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "adaption_oracle.c")
_BUILD = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_BUILD, "libadaption_oracle.so")
_lib = None
BUILD_FLAGS = ["-O2", "-fopenmp", "-std=c11"]


def build(force: bool = False) -> str:
    """Compile the C oracle into ``oracle/_build`` (gcc, -O2, OpenMP)."""
    os.makedirs(_BUILD, exist_ok=True)
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC):
        tmp = _LIB_PATH + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc"] + BUILD_FLAGS + ["-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        P = c.c_void_p
        lib.oracle_num_threads.restype = c.c_int
        lib.oracle_quantize.argtypes = [P, c.c_size_t, c.c_int, c.c_int, c.c_int, P, P]
        lib.oracle_dequantize.argtypes = [P, c.c_size_t, c.c_int, P]
        lib.oracle_split_planes.argtypes = [P, c.c_size_t, P, P]
        lib.oracle_max_abs.argtypes = [P, c.c_size_t]
        lib.oracle_max_abs.restype = c.c_float
        lib.oracle_int_bits_from_max.argtypes = [c.c_float, c.c_int]
        lib.oracle_int_bits_from_max.restype = c.c_int
        lib.oracle_int_bits_from_acc.argtypes = [c.c_int64, c.c_int, c.c_int]
        lib.oracle_int_bits_from_acc.restype = c.c_int
        lib.oracle_conv_acc.argtypes = [P, P] + [c.c_int] * 11 + [P]
        lib.oracle_conv_acc_at.argtypes = [P, P] + [c.c_int] * 15
        lib.oracle_conv_acc_at.restype = c.c_int64
        lib.oracle_ip_acc.argtypes = [P, P, c.c_int64, c.c_int64, c.c_int64, P]
        lib.oracle_shift_round.argtypes = [c.c_int64, c.c_int]
        lib.oracle_shift_round.restype = c.c_int64
        lib.oracle_epilogue.argtypes = [P, c.c_size_t, c.c_size_t, P, c.c_int, c.c_int, c.c_int,
                                        c.c_int, c.c_int, P, P]
        lib.oracle_epilogue_range.argtypes = [P, c.c_size_t, c.c_size_t, P, c.c_int, c.c_int, c.c_int]
        lib.oracle_epilogue_range.restype = c.c_int64
        lib.oracle_requantize.argtypes = [P, c.c_size_t, c.c_int, c.c_int, c.c_int, c.c_int, P, P]
        lib.oracle_maxpool2x2.argtypes = [P, c.c_int, c.c_int, c.c_int, c.c_int, P]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


@dataclass
class Counters:
    """Sparsity / saturation counters (Sec. 3.1: sparsity = zeros / total)."""
    zeros: int = 0
    sat_pos: int = 0
    sat_neg: int = 0


def _counters_out(buf: np.ndarray) -> Counters:
    return Counters(int(buf[0]), int(buf[1]), int(buf[2]))


# ----------------------------------------------------------------------------------------
# Sec. 2: the quantizer
# ----------------------------------------------------------------------------------------
def quantize(x, n_bits: int, frac_bits: int, relu: bool = False):
    """fp32 -> canonical integers (int16), deterministic rounding + saturation."""
    _check_fmt(n_bits, frac_bits)
    x = _c(x, np.float32)
    q = np.empty(x.shape, dtype=np.int16)
    cnt = np.zeros(3, dtype=np.uint64)
    _load().oracle_quantize(_ptr(x), x.size, n_bits, frac_bits, int(relu), _ptr(q), _ptr(cnt))
    return q, _counters_out(cnt)


def dequantize(q, frac_bits: int) -> np.ndarray:
    q = _c(q, np.int16)
    out = np.empty(q.shape, dtype=np.float64)
    _load().oracle_dequantize(_ptr(q), q.size, frac_bits, _ptr(out))
    return out


def split_planes(q):
    """q = 256*hi + lo, hi signed int8, lo uint8."""
    q = _c(q, np.int16)
    hi = np.empty(q.shape, dtype=np.int8)
    lo = np.empty(q.shape, dtype=np.uint8)
    _load().oracle_split_planes(_ptr(q), q.size, _ptr(hi), _ptr(lo))
    return hi, lo


# ----------------------------------------------------------------------------------------
# Sec. 2.1 / 2.3: dynamic range -> decimal point
# ----------------------------------------------------------------------------------------
def max_abs(x) -> float:
    x = _c(x, np.float32)
    return float(_load().oracle_max_abs(_ptr(x), x.size))


def int_bits_from_max(m: float, n_bits: int) -> int:
    return int(_load().oracle_int_bits_from_max(ctypes.c_float(m), n_bits))


def measure_range(x, n_bits: int):
    """Returns (max_abs, m, frac_bits) with frac_bits = n-1-m."""
    M = max_abs(x)
    m = int_bits_from_max(M, n_bits)
    return M, m, n_bits - 1 - m


def int_bits_from_acc(max_abs_acc: int, acc_frac_bits: int, n_bits: int) -> int:
    return int(_load().oracle_int_bits_from_acc(int(max_abs_acc), acc_frac_bits, n_bits))


# ----------------------------------------------------------------------------------------
# Sec. 2: LPConvolution / LPInnerProduct accumulators, epilogue, pooling
# ----------------------------------------------------------------------------------------
def conv_acc(xq, wq, pad=(0, 0), stride=(1, 1)) -> np.ndarray:
    xq = _c(xq, np.int16)
    wq = _c(wq, np.int16)
    N, H, W, C = xq.shape
    K, R, S, C2 = wq.shape
    assert C == C2
    OH = (H + 2 * pad[0] - R) // stride[0] + 1
    OW = (W + 2 * pad[1] - S) // stride[1] + 1
    acc = np.empty((N, OH, OW, K), dtype=np.int64)
    _load().oracle_conv_acc(_ptr(xq), _ptr(wq), N, H, W, C, K, R, S, pad[0], pad[1],
                            stride[0], stride[1], _ptr(acc))
    return acc


def conv_acc_at(xq, wq, pad, stride, n, oh, ow, k) -> int:
    xq = _c(xq, np.int16)
    wq = _c(wq, np.int16)
    N, H, W, C = xq.shape
    K, R, S, _ = wq.shape
    return int(_load().oracle_conv_acc_at(_ptr(xq), _ptr(wq), N, H, W, C, K, R, S, pad[0], pad[1],
                                          stride[0], stride[1], n, oh, ow, k))


def ip_acc(xq, wq) -> np.ndarray:
    xq = _c(xq, np.int16)
    wq = _c(wq, np.int16)
    B, K = xq.shape
    O, K2 = wq.shape
    assert K == K2
    acc = np.empty((B, O), dtype=np.int64)
    _load().oracle_ip_acc(_ptr(xq), _ptr(wq), B, K, O, _ptr(acc))
    return acc


def shift_round(v: int, s: int) -> int:
    return int(_load().oracle_shift_round(int(v), int(s)))


def epilogue(acc, bias_q, bias_frac_bits: int, acc_frac_bits: int, relu: bool,
             out_n_bits: int, out_frac_bits: int):
    """Bias + ReLU + requantize (+counters) of an accumulator tensor [..., channels]."""
    _check_fmt(out_n_bits, out_frac_bits)
    acc = _c(acc, np.int64)
    ch = acc.shape[-1]
    outer = acc.size // ch
    y = np.empty(acc.shape, dtype=np.int16)
    cnt = np.zeros(3, dtype=np.uint64)
    b = None if bias_q is None else _c(bias_q, np.int16)
    if b is not None:
        assert b.size == ch and bias_frac_bits <= acc_frac_bits
    _load().oracle_epilogue(_ptr(acc), outer, ch, None if b is None else _ptr(b), bias_frac_bits,
                            acc_frac_bits, int(relu), out_n_bits, out_frac_bits, _ptr(y), _ptr(cnt))
    return y, _counters_out(cnt)


def epilogue_range(acc, bias_q, bias_frac_bits: int, acc_frac_bits: int, relu: bool) -> int:
    acc = _c(acc, np.int64)
    ch = acc.shape[-1]
    b = None if bias_q is None else _c(bias_q, np.int16)
    return int(_load().oracle_epilogue_range(_ptr(acc), acc.size // ch, ch,
                                             None if b is None else _ptr(b), bias_frac_bits,
                                             acc_frac_bits, int(relu)))


def requantize(xq, in_frac_bits: int, relu: bool, out_n_bits: int, out_frac_bits: int):
    xq = _c(xq, np.int16)
    y = np.empty(xq.shape, dtype=np.int16)
    cnt = np.zeros(3, dtype=np.uint64)
    _load().oracle_requantize(_ptr(xq), xq.size, in_frac_bits, int(relu), out_n_bits,
                              out_frac_bits, _ptr(y), _ptr(cnt))
    return y, _counters_out(cnt)


def maxpool2x2(xq) -> np.ndarray:
    xq = _c(xq, np.int16)
    N, H, W, C = xq.shape
    assert H % 2 == 0 and W % 2 == 0
    y = np.empty((N, H // 2, W // 2, C), dtype=np.int16)
    _load().oracle_maxpool2x2(_ptr(xq), N, H, W, C, _ptr(y))
    return y


def _check_fmt(n_bits: int, frac_bits: int):
    if not (1 <= n_bits <= 16 and 0 <= frac_bits <= n_bits - 1):
        raise ValueError(f"bad fixed-point format n={n_bits} f={frac_bits}")


# ----------------------------------------------------------------------------------------
# Layer-level helpers and the network driver (Sec. 2.1 workflow: measure ranges on a
# batch, fix one decimal point per layer, run the low-precision forward pass)
# ----------------------------------------------------------------------------------------
@dataclass
class LayerResult:
    y: np.ndarray            # int16 canonical integers of the layer output
    n_bits: int
    frac_bits: int
    counters: Counters
    max_abs_acc: int         # range of the pre-requantization values (accumulator units)
    acc_frac_bits: int


def lp_layer(acc, fx: int, fw: int, bias_q, bias_frac_bits: int, relu: bool, out_n_bits: int,
             out_frac_bits=None) -> LayerResult:
    """Epilogue of an LP layer; if ``out_frac_bits`` is None the decimal point is chosen from
    the measured range of this very batch (calibration)."""
    F = fx + fw
    A = epilogue_range(acc, bias_q, bias_frac_bits, F, relu)
    if out_frac_bits is None:
        out_frac_bits = out_n_bits - 1 - int_bits_from_acc(A, F, out_n_bits)
    y, cnt = epilogue(acc, bias_q, bias_frac_bits, F, relu, out_n_bits, out_frac_bits)
    return LayerResult(y, out_n_bits, out_frac_bits, cnt, A, F)


def quantize_param(w, n_bits: int):
    """Weights / biases: decimal point from max|w| (Sec. 2.3), then quantize."""
    _, _, f = measure_range(w, n_bits)
    q, _ = quantize(w, n_bits, f)
    return q, f


def _thresholded_fmt(t, n_bits: int, threshold: float) -> int:
    """Fractional bits of an fp32 tensor by the thresholded allocation of Sec. 2.3."""
    from . import bit_allocation as ba
    return ba.choose_frac_bits(ba.bit_histogram(t), n_bits, threshold)


def rounding_seeds(rounding_seed: int, layer_index: int | None):
    """Seeds of the stochastic-rounding draws of one network pass (Sec. 2.4): every tensor that is
    rounded gets its own stream.  Input: base; layer li (counting conv / inner-product layers from 0):
    weights base + 16 li + 1, biases base + 16 li + 2, output base + 16 li + 3, with
    base = rounding_seed * 1000003, all modulo 2^64."""
    base = (int(rounding_seed) * 1000003) & 0xFFFFFFFFFFFFFFFF
    if layer_index is None:
        return base
    return tuple((base + 16 * layer_index + k) & 0xFFFFFFFFFFFFFFFF for k in (1, 2, 3))


def run_network(layers, x, x_fmt, n_bits: int, fixed_formats=None, threshold: float = 0.0,
                rounding_seed: int | None = None):
    """Forward pass of a stack of LP layers on a batch.

    ``rounding_seed`` not None: every LP layer's rounding_scheme is STOCHASTIC (Sec. 2, Sec. 2.4):
    the input, the weights, the biases and every layer output are rounded stochastically with the
    seeds of ``rounding_seeds``; decimal points still come from the measured ranges (of the unrounded
    values), and pooling is unaffected.

    ``threshold`` > 0 (only without ``fixed_formats``): decimal points by the thresholded allocation
    of Sec. 2.3 instead of the maximum: fp32 tensors (input, weights) from their bit-occupancy
    histogram; a layer output is first quantized with the max-based format (nothing clipped), the
    widths of those integers decide how many integer bits may go, and the layer is requantized
    from its exact accumulators with the final format.

    ``layers``: list of dicts, each one of
        {"type": "conv", "w": fp32 [K][R][S][C], "b": fp32 [K], "pad": p, "stride": s, "relu": bool}
        {"type": "ip",   "w": fp32 [O][K], "b": fp32 [O], "relu": bool}
        {"type": "pool"}
    ``x``: fp32 NHWC input; ``x_fmt`` = (n, f) or None to measure it on the batch.
    Weights and biases share the layer's weight format (one BD/AD pair per layer, Sec. 2).
    Returns a list of per-layer records (dicts) including every chosen decimal point.
    """
    records = []
    if x_fmt is None:
        fx = _thresholded_fmt(x, n_bits, threshold) if threshold > 0 else measure_range(x, n_bits)[2]
        nx = n_bits
    else:
        nx, fx = x_fmt
    if rounding_seed is not None:
        from . import stochastic as st
        a, c3 = st.quantize_stochastic(x, nx, fx, rounding_seeds(rounding_seed, None))
        cnt = Counters(*c3)
    else:
        a, cnt = quantize(x, nx, fx)
    records.append({"type": "input", "y": a, "n_bits": nx, "frac_bits": fx, "counters": cnt})
    li = 0
    for L in layers:
        if L["type"] == "pool":
            a = maxpool2x2(a)
            records.append({"type": "pool", "y": a, "n_bits": nx, "frac_bits": fx})
            continue
        if threshold > 0 and fixed_formats is None:
            fw = _thresholded_fmt(L["w"], n_bits, threshold)
            wq, _ = quantize(L["w"], n_bits, fw)
        else:
            wq, fw = quantize_param(L["w"], n_bits)
        bq, _ = quantize(L["b"], n_bits, fw)
        if rounding_seed is not None:
            sw, sb, sy = rounding_seeds(rounding_seed, li)
            wq, _ = st.quantize_stochastic(L["w"], n_bits, fw, sw)
            bq, _ = st.quantize_stochastic(L["b"], n_bits, fw, sb)
        if L["type"] == "conv":
            p, s = L["pad"], L["stride"]
            acc = conv_acc(a, wq, (p, p), (s, s))
        else:
            acc = ip_acc(a.reshape(a.shape[0], -1), wq)
        f_out = None if fixed_formats is None else fixed_formats[li]

        def layer_with(f):
            """Epilogue with the given output decimal point (None: chosen from the measured range),
            rounding as the network's rounding_scheme says."""
            r = lp_layer(acc, fx, fw, bq, fw, L["relu"], n_bits, f)
            if rounding_seed is None:
                return r
            y, c3 = st.epilogue_stochastic(acc, bq, fw, fx + fw, L["relu"], n_bits, r.frac_bits, sy)
            return LayerResult(y, n_bits, r.frac_bits, Counters(*c3), r.max_abs_acc, r.acc_frac_bits)

        res = layer_with(f_out)
        if threshold > 0 and fixed_formats is None:
            from . import bit_allocation as ba
            m = ba.choose_int_bits_from_widths(ba.width_histogram(res.y), res.frac_bits, n_bits, threshold)
            if n_bits - 1 - m != res.frac_bits:
                res = layer_with(n_bits - 1 - m)
        records.append({"type": L["type"], "y": res.y, "n_bits": n_bits, "frac_bits": res.frac_bits,
                        "w_frac_bits": fw, "wq": wq, "bq": bq, "counters": res.counters,
                        "max_abs_acc": res.max_abs_acc, "acc_frac_bits": res.acc_frac_bits})
        a, nx, fx = res.y, n_bits, res.frac_bits
        li += 1
    return records
