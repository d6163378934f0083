"""Time one low-precision layer (or one streaming kernel) in isolation on the current GPU.

    python -m paper_1711_04713_b200.layer_bench conv --N 8 --H 28 --C 512 --K 512 --R 3 --n-bits 16
    python -m paper_1711_04713_b200.layer_bench ip --B 64 --Kin 25088 --O 4096
    python -m paper_1711_04713_b200.layer_bench quantize --numel 268435456
    python -m paper_1711_04713_b200.layer_bench range|act|pool|hist|squantize|params ...

Prints one JSON line with the CUDA-event time per call and the achieved rate (logical TOPS for
the layers, algorithmic GB/s for the streaming kernels).  Inputs are seeded synthetic tensors
(post-ReLU-like activations, He-normal weights).  This is also the small case the ncu captures
under profiles/ are taken on.
"""
from __future__ import annotations

import argparse
import json
import math

import torch

from . import binding as B
from . import build as bld


def _time(fn, iters: int, warmup: int = 3) -> float:
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _quantized(x: torch.Tensor, outer: int, inner: int, n_bits: int, c_stride: int) -> B.QTensor:
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    B.adaption_measure_range(x, n_bits, mx, fmt)
    q = B.QTensor.empty(outer, inner, n_bits, int(fmt.cpu()[1]), c_stride)
    B.adaption_quantize(x, outer, inner, q)
    return q


def _layer_output_format(run, fx: int, fw: int, n_bits: int) -> int:
    st = B.new_stats()
    run(B.MODE_RANGE, None, st)
    s = B.read_stats(st)
    if s.status != 0:
        raise B.AdaptionError(s.status, "range pass")
    return B.adaption_choose_frac_bits_from_acc(int(s.max_abs_acc), fx + fw, n_bits)


def bench_conv(a) -> dict:
    g = torch.Generator(device="cuda").manual_seed(a.seed)
    cs = B.pad_to(a.C, 32)
    x = torch.randn(a.N * a.H * a.H, a.C, device="cuda", generator=g).clamp_(min=0)
    w = torch.randn(a.K * a.R * a.R, a.C, device="cuda", generator=g) * math.sqrt(2.0 / (a.R * a.R * a.C))
    xq = _quantized(x, a.N * a.H * a.H, a.C, a.n_bits, cs)
    wq = _quantized(w, a.K * a.R * a.R, a.C, a.n_bits, cs)
    shp = B.conv_shape(a.N, a.H, a.H, a.C, a.K, a.R, a.R, a.pad, a.stride)
    OH = (a.H + 2 * a.pad - a.R) // a.stride + 1
    need = B.adaption_lp_conv_workspace_bytes(shp, xq.fmt(), wq.fmt(), cs, a.algo)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None

    def run(mode, y, st):
        B.adaption_lp_conv_fwd(shp, xq, wq, None, 0, True, mode, a.algo, y, st, ws)

    f_out = _layer_output_format(run, xq.frac_bits, wq.frac_bits, a.n_bits)
    y = B.QTensor.empty(a.N * OH * OH, a.K, a.n_bits, f_out, B.pad_to(a.K, 32))
    st = B.new_stats()
    ms = _time(lambda: run(B.MODE_REQUANT, y, st), a.iters)
    macs = a.N * OH * OH * a.K * a.R * a.R * a.C
    if B.read_stats(st).status != 0:
        raise B.AdaptionError(B.read_stats(st).status, "conv")
    return {"kind": "conv", "shape": [a.N, a.H, a.H, a.C, a.K, a.R], "n_bits": a.n_bits, "ms": ms,
            "tops": 2.0 * macs / (ms / 1e3) / 1e12, "gmac": macs / 1e9, "workspace_bytes": need}


def bench_ip(a) -> dict:
    g = torch.Generator(device="cuda").manual_seed(a.seed)
    x = torch.randn(a.B, a.Kin, device="cuda", generator=g).clamp_(min=0)
    w = torch.randn(a.O, a.Kin, device="cuda", generator=g) * math.sqrt(2.0 / a.Kin)
    cs = B.pad_to(a.Kin, 16)
    xq = _quantized(x, a.B, a.Kin, a.n_bits, cs)
    wq = _quantized(w, a.O, a.Kin, a.n_bits, cs)
    need = B.adaption_lp_ip_workspace_bytes(a.B, a.Kin, a.O, xq.fmt(), wq.fmt(), a.algo)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None

    def run(mode, y, st):
        B.adaption_lp_ip_fwd(a.B, a.Kin, a.O, xq, wq, None, 0, True, mode, a.algo, y, st, ws)

    f_out = _layer_output_format(run, xq.frac_bits, wq.frac_bits, a.n_bits)
    y = B.QTensor.empty(a.B, a.O, a.n_bits, f_out)
    st = B.new_stats()
    ms = _time(lambda: run(B.MODE_REQUANT, y, st), a.iters)
    macs = a.B * a.Kin * a.O
    bytes_w = a.O * a.Kin * (2 if a.n_bits > 8 else 1)
    return {"kind": "ip", "shape": [a.B, a.Kin, a.O], "n_bits": a.n_bits, "ms": ms,
            "tops": 2.0 * macs / (ms / 1e3) / 1e12, "weight_gbs": bytes_w / (ms / 1e3) / 1e9,
            "workspace_bytes": need}


def bench_stream(a) -> dict:
    g = torch.Generator(device="cuda").manual_seed(a.seed)
    inner = a.inner
    outer = a.numel // inner
    n = outer * inner
    x = torch.randn(outer, inner, device="cuda", generator=g)
    plane_b = 2 if a.n_bits > 8 else 1
    if a.kind == "range":
        mx = torch.zeros(1, dtype=torch.float32, device="cuda")
        fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
        ms = _time(lambda: B.adaption_measure_range(x, a.n_bits, mx, fmt), a.iters)
        bytes_ = 4 * n
    elif a.kind == "hist":
        hist = B.new_hist()
        ms = _time(lambda: B.adaption_bit_histogram(x, hist), a.iters)
        bytes_ = 4 * n
    elif a.kind == "squantize":
        q = B.QTensor.empty(outer, inner, a.n_bits, a.n_bits - 3)
        st = B.new_stats()
        ms = _time(lambda: B.adaption_quantize_stochastic(x, outer, inner, q, 42, False, None, st), a.iters)
        bytes_ = (4 + plane_b) * n
    elif a.kind in ("quantize", "act"):
        q = B.QTensor.empty(outer, inner, a.n_bits, a.n_bits - 3)
        st = B.new_stats()
        if a.kind == "quantize":
            ms = _time(lambda: B.adaption_quantize(x, outer, inner, q, None, B.ROUND_DETERMINISTIC, st), a.iters)
        else:
            ms = _time(lambda: B.adaption_lp_act(x, None, outer, inner, True, q, None, B.ROUND_DETERMINISTIC, st),
                       a.iters)
        bytes_ = (4 + plane_b) * n
    elif a.kind == "requant":
        qin = B.QTensor.empty(outer, inner, a.n_bits, a.n_bits - 3)
        B.adaption_quantize(x, outer, inner, qin)
        q = B.QTensor.empty(outer, inner, a.n_bits, a.n_bits - 5)
        st = B.new_stats()
        ms = _time(lambda: B.adaption_lp_act(None, qin, outer, inner, True, q, None, B.ROUND_DETERMINISTIC, st),
                   a.iters)
        bytes_ = 2 * plane_b * n
    else:  # pool: numel = N*H*W*C with H = W = a.H
        Cc = inner
        N = max(1, n // (a.H * a.H * Cc))
        qin = B.QTensor.empty(N * a.H * a.H, Cc, a.n_bits, 5)
        B.adaption_quantize(x[:N * a.H * a.H], N * a.H * a.H, Cc, qin)
        q = B.QTensor.empty(N * (a.H // 2) ** 2, Cc, a.n_bits, 5)
        ms = _time(lambda: B.adaption_maxpool2x2(qin, N, a.H, a.H, Cc, q), a.iters)
        n = N * a.H * a.H * Cc
        bytes_ = int(plane_b * n * 1.25)
    return {"kind": a.kind, "numel": n, "n_bits": a.n_bits, "ms": ms, "gbs": bytes_ / (ms / 1e3) / 1e9,
            "algorithmic_bytes": bytes_}


def bench_params(a) -> dict:
    """All weight and bias tensors of VGG16 (138 M parameters) quantized with fixed formats, as every
    forward pass does: one adaption_quantize_batch call."""
    from . import workloads as wl
    from .network import LPNetwork
    net = LPNetwork(wl.make_params(wl.vgg16_specs(), seed=a.seed), 1, (224, 224), 3, a.n_bits)
    net.quantize_params(measure=True)
    ms = _time(lambda: net.quantize_params(measure=False), a.iters)
    n = sum(L.w_f32.numel() + L.b_f32.numel() for L in net.layers if L.type in ("conv", "ip"))
    bytes_ = n * (4 + (2 if a.n_bits > 8 else 1))
    return {"kind": "params", "numel": n, "n_bits": a.n_bits, "ms": ms, "gbs": bytes_ / (ms / 1e3) / 1e9,
            "algorithmic_bytes": bytes_, "launches": net.param_quantize_launches()}


def bench_peak(a) -> dict:
    """Back-to-back int8 tensor-core instructions on resident operands (the roofline denominator)."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    out = {"kind": "peak", "iters": a.iters, "sms": sms, "configs": []}
    for pair, bn, ce in [(False, 64, 0), (False, 128, 0), (False, 256, 0), (True, 64, 0), (True, 128, 0),
                         (True, 256, 0), (False, 128, 4), (False, 128, 1), (True, 128, 4), (True, 128, 1)]:
        if True:
            cyc = torch.zeros(max(sms, 148), dtype=torch.int64, device="cuda")
            st = torch.zeros(1, dtype=torch.int32, device="cuda")
            n = 4096

            def run():
                B.adaption_probe_i8_peak(bn, pair, n, cyc, st, ce)

            ms = _time(run, max(a.iters, 3))
            if int(st.cpu()[0]) != 0:
                raise B.AdaptionError(int(st.cpu()[0]), "peak probe")
            c = cyc.cpu()
            issuing = c[c > 0].double()
            units = sms // 2 if pair else sms
            macs = units * 4 * n * (256 if pair else 128) * bn * 32
            out["configs"].append({"pair": pair, "bn": bn, "commit_every": ce, "cycles_per_mma": float(issuing.mean()) / (4 * n),
                                   "int8_tops": 2.0 * macs / (ms / 1e3) / 1e12, "ms": ms})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["conv", "ip", "range", "quantize", "act", "requant", "pool", "peak", "hist", "squantize", "params"])
    ap.add_argument("--N", type=int, default=8)
    ap.add_argument("--H", type=int, default=28)
    ap.add_argument("--C", type=int, default=512)
    ap.add_argument("--K", type=int, default=512)
    ap.add_argument("--R", type=int, default=3)
    ap.add_argument("--pad", type=int, default=1)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--Kin", type=int, default=25088)
    ap.add_argument("--O", type=int, default=4096)
    ap.add_argument("--numel", type=int, default=1 << 28)
    ap.add_argument("--inner", type=int, default=256)
    ap.add_argument("--n-bits", type=int, default=16)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--algo", type=int, default=B.ALGO_AUTO)
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("layer_bench needs a CUDA device")
    bld.build_library()
    B.load()
    if a.kind == "conv":
        out = bench_conv(a)
    elif a.kind == "ip":
        out = bench_ip(a)
    elif a.kind == "peak":
        out = bench_peak(a)
    elif a.kind == "params":
        out = bench_params(a)
    else:
        out = bench_stream(a)
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
