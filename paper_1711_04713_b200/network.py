"""Host-side orchestration of a stack of low-precision layers on one GPU.

Only sequencing, buffer ownership and format bookkeeping live here; every step of the path
(range measurement, quantization, convolution / inner product with fused bias + ReLU +
requantization, pooling) is a call into the CUDA library through ``binding``.

Workflow (paper Sec. 2.1): ``calibrate`` runs a batch through the stack and fixes one decimal
point per layer from the measured ranges; ``forward`` then runs with those fixed formats and
never synchronises with the host.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import binding as B
from . import replicas


def calibration_loop(be, kinds: list[str], threshold: float = 0.0, group=None, device="cpu"):
    """The calibration workflow of paper Sec. 2.1 / 2.3 as host logic over a backend `be` that runs the
    layers (the CUDA library for LPNetwork; anything with the same methods in tests): measure the
    input's range, quantize it, then per layer a RANGE pass, the decimal point from the measured
    range, a REQUANT pass (and, with `threshold` > 0, the width histogram of that output and a second
    REQUANT pass if integer bits can go).  With a process group every range, histogram and counter
    is reduced over the replicas, so that all of them fix the same decimal points (each replica holds
    its own shard of the batch, the weights are replicated).  Returns the per-layer records."""
    rec = []
    fx = be.input_frac_bits(threshold, group)
    rec.append({"type": "input", "frac_bits": fx, "stats": be.quantize_input(fx)})
    for i, kind in enumerate(kinds):
        if kind == "pool":
            rec.append({"type": "pool", "frac_bits": be.pool(i)})
            continue
        local = int(be.range_pass(i))
        A = replicas.agree_on_range(local, device, group)
        F = be.acc_frac_bits(i)
        f = be.choose_from_acc(A, F)
        st = be.requant_pass(i, f)
        if threshold > 0:
            hist = replicas.sum_histogram(be.width_histogram(i), device, group)
            f2 = be.choose_from_widths(hist, f, threshold)
            if f2 != f:
                f = f2
                st = be.requant_pass(i, f)
        totals = replicas.sum_counters(int(st.zeros), int(st.sat_pos), int(st.sat_neg), device, group)
        rec.append({"type": kind, "name": be.layer_name(i), "frac_bits": f, "w_frac_bits": be.w_frac_bits(i),
                    "max_abs_acc": A, "local_max_abs_acc": local, "acc_frac_bits": F, "stats": st,
                    "counters_all_replicas": totals})
    return rec


def rounding_seeds(rounding_seed: int, layer_index: int | None):
    """Seeds of the stochastic-rounding draws of one pass: input = base; layer li (conv / inner-product
    layers counted from 0): weights base + 16 li + 1, biases + 2, output + 3; base = rounding_seed *
    1000003; all modulo 2^64."""
    base = (int(rounding_seed) * 1000003) & 0xFFFFFFFFFFFFFFFF
    if layer_index is None:
        return base
    return tuple((base + 16 * layer_index + k) & 0xFFFFFFFFFFFFFFFF for k in (1, 2, 3))


def act_c_stride(c: int) -> int:
    """Channel pitch of activation / weight planes: a multiple of 32 so that every layer can take
    the tensor-core path."""
    return B.pad_to(c, 32)


@dataclass
class _Layer:
    type: str
    name: str = ""
    relu: bool = True
    # geometry
    N: int = 0
    H: int = 0
    W: int = 0
    C: int = 0
    K: int = 0
    R: int = 0
    pad: int = 0
    stride: int = 1
    OH: int = 0
    OW: int = 0
    ip_k: int = 0            # reduction length of an inner product (padded flatten)
    # buffers
    w_f32: torch.Tensor | None = None
    b_f32: torch.Tensor | None = None
    w: B.QTensor | None = None
    b: B.QTensor | None = None
    w_fmt_dev: torch.Tensor | None = None
    w_max_dev: torch.Tensor | None = None
    y: B.QTensor | None = None
    stats: torch.Tensor | None = None
    workspace: torch.Tensor | None = None
    shape: object = None
    macs: int = 0
    extra: dict = field(default_factory=dict)


class LPNetwork:
    def __init__(self, params: list[dict], batch: int, in_hw: tuple[int, int], in_c: int, n_bits: int,
                 algo: int = B.ALGO_AUTO, keep_q16: bool = False, device="cuda", fuse_pool: bool = True,
                 rounding_seed: int | None = None):
        """``rounding_seed`` not None: rounding_scheme STOCHASTIC for every layer (paper Sec. 2, 2.4): the
        input, weights, biases and layer outputs are rounded stochastically, each tensor with its own
        seed (see ``rounding_seeds``); decimal points still come from the measured ranges."""
        self.rounding_seed = rounding_seed
        self.n_bits = n_bits
        self.fuse_pool = fuse_pool
        self.algo = algo
        self.device = device
        self.batch = batch
        self.in_h, self.in_w = in_hw
        self.in_c = in_c
        self.keep_q16 = keep_q16
        self.layers: list[_Layer] = []
        self.calibrated = False
        self.launches_per_forward = 0

        self.x_fmt_dev = torch.zeros(2, dtype=torch.int32, device=device)
        self.x_max_dev = torch.zeros(1, dtype=torch.float32, device=device)
        self.x_stats = B.new_stats(device)
        # A first convolution with few input channels gathers its taps into packed rows inside the
        # library (it needs no 32-byte pitch), so the network input keeps the smallest pitch.
        first = params[0] if params else None
        few = (first is not None and first["type"] == "conv" and in_c <= 4
               and first["w"].shape[1] * first["w"].shape[2] * in_c <= 32)
        in_cs = B.pad_to(in_c, 16) if few else act_c_stride(in_c)
        self.xq = B.QTensor.empty(batch * self.in_h * self.in_w, in_c, n_bits, 0, in_cs, keep_q16, device)
        h, w, c, cs = self.in_h, self.in_w, in_c, self.xq.c_stride
        flat = False
        for p in params:
            L = _Layer(p["type"], p.get("name", ""))
            if p["type"] == "pool":
                L.N, L.H, L.W, L.C = batch, h, w, c
                h, w = h // 2, w // 2
                L.y = B.QTensor.empty(batch * h * w, c, n_bits, 0, cs, keep_q16, device)
            elif p["type"] == "conv":
                K, R, S, Cin = p["w"].shape
                assert Cin == c and R == S and not flat
                L.N, L.H, L.W, L.C, L.K, L.R = batch, h, w, c, K, R
                L.pad, L.stride, L.relu = p["pad"], p["stride"], p["relu"]
                L.OH = (h + 2 * L.pad - R) // L.stride + 1
                L.OW = (w + 2 * L.pad - S) // L.stride + 1
                L.shape = B.conv_shape(batch, h, w, c, K, R, S, L.pad, L.stride)
                L.w_f32 = torch.from_numpy(np.ascontiguousarray(p["w"])).to(device)
                L.w = B.QTensor.empty(K * R * S, c, n_bits, 0, cs, False, device)
                L.macs = batch * L.OH * L.OW * K * R * S * c
                h, w, c = L.OH, L.OW, K
                cs = act_c_stride(K)
                L.y = B.QTensor.empty(batch * h * w, K, n_bits, 0, cs, keep_q16, device)
            elif p["type"] == "ip":
                O, Kin = p["w"].shape
                L.relu = p["relu"]
                if not flat:
                    assert Kin == h * w * c
                    # weights follow the padded NHWC flatten of the previous activation
                    L.ip_k = h * w * cs
                    wsrc = np.ascontiguousarray(p["w"]).reshape(O * h * w, c)
                    L.w = B.QTensor.empty(O * h * w, c, n_bits, 0, cs, False, device)
                    L.extra["w_view"] = (O, L.ip_k)
                    flat = True
                else:
                    assert Kin == c
                    L.ip_k = cs
                    wsrc = np.ascontiguousarray(p["w"])
                    L.w = B.QTensor.empty(O, c, n_bits, 0, cs, False, device)
                    L.extra["w_view"] = (O, cs)
                L.w_f32 = torch.from_numpy(wsrc).to(device)
                L.N, L.C, L.K = batch, Kin, O
                L.macs = batch * Kin * O
                h, w, c = 1, 1, O
                cs = B.pad_to(O, 16)
                L.y = B.QTensor.empty(batch, O, n_bits, 0, cs, keep_q16, device)
            else:
                raise ValueError(p["type"])
            if L.type in ("conv", "ip"):
                L.b_f32 = torch.from_numpy(np.ascontiguousarray(p["b"])).to(device)
                L.b = B.QTensor.empty(1, L.K, n_bits, 0, None, True, device)
                L.w_fmt_dev = torch.zeros(2, dtype=torch.int32, device=device)
                L.w_max_dev = torch.zeros(1, dtype=torch.float32, device=device)
                L.stats = B.new_stats(device)
            self.layers.append(L)
        self.total_macs = sum(L.macs for L in self.layers)

    # ------------------------------------------------------------------ parameters
    def _fp32_fmt_by_threshold(self, t: torch.Tensor, threshold: float) -> int:
        """Fractional bits of an fp32 device tensor by the thresholded allocation (Sec. 2.3)."""
        hist = B.new_hist(self.device)
        B.adaption_bit_histogram(t, hist)
        return B.adaption_choose_frac_bits_from_hist(hist.cpu().tolist(), self.n_bits, threshold)

    def quantize_params(self, measure: bool = True, threshold: float = 0.0):
        """Weights and biases -> fixed point (paper Sec. 2.1: quantized in the forward pass).  With
        ``measure`` the decimal point of each layer's weights is taken from max|w| on the device, or,
        with ``threshold`` > 0, from the thresholded allocation of Sec. 2.3."""
        if self.rounding_seed is not None:
            return self._quantize_params_stochastic(measure, threshold)
        if not measure:
            # fixed formats: every weight and bias tensor of the network in one library call
            entries = []
            for L in self.layers:
                if L.type in ("conv", "ip"):
                    entries.append((L.w_f32, L.w.outer, L.w.inner, L.w, None))
                    entries.append((L.b_f32, 1, L.K, L.b, None))
            B.adaption_quantize_batch(B.quantize_items(entries))
            return
        for L in self.layers:
            if L.type not in ("conv", "ip"):
                continue
            if measure and threshold > 0:
                L.w.frac_bits = L.b.frac_bits = self._fp32_fmt_by_threshold(L.w_f32, threshold)
                L.w_fmt_dev.copy_(torch.tensor([self.n_bits, L.w.frac_bits], dtype=torch.int32))
                B.adaption_quantize(L.w_f32, L.w.outer, L.w.inner, L.w)
                B.adaption_quantize(L.b_f32, 1, L.K, L.b)
            elif measure:
                L.w_max_dev.zero_()
                B.adaption_measure_range(L.w_f32, self.n_bits, L.w_max_dev, L.w_fmt_dev)
                B.adaption_quantize(L.w_f32, L.w.outer, L.w.inner, L.w, L.w_fmt_dev)
                B.adaption_quantize(L.b_f32, 1, L.K, L.b, L.w_fmt_dev)
        for L in self.layers:
            if L.type in ("conv", "ip"):
                f = int(L.w_fmt_dev.cpu()[1])
                L.w.frac_bits = f
                L.b.frac_bits = f

    def _quantize_params_stochastic(self, measure: bool, threshold: float):
        """Weights and biases with rounding_scheme STOCHASTIC: formats as in the deterministic case
        (from max|w| or the thresholded allocation), values by the stochastic quantizer."""
        li = 0
        for L in self.layers:
            if L.type not in ("conv", "ip"):
                continue
            if measure and threshold > 0:
                L.w.frac_bits = L.b.frac_bits = self._fp32_fmt_by_threshold(L.w_f32, threshold)
            elif measure:
                L.w_max_dev.zero_()
                B.adaption_measure_range(L.w_f32, self.n_bits, L.w_max_dev, L.w_fmt_dev)
                L.w.frac_bits = L.b.frac_bits = int(L.w_fmt_dev.cpu()[1])
            sw, sb, _ = rounding_seeds(self.rounding_seed, li)
            B.adaption_quantize_stochastic(L.w_f32, L.w.outer, L.w.inner, L.w, sw)
            B.adaption_quantize_stochastic(L.b_f32, 1, L.K, L.b, sb)
            L.extra["li"] = li
            li += 1

    @staticmethod
    def helper_launches(L: _Layer) -> int:
        """Launches beside the layer's own kernel when it runs with a workspace: the tap packing of a
        first layer with at most 4 channels (activations, weights), else the split-K finalize."""
        if L.workspace is None:
            return 0
        return 2 if L.type == "conv" and L.C <= 4 else 1

    def param_quantize_launches(self) -> int:
        """Kernel launches of one quantize_params(measure=False): dense tensors share one launch per
        40, a tensor with padded rows takes one of its own."""
        dense = padded = 0
        for L in self.layers:
            if L.type in ("conv", "ip"):
                for q in (L.w, L.b):
                    if q.inner == q.c_stride:
                        dense += 1
                    else:
                        padded += 1
        return (dense + 39) // 40 + padded

    # ------------------------------------------------------------------ one layer
    def _workspace(self, L: _Layer, x: B.QTensor) -> torch.Tensor | None:
        if L.type == "conv":
            need = B.adaption_lp_conv_workspace_bytes(L.shape, x.fmt(), L.w.fmt(), x.c_stride, self.algo)
        else:
            need = B.adaption_lp_ip_workspace_bytes(L.N, L.ip_k, L.K, x.fmt(), L.w.fmt(), self.algo)
        if need == 0:
            return None
        if L.workspace is None or L.workspace.numel() < need:
            L.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        return L.workspace

    def fused_pool_after(self, i: int) -> bool:
        """True where layer i is a convolution whose output only feeds the 2x2 max-pool after it, so
        that inference may run the pair as one library call (the convolution's own output is then not
        materialised in ``layers[i].y``)."""
        if not self.fuse_pool or self.keep_q16 or i + 1 >= len(self.layers) or self.rounding_seed is not None:
            return False
        L, P = self.layers[i], self.layers[i + 1]
        return L.type == "conv" and P.type == "pool" and L.OH % 2 == 0 and L.OW % 2 == 0

    def _run_conv_pool(self, L: _Layer, P: _Layer, x: B.QTensor, phases: int = 3) -> B.QTensor:
        P.y.frac_bits = L.y.frac_bits
        need = B.adaption_lp_conv_pool_workspace_bytes(L.shape, x.fmt(), L.w.fmt(), P.y.fmt(), x.c_stride,
                                                       P.y.c_stride, self.algo)
        if P.workspace is None or P.workspace.numel() < need:
            P.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        B.adaption_lp_conv_pool_fwd(L.shape, x, L.w, L.b.q16, L.b.frac_bits, L.relu, self.algo, P.y, L.stats,
                                    P.workspace, phases)
        return P.y

    def _run_layer(self, L: _Layer, x: B.QTensor, mode: int) -> B.QTensor:
        if L.type == "pool":
            L.y.frac_bits = x.frac_bits
            B.adaption_maxpool2x2(x, L.N, L.H, L.W, L.C, L.y)
            return L.y
        ws = self._workspace(L, x)
        y = L.y if mode == B.MODE_REQUANT else None
        stochastic = self.rounding_seed is not None and mode == B.MODE_REQUANT
        seed_y = rounding_seeds(self.rounding_seed, L.extra["li"])[2] if stochastic else 0
        if L.type == "conv":
            if stochastic:
                B.adaption_lp_conv_fwd_stochastic(L.shape, x, L.w, L.b.q16, L.b.frac_bits, L.relu, self.algo, y,
                                                  seed_y, L.stats, ws)
            else:
                B.adaption_lp_conv_fwd(L.shape, x, L.w, L.b.q16, L.b.frac_bits, L.relu, mode, self.algo, y,
                                       L.stats, ws)
        else:
            xin = x.reshaped(L.N, L.ip_k, L.ip_k)
            O, kp = L.extra["w_view"]
            win = L.w.reshaped(O, kp, kp)
            if stochastic:
                B.adaption_lp_ip_fwd_stochastic(L.N, L.ip_k, L.K, xin, win, L.b.q16, L.b.frac_bits, L.relu,
                                                self.algo, y, seed_y, L.stats, ws)
            else:
                B.adaption_lp_ip_fwd(L.N, L.ip_k, L.K, xin, win, L.b.q16, L.b.frac_bits, L.relu, mode,
                                     self.algo, y, L.stats, ws)
        return L.y

    # ------------------------------------------------------------------ calibration
    def calibrate(self, x_f32: torch.Tensor, x_fmt: tuple[int, int] | None = None, threshold: float = 0.0,
                  group=None):
        """Run one batch layer by layer, measuring each layer's range on it and fixing its decimal
        point (paper Sec. 2.1, 2.3).  Returns the per-layer records (formats, counters, ranges).
        ``threshold`` > 0: thresholded allocation of the integer bits instead of the maximum (fp32
        tensors from their bit-occupancy histogram; a layer output is first stored with the
        max-based format, the widths of those integers decide, then the layer is run again).
        ``group`` (or an initialised default process group): data-parallel replicas, each calibrating
        on its own shard of the batch, agree on every decimal point (see ``calibration_loop``)."""
        self.quantize_params(measure=True, threshold=threshold)
        self._cal_x, self._cal_x_fmt, self._cal_in = x_f32, x_fmt, {}
        try:
            rec = calibration_loop(self, [L.type for L in self.layers], threshold, group, self.device)
        finally:
            self._cal_x, self._cal_in = None, {}
        self.calibrated = True
        return rec

    # ---- backend of calibration_loop: every method is one or two library calls
    def input_frac_bits(self, threshold: float, group) -> int:
        x = self._cal_x
        if self._cal_x_fmt is not None:
            assert self._cal_x_fmt[0] == self.n_bits
            return self._cal_x_fmt[1]
        if threshold > 0:
            hist = B.new_hist(self.device)
            B.adaption_bit_histogram(x, hist)
            total = replicas.sum_histogram(hist.cpu().tolist(), self.device, group)
            return B.adaption_choose_frac_bits_from_hist(total, self.n_bits, threshold)
        self.x_max_dev.zero_()
        B.adaption_measure_range(x, self.n_bits, self.x_max_dev, self.x_fmt_dev)
        local = float(self.x_max_dev.cpu()[0])
        agreed = replicas.largest_float(local, self.device, group)
        if agreed != local:
            # fold the replicas' maximum in and let the library derive the format from it
            self.x_max_dev.fill_(agreed)
            B.adaption_measure_range(x[:0], self.n_bits, self.x_max_dev, self.x_fmt_dev)
        return int(self.x_fmt_dev.cpu()[1])

    def quantize_input(self, frac_bits: int):
        self.x_stats.zero_()
        self.xq.frac_bits = frac_bits
        self._quantize_input(self._cal_x)
        self._cal_act = self.xq
        return B.read_stats(self.x_stats)

    def pool(self, i: int) -> int:
        self._cal_act = self._run_layer(self.layers[i], self._cal_act, B.MODE_REQUANT)
        return self._cal_act.frac_bits

    def range_pass(self, i: int) -> int:
        L = self.layers[i]
        L.stats.zero_()
        self._cal_in[i] = self._cal_act
        self._run_layer(L, self._cal_act, B.MODE_RANGE)
        st = B.read_stats(L.stats)
        if st.status != 0:
            raise B.AdaptionError(st.status, f"layer {L.name} (range)")
        return int(st.max_abs_acc)

    def acc_frac_bits(self, i: int) -> int:
        return self._cal_in[i].frac_bits + self.layers[i].w.frac_bits

    def choose_from_acc(self, max_abs_acc: int, acc_frac_bits: int) -> int:
        return B.adaption_choose_frac_bits_from_acc(max_abs_acc, acc_frac_bits, self.n_bits)

    def requant_pass(self, i: int, frac_bits: int):
        L = self.layers[i]
        L.y.frac_bits = frac_bits
        L.stats.zero_()
        self._cal_act = self._run_layer(L, self._cal_in[i], B.MODE_REQUANT)
        st = B.read_stats(L.stats)
        if st.status != 0:
            raise B.AdaptionError(st.status, f"layer {L.name}")
        return st

    def width_histogram(self, i: int) -> list[int]:
        hist = B.new_hist(self.device)
        B.adaption_width_histogram(self.layers[i].y, hist)
        return hist.cpu().tolist()

    def choose_from_widths(self, hist: list[int], frac_bits: int, threshold: float) -> int:
        return B.adaption_choose_frac_bits_from_widths(hist, frac_bits, self.n_bits, threshold)

    def layer_name(self, i: int) -> str:
        return self.layers[i].name

    def w_frac_bits(self, i: int) -> int:
        return self.layers[i].w.frac_bits

    def set_formats(self, x_frac_bits: int, layer_frac_bits: list[int]):
        """Fix the decimal points without a calibration run (formats chosen elsewhere, e.g. on another
        batch): ``x_frac_bits`` for the network input, one entry per conv / inner-product layer for
        its output.  Weight formats still come from max|w| on the device."""
        self.quantize_params(measure=True)
        self.xq.frac_bits = x_frac_bits
        it = iter(layer_frac_bits)
        for L in self.layers:
            if L.type in ("conv", "ip"):
                L.y.frac_bits = int(next(it))
        self.calibrated = True

    def _quantize_input(self, x_f32: torch.Tensor):
        if self.rounding_seed is not None:
            B.adaption_quantize_stochastic(x_f32, self.xq.outer, self.xq.inner, self.xq,
                                           rounding_seeds(self.rounding_seed, None), False, None, self.x_stats)
        else:
            B.adaption_quantize(x_f32, self.xq.outer, self.xq.inner, self.xq, None, B.ROUND_DETERMINISTIC,
                                self.x_stats)

    # ------------------------------------------------------------------ inference
    def forward(self, x_f32: torch.Tensor, requantize_params: bool = True, measure_input: bool = True):
        """One forward pass with the calibrated formats; enqueues work only (no host sync).
        Returns the output QTensor and the number of kernel launches issued."""
        assert self.calibrated
        launches = 0
        if measure_input:
            # range of the incoming batch (monitoring; the calibrated input format stays in force)
            B.adaption_measure_range(x_f32, self.n_bits, self.x_max_dev, self.x_fmt_dev)
            launches += 2
        self._quantize_input(x_f32)
        launches += 1
        if requantize_params:
            self.quantize_params(measure=False)
            launches += self.param_quantize_launches()
        a = self.xq
        i = 0
        while i < len(self.layers):
            L = self.layers[i]
            if self.fused_pool_after(i):
                a = self._run_conv_pool(L, self.layers[i + 1], a)
                launches += 1
                i += 1
            else:
                a = self._run_layer(L, a, B.MODE_REQUANT)
            launches += 1
            if L.workspace is not None and L.type != "pool":
                launches += self.helper_launches(L)
            i += 1
        self.launches_per_forward = launches
        return a, launches

    def zero_stats(self):
        self.x_stats.zero_()
        for L in self.layers:
            if L.stats is not None:
                L.stats.zero_()

    def layer_stats(self):
        out = []
        for L in self.layers:
            if L.stats is not None:
                st = B.read_stats(L.stats)
                total = L.y.outer * L.y.inner
                out.append({"name": L.name, "zeros": int(st.zeros), "sat_pos": int(st.sat_pos),
                            "sat_neg": int(st.sat_neg), "total": total, "status": int(st.status),
                            "frac_bits": L.y.frac_bits})
        return out
