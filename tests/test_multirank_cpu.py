"""Replica bookkeeping with two gloo ranks on CPU: all replicas must end up with the same per-layer
decimal point (max-reduced range), counters add up, and the step time is the slowest rank's."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import reference as orc
from paper_1711_04713_b200 import binding as B
from paper_1711_04713_b200 import build
from paper_1711_04713_b200 import replicas
from paper_1711_04713_b200 import workloads as wl


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank: its own shard of images, shared weights
        x = wl.relu_normal((2, 6, 6, 8), seed=replicas.shard_seed(100, rank)) * (1.0 + 3.0 * rank)
        w = wl.he_conv_weight(4, 3, 3, 8, seed=7)
        fx = 10
        xq, _ = orc.quantize(x, 16, fx)
        wq, fw = orc.quantize_param(w, 16)
        acc = orc.conv_acc(xq, wq, (1, 1))
        local_range = orc.epilogue_range(acc, None, 0, fx + fw, True)
        agreed = replicas.agree_on_range(local_range)
        f_out = B.adaption_choose_frac_bits_from_acc(agreed, fx + fw, 16)
        y, cnt = orc.epilogue(acc, None, 0, fx + fw, True, 16, f_out)
        z, sp, sn = replicas.sum_counters(cnt.zeros, cnt.sat_pos, cnt.sat_neg)
        slow = replicas.slowest_rank_ms(10.0 + rank)
        np.save(os.path.join(out_dir, f"r{rank}.npy"),
                np.array([local_range, agreed, f_out, cnt.zeros, z, sp, sn, int(slow * 1000)], dtype=np.int64))
    finally:
        dist.destroy_process_group()


def test_two_replicas_agree_on_formats_and_counters(tmp_path):
    build.build_library()           # the host helper lives in the library; no GPU needed
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(world))
    assert r0[0] != r1[0]                                   # shards have different ranges ...
    assert r0[1] == r1[1] == max(r0[0], r1[0])              # ... but agree on the larger one
    assert r0[2] == r1[2]                                   # hence on the same decimal point
    assert r0[4] == r1[4] == r0[3] + r1[3]                  # zero counts add up
    assert r0[5] == r1[5] == 0 and r0[6] == r1[6] == 0      # nothing saturates at the agreed format
    assert r0[7] == r1[7] == 11000                          # the slowest replica defines the step
    assert replicas.whole_job_rate(64, 2, 5.0) == 25600.0


class _OracleBackend:
    """The calibration backend protocol of network.calibration_loop with the CPU oracle standing in
    for the CUDA library: lets the replica logic run on CPU ranks."""

    def __init__(self, params, x, n_bits):
        from types import SimpleNamespace
        self.ns = SimpleNamespace
        self.params, self.x, self.n = params, x, n_bits
        self.outputs = []

    def input_frac_bits(self, threshold, group):
        from oracle import bit_allocation as ba
        if threshold > 0:
            return ba.choose_frac_bits(replicas.sum_histogram(ba.bit_histogram(self.x), "cpu", group), self.n, threshold)
        m = replicas.largest_float(orc.max_abs(self.x), "cpu", group)
        return self.n - 1 - orc.int_bits_from_max(m, self.n)

    def quantize_input(self, fx):
        self.a, cnt = orc.quantize(self.x, self.n, fx)
        self.fx = fx
        self.outputs.append(self.a)
        return self.ns(zeros=cnt.zeros, sat_pos=cnt.sat_pos, sat_neg=cnt.sat_neg)

    def pool(self, i):
        self.a = orc.maxpool2x2(self.a)
        self.outputs.append(self.a)
        return self.fx

    def range_pass(self, i):
        L = self.params[i]
        self.threshold_w = getattr(self, "threshold_w", 0.0)
        if self.threshold_w > 0:
            from oracle import bit_allocation as ba
            self.fw = ba.choose_frac_bits(ba.bit_histogram(L["w"]), self.n, self.threshold_w)
            self.wq, _ = orc.quantize(L["w"], self.n, self.fw)
        else:
            self.wq, self.fw = orc.quantize_param(L["w"], self.n)
        self.bq, _ = orc.quantize(L["b"], self.n, self.fw)
        if L["type"] == "conv":
            self.acc = orc.conv_acc(self.a, self.wq, (L["pad"], L["pad"]), (L["stride"], L["stride"]))
        else:
            self.acc = orc.ip_acc(self.a.reshape(self.a.shape[0], -1), self.wq)
        self.F = self.fx + self.fw
        return orc.epilogue_range(self.acc, self.bq, self.fw, self.F, L["relu"])

    def acc_frac_bits(self, i):
        return self.F

    def choose_from_acc(self, A, F):
        return self.n - 1 - orc.int_bits_from_acc(A, F, self.n)

    def requant_pass(self, i, f):
        y, cnt = orc.epilogue(self.acc, self.bq, self.fw, self.F, self.params[i]["relu"], self.n, f)
        self.y, self.y_f = y, f
        self.pending = (y, f)
        return self.ns(zeros=cnt.zeros, sat_pos=cnt.sat_pos, sat_neg=cnt.sat_neg)

    def width_histogram(self, i):
        from oracle import bit_allocation as ba
        return ba.width_histogram(self.y).tolist()

    def choose_from_widths(self, hist, f, threshold):
        from oracle import bit_allocation as ba
        return self.n - 1 - ba.choose_int_bits_from_widths(hist, f, self.n, threshold)

    def layer_name(self, i):
        return self.params[i].get("name", str(i))

    def w_frac_bits(self, i):
        self.a, self.fx = self.y, self.y_f          # called last for a layer: its output feeds the next one
        self.outputs.append(self.a)
        return self.fw


def _small_stack():
    specs = [wl.LayerSpec("conv", "c1", 3, 8, 3, 1, 1, True), wl.LayerSpec("pool", "p1"),
             wl.LayerSpec("conv", "c2", 8, 12, 3, 1, 1, True), wl.LayerSpec("ip", "f1", 4 * 4 * 12, 10, relu=False)]
    return wl.make_params(specs, seed=9)


def _calibration_rank(rank: int, world: int, port: int, out_dir: str, threshold: float):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_1711_04713_b200.network import calibration_loop
        params = _small_stack()
        x = wl.vgg16_input(4, seed=9, hw=8)
        x[2:] *= 3.0                                   # the second shard has the larger ranges
        be = _OracleBackend(params, x[2 * rank:2 * rank + 2], 16)
        be.threshold_w = threshold
        rec = calibration_loop(be, [p["type"] for p in params], threshold, None, "cpu")
        np.save(os.path.join(out_dir, f"fmt{rank}.npy"), np.array([r["frac_bits"] for r in rec], dtype=np.int64))
        np.save(os.path.join(out_dir, f"cnt{rank}.npy"),
                np.array([r["counters_all_replicas"] for r in rec if "counters_all_replicas" in r], dtype=np.int64))
        np.save(os.path.join(out_dir, f"out{rank}.npy"), be.outputs[-1])
    finally:
        dist.destroy_process_group()


def test_two_replicas_calibrate_like_one_process_on_the_whole_batch(tmp_path):
    """The calibration loop LPNetwork.calibrate runs, driven by two gloo ranks that each hold half of
    the batch (the oracle stands in for the layer calls): both end with the same decimal points, and
    these, the summed counters and each rank's outputs are those of one calibration of the whole
    batch, with the maximum-based rule and with the thresholded allocation."""
    build.build_library()
    params = _small_stack()
    x = wl.vgg16_input(4, seed=9, hw=8)
    x[2:] *= 3.0
    for threshold in (0.0, 0.02):
        d = tmp_path / f"t{threshold}"
        d.mkdir()
        mp.spawn(_calibration_rank, args=(2, _free_port(), str(d), threshold), nprocs=2, join=True)
        whole = orc.run_network(params, x, None, 16, threshold=threshold)
        f0, f1 = np.load(d / "fmt0.npy"), np.load(d / "fmt1.npy")
        assert f0.tolist() == f1.tolist() == [r["frac_bits"] for r in whole]
        want_cnt = [[r["counters"].zeros, r["counters"].sat_pos, r["counters"].sat_neg]
                    for r in whole if r["type"] in ("conv", "ip")]
        assert np.load(d / "cnt0.npy").tolist() == np.load(d / "cnt1.npy").tolist() == want_cnt
        assert np.array_equal(np.load(d / "out0.npy"), whole[-1]["y"][:2])
        assert np.array_equal(np.load(d / "out1.npy"), whole[-1]["y"][2:])
    # a single shard calibrated alone would have chosen other decimal points: the exchange matters
    alone = orc.run_network(params, x[:2], None, 16)
    assert [r["frac_bits"] for r in alone] != [r["frac_bits"] for r in orc.run_network(params, x, None, 16)]


def test_single_process_paths_need_no_process_group():
    assert replicas.agree_on_range(123) == 123
    assert replicas.sum_counters(1, 2, 3) == (1, 2, 3)
    assert replicas.slowest_rank_ms(4.5) == 4.5
    assert replicas.shard_seed(100, 3) == 103
    assert replicas.largest_float(2.5) == 2.5
    assert replicas.sum_histogram([1, 2, 3]) == [1, 2, 3]
