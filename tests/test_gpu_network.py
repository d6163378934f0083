"""GPU parity at the level of whole workloads: the LeNet-style stack (every tensor, every chosen
decimal point, every counter) and VGG16-shaped layers at full size on sampled outputs."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_1711_04713_b200 import binding as B
from paper_1711_04713_b200 import workloads as wl
from paper_1711_04713_b200.network import LPNetwork
from tests.util import dev, from_qtensor

pytestmark = pytest.mark.gpu


def _compare_stack(params, x, x_fmt, n_bits, in_hw, in_c, algo, threshold=0.0):
    rec = orc.run_network(params, x, x_fmt, n_bits, threshold=threshold)
    net = LPNetwork(params, x.shape[0], in_hw, in_c, n_bits, algo=algo)
    xd = dev(x.reshape(-1, in_c))
    grec = net.calibrate(xd, x_fmt, threshold=threshold)
    assert len(grec) == len(rec)
    assert grec[0]["frac_bits"] == rec[0]["frac_bits"]
    assert np.array_equal(from_qtensor(net.xq).reshape(rec[0]["y"].shape), rec[0]["y"])
    for L, g, r in zip(net.layers, grec[1:], rec[1:]):
        assert g["type"] == r["type"]
        assert g["frac_bits"] == r["frac_bits"], L.name
        got = from_qtensor(L.y).reshape(r["y"].shape)
        assert np.array_equal(got, r["y"]), L.name
        assert L.y.padding_is_zero()
        if r["type"] in ("conv", "ip"):
            assert g["w_frac_bits"] == r["w_frac_bits"]
            assert g["max_abs_acc"] == r["max_abs_acc"]
            assert np.array_equal(from_qtensor(L.w).reshape(r["wq"].shape), r["wq"])
            c = r["counters"]
            assert (int(g["stats"].zeros), int(g["stats"].sat_pos), int(g["stats"].sat_neg)) == \
                   (c.zeros, c.sat_pos, c.sat_neg), L.name
    # inference with the calibrated formats reproduces the calibration run, with and without
    # re-quantizing the parameters
    for requant in (True, False):
        net.zero_stats()
        out, _ = net.forward(xd, requantize_params=requant)
        torch.cuda.synchronize()
        assert np.array_equal(from_qtensor(out).reshape(rec[-1]["y"].shape), rec[-1]["y"])
        for s, r in zip(net.layer_stats(), [r for r in rec if r["type"] in ("conv", "ip")]):
            assert s["status"] == 0
            assert (s["zeros"], s["sat_pos"], s["sat_neg"]) == \
                   (r["counters"].zeros, r["counters"].sat_pos, r["counters"].sat_neg)
    # dequantized logits stay within one LSB of the real-valued last layer on the same operands
    last, prev = rec[-1], rec[-2]
    real = (prev["y"].reshape(prev["y"].shape[0], -1).astype(np.float64) * 2.0 ** -prev["frac_bits"]) @ \
           (last["wq"].astype(np.float64) * 2.0 ** -last["w_frac_bits"]).T + \
           last["bq"].astype(np.float64) * 2.0 ** -last["w_frac_bits"]
    deq = from_qtensor(out).astype(np.float64) * 2.0 ** -last["frac_bits"]
    assert np.all(np.abs(deq - real) <= 2.0 ** -last["frac_bits"])
    return rec


@pytest.mark.parametrize("algo", [B.ALGO_AUTO, B.ALGO_DIRECT])
@pytest.mark.parametrize("n_bits", [16, 8])
def test_lenet_stack(algo, n_bits):
    specs = wl.lenet_specs()
    params = wl.make_params(specs, seed=0)
    x = wl.lenet_input(8, seed=0)
    _compare_stack(params, x, (n_bits, n_bits - 1), n_bits, (28, 28), 1, algo)


def test_small_vgg_like_stack_tensor_path():
    """Three VGG-style blocks on 32x32 inputs: conv(3->64), conv(64->64), pool, conv(64->128), pool,
    two inner products; channel padding, pooling and flatten all on the tensor-core path."""
    specs = [wl.LayerSpec("conv", "c1", 3, 64, 3, 1, 1, True), wl.LayerSpec("conv", "c2", 64, 64, 3, 1, 1, True),
             wl.LayerSpec("pool", "p1"), wl.LayerSpec("conv", "c3", 64, 128, 3, 1, 1, True),
             wl.LayerSpec("pool", "p2"), wl.LayerSpec("ip", "f1", 8 * 8 * 128, 256, relu=True),
             wl.LayerSpec("ip", "f2", 256, 10, relu=False)]
    params = wl.make_params(specs, seed=3)
    x = wl.vgg16_input(8, seed=3, hw=32)
    _compare_stack(params, x, None, 16, (32, 32), 3, B.ALGO_AUTO)


@pytest.mark.parametrize("threshold", [0.002, 0.02])
def test_stacks_with_thresholded_bit_allocation(threshold):
    """Sec. 2.3: decimal points by the thresholded allocation instead of the maximum.  Formats differ
    from the max-based ones (more fractional bits, some values saturate) and every tensor, format
    and counter still matches the oracle."""
    params = wl.make_params(wl.lenet_specs(), seed=0)
    x = wl.lenet_input(8, seed=0)
    rec = _compare_stack(params, x, None, 16, (28, 28), 1, B.ALGO_AUTO, threshold=threshold)
    base = orc.run_network(params, x, None, 16)
    assert all(r["frac_bits"] >= b["frac_bits"] for r, b in zip(rec, base))
    if threshold >= 0.02:     # large enough to move decimal points on this stack
        assert any(r["frac_bits"] > b["frac_bits"] for r, b in zip(rec, base))
        assert sum(r["counters"].sat_pos for r in rec if "counters" in r) > 0
    specs = [wl.LayerSpec("conv", "c1", 3, 64, 3, 1, 1, True), wl.LayerSpec("conv", "c2", 64, 64, 3, 1, 1, True),
             wl.LayerSpec("pool", "p1"), wl.LayerSpec("conv", "c3", 64, 128, 3, 1, 1, True),
             wl.LayerSpec("pool", "p2"), wl.LayerSpec("ip", "f1", 8 * 8 * 128, 256, relu=True),
             wl.LayerSpec("ip", "f2", 256, 10, relu=False)]
    _compare_stack(wl.make_params(specs, seed=4), wl.vgg16_input(8, seed=4, hw=32), None, 8, (32, 32), 3,
                   B.ALGO_AUTO, threshold=threshold)


def test_giga1net_stack():
    """Giga1Net (paper Table 1): kernels of 1, 7, 5 and 3, 3 to 128 channels, four pools, two inner
    products; every tensor, decimal point and counter against the oracle on a small batch."""
    specs = wl.giga1net_specs()
    assert abs(wl.giga1net_macs_per_image() * 2 / 1e9 - 1.0) < 0.2      # "1 GOp/frame"
    params = wl.make_params(specs, seed=5)
    x = wl.vgg16_input(3, seed=5)
    _compare_stack(params, x, None, 16, (224, 224), 3, B.ALGO_AUTO)


def _sampled_conv_check(N, H, Cin, K, n_bits, seed, samples=1500):
    rng = np.random.default_rng(seed)
    x = wl.relu_normal((N, H, H, Cin), seed)
    w = wl.he_conv_weight(K, 3, 3, Cin, seed + 1)
    b = wl.bias(K, seed + 2)
    fx = orc.measure_range(x, n_bits)[2]
    xq, _ = orc.quantize(x, n_bits, fx)
    wq, fw = orc.quantize_param(w, n_bits)
    bq, _ = orc.quantize(b, n_bits, fw)
    xd = dev(x.reshape(-1, Cin))
    xg = B.QTensor.empty(N * H * H, Cin, n_bits, fx, Cin)
    B.adaption_quantize(xd, N * H * H, Cin, xg)
    wg = B.QTensor.empty(K * 9, Cin, n_bits, fw, Cin)
    B.adaption_quantize(dev(w.reshape(-1, Cin)), K * 9, Cin, wg)
    bg = B.QTensor.empty(1, K, n_bits, fw, None, with_q16=True)
    B.adaption_quantize(dev(b), 1, K, bg)
    shp = B.conv_shape(N, H, H, Cin, K, 3, 3, 1, 1)
    st = B.new_stats()
    B.adaption_lp_conv_fwd(shp, xg, wg, bg.q16, fw, True, B.MODE_RANGE, B.ALGO_TENSOR, None, st, None)
    A = int(B.read_stats(st).max_abs_acc)
    F = fx + fw
    f_out = B.adaption_choose_frac_bits_from_acc(A, F, n_bits)
    y = B.QTensor.empty(N * H * H, K, n_bits, f_out, K)
    st = B.new_stats()
    B.adaption_lp_conv_fwd(shp, xg, wg, bg.q16, fw, True, B.MODE_REQUANT, B.ALGO_TENSOR, y, st, None)
    s = B.read_stats(st)
    assert s.status == 0
    got = from_qtensor(y).reshape(N, H, H, K)
    # sampled outputs, computed one by one by the oracle; image corners and edges always included
    pts = [(0, 0, 0, 0), (N - 1, H - 1, H - 1, K - 1), (N - 1, 0, H - 1, 1), (0, H - 1, 0, K // 2)]
    pts += [tuple(int(v) for v in (rng.integers(N), rng.integers(H), rng.integers(H), rng.integers(K)))
            for _ in range(samples)]
    vmax_seen = 0
    for (n, oh, ow, k) in pts:
        acc = np.array([[orc.conv_acc_at(xq, wq, (1, 1), (1, 1), n, oh, ow, k)]], dtype=np.int64)
        want, _ = orc.epilogue(acc, bq[k:k + 1], fw, F, True, n_bits, f_out)
        assert int(got[n, oh, ow, k]) == int(want[0, 0]), (n, oh, ow, k)
        vmax_seen = max(vmax_seen, orc.epilogue_range(acc, bq[k:k + 1], fw, F, True))
    # properties that hold at any size
    assert A >= vmax_seen
    assert f_out == n_bits - 1 - orc.int_bits_from_acc(A, F, n_bits)
    assert got.min() >= 0 and int(s.sat_neg) == 0 and int(s.sat_pos) <= 1
    assert int(s.zeros) == int((got == 0).sum())
    return got


def test_vgg16_conv3_2_batch32_sampled():
    """The single-layer workload at full size (32 x 56 x 56 x 256 -> 256, 59 GMAC)."""
    _sampled_conv_check(32, 56, 256, 256, 16, seed=0)


def test_vgg16_conv4_1_precision_sweep_sampled():
    for n_bits, seed in [(4, 0), (8, 1), (12, 2), (16, 3)]:
        _sampled_conv_check(16, 28, 256, 512, n_bits, seed, samples=300)


@pytest.mark.parametrize("n_bits,batch", [(16, 64), (8, 128)])
def test_vgg16_full_batch_in_the_benchmark_configuration(n_bits, batch):
    """The whole VGG16 stack at the benchmark's batch size and launch configuration (same network
    object, same forward call).  The oracle runs the first two images of the batch, with decimal
    points it chose itself on those two images; the GPU gets these formats and must reproduce every
    layer's output for the two images bit for bit (images are independent).  Counters and padding are
    checked on the full batch through properties that hold at any size."""
    specs = wl.vgg16_specs()
    params = wl.make_params(specs, seed=0)
    x = wl.vgg16_input(batch, seed=0)
    sub = 2
    rec = orc.run_network(params, x[:sub], None, n_bits)
    xd = dev(x.reshape(-1, 3))
    counters = {}
    # first with every layer's output materialised, then as the benchmark runs it: a convolution
    # whose output only feeds a pooling layer hands over pooled data and keeps no tensor of its own
    for fuse_pool in (False, True):
        net = LPNetwork(params, batch, (224, 224), 3, n_bits, fuse_pool=fuse_pool)
        net.set_formats(rec[0]["frac_bits"], [r["frac_bits"] for r in rec[1:] if r["type"] in ("conv", "ip")])
        net.zero_stats()
        out, _ = net.forward(xd)
        torch.cuda.synchronize()
        got_in = from_qtensor(net.xq)
        assert np.array_equal(got_in[:sub * 224 * 224].reshape(rec[0]["y"].shape), rec[0]["y"])
        n_fused = 0
        for i, (L, r) in enumerate(zip(net.layers, rec[1:])):
            if r["type"] in ("conv", "ip"):
                assert L.w.frac_bits == r["w_frac_bits"], L.name
                st = B.read_stats(L.stats)
                assert int(st.status) == 0
                got = (int(st.zeros), int(st.sat_pos), int(st.sat_neg))
            if net.fused_pool_after(i):
                # counters are those of the convolution's own output: equal to the unfused run's
                assert got == counters[L.name], L.name
                n_fused += 1
                continue
            full = from_qtensor(L.y)
            rows = full.shape[0] // batch * sub
            assert np.array_equal(full[:rows].reshape(r["y"].shape), r["y"]), L.name
            assert L.y.padding_is_zero(), L.name
            if r["type"] in ("conv", "ip"):
                counters.setdefault(L.name, got)
                assert got == counters[L.name], L.name
                assert got[0] == int((full == 0).sum()), L.name
                qmax, qmin = (1 << (n_bits - 1)) - 1, -(1 << (n_bits - 1))
                assert got[1] <= int((full == qmax).sum()) and got[2] <= int((full == qmin).sum())
                if L.relu:
                    assert int(full.min()) >= 0 and got[2] == 0
            del full
        assert n_fused == (5 if fuse_pool else 0)
        del net


@pytest.mark.parametrize("n_bits,seed", [(4, 0), (8, 1), (12, 2), (16, 3)])
def test_fc6_batch256_precision_sweep(n_bits, seed):
    """The inner-product half of the precision sweep at full size: 25088 -> 4096 at batch 256,
    ReLU'd N(0,1) inputs, He-normal weights, formats from range measurement; every output compared."""
    Bsz, K, O = 256, 25088, 4096
    x = wl.relu_normal((Bsz, K), seed)
    w = wl.he_ip_weight(O, K, seed + 1)
    b = wl.bias(O, seed + 2)
    fx = orc.measure_range(x, n_bits)[2]
    xq, _ = orc.quantize(x, n_bits, fx)
    wq, fw = orc.quantize_param(w, n_bits)
    bq, _ = orc.quantize(b, n_bits, fw)
    acc = orc.ip_acc(xq, wq)
    F = fx + fw
    A = orc.epilogue_range(acc, bq, fw, F, True)
    f_out = n_bits - 1 - orc.int_bits_from_acc(A, F, n_bits)
    want, cnt = orc.epilogue(acc, bq, fw, F, True, n_bits, f_out)

    # the GPU measures the same formats itself
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    xd, wd = dev(x), dev(w)
    B.adaption_measure_range(xd, n_bits, mx, fmt)
    assert int(fmt.cpu()[1]) == fx
    xg = B.QTensor.empty(Bsz, K, n_bits, fx, K)
    B.adaption_quantize(xd, Bsz, K, xg)
    mx.zero_()
    B.adaption_measure_range(wd, n_bits, mx, fmt)
    assert int(fmt.cpu()[1]) == fw
    wg = B.QTensor.empty(O, K, n_bits, fw, K)
    B.adaption_quantize(wd, O, K, wg)
    bg = B.QTensor.empty(1, O, n_bits, fw, None, with_q16=True)
    B.adaption_quantize(dev(b), 1, O, bg)
    need = B.adaption_lp_ip_workspace_bytes(Bsz, K, O, xg.fmt(), wg.fmt(), B.ALGO_AUTO)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda") if need else None
    st = B.new_stats()
    B.adaption_lp_ip_fwd(Bsz, K, O, xg, wg, bg.q16, fw, True, B.MODE_RANGE, B.ALGO_AUTO, None, st, ws)
    assert int(B.read_stats(st).max_abs_acc) == A
    assert B.adaption_choose_frac_bits_from_acc(A, F, n_bits) == f_out
    y = B.QTensor.empty(Bsz, O, n_bits, f_out, O)
    st = B.new_stats()
    B.adaption_lp_ip_fwd(Bsz, K, O, xg, wg, bg.q16, fw, True, B.MODE_REQUANT, B.ALGO_AUTO, y, st, ws)
    s = B.read_stats(st)
    assert s.status == 0
    assert np.array_equal(from_qtensor(y), want)
    assert (int(s.zeros), int(s.sat_pos), int(s.sat_neg)) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
