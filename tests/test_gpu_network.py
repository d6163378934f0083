"""GPU parity at the level of whole workloads: the LeNet-style stack, single VGG16 layers and the
whole VGG16 stack at the sizes the benchmark runs, each with every tensor, every chosen decimal
point and every counter compared with the oracle.  The full-size cases carry the extra marker
``slow`` (they still belong to ``-m gpu``); ``-m "gpu and not slow"`` leaves them out."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_1711_04713_b200 import binding as B
from paper_1711_04713_b200 import workloads as wl
from paper_1711_04713_b200.network import LPNetwork
from tests.util import dev, from_qtensor

pytestmark = pytest.mark.gpu


def _compare_stack(params, x, x_fmt, n_bits, in_hw, in_c, algo, threshold=0.0, rounding_seed=None):
    rec = orc.run_network(params, x, x_fmt, n_bits, threshold=threshold, rounding_seed=rounding_seed)
    net = LPNetwork(params, x.shape[0], in_hw, in_c, n_bits, algo=algo, rounding_seed=rounding_seed)
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
    # (stochastic rounding may land on either neighbour: up to one LSB; deterministic: half an LSB plus
    # the one-LSB saturation edge)
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


@pytest.mark.parametrize("algo", [B.ALGO_AUTO, B.ALGO_DIRECT])
def test_stacks_with_stochastic_rounding(algo):
    """rounding_scheme STOCHASTIC for every layer (paper Sec. 2, 2.4): input, weights, biases and layer
    outputs rounded stochastically with per-tensor seeds; every tensor, decimal point and counter equals
    the oracle's, in calibration and in inference, on the tensor-core path and on the plain kernels;
    also together with the thresholded allocation."""
    params = wl.make_params(wl.lenet_specs(), seed=0)
    x = wl.lenet_input(8, seed=0)
    rec = _compare_stack(params, x, None, 16, (28, 28), 1, algo, rounding_seed=11)
    base = orc.run_network(params, x, None, 16)
    assert any(not np.array_equal(r["y"], b["y"]) for r, b in zip(rec, base))      # it is another rounding
    specs = [wl.LayerSpec("conv", "c1", 3, 64, 3, 1, 1, True), wl.LayerSpec("conv", "c2", 64, 64, 3, 1, 1, True),
             wl.LayerSpec("pool", "p1"), wl.LayerSpec("conv", "c3", 64, 128, 3, 1, 1, True),
             wl.LayerSpec("pool", "p2"), wl.LayerSpec("ip", "f1", 8 * 8 * 128, 256, relu=True),
             wl.LayerSpec("ip", "f2", 256, 10, relu=False)]
    for n_bits, thr in ((16, 0.0), (8, 0.0), (16, 0.01)):
        _compare_stack(wl.make_params(specs, seed=6), wl.vgg16_input(8, seed=6, hw=32), None, n_bits, (32, 32), 3,
                       algo, threshold=thr, rounding_seed=12)


@pytest.mark.slow
def test_vgg16_with_stochastic_rounding():
    """The real VGG16 shapes (224 x 224 inputs, every tile family of the tensor-core path, the split
    inner products) with rounding_scheme STOCHASTIC for every layer, on a batch small enough for the
    oracle's generator: every tensor, decimal point and counter."""
    params = wl.make_params(wl.vgg16_specs(), seed=0)
    x = wl.vgg16_input(4, seed=7)
    _compare_stack(params, x, None, 16, (224, 224), 3, B.ALGO_AUTO, rounding_seed=21)


def test_giga1net_stack():
    """Giga1Net (paper Table 1): kernels of 1, 7, 5 and 3, 3 to 128 channels, four pools, two inner
    products; every tensor, decimal point and counter against the oracle on a small batch."""
    specs = wl.giga1net_specs()
    assert abs(wl.giga1net_macs_per_image() * 2 / 1e9 - 1.0) < 0.2      # "1 GOp/frame"
    params = wl.make_params(specs, seed=5)
    x = wl.vgg16_input(3, seed=5)
    _compare_stack(params, x, None, 16, (224, 224), 3, B.ALGO_AUTO)


def _full_conv_check(N, H, Cin, K, n_bits, seed):
    """One 3x3 / pad 1 LPConvolution at full size, ReLU'd N(0,1) input, He-normal weights, every format
    from range measurement: the GPU's measured range, chosen decimal point, every output element and
    all three counters against the oracle's direct convolution."""
    x = wl.relu_normal((N, H, H, Cin), seed)
    w = wl.he_conv_weight(K, 3, 3, Cin, seed + 1)
    b = wl.bias(K, seed + 2)
    fx = orc.measure_range(x, n_bits)[2]
    xq, _ = orc.quantize(x, n_bits, fx)
    wq, fw = orc.quantize_param(w, n_bits)
    bq, _ = orc.quantize(b, n_bits, fw)
    F = fx + fw
    acc = orc.conv_acc(xq, wq, (1, 1), (1, 1))
    A_want = orc.epilogue_range(acc, bq, fw, F, True)
    f_want = n_bits - 1 - orc.int_bits_from_acc(A_want, F, n_bits)
    want, cnt = orc.epilogue(acc, bq, fw, F, True, n_bits, f_want)
    del acc

    # the GPU measures every format itself
    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    xd = dev(x.reshape(-1, Cin))
    B.adaption_measure_range(xd, n_bits, mx, fmt)
    assert int(fmt.cpu()[1]) == fx
    xg = B.QTensor.empty(N * H * H, Cin, n_bits, fx, Cin)
    B.adaption_quantize(xd, N * H * H, Cin, xg)
    wd = dev(w.reshape(-1, Cin))
    mx.zero_()
    B.adaption_measure_range(wd, n_bits, mx, fmt)
    assert int(fmt.cpu()[1]) == fw
    wg = B.QTensor.empty(K * 9, Cin, n_bits, fw, Cin)
    B.adaption_quantize(wd, K * 9, Cin, wg)
    bg = B.QTensor.empty(1, K, n_bits, fw, None, with_q16=True)
    B.adaption_quantize(dev(b), 1, K, bg)
    shp = B.conv_shape(N, H, H, Cin, K, 3, 3, 1, 1)
    st = B.new_stats()
    B.adaption_lp_conv_fwd(shp, xg, wg, bg.q16, fw, True, B.MODE_RANGE, B.ALGO_TENSOR, None, st, None)
    assert int(B.read_stats(st).max_abs_acc) == A_want
    f_out = B.adaption_choose_frac_bits_from_acc(A_want, F, n_bits)
    assert f_out == f_want
    y = B.QTensor.empty(N * H * H, K, n_bits, f_out, K)
    st = B.new_stats()
    B.adaption_lp_conv_fwd(shp, xg, wg, bg.q16, fw, True, B.MODE_REQUANT, B.ALGO_TENSOR, y, st, None)
    s = B.read_stats(st)
    assert s.status == 0
    assert np.array_equal(from_qtensor(y).reshape(want.shape), want)
    assert (int(s.zeros), int(s.sat_pos), int(s.sat_neg)) == (cnt.zeros, cnt.sat_pos, cnt.sat_neg)
    # the dequantized view is within one LSB of the real-valued layer on the same operands (sampled)
    rng = np.random.default_rng(seed)
    for _ in range(64):
        n, oh, ow, k = (int(rng.integers(v)) for v in (N, H, H, K))
        v = orc.conv_acc_at(xq, wq, (1, 1), (1, 1), n, oh, ow, k) + (int(bq[k]) << fx)
        real = max(v, 0) * 2.0 ** -F
        assert abs(float(want[n, oh, ow, k]) * 2.0 ** -f_out - real) <= 2.0 ** -f_out


@pytest.mark.slow
def test_vgg16_conv3_2_batch32_whole_tensor():
    """The single-layer workload at full size (32 x 56 x 56 x 256 -> 256, 59 GMAC): every output."""
    _full_conv_check(32, 56, 256, 256, 16, seed=0)


@pytest.mark.slow
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
@pytest.mark.parametrize("n_bits", [4, 8, 12, 16])
def test_vgg16_conv4_1_batch64_precision_sweep(n_bits, seed):
    """The convolution half of the precision sweep as specified: 64 x 28 x 28 x 256 -> 512 at four
    widths and four seeds, every output."""
    _full_conv_check(64, 28, 256, 512, n_bits, seed)


@pytest.mark.slow
@pytest.mark.parametrize("n_bits,batch", [(16, 64), (8, 128)])
def test_vgg16_whole_batch_calibration_and_forward(n_bits, batch):
    """The whole VGG16 stack as the benchmark runs it (16-bit at batch 64, 8-bit at batch 128): the
    GPU calibrates on the whole batch (range measurement and decimal point per layer), the oracle does
    the same on the same images; every decimal point, every stored tensor of every layer, every
    counter and the measured ranges must agree, and the inference pass with those formats (pooling
    fused into the producing convolutions, parameters requantized or kept) reproduces the logits
    and counters."""
    params = wl.make_params(wl.vgg16_specs(), seed=0)
    x = wl.vgg16_input(batch, seed=0)
    _compare_stack(params, x, None, n_bits, (224, 224), 3, B.ALGO_AUTO)


@pytest.mark.slow
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
@pytest.mark.parametrize("n_bits", [4, 8, 12, 16])
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
