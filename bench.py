#!/usr/bin/env python
"""Benchmark of the low-precision forward path on B200.

Workload: full VGG16 forward, 16-bit weights and activations, batch 64 per GPU, seeded synthetic
input (N(0,1) images, He-normal weights), every decimal point fixed beforehand by range
measurement on the batch.  One step = one forward pass of the batch through the whole path:
range measurement of the input, LPAct of the input, quantization of all weights and biases,
13 LPConvolution + 3 LPInnerProduct layers with fused bias / ReLU / requantization / zero
counting, 5 max-pools.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--batch B] [--n-bits 16]

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample of
the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "effective fixed-point TOPS & images/s for VGG16 16-bit forward; % of INT8 peak"
INT8_NOMINAL_TOPS = 4500.0          # dense INT8, datasheet
NOMINAL_INT8_OVER_BF16 = 2.0        # nominal dense INT8 : bf16 ratio (4.5 : 2.25 POPS)
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_BF16_SUSTAINED = 1400.0
# DRAM traffic of the layer GEMM per launch comes from a small text record next to the ncu summary it
# was read from; it names the kernel source it is valid for.
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "lp_gemm_dram_traffic.txt")


def gemm_traffic(n_bits: int, batch: int):
    """DRAM bytes per layer-GEMM launch from the committed ncu record, or None when the record is
    missing, was taken on another workload, or the kernel source has changed since."""
    import hashlib
    try:
        rec = dict(line.split(None, 1) for line in open(TRAFFIC_RECORD) if line.strip() and not line.startswith("#"))
        src = os.path.join(ROOT, "paper_1711_04713_b200", "csrc", "gemm_tc.cu")
        sha = hashlib.sha1(open(src, "rb").read()).hexdigest()
        if not sha.startswith(rec["source_sha1"].strip()):
            return None
        if int(rec["n_bits"]) != n_bits or int(rec["batch"]) != batch:
            return None
        return float(rec["bytes_per_launch"])
    except (OSError, KeyError, ValueError):
        return None


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_burst": float(p["bf16_tflops"]),
                "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_burst": FALLBACK_BF16_TFLOPS, "bf16_sustained": FALLBACK_BF16_SUSTAINED,
                "source": "fallback"}


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = f"/tmp/adaption_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu)], stdout=self.fh, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin: float | None = None, t_end: float | None = None) -> dict:
        """Median SM clock and the throttle reasons seen; with t_begin/t_end (time.time()) only the
        samples taken inside that window count."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, mx, pw, reasons = [], [], [], set()
        try:
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                if t_begin is not None:
                    try:
                        ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    except ValueError:
                        continue
                    if ts < t_begin - 0.05 or ts > t_end + 0.05:
                        continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                    pw.append(float(f[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["sm_max_mhz"] = max(mx)
            out["power_w_max"] = max(pw) if pw else None
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------------------------------
# reference arm: the CPU oracle on a bounded sample
# ---------------------------------------------------------------------------------------------
def oracle_sample_step(params, x_sample, formats, n_bits):
    from oracle import reference as orc
    t0 = time.perf_counter()
    orc.run_network(params, x_sample, formats["input"], n_bits, fixed_formats=formats["layers"])
    return time.perf_counter() - t0


def oracle_formats(params, x_sample, n_bits):
    """Formats fixed by a calibration pass of the oracle on the sample itself (untimed)."""
    from oracle import reference as orc
    rec = orc.run_network(params, x_sample, None, n_bits)
    return {"input": (rec[0]["n_bits"], rec[0]["frac_bits"]),
            "layers": [r["frac_bits"] for r in rec if r["type"] in ("conv", "ip")]}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        # the multi-process launcher pins every rank to one OpenMP thread; only this rank computes here,
        # so it takes the host cores it may run on (read by the OpenMP runtime when the oracle loads)
        os.environ["OMP_NUM_THREADS"] = str(len(os.sched_getaffinity(0)))
    from oracle import reference as orc
    from paper_1711_04713_b200 import workloads as wl
    params = wl.make_params(wl.vgg16_specs(), seed=0)
    macs_img = wl.vgg16_macs_per_image()
    sample_images = 1
    x = wl.vgg16_input(sample_images, seed=0)
    formats = oracle_formats(params, x, args.n_bits)
    # keep the whole run within a few minutes: the oracle is slow by design, so when K + W steps
    # of one image each would take longer than the budget, fewer steps are executed and said so
    budget_s = 240.0
    t_probe = oracle_sample_step(params, x, formats, args.n_bits)
    can_run = max(1, int(budget_s / max(t_probe, 1e-3)))
    warm = min(args.warmup, max(0, can_run - 1) // 4)
    steps_exec = max(1, min(args.steps, can_run - warm))
    for _ in range(warm):
        oracle_sample_step(params, x, formats, args.n_bits)
    t = 0.0
    for _ in range(steps_exec):
        t += oracle_sample_step(params, x, formats, args.n_bits)
    ms = t / steps_exec * 1e3
    ips = sample_images / (ms / 1e3)
    cores = orc.num_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": ips, "unit": "images/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "steps_executed": steps_exec, "warmup_executed": warm,
        "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": f"int{args.n_bits}", "data": "synthetic",
        "effective_tops": 2.0 * macs_img * ips / 1e12,
        "config": {"workload": f"VGG16 forward, {args.n_bits}-bit weights and activations (full stack); "
                               f"each step = {sample_images} image through the CPU oracle",
                   "global_batch": sample_images, "n_bits": args.n_bits},
        "cpu_baseline": {"value": ips, "unit": "images/s", "cores": cores, "kind": "oracle",
                         "sample": f"{sample_images} image(s) per step, whole VGG16 stack, fixed formats"},
        "e2e": {"value": ips, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# single kernels: timing helpers shared by the headline run and by `--kernel`
# ---------------------------------------------------------------------------------------------
def _time_ms(torch, fn, iters: int, warmup: int = 3) -> float:
    """CUDA-event time per call on the current stream, after warm-up, synchronised on both sides."""
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


def int8_probe(B, torch, gpu_index: int, repeats: int = 5, iters: int = 400000) -> dict:
    """The int8 tensor pipe's issue rate: every SM runs 4 * iters back-to-back 128x128x32 int8 MMAs on
    operands resident in shared memory (about 55 ms per run at 1.85 GHz).  Median of `repeats` runs by
    CUDA events; the SM clock is sampled while they run."""
    out = {"int8_tops": None}
    try:
        sms = torch.cuda.get_device_properties(gpu_index).multi_processor_count
        cyc = torch.zeros(max(sms, 256), dtype=torch.int64, device="cuda")
        pst = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.adaption_probe_i8_peak(128, False, 4096, cyc, pst)      # warm-up
        torch.cuda.synchronize()
        sampler = ClockSampler(gpu_index)
        sampler.start()
        time.sleep(0.3)
        w0 = time.time()
        times = []
        for _ in range(repeats):
            times.append(_time_ms(torch, lambda: B.adaption_probe_i8_peak(128, False, iters, cyc, pst), 1, warmup=0))
        w1 = time.time()
        clk = sampler.stop(w0, w1)
        if int(pst.cpu()[0]) != 0:
            raise RuntimeError("probe reported a timeout")
        ms = statistics.median(times)
        c = cyc.cpu()
        issuing = c[c > 0].double()
        out = {"int8_tops": 2.0 * sms * 4 * iters * 128 * 128 * 32 / (ms / 1e3) / 1e12, "repeats": repeats,
               "ms_per_run": ms, "cycles_per_mma": float(issuing.mean()) / (4 * iters), "sm_mhz": clk.get("sm_mhz"),
               "reasons": clk.get("reasons")}
    except Exception as exc:  # the probe only feeds the denominator
        out["error"] = str(exc)
    return out


def streaming_kernels(B, torch, hbm_gbs: float, numel: int = 1 << 28, iters: int = 10) -> dict:
    """The HBM-bound steps of the path, each alone on buffers far larger than L2 (numel fp32 values =
    1 GiB in): algorithmic GB/s (bytes the step must read and write / CUDA-event time) and the
    fraction of the measured copy bandwidth."""
    out = {}
    inner = 256
    outer = numel // inner
    g = torch.Generator(device="cuda").manual_seed(0)
    x = torch.randn(outer, inner, device="cuda", generator=g)

    def rec(name, ms, nbytes, note):
        gbs = nbytes / (ms / 1e3) / 1e9
        out[name] = {"gbs": gbs, "frac_of_hbm": gbs / hbm_gbs, "ms": ms, "algorithmic_bytes": nbytes, "what": note}

    mx = torch.zeros(1, dtype=torch.float32, device="cuda")
    fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
    rec("range", _time_ms(torch, lambda: B.adaption_measure_range(x, 16, mx, fmt), iters), 4 * numel,
        "adaption_measure_range: 4 B read per element")
    st = B.new_stats()
    for n_bits in (16, 8):
        pb = 2 if n_bits > 8 else 1
        q = B.QTensor.empty(outer, inner, n_bits, n_bits - 3)
        rec(f"quantize_n{n_bits}",
            _time_ms(torch, lambda: B.adaption_quantize(x, outer, inner, q, None, B.ROUND_DETERMINISTIC, st), iters),
            (4 + pb) * numel, f"adaption_quantize fp32 -> {n_bits}-bit planes: 4 B read + {pb} B written per element")
        if n_bits == 16:
            rec("lp_act_fp32_relu_n16",
                _time_ms(torch, lambda: B.adaption_lp_act(x, None, outer, inner, True, q, None,
                                                          B.ROUND_DETERMINISTIC, st), iters),
                (4 + pb) * numel, "adaption_lp_act on fp32 input with ReLU (same kernel as the quantizer)")
            q2 = B.QTensor.empty(outer, inner, n_bits, n_bits - 5)
            rec("lp_act_requant_n16",
                _time_ms(torch, lambda: B.adaption_lp_act(None, q, outer, inner, True, q2, None,
                                                          B.ROUND_DETERMINISTIC, st), iters),
                2 * pb * numel, "adaption_lp_act on a stored 16-bit tensor (format change): 2 B read + 2 B written")
            H = 112
            N = numel // (H * H * inner)
            qp = B.QTensor.empty(N * (H // 2) ** 2, inner, n_bits, n_bits - 3)
            qin = q
            rec("maxpool2x2_n16", _time_ms(torch, lambda: B.adaption_maxpool2x2(qin, N, H, H, inner, qp), iters),
                int(pb * N * H * H * inner * 1.25), "adaption_maxpool2x2, 16-bit: 2 B read + 0.5 B written per input element")
            del q2, qp
        del q
    del x
    return out


def params_quantizer(B, torch, net, hbm_gbs: float, iters: int = 10) -> dict:
    """All weight and bias tensors of the network quantized with fixed formats by one library call, as
    every forward pass of the headline does."""
    ms = _time_ms(torch, lambda: net.quantize_params(measure=False), iters)
    n = sum(L.w_f32.numel() + L.b_f32.numel() for L in net.layers if L.type in ("conv", "ip"))
    nbytes = n * (4 + (2 if net.n_bits > 8 else 1))
    gbs = nbytes / (ms / 1e3) / 1e9
    return {"gbs": gbs, "frac_of_hbm": gbs / hbm_gbs, "ms": ms, "algorithmic_bytes": nbytes,
            "what": f"adaption_quantize_batch over {n} parameters ({net.param_quantize_launches()} launches)"}


def oracle_single_thread() -> dict | None:
    """One image of the single-layer workload (56 x 56 x 256 -> 256, 3x3) through the oracle's direct
    convolution on ONE host thread (a child process with OMP_NUM_THREADS=1)."""
    code = ("import time, numpy as np\n"
            "from oracle import reference as orc\n"
            "rng = np.random.default_rng(0)\n"
            "x = rng.integers(0, 32768, (1, 56, 56, 256)).astype(np.int16)\n"
            "w = rng.integers(-32768, 32768, (256, 3, 3, 256)).astype(np.int16)\n"
            "orc.conv_acc(x[:, :8], w, (1, 1))\n"
            "t = time.perf_counter(); orc.conv_acc(x, w, (1, 1)); t = time.perf_counter() - t\n"
            "print(t, orc.num_threads())\n")
    try:
        env = dict(os.environ, OMP_NUM_THREADS="1")
        r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=120)
        t, threads = r.stdout.split()
        gmac = 56 * 56 * 256 * 9 * 256 / 1e9
        return {"gmac_per_s": gmac / float(t), "threads": int(threads), "seconds": float(t),
                "sample": "direct convolution of one 56x56x256 -> 256 image (1.85 GMAC)"}
    except Exception:
        return None


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------
def run_gpu(args):
    import torch

    from paper_1711_04713_b200 import binding as B
    from paper_1711_04713_b200 import build as bld
    from paper_1711_04713_b200 import replicas
    from paper_1711_04713_b200 import workloads as wl
    from paper_1711_04713_b200.network import LPNetwork

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (no CPU fallback exists)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        bld.build_library()
    if dist is not None:
        dist.barrier()
    B.load()
    apply_overrides(B, args)
    peaks = read_peaks()

    # ---- workload: each rank owns its own batch of images (weak scaling, no data-path collective)
    specs = wl.vgg16_specs()
    params = wl.make_params(specs, seed=0)
    batch = args.batch
    x_host = torch.from_numpy(wl.vgg16_input(batch, seed=replicas.shard_seed(100, rank)).reshape(-1, 3)).pin_memory()
    x_dev = x_host.cuda()
    net = LPNetwork(params, batch, (224, 224), 3, args.n_bits)
    del params
    net.calibrate(x_dev)
    macs_step = net.total_macs
    torch.cuda.synchronize()

    gemm_layers = [L for L in net.layers if L.type in ("conv", "ip")]
    n_gemm = len(gemm_layers)

    def step(timed_events=None, x_in=None, requantize=True):
        """One forward pass of the batch; optional CUDA events around every layer-GEMM launch.
        `requantize=False` is the inference mode with the parameters quantized beforehand."""
        x_in = x_dev if x_in is None else x_in
        B.adaption_measure_range(x_in, net.n_bits, net.x_max_dev, net.x_fmt_dev)
        B.adaption_lp_act(x_in, None, net.xq.outer, net.xq.inner, False, net.xq, None,
                          B.ROUND_DETERMINISTIC, net.x_stats)
        if requantize:
            net.quantize_params(measure=False)
        a = net.xq
        i = 0
        while i < len(net.layers):
            L = net.layers[i]
            fused = net.fused_pool_after(i)
            timed = timed_events is not None and L.type != "pool"
            if timed:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            if fused:
                # convolution with the horizontal half of the pooling in its epilogue, then (outside the
                # layer-GEMM events) the vertical half
                P = net.layers[i + 1]
                net._run_conv_pool(L, P, a, B.PHASE_CONV)
            else:
                a = net._run_layer(L, a, B.MODE_REQUANT)
            if timed:
                e1.record()
                timed_events.append((L, e0, e1))
            if fused:
                a = net._run_conv_pool(L, P, a, B.PHASE_POOL)
                i += 1
            i += 1
        return a

    # kernels of ours per step: range (2) + input LPAct (1) + weight/bias quantization (dense tensors
    # batched into one launch) + one per layer (+1 finalize where K is split, +2 first-layer tap packing)
    launches_step = (3 + net.param_quantize_launches() + len(net.layers) +
                     sum(net.helper_launches(L) for L in gemm_layers))

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()          # nvidia-smi needs a moment to start: launch it before the warm-up
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if rank == 0:
        t_spin = time.time()
        while time.time() - t_spin < 1.0:       # untimed extra warm-up until the sampler is running
            step()
            torch.cuda.synchronize()

    net.zero_stats()
    events = []
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    t0.record()
    # CUDA events around every layer GEMM cost a few microseconds each (the next kernel cannot start
    # under the tail of the previous one): they are recorded on every event_every-th step of the timed
    # region only, which still gives the kernel's duration live inside it
    every = max(1, args.event_every)
    steps_sampled = 0
    for k in range(args.steps):
        if k % every == 0:
            out = step(events)
            steps_sampled += 1
        else:
            out = step()
    t1.record()
    torch.cuda.synchronize()
    wall1 = time.time()
    if dist is not None:
        dist.barrier()
    elapsed_ms = t0.elapsed_time(t1)
    clocks = sampler.stop(wall0, wall1) if rank == 0 else {}
    elapsed_ms = replicas.slowest_rank_ms(elapsed_ms, device="cuda")
    ms_per_step = elapsed_ms / args.steps
    ips = replicas.whole_job_rate(batch, world, ms_per_step)
    eff_tops = 2.0 * macs_step * world / (ms_per_step / 1e3) / 1e12

    # ---- per-launch durations of the dominant kernel (the tensor-core layer GEMM), from the
    #      events recorded inside the timed region
    per_layer = {}
    gemm_ms = 0.0
    for L, e0, e1 in events:
        d = e0.elapsed_time(e1)
        per_layer.setdefault(L.name, []).append(d)
        gemm_ms += d
    gemm_launches = len(events)
    gemm_ops = 2.0 * macs_step * steps_sampled               # logical n-bit operations in those launches
    achieved_tops = gemm_ops / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else 0.0
    planes = 4.0 if args.n_bits > 8 else 1.0                  # int8 products per logical MAC
    # Denominator: the int8 tensor pipe's own rate as the library's probe measures it on this GPU
    # (back-to-back tcgen05.mma kind::i8 on operands resident in shared memory), several repeats of
    # 50 ms and more each, median; the SM clock it ran at is sampled beside it.  The figures derived
    # from the measured bf16 GEMM (x2, the nominal INT8 : bf16 ratio) and the datasheet's 4.5 POPS are
    # reported as side keys.
    probe = int8_probe(B, torch, local_rank)
    bf16_burst_int8 = peaks["bf16_burst"] * NOMINAL_INT8_OVER_BF16
    if probe and probe.get("int8_tops"):
        peak_int8 = max(probe["int8_tops"], bf16_burst_int8)
        peak_source = ("int8 issue-rate probe of this run (adaption_probe_i8_peak, 128x128x32, median of "
                       f"{probe['repeats']} runs of {probe['ms_per_run']:.0f} ms at {probe['sm_mhz']} MHz)"
                       if probe["int8_tops"] >= bf16_burst_int8 else
                       f"{peaks['source']} bf16 burst {peaks['bf16_burst']} x{NOMINAL_INT8_OVER_BF16:g}")
    else:
        peak_int8 = bf16_burst_int8
        peak_source = f"{peaks['source']} bf16 burst {peaks['bf16_burst']} x{NOMINAL_INT8_OVER_BF16:g} (probe failed)"
    peak = peak_int8 / planes
    roofline = {
        "bound": "tensor", "kernel": "lp_gemm_kernel (all LPConvolution / LPInnerProduct launches)",
        "achieved": achieved_tops, "peak": peak, "unit": "TFLOP/s", "frac": achieved_tops / peak,
        "traffic": gemm_traffic(args.n_bits, batch), "traffic_unit": "bytes per launch (DRAM read + write)",
        "peak_source": f"{peak_source} / {planes:g} int8 products per {args.n_bits}-bit MAC",
        "int8_probe": probe,
        "frac_of_nominal_int8": achieved_tops / (INT8_NOMINAL_TOPS / planes),
        "frac_of_measured_bf16_burst_x2": achieved_tops / (bf16_burst_int8 / planes),
        "frac_of_measured_bf16_sustained_x2": achieved_tops / (peaks["bf16_sustained"] * NOMINAL_INT8_OVER_BF16 / planes),
        "launches": gemm_launches, "avg_launch_ms": gemm_ms / max(gemm_launches, 1),
        "steps_with_events": steps_sampled,
        "share_of_step": (gemm_ms / max(steps_sampled, 1)) / ms_per_step if world == 1 else None,
    }
    layer_table = {k: {"ms": statistics.mean(v)} for k, v in per_layer.items()}
    for L in gemm_layers:
        layer_table[L.name]["tops"] = 2.0 * L.macs / (layer_table[L.name]["ms"] / 1e3) / 1e12
        layer_table[L.name]["frac_of_nominal_int8"] = layer_table[L.name]["tops"] / (INT8_NOMINAL_TOPS / planes)
    conv_ms = sum(layer_table[L.name]["ms"] for L in gemm_layers if L.type == "conv")
    conv_tops = 2.0 * sum(L.macs for L in gemm_layers if L.type == "conv") / (conv_ms / 1e3) / 1e12
    roofline["conv_layers"] = {"tops": conv_tops, "ms": conv_ms,
                               "frac_of_nominal_int8": conv_tops / (INT8_NOMINAL_TOPS / planes),
                               "frac_of_probe": conv_tops / peak,
                               "target": "at least 0.60 of the dense INT8 peak / int8 products per MAC"}

    stats = net.layer_stats()
    sparsity = {s["name"]: round(s["zeros"] / max(s["total"], 1) / args.steps, 4) for s in stats}
    sat = {s["name"]: [s["sat_pos"] // args.steps, s["sat_neg"] // args.steps] for s in stats}

    # ---- end to end: host buffers in, host result out, copies inside the timed region
    out_host_lo = torch.empty_like(out.lo, device="cpu").pin_memory()
    out_host_hi = torch.empty_like(out.hi, device="cpu").pin_memory() if out.hi is not None else None
    e2e_steps = max(3, min(args.steps, 10))
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # Every step copies its own input from pinned host memory and reads its result back; the copy
    # of step i + 1 runs on a second stream into a second buffer while step i computes (what a
    # serving loop does), and the host waits only once, at the end.
    cur = torch.cuda.current_stream()
    copy_stream = torch.cuda.Stream()
    x_bufs = [x_dev, torch.empty_like(x_dev)]
    ready = [torch.cuda.Event(), torch.cuda.Event()]
    consumed = [torch.cuda.Event(), torch.cuda.Event()]
    e0.record()
    copy_stream.wait_stream(cur)
    with torch.cuda.stream(copy_stream):
        x_bufs[0].copy_(x_host, non_blocking=True)
        ready[0].record(copy_stream)
    for i in range(e2e_steps):
        b = i % 2
        if i + 1 < e2e_steps:
            with torch.cuda.stream(copy_stream):
                if i >= 1:
                    copy_stream.wait_event(consumed[1 - b])     # the buffer's previous step has read it
                x_bufs[1 - b].copy_(x_host, non_blocking=True)
                ready[1 - b].record(copy_stream)
        cur.wait_event(ready[b])
        o = step(x_in=x_bufs[b])
        consumed[b].record(cur)
        out_host_lo.copy_(o.lo, non_blocking=True)
        if out_host_hi is not None:
            out_host_hi.copy_(o.hi, non_blocking=True)
    cur.synchronize()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = replicas.slowest_rank_ms(e2e_ms, device="cuda")
    e2e_ips = replicas.whole_job_rate(batch, world, e2e_ms / e2e_steps)
    h2d = x_host.numel() * 4
    d2h = out.lo.numel() + (out.hi.numel() if out.hi is not None else 0)

    bad = [s for s in net.layer_stats() if s["status"] != 0]
    if bad:
        raise RuntimeError(f"device-side timeout flagged in {bad}")

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- side measurements (rank 0, one GPU): other modes of the same stack, the HBM-bound steps alone
    side = {}
    streaming = None
    if world == 1 and not args.headline_only:
        k_side = max(5, min(args.steps, 20))
        ms_inf = _time_ms(torch, lambda: step(requantize=False), k_side)
        side["inference_mode"] = {
            "what": "same step with weights and biases quantized beforehand (no per-forward parameter quantization)",
            "ms_per_step": ms_inf, "images_per_s": batch / (ms_inf / 1e3),
            "effective_tops": 2.0 * macs_step / (ms_inf / 1e3) / 1e12}
        t_c = time.perf_counter()
        n_cal = 3
        for _ in range(n_cal):
            net.calibrate(x_dev)
        torch.cuda.synchronize()
        ms_cal = (time.perf_counter() - t_c) / n_cal * 1e3
        side["calibration_forward"] = {
            "what": "LPNetwork.calibrate on the batch: per layer a RANGE pass, a host read of the range, a "
                    "REQUANT pass; parameters measured and quantized; wall clock including the host reads",
            "ms_per_batch": ms_cal, "images_per_s": batch / (ms_cal / 1e3)}
        streaming = streaming_kernels(B, torch, peaks["hbm_gbs"])
        streaming["quantize_batch_params"] = params_quantizer(B, torch, net, peaks["hbm_gbs"])
        other_bits, other_batch = (8, 128) if args.n_bits > 8 else (16, 64)
        try:
            del net
            torch.cuda.empty_cache()
            params2 = wl.make_params(specs, seed=0)
            x2 = torch.from_numpy(wl.vgg16_input(other_batch, seed=100).reshape(-1, 3)).cuda()
            net2 = LPNetwork(params2, other_batch, (224, 224), 3, other_bits)
            del params2
            net2.calibrate(x2)

            def step2():
                B.adaption_measure_range(x2, net2.n_bits, net2.x_max_dev, net2.x_fmt_dev)
                net2.forward(x2, requantize_params=True, measure_input=False)

            ms2 = _time_ms(torch, step2, k_side)
            side[f"vgg16_{other_bits}bit_batch{other_batch}"] = {
                "what": f"the same stack and step at {other_bits}-bit weights and activations, batch {other_batch}",
                "ms_per_step": ms2, "images_per_s": other_batch / (ms2 / 1e3),
                "effective_tops": 2.0 * net2.total_macs / (ms2 / 1e3) / 1e12,
                "sparsity": {s_["name"]: round(s_["zeros"] / max(s_["total"], 1) / (k_side + 4), 4)
                             for s_ in net2.layer_stats()},
                "saturations": {s_["name"]: [s_["sat_pos"] // (k_side + 4), s_["sat_neg"] // (k_side + 4)]
                                for s_ in net2.layer_stats()}}
            del net2, x2
        except Exception as exc:  # a side key must not take the headline down
            side[f"vgg16_{other_bits}bit_batch{other_batch}"] = {"error": str(exc)}

    # ---- the oracle on the host cores, on a bounded sample of the same workload
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import reference as orc
        params = wl.make_params(specs, seed=0)
        xs = wl.vgg16_input(1, seed=100)
        formats = oracle_formats(params, xs, args.n_bits)
        t_one = oracle_sample_step(params, xs, formats, args.n_bits)
        n_img = int(max(1, min(8, 12.0 / max(t_one, 1e-3))))
        xs = wl.vgg16_input(n_img, seed=100)
        t_s = oracle_sample_step(params, xs, formats, args.n_bits)
        cpu_baseline = {"value": n_img / t_s, "unit": "images/s", "cores": orc.num_threads(), "kind": "oracle",
                        "sample": f"{n_img} image(s) of the same VGG16 {args.n_bits}-bit forward "
                                  f"(whole stack, fixed formats), {t_s:.1f} s",
                        "effective_tops": 2.0 * wl.vgg16_macs_per_image() * n_img / t_s / 1e12,
                        "gmac_per_s": wl.vgg16_macs_per_image() * n_img / t_s / 1e9,
                        "compiler_flags": orc.BUILD_FLAGS, "single_thread": oracle_single_thread()}

    line = {
        "metric": METRIC, "value": ips, "unit": "images/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": f"int{args.n_bits}", "data": "synthetic",
        "effective_tops": eff_tops,
        "pct_of_int8_peak": {"nominal_4500_div_planes": 100.0 * eff_tops / (INT8_NOMINAL_TOPS / planes),
                             "int8_probe_div_planes": 100.0 * eff_tops / peak},
        "config": {"workload": f"VGG16 full forward, {args.n_bits}-bit weights and activations, batch {batch} "
                               "per GPU, 224x224x3 N(0,1) inputs, He-normal weights, per-layer decimal points "
                               "from range measurement; step includes input range + LPAct and per-forward "
                               "weight/bias quantization",
                   "global_batch": batch * world, "n_bits": args.n_bits,
                   "l2": "activations and weights touched per step (about 2.5 GB) exceed the 126 MB L2; "
                         "no explicit flush"},
        "clocks": clocks, "gpu_launches": launches_step * args.steps,
        "e2e": {"value": e2e_ips, "unit": "images/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps,
                "note": "every step copies the batch (the same pinned host buffer each time) to the device and "
                        "reads the logits back; the copy of step i+1 runs on a second stream under step i, and "
                        "this loop records no per-layer events, which is why it can come out ahead of `value`"},
        "roofline": roofline, "streaming": streaming, "modes": side, "cpu_baseline": cpu_baseline,
        "layers": layer_table, "sparsity": sparsity, "saturations": sat,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# one layer or one streaming kernel alone (`--kernel`): the small cases the ncu captures use
# ---------------------------------------------------------------------------------------------
def run_kernel(args):
    import math

    import torch

    from paper_1711_04713_b200 import binding as B
    from paper_1711_04713_b200 import build as bld

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py --kernel needs a CUDA device")
    bld.build_library()
    B.load()
    apply_overrides(B, args)
    a = args
    peaks = read_peaks()
    g = torch.Generator(device="cuda").manual_seed(a.seed)

    def quantized(x, outer, inner, c_stride):
        mx = torch.zeros(1, dtype=torch.float32, device="cuda")
        fmt = torch.zeros(2, dtype=torch.int32, device="cuda")
        B.adaption_measure_range(x, a.n_bits, mx, fmt)
        q = B.QTensor.empty(outer, inner, a.n_bits, int(fmt.cpu()[1]), c_stride)
        B.adaption_quantize(x, outer, inner, q)
        return q

    def output_format(run, fx, fw):
        st = B.new_stats()
        run(B.MODE_RANGE, None, st)
        s = B.read_stats(st)
        if s.status != 0:
            raise B.AdaptionError(s.status, "range pass")
        return B.adaption_choose_frac_bits_from_acc(int(s.max_abs_acc), fx + fw, a.n_bits)

    if a.kernel == "conv":
        cs = B.pad_to(a.C, 32)
        x = torch.randn(a.N * a.H * a.H, a.C, device="cuda", generator=g).clamp_(min=0)
        w = torch.randn(a.K * a.R * a.R, a.C, device="cuda", generator=g) * math.sqrt(2.0 / (a.R * a.R * a.C))
        xq, wq = quantized(x, a.N * a.H * a.H, a.C, cs), quantized(w, a.K * a.R * a.R, a.C, cs)
        shp = B.conv_shape(a.N, a.H, a.H, a.C, a.K, a.R, a.R, a.pad, a.stride)
        OH = (a.H + 2 * a.pad - a.R) // a.stride + 1
        pooled = bool(a.pool)
        y = None
        if pooled:
            y = B.QTensor.empty(a.N * (OH // 2) ** 2, a.K, a.n_bits, 0, B.pad_to(a.K, 32))
            need = B.adaption_lp_conv_pool_workspace_bytes(shp, xq.fmt(), wq.fmt(), y.fmt(), cs, y.c_stride, a.algo)
        else:
            need = B.adaption_lp_conv_workspace_bytes(shp, xq.fmt(), wq.fmt(), cs, a.algo)
        ws = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None
        ws_r = ws
        if pooled:
            nr = B.adaption_lp_conv_workspace_bytes(shp, xq.fmt(), wq.fmt(), cs, a.algo)
            ws_r = torch.empty(nr, dtype=torch.uint8, device="cuda") if nr else None

        def run(mode, yy, st):
            if pooled and mode == B.MODE_REQUANT:
                B.adaption_lp_conv_pool_fwd(shp, xq, wq, None, 0, True, a.algo, yy, st, ws, B.PHASE_CONV)
            else:
                B.adaption_lp_conv_fwd(shp, xq, wq, None, 0, True, mode, a.algo, yy, st, ws_r)

        f_out = output_format(run, xq.frac_bits, wq.frac_bits)
        if pooled:
            y.frac_bits = f_out
        else:
            y = B.QTensor.empty(a.N * OH * OH, a.K, a.n_bits, f_out, B.pad_to(a.K, 32))
        st = B.new_stats()
        ms = _time_ms(torch, lambda: run(B.MODE_REQUANT, y, st), a.iters)
        if B.read_stats(st).status != 0:
            raise B.AdaptionError(B.read_stats(st).status, "conv")
        macs = a.N * OH * OH * a.K * a.R * a.R * a.C
        planes = 4.0 if a.n_bits > 8 else 1.0
        out = {"kernel": "conv", "shape": [a.N, a.H, a.H, a.C, a.K, a.R], "n_bits": a.n_bits, "ms": ms,
               "tops": 2.0 * macs / (ms / 1e3) / 1e12, "gmac": macs / 1e9, "workspace_bytes": need,
               "pooled_store": pooled,
               "frac_of_nominal_int8": 2.0 * macs / (ms / 1e3) / 1e12 / (INT8_NOMINAL_TOPS / planes)}
    elif a.kernel == "ip":
        x = torch.randn(a.B, a.Kin, device="cuda", generator=g).clamp_(min=0)
        w = torch.randn(a.O, a.Kin, device="cuda", generator=g) * math.sqrt(2.0 / a.Kin)
        cs = B.pad_to(a.Kin, 16)
        xq, wq = quantized(x, a.B, a.Kin, cs), quantized(w, a.O, a.Kin, cs)
        need = B.adaption_lp_ip_workspace_bytes(a.B, a.Kin, a.O, xq.fmt(), wq.fmt(), a.algo)
        ws = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None

        def run(mode, yy, st):
            B.adaption_lp_ip_fwd(a.B, a.Kin, a.O, xq, wq, None, 0, True, mode, a.algo, yy, st, ws)

        f_out = output_format(run, xq.frac_bits, wq.frac_bits)
        y = B.QTensor.empty(a.B, a.O, a.n_bits, f_out)
        st = B.new_stats()
        ms = _time_ms(torch, lambda: run(B.MODE_REQUANT, y, st), a.iters)
        macs = a.B * a.Kin * a.O
        bytes_w = a.O * a.Kin * (2 if a.n_bits > 8 else 1)
        out = {"kernel": "ip", "shape": [a.B, a.Kin, a.O], "n_bits": a.n_bits, "ms": ms,
               "tops": 2.0 * macs / (ms / 1e3) / 1e12, "weight_gbs": bytes_w / (ms / 1e3) / 1e9,
               "frac_of_hbm": bytes_w / (ms / 1e3) / 1e9 / peaks["hbm_gbs"], "workspace_bytes": need}
    elif a.kernel == "peak":
        sms = torch.cuda.get_device_properties(0).multi_processor_count
        out = {"kernel": "peak", "sms": sms, "configs": []}
        n = 4096
        for pair, bn, ce in [(False, 64, 0), (False, 128, 0), (False, 256, 0), (True, 64, 0), (True, 128, 0),
                             (True, 256, 0), (False, 128, 4), (False, 128, 1), (True, 128, 4), (True, 128, 1)]:
            cyc = torch.zeros(max(sms, 148), dtype=torch.int64, device="cuda")
            st = torch.zeros(1, dtype=torch.int32, device="cuda")
            ms = _time_ms(torch, lambda: B.adaption_probe_i8_peak(bn, pair, n, cyc, st, ce), max(a.iters, 3))
            if int(st.cpu()[0]) != 0:
                raise B.AdaptionError(int(st.cpu()[0]), "peak probe")
            c = cyc.cpu()
            units = sms // 2 if pair else sms
            macs = units * 4 * n * (256 if pair else 128) * bn * 32
            out["configs"].append({"pair": pair, "bn": bn, "commit_every": ce,
                                   "cycles_per_mma": float(c[c > 0].double().mean()) / (4 * n),
                                   "int8_tops": 2.0 * macs / (ms / 1e3) / 1e12, "ms": ms})
        out["long_run"] = int8_probe(B, torch, 0)
    elif a.kernel == "streaming":
        out = {"kernel": "streaming", "hbm_gbs": peaks["hbm_gbs"],
               "streaming": streaming_kernels(B, torch, peaks["hbm_gbs"], a.numel, a.iters)}
    else:
        inner = a.inner
        outer = a.numel // inner
        n = outer * inner
        x = torch.randn(outer, inner, device="cuda", generator=g)
        pb = 2 if a.n_bits > 8 else 1
        if a.kernel == "hist":
            hist = B.new_hist()
            ms = _time_ms(torch, lambda: B.adaption_bit_histogram(x, hist), a.iters)
            nbytes = 4 * n
        elif a.kernel == "squantize":
            q = B.QTensor.empty(outer, inner, a.n_bits, a.n_bits - 3)
            st = B.new_stats()
            ms = _time_ms(torch, lambda: B.adaption_quantize_stochastic(x, outer, inner, q, 42, False, None, st), a.iters)
            nbytes = (4 + pb) * n
        elif a.kernel == "quantize":
            q = B.QTensor.empty(outer, inner, a.n_bits, a.n_bits - 3)
            st = B.new_stats()
            ms = _time_ms(torch, lambda: B.adaption_quantize(x, outer, inner, q, None, B.ROUND_DETERMINISTIC, st), a.iters)
            nbytes = (4 + pb) * n
        else:
            raise SystemExit(f"unknown kernel {a.kernel}")
        out = {"kernel": a.kernel, "numel": n, "n_bits": a.n_bits, "ms": ms, "gbs": nbytes / (ms / 1e3) / 1e9,
               "frac_of_hbm": nbytes / (ms / 1e3) / 1e9 / peaks["hbm_gbs"], "algorithmic_bytes": nbytes}
    print(json.dumps(out), flush=True)


def apply_overrides(B, args):
    for kv in args.set:
        name, _, value = kv.partition("=")
        B.adaption_debug_set(name, int(value))


def respawn_ranks(args) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script, one per GPU."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--n-bits", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the side measurements (other modes, streaming kernels)")
    ap.add_argument("--event-every", type=int, default=4,
                    help="record per-layer CUDA events on every n-th timed step (roofline durations)")
    # one layer or one streaming kernel alone
    ap.add_argument("--kernel", default=None,
                    choices=["conv", "ip", "peak", "streaming", "quantize", "squantize", "hist"])
    ap.add_argument("--N", type=int, default=8)
    ap.add_argument("--H", type=int, default=28)
    ap.add_argument("--C", type=int, default=512)
    ap.add_argument("--K", type=int, default=512)
    ap.add_argument("--R", type=int, default=3)
    ap.add_argument("--pad", type=int, default=1)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--pool", type=int, default=0, help="conv: store through the fused 2x2 max-pool call")
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--Kin", type=int, default=25088)
    ap.add_argument("--O", type=int, default=4096)
    ap.add_argument("--numel", type=int, default=1 << 28)
    ap.add_argument("--inner", type=int, default=256)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--algo", type=int, default=0)
    ap.add_argument("--set", action="append", default=[], metavar="NAME=VALUE",
                    help="experiment override of a tile heuristic (adaption_debug_set), e.g. --set pdl=0")
    args = ap.parse_args()
    if args.kernel is not None:
        run_kernel(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(respawn_ranks(args))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
