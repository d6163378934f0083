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


def test_single_process_paths_need_no_process_group():
    assert replicas.agree_on_range(123) == 123
    assert replicas.sum_counters(1, 2, 3) == (1, 2, 3)
    assert replicas.slowest_rank_ms(4.5) == 4.5
    assert replicas.shard_seed(100, 3) == 103
