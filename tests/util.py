"""Test helpers: move canonical integers between numpy and device byte planes (no arithmetic of
the method beyond the definition q = 256*hi + lo used to lay test data out)."""
import numpy as np
import torch

from paper_1711_04713_b200 import binding as B


def to_qtensor(q: np.ndarray, n_bits: int, frac_bits: int, c_stride: int | None = None,
               with_q16: bool = False) -> B.QTensor:
    q = np.ascontiguousarray(q, dtype=np.int16)
    inner = q.shape[-1]
    outer = q.size // inner
    cs = B.pad_to(inner, 16) if c_stride is None else c_stride
    padded = np.zeros((outer, cs), dtype=np.int16)
    padded[:, :inner] = q.reshape(outer, inner)
    qt = B.QTensor.empty(outer, inner, n_bits, frac_bits, cs, with_q16)
    if n_bits > 8:
        qt.hi.copy_(torch.from_numpy((padded >> 8).astype(np.int8).ravel()))
        qt.lo.copy_(torch.from_numpy((padded & 255).astype(np.uint8).ravel()))
    else:
        qt.lo.copy_(torch.from_numpy(padded.astype(np.int8).view(np.uint8).ravel()))
    return qt


def from_qtensor(qt: B.QTensor) -> np.ndarray:
    return qt.to_int16().numpy()


def q16_of(qt: B.QTensor) -> np.ndarray:
    return qt.q16.view(qt.outer, qt.c_stride)[:, :qt.inner].cpu().numpy()


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def stats_tuple(stats: torch.Tensor):
    s = B.read_stats(stats)
    return int(s.zeros), int(s.sat_pos), int(s.sat_neg)
