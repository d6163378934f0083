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


# ---- canary guards: a stand-in for a memory checker -----------------------------------------
GUARD_BYTES = 4096
GUARD_BYTE = 0xC7


class Guards:
    """Allocates device buffers with GUARD_BYTES of a fixed byte in front of and behind each one
    (same allocation), so that a kernel writing just outside a buffer it was given is caught by
    ``check()`` instead of landing unseen in allocator slack."""

    def __init__(self):
        self._bufs = []

    def alloc(self, nbytes: int, dtype=torch.uint8, fill: int | None = None) -> torch.Tensor:
        item = torch.empty((), dtype=dtype).element_size()
        assert GUARD_BYTES % item == 0
        raw = torch.full((nbytes + 2 * GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device="cuda")
        body = raw[GUARD_BYTES:GUARD_BYTES + nbytes]
        if fill is not None:
            body.fill_(fill)
        self._bufs.append((raw, nbytes))
        return body.view(dtype)

    def qtensor(self, outer: int, inner: int, n_bits: int, frac_bits: int = 0, c_stride: int | None = None,
                with_q16: bool = False, fill: int | None = 0x3C) -> B.QTensor:
        cs = B.pad_to(inner, 16) if c_stride is None else c_stride
        n = outer * cs
        lo = self.alloc(n, torch.uint8, fill)
        hi = self.alloc(n, torch.int8, fill) if n_bits > 8 else None
        q16 = self.alloc(2 * n, torch.int16, fill) if with_q16 else None
        return B.QTensor(outer, inner, cs, n_bits, frac_bits, lo, hi, q16)

    def check(self):
        torch.cuda.synchronize()
        for raw, nbytes in self._bufs:
            front = raw[:GUARD_BYTES]
            back = raw[GUARD_BYTES + nbytes:]
            assert bool((front == GUARD_BYTE).all()), "write in front of a buffer"
            assert bool((back == GUARD_BYTE).all()), "write behind a buffer"
