"""Helpers for the GPU parity tests: a heap backed by a torch byte tensor (so the tests can read every
byte back), upload of the seeded 16-bit inputs, and comparison against the oracle's heap image."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2511_12500_b200 as iris

SENTINEL = 0xA5


def align(x: int, a: int = 256) -> int:
    return (x + a - 1) // a * a


class GpuHeap:
    def __init__(self, world: int, bytes_per_rank: int, fill: int = SENTINEL):
        self.world, self.bpr = world, bytes_per_rank
        self.mem = torch.full((world * bytes_per_rank,), fill, dtype=torch.uint8, device="cuda")
        self.h = iris.iris_heap_create(world, bytes_per_rank, external_base=self.mem.data_ptr())
        self.bases = iris.iris_heap_bases(self.h)

    def close(self):
        if self.h:
            iris.iris_heap_destroy(self.h)
            self.h = 0

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def addr(self, rank: int, off: int) -> int:
        return self.bases[rank] + off

    def slot(self, r: int) -> torch.Tensor:
        return self.mem[r * self.bpr:(r + 1) * self.bpr]

    def view(self, r: int, off: int, nbytes: int, dtype=torch.uint8) -> torch.Tensor:
        return self.slot(r)[off:off + nbytes].view(dtype)

    def write(self, r: int, off: int, data: np.ndarray):
        b = np.ascontiguousarray(data).view(np.uint8).reshape(-1)
        self.slot(r)[off:off + b.size] = torch.from_numpy(b).cuda()

    def to_host(self) -> np.ndarray:
        torch.cuda.synchronize()
        return self.mem.cpu().numpy()

    def image(self, fill: int = SENTINEL) -> oracle.HeapImage:
        return oracle.HeapImage(self.world, self.bpr, fill=fill)


def dev16(a: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> device tensor (int16 storage; only the address is used)."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def gemm_layout(M: int, N: int, world: int, with_out: bool = False):
    """c_off, flag_off, lock_off, out_off, bytes_per_rank with guard gaps between the regions."""
    nt = max(1, oracle.num_tiles(M, N, world)) if M and N else 1
    c_off = 256
    flag_off = align(c_off + M * N * 2 + 64)
    lock_off = align(flag_off + nt * 4 + 64)
    out_off = align(lock_off + nt * 4 + 64)
    end = out_off + (M * N * 2 if with_out else 0)
    return c_off, flag_off, lock_off, out_off, align(end + 256)


def first_diff(a: np.ndarray, b: np.ndarray) -> str:
    idx = np.flatnonzero(a != b)
    return f"{idx.size} differing bytes, first at {idx[:5].tolist()}" if idx.size else "equal"


def check_tolerance(got16: np.ndarray, ref16: np.ndarray, dtype: str):
    """The stated tolerance: max |gpu - ref| <= 1e-2 (|ref| + 1) elementwise and relative Frobenius error <= 2e-3."""
    g, r = oracle.decode(got16, dtype), oracle.decode(ref16, dtype)
    assert np.all(np.isfinite(g))
    assert np.all(np.abs(g - r) <= 1e-2 * (np.abs(r) + 1.0)), float(np.max(np.abs(g - r)))
    denom = np.linalg.norm(r)
    rel = np.linalg.norm(g - r) / denom if denom > 0 else np.linalg.norm(g - r)
    assert rel <= 2e-3, rel
    return rel
