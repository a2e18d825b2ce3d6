"""Seeded synthetic inputs for the GEMM + all-scatter path and the heap microbenchmarks.

This module only draws numbers.  It holds none of the method's arithmetic (no GEMM, no
scatter, no flag logic) so that both the CPU oracle's tests and the CUDA path's tests can be
fed the very same 16-bit arrays without sharing any code of the method itself.

Generator: a counter-based 64-bit mixer.  Element ``i`` of stream ``q`` under seed ``s`` depends
only on ``(s, q, i)``, so any row range of a huge matrix can be produced on its own (the oracle
needs only the rows of a few sampled tiles).

    key   = mix64(s * 0x9E3779B97F4A7C15 + mix64(q + 0xD1B54A32D192ED03))
    x(i)  = mix64(key + i * 0x9E3779B97F4A7C15)
    u(i)  = (x(i) >> 11) * 2**-53                                  in [0, 1)
    uniform[-1,1):   2 u - 1
    normal(0, sd):   sd * sqrt(-2 ln(1 - u_q(i))) * cos(2 pi u_{q + 2**31}(i))     (Box-Muller)

Values are rounded float64 -> float32 (numpy) -> fp16 (numpy) or bf16 (torch), all
round-to-nearest-even library casts; the resulting uint16 bit patterns *are* the inputs.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

SEED0 = 251112500  # seeds used by configs: SEED0 + config index

STREAM_A = 0          # A
STREAM_B0 = 1         # B_r uses STREAM_B0 + r
STREAM_BIAS = 100     # bias
STREAM_PAYLOAD0 = 200  # payload of rank r uses STREAM_PAYLOAD0 + r

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_QOFF = np.uint64(0xD1B54A32D192ED03)
_CHUNK = 1 << 22


def _mix64(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.uint64, copy=True)
    x ^= x >> np.uint64(30)
    x *= _M1
    x ^= x >> np.uint64(27)
    x *= _M2
    x ^= x >> np.uint64(31)
    return x


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        q = _mix64(np.array([np.uint64(stream & 0xFFFFFFFFFFFFFFFF) + _QOFF], dtype=np.uint64))
        k = _mix64(np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _GOLD + q[0]], dtype=np.uint64))
    return k[0]


def raw_u64(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """x(i) for i in [start, start+count)."""
    with np.errstate(over="ignore"):
        i = np.arange(start, start + count, dtype=np.uint64)
        return _mix64(_key(seed, stream) + i * _GOLD)


def unit(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """u(i) in [0,1) as float64."""
    return (raw_u64(seed, stream, start, count) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def _values(seed: int, stream: int, start: int, count: int, dist: str) -> np.ndarray:
    if dist == "uniform":          # uniform[-1, 1)
        return 2.0 * unit(seed, stream, start, count) - 1.0
    if dist == "normal002":        # normal(0, 0.02)
        u1 = unit(seed, stream, start, count)
        u2 = unit(seed, stream + (1 << 31), start, count)
        return 0.02 * np.sqrt(-2.0 * np.log1p(-u1)) * np.cos(2.0 * np.pi * u2)
    if dist.startswith("ternary"):  # {-1, 0, +1}; "ternary:0.25" = P(non-zero)
        density = float(dist.split(":")[1]) if ":" in dist else 0.25
        u = unit(seed, stream, start, count)
        s = raw_u64(seed, stream + (1 << 31), start, count) & np.uint64(1)
        return np.where(u < density, np.where(s == 1, 1.0, -1.0), 0.0)
    if dist.startswith("smallint"):  # integers in [-k, k]; "smallint:3"
        k = int(dist.split(":")[1]) if ":" in dist else 3
        x = raw_u64(seed, stream, start, count) >> np.uint64(33)
        return (x % np.uint64(2 * k + 1)).astype(np.float64) - float(k)
    raise ValueError(f"unknown distribution {dist!r}")


def to16(values: np.ndarray, dtype: str) -> np.ndarray:
    """float64 -> float32 -> fp16/bf16 bit patterns (uint16), library RNE casts."""
    f32 = np.ascontiguousarray(values, dtype=np.float64).astype(np.float32)
    if dtype == "fp16":
        return f32.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        t = torch.from_numpy(f32).to(torch.bfloat16)
        return t.view(torch.int16).numpy().view(np.uint16)
    raise ValueError(f"unknown dtype {dtype!r}")


def matrix(seed: int, stream: int, rows: int, cols: int, dist: str, dtype: str,
           row_begin: int = 0, row_end: int | None = None) -> np.ndarray:
    """Rows [row_begin, row_end) of a row-major ``rows x cols`` matrix as uint16 bit patterns.

    Element (r, c) is element ``r*cols + c`` of the stream, whatever range is asked for.
    """
    if row_end is None:
        row_end = rows
    assert 0 <= row_begin <= row_end <= rows
    n = (row_end - row_begin) * cols
    out = np.empty(n, dtype=np.uint16)
    base = row_begin * cols

    def fill(off: int):
        cnt = min(_CHUNK, n - off)
        out[off:off + cnt] = to16(_values(seed, stream, base + off, cnt, dist), dtype)

    offsets = range(0, n, _CHUNK)
    if len(offsets) > 1:       # chunks are independent (counter-based): generate them on several host threads
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
            list(pool.map(fill, offsets))
    else:
        for off in offsets:
            fill(off)
    return out.reshape(row_end - row_begin, cols)


def vector(seed: int, stream: int, n: int, dist: str, dtype: str) -> np.ndarray:
    return matrix(seed, stream, 1, n, dist, dtype)[0]


def payload_bytes(seed: int, stream: int, nbytes: int) -> np.ndarray:
    """Random bytes (any fp16 bit pattern may occur, NaNs included: the payload is bytes only)."""
    n8 = (nbytes + 7) // 8
    out = np.empty(n8, dtype=np.uint64)
    for off in range(0, n8, _CHUNK):
        cnt = min(_CHUNK, n8 - off)
        out[off:off + cnt] = raw_u64(seed, stream, off, cnt)
    return out.view(np.uint8)[:nbytes].copy()


def gemm_inputs(seed: int, world: int, M: int, N: int, K: int, dist: str, dtype: str):
    """A [M,K] and the W shards B_r [N/W, K] (K contiguous) as uint16 arrays."""
    assert N % world == 0
    nl = N // world
    A = matrix(seed, STREAM_A, M, K, dist, dtype)
    Bs = [matrix(seed, STREAM_B0 + r, nl, K, dist, dtype) for r in range(world)]
    return A, Bs
