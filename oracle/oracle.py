"""ctypes front end of the CPU oracle in ``iris_oracle.cpp``.

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's cpu_baseline
leg.  It never touches the CUDA library.  Everything here is argument marshalling plus the
composition "GEMM block -> all-scatter -> flags" that mirrors the order of the paper's listings;
the arithmetic lives in the C++ file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

F16, BF16 = 0, 1
DTYPES = {"fp16": F16, "bf16": BF16}
TILE = 128

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "iris_oracle.cpp")
_LIB = os.path.join(_HERE, "build", "libiris_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            i64, u64, i32, u16p, u8p = C.c_int64, C.c_uint64, C.c_int32, C.POINTER(C.c_uint16), C.POINTER(C.c_uint8)
            L.orc_hw_threads.restype = C.c_int
            L.orc_decode1.restype = C.c_double
            L.orc_decode1.argtypes = [C.c_int, C.c_uint16]
            L.orc_encode1.restype = C.c_uint16
            L.orc_encode1.argtypes = [C.c_int, C.c_double]
            L.orc_decode.argtypes = [C.c_int, u16p, i64, C.POINTER(C.c_double)]
            L.orc_encode.argtypes = [C.c_int, C.POINTER(C.c_double), i64, u16p]
            L.orc_translate.argtypes = [C.POINTER(u64), C.c_int, u64, u64, C.c_int, C.c_int, C.POINTER(u64)]
            L.orc_gemm_block.argtypes = [C.c_int, u16p, C.POINTER(u16p), i64, i64, i64, C.c_int, i64, i64, i64, i64,
                                         u16p, C.POINTER(C.c_double), C.c_int]
            L.orc_all_scatter.argtypes = [u8p, C.c_int, u64, u64, i64, i64, u16p]
            L.orc_num_tiles.restype = i64
            L.orc_num_tiles.argtypes = [i64, i64, C.c_int]
            L.orc_publish_flags.argtypes = [u8p, C.c_int, u64, u64, i64, i32]
            L.orc_consume_locks.argtypes = [u8p, C.c_int, u64, u64, i64, i64]
            for f in (L.orc_put, L.orc_get):
                f.argtypes = [u8p, C.c_int, u64, u64, u64, i64, i64, i64, i64, C.c_int, C.c_int]
            L.orc_atomic_add.argtypes = [u8p, C.c_int, u64, u64, i64, i64, C.c_int, i32, C.POINTER(i32)]
            L.orc_atomic_cas.argtypes = [u8p, C.c_int, u64, u64, i64, i64, C.c_int, i32, i32, C.POINTER(i32)]
            L.orc_atomic_add_u64.argtypes = [u8p, C.c_int, u64, u64, i64, i64, C.c_int, u64, C.POINTER(u64)]
            L.orc_atomic_cas_u64.argtypes = [u8p, C.c_int, u64, u64, i64, i64, C.c_int, u64, u64, C.POINTER(u64)]
            L.orc_atomic_rmw.argtypes = [u8p, C.c_int, u64, C.c_int, u64, i64, i64, C.c_int, i32, C.POINTER(i32)]
            L.orc_copy.argtypes = [u8p, C.c_int, u64, u64, u64, i64, i64, i64, i64, C.c_int, C.c_int]
            L.orc_consume_bias.argtypes = [u8p, C.c_int, u64, C.c_int, u64, u64, i64, i64, u16p]
            L.orc_all_store.argtypes = [u8p, C.c_int, u64, u64, u64, u64, u64, u64, i32]
            _lib = L
    return _lib


def _u16p(a: np.ndarray):
    assert a.dtype == np.uint16 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_uint16))


def _u8p(a: np.ndarray):
    assert a.dtype == np.uint8 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_uint8))


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what}: error {rc}")


def hw_threads() -> int:
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else lib().orc_hw_threads()


def decode(bits: np.ndarray, dtype: str) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    lib().orc_decode(DTYPES[dtype], _u16p(bits.reshape(-1)), bits.size, out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


def encode(values: np.ndarray, dtype: str) -> np.ndarray:
    values = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty(values.shape, dtype=np.uint16)
    lib().orc_encode(DTYPES[dtype], values.ctypes.data_as(C.POINTER(C.c_double)), values.size, _u16p(out.reshape(-1)))
    return out


def translate(bases, bytes_per_rank: int, ptr: int, from_rank: int, to_rank: int) -> int:
    arr = (C.c_uint64 * len(bases))(*bases)
    out = C.c_uint64(0)
    rc = lib().orc_translate(arr, len(bases), bytes_per_rank, ptr, from_rank, to_rank, C.byref(out))
    if rc == -1:
        raise ValueError("bad rank")
    if rc == -2:
        raise IndexError("pointer outside the source rank's heap")
    return out.value


def gemm_block(A: np.ndarray, Bs, dtype: str, m0=0, m1=None, n0=0, n1=None, threads=None, want_exact=False):
    """Rounded (and optionally unrounded fp64) block [m0,m1) x [n0,n1) of A . [B_0|...|B_{W-1}]."""
    M, K = A.shape
    W = len(Bs)
    nl = Bs[0].shape[0]
    N = W * nl
    m1 = M if m1 is None else m1
    n1 = N if n1 is None else n1
    for b in Bs:
        assert b.shape == (nl, K)
    ptrs = (C.POINTER(C.c_uint16) * W)(*[_u16p(b) for b in Bs])
    c16 = np.empty((m1 - m0, n1 - n0), dtype=np.uint16)
    c64 = np.empty((m1 - m0, n1 - n0), dtype=np.float64) if want_exact else None
    rc = lib().orc_gemm_block(DTYPES[dtype], _u16p(A), ptrs, M, N, K, W, m0, m1, n0, n1, _u16p(c16.reshape(-1)),
                              c64.ctypes.data_as(C.POINTER(C.c_double)) if want_exact else None,
                              threads or hw_threads())
    _check(rc, "gemm_block")
    return (c16, c64) if want_exact else c16


def num_tiles(M: int, N: int, world: int) -> int:
    return int(lib().orc_num_tiles(M, N, world))


def tile_rect(t: int, M: int, N: int, world: int):
    """(m0, m1, n0, n1) of publication tile t in global coordinates."""
    nl = N // world
    tnl = -(-nl // TILE)
    tn_all = world * tnl
    tm, rem = divmod(t, tn_all)
    r, j = divmod(rem, tnl)
    m0, n0 = tm * TILE, r * nl + j * TILE
    return m0, min(M, m0 + TILE), n0, min((r + 1) * nl, n0 + TILE)


class HeapImage:
    """Host model of the emulated symmetric heap: W slots of bytes_per_rank bytes."""

    def __init__(self, world: int, bytes_per_rank: int, fill: int = 0):
        self.world, self.bpr = world, bytes_per_rank
        self.mem = np.full(world * bytes_per_rank, fill, dtype=np.uint8)

    def slot(self, r: int) -> np.ndarray:
        return self.mem[r * self.bpr:(r + 1) * self.bpr]

    def view(self, r: int, off: int, nbytes: int, dtype=np.uint8) -> np.ndarray:
        return self.slot(r)[off:off + nbytes].view(dtype)

    # --- Table 3 operations -------------------------------------------------------------
    def put(self, src_off, dst_off, rows, row_bytes, src_pitch, dst_pitch, from_rank, to_rank):
        _check(lib().orc_put(_u8p(self.mem), self.world, self.bpr, src_off, dst_off, rows, row_bytes, src_pitch,
                             dst_pitch, from_rank, to_rank), "put")

    def get(self, src_off, dst_off, rows, row_bytes, src_pitch, dst_pitch, from_rank, to_rank):
        _check(lib().orc_get(_u8p(self.mem), self.world, self.bpr, src_off, dst_off, rows, row_bytes, src_pitch,
                             dst_pitch, from_rank, to_rank), "get")

    def atomic_add(self, off, count, stride, to_rank, val) -> np.ndarray:
        old = np.empty(count, dtype=np.int32)
        _check(lib().orc_atomic_add(_u8p(self.mem), self.world, self.bpr, off, count, stride, to_rank, val,
                                    old.ctypes.data_as(C.POINTER(C.c_int32))), "atomic_add")
        return old

    def atomic_cas(self, off, count, stride, to_rank, cmp, val) -> np.ndarray:
        old = np.empty(count, dtype=np.int32)
        _check(lib().orc_atomic_cas(_u8p(self.mem), self.world, self.bpr, off, count, stride, to_rank, cmp, val,
                                    old.ctypes.data_as(C.POINTER(C.c_int32))), "atomic_cas")
        return old

    def atomic_add_u64(self, off, count, stride, to_rank, val) -> np.ndarray:
        old = np.empty(count, dtype=np.uint64)
        _check(lib().orc_atomic_add_u64(_u8p(self.mem), self.world, self.bpr, off, count, stride, to_rank, val,
                                        old.ctypes.data_as(C.POINTER(C.c_uint64))), "atomic_add_u64")
        return old

    def atomic_cas_u64(self, off, count, stride, to_rank, cmp, val) -> np.ndarray:
        old = np.empty(count, dtype=np.uint64)
        _check(lib().orc_atomic_cas_u64(_u8p(self.mem), self.world, self.bpr, off, count, stride, to_rank, cmp, val,
                                        old.ctypes.data_as(C.POINTER(C.c_uint64))), "atomic_cas_u64")
        return old

    ATOMIC_OPS = {"add": 0, "xchg": 1, "and": 2, "or": 3, "xor": 4, "min": 5, "max": 6}

    def atomic_rmw(self, op: str, off, count, stride, to_rank, val) -> np.ndarray:
        old = np.empty(count, dtype=np.int32)
        _check(lib().orc_atomic_rmw(_u8p(self.mem), self.world, self.bpr, self.ATOMIC_OPS[op], off, count, stride, to_rank, val,
                                    old.ctypes.data_as(C.POINTER(C.c_int32))), "atomic_rmw")
        return old

    def copy(self, src_off, dst_off, rows, row_bytes, src_pitch, dst_pitch, from_rank, to_rank):
        """copy between any two ranks (Table 3); load/store to a buffer outside the heap are the caller's slices of this."""
        _check(lib().orc_copy(_u8p(self.mem), self.world, self.bpr, src_off, dst_off, rows, row_bytes, src_pitch, dst_pitch,
                              from_rank, to_rank), "copy")

    # --- GEMM + all-scatter -------------------------------------------------------------
    def all_scatter(self, c_off: int, c_full: np.ndarray):
        M, N = c_full.shape
        _check(lib().orc_all_scatter(_u8p(self.mem), self.world, self.bpr, c_off, M, N,
                                     _u16p(np.ascontiguousarray(c_full).reshape(-1))), "all_scatter")

    def publish_flags(self, flag_off: int, ntiles: int, epoch: int):
        _check(lib().orc_publish_flags(_u8p(self.mem), self.world, self.bpr, flag_off, ntiles, epoch), "publish_flags")

    def consume_locks(self, lock_off: int, M: int, N: int):
        _check(lib().orc_consume_locks(_u8p(self.mem), self.world, self.bpr, lock_off, M, N), "consume_locks")

    def gemm_all_scatter(self, A, Bs, dtype: str, c_off: int, flag_off: int, epoch: int, lock_off=None, threads=None):
        """Expected heap after gemm_all_scatter in any mode (lock_off given: workgroup-specialised)."""
        M, N = A.shape[0], len(Bs) * Bs[0].shape[0]
        c_full = gemm_block(A, Bs, dtype, threads=threads)
        self.all_scatter(c_off, c_full)
        self.publish_flags(flag_off, num_tiles(M, N, self.world), epoch)
        if lock_off is not None:
            self.consume_locks(lock_off, M, N)
        return c_full

    def consume_bias(self, dtype: str, c_off: int, out_off: int, M: int, N: int, bias: np.ndarray):
        _check(lib().orc_consume_bias(_u8p(self.mem), self.world, self.bpr, DTYPES[dtype], c_off, out_off, M, N,
                                      _u16p(np.ascontiguousarray(bias))), "consume_bias")

    def all_store(self, payload_off, recv_off, flag_off, S, tile_bytes, epoch):
        _check(lib().orc_all_store(_u8p(self.mem), self.world, self.bpr, payload_off, recv_off, flag_off, S,
                                   tile_bytes, epoch), "all_store")


def consume_bias_rows(c_rows: np.ndarray, bias: np.ndarray, dtype: str) -> np.ndarray:
    """OUT rows for given C rows (one slot): the consumer definition on a standalone array."""
    M, N = c_rows.shape
    img = HeapImage(1, 2 * M * N * 2)
    img.view(0, 0, M * N * 2, np.uint16)[:] = np.ascontiguousarray(c_rows).reshape(-1)
    img.consume_bias(dtype, 0, M * N * 2, M, N, bias)
    return img.view(0, M * N * 2, M * N * 2, np.uint16).reshape(M, N).copy()
