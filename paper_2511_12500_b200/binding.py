"""Thin ctypes binding of libiris_b200.so: same names as include/iris_b200.h, argument marshalling only.

PyTorch appears here only to obtain device pointers and the current stream.  There is no fallback:
if the shared library is missing or cannot be loaded, importing a symbol raises.
"""
from __future__ import annotations

import ctypes as C
import os

IRIS_OK = 0
IRIS_ERR_ARG, IRIS_ERR_RANGE, IRIS_ERR_NOMEM, IRIS_ERR_CUDA = -1, -2, -3, -4
IRIS_ERR_UNSUPPORTED, IRIS_ERR_TIMEOUT, IRIS_ERR_STATE = -5, -6, -7
IRIS_F16, IRIS_BF16 = 0, 1
DTYPES = {"fp16": IRIS_F16, "bf16": IRIS_BF16}
IRIS_MODE_BULK_SYNCHRONOUS, IRIS_MODE_FUSED_SEQUENTIAL, IRIS_MODE_WORKGROUP_SPECIALIZED = 0, 1, 2
MODES = {"bulk_synchronous": 0, "fused_sequential": 1, "workgroup_specialized": 2}
IRIS_SEM_RELAXED, IRIS_SEM_ACQUIRE, IRIS_SEM_RELEASE, IRIS_SEM_ACQ_REL = 0, 1, 2, 3
IRIS_SCOPE_BLOCK, IRIS_SCOPE_GPU, IRIS_SCOPE_SYS = 0, 1, 2
IRIS_OP_ADD, IRIS_OP_XCHG, IRIS_OP_AND, IRIS_OP_OR, IRIS_OP_XOR, IRIS_OP_MIN, IRIS_OP_MAX = range(7)
ATOMIC_OPS = {"add": 0, "xchg": 1, "and": 2, "or": 3, "xor": 4, "min": 5, "max": 6}
IRIS_B_N_BY_K, IRIS_B_K_BY_N = 0, 1
IRIS_MAX_WORLD = 8
IRIS_TILE = 128

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libiris_b200.so")

# Every symbol include/iris_b200.h declares.
EXPORTS = [
    "iris_last_error", "iris_version", "iris_heap_create", "iris_heap_create_ex", "iris_heap_destroy", "iris_heap_world",
    "iris_heap_bytes_per_rank", "iris_heap_base", "iris_heap_bases", "iris_malloc", "iris_heap_reset", "iris_translate",
    "iris_status_check", "iris_put_tile", "iris_get_tile", "iris_atomic_add", "iris_atomic_cas",
    "iris_atomic_add_contended", "iris_atomic_cas_contended", "iris_flags_fill", "iris_all_store_bench",
    "iris_gemm_all_scatter_ex", "iris_gemm_all_scatter_unfused", "gemm_all_scatter", "iris_gemm_heap_bytes", "iris_heap_epoch", "iris_num_tiles",
    "iris_consume_bias", "iris_consume_bias_ranks", "iris_gemm_all_scatter_host", "iris_gemm_out_offset", "iris_gemm_takeover_stats",
    "iris_gemm_all_scatter_noalloc", "iris_heap_create_from_bases", "iris_heap_local_rank", "iris_ipc_alloc", "iris_ipc_free", "iris_ipc_export",
    "iris_ipc_open", "iris_ipc_close", "iris_atomic_add_u64", "iris_atomic_cas_u64", "iris_copy_tile", "iris_load_tile", "iris_store_tile", "iris_atomic_rmw",
]


class IrisError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"iris error {code}: {msg}")
        self.code = code


class GemmArgs(C.Structure):
    _fields_ = [
        ("A", C.c_void_p), ("B_shards", C.POINTER(C.c_void_p)), ("heap", C.c_void_p),
        ("M", C.c_int), ("N", C.c_int), ("K", C.c_int), ("world", C.c_int), ("mode", C.c_int), ("dtype", C.c_int),
        ("c_off", C.c_uint64), ("flag_off", C.c_uint64), ("lock_off", C.c_uint64),
        ("epoch", C.c_int32), ("comm_ctas", C.c_int), ("max_ctas", C.c_int), ("raster_group", C.c_int),
        ("block_n", C.c_int), ("spin_timeout_ns", C.c_uint64), ("cta_pair", C.c_int), ("static_schedule", C.c_int), ("stream_k", C.c_int), ("wg_tail", C.c_int), ("rank_first", C.c_int), ("rank_count", C.c_int), ("pace_stores", C.c_int),
        ("consumer_bias", C.c_void_p), ("consumer_out_off", C.c_uint64), ("b_layout", C.c_int), ("fuse_tail", C.c_int), ("stage_k", C.c_int),
    ]


_lib = None


def lib() -> C.CDLL:
    """Load the library (no CUDA call is made by loading it)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2511_12500_b200.build` (needs nvcc); there is no fallback")
    L = C.CDLL(LIB_PATH)
    vp, u64, sz, i32, ci = C.c_void_p, C.c_uint64, C.c_size_t, C.c_int32, C.c_int
    L.iris_last_error.restype = C.c_char_p
    L.iris_version.restype = C.c_char_p
    L.iris_heap_create.restype = vp
    L.iris_heap_create.argtypes = [ci, sz]
    L.iris_heap_create_ex.argtypes = [ci, sz, vp, C.POINTER(vp)]
    L.iris_heap_create_from_bases.argtypes = [ci, sz, C.POINTER(u64), ci, C.POINTER(vp)]
    L.iris_heap_local_rank.argtypes = [vp]
    L.iris_ipc_alloc.argtypes = [sz, C.POINTER(vp)]
    L.iris_ipc_free.argtypes = [vp]
    L.iris_ipc_export.argtypes = [vp, C.c_char_p]
    L.iris_ipc_open.argtypes = [C.c_char_p, C.POINTER(vp)]
    L.iris_ipc_close.argtypes = [vp]
    L.iris_heap_destroy.argtypes = [vp]
    L.iris_heap_world.argtypes = [vp]
    L.iris_heap_bytes_per_rank.restype = sz
    L.iris_heap_bytes_per_rank.argtypes = [vp]
    L.iris_heap_base.restype = vp
    L.iris_heap_base.argtypes = [vp, ci]
    L.iris_heap_bases.argtypes = [vp, C.POINTER(u64)]
    L.iris_malloc.argtypes = [vp, sz, sz, C.POINTER(u64)]
    L.iris_heap_reset.argtypes = [vp]
    L.iris_translate.argtypes = [vp, vp, ci, ci, C.POINTER(vp)]
    L.iris_status_check.argtypes = [vp, vp, C.POINTER(i32)]
    for f in (L.iris_put_tile, L.iris_get_tile):
        f.argtypes = [vp, vp, vp, sz, sz, sz, sz, ci, ci, vp]
    L.iris_copy_tile.argtypes = [vp, vp, vp, sz, sz, sz, sz, ci, ci, ci, vp]
    for f in (L.iris_load_tile, L.iris_store_tile):
        f.argtypes = [vp, vp, vp, sz, sz, sz, sz, ci, ci, vp]
    L.iris_atomic_rmw.argtypes = [vp, ci, vp, sz, sz, ci, ci, i32, ci, ci, vp, vp]
    L.iris_atomic_add.argtypes = [vp, vp, sz, sz, ci, ci, i32, ci, ci, vp, vp]
    L.iris_atomic_cas.argtypes = [vp, vp, sz, sz, ci, ci, i32, i32, ci, ci, vp, vp]
    L.iris_atomic_add_u64.argtypes = [vp, vp, sz, sz, ci, ci, u64, ci, ci, vp, vp]
    L.iris_atomic_cas_u64.argtypes = [vp, vp, sz, sz, ci, ci, u64, u64, ci, ci, vp, vp]
    L.iris_atomic_add_contended.argtypes = [vp, vp, sz, ci, ci, i32, ci, ci, vp, vp]
    L.iris_atomic_cas_contended.argtypes = [vp, vp, sz, ci, ci, i32, i32, ci, ci, vp, vp]
    L.iris_flags_fill.argtypes = [vp, u64, sz, i32, vp]
    L.iris_all_store_bench.argtypes = [vp, u64, u64, u64, sz, sz, i32, ci, ci, vp]
    L.iris_gemm_all_scatter_ex.argtypes = [C.POINTER(GemmArgs), vp]
    L.iris_gemm_all_scatter_unfused.argtypes = [C.POINTER(GemmArgs), vp, vp]
    L.gemm_all_scatter.argtypes = [vp, C.POINTER(vp), vp, ci, ci, ci, ci, ci]
    L.iris_gemm_heap_bytes.restype = sz
    L.iris_gemm_heap_bytes.argtypes = [ci, ci, ci]
    L.iris_heap_epoch.restype = i32
    L.iris_heap_epoch.argtypes = [vp]
    L.iris_num_tiles.restype = C.c_int64
    L.iris_num_tiles.argtypes = [ci, ci, ci]
    L.iris_consume_bias.argtypes = [vp, u64, u64, u64, vp, ci, ci, ci, ci, i32, ci, u64, vp]
    L.iris_consume_bias_ranks.argtypes = [vp, u64, u64, u64, vp, ci, ci, ci, ci, ci, ci, i32, ci, u64, vp]
    L.iris_gemm_all_scatter_host.argtypes = [vp, C.POINTER(vp), vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci]
    L.iris_gemm_takeover_stats.argtypes = [vp, C.POINTER(C.c_int32)]
    L.iris_gemm_out_offset.restype = u64
    L.iris_gemm_out_offset.argtypes = [ci, ci, ci]
    L.iris_gemm_all_scatter_noalloc.argtypes = [vp, C.POINTER(vp), C.POINTER(u64), sz, ci, ci, ci, ci, ci, u64, u64, i32, vp]
    _lib = L
    return L


def iris_last_error() -> str:
    return lib().iris_last_error().decode()


def _ck(rc: int) -> int:
    if rc != IRIS_OK:
        raise IrisError(rc, iris_last_error())
    return rc


def _ptr(x) -> int | None:
    """Device/host address of a torch tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _stream(stream) -> int | None:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream


# ---------------------------------------------------------------------------------------------- heap
def iris_heap_create(world: int, bytes_per_rank: int, external_base=None) -> int:
    h = C.c_void_p()
    _ck(lib().iris_heap_create_ex(world, bytes_per_rank, _ptr(external_base), C.byref(h)))
    return h.value


def iris_heap_create_from_bases(world: int, bytes_per_rank: int, bases, local_rank: int) -> int:
    """Heap over several processes: bases[r] = this process's device address of rank r's slot."""
    if len(bases) != world:
        raise ValueError("one base per rank")
    arr = (C.c_uint64 * world)(*[int(b) for b in bases])
    h = C.c_void_p()
    _ck(lib().iris_heap_create_from_bases(world, bytes_per_rank, arr, local_rank, C.byref(h)))
    return h.value


def iris_heap_local_rank(heap: int) -> int:
    return lib().iris_heap_local_rank(heap)


IRIS_IPC_HANDLE_BYTES = 64


def iris_ipc_alloc(nbytes: int) -> int:
    p = C.c_void_p()
    _ck(lib().iris_ipc_alloc(nbytes, C.byref(p)))
    return p.value


def iris_ipc_free(ptr: int):
    _ck(lib().iris_ipc_free(ptr))


def iris_ipc_export(ptr: int) -> bytes:
    buf = C.create_string_buffer(IRIS_IPC_HANDLE_BYTES)
    _ck(lib().iris_ipc_export(ptr, buf))
    return buf.raw


def iris_ipc_open(handle: bytes) -> int:
    if len(handle) != IRIS_IPC_HANDLE_BYTES:
        raise ValueError("an exported handle has IRIS_IPC_HANDLE_BYTES bytes")
    p = C.c_void_p()
    _ck(lib().iris_ipc_open(handle, C.byref(p)))
    return p.value


def iris_ipc_close(ptr: int):
    _ck(lib().iris_ipc_close(ptr))


def iris_heap_destroy(heap: int):
    _ck(lib().iris_heap_destroy(heap))


def iris_heap_world(heap: int) -> int:
    return lib().iris_heap_world(heap)


def iris_heap_bytes_per_rank(heap: int) -> int:
    return lib().iris_heap_bytes_per_rank(heap)


def iris_heap_base(heap: int, rank: int) -> int:
    p = lib().iris_heap_base(heap, rank)
    if not p:
        raise IrisError(IRIS_ERR_ARG, iris_last_error())
    return p


def iris_heap_bases(heap: int) -> list[int]:
    out = (C.c_uint64 * IRIS_MAX_WORLD)()
    _ck(lib().iris_heap_bases(heap, out))
    return list(out[: iris_heap_world(heap)])


def iris_malloc(heap: int, nbytes: int, align: int = 0) -> int:
    off = C.c_uint64()
    _ck(lib().iris_malloc(heap, nbytes, align, C.byref(off)))
    return off.value


def iris_heap_reset(heap: int):
    _ck(lib().iris_heap_reset(heap))


def iris_translate(heap: int, ptr: int, from_rank: int, to_rank: int) -> int:
    out = C.c_void_p()
    _ck(lib().iris_translate(heap, ptr, from_rank, to_rank, C.byref(out)))
    return out.value


def iris_status_check(heap: int, stream=None):
    """Synchronise and raise IrisError(IRIS_ERR_TIMEOUT) if a device-side wait expired."""
    detail = (C.c_int32 * 8)()
    rc = lib().iris_status_check(heap, _stream(stream), detail)
    if rc != IRIS_OK:
        e = IrisError(rc, iris_last_error())
        e.detail = list(detail)
        raise e


# ---------------------------------------------------------------------------------------- tile ops
def iris_put_tile(heap, src, dst, rows, row_bytes, src_pitch, dst_pitch, from_rank, to_rank, stream=None):
    _ck(lib().iris_put_tile(heap, src, dst, rows, row_bytes, src_pitch, dst_pitch, from_rank, to_rank, _stream(stream)))


def iris_get_tile(heap, src, dst, rows, row_bytes, src_pitch, dst_pitch, from_rank, to_rank, stream=None):
    _ck(lib().iris_get_tile(heap, src, dst, rows, row_bytes, src_pitch, dst_pitch, from_rank, to_rank, _stream(stream)))


def iris_copy_tile(heap, src, dst, rows, row_bytes, src_pitch, dst_pitch, cur_rank, from_rank, to_rank, stream=None):
    _ck(lib().iris_copy_tile(heap, src, dst, rows, row_bytes, src_pitch, dst_pitch, cur_rank, from_rank, to_rank, _stream(stream)))


def iris_load_tile(heap, src, out, rows, row_bytes, src_pitch, out_pitch, from_rank, to_rank, stream=None):
    _ck(lib().iris_load_tile(heap, src, _ptr(out), rows, row_bytes, src_pitch, out_pitch, from_rank, to_rank, _stream(stream)))


def iris_store_tile(heap, values, dst, rows, row_bytes, values_pitch, dst_pitch, from_rank, to_rank, stream=None):
    _ck(lib().iris_store_tile(heap, _ptr(values), dst, rows, row_bytes, values_pitch, dst_pitch, from_rank, to_rank, _stream(stream)))


def iris_atomic_rmw(heap, op, ptr, count, stride_bytes, from_rank, to_rank, value, sem=IRIS_SEM_RELAXED, scope=IRIS_SCOPE_GPU,
                    old_out=None, stream=None):
    _ck(lib().iris_atomic_rmw(heap, op, ptr, count, stride_bytes, from_rank, to_rank, value, sem, scope, _ptr(old_out), _stream(stream)))


def iris_atomic_add(heap, ptr, count, stride_bytes, from_rank, to_rank, value, sem=IRIS_SEM_RELAXED,
                    scope=IRIS_SCOPE_GPU, old_out=None, stream=None):
    _ck(lib().iris_atomic_add(heap, ptr, count, stride_bytes, from_rank, to_rank, value, sem, scope, _ptr(old_out), _stream(stream)))


def iris_atomic_cas(heap, ptr, count, stride_bytes, from_rank, to_rank, compare, value, sem=IRIS_SEM_RELAXED,
                    scope=IRIS_SCOPE_GPU, old_out=None, stream=None):
    _ck(lib().iris_atomic_cas(heap, ptr, count, stride_bytes, from_rank, to_rank, compare, value, sem, scope, _ptr(old_out), _stream(stream)))


def iris_atomic_add_u64(heap, ptr, count, stride_bytes, from_rank, to_rank, value, sem=IRIS_SEM_RELAXED,
                        scope=IRIS_SCOPE_GPU, old_out=None, stream=None):
    _ck(lib().iris_atomic_add_u64(heap, ptr, count, stride_bytes, from_rank, to_rank, value, sem, scope, _ptr(old_out), _stream(stream)))


def iris_atomic_cas_u64(heap, ptr, count, stride_bytes, from_rank, to_rank, compare, value, sem=IRIS_SEM_RELAXED,
                        scope=IRIS_SCOPE_GPU, old_out=None, stream=None):
    _ck(lib().iris_atomic_cas_u64(heap, ptr, count, stride_bytes, from_rank, to_rank, compare, value, sem, scope, _ptr(old_out), _stream(stream)))


def iris_atomic_add_contended(heap, ptr, threads, from_rank, to_rank, value, sem=IRIS_SEM_RELAXED, scope=IRIS_SCOPE_GPU,
                              old_out=None, stream=None):
    _ck(lib().iris_atomic_add_contended(heap, ptr, threads, from_rank, to_rank, value, sem, scope, _ptr(old_out), _stream(stream)))


def iris_atomic_cas_contended(heap, ptr, threads, from_rank, to_rank, compare, value_base, sem=IRIS_SEM_RELAXED,
                              scope=IRIS_SCOPE_GPU, old_out=None, stream=None):
    _ck(lib().iris_atomic_cas_contended(heap, ptr, threads, from_rank, to_rank, compare, value_base, sem, scope, _ptr(old_out), _stream(stream)))


def iris_flags_fill(heap, off, count, value, stream=None):
    _ck(lib().iris_flags_fill(heap, off, count, value, _stream(stream)))


def iris_all_store_bench(heap, payload_off, recv_off, flag_off, S, tile_bytes, epoch, ctas=0, pull=0, stream=None):
    _ck(lib().iris_all_store_bench(heap, payload_off, recv_off, flag_off, S, tile_bytes, epoch, ctas, pull, _stream(stream)))


# ------------------------------------------------------------------------------- GEMM + all-scatter
def iris_num_tiles(M: int, N: int, world: int) -> int:
    n = lib().iris_num_tiles(M, N, world)
    if n < 0:
        raise IrisError(int(n), iris_last_error())
    return int(n)


def iris_gemm_heap_bytes(M: int, N: int, world: int) -> int:
    return lib().iris_gemm_heap_bytes(M, N, world)


def iris_heap_epoch(heap: int) -> int:
    return lib().iris_heap_epoch(heap)


def _shards(B_shards):
    arr = (C.c_void_p * len(B_shards))(*[_ptr(b) for b in B_shards])
    return arr


def iris_gemm_all_scatter_ex(heap, A, B_shards, M, N, K, world, mode, dtype, c_off, flag_off, lock_off=0, epoch=1,
                             comm_ctas=0, max_ctas=0, raster_group=0, block_n=0, spin_timeout_ns=0, cta_pair=0, static_schedule=0, stream_k=0, wg_tail=0, rank_first=0, rank_count=0, pace_stores=0, consumer_bias=None, consumer_out_off=0, b_layout=0, fuse_tail=0, stage_k=0, stream=None, comm_stream=None):
    arr = _shards(B_shards)
    a = GemmArgs(_ptr(A), C.cast(arr, C.POINTER(C.c_void_p)), heap, M, N, K, world, mode, dtype, c_off, flag_off, lock_off,
                 epoch, comm_ctas, max_ctas, raster_group, block_n, spin_timeout_ns, cta_pair, static_schedule, stream_k, wg_tail, rank_first, rank_count, pace_stores, _ptr(consumer_bias), consumer_out_off, b_layout, fuse_tail, stage_k)
    if comm_stream is not None:     # the two-kernel, two-stream form (producers on `stream`, communication kernel on `comm_stream`)
        _ck(lib().iris_gemm_all_scatter_unfused(C.byref(a), _stream(stream), _stream(comm_stream)))
    else:
        _ck(lib().iris_gemm_all_scatter_ex(C.byref(a), _stream(stream)))


def iris_gemm_all_scatter_unfused(heap, A, B_shards, M, N, K, world, dtype, c_off, flag_off, lock_off, epoch, producer_stream, comm_stream, **kw):
    """Workgroup-specialised schedule as two kernels on two streams (see the header)."""
    iris_gemm_all_scatter_ex(heap, A, B_shards, M, N, K, world, IRIS_MODE_WORKGROUP_SPECIALIZED, dtype, c_off, flag_off, lock_off, epoch,
                             stream=producer_stream, comm_stream=comm_stream, **kw)


def gemm_all_scatter(A, B_shards, heap, M, N, K, world, mode):
    """The short form: bf16, C at offset 0, default stream (see the header)."""
    arr = _shards(B_shards)
    _ck(lib().gemm_all_scatter(_ptr(A), C.cast(arr, C.POINTER(C.c_void_p)), heap, M, N, K, world, mode))


def iris_consume_bias(heap, c_off, out_off, flag_off, bias, M, N, world, dtype, epoch, ctas=0, timeout_ns=0, stream=None):
    _ck(lib().iris_consume_bias(heap, c_off, out_off, flag_off, _ptr(bias), M, N, world, dtype, epoch, ctas, timeout_ns, _stream(stream)))


def iris_consume_bias_ranks(heap, c_off, out_off, flag_off, bias, M, N, world, rank_first, rank_count, dtype, epoch, ctas=0, timeout_ns=0, stream=None):
    _ck(lib().iris_consume_bias_ranks(heap, c_off, out_off, flag_off, _ptr(bias), M, N, world, rank_first, rank_count, dtype, epoch, ctas, timeout_ns,
                                      _stream(stream)))


def iris_gemm_takeover_stats(heap):
    """(half tiles kept by their producers, publication tiles still queued) of the last workgroup-specialised pair launch."""
    out = (C.c_int32 * 2)()
    _ck(lib().iris_gemm_takeover_stats(heap, out))
    return int(out[0]), int(out[1])


def iris_gemm_out_offset(M: int, N: int, world: int) -> int:
    return lib().iris_gemm_out_offset(M, N, world)


def iris_gemm_all_scatter_host(A_host, B_shards_host, C_host, flags_host, bias_host, OUT_host, heap, M, N, K, world, mode, dtype,
                               out_slot=0):
    arr = _shards(B_shards_host)
    _ck(lib().iris_gemm_all_scatter_host(_ptr(A_host), C.cast(arr, C.POINTER(C.c_void_p)), _ptr(C_host), _ptr(flags_host),
                                         _ptr(bias_host), _ptr(OUT_host), heap, M, N, K, world, mode, dtype, out_slot))


def iris_gemm_all_scatter_noalloc(A, B_shards, slot_bases, bytes_per_rank, M, N, K, world, dtype, c_off, flag_off, epoch, stream=None):
    """Workgroup-specialised gemm_all_scatter for callers that must not allocate device memory: no heap handle, the
    locks and the status block sit in a fixed array inside the library (at most 16384 publication tiles).  Blocks
    until the work on `stream` has finished.  Calls that overlap on the GPU race on that array."""
    arr = _shards(B_shards)
    bases = (C.c_uint64 * len(slot_bases))(*slot_bases)
    _ck(lib().iris_gemm_all_scatter_noalloc(_ptr(A), C.cast(arr, C.POINTER(C.c_void_p)), bases, bytes_per_rank, M, N, K, world, dtype,
                                            c_off, flag_off, epoch, _stream(stream)))
