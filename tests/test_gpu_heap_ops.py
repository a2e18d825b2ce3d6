"""GPU parity: heap, translation, tile put/get, atomics, flags and the all-store microbenchmark against
the CPU oracle, byte for byte, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import SENTINEL, GpuHeap

pytestmark = pytest.mark.gpu


def test_heap_create_queries_and_errors():
    h = iris.iris_heap_create(4, 1 << 20)
    try:
        assert iris.iris_heap_world(h) == 4 and iris.iris_heap_bytes_per_rank(h) == 1 << 20
        bases = iris.iris_heap_bases(h)
        assert [b - bases[0] for b in bases] == [r << 20 for r in range(4)]       # W equal partitions of one allocation
        assert [iris.iris_heap_base(h, r) for r in range(4)] == bases
        a = iris.iris_malloc(h, 1000)
        b = iris.iris_malloc(h, 16, 16)
        c = iris.iris_malloc(h, 4096, 4096)
        assert (a, b, c) == (0, 1008, 4096)
        with pytest.raises(iris.IrisError) as e:
            iris.iris_malloc(h, 1 << 20)
        assert e.value.code == iris.IRIS_ERR_NOMEM
        with pytest.raises(iris.IrisError):
            iris.iris_malloc(h, 16, 24)
        iris.iris_heap_reset(h)
        assert iris.iris_malloc(h, 1 << 20) == 0
    finally:
        iris.iris_heap_destroy(h)
    for world, bpr in [(0, 256), (9, 256), (2, 0), (2, 100)]:
        with pytest.raises(iris.IrisError) as e:
            iris.iris_heap_create(world, bpr)
        assert e.value.code == iris.IRIS_ERR_ARG
    assert iris.lib().iris_heap_create(0, 256) is None      # the short form returns NULL on failure


def test_translate_matches_oracle_and_rejects_out_of_range():
    with GpuHeap(3, 4096) as g:
        for frm in range(3):
            for to in range(3):
                for off in (0, 1, 17, 4095):
                    p = g.addr(frm, off)
                    assert iris.iris_translate(g.h, p, frm, to) == oracle.translate(g.bases, g.bpr, p, frm, to)
        for bad in (g.addr(0, 0) - 1, g.addr(0, 0) + 4096):
            with pytest.raises(iris.IrisError) as e:
                iris.iris_translate(g.h, bad, 0, 1)
            assert e.value.code == iris.IRIS_ERR_RANGE
        with pytest.raises(iris.IrisError) as e:
            iris.iris_translate(g.h, g.addr(0, 0), 0, 3)
        assert e.value.code == iris.IRIS_ERR_ARG


def _random_heap(g: GpuHeap, seed: int) -> oracle.HeapImage:
    img = g.image()
    img.mem[:] = inputs.payload_bytes(seed, 7, img.mem.size)
    g.mem.copy_(torch.from_numpy(img.mem).cuda())
    return img


@pytest.mark.parametrize("rows,row_bytes,sp,dp,so,do", [
    (128, 256, 512, 1024, 0, 65536),       # a 128 x 128 fp16 tile between pitched matrices (vector path)
    (37, 48, 80, 64, 4096 + 16, 90000),    # odd row count, 16-byte aligned
    (5, 23, 40, 31, 101, 70001),           # unaligned: byte path
    (1, 16, 16, 16, 0, 16),
    (300, 4096, 4096, 4096, 8192, 8192 + 300 * 4096),   # > one grid sweep
])
def test_put_get_byte_exact(rows, row_bytes, sp, dp, so, do):
    W, bpr = 4, 3 << 20
    with GpuHeap(W, bpr) as g:
        img = _random_heap(g, 3)
        iris.iris_put_tile(g.h, g.addr(1, so), g.addr(1, do), rows, row_bytes, sp, dp, 1, 3)
        img.put(so, do, rows, row_bytes, sp, dp, 1, 3)
        iris.iris_get_tile(g.h, g.addr(0, do), g.addr(0, so), rows, row_bytes, dp, sp, 0, 3)   # rank 0 pulls it from rank 3
        img.get(do, so, rows, row_bytes, dp, sp, 0, 3)
        assert np.array_equal(g.to_host(), img.mem)


def test_put_get_edge_cases_and_errors():
    with GpuHeap(2, 8192) as g:
        img = _random_heap(g, 4)
        iris.iris_put_tile(g.h, g.addr(0, 0), g.addr(0, 64), 0, 16, 16, 16, 0, 1)    # empty: no-op
        iris.iris_put_tile(g.h, g.addr(0, 0), g.addr(0, 64), 4, 0, 16, 16, 0, 1)
        iris.iris_put_tile(g.h, g.addr(0, 8192 - 32), g.addr(0, 8192 - 16), 1, 16, 16, 16, 0, 1)   # last bytes of the slot
        img.put(8192 - 32, 8192 - 16, 1, 16, 16, 16, 0, 1)
        assert np.array_equal(g.to_host(), img.mem)
        for args, code in [((g.addr(0, 8192 - 8), g.addr(0, 0), 1, 16, 16, 16, 0, 1), iris.IRIS_ERR_RANGE),
                           ((g.addr(0, 0), g.addr(0, 8000), 2, 128, 128, 128, 0, 1), iris.IRIS_ERR_RANGE),
                           ((g.addr(1, 0), g.addr(0, 0), 1, 16, 16, 16, 0, 1), iris.IRIS_ERR_RANGE),   # src not in from_rank's slot
                           ((g.addr(0, 0), g.addr(0, 64), 2, 32, 16, 32, 0, 1), iris.IRIS_ERR_ARG),    # pitch < row
                           ((g.addr(0, 0), g.addr(0, 64), 1, 16, 16, 16, 0, 2), iris.IRIS_ERR_ARG)]:
            with pytest.raises(iris.IrisError) as e:
                iris.iris_put_tile(g.h, *args)
            assert e.value.code == code
        assert np.array_equal(g.to_host(), img.mem)      # nothing was launched


@pytest.mark.parametrize("sem", [iris.IRIS_SEM_RELAXED, iris.IRIS_SEM_ACQUIRE, iris.IRIS_SEM_RELEASE, iris.IRIS_SEM_ACQ_REL])
@pytest.mark.parametrize("scope", [iris.IRIS_SCOPE_BLOCK, iris.IRIS_SCOPE_GPU, iris.IRIS_SCOPE_SYS])
def test_atomic_vector_forms_match_oracle(sem, scope):
    with GpuHeap(3, 1 << 16, fill=0) as g:
        img = g.image(fill=0)
        n, stride, off = 1000, 8, 256
        old = torch.empty(n, dtype=torch.int32, device="cuda")
        for val in (5, -7):
            iris.iris_atomic_add(g.h, g.addr(0, off), n, stride, 0, 2, val, sem, scope, old)
            assert np.array_equal(old.cpu().numpy(), img.atomic_add(off, n, stride, 2, val))
        iris.iris_atomic_cas(g.h, g.addr(1, off), n, stride, 1, 2, -2, 9, sem, scope, old)        # hits everywhere
        assert np.array_equal(old.cpu().numpy(), img.atomic_cas(off, n, stride, 2, -2, 9))
        iris.iris_atomic_cas(g.h, g.addr(1, off), n // 2, 2 * stride, 1, 2, 4, 1, sem, scope, old[: n // 2])   # misses
        assert np.array_equal(old[: n // 2].cpu().numpy(), img.atomic_cas(off, n // 2, 2 * stride, 2, 4, 1))
        assert np.array_equal(g.to_host(), img.mem)


@pytest.mark.parametrize("sem", [iris.IRIS_SEM_RELAXED, iris.IRIS_SEM_ACQUIRE, iris.IRIS_SEM_RELEASE, iris.IRIS_SEM_ACQ_REL])
@pytest.mark.parametrize("scope", [iris.IRIS_SCOPE_BLOCK, iris.IRIS_SCOPE_GPU, iris.IRIS_SCOPE_SYS])
def test_u64_atomic_vector_forms_match_oracle(sem, scope):
    """atomic_add / atomic_cas on uint64 words: previous values and the whole heap image equal the oracle's, with
    operands that carry out of the low 32 bits and wrap at 2**64."""
    with GpuHeap(3, 1 << 16, fill=0) as g:
        img = g.image(fill=0)
        n, stride, off = 777, 16, 512
        rng = np.random.default_rng(21)
        init = rng.integers(0, 2**64, n, dtype=np.uint64)
        init[:3] = [2**64 - 1, 2**32 - 1, 0]
        words = np.zeros(n * 2, dtype=np.uint64)
        words[::2] = init
        g.write(2, off, words)
        img.view(2, off, n * stride, np.uint64)[:] = words
        old = torch.empty(n, dtype=torch.int64, device="cuda")
        for val in (1, 2**32 + 3, 2**64 - 1):
            iris.iris_atomic_add_u64(g.h, g.addr(0, off), n, stride, 0, 2, val, sem, scope, old)
            assert np.array_equal(old.cpu().numpy().view(np.uint64), img.atomic_add_u64(off, n, stride, 2, val))
        cur = img.view(2, off, n * stride, np.uint64)[::2].copy()
        target = int(cur[5])
        iris.iris_atomic_cas_u64(g.h, g.addr(1, off), n, stride, 1, 2, target, 42, sem, scope, old)   # hits where the word equals cur[5]
        assert np.array_equal(old.cpu().numpy().view(np.uint64), img.atomic_cas_u64(off, n, stride, 2, target, 42))
        iris.iris_atomic_cas_u64(g.h, g.addr(1, off), n, stride, 1, 2, target ^ (1 << 40), 43, sem, scope, old)   # differs in the high half only
        assert np.array_equal(old.cpu().numpy().view(np.uint64), img.atomic_cas_u64(off, n, stride, 2, target ^ (1 << 40), 43))
        assert np.array_equal(g.to_host(), img.mem)
        for bad in (dict(ptr=g.addr(0, off + 4)), dict(stride=12)):        # 8-byte alignment of address and stride
            with pytest.raises(iris.IrisError) as e:
                iris.iris_atomic_add_u64(g.h, bad.get("ptr", g.addr(0, off)), 2, bad.get("stride", 8), 0, 1, 1)
            assert e.value.code == iris.IRIS_ERR_ARG
        with pytest.raises(iris.IrisError) as e:
            iris.iris_atomic_cas_u64(g.h, g.addr(0, (1 << 16) - 8), 2, 8, 0, 1, 0, 1)
        assert e.value.code == iris.IRIS_ERR_RANGE
        assert np.array_equal(g.to_host(), img.mem)


def test_region_checks_do_not_wrap_on_huge_sizes():
    """rows, pitch and count large enough to wrap a 64-bit product are refused with IRIS_ERR_RANGE before any launch."""
    with GpuHeap(2, 4096) as g:
        before = g.to_host().copy()
        with pytest.raises(iris.IrisError) as e:
            iris.iris_put_tile(g.h, g.addr(0, 0), g.addr(0, 2048), 2**62, 4, 4, 4, 0, 1)
        assert e.value.code == iris.IRIS_ERR_RANGE
        with pytest.raises(iris.IrisError) as e:
            iris.iris_get_tile(g.h, g.addr(0, 0), g.addr(0, 2048), 2**61 + 1, 8, 8, 8, 0, 1)
        assert e.value.code == iris.IRIS_ERR_RANGE
        with pytest.raises(iris.IrisError) as e:
            iris.iris_atomic_add(g.h, g.addr(0, 0), 2**62, 4, 0, 1, 1)
        assert e.value.code == iris.IRIS_ERR_RANGE
        with pytest.raises(iris.IrisError) as e:
            iris.iris_atomic_add_u64(g.h, g.addr(0, 0), 2**61, 8, 0, 1, 1)
        assert e.value.code == iris.IRIS_ERR_RANGE
        assert np.array_equal(g.to_host(), before)


def test_contended_atomics_invariants():
    with GpuHeap(2, 4096, fill=0) as g:
        n = 100000
        old = torch.empty(n, dtype=torch.int32, device="cuda")
        iris.iris_atomic_add_contended(g.h, g.addr(0, 64), n, 0, 1, 1, iris.IRIS_SEM_ACQ_REL, iris.IRIS_SCOPE_GPU, old)
        assert int(g.view(1, 64, 4, torch.int32)[0]) == n and int(g.view(0, 64, 4, torch.int32)[0]) == 0
        assert torch.equal(torch.sort(old).values, torch.arange(n, dtype=torch.int32, device="cuda"))  # a permutation of 0..n-1
        iris.iris_atomic_cas_contended(g.h, g.addr(0, 128), n, 0, 1, 0, 1000, iris.IRIS_SEM_RELAXED, iris.IRIS_SCOPE_GPU, old)
        winners = torch.nonzero(old == 0).flatten()
        assert winners.numel() == 1                                                  # exactly one contender saw 0
        final = int(g.view(1, 128, 4, torch.int32)[0])
        assert final == 1000 + int(winners[0]) and bool(torch.all((old == 0) | (old == final)))


def test_flags_fill_touches_exactly_the_region():
    with GpuHeap(4, 8192) as g:
        img = g.image()
        iris.iris_flags_fill(g.h, 1024, 100, 7)
        for s in range(4):
            img.view(s, 1024, 400, np.int32)[:] = 7
        assert np.array_equal(g.to_host(), img.mem)
        with pytest.raises(iris.IrisError) as e:
            iris.iris_flags_fill(g.h, 8192 - 8, 3, 1)
        assert e.value.code == iris.IRIS_ERR_RANGE


@pytest.mark.parametrize("W,S,tile", [(8, 1024, 32768), (8, 1 << 18, 32768), (4, 100000 - 100000 % 16, 4096), (2, 48, 16), (8, 1 << 22, 32768)])
@pytest.mark.parametrize("pull", [0, 1])
def test_all_store_matches_oracle(W, S, tile, pull):
    tile = min(tile, 32768)
    T = -(-S // tile)
    payload_off, recv_off = 256, 256 + ((S + 255) // 256) * 256 + 256
    flag_off = recv_off + ((W * S + 255) // 256) * 256 + 256
    bpr = flag_off + ((W * T * 4 + 255) // 256) * 256 + 256
    with GpuHeap(W, bpr) as g:
        img = g.image()
        for r in range(W):
            pay = inputs.payload_bytes(inputs.SEED0 + 1, inputs.STREAM_PAYLOAD0 + r, S)
            img.view(r, payload_off, S)[:] = pay
            g.write(r, payload_off, pay)
            img.view(r, flag_off, W * T * 4, np.int32)[:] = 0
        iris.iris_flags_fill(g.h, flag_off, W * T, 0)
        for epoch in (1, 2):                                   # two rounds: cas(epoch-1 -> epoch) without resets
            iris.iris_all_store_bench(g.h, payload_off, recv_off, flag_off, S, tile, epoch, 0, pull)
            img.all_store(payload_off, recv_off, flag_off, S, tile, epoch)
            assert np.array_equal(g.to_host(), img.mem)
        iris.iris_status_check(g.h)


def test_all_store_argument_errors():
    with GpuHeap(2, 1 << 16) as g:
        for args, code in [((0, 4096, 32768, 1000, 512, 1), iris.IRIS_ERR_ARG),        # S not multiple of 16
                           ((0, 4096, 32768, 1024, 100, 1), iris.IRIS_ERR_ARG),        # tile not multiple of 16
                           ((0, 512, 32768, 1024, 512, 1), iris.IRIS_ERR_ARG),         # payload overlaps receive area
                           ((0, 4096, 32768, 1 << 15, 512, 1), iris.IRIS_ERR_RANGE)]:  # receive area leaves the slot
            with pytest.raises(iris.IrisError) as e:
                iris.iris_all_store_bench(g.h, *args)
            assert e.value.code == code
        assert bool(torch.all(g.mem == SENTINEL))


@pytest.mark.parametrize("op", ["add", "xchg", "and", "or", "xor", "min", "max"])
def test_remaining_atomics_match_oracle(op):
    with GpuHeap(3, 1 << 14) as g:
        img = _random_heap(g, 11)
        n, stride, off = 500, 12, 512
        old = torch.empty(n, dtype=torch.int32, device="cuda")
        for val, sem, scope in [(0x5A5A1234, iris.IRIS_SEM_RELAXED, iris.IRIS_SCOPE_GPU), (-77, iris.IRIS_SEM_ACQ_REL, iris.IRIS_SCOPE_SYS),
                                (3, iris.IRIS_SEM_RELEASE, iris.IRIS_SCOPE_BLOCK)]:
            iris.iris_atomic_rmw(g.h, iris.ATOMIC_OPS[op], g.addr(2, off), n, stride, 2, 0, val, sem, scope, old)
            assert np.array_equal(old.cpu().numpy(), img.atomic_rmw(op, off, n, stride, 0, val)), (op, val)
        assert np.array_equal(g.to_host(), img.mem)
        with pytest.raises(iris.IrisError) as e:
            iris.iris_atomic_rmw(g.h, 9, g.addr(0, 0), 1, 4, 0, 1, 1)
        assert e.value.code == iris.IRIS_ERR_ARG


def test_copy_load_store_byte_exact():
    W, bpr = 4, 1 << 16
    with GpuHeap(W, bpr) as g:
        img = _random_heap(g, 12)
        # copy: rank 0 moves a region from rank 1's memory to rank 3's
        iris.iris_copy_tile(g.h, g.addr(0, 1024), g.addr(0, 20480), 17, 80, 96, 112, 0, 1, 3)
        img.copy(1024, 20480, 17, 80, 96, 112, 1, 3)
        assert np.array_equal(g.to_host(), img.mem)
        # load: rank 2 reads rank 1's memory into a buffer outside the heap
        out = torch.zeros(9 * 48, dtype=torch.uint8, device="cuda")
        iris.iris_load_tile(g.h, g.addr(2, 4096 + 3), out, 9, 37, 64, 48, 2, 1)       # unaligned: byte path
        host = img.mem.reshape(W, bpr)
        exp = np.zeros((9, 48), dtype=np.uint8)
        for i in range(9):
            exp[i, :37] = host[1, 4099 + i * 64: 4099 + i * 64 + 37]
        assert np.array_equal(out.cpu().numpy().reshape(9, 48), exp)
        # store: rank 2 writes values from outside the heap into rank 0's memory
        vals = torch.from_numpy(inputs.payload_bytes(13, 1, 32 * 256)).cuda()
        iris.iris_store_tile(g.h, vals, g.addr(2, 32768), 32, 256, 256, 512, 2, 0)
        v = vals.cpu().numpy().reshape(32, 256)
        for i in range(32):
            img.view(0, 32768 + i * 512, 256)[:] = v[i]
        assert np.array_equal(g.to_host(), img.mem)
        with pytest.raises(iris.IrisError) as e:
            iris.iris_load_tile(g.h, g.addr(2, bpr - 16), out, 2, 32, 32, 48, 2, 1)
        assert e.value.code == iris.IRIS_ERR_RANGE
