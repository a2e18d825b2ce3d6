"""GPU parity for gemm_all_scatter in its three schedules, against the CPU oracle.

Layout, replication, flags and locks are compared bit-exactly (whole heap image); values are compared
bit-exactly where the arithmetic is exact (integer-valued inputs) and within the stated tolerance
otherwise: max |gpu - ref| <= 1e-2 (|ref| + 1) elementwise, relative Frobenius error <= 2e-3.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import SENTINEL, GpuHeap, check_tolerance, dev16, first_diff, gemm_layout

pytestmark = pytest.mark.gpu

MODES = [iris.IRIS_MODE_BULK_SYNCHRONOUS, iris.IRIS_MODE_FUSED_SEQUENTIAL, iris.IRIS_MODE_WORKGROUP_SPECIALIZED]
MODE_IDS = ["bulk_synchronous", "fused_sequential", "workgroup_specialized"]


def run_gemm(g, A, Bs, dtype, mode, epoch=1, with_locks_zeroed=True, **kw):
    M, K = A.shape
    W, nl = len(Bs), Bs[0].shape[0]
    N = W * nl
    c_off, flag_off, lock_off, out_off, _ = gemm_layout(M, N, W, with_out=True)
    # b_layout = 1: the shards are handed over as [K, N_local] row-major (the oracle keeps reading the [N_local, K] arrays)
    dA, dB = dev16(A), [dev16(np.ascontiguousarray(b.T) if kw.get("b_layout", 0) == 1 else b) for b in Bs]
    nt = oracle.num_tiles(M, N, W) if M and N else 0
    if with_locks_zeroed and nt:
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
    # These shapes are a wave or two: by default the producers would scatter most tiles themselves.  Unless a test
    # asks otherwise, every tile takes the lock handshake and the communication CTAs (Listing 5 as printed).
    if mode == iris.IRIS_MODE_WORKGROUP_SPECIALIZED:
        kw.setdefault("wg_tail", -1)
    iris.iris_gemm_all_scatter_ex(g.h, dA, dB, M, N, K, W, mode, iris.DTYPES[dtype], c_off, flag_off, lock_off, epoch, **kw)
    iris.iris_status_check(g.h)
    return c_off, flag_off, lock_off, out_off, nt


def expected_image(g, A, Bs, dtype, mode, epoch=1, c_full=None):
    M = A.shape[0]
    W, nl = len(Bs), Bs[0].shape[0]
    N = W * nl
    c_off, flag_off, lock_off, out_off, _ = gemm_layout(M, N, W, with_out=True)
    img = g.image()
    nt = oracle.num_tiles(M, N, W) if M and N else 0
    for s in range(W):                       # the caller zeroes the lock array in every slot
        img.view(s, lock_off, nt * 4, np.int32)[:] = 0
    if M and N:
        if c_full is None:
            c_full = oracle.gemm_block(A, Bs, dtype)
        img.all_scatter(c_off, c_full)
        img.publish_flags(flag_off, nt, epoch)
        if mode == iris.IRIS_MODE_WORKGROUP_SPECIALIZED:
            img.consume_locks(lock_off, M, N)
    return img, c_full


def c_slot(host, g, s, c_off, M, N):
    return host[s * g.bpr + c_off: s * g.bpr + c_off + M * N * 2].view(np.uint16).reshape(M, N)


# ------------------------------------------------------------------------------------------------
# Config 1 of the benchmark definition: W=2, M=N=K=256, fp16 uniform[-1,1], 128x128 tiles.
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_config1_all_modes(mode):
    W, M, N, K, dtype = 2, 256, 256, 256, "fp16"
    A, Bs = inputs.gemm_inputs(inputs.SEED0 + 0, W, M, N, K, "uniform", dtype)
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        c_off, flag_off, lock_off, _, nt = run_gemm(g, A, Bs, dtype, mode)
        host = g.to_host()
        img, c_ref = expected_image(g, A, Bs, dtype, mode)
        # values: within tolerance in slot 0 ...
        check_tolerance(c_slot(host, g, 0, c_off, M, N), c_ref, dtype)
        # ... layout / replication / flags / locks / sentinel: bit-exact once the oracle image carries the GPU's values
        img2, _ = expected_image(g, A, Bs, dtype, mode, c_full=c_slot(host, g, 0, c_off, M, N).copy())
        assert np.array_equal(host, img2.mem), first_diff(host, img2.mem)
        assert nt == 4


# ------------------------------------------------------------------------------------------------
# Exact-arithmetic inputs: every dot product is a small integer, so any correct fp32-accumulating GEMM
# equals the oracle byte for byte.  This pins tile placement, rank offsets, replication, flags and locks.
# ------------------------------------------------------------------------------------------------
EXACT_SHAPES = [
    # W, M, N_local, K
    (1, 128, 128, 64),
    (2, 256, 128, 256),
    (2, 384, 256, 192),        # BN=256 path, 3 tile rows
    (4, 130, 136, 72),         # ragged M, ragged N_local (not a multiple of 128), ragged K (not a multiple of 64)
    (8, 128, 512, 128),
    (3, 520, 392, 328),        # odd world, everything ragged, several tiles
    (8, 1, 8, 8),              # smallest legal problem
    (2, 300, 640, 64),         # N_local > 512 and not a multiple of 256
    (2, 1000, 512, 200),       # CTA-pair tiles (256 x 256), ragged M: the last pair's second CTA has no rows
    (8, 257, 256, 64),         # CTA-pair tiles, one row in the second tile row
    (2, 600, 448, 136),        # CTA-pair tiles with a ragged shard (448 = 256 + 192): masked stores, 4 flags of 4 + 2 of 4
    (3, 384, 904, 64),         # 904 = 3 * 256 + 136: the last pair tile has two publication tiles, the second 8 columns wide
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("W,M,nl,K", EXACT_SHAPES)
def test_exact_integer_gemm_full_heap_image(mode, dtype, W, M, nl, K):
    N = W * nl
    A = inputs.matrix(41, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(41, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        run_gemm(g, A, Bs, dtype, mode)
        host = g.to_host()
        img, _ = expected_image(g, A, Bs, dtype, mode)
        assert np.array_equal(host, img.mem), first_diff(host, img.mem)


B_ROW_MAJOR_SHAPES = [
    # W, M, N_local, K, kwargs: B shards stored [K, N_local] (Listing 2's operand as printed), read as an MN-major operand
    (1, 128, 128, 64, dict()),
    (4, 130, 136, 72, dict()),                          # single-CTA kernel, everything ragged
    (3, 520, 392, 328, dict()),                         # CTA pairs, ragged shard (392 = 256 + 136)
    (3, 520, 392, 328, dict(cta_pair=-1)),              # the same on the single-CTA kernel
    (3, 384, 904, 64, dict()),                          # 904 = 3 * 256 + 136
    (2, 600, 448, 136, dict()),                         # 448 = 256 + 192: a 192-wide last pair tile, 96 columns per CTA
    (2, 384, 256, 192, dict(cta_pair=-1, block_n=256)), # single-CTA kernel, 256-wide tiles: four 64-column blocks per stage
    (8, 128, 512, 128, dict(block_n=128)),
    (2, 1000, 512, 200, dict()),
    (4, 100, 136, 4096, dict(stream_k=1)),              # k ranges of a tile computed by different CTAs
    (8, 8, 8, 8, dict()),                               # a shard narrower than one 64-column block
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("W,M,nl,K,kw", B_ROW_MAJOR_SHAPES)
def test_b_shards_row_major_k_by_n_full_heap_image(mode, dtype, W, M, nl, K, kw):
    N = W * nl
    A = inputs.matrix(71, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(71, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        run_gemm(g, A, Bs, dtype, mode, b_layout=1, **kw)
        host = g.to_host()
        img, _ = expected_image(g, A, Bs, dtype, mode)
        assert np.array_equal(host, img.mem), first_diff(host, img.mem)


def test_b_layouts_agree_bit_for_bit_on_real_valued_inputs():
    """Same sums in the same order whichever way B is stored: C from [K, N_local] shards equals C from [N_local, K] shards."""
    W, M, nl, K, dtype = 4, 384, 320, 1024, "bf16"
    N = W * nl
    A, Bs = inputs.gemm_inputs(inputs.SEED0 + 2, W, M, N, K, "normal002", dtype)
    c_ref = oracle.gemm_block(A, Bs, dtype)
    bpr = gemm_layout(M, N, W, True)[4]
    for kw in (dict(), dict(cta_pair=-1)):
        outs = []
        for b_layout in (0, 1):
            with GpuHeap(W, bpr) as g:
                c_off = run_gemm(g, A, Bs, dtype, iris.IRIS_MODE_FUSED_SEQUENTIAL, b_layout=b_layout, **kw)[0]
                outs.append(c_slot(g.to_host(), g, W - 1, c_off, M, N).copy())
        check_tolerance(outs[1], c_ref, dtype)
        assert np.array_equal(outs[0], outs[1])


RAGGED_PAIR_SHAPES = [
    # W, M, N_local, K: CTA-pair kernel, N_local > 256 and not a multiple of 256
    (2, 600, 448, 136),      # 256 + 192
    (3, 384, 904, 64),       # 3 x 256 + 136: two plain units and a fused one per shard; the remainder's last publication tile is 8 wide
    (3, 520, 392, 328),      # 256 + 136
    (2, 300, 640, 64),       # 2 x 256 + 128
    (4, 1100, 576, 256),     # 2 x 256 + 64 (the paper's 4608 / 8), ragged M
    (2, 512, 320, 128),      # 256 + 64
    (8, 2048, 288, 64),      # 256 + 32: the narrowest remainder an MMA group can have
    (2, 700, 504, 72),       # 256 + 248: remainder rounded up to a full 256-wide group
    (2, 512, 320, 1096),     # 256 + 64, 18 k-blocks (the last one 8 wide): the 2 + 2 + 1 k-block ring goes round several times
    (4, 520, 352, 840),      # 256 + 96: the widest remainder that still gets two k-blocks per stage by default
]


@pytest.mark.parametrize("kw", [dict(), dict(fuse_tail=1), dict(fuse_tail=-1), dict(fuse_tail=-1, stage_k=64), dict(fuse_tail=1, stage_k=64), dict(fuse_tail=1, stage_k=128),
                                dict(fuse_tail=1, max_ctas=6, comm_ctas=2),
                                dict(fuse_tail=1, static_schedule=1, raster_group=1), dict(fuse_tail=1, wg_tail=0),
                                dict(fuse_tail=1, wg_tail=0, comm_ctas=2, max_ctas=12)],
                         ids=["default", "fused", "separate_tail_tile", "separate_tail_tile_k64", "fused_k64", "fused_k128", "small_grid", "static", "tail_rule", "takeover"])
@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("W,M,nl,K", RAGGED_PAIR_SHAPES)
def test_ragged_shard_remainder_fused_with_last_full_tile(mode, W, M, nl, K, kw):
    """A shard that is not a whole number of 256-column tiles: by default the pair that computes the last full tile also
    computes the remainder columns (second MMA group on the same A stages, second accumulator); fuse_tail = -1 makes the
    remainder a tile of its own.  Either way the heap image is the oracle's, twice in a row."""
    N, dtype = W * nl, "bf16"
    A = inputs.matrix(73, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(73, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        c_full = None
        for epoch in (1, 2):
            run_gemm(g, A, Bs, dtype, mode, epoch=epoch, with_locks_zeroed=(epoch == 1), **kw)
            host = g.to_host()
            img, c_full = expected_image(g, A, Bs, dtype, mode, epoch=epoch, c_full=c_full)
            assert np.array_equal(host, img.mem), (epoch, first_diff(host, img.mem))


@pytest.mark.parametrize("block_n", [128, 256])
@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_exact_integer_gemm_tile_width_and_grid_knobs(block_n, mode):
    W, M, nl, K, dtype = 4, 640, 512, 320, "bf16"
    N = W * nl
    A = inputs.matrix(43, inputs.STREAM_A, M, K, "smallint:2", dtype)
    Bs = [inputs.matrix(43, inputs.STREAM_B0 + r, nl, K, "ternary:0.5", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        img = None
        for kw in (dict(), dict(max_ctas=7, comm_ctas=3, raster_group=2), dict(max_ctas=148, comm_ctas=32, raster_group=1),
                   dict(cta_pair=-1), dict(cta_pair=-1, max_ctas=5, comm_ctas=2), dict(cta_pair=1 if block_n == 256 else 0, comm_ctas=8), dict(static_schedule=1), dict(static_schedule=1, max_ctas=10, raster_group=3),
                   dict(stage_k=64), dict(stage_k=64, max_ctas=6, comm_ctas=2), dict(stage_k=128, static_schedule=1)):
            g.mem.fill_(SENTINEL)
            run_gemm(g, A, Bs, dtype, mode, block_n=block_n, **kw)
            host = g.to_host()
            if img is None:
                img, _ = expected_image(g, A, Bs, dtype, mode)
            assert np.array_equal(host, img.mem), (kw, first_diff(host, img.mem))


# ------------------------------------------------------------------------------------------------
# Real-valued inputs: tolerance vs the oracle; all W copies byte-identical; the three schedules agree
# bit for bit (they share one main loop).
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,dist", [("bf16", "normal002"), ("bf16", "uniform"), ("fp16", "uniform")])
def test_real_valued_tolerance_replication_and_cross_mode_equality(dtype, dist):
    W, M, nl, K = 4, 384, 256, 1024
    N = W * nl
    A, Bs = inputs.gemm_inputs(inputs.SEED0 + 2, W, M, N, K, dist, dtype)
    c_ref = oracle.gemm_block(A, Bs, dtype)
    bpr = gemm_layout(M, N, W, True)[4]
    results = []
    with GpuHeap(W, bpr) as g:
        for mode in MODES:
            g.mem.fill_(SENTINEL)
            c_off, flag_off, lock_off, _, nt = run_gemm(g, A, Bs, dtype, mode)
            host = g.to_host()
            c0 = c_slot(host, g, 0, c_off, M, N).copy()
            check_tolerance(c0, c_ref, dtype)
            for s in range(1, W):
                assert np.array_equal(c_slot(host, g, s, c_off, M, N), c0)
            img, _ = expected_image(g, A, Bs, dtype, mode, c_full=c0)
            assert np.array_equal(host, img.mem), first_diff(host, img.mem)
            results.append(c0)
    assert np.array_equal(results[0], results[1]) and np.array_equal(results[0], results[2])


def test_identity_B_reproduces_A_and_zero_A_gives_zero():
    W, M, K, dtype = 2, 256, 256, "bf16"
    A = inputs.matrix(5, 0, M, K, "uniform", dtype)
    A[A == 0x8000] = 0
    eye = oracle.encode(np.eye(K), dtype)
    Bs = [np.ascontiguousarray(eye[r * 128:(r + 1) * 128]) for r in range(W)]
    bpr = gemm_layout(M, K, W, True)[4]
    with GpuHeap(W, bpr) as g:
        c_off = run_gemm(g, A, Bs, dtype, iris.IRIS_MODE_FUSED_SEQUENTIAL)[0]
        host = g.to_host()
        for s in range(W):
            assert np.array_equal(c_slot(host, g, s, c_off, M, K), A)
        c_off = run_gemm(g, np.zeros_like(A), Bs, dtype, iris.IRIS_MODE_WORKGROUP_SPECIALIZED, epoch=2)[0]
        host = g.to_host()
        for s in range(W):
            assert not c_slot(host, g, s, c_off, M, K).any()


def test_epochs_advance_without_resets_and_runs_are_deterministic():
    W, M, nl, K, dtype = 2, 256, 256, 512, "bf16"
    N = W * nl
    A, Bs = inputs.gemm_inputs(77, W, M, N, K, "uniform", dtype)
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        first = None
        for epoch in range(1, 6):
            mode = MODES[epoch % 3]
            c_off, flag_off, lock_off, _, nt = run_gemm(g, A, Bs, dtype, mode, epoch=epoch, with_locks_zeroed=(epoch == 1))
            host = g.to_host()
            for s in range(W):
                f = host[s * g.bpr + flag_off: s * g.bpr + flag_off + nt * 4].view(np.int32)
                assert np.all(f == epoch)
                lk = host[s * g.bpr + lock_off: s * g.bpr + lock_off + nt * 4].view(np.int32)
                assert np.all(lk == 0)                      # locks reset themselves (cas 1 -> 0)
            c0 = c_slot(host, g, 0, c_off, M, N).copy()
            if first is None:
                first = c0
            assert np.array_equal(first, c0)


def test_empty_problems_and_K_zero():
    with GpuHeap(2, 1 << 20) as g:
        dummy = torch.zeros(64, dtype=torch.int16, device="cuda")
        for (M, N, K) in [(0, 256, 64), (128, 0, 64)]:
            iris.iris_gemm_all_scatter_ex(g.h, dummy, [dummy, dummy], M, N, K, 2, 1, iris.IRIS_BF16, 0, 65536, 0, 1)
        iris.iris_status_check(g.h)
        assert bool(torch.all(g.mem == SENTINEL))           # nothing written, nothing published
        # K = 0: the empty sum, C = +0 everywhere, flags published
        M, N = 128, 256
        c_off, flag_off, lock_off, _, _ = gemm_layout(M, N, 2, True)
        for mode in MODES:
            g.mem.fill_(SENTINEL)
            iris.iris_flags_fill(g.h, lock_off, 2, 0)
            iris.iris_gemm_all_scatter_ex(g.h, None, [None, None], M, N, 0, 2, mode, iris.IRIS_BF16, c_off, flag_off, lock_off, 3)
            iris.iris_status_check(g.h)
            host = g.to_host()
            img = g.image()
            for s in range(2):
                img.view(s, lock_off, 8, np.int32)[:] = 0
            img.all_scatter(c_off, np.zeros((M, N), dtype=np.uint16))
            img.publish_flags(flag_off, 2, 3)
            assert np.array_equal(host, img.mem), first_diff(host, img.mem)


def test_argument_errors_are_reported_before_any_launch():
    with GpuHeap(2, 1 << 20) as g:
        d = torch.zeros(1 << 16, dtype=torch.int16, device="cuda")
        ok = dict(M=128, N=256, K=64, world=2, mode=1, dtype=iris.IRIS_BF16, c_off=0, flag_off=65536, lock_off=66560, epoch=1)
        cases = [
            (dict(N=250), iris.IRIS_ERR_ARG), (dict(N=264, K=64), iris.IRIS_ERR_ARG), (dict(K=60), iris.IRIS_ERR_ARG),
            (dict(mode=3), iris.IRIS_ERR_ARG), (dict(dtype=2), iris.IRIS_ERR_ARG), (dict(world=4), iris.IRIS_ERR_ARG),
            (dict(epoch=0), iris.IRIS_ERR_ARG), (dict(c_off=128), iris.IRIS_ERR_ARG), (dict(block_n=64), iris.IRIS_ERR_ARG),
            (dict(M=4096, N=256), iris.IRIS_ERR_RANGE), (dict(flag_off=(1 << 20) - 4), iris.IRIS_ERR_RANGE),
            (dict(flag_off=1024), iris.IRIS_ERR_ARG),                   # flags inside C
            (dict(mode=2, lock_off=65536), iris.IRIS_ERR_ARG),          # locks on top of flags
            (dict(cta_pair=1), iris.IRIS_ERR_UNSUPPORTED),              # M = 128: no room for a 256-row pair tile
            (dict(cta_pair=2), iris.IRIS_ERR_ARG),
        ]
        for delta, code in cases:
            kw = {**ok, **delta}
            with pytest.raises(iris.IrisError) as e:
                iris.iris_gemm_all_scatter_ex(g.h, d, [d, d], kw["M"], kw["N"], kw["K"], kw["world"], kw["mode"], kw["dtype"],
                                              kw["c_off"], kw["flag_off"], kw["lock_off"], kw["epoch"], block_n=kw.get("block_n", 0),
                                              cta_pair=kw.get("cta_pair", 0))
            assert e.value.code == code, (delta, e.value)
        torch.cuda.synchronize()
        assert bool(torch.all(g.mem == SENTINEL))


def test_short_form_and_host_entry_point():
    W, M, N, K = 2, 256, 512, 256
    A, Bs = inputs.gemm_inputs(9, W, M, N, K, "smallint:2", "bf16")
    c_ref = oracle.gemm_block(A, Bs, "bf16")
    nt = oracle.num_tiles(M, N, W)
    bpr = iris.iris_gemm_heap_bytes(M, N, W)
    flag_off = (M * N * 2 + 255) // 256 * 256
    lock_off = flag_off + (nt * 4 + 255) // 256 * 256
    assert bpr == lock_off + (nt * 4 + 255) // 256 * 256 + 256
    with GpuHeap(W, bpr) as g:                                         # backing bytes pre-filled with 0xA5: stale flags and locks
        dA, dB = dev16(A), [dev16(b) for b in Bs]
        for i, mode in enumerate(MODES):
            iris.gemm_all_scatter(dA, dB, g.h, M, N, K, W, mode)       # default stream
            iris.iris_status_check(g.h, 0)
            assert iris.iris_heap_epoch(g.h) == i + 1
            host = g.to_host()
            for s in range(W):
                assert np.array_equal(c_slot(host, g, s, 0, M, N), c_ref)
                assert np.all(host[s * bpr + flag_off: s * bpr + flag_off + nt * 4].view(np.int32) == i + 1)
        # host buffers in, host buffers out
        C_host = np.empty((M, N), dtype=np.uint16)
        flags = np.empty((W, nt), dtype=np.int32)
        iris.iris_gemm_all_scatter_host(A, Bs, C_host, flags, None, None, g.h, M, N, K, W, iris.IRIS_MODE_WORKGROUP_SPECIALIZED,
                                        iris.IRIS_BF16, 1)
        assert np.array_equal(C_host, c_ref) and np.all(flags == 4)
    # with the consumer: OUT comes back too
    out_off = iris.iris_gemm_out_offset(M, N, W)
    assert out_off == bpr - 256
    bias = inputs.vector(9, inputs.STREAM_BIAS, N, "smallint:2", "bf16")
    with GpuHeap(W, out_off + M * N * 2) as g:
        C_host, OUT_host = np.empty((M, N), dtype=np.uint16), np.empty((M, N), dtype=np.uint16)
        iris.iris_gemm_all_scatter_host(A, Bs, C_host, None, bias, OUT_host, g.h, M, N, K, W, iris.IRIS_MODE_FUSED_SEQUENTIAL,
                                        iris.IRIS_BF16, 0)
        assert np.array_equal(C_host, c_ref) and np.array_equal(OUT_host, oracle.consume_bias_rows(c_ref, bias, "bf16"))


def test_short_form_clears_stale_flags_and_locks_when_its_layout_changes():
    """The short form places flags and locks itself, so it also initialises them: on a heap whose bytes are a non-zero
    pattern (locks that are neither 0, 1 nor 2; flags far above any epoch), in the workgroup-specialised schedule, first
    for one shape and then for a smaller one whose lock array lands inside the first shape's C."""
    W, K = 2, 128
    shapes = [(512, 1024), (256, 512)]
    bpr = iris.iris_gemm_heap_bytes(*shapes[0], W)
    with GpuHeap(W, bpr, fill=0x7B) as g:
        epoch = 0
        for M, N in shapes:
            A, Bs = inputs.gemm_inputs(13, W, M, N, K, "smallint:2", "bf16")
            c_ref = oracle.gemm_block(A, Bs, "bf16")
            nt = oracle.num_tiles(M, N, W)
            flag_off = (M * N * 2 + 255) // 256 * 256
            lock_off = flag_off + (nt * 4 + 255) // 256 * 256
            dA, dB = dev16(A), [dev16(b) for b in Bs]
            for _ in range(2):
                iris.gemm_all_scatter(dA, dB, g.h, M, N, K, W, iris.IRIS_MODE_WORKGROUP_SPECIALIZED)
                iris.iris_status_check(g.h, 0)
                epoch += 1
                host = g.to_host()
                for s in range(W):
                    assert np.array_equal(c_slot(host, g, s, 0, M, N), c_ref)
                    assert np.all(host[s * bpr + flag_off: s * bpr + flag_off + nt * 4].view(np.int32) == epoch)
                    assert np.all(host[s * bpr + lock_off: s * bpr + lock_off + nt * 4].view(np.int32) == 0)


STREAMK_SHAPES = [
    # W, M, N_local, K, kwargs  (single-CTA kernel; K long enough to be cut into ranges)
    (8, 128, 512, 2048, dict()),                         # one tile row, 16 tiles for 148 SMs: chosen automatically
    (8, 128, 512, 2048, dict(stream_k=1, block_n=128)),
    (2, 300, 640, 1024, dict(stream_k=1, cta_pair=-1)),  # ragged M and N_local, tiles split at arbitrary k
    (4, 100, 136, 4096, dict(stream_k=1)),               # a single ragged tile row
    (8, 128, 3584, 512, dict(stream_k=1, max_ctas=37, comm_ctas=5)),
    (3, 640, 256, 1536, dict(stream_k=1, cta_pair=-1, max_ctas=13)),   # ranges longer than a tile: whole tiles + two parts
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("W,M,nl,K,kw", STREAMK_SHAPES)
def test_stream_k_exact_integer_full_heap_image(mode, dtype, W, M, nl, K, kw):
    """Tiles computed in k-range parts and reduced through the workspace: with integer-valued inputs the sums are
    exact in any order, so the whole heap image must still equal the oracle's byte for byte; run twice so that the
    arrival counters and the workspace are seen to be reusable."""
    N = W * nl
    A = inputs.matrix(47, inputs.STREAM_A, M, K, "ternary:0.25", dtype)
    Bs = [inputs.matrix(47, inputs.STREAM_B0 + r, nl, K, "smallint:1", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        img = None
        for epoch in (1, 2):
            run_gemm(g, A, Bs, dtype, mode, epoch=epoch, with_locks_zeroed=(epoch == 1), **kw)
            host = g.to_host()
            img, _ = expected_image(g, A, Bs, dtype, mode, epoch=epoch, c_full=None if img is None else c_slot(img.mem, g, 0, gemm_layout(M, N, W, True)[0], M, N).copy())
            assert np.array_equal(host, img.mem), (epoch, first_diff(host, img.mem))


def test_stream_k_real_valued_is_deterministic_and_within_tolerance():
    W, M, nl, K, dtype = 8, 128, 1024, 4096, "bf16"
    N = W * nl
    A, Bs = inputs.gemm_inputs(inputs.SEED0 + 3, W, M, N, K, "normal002", dtype)
    c_ref = oracle.gemm_block(A, Bs, dtype)
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        outs = []
        for rep in range(3):
            g.mem.fill_(SENTINEL)
            c_off = run_gemm(g, A, Bs, dtype, iris.IRIS_MODE_WORKGROUP_SPECIALIZED, stream_k=1)[0]
            host = g.to_host()
            c0 = c_slot(host, g, 0, c_off, M, N).copy()
            check_tolerance(c0, c_ref, dtype)
            for s in range(1, W):
                assert np.array_equal(c_slot(host, g, s, c_off, M, N), c0)
            outs.append(c0)
        assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])   # the parts are added in a fixed order


@pytest.mark.parametrize("wg_tail", [0, 1, 3, 1000])
@pytest.mark.parametrize("W,M,nl,K,kw", [
    (2, 1000, 512, 200, dict()),                            # CTA pairs, 4 x 4 pair tiles
    (2, 1000, 512, 200, dict(static_schedule=1, max_ctas=8)),
    (8, 1280, 384, 64, dict(max_ctas=24, comm_ctas=4)),     # single-CTA kernel, several waves
    (3, 520, 392, 328, dict(cta_pair=-1, max_ctas=9)),
    (4, 640, 512, 1024, dict(cta_pair=-1, stream_k=1, max_ctas=21)),
    (2, 600, 448, 136, dict(max_ctas=6)),                   # CTA pairs with a ragged shard: 2 producer pairs, 1 communication pair
])
def test_workgroup_specialized_tail_tiles_scattered_by_producers(wg_tail, W, M, nl, K, kw):
    """The last wave's tiles (or the last n) are written to all slots by their producers, the rest go through the lock
    handshake: the heap image -- C everywhere, flags, locks back at 0 -- is the oracle's either way."""
    N, dtype, mode = W * nl, "bf16", iris.IRIS_MODE_WORKGROUP_SPECIALIZED
    A = inputs.matrix(53, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(53, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        run_gemm(g, A, Bs, dtype, mode, wg_tail=wg_tail, **kw)
        host = g.to_host()
        img, _ = expected_image(g, A, Bs, dtype, mode)
        assert np.array_equal(host, img.mem), first_diff(host, img.mem)


def test_producers_take_over_what_the_communication_ctas_cannot_finish():
    """Two communication CTAs for a scatter that needs many more: with the default rule the producers keep most tiles
    (and say so), with Listing 5 throughout they keep none; the heap image is the oracle's in both cases."""
    W, M, nl, K, dtype, mode = 8, 2048, 512, 512, "bf16", iris.IRIS_MODE_WORKGROUP_SPECIALIZED
    N = W * nl
    A = inputs.matrix(59, inputs.STREAM_A, M, K, "ternary:0.25", dtype)
    Bs = [inputs.matrix(59, inputs.STREAM_B0 + r, nl, K, "smallint:1", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    c_full = None
    for wg_tail, comm in ((0, 2), (0, 0), (-1, 2), (0, 40)):
        with GpuHeap(W, bpr) as g:
            run_gemm(g, A, Bs, dtype, mode, wg_tail=wg_tail, comm_ctas=comm)
            kept, queued = iris.iris_gemm_takeover_stats(g.h)
            host = g.to_host()
            img, c_full = expected_image(g, A, Bs, dtype, mode, c_full=c_full)
            assert np.array_equal(host, img.mem), (wg_tail, comm, first_diff(host, img.mem))
            assert queued == 0
            if wg_tail < 0:
                assert kept == 0
            elif comm == 2:
                assert kept > 0          # 8 x 16 pair tiles, 73 producer pairs: one full wave before the last, far too much for 12 warps


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("W,M,nl,K", [(4, 1300, 384, 136),     # A is the smaller operand: one block per rank's shard
                                      (2, 1300, 256, 136)],    # B is smaller: row blocks of A (512, 512, 276)
                         ids=["by_ranks", "by_rows"])
def test_host_buffer_call_pipelined_over_blocks(mode, W, M, nl, K):
    """The host-buffer call copies, computes and copies back block by block on three streams: the host outputs and
    the whole heap image must be what the single call on device buffers gives (the oracle's)."""
    dtype = "bf16"
    N = W * nl
    A = inputs.matrix(61, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(61, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bias = inputs.vector(61, inputs.STREAM_BIAS, N, "smallint:3", dtype)
    nt = oracle.num_tiles(M, N, W)
    c_off, flag_off = 0, (M * N * 2 + 255) // 256 * 256                  # the short form's layout
    lock_off = flag_off + (nt * 4 + 255) // 256 * 256
    out_off = lock_off + (nt * 4 + 255) // 256 * 256
    assert out_off == iris.iris_gemm_out_offset(M, N, W)
    bpr = out_off + (M * N * 2 + 255) // 256 * 256 + 256
    with GpuHeap(W, bpr) as g:
        img = g.image()
        for s in range(W):                       # the call clears its own flag and lock arrays (in whole 256-byte units)
            img.view(s, flag_off, out_off - flag_off)[:] = 0
        C_host, OUT_host = np.zeros((M, N), dtype=np.uint16), np.zeros((M, N), dtype=np.uint16)
        flags = np.zeros((W, nt), dtype=np.int32)
        for call in (1, 2):                      # the second call reuses the handle's streams, events and staging
            iris.iris_gemm_all_scatter_host(A, Bs, C_host, flags, bias, OUT_host, g.h, M, N, K, W, mode, iris.IRIS_BF16, W - 1)
            assert np.all(flags == call)
        img.gemm_all_scatter(A, Bs, dtype, c_off, flag_off, 2, lock_off if mode == iris.IRIS_MODE_WORKGROUP_SPECIALIZED else None)
        img.consume_bias(dtype, c_off, out_off, M, N, bias)
        host = g.to_host()
        assert np.array_equal(host, img.mem), first_diff(host, img.mem)
        c_ref = c_slot(img.mem, g, 0, c_off, M, N)
        assert np.array_equal(C_host, c_ref)
        assert np.array_equal(OUT_host, oracle.consume_bias_rows(c_ref, bias, dtype))


RANK_RANGE_SHAPES = [
    # W, M, N_local, K, kwargs
    (4, 520, 512, 136, dict()),                              # CTA pairs
    (8, 384, 256, 192, dict(max_ctas=20, comm_ctas=4)),
    (3, 130, 136, 72, dict()),                               # single-CTA kernel, ragged everything
    (4, 640, 512, 1024, dict(cta_pair=-1, stream_k=1, max_ctas=21)),
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("W,M,nl,K,kw", RANK_RANGE_SHAPES)
def test_rank_range_one_call_touches_only_its_ranks(mode, W, M, nl, K, kw):
    """rank_first / rank_count: one call computes and scatters only those ranks' column shards (what one rank of a real
    job would run).  After a call for ranks [1, W-1) the other ranks' columns, flags and locks are still the sentinel;
    after the remaining ranks' calls the heap image is the full call's (the oracle's)."""
    N, dtype = W * nl, "bf16"
    A = inputs.matrix(67, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(67, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bias = inputs.vector(67, inputs.STREAM_BIAS, N, "smallint:3", dtype)
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    tm_n, ppr = -(-M // 128), -(-nl // 128)
    c_full = oracle.gemm_block(A, Bs, dtype)
    out_full = oracle.consume_bias_rows(c_full, bias, dtype)
    with GpuHeap(W, bpr) as g:
        img = g.image()
        for s in range(W):
            img.view(s, lock_off, nt * 4, np.int32)[:] = 0
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        dA, dbias = dev16(A), dev16(bias)

        def call(first, count):
            dB = [dev16(Bs[r]) if first <= r < first + count else None for r in range(W)]     # the others are not needed
            iris.iris_gemm_all_scatter_ex(g.h, dA, dB, M, N, K, W, mode, iris.IRIS_BF16, c_off, flag_off, lock_off, 5, rank_first=first,
                                          rank_count=count, consumer_bias=dbias, consumer_out_off=out_off, **kw)
            iris.iris_status_check(g.h)
            for s in range(W):                                   # the oracle's image, restricted to these ranks
                cv = img.view(s, c_off, M * N * 2, np.uint16).reshape(M, N)
                ov = img.view(s, out_off, M * N * 2, np.uint16).reshape(M, N)
                fv = img.view(s, flag_off, nt * 4, np.int32).reshape(tm_n, W, ppr)
                for r in range(first, first + count):
                    cv[:, r * nl:(r + 1) * nl] = c_full[:, r * nl:(r + 1) * nl]
                    ov[:, r * nl:(r + 1) * nl] = out_full[:, r * nl:(r + 1) * nl]
                    fv[:, r, :] = 5
            host = g.to_host()
            assert np.array_equal(host, img.mem), (first, count, first_diff(host, img.mem))

        call(1, W - 2)
        call(0, 1)
        call(W - 1, 1)
        full, _ = expected_image(g, A, Bs, dtype, mode, epoch=5, c_full=c_full)
        full.consume_bias(dtype, c_off, out_off, M, N, bias)
        assert np.array_equal(img.mem, full.mem)                 # the three partial images add up to the oracle's full one
