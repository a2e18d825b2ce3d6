"""Parity at the benchmark's full sizes, in every launch configuration bench.py times.

The oracle cannot finish a 4.4 TFLOP fp64 GEMM, so values are checked on publication tiles that the oracle computes one
by one from the same seeded inputs: a seeded random sample plus the first and last tile row and the first and last tile
column of every rank shard (where a wrong edge, rank offset or raster wrap would show).  Replication (all W copies
byte-identical), flags, locks and the consumer's output are checked at full size on the device (they are memcmp / scans).
The oracle's tiles are computed once per workload and shared by the schedules that are checked on it: every schedule
must produce the same C.
"""
import functools

import numpy as np
import pytest
import torch

import oracle
import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import check_tolerance

pytestmark = pytest.mark.gpu


def align(x, a=256):
    return (x + a - 1) // a * a


@functools.lru_cache(maxsize=1)
def _workload(W, M, N, K, dist, dtype, seed):
    """Host inputs and their device copies (kept for the schedules that share a workload; one workload at a time)."""
    A, Bs = inputs.gemm_inputs(seed, W, M, N, K, dist, dtype)
    bias = inputs.vector(seed, inputs.STREAM_BIAS, N, "uniform", dtype)
    dA = torch.from_numpy(A.view(np.int16)).cuda()
    dB = [torch.from_numpy(b.view(np.int16)).cuda() for b in Bs]
    dbias = torch.from_numpy(bias.view(np.int16)).cuda()
    return A, Bs, bias, dA, dB, dbias, {}


def sample_tiles(M, N, W, n_random, seed, edges):
    """Publication tile ids: n_random seeded picks, tiles 0 and nt-1, and (edges) the first / last tile row and the
    first / last tile column of every rank shard."""
    nl = N // W
    tm_n, tnl = -(-M // 128), -(-nl // 128)
    nt = tm_n * W * tnl
    rng = np.random.default_rng(seed)
    picks = {0, nt - 1} | {int(t) for t in rng.choice(nt, size=min(n_random, nt), replace=False)}
    if edges:
        per_row = W * tnl
        picks |= set(range(per_row)) | set(range((tm_n - 1) * per_row, nt))
        for tm in range(tm_n):
            for r in range(W):
                picks.add(tm * per_row + r * tnl)
                picks.add(tm * per_row + r * tnl + tnl - 1)
    return sorted(picks)


def _run_fullsize(W, M, N, K, dist, dtype, mode, seed, n_random, edges=False, with_consumer=True, fused=True, two_streams=False, **kw):
    nl = N // W
    nt = iris.iris_num_tiles(M, N, W)
    flag_off = align(M * N * 2)
    lock_off = flag_off + align(nt * 4)
    out_off = iris.iris_gemm_out_offset(M, N, W)
    bpr = align(out_off + M * N * 2)
    A, Bs, bias, dA, dB, dbias, refs = _workload(W, M, N, K, dist, dtype, seed)
    mem = torch.full((W * bpr,), 0xFF, dtype=torch.uint8, device="cuda")      # NaN poison
    h = iris.iris_heap_create(W, bpr, external_base=mem.data_ptr())
    s1, s2, s3 = (torch.cuda.Stream() for _ in range(3)) if two_streams else (None, None, None)
    try:
        iris.iris_flags_fill(h, flag_off, nt, 0)
        iris.iris_flags_fill(h, lock_off, nt, 0)
        torch.cuda.synchronize()
        for epoch in (1, 2):           # the second pass runs over the first one's data, as the timed loop does
            if two_streams:
                # the unfused form: producers on one stream, communication kernel on a second, consumer on a third
                iris.iris_gemm_all_scatter_unfused(h, dA, dB, M, N, K, W, iris.DTYPES[dtype], 0, flag_off, lock_off, epoch, s1, s2, **kw)
                if with_consumer:
                    iris.iris_consume_bias(h, 0, out_off, flag_off, dbias, M, N, W, iris.DTYPES[dtype], epoch, ctas=592, stream=s3)
                    s3.synchronize()
                iris.iris_status_check(h, s1)
                continue
            # fused: the consumer rides inside the GEMM launch where the kernel supports it; otherwise it is the second
            # kernel of the step, exactly as bench.py's default step launches it
            iris.iris_gemm_all_scatter_ex(h, dA, dB, M, N, K, W, iris.MODES[mode], iris.DTYPES[dtype], 0, flag_off, lock_off, epoch,
                                          consumer_bias=dbias if (with_consumer and fused) else None, consumer_out_off=out_off, **kw)
            if with_consumer and not fused:
                iris.iris_consume_bias(h, 0, out_off, flag_off, dbias, M, N, W, iris.DTYPES[dtype], epoch)
            iris.iris_status_check(h)
        slots = mem.view(W, bpr)
        c0 = slots[0, : M * N * 2]
        for s in range(1, W):                                       # replication: all W copies byte-identical
            assert torch.equal(slots[s, : M * N * 2], c0), f"slot {s} differs from slot 0"
            if with_consumer:
                assert torch.equal(slots[s, out_off: out_off + M * N * 2], slots[0, out_off: out_off + M * N * 2])
        for s in range(W):                                          # flags == epoch, locks consumed, everywhere
            assert bool(torch.all(slots[s, flag_off: flag_off + nt * 4].view(torch.int32) == 2))
            assert bool(torch.all(slots[s, lock_off: lock_off + nt * 4].view(torch.int32) == 0))
        c_host = c0.view(torch.int16).view(M, N)
        out_host = slots[0, out_off: out_off + M * N * 2].view(torch.int16).view(M, N)
        tiles = sample_tiles(M, N, W, n_random, seed, edges)
        for t in tiles:
            m0, m1, n0, n1 = oracle.tile_rect(t, M, N, W)
            r = n0 // nl
            if t not in refs:
                refs[t] = oracle.gemm_block(A[m0:m1], [Bs[r][n0 - r * nl: n1 - r * nl]], dtype)
            got = c_host[m0:m1, n0:n1].cpu().numpy().view(np.uint16)
            check_tolerance(got, refs[t], dtype)
            if with_consumer:                                       # consumer: bit-exact on the GPU's own C
                exp = oracle.consume_bias_rows(np.ascontiguousarray(got), bias[n0:n1], dtype)
                assert np.array_equal(out_host[m0:m1, n0:n1].cpu().numpy().view(np.uint16), exp)
        return len(tiles)
    finally:
        iris.iris_heap_destroy(h)


# W=8, M=8192, N=K=16384, bf16 uniform[-1,1): the workload the headline figure is quoted on, in every schedule bench.py's
# `modes` block times on it, plus the two forms of the consumer.  256 random publication tiles of 8192 plus the edge
# tiles (about 1500 tiles in all, computed by the oracle once and shared).
HEADLINE = (8, 8192, 16384, 16384, "uniform", "bf16")
HEADLINE_CASES = [
    ("workgroup_specialized", dict(fused=False)),                       # the default step: consumer as a second kernel
    ("workgroup_specialized", dict(fused=True)),                        # consumer warps inside the GEMM launch
    ("workgroup_specialized", dict(fused=False, wg_tail=-1)),           # Listing 5 for every tile
    ("fused_sequential", dict(fused=True)),
    ("bulk_synchronous", dict(fused=False)),
    ("workgroup_specialized", dict(two_streams=True)),                  # unfused: two kernels on two streams, consumer on a third
]


@pytest.mark.parametrize("mode,kw", HEADLINE_CASES,
                         ids=["wg_consumer_kernel", "wg_consumer_warps", "wg_every_tile_via_comm_ctas", "fused_sequential", "bulk_synchronous",
                              "unfused_two_streams"])
def test_headline_workload_every_schedule_sampled_tiles(mode, kw):
    n = _run_fullsize(*HEADLINE, mode, inputs.SEED0 + 4, n_random=256, edges=True, **kw)
    assert n >= 1400


@pytest.mark.parametrize("mode", ["bulk_synchronous", "fused_sequential", "workgroup_specialized"])
def test_config3_sampled_tiles(mode):
    """W=8, M=4096, N=8192, K=8192, bf16 normal(0, 0.02): 64 random tiles plus the edge tiles (about 600 of 2048)."""
    _run_fullsize(8, 4096, 8192, 8192, "normal002", "bf16", mode, inputs.SEED0 + 2, n_random=64, edges=True)


@pytest.mark.parametrize("comm_ctas", [8, 16, 32])
def test_config4_skinny_workgroup_specialized(comm_ctas):
    """W=8, M=128, N=28672, K=8192, bf16 normal(0, 0.02): the memory-bound decode-like shape; every tile of its one tile row."""
    _run_fullsize(8, 128, 28672, 8192, "normal002", "bf16", "workgroup_specialized", inputs.SEED0 + 3, n_random=32, edges=True, comm_ctas=comm_ctas)


@pytest.mark.parametrize("mode", ["fused_sequential", "bulk_synchronous"])
def test_config4_skinny_other_schedules(mode):
    _run_fullsize(8, 128, 28672, 8192, "normal002", "bf16", mode, inputs.SEED0 + 3, n_random=32, edges=True)


@pytest.mark.parametrize("W,M", [(2, 8192), (4, 8192), (2, 1024), (4, 1024), (8, 1024)])
def test_config5_sweep_members_sampled_tiles(W, M):
    """The other members of the W x M sweep on N = K = 16384 (bench.py times them in all schedules; here the
    workgroup-specialised one, 48 random tiles plus the corner tiles of the output)."""
    _run_fullsize(W, M, 16384, 16384, "uniform", "bf16", "workgroup_specialized", inputs.SEED0 + 4, n_random=48)


@pytest.mark.parametrize("mode", ["fused_sequential", "workgroup_specialized", "bulk_synchronous"])
@pytest.mark.parametrize("N,K", [(3584, 14336), (4608, 36864)], ids=["8192x3584x14336", "8192x4608x36864"])
def test_paper_shapes_with_global_n_ragged_shards(N, K, mode):
    """The two shapes Section 5.2 names, read with N global (W=8, M=8192, bf16 normal(0, 0.02)): shards of 448 = 256 + 192
    and 576 = 2 x 256 + 64 columns, so every shard ends in a fused unit (and, for 576, on the ring of two two-k-block
    stages and one one-k-block stage) and in a narrow publication tile.  24 random tiles plus the corner tiles."""
    _run_fullsize(8, 8192, N, K, "normal002", "bf16", mode, inputs.SEED0 + 6, n_random=24)


def test_paper_shape_with_n_per_rank():
    """8192 x (8 x 3584) x 14336, the same shape read with N per rank (bench.py's sweep times it): 16 random tiles."""
    _run_fullsize(8, 8192, 8 * 3584, 14336, "normal002", "bf16", "workgroup_specialized", inputs.SEED0 + 7, n_random=16)
