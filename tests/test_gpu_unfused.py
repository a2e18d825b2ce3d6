"""GPU parity for the unfused producer-consumer pattern (Section 4.1): the workgroup-specialised schedule as two
kernels on two streams -- GEMM producers on one, the communication kernel (lock poll, copy, flag publication) on the
other -- against the CPU oracle.  The heap image must be the one every other schedule produces: C in all W slots,
flags == epoch, locks back at 0.  A consumer on a third stream overlaps both.

The dependency between the two kernels runs one way (the second waits for locks the first sets), the producers are
launched first and every wait has a deadline, so nothing here can hang: the timeout test shows that a handshake that
can never complete ends with a status code and a usable context.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import SENTINEL, GpuHeap, check_tolerance, dev16, first_diff, gemm_layout

pytestmark = pytest.mark.gpu

WG = iris.IRIS_MODE_WORKGROUP_SPECIALIZED

SHAPES = [
    # W, M, N_local, K, kwargs
    (2, 256, 128, 256, dict()),                                  # single-CTA kernel, 128-wide tiles
    (4, 130, 136, 72, dict()),                                   # everything ragged
    (3, 520, 392, 328, dict()),                                  # CTA pairs, ragged shard
    (3, 520, 392, 328, dict(cta_pair=-1, max_ctas=9, comm_ctas=3)),
    (2, 1000, 512, 200, dict(comm_ctas=8)),                      # CTA pairs, 4 x 4 pair tiles
    (8, 1280, 384, 64, dict(max_ctas=24, comm_ctas=4)),          # several waves on 20 producers
    (2, 384, 256, 192, dict(cta_pair=-1, block_n=256)),          # single-CTA kernel, 256-wide tiles
    (8, 2048, 512, 128, dict(comm_ctas=2)),                      # far too few communication CTAs: producers take tiles over
]


def _expected(g, A, Bs, dtype, epoch, c_full=None):
    M = A.shape[0]
    W, nl = len(Bs), Bs[0].shape[0]
    N = W * nl
    c_off, flag_off, lock_off, _, _ = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    img = g.image()
    for s in range(W):
        img.view(s, lock_off, nt * 4, np.int32)[:] = 0
    if c_full is None:
        c_full = oracle.gemm_block(A, Bs, dtype)
    img.all_scatter(c_off, c_full)
    img.publish_flags(flag_off, nt, epoch)
    img.consume_locks(lock_off, M, N)
    return img, c_full


@pytest.mark.parametrize("wg_tail", [-1, 0], ids=["every_tile_handed_over", "default_tail_rule"])
@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("W,M,nl,K,kw", SHAPES)
def test_unfused_two_streams_full_heap_image(wg_tail, dtype, W, M, nl, K, kw):
    N = W * nl
    A = inputs.matrix(83, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(83, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    c_off, flag_off, lock_off, _, bpr = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    with GpuHeap(W, bpr) as g:
        dA, dB = dev16(A), [dev16(b) for b in Bs]
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        torch.cuda.synchronize()
        c_full = None
        for epoch in (1, 2):             # the second pass finds the first one's data, flags and (reset) locks
            iris.iris_gemm_all_scatter_unfused(g.h, dA, dB, M, N, K, W, iris.DTYPES[dtype], c_off, flag_off, lock_off, epoch, s1, s2,
                                               wg_tail=wg_tail, **kw)
            iris.iris_status_check(g.h, s1)      # the producer stream has joined the communication stream
            host = g.to_host()
            img, c_full = _expected(g, A, Bs, dtype, epoch, c_full)
            assert np.array_equal(host, img.mem), (epoch, first_diff(host, img.mem))


def test_unfused_with_consumer_on_a_third_stream_real_valued():
    """Producers, communication kernel and the flag-gated consumer as three kernels on three streams, launched back to
    back: C within tolerance of the oracle, every copy identical, OUT = C + bias bit-exact on the GPU's own C."""
    W, M, nl, K, dtype = 8, 1024, 512, 1024, "bf16"
    N = W * nl
    A, Bs = inputs.gemm_inputs(inputs.SEED0 + 2, W, M, N, K, "normal002", dtype)
    bias = inputs.vector(inputs.SEED0 + 2, inputs.STREAM_BIAS, N, "uniform", dtype)
    c_ref = oracle.gemm_block(A, Bs, dtype)
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    s1, s2, s3 = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    with GpuHeap(W, bpr, fill=0xFF) as g:                               # NaN poison: a consumer that reads early is caught
        dA, dB, dbias = dev16(A), [dev16(b) for b in Bs], dev16(bias)
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        iris.iris_flags_fill(g.h, flag_off, nt, 0)
        torch.cuda.synchronize()
        for epoch in (1, 2, 3):
            iris.iris_gemm_all_scatter_unfused(g.h, dA, dB, M, N, K, W, iris.DTYPES[dtype], c_off, flag_off, lock_off, epoch, s1, s2)
            iris.iris_consume_bias(g.h, c_off, out_off, flag_off, dbias, M, N, W, iris.DTYPES[dtype], epoch, ctas=64, stream=s3)
            s3.synchronize()
            iris.iris_status_check(g.h, s1)
            host = g.to_host()
            c0 = host[c_off: c_off + M * N * 2].view(np.uint16).reshape(M, N)
            check_tolerance(c0, c_ref, dtype)
            exp_out = oracle.consume_bias_rows(np.ascontiguousarray(c0), bias, dtype)
            for s in range(W):
                assert np.array_equal(host[s * bpr + c_off: s * bpr + c_off + M * N * 2].view(np.uint16).reshape(M, N), c0)
                assert np.array_equal(host[s * bpr + out_off: s * bpr + out_off + M * N * 2].view(np.uint16).reshape(M, N), exp_out)
                assert np.all(host[s * bpr + flag_off: s * bpr + flag_off + nt * 4].view(np.int32) == epoch)
                assert np.all(host[s * bpr + lock_off: s * bpr + lock_off + nt * 4].view(np.int32) == 0)


def test_unfused_argument_errors():
    W, M, nl, K = 2, 256, 128, 64
    N = W * nl
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    with GpuHeap(W, bpr) as g:
        d = torch.zeros(1 << 16, dtype=torch.int16, device="cuda")
        with pytest.raises(iris.IrisError) as e:      # one stream for both kernels
            iris.iris_gemm_all_scatter_unfused(g.h, d, [d, d], M, N, K, W, iris.IRIS_BF16, c_off, flag_off, lock_off, 1, s1, s1)
        assert e.value.code == iris.IRIS_ERR_ARG
        with pytest.raises(iris.IrisError) as e:      # another schedule
            iris.iris_gemm_all_scatter_ex(g.h, d, [d, d], M, N, K, W, iris.IRIS_MODE_FUSED_SEQUENTIAL, iris.IRIS_BF16, c_off, flag_off, lock_off, 1,
                                          stream=s1, comm_stream=s2)
        assert e.value.code == iris.IRIS_ERR_ARG
        with pytest.raises(iris.IrisError) as e:      # consumer warps inside the producer kernel would wait on the second kernel
            iris.iris_gemm_all_scatter_unfused(g.h, d, [d, d], M, N, K, W, iris.IRIS_BF16, c_off, flag_off, lock_off, 1, s1, s2,
                                               consumer_bias=d, consumer_out_off=out_off)
        assert e.value.code == iris.IRIS_ERR_UNSUPPORTED
        torch.cuda.synchronize()
        assert bool(torch.all(g.mem == SENTINEL))


def test_unfused_handshake_that_cannot_complete_times_out_and_leaves_the_context_usable():
    """Locks preset to 3: the producers' cas(0 -> 1) never succeeds, so the communication kernel never sees a tile
    handed over.  Its bounded wait (3 ms here) runs out, the status block says so, and the next call works."""
    W, M, nl, K, dtype = 2, 256, 128, 128, "bf16"
    N = W * nl
    A = inputs.matrix(89, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(89, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    c_off, flag_off, lock_off, _, bpr = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    with GpuHeap(W, bpr) as g:
        dA, dB = dev16(A), [dev16(b) for b in Bs]
        iris.iris_flags_fill(g.h, lock_off, nt, 3)
        torch.cuda.synchronize()
        iris.iris_gemm_all_scatter_unfused(g.h, dA, dB, M, N, K, W, iris.DTYPES[dtype], c_off, flag_off, lock_off, 1, s1, s2,
                                           wg_tail=-1, spin_timeout_ns=3_000_000)
        with pytest.raises(iris.IrisError) as e:
            iris.iris_status_check(g.h, s1)
        assert e.value.code == iris.IRIS_ERR_TIMEOUT
        # the context is intact: the same call with the locks in their initial state completes and matches the oracle
        g.mem.fill_(SENTINEL)
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        torch.cuda.synchronize()
        iris.iris_gemm_all_scatter_unfused(g.h, dA, dB, M, N, K, W, iris.DTYPES[dtype], c_off, flag_off, lock_off, 2, s1, s2, wg_tail=-1)
        iris.iris_status_check(g.h, s1)
        host = g.to_host()
        img, _ = _expected(g, A, Bs, dtype, 2)
        assert np.array_equal(host, img.mem), first_diff(host, img.mem)
