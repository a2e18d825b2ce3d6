"""Protocol stress and randomised shapes for gemm_all_scatter.

No sanitizer is available for these kernels, so ordering bugs (a flag published before its tile, a consumer that
reads before acquiring, a lock taken twice) are hunted by repetition: small-K problems make the scatter, not the
GEMM, the bottleneck, so producers, communication CTAs and consumer warps all run at once; the heap is re-poisoned
with NaN patterns before every launch and the result is compared bit for bit with the first (oracle-checked) one.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import GpuHeap, dev16, first_diff, gemm_layout

pytestmark = pytest.mark.gpu

MODES = [iris.IRIS_MODE_BULK_SYNCHRONOUS, iris.IRIS_MODE_FUSED_SEQUENTIAL, iris.IRIS_MODE_WORKGROUP_SPECIALIZED]


@pytest.mark.parametrize("mode", [iris.IRIS_MODE_FUSED_SEQUENTIAL, iris.IRIS_MODE_WORKGROUP_SPECIALIZED])
@pytest.mark.parametrize("W,M,nl,K,kw", [
    (8, 2048, 256, 64, dict()),                              # pair kernel, K tiny: every tile is ready almost at once
    (8, 2048, 256, 64, dict(comm_ctas=2)),                   # communicators are the bottleneck
    (4, 1024, 512, 128, dict(static_schedule=1, comm_ctas=40)),
    (8, 1280, 384, 64, dict()),                              # single-CTA kernel (N_local % 256 != 0)
    (8, 2048, 256, 64, dict(wg_tail=-1)),                    # one wave: every tile through the lock handshake
    (8, 2048, 512, 64, dict(max_ctas=40)),                   # several waves, the last one scattered by its producers
    (8, 1280, 384, 64, dict(wg_tail=-1, comm_ctas=3)),
])
def test_repeated_launches_on_a_poisoned_heap(mode, W, M, nl, K, kw):
    N, dtype = W * nl, "bf16"
    A = inputs.matrix(81, inputs.STREAM_A, M, K, "smallint:2", dtype)
    Bs = [inputs.matrix(81, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bias = inputs.vector(81, inputs.STREAM_BIAS, N, "smallint:3", dtype)
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    with GpuHeap(W, bpr, fill=0xFF) as g:
        img = g.image(fill=0xFF)
        for s in range(W):
            img.view(s, lock_off, nt * 4, np.int32)[:] = 0
            img.view(s, flag_off, nt * 4, np.int32)[:] = 0
        iris.iris_flags_fill(g.h, flag_off, nt, 0)
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        dA, dB, dbias = dev16(A), [dev16(b) for b in Bs], dev16(bias)
        slots = g.mem.view(W, bpr)
        want_c = want_out = None
        for epoch in range(1, 61):
            slots[:, c_off:c_off + M * N * 2] = 0xFF            # poison C and OUT again (flags and locks stay)
            slots[:, out_off:out_off + M * N * 2] = 0xFF
            iris.iris_gemm_all_scatter_ex(g.h, dA, dB, M, N, K, W, mode, iris.IRIS_BF16, c_off, flag_off, lock_off, epoch,
                                          consumer_bias=dbias, consumer_out_off=out_off, **kw)
            if epoch == 1:                                       # first launch: the whole heap image against the oracle
                iris.iris_status_check(g.h)
                img.gemm_all_scatter(A, Bs, dtype, c_off, flag_off, 1, lock_off if mode == iris.IRIS_MODE_WORKGROUP_SPECIALIZED else None)
                img.consume_bias(dtype, c_off, out_off, M, N, bias)
                host = g.to_host()
                assert np.array_equal(host, img.mem), first_diff(host, img.mem)
                want_c = slots[:, c_off:c_off + M * N * 2].clone()
                want_out = slots[:, out_off:out_off + M * N * 2].clone()
            else:                                                # later launches: bit-identical C and OUT in every slot
                assert torch.equal(slots[:, c_off:c_off + M * N * 2], want_c), f"C differs at epoch {epoch}"
                assert torch.equal(slots[:, out_off:out_off + M * N * 2], want_out), f"OUT differs at epoch {epoch}"
                assert bool(torch.all(slots[:, flag_off:flag_off + nt * 4].view(torch.int32) == epoch))
                assert bool(torch.all(slots[:, lock_off:lock_off + nt * 4].view(torch.int32) == 0))
        iris.iris_status_check(g.h)


def test_random_shapes_exact_heap_image():
    """Seeded random (W, M, N_local, K, mode, knobs): integer-valued inputs, whole heap image byte for byte."""
    rng = np.random.default_rng(20251125)
    for case in range(24):
        W = int(rng.choice([1, 2, 3, 4, 5, 8]))
        M = int(rng.integers(1, 900))
        nl = int(rng.integers(1, 90)) * 8
        K = int(rng.integers(1, 60)) * 8
        mode = MODES[case % 3]
        kw = {}
        if rng.random() < 0.4:
            kw["max_ctas"] = int(rng.integers(2, 30))
        if rng.random() < 0.4:
            kw["comm_ctas"] = int(rng.integers(1, 12))
        if rng.random() < 0.3:
            kw["raster_group"] = int(rng.integers(1, 6))
        if rng.random() < 0.3:
            kw["static_schedule"] = 1
        if rng.random() < 0.2:
            kw["cta_pair"] = -1
        elif rng.random() < 0.4 and M > 128 and nl > 128:
            kw["cta_pair"] = 1      # pairs even where the shard is ragged
        if rng.random() < 0.5:
            kw["wg_tail"] = int(rng.choice([-1, 1, 2, 5]))
        if rng.random() < 0.3:
            kw["pace_stores"] = -1
        if kw.get("cta_pair") == -1 and rng.random() < 0.6:
            kw["stream_k"] = 1
        dtype = "bf16" if case % 2 else "fp16"
        N = W * nl
        A = inputs.matrix(900 + case, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
        Bs = [inputs.matrix(900 + case, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
        c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=False)
        nt = oracle.num_tiles(M, N, W)
        with GpuHeap(W, bpr) as g:
            img = g.image()
            for s in range(W):
                img.view(s, lock_off, nt * 4, np.int32)[:] = 0
            iris.iris_flags_fill(g.h, lock_off, nt, 0)
            iris.iris_gemm_all_scatter_ex(g.h, dev16(A), [dev16(b) for b in Bs], M, N, K, W, mode, iris.DTYPES[dtype], c_off, flag_off,
                                          lock_off, 7, **kw)
            iris.iris_status_check(g.h)
            img.gemm_all_scatter(A, Bs, dtype, c_off, flag_off, 7, lock_off if mode == iris.IRIS_MODE_WORKGROUP_SPECIALIZED else None)
            host = g.to_host()
            assert np.array_equal(host, img.mem), (case, W, M, nl, K, mode, kw, first_diff(host, img.mem))
