"""GPU parity for the flag-gated consumer (OUT = C + bias after acquiring each tile's flag) and for the
bounded device-side waits: a wait that can never be satisfied returns an error status, and the GPU
stays usable (nothing traps, nothing spins forever)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import SENTINEL, GpuHeap, dev16, first_diff, gemm_layout

pytestmark = pytest.mark.gpu

MODES = [iris.IRIS_MODE_BULK_SYNCHRONOUS, iris.IRIS_MODE_FUSED_SEQUENTIAL, iris.IRIS_MODE_WORKGROUP_SPECIALIZED]


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("W,M,nl", [(2, 256, 128), (4, 130, 136), (8, 384, 256)])
def test_consumer_matches_oracle_on_seeded_C(dtype, W, M, nl):
    """C, bias and flags are written directly; the consumer's output must equal the oracle's bit for bit."""
    N = W * nl
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    C = inputs.matrix(51, 0, M, N, "uniform", dtype)
    bias = inputs.vector(51, inputs.STREAM_BIAS, N, "uniform", dtype)
    nt = oracle.num_tiles(M, N, W)
    with GpuHeap(W, bpr) as g:
        img = g.image()
        for s in range(W):
            g.write(s, c_off, C)
            img.view(s, c_off, M * N * 2, np.uint16)[:] = C.reshape(-1)
        iris.iris_flags_fill(g.h, flag_off, nt, 9)
        img.publish_flags(flag_off, nt, 9)
        iris.iris_consume_bias(g.h, c_off, out_off, flag_off, dev16(bias), M, N, W, iris.DTYPES[dtype], 9)   # flag == epoch
        iris.iris_status_check(g.h)
        img.consume_bias(dtype, c_off, out_off, M, N, bias)
        host = g.to_host()
        assert np.array_equal(host, img.mem), first_diff(host, img.mem)
        iris.iris_consume_bias(g.h, c_off, out_off, flag_off, dev16(bias), M, N, W, iris.DTYPES[dtype], 5)   # flag > epoch passes too
        iris.iris_status_check(g.h)


@pytest.mark.parametrize("mode", MODES)
def test_producer_then_consumer_on_poisoned_heap(mode):
    """The heap starts as NaN patterns (0xFFFF); a consumer that read a tile before its flag would emit NaNs.
    OUT must equal the consumer definition applied to the GPU's own C, bit for bit (fp32 add + one rounding
    is deterministic), and C must be within tolerance of the oracle."""
    W, M, nl, K, dtype = 4, 512, 256, 512, "bf16"
    N = W * nl
    A, Bs = inputs.gemm_inputs(inputs.SEED0 + 4, W, M, N, K, "uniform", dtype)
    bias = inputs.vector(inputs.SEED0 + 4, inputs.STREAM_BIAS, N, "uniform", dtype)
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    with GpuHeap(W, bpr, fill=0xFF) as g:
        iris.iris_flags_fill(g.h, flag_off, nt, 0)
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        dA, dB, dbias = dev16(A), [dev16(b) for b in Bs], dev16(bias)
        for epoch in (1, 2):
            iris.iris_gemm_all_scatter_ex(g.h, dA, dB, M, N, K, W, mode, iris.IRIS_BF16, c_off, flag_off, lock_off, epoch)
            iris.iris_consume_bias(g.h, c_off, out_off, flag_off, dbias, M, N, W, iris.IRIS_BF16, epoch)
            iris.iris_status_check(g.h)
        host = g.to_host()
        c0 = host[c_off:c_off + M * N * 2].view(np.uint16).reshape(M, N)
        exp_out = oracle.consume_bias_rows(c0, bias, dtype)
        for s in range(W):
            out = host[s * bpr + out_off: s * bpr + out_off + M * N * 2].view(np.uint16).reshape(M, N)
            assert np.array_equal(out, exp_out)
        assert not np.isnan(oracle.decode(exp_out, dtype)).any()


def test_consumer_wait_that_cannot_be_satisfied_times_out_cleanly():
    W, M, nl = 2, 256, 128
    N = W * nl
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    with GpuHeap(W, bpr) as g:
        nt = oracle.num_tiles(M, N, W)
        iris.iris_flags_fill(g.h, flag_off, nt, 0)                      # nothing will ever publish epoch 1
        bias = torch.zeros(N, dtype=torch.int16, device="cuda")
        iris.iris_consume_bias(g.h, c_off, out_off, flag_off, bias, M, N, W, iris.IRIS_BF16, 1, 0, 2_000_000)   # 2 ms deadline
        with pytest.raises(iris.IrisError) as e:
            iris.iris_status_check(g.h)
        assert e.value.code == iris.IRIS_ERR_TIMEOUT
        assert e.value.detail[1] == 3 and e.value.detail[5] == 0 and e.value.detail[6] == 1   # consumer, seen 0, wanted 1
        out = g.view(0, out_off, M * N * 2)
        assert bool(torch.all(out == SENTINEL))                         # no tile was touched
        iris.iris_status_check(g.h)                                     # status cleared; context still healthy
        iris.iris_flags_fill(g.h, flag_off, nt, 1)
        iris.iris_consume_bias(g.h, c_off, out_off, flag_off, bias, M, N, W, iris.IRIS_BF16, 1)
        iris.iris_status_check(g.h)


def test_communication_ctas_give_up_when_a_lock_is_never_released():
    """Workgroup-specialised mode with the lock array pre-set to a value the handshake never produces for the
    communicators (2): producers' cas(0->1) misses, communicators never see 1, and their bounded wait expires."""
    W, M, nl, K = 2, 256, 128, 64
    N = W * nl
    A, Bs = inputs.gemm_inputs(3, W, M, N, K, "uniform", "bf16")
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    with GpuHeap(W, bpr) as g:
        nt = oracle.num_tiles(M, N, W)
        iris.iris_flags_fill(g.h, lock_off, nt, 3)    # neither free (0) nor a state the communicators act on (1, 2)
        iris.iris_flags_fill(g.h, flag_off, nt, 0)
        iris.iris_gemm_all_scatter_ex(g.h, dev16(A), [dev16(b) for b in Bs], M, N, K, W, iris.IRIS_MODE_WORKGROUP_SPECIALIZED,
                                      iris.IRIS_BF16, c_off, flag_off, lock_off, 1, spin_timeout_ns=3_000_000, wg_tail=-1)
        with pytest.raises(iris.IrisError) as e:
            iris.iris_status_check(g.h)
        assert e.value.code == iris.IRIS_ERR_TIMEOUT and e.value.detail[1] == 1
        flags = g.view(0, flag_off, nt * 4, torch.int32)
        assert bool(torch.all(flags == 0))                              # nothing was published
        # the device is still usable: a correct run right after succeeds
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        iris.iris_gemm_all_scatter_ex(g.h, dev16(A), [dev16(b) for b in Bs], M, N, K, W, iris.IRIS_MODE_WORKGROUP_SPECIALIZED,
                                      iris.IRIS_BF16, c_off, flag_off, lock_off, 1)
        iris.iris_status_check(g.h)
        assert bool(torch.all(flags == 1))


FUSED_SHAPES = [
    # W, M, N_local, K, kwargs
    (2, 1000, 512, 200, dict()),                     # CTA-pair kernel: consumer warps inside the GEMM launch
    (8, 512, 256, 320, dict(comm_ctas=4)),
    (4, 640, 512, 128, dict(static_schedule=1, max_ctas=12, comm_ctas=4)),
    (4, 130, 136, 72, dict()),                       # ragged: single-CTA kernel, consumer follows as a kernel
    (2, 384, 256, 192, dict(cta_pair=-1)),
    (3, 520, 392, 328, dict(fuse_tail=1)),           # CTA pairs, ragged shard: the remainder rides with the last full tile
    (2, 600, 576, 136, dict(fuse_tail=1, comm_ctas=4)),   # 576 = 2 x 256 + 64: one plain unit and one fused unit per shard
    (2, 600, 576, 136, dict(fuse_tail=-1)),          # the same with the remainder as a tile of its own
]


@pytest.mark.parametrize("mode,wg_tail", [(MODES[0], 0), (MODES[1], 0), (MODES[2], -1), (MODES[2], 0), (MODES[2], 2)],
                         ids=["bulk_synchronous", "fused_sequential", "workgroup_specialized_no_tail", "workgroup_specialized", "workgroup_specialized_tail2"])
@pytest.mark.parametrize("W,M,nl,K,kw", FUSED_SHAPES)
def test_consumer_as_part_of_the_gemm_call(mode, wg_tail, W, M, nl, K, kw):
    """gemm_all_scatter with consumer_bias set: C, flags, locks and OUT must equal the oracle's heap image byte for
    byte (integer-valued inputs make the GEMM exact).  The heap starts as NaN patterns, so a consumer warp that read
    a tile before its flag was published would leave NaNs in OUT."""
    N, dtype = W * nl, "bf16"
    A = inputs.matrix(71, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(71, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bias = inputs.vector(71, inputs.STREAM_BIAS, N, "smallint:3", dtype)
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    nt = oracle.num_tiles(M, N, W)
    with GpuHeap(W, bpr, fill=0xFF) as g:
        img = g.image(fill=0xFF)
        iris.iris_flags_fill(g.h, flag_off, nt, 0)
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        for s in range(W):
            img.view(s, lock_off, nt * 4, np.int32)[:] = 0
        dA, dB, dbias = dev16(A), [dev16(b) for b in Bs], dev16(bias)
        for epoch in (1, 2, 3):
            iris.iris_gemm_all_scatter_ex(g.h, dA, dB, M, N, K, W, mode, iris.IRIS_BF16, c_off, flag_off, lock_off, epoch,
                                          consumer_bias=dbias, consumer_out_off=out_off, wg_tail=wg_tail, **kw)
        iris.iris_status_check(g.h)
        img.gemm_all_scatter(A, Bs, dtype, c_off, flag_off, 3, lock_off if mode == iris.IRIS_MODE_WORKGROUP_SPECIALIZED else None)
        img.consume_bias(dtype, c_off, out_off, M, N, bias)
        host = g.to_host()
        assert np.array_equal(host, img.mem), first_diff(host, img.mem)


def test_consumer_arguments_are_checked():
    W, M, nl, K = 2, 256, 256, 64
    N = W * nl
    c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
    with GpuHeap(W, bpr) as g:
        d = torch.zeros(1 << 16, dtype=torch.int16, device="cuda")
        for out, code in [(c_off, iris.IRIS_ERR_ARG), (flag_off, iris.IRIS_ERR_ARG), (bpr - 256, iris.IRIS_ERR_RANGE), (out_off + 8, iris.IRIS_ERR_ARG)]:
            with pytest.raises(iris.IrisError) as e:
                iris.iris_gemm_all_scatter_ex(g.h, d, [d, d], M, N, K, W, 1, iris.IRIS_BF16, c_off, flag_off, lock_off, 1,
                                              consumer_bias=d, consumer_out_off=out)
            assert e.value.code == code, (out, e.value)
        torch.cuda.synchronize()
        assert bool(torch.all(g.mem == SENTINEL))

