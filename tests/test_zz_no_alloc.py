"""The allocation-free entry point against the regular one.

iris_gemm_all_scatter_noalloc() serves callers that cannot allocate device memory (a process whose HBM is
already handed out to a framework's pool, a loop that cannot take the synchronisation an allocation implies):
it takes raw slot addresses instead of a heap handle and keeps its locks and status block in a fixed array
inside the library.  That array is shared by all calls and keeps its old contents, so the test calls it twice
in a row, with different inputs, and compares every byte of C and every flag in every slot with what
iris_gemm_all_scatter_ex (workgroup-specialised, default tuning) produced for the same inputs.  Both paths build
their plan with the same code and run the same kernels, so the comparison is bit-exact, which is tighter than the tolerance the other GPU tests use.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import SENTINEL, GpuHeap, check_tolerance, dev16, gemm_layout

pytestmark = pytest.mark.gpu


def _reference_run(W, M, N, K, dtype, A, Bs, epoch):
    """Existing entry point, workgroup-specialised, on a heap object."""
    c_off, flag_off, lock_off, _, bpr = gemm_layout(M, N, W)
    nt = oracle.num_tiles(M, N, W)
    with GpuHeap(W, bpr) as g:
        iris.iris_flags_fill(g.h, lock_off, nt, 0)
        iris.iris_gemm_all_scatter_ex(g.h, dev16(A), [dev16(b) for b in Bs], M, N, K, W, iris.IRIS_MODE_WORKGROUP_SPECIALIZED,
                                      iris.DTYPES[dtype], c_off, flag_off, lock_off, epoch)
        iris.iris_status_check(g.h)
        host = g.to_host().reshape(W, bpr)
        return (host[:, c_off:c_off + M * N * 2].copy(), host[:, flag_off:flag_off + nt * 4].copy())


@pytest.mark.parametrize("W,M,nl,K,dtype", [
    (4, 128, 392, 328, "bf16"),      # single-CTA kernel, 128-wide compute tiles; ragged in N_local and K
    (8, 100, 512, 192, "fp16"),      # single-CTA kernel (one tile row), N_local a multiple of 256
    (4, 520, 392, 328, "bf16"),      # CTA-pair kernel, ragged in M, N_local (256 + 136: a fused unit) and K
    (8, 640, 512, 192, "fp16"),      # CTA-pair kernel, more units than pairs
    (2, 900, 1280, 136, "bf16"),     # CTA-pair kernel, five units per shard, ragged M and K
], ids=["single_bn128_bf16", "single_fp16", "pair_ragged_bf16", "pair_fp16", "pair_bf16_wide"])
def test_noalloc_matches_regular_entry_point_twice_in_a_row(W, M, nl, K, dtype):
    N = W * nl
    c_off, flag_off, _, _, bpr = gemm_layout(M, N, W)
    nt = oracle.num_tiles(M, N, W)
    mem = torch.full((W * bpr,), SENTINEL, dtype=torch.uint8, device="cuda")   # the caller's memory: no heap handle
    bases = [mem.data_ptr() + s * bpr for s in range(W)]
    assert bases[0] % 256 == 0
    for call, (seed, epoch) in enumerate([(61, 1), (62, 2)]):
        A, Bs = inputs.gemm_inputs(seed, W, M, N, K, "uniform", dtype)
        dA, dB = dev16(A), [dev16(b) for b in Bs]
        iris.iris_gemm_all_scatter_noalloc(dA, dB, bases, bpr, M, N, K, W, iris.DTYPES[dtype], c_off, flag_off, epoch)
        host = mem.cpu().numpy().reshape(W, bpr)           # the call has already waited for the stream
        ref_c, ref_flags = _reference_run(W, M, N, K, dtype, A, Bs, epoch)
        assert np.array_equal(host[:, c_off:c_off + M * N * 2], ref_c), f"call {call}: C differs"
        assert np.array_equal(host[:, flag_off:flag_off + nt * 4], ref_flags), f"call {call}: flags differ"
        assert np.all(host[:, flag_off:flag_off + nt * 4].view(np.int32) == epoch)
        # outside C and the flags the caller's memory is untouched (the locks are not in it)
        assert np.all(host[:, :c_off] == SENTINEL) and np.all(host[:, flag_off + nt * 4:] == SENTINEL)
        check_tolerance(host[0, c_off:c_off + M * N * 2].view(np.uint16).reshape(M, N), oracle.gemm_block(A, Bs, dtype), dtype)


def test_noalloc_rejects_problems_beyond_its_static_scratch():
    W, M, N, K = 8, 128 * 129, 128 * 128, 64               # 129 * 128 = 16512 publication tiles > 16384
    with pytest.raises(iris.IrisError) as e:
        iris.iris_gemm_all_scatter_noalloc(256, [256] * W, [4096 * (s + 1) for s in range(W)], 1 << 40, M, N, K, W, iris.IRIS_BF16, 0,
                                           1 << 39, 1)
    assert e.value.code == iris.IRIS_ERR_UNSUPPORTED and "16384" in str(e.value)
