"""Property test: for ANY legal small shape and any combination of the tuning knobs, gemm_all_scatter leaves exactly the
oracle's heap image (exact-arithmetic inputs, so the comparison is byte for byte: values, placement, replication, flags,
locks, and every byte outside the regions untouched).

The examples are drawn by hypothesis from a fixed seed (derandomize), so a run is reproducible; the domain covers what the
hand-picked shapes of the other files cannot enumerate: odd worlds, shards narrower than a tile, ragged everything, each
knob against each kernel.  Arguments the header declares illegal are not drawn."""
import os

import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import inputs
from gpu_util import GpuHeap, first_diff, gemm_layout
from test_gpu_gemm_all_scatter import expected_image, run_gemm

pytestmark = pytest.mark.gpu

MODES = [iris.IRIS_MODE_BULK_SYNCHRONOUS, iris.IRIS_MODE_FUSED_SEQUENTIAL, iris.IRIS_MODE_WORKGROUP_SPECIALIZED]


@st.composite
def problems(draw):
    W = draw(st.integers(1, 8))
    nl = 8 * draw(st.integers(1, 80))            # N/world: a multiple of 8, up to 640 (2.5 pair tiles)
    if W * nl > 2560:
        nl = max(8, (2560 // W) // 8 * 8)
    M = draw(st.one_of(st.integers(1, 130), st.integers(131, 700)))
    K = 8 * draw(st.one_of(st.integers(1, 9), st.integers(10, 60)))
    mode = draw(st.sampled_from(MODES))
    dtype = draw(st.sampled_from(["bf16", "fp16"]))
    kw = {}
    if draw(st.booleans()):
        kw["cta_pair"] = -1
    bn = draw(st.sampled_from([0, 0, 128, 256]))
    if bn:
        kw["block_n"] = bn
    if draw(st.booleans()):
        kw["static_schedule"] = 1
    kw["raster_group"] = draw(st.sampled_from([0, 1, 3]))
    mc = draw(st.sampled_from([0, 0, 12, 24]))
    if mc:
        kw["max_ctas"] = mc
    if mode == iris.IRIS_MODE_WORKGROUP_SPECIALIZED:
        kw["wg_tail"] = draw(st.sampled_from([-1, 0, 3]))
        kw["comm_ctas"] = draw(st.sampled_from([0, 2, 4]))
    kw["fuse_tail"] = draw(st.sampled_from([-1, 0, 1]))
    kw["stage_k"] = draw(st.sampled_from([0, 64, 128]))
    kw["b_layout"] = draw(st.sampled_from([0, 0, 1]))
    if draw(st.booleans()):
        kw["pace_stores"] = -1
    seed = draw(st.integers(0, 1 << 20))
    return W, M, nl, K, mode, dtype, kw, seed


# 200 examples take about 20 s; IRIS_PROPERTY_EXAMPLES=N widens the search
@settings(max_examples=int(os.environ.get("IRIS_PROPERTY_EXAMPLES", "200")), deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))
@given(problems())
def test_any_small_problem_leaves_the_oracles_heap_image(problem):
    W, M, nl, K, mode, dtype, kw, seed = problem
    N = W * nl
    A = inputs.matrix(seed, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
    Bs = [inputs.matrix(seed, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
    bpr = gemm_layout(M, N, W, True)[4]
    with GpuHeap(W, bpr) as g:
        c_full = None
        for epoch in (1, 2):          # a second call over the first one's data, flags and (reset) locks
            run_gemm(g, A, Bs, dtype, mode, epoch=epoch, with_locks_zeroed=(epoch == 1), **dict(kw))
            host = g.to_host()
            img, c_full = expected_image(g, A, Bs, dtype, mode, epoch=epoch, c_full=c_full)
            assert np.array_equal(host, img.mem), (problem, epoch, first_diff(host, img.mem))
