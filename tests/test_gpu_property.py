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
from gpu_util import GpuHeap, dev16, first_diff, gemm_layout
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
        # ... and the flag-gated consumer on top of it: OUT = C + bias in every slot, nothing else touched
        bias = inputs.matrix(seed, inputs.STREAM_BIAS, 1, N, "smallint:2", dtype).reshape(-1)
        c_off, flag_off, _, out_off, _ = gemm_layout(M, N, W, True)
        iris.iris_consume_bias(g.h, c_off, out_off, flag_off, dev16(bias), M, N, W, iris.DTYPES[dtype], 2)
        iris.iris_status_check(g.h)
        img.consume_bias(dtype, c_off, out_off, M, N, bias)
        host = g.to_host()
        assert np.array_equal(host, img.mem), (problem, "consumer", first_diff(host, img.mem))


# ------------------------------------------------------------------------------------------------
# Table 3 on random arguments: a sequence of put / get / copy / atomic operations with arbitrary (legal) sizes, pitches,
# alignments and rank triples, applied to the GPU heap and to the oracle's image; the two must agree byte for byte after
# the whole sequence (any misplaced, missing or extra byte shows), and the atomics' returned old values must agree too.
# ------------------------------------------------------------------------------------------------
BPR = 1 << 16


@st.composite
def region_op(draw, W):
    kind = draw(st.sampled_from(["put", "get", "copy"]))
    vec = draw(st.booleans())                       # 16-byte aligned everything (vector path) or arbitrary (byte path)
    unit = 16 if vec else 1
    rows = draw(st.integers(1, 40))
    row_bytes = unit * draw(st.integers(1, 600 // unit if vec else 300))
    sp = row_bytes + unit * draw(st.integers(0, 8))
    dp = row_bytes + unit * draw(st.integers(0, 8))
    span_s, span_d = (rows - 1) * sp + row_bytes, (rows - 1) * dp + row_bytes
    so = unit * draw(st.integers(0, (BPR - span_s) // unit))
    do = unit * draw(st.integers(0, (BPR - span_d) // unit))
    ranks = [draw(st.integers(0, W - 1)) for _ in range(3)]
    return kind, rows, row_bytes, sp, dp, so, do, ranks


@st.composite
def atomic_op(draw, W):
    op = draw(st.sampled_from(["add", "xchg", "and", "or", "xor", "min", "max", "cas", "add64", "cas64"]))
    wide = op.endswith("64")
    word = 8 if wide else 4
    count = draw(st.integers(1, 300))
    stride = word * draw(st.integers(1, 5))
    off = word * draw(st.integers(0, (BPR - ((count - 1) * stride + word)) // word))
    frm, to = draw(st.integers(0, W - 1)), draw(st.integers(0, W - 1))
    val = draw(st.integers(0, (1 << 64) - 1) if wide else st.integers(-(1 << 31), (1 << 31) - 1))
    cmp_ = draw(st.integers(0, 3))
    return op, count, stride, off, frm, to, val, cmp_


@st.composite
def op_sequences(draw):
    W = draw(st.integers(1, 5))
    n = draw(st.integers(1, 8))
    ops = [draw(st.one_of(region_op(W), atomic_op(W))) for _ in range(n)]
    return W, ops, draw(st.integers(0, 1 << 20))


@settings(max_examples=int(os.environ.get("IRIS_PROPERTY_EXAMPLES", "150")), deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))
@given(op_sequences())
def test_any_sequence_of_tile_operations_and_atomics_matches_the_oracle(case):
    import torch
    W, ops, seed = case
    with GpuHeap(W, BPR) as g:
        img = g.image()
        img.mem[:] = inputs.payload_bytes(seed, 7, img.mem.size)
        # a sprinkling of small values so that cas (compare with 0..3) and min/max take both branches
        img.mem[::97] = 0
        g.mem.copy_(torch.from_numpy(img.mem).cuda())
        for op in ops:
            if op[0] in ("put", "get", "copy"):
                kind, rows, rb, sp, dp, so, do, (a, b, c) = op
                overlap = so < do + (rows - 1) * dp + rb and do < so + (rows - 1) * sp + rb
                # source and destination overlapping in one slot: the order of the bytes is unspecified
                if overlap and ((kind in ("put", "get") and a == b) or (kind == "copy" and b == c)):
                    continue
                if kind == "put":
                    iris.iris_put_tile(g.h, g.addr(a, so), g.addr(a, do), rows, rb, sp, dp, a, b)
                    img.put(so, do, rows, rb, sp, dp, a, b)
                elif kind == "get":
                    iris.iris_get_tile(g.h, g.addr(a, so), g.addr(a, do), rows, rb, sp, dp, a, b)
                    img.get(so, do, rows, rb, sp, dp, a, b)
                else:
                    iris.iris_copy_tile(g.h, g.addr(a, so), g.addr(a, do), rows, rb, sp, dp, a, b, c)
                    img.copy(so, do, rows, rb, sp, dp, b, c)
                continue
            name, count, stride, off, frm, to, val, cmp_ = op
            wide = name.endswith("64")
            old = torch.empty(count, dtype=torch.int64 if wide else torch.int32, device="cuda")
            ptr = g.addr(frm, off)
            if name == "add64":
                iris.iris_atomic_add_u64(g.h, ptr, count, stride, frm, to, val, old_out=old)
                exp = img.atomic_add_u64(off, count, stride, to, val)
            elif name == "cas64":
                iris.iris_atomic_cas_u64(g.h, ptr, count, stride, frm, to, cmp_, val, old_out=old)
                exp = img.atomic_cas_u64(off, count, stride, to, cmp_, val)
            elif name == "cas":
                iris.iris_atomic_cas(g.h, ptr, count, stride, frm, to, cmp_, val, old_out=old)
                exp = img.atomic_cas(off, count, stride, to, cmp_, val)
            else:
                iris.iris_atomic_rmw(g.h, iris.ATOMIC_OPS[name], ptr, count, stride, frm, to, val, old_out=old)
                exp = img.atomic_rmw(name, off, count, stride, to, val)
            got = old.cpu().numpy()
            assert np.array_equal(got.view(exp.dtype), exp), (op, "returned old values differ")
        assert np.array_equal(g.to_host(), img.mem), (case, first_diff(g.to_host(), img.mem))
