"""The heap over several processes on real device memory: two processes share one GPU, each owns one slot, maps the
other's through an exported handle, computes its own shard of N and scatters it into both slots; every rank's slot
must equal the oracle's image byte for byte (exact-arithmetic inputs), flags and consumer output included.

No kernel of one process waits for a kernel of the other: the only cross-process wait is the consumer's, and it runs
after a host barrier behind which every flag is already set."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import paper_2511_12500_b200 as iris
from gpu_util import GpuHeap

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


def test_two_processes_share_a_heap_through_exported_handles(tmp_path):
    rdv = tmp_path / "rendezvous"
    env = {**os.environ, "OMP_NUM_THREADS": "4"}
    procs = [subprocess.Popen([sys.executable, os.path.join(HERE, "ipc_rank_worker.py"), str(r), "2", str(rdv)], env=env,
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = []
    try:
        for p in procs:
            outs.append(p.communicate(timeout=600)[0])
    finally:
        for p in procs:
            if p.poll() is None:
                p.kill()
    for r, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, f"rank {r}:\n{out[-3000:]}"
        assert f"RANK {r} OK" in out, out[-2000:]


def test_heap_from_bases_in_one_process_matches_the_contiguous_heap():
    """Slots at unrelated addresses (three separate allocations, shuffled): translation, the base table and a put follow the table."""
    W, bpr = 3, 4096
    bufs = [torch.zeros(bpr, dtype=torch.uint8, device="cuda") for _ in range(W)]
    bases = [b.data_ptr() for b in (bufs[2], bufs[0], bufs[1])]
    h = iris.iris_heap_create_from_bases(W, bpr, bases, 1)
    try:
        assert iris.iris_heap_bases(h) == bases and iris.iris_heap_local_rank(h) == 1
        assert iris.iris_translate(h, bases[1] + 100, 1, 0) == bases[0] + 100
        assert iris.iris_translate(h, bases[0] + 4095, 0, 2) == bases[2] + 4095
        with pytest.raises(iris.IrisError) as e:
            iris.iris_translate(h, bases[1] + bpr, 1, 0)
        assert e.value.code == iris.IRIS_ERR_RANGE
        src = torch.arange(256, dtype=torch.uint8, device="cuda")
        iris.iris_store_tile(h, src, bases[1] + 512, 1, 256, 256, 256, 1, 1)         # into the local slot
        iris.iris_put_tile(h, bases[1] + 512, bases[1] + 1024, 1, 256, 256, 256, 1, 2)   # local -> rank 2's slot
        torch.cuda.synchronize()
        assert torch.equal(bufs[1][1024:1280], src)          # rank 2's slot is the third allocation listed, bufs[1]
        assert int(bufs[2].sum()) == 0 and int(bufs[1][:1024].sum()) == 0
        for fn in (lambda: iris.gemm_all_scatter(src, [src] * W, h, 128, 3 * 128, 64, W, 1),):
            with pytest.raises(iris.IrisError) as e:
                fn()
            assert e.value.code == iris.IRIS_ERR_UNSUPPORTED
    finally:
        iris.iris_heap_destroy(h)


def test_heap_from_bases_rejects_bad_tables():
    buf = torch.zeros(3 * 4096, dtype=torch.uint8, device="cuda")
    b = buf.data_ptr()
    for bases, local, bpr in (([b, b + 2048], 0, 4096),        # overlap
                              ([b, b + 4096 + 8], 0, 4096),    # misaligned
                              ([b, 0], 0, 4096),               # missing
                              ([b, 1 << 20], 0, 4096),         # not memory of this process
                              ([b, b + 4096], 2, 4096),        # local rank outside the world
                              ([b, b + 4096], 0, 100)):        # slot size
        with pytest.raises(iris.IrisError) as e:
            iris.iris_heap_create_from_bases(len(bases), bpr, bases, local)
        assert e.value.code == iris.IRIS_ERR_ARG


def test_ipc_alloc_is_zeroed_and_exports_a_handle():
    n = 1 << 20
    p = iris.iris_ipc_alloc(n)
    try:
        hd = iris.iris_ipc_export(p)
        assert len(hd) == iris.IRIS_IPC_HANDLE_BYTES and any(hd)
        h = iris.iris_heap_create_from_bases(1, n, [p], 0)
        try:
            out = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
            iris.iris_load_tile(h, p, out, 1, n, n, n, 0, 0)
            torch.cuda.synchronize()
            assert int(out.max()) == 0
        finally:
            iris.iris_heap_destroy(h)
    finally:
        iris.iris_ipc_free(p)
    with pytest.raises(ValueError):
        iris.iris_ipc_open(b"short")
