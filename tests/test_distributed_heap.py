"""Host side of the heap over several processes (Section 3.2 initialisation): handle exchange, table of bases,
order of release.  No GPU: the memory operations are fakes that record what was called; the ranks are two gloo
processes."""
import os
import subprocess
import sys
import textwrap

import pytest

from paper_2511_12500_b200 import distributed as D

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _gather_of(entries):
    return lambda obj: list(entries)


def test_own_slot_is_the_local_allocation_and_peers_are_opened_in_rank_order():
    opened = []

    def open_handle(h):
        opened.append(h)
        return 0x7000_0000 + 0x1000 * h[0]

    entries = [(0, bytes([0]) * 64), (1, bytes([1]) * 64), (2, bytes([2]) * 64)]
    bases, mapped = D.exchange_bases(0x1234_0000, entries[1][1], 1, 3, _gather_of(entries), open_handle)
    assert bases == [0x7000_0000, 0x1234_0000, 0x7000_2000]
    assert mapped == [0x7000_0000, 0x7000_2000]
    assert opened == [entries[0][1], entries[2][1]]          # never its own handle


def test_exchange_rejects_a_scrambled_or_short_gather():
    e = [(1, b"b" * 64), (0, b"a" * 64)]
    with pytest.raises(RuntimeError, match="rank order"):
        D.exchange_bases(1, b"a" * 64, 0, 2, _gather_of(e), lambda h: 2)
    with pytest.raises(RuntimeError, match="entries"):
        D.exchange_bases(1, b"a" * 64, 0, 2, _gather_of(e[:1]), lambda h: 2)
    with pytest.raises(ValueError):
        D.exchange_bases(1, b"a" * 64, 2, 2, _gather_of(e), lambda h: 2)


def test_exchange_rejects_two_slots_at_one_address():
    e = [(0, b"a" * 64), (1, b"b" * 64)]
    with pytest.raises(RuntimeError, match="twice"):
        D.exchange_bases(0x5000, b"a" * 64, 0, 2, _gather_of(e), lambda h: 0x5000)


WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    from paper_2511_12500_b200 import distributed as D

    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    log = []

    class FakeOps:
        # addresses encode (owner rank, mapping process): a mapping of rank q's slot in process p is 0x100000*(q+1) + 0x100*(p+1)
        @staticmethod
        def alloc(n):
            log.append(("alloc", n)); return 0x100000 * (rank + 1)
        @staticmethod
        def export(p):
            assert p == 0x100000 * (rank + 1)
            return bytes([rank + 1]) * 64
        @staticmethod
        def open(h):
            q = h[0] - 1
            assert q != rank, "a process must not open its own handle"
            log.append(("open", q)); return 0x100000 * (q + 1) + 0x100 * (rank + 1)
        @staticmethod
        def close(p):
            log.append(("close", p))
        @staticmethod
        def free(p):
            log.append(("free", p))
        @staticmethod
        def heap_create(world_, bpr, bases, local_rank):
            log.append(("heap", world_, bpr, tuple(bases), local_rank)); return 42
        @staticmethod
        def heap_destroy(h):
            log.append(("destroy", h))

    with D.DistributedHeap(4096, ops=FakeOps) as heap:
        assert heap.rank == rank and heap.world == world == 2
        other = 1 - rank
        want = [0, 0]
        want[rank] = 0x100000 * (rank + 1)
        want[other] = 0x100000 * (other + 1) + 0x100 * (rank + 1)
        assert heap.bases == want, (heap.bases, want)
        assert heap.handle == 42
        assert ("heap", 2, 4096, tuple(want), rank) in log
    names = [e[0] for e in log]
    # peers' mappings are closed, and the heap handle destroyed, before the local slot is freed
    assert names == ["alloc", "open", "heap", "destroy", "close", "free"], names
    assert log[-2] == ("close", want[other]) and log[-1] == ("free", want[rank])
    try:
        D.DistributedHeap(100, ops=FakeOps)
    except ValueError:
        pass
    else:
        raise AssertionError("bytes_per_rank = 100 accepted")
    dist.barrier()
    if rank == 0:
        print("EXCHANGE OK")
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_build_matching_tables(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
                          "--master-port", "29671", str(script)], capture_output=True, text=True, timeout=240,
                         env={**os.environ, "OMP_NUM_THREADS": "1"})
    assert out.returncode == 0, out.stderr[-3000:]
    assert "EXCHANGE OK" in out.stdout
