"""One rank of the two-process heap test (run by test_gpu_distributed_heap.py, never collected by pytest).

usage: ipc_rank_worker.py RANK WORLD RENDEZVOUS_FILE
Every process uses cuda:0.  A process launches only kernels that wait for nothing another process does: the GEMM +
scatter of its own shard, then -- after a host barrier that follows every rank's device synchronisation -- the
consumer, whose flags are all set by then.  Each rank compares its own slot, byte for byte, with the oracle's.
"""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402
import paper_2511_12500_b200 as iris  # noqa: E402
from paper_2511_12500_b200 import inputs  # noqa: E402
from paper_2511_12500_b200.distributed import DistributedHeap  # noqa: E402
from gpu_util import dev16, first_diff, gemm_layout  # noqa: E402

SEQ, WG, BSP = iris.IRIS_MODE_FUSED_SEQUENTIAL, iris.IRIS_MODE_WORKGROUP_SPECIALIZED, iris.IRIS_MODE_BULK_SYNCHRONOUS
CASES = [
    # mode, dtype, M, N_local, K, extra arguments
    (SEQ, "bf16", 256, 128, 128, {}),                          # single-CTA tiles
    (WG, "fp16", 300, 136, 72, {"wg_tail": -1}),               # ragged everything, every tile through the lock handshake
    (BSP, "bf16", 384, 256, 192, {"cta_pair": -1}),
    (SEQ, "bf16", 520, 448, 136, {}),                          # CTA-pair tiles through per-slot store maps, ragged shard (fused tail)
    (WG, "bf16", 1000, 512, 200, {"wg_tail": -1}),             # CTA-pair tiles, communication CTAs copy to the peer's slot
    (WG, "fp16", 768, 256, 256, {}),                           # default tail rule: producers scatter the last wave themselves
    (BSP, "fp16", 512, 384, 64, {}),
    (WG, "bf16", 640, 256, 192, {"wg_tail": -1, "two_streams": True}),   # the unfused form: communication kernel on a second stream
]


def slot_to_host(heap, bpr):
    out = torch.empty(bpr, dtype=torch.uint8, device="cuda")
    iris.iris_load_tile(heap.handle, heap.bases[heap.rank], out, 1, bpr, bpr, bpr, heap.rank, heap.rank)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def main():
    rank, world, rdv = int(sys.argv[1]), int(sys.argv[2]), sys.argv[3]
    dist.init_process_group("gloo", init_method=f"file://{rdv}", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    for ci, (mode, dtype, M, nl, K, kw) in enumerate(CASES):
        W, N = world, world * nl
        A = inputs.matrix(77 + ci, inputs.STREAM_A, M, K, "ternary:0.5", dtype)
        Bs = [inputs.matrix(77 + ci, inputs.STREAM_B0 + r, nl, K, "smallint:2", dtype) for r in range(W)]
        bias = inputs.matrix(77 + ci, inputs.STREAM_BIAS, 1, N, "smallint:2", dtype).reshape(-1)
        c_off, flag_off, lock_off, out_off, bpr = gemm_layout(M, N, W, with_out=True)
        nt = oracle.num_tiles(M, N, W)
        with DistributedHeap(bpr) as heap:
            assert iris.iris_heap_local_rank(heap.handle) == rank
            assert iris.iris_heap_bases(heap.handle) == heap.bases
            dA, dBias = dev16(A), dev16(bias)
            shards = [None] * W
            shards[rank] = dev16(Bs[rank])                      # a rank holds its own shard of B only
            epoch = 3
            # what the header says such a heap refuses
            for bad in (dict(rank_first=0, rank_count=0), dict(rank_first=(rank + 1) % W, rank_count=1)):
                try:
                    iris.iris_gemm_all_scatter_ex(heap.handle, dA, [shards[rank]] * W, M, N, K, W, mode, iris.DTYPES[dtype], c_off, flag_off, lock_off, epoch, **bad)
                except iris.IrisError as e:
                    assert e.code == iris.IRIS_ERR_ARG, e
                else:
                    raise AssertionError(f"accepted {bad}")
            kw = dict(kw)
            if kw.pop("two_streams", False):
                kw["comm_stream"] = torch.cuda.Stream()
                kw["stream"] = torch.cuda.current_stream()
            iris.iris_gemm_all_scatter_ex(heap.handle, dA, shards, M, N, K, W, mode, iris.DTYPES[dtype], c_off, flag_off, lock_off, epoch,
                                          rank_first=rank, rank_count=1, **kw)
            iris.iris_status_check(heap.handle)                 # synchronises: this rank's tiles and flags are in every slot
            heap.barrier()                                      # ... and so are every other rank's
            iris.iris_consume_bias(heap.handle, c_off, out_off, flag_off, dBias, M, N, W, iris.DTYPES[dtype], epoch)
            iris.iris_status_check(heap.handle)
            got = slot_to_host(heap, bpr)
            img = oracle.HeapImage(W, bpr, fill=0)
            img.gemm_all_scatter(A, Bs, dtype, c_off, flag_off, epoch, lock_off=lock_off if mode == WG else None)
            img.consume_bias(dtype, c_off, out_off, M, N, bias)
            want = img.slot(rank)
            assert np.array_equal(got, want), f"case {ci} rank {rank}: {first_diff(got, want)}"
            assert nt > 0 and (img.view(rank, flag_off, nt * 4, np.int32) == epoch).all()
            torch.cuda.synchronize()
    dist.barrier()
    print(f"RANK {rank} OK {len(CASES)} cases", flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
