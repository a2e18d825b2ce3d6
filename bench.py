#!/usr/bin/env python
"""Benchmark of the GEMM + all-scatter hot path on B200 (one JSON line on stdout).

A step = one pass of the whole path on one batch of synthetic input:
    gemm_all_scatter (workgroup_specialized)  ->  flag-gated consumer (OUT = C + bias)
on the workload the target is quoted on: W=8 emulated ranks, M=8192, N=K=16384, bf16 uniform[-1,1).

  python bench.py [--gpus N] [--steps K] [--warmup W]            # the CUDA path
  python bench.py --impl reference [--steps K] [--warmup W]      # the CPU oracle on a bounded sample

`value` is TFLOP/s of the step (2*M*N*K flops per step) with inputs resident in HBM; `e2e` is the same
metric through the host-buffer entry point (H2D of A, B, bias and D2H of C, OUT, flags inside the timed
region); `roofline` describes the dominant kernel (the GEMM + scatter kernel) against the measured
tensor peak; `cpu_baseline` is the oracle timed on this machine's host cores on a sample of the same workload.
With --gpus N > 1 every rank runs an independent replica (the path is emulated inside one GPU and has no
cross-GPU exchange step); the value is the sum over ranks, timed as the max over ranks.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

WORKLOADS = {
    # name: (W, M, N, K, dist, dtype)
    "cfg5_w8_m8192_n16384_k16384": (8, 8192, 16384, 16384, "uniform", "bf16"),
    "cfg5_w8_m1024_n16384_k16384": (8, 1024, 16384, 16384, "uniform", "bf16"),
    "cfg5_w8_m2048_n16384_k16384": (8, 2048, 16384, 16384, "uniform", "bf16"),   # a quarter of the headline's rows: the size ncu's full set is taken on
    "cfg5_w4_m8192_n16384_k16384": (4, 8192, 16384, 16384, "uniform", "bf16"),
    "cfg5_w4_m1024_n16384_k16384": (4, 1024, 16384, 16384, "uniform", "bf16"),
    "cfg5_w2_m8192_n16384_k16384": (2, 8192, 16384, 16384, "uniform", "bf16"),
    "cfg5_w2_m1024_n16384_k16384": (2, 1024, 16384, 16384, "uniform", "bf16"),
    "cfg3_w8_m4096_n8192_k8192": (8, 4096, 8192, 8192, "normal002", "bf16"),
    "cfg4_w8_m128_n28672_k8192": (8, 128, 28672, 8192, "normal002", "bf16"),
    "cfg1_w2_256": (2, 256, 256, 256, "uniform", "fp16"),
    # the two shapes the paper names in Section 5.2 (M x N x K = 8192 x 4608 x 36864 and 8192 x 3584 x 14336, 8 ranks);
    # the text does not say whether N is per rank or global, so both readings are available
    "paper_8192x4608x36864_w8_n_per_rank": (8, 8192, 8 * 4608, 36864, "normal002", "bf16"),
    "paper_8192x3584x14336_w8_n_per_rank": (8, 8192, 8 * 3584, 14336, "normal002", "bf16"),
    "paper_8192x4608x36864_w8_n_global": (8, 8192, 4608, 36864, "normal002", "bf16"),
    "paper_8192x3584x14336_w8_n_global": (8, 8192, 3584, 14336, "normal002", "bf16"),
}
DEFAULT_WORKLOAD = "cfg5_w8_m8192_n16384_k16384"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
METRIC = "gemm_all_scatter_tflops"
UNIT = "TFLOP/s"
# DRAM traffic of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum per launch) is not typed in here: it is
# read from the ncu summary under profiles/ that records it together with a digest of the kernel sources it was taken on.
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "gemm_all_scatter_dram_traffic.md")
KERNEL_SOURCES = ["gemm_all_scatter.cu", "sm100_ptx.cuh", "iris_device.cuh", "iris_internal.h"]


def kernel_sources_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2511_12500_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, mode: str):
    """(bytes per launch or None, note) from the tracked ncu record; None when there is no record for this workload and
    schedule or when the kernel sources have changed since it was captured."""
    try:
        text = open(TRAFFIC_RECORD).read()
    except OSError:
        return None, "no ncu record under profiles/"
    for block in text.split("\n## ")[1:]:
        kv = {}
        for line in block.splitlines():
            if ":" in line and line.startswith("- "):
                k, v = line[2:].split(":", 1)
                kv[k.strip()] = v.strip()
        if kv.get("workload") == workload and kv.get("mode") == mode:
            if kv.get("kernel_sources_sha256") != kernel_sources_digest():
                return None, f"ncu record is for older kernel sources (commit {kv.get('commit', '?')}); not carried over"
            return float(kv["dram_bytes_read"]) + float(kv["dram_bytes_write"]), f"ncu 1-pass capture at commit {kv.get('commit', '?')}"
    return None, "no ncu record for this workload and schedule"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def align(x, a=256):
    return (x + a - 1) // a * a


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 20 ms.  The sampler is started before the warm-up (nvidia-smi
    needs 100-200 ms to deliver its first line); only the lines stamped inside the timed region [mark(), stop()] count."""

    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,power.limit,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path, self.t0 = index, None, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark(self):
        self.t0 = datetime.datetime.now()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        t1 = datetime.datetime.now()
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons, lim = [], [], [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                stamp = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                if self.t0 is not None and not (self.t0 <= stamp <= t1):
                    continue
                vals = (float(f[1]), float(f[2]), float(f[3]), float(f[4]))
            except ValueError:
                continue
            sm.append(vals[0]); mx.append(vals[1]); pw.append(vals[2]); lim = vals[3]
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), power_w_max=float(max(pw)), reasons=sorted(reasons),
                       samples=len(sm), power_limit_w=lim)
        return out


def sample_strips(M: int, W: int, count: int, seed: int = 1):
    """Seeded sample of (tile row, rank) strips: 128 rows x one rank's whole column shard."""
    rng = np.random.default_rng(seed)
    tiles_m = -(-M // 128)
    total = tiles_m * W
    picks = rng.choice(total, size=min(count, total), replace=False)
    return [(int(p) // W, int(p) % W) for p in picks]


def oracle_strip_sample(workload, seed, strips, threads=None):
    """Oracle (as it stands: fp64 accumulation, one rounding) on the given strips: (seconds, flops, cores).
    Only the oracle call is timed; drawing the strip's input rows is not."""
    import oracle
    from paper_2511_12500_b200 import inputs
    W, M, N, K, dist, dtype = workload
    nl = N // W
    secs, flops = 0.0, 0.0
    cores = threads or oracle.hw_threads()
    for tm, r in strips:
        m0, m1 = tm * 128, min(M, tm * 128 + 128)
        A = inputs.matrix(seed, inputs.STREAM_A, M, K, dist, dtype, m0, m1)
        B = inputs.matrix(seed, inputs.STREAM_B0 + r, nl, K, dist, dtype)
        t0 = time.perf_counter()
        oracle.gemm_block(A, [B], dtype, threads=cores)
        secs += time.perf_counter() - t0
        flops += 2.0 * (m1 - m0) * nl * K
    return secs, flops, cores


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    workload = WORKLOADS[args.workload]
    W, M, N, K, dist, dtype = workload
    seed = 251112500 + 4
    strips = sample_strips(M, W, args.steps + args.warmup, seed=7)
    while len(strips) < args.steps + args.warmup:
        strips += strips
    for i in range(args.warmup):
        oracle_strip_sample(workload, seed, strips[i:i + 1])
    secs, flops, cores = 0.0, 0.0, 0
    for i in range(args.warmup, args.warmup + args.steps):
        s, f, cores = oracle_strip_sample(workload, seed, strips[i:i + 1])
        secs += s
        flops += f
    value = flops / secs / 1e12
    sample = f"one strip (128 rows x one rank's {N // W}-column shard, K={K}) of {args.workload} per step, fp64 accumulation"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "world": W, "M": M, "N": N, "K": K, "mode": "oracle", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def gpu_gate(torch):
    """Keep the GPU busy for ~0.2 ms before a single launch is timed between two synchronisations.

    A start event recorded on an idle GPU is stamped at once, so everything the host still does before the kernel is
    queued (argument marshalling, plan lookup, the launch call itself: 20-25 us, for the library GEMM as for this
    path) would be counted as kernel time -- a fifth of a 0.1 ms kernel.  With the GPU busy the host runs ahead and the
    interval between the two events is device time only."""
    torch.cuda._sleep(400_000)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar over the process group (the job's time is its slowest rank's)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world_size: int, flops_per_rank_step: float, ms_per_step_max: float) -> float:
    """Whole-job TFLOP/s of `world_size` replicas, each doing flops_per_rank_step per step, timed by the slowest."""
    return world_size * flops_per_rank_step / (ms_per_step_max * 1e-3) / 1e12


def run_ours(args):
    import torch
    import paper_2511_12500_b200 as iris
    from paper_2511_12500_b200 import inputs

    world_size = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist_on = world_size > 1
    if dist_on:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    pk, pk_kind = peaks()

    workload = WORKLOADS[args.workload]
    W, M, N, K, dist_name, dtype = workload
    seed = 251112500 + 4 + rank                     # independent batch per replica
    nl = N // W
    nt = iris.iris_num_tiles(M, N, W)
    flag_off = align(M * N * 2)
    lock_off = flag_off + align(nt * 4)
    out_off = iris.iris_gemm_out_offset(M, N, W)
    bpr = align(out_off + M * N * 2)
    mode = iris.MODES[args.mode]
    dt = iris.DTYPES[dtype]

    A, Bs = inputs.gemm_inputs(seed, W, M, N, K, dist_name, dtype)
    bias = inputs.vector(seed, inputs.STREAM_BIAS, N, "uniform", dtype)
    sampler = ClockSampler(local_rank)
    sampler.start()           # long before the timed region: see the class
    dA = torch.from_numpy(A.view(np.int16)).cuda()
    dB = [torch.from_numpy(b.view(np.int16)).cuda() for b in Bs]
    dbias = torch.from_numpy(bias.view(np.int16)).cuda()
    heap_mem = torch.zeros(W * bpr, dtype=torch.uint8, device="cuda")
    h = iris.iris_heap_create(W, bpr, external_base=heap_mem.data_ptr())
    stream = torch.cuda.current_stream()
    flops = 2.0 * M * N * K
    store_bytes = float(W) * M * N * 2

    def gemm(epoch, m=mode, fused=False, wg_tail=None, **kw):
        kw.setdefault("stream", None)
        kw.setdefault("fuse_tail", args.fuse_tail)
        kw.setdefault("stage_k", args.stage_k)
        iris.iris_gemm_all_scatter_ex(h, dA, dB, M, N, K, W, m, dt, 0, flag_off, lock_off, epoch, comm_ctas=args.comm_ctas,
                                      raster_group=args.raster_group, block_n=args.block_n, cta_pair=args.cta_pair, static_schedule=args.static_schedule, stream_k=args.stream_k,
                                      wg_tail=args.wg_tail if wg_tail is None else wg_tail,
                                      consumer_bias=dbias if fused else None, consumer_out_off=out_off, **kw)

    def consume(epoch):
        iris.iris_consume_bias(h, 0, out_off, flag_off, dbias, M, N, W, dt, epoch)

    def barrier():
        torch.cuda.synchronize()
        if dist_on:
            dist.barrier()
            torch.cuda.synchronize()

    fused = bool(args.fused_consumer)

    def step(epoch, events=None):
        """One pass of the path: GEMM + all-scatter + flag publication + flag-gated consumer."""
        if events:
            events[0].record(stream)
        if fused:
            gemm(epoch, fused=True)          # the consumer's warps acquire the flags inside the same launch
            if events:
                events[1].record(stream)
        else:
            gemm(epoch)
            if events:
                events[1].record(stream)
            consume(epoch)
        if events:
            events[2].record(stream)

    epoch = 0
    for _ in range(args.warmup):
        epoch += 1
        step(epoch)
    iris.iris_status_check(h)

    # ---------------- timed region: exactly K steps ----------------
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    sampler.mark()
    gpu_gate(torch)
    for i in range(args.steps):
        epoch += 1
        step(epoch, ev[i])
    barrier()
    clocks = sampler.stop()
    iris.iris_status_check(h)
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    gemm_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    cons_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    total_ms = max_over_ranks(total_ms, device="cuda")
    ms_per_step = total_ms / args.steps
    value = job_value(world_size, flops, ms_per_step)

    result = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world_size, "steps": args.steps, "warmup": args.warmup,
              "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if dtype == "bf16" else "f16",
              "data": "synthetic",
              "config": {"workload": args.workload, "world": W, "M": M, "N": N, "K": K, "mode": args.mode, "comm_ctas": args.comm_ctas or "auto",
                         "step": "gemm_all_scatter + flag-gated consumer (OUT = C + bias)" + (", consumer warps inside the GEMM launch" if fused else ", consumer as a second kernel"), "accumulate": "fp32",
                         "l2": "inputs (0.8 GB) and outputs (4.3 GB) far exceed the 126 MB L2; no explicit flush",
                         "multi_gpu": "replicas only (ranks are emulated inside one GPU)"},
              "clocks": clocks, "gpu_launches": (1 if fused else 2) * args.steps}

    if rank == 0:
        # ---------------- roofline of the dominant kernel ----------------
        t_tensor = flops / (pk["bf16_tflops"] * 1e12) * 1e3
        t_store = store_bytes / (pk["hbm_gbs"] * 1e9) * 1e3
        t_bytes = ((M * K + N * K) * 2.0 + store_bytes) / (pk["hbm_gbs"] * 1e9) * 1e3   # operand reads + replicated stores
        achieved = flops / (gemm_ms * 1e-3) / 1e12
        traffic, traffic_note = recorded_traffic(args.workload, args.mode)
        result["roofline"] = {"kernel": f"gemm_all_scatter_pair_kernel<bf16> ({args.mode}); single-CTA kernel when --cta-pair -1 or the shape needs it", "bound": "tensor", "achieved": achieved,
                              "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / pk["bf16_tflops"],
                              "peak_kind": f"{pk_kind} burst (of {pk_kind})", "peak_sustained": pk["bf16_tflops_sustained"],
                              "traffic": traffic, "traffic_note": traffic_note,
                              "algorithmic_bytes": (M * K + N * K) * 2.0 + store_bytes,
                              "kernel_ms": gemm_ms, "combined_roofline_ms": max(t_tensor, t_store),
                              "frac_of_combined_roofline": max(t_tensor, t_store) / gemm_ms,
                              "full_traffic_roofline_ms": max(t_tensor, t_bytes), "frac_of_full_traffic_roofline": max(t_tensor, t_bytes) / gemm_ms,
                              "replicated_store_gbs": store_bytes / (gemm_ms * 1e-3) / 1e9}
        # ---------------- the same kernel in steady state: >= 1 s of back-to-back launches under the power cap ----------------
        # (the timed region above may last well under 100 ms, during which the clocks are still on their way down)
        if args.steady_seconds > 0:
            n_steady = max(10, int(np.ceil(args.steady_seconds * 1e3 / max(gemm_ms, 1e-3))))
            s2 = ClockSampler(local_rank)
            s2.start()
            for _ in range(3):
                epoch += 1
                gemm(epoch)
            time.sleep(0.3)               # nvidia-smi needs a moment before its first line
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            s2.mark()
            e0.record(stream)
            for _ in range(n_steady):
                epoch += 1
                gemm(epoch)
            e1.record(stream)
            torch.cuda.synchronize()
            ck = s2.stop()
            iris.iris_status_check(h)
            sms = e0.elapsed_time(e1) / n_steady
            st_ach = flops / (sms * 1e-3) / 1e12
            result["roofline"]["steady"] = {"launches": n_steady, "seconds": sms * n_steady * 1e-3, "kernel_ms": sms, "achieved": st_ach,
                                            "frac": st_ach / pk["bf16_tflops"], "frac_vs_sustained": st_ach / pk["bf16_tflops_sustained"],
                                            "sm_mhz": ck.get("sm_mhz"), "clock_samples": ck.get("samples"), "reasons": ck.get("reasons"),
                                            "power_w_max": ck.get("power_w_max"),
                                            "ms_times_mhz": (sms * ck["sm_mhz"]) if ck.get("sm_mhz") else None,
                                            "note": "back-to-back launches of the dominant kernel alone; frac against the burst peak, frac_vs_sustained "
                                                    "against the peak measured the same way (a seconds-long loop)"}
        cons_bytes = 2.0 * store_bytes + N * 2
        if fused:   # time the stand-alone consumer kernel too, for its own HBM figure
            ts = []
            for _ in range(4):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                gpu_gate(torch)
                e0.record(stream)
                consume(epoch)
                e1.record(stream)
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            cons_ms = float(np.median(ts[1:]))
        result["consumer"] = {"kernel_ms": cons_ms, "gbs": cons_bytes / (cons_ms * 1e-3) / 1e9,
                              "frac_of_hbm_peak": cons_bytes / (cons_ms * 1e-3) / 1e9 / pk["hbm_gbs"], "bytes": cons_bytes,
                              "note": "stand-alone consumer kernel after the producer" + ("; in the timed step the consumer runs inside the GEMM launch" if fused else "")}

        # ---------------- the three schedules on the same workload (context for the headline) ----------------
        modes = {}
        # Round-robin over the variants, one launch each per round, so that clock drift under the power cap (launch times
        # grow by 10-30 % over the first few hundred ms of continuous load) hits all of them alike.
        variants = list(iris.MODES.items()) + [("workgroup_specialized_every_tile_via_comm_ctas", iris.IRIS_MODE_WORKGROUP_SPECIALIZED)]
        tA = dA.view(torch.bfloat16 if dtype == "bf16" else torch.float16).view(M, K)
        tB = torch.cat([b.view(tA.dtype).view(nl, K) for b in dB], dim=0)
        variants.append(("unfused_two_streams", "unfused"))   # Section 4.1: producers and communication kernel as two launches
        variants.append(("library_gemm_no_scatter", None))   # context: cuBLAS through torch.matmul, same operands, same moment
        comm_stream = torch.cuda.Stream()
        series = {name: [] for name, _ in variants}
        for it in range(1 + args.mode_iters if args.mode_iters > 0 else 0):
            for name, m in variants:
                epoch += 1
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                gpu_gate(torch)
                e0.record(stream)
                if m is None:
                    tC = tA @ tB.t()
                elif m == "unfused":
                    gemm(epoch, iris.IRIS_MODE_WORKGROUP_SPECIALIZED, stream=stream, comm_stream=comm_stream)   # `stream` joins the second one
                else:
                    gemm(epoch, m, wg_tail=-1 if name.endswith("comm_ctas") else None)
                e1.record(stream)
                torch.cuda.synchronize()
                if it > 0:
                    series[name].append(e0.elapsed_time(e1))
        kept = {}
        for name, m in (variants if args.mode_iters > 0 else ()):
            if m == iris.IRIS_MODE_WORKGROUP_SPECIALIZED and not name.endswith("comm_ctas"):
                epoch += 1
                gemm(epoch, m)
                kept[name] = iris.iris_gemm_takeover_stats(h)[0]
        for name, ts in series.items():
            if not ts:
                continue
            ms = float(np.median(ts))
            modes[name] = {"ms": ms, "ms_min": float(min(ts)), "tflops": flops / ms / 1e9, "store_gbs": store_bytes / ms / 1e6,
                           "frac_of_combined_roofline": max(t_tensor, t_store) / ms}
            if name in kept:
                modes[name]["half_tiles_kept_by_producers_before_the_last_wave"] = kept[name]
        iris.iris_status_check(h)
        result["modes"] = modes

        # ---------------- consumer launched on a second stream right after the producer (it overlaps the GEMM) ----------------
        # End-to-end time from the producer's launch to the end of the last kernel, next to the same two kernels on one stream.
        # (not in bulk_synchronous mode: there the flags come from the second kernel of the call, after the GEMM has ended, so
        # nothing of the consumer can overlap the GEMM -- and a consumer grid that fills every SM's thread slots while it
        # waits would keep that second kernel from ever starting; the consumer's deadline, not a hang, is what ends that)
        if args.mode_iters > 0 and args.mode != "bulk_synchronous":
            cons_stream = torch.cuda.Stream()
            sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
            joined = torch.cuda.Event()
            ts2, ts1 = [], []
            for it in range(1 + args.mode_iters):
                for overlapped in (True, False):
                    epoch += 1
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    torch.cuda.synchronize()
                    # (no busy kernel in front here: two streams released by one event start in no fixed order, and a consumer
                    # that becomes resident first keeps the GEMM's CTAs off the SMs; 20 us of host time in 4 ms do not matter)
                    e0.record(stream)
                    gemm(epoch)
                    if overlapped:
                        # launched after the producer, whose CTAs are all resident by then; beside a GEMM CTA of the pair kernel
                        # one consumer CTA fits per SM (shared memory), the rest of the grid follows as the GEMM's CTAs leave
                        iris.iris_consume_bias(h, 0, out_off, flag_off, dbias, M, N, W, dt, epoch, ctas=4 * sm_count, stream=cons_stream)
                        joined.record(cons_stream)
                        stream.wait_event(joined)
                    else:
                        consume(epoch)
                    e1.record(stream)
                    torch.cuda.synchronize()
                    if it > 0:
                        (ts2 if overlapped else ts1).append(e0.elapsed_time(e1))
            iris.iris_status_check(h)
            result["consumer_on_second_stream"] = {"ms": float(np.median(ts2)), "ms_min": float(min(ts2)), "tflops": flops / float(np.median(ts2)) / 1e9,
                                                   "same_two_kernels_on_one_stream_ms": float(np.median(ts1)),
                                                   "note": "producer kernel on one stream, iris_consume_bias on a second stream right after it; first launch to last kernel done"}

        # ---------------- the same step with the consumer's warps inside the GEMM launch ----------------
        if not fused and args.mode != "bulk_synchronous":
            for _ in range(2):
                epoch += 1
                gemm(epoch, fused=True)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(args.steps):
                epoch += 1
                gemm(epoch, fused=True)
            e1.record(stream)
            torch.cuda.synchronize()
            iris.iris_status_check(h)
            fms = e0.elapsed_time(e1) / args.steps
            result["fused_consumer_step"] = {"ms_per_step": fms, "value": flops / fms / 1e9, "unit": UNIT, "gpu_launches_per_step": 1,
                                             "note": "consumer warps acquire each tile's flag inside the GEMM launch (consumer_bias set); same outputs"}

        # ---------------- context only: the library GEMM (cuBLAS via torch.matmul) on the same operands ----------------
        # Not part of the path and not a target: it shows what the same data, clocks and power cap give a plain
        # GEMM without any scatter, next to the burst / sustained peaks measured on other data.
        try:
            for _ in range(3):
                tC = tA @ tB.t()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(args.steps):
                tC = tA @ tB.t()
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            result["context"] = {"torch_matmul_same_operands": {"ms": ms, "tflops": flops / ms / 1e9, "note": "library GEMM only, no scatter, no flags"}}
            del tB, tC
        except Exception as exc:  # pragma: no cover
            result["context"] = {"error": str(exc)}

        # ---------------- end to end through the host-buffer entry point ----------------
        try:
            if args.e2e_steps <= 0:
                raise RuntimeError("skipped (--e2e-steps 0)")
            pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()  # noqa: E731
            hA, hB, hbias = pin(A), [pin(b) for b in Bs], pin(bias)
            hC = torch.empty(M * N, dtype=torch.int16).pin_memory()
            hOUT = torch.empty(M * N, dtype=torch.int16).pin_memory()
            hflags = torch.empty(W * nt, dtype=torch.int32).pin_memory()
            iris.iris_flags_fill(h, flag_off, nt, 0)
            torch.cuda.synchronize()
            e2e_t = []
            for i in range(1 + args.e2e_steps):
                t0 = time.perf_counter()
                iris.iris_gemm_all_scatter_host(hA, hB, hC, hflags, hbias, hOUT, h, M, N, K, W, mode, dt, 0)
                e2e_t.append(time.perf_counter() - t0)
            e2e_s = float(np.mean(e2e_t[1:]))
            h2d = (M * K + N * K + N) * 2
            d2h = 2 * M * N * 2 + W * nt * 4
            result["e2e"] = {"value": flops / e2e_s / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                             "ms_per_step": e2e_s * 1e3, "api": "iris_gemm_all_scatter_host (pinned host buffers; one block per rank shard, pipelined over copy-in, compute and copy-out streams)"}
            del hA, hB, hC, hOUT
        except Exception as exc:  # pragma: no cover
            result["e2e"] = {"value": None, "unit": UNIT, "error": str(exc)}

        # ---------------- all-store microbenchmark (replicated-store GB/s vs HBM peak) ----------------
        if args.sweep != "none":
            result["all_store"] = all_store_sweep(iris, pk, args.sweep, pull=0)
            result["all_load"] = all_store_sweep(iris, pk, args.sweep, pull=1)
            result["p2p"] = p2p_microbench(iris, pk)

        # ---------------- CPU oracle on a bounded sample of the same workload ----------------
        if not args.no_cpu_baseline:
            strips = sample_strips(M, W, args.cpu_strips, seed=3)
            secs, fl, cores = oracle_strip_sample(workload, seed, strips)
            result["cpu_baseline"] = {"value": fl / secs / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": secs,
                                      "sample": f"{len(strips)} strips (128 rows x one rank's {nl}-column shard, K={K}) of {args.workload}, "
                                                f"{fl / flops:.4f} of one step's flops, fp64 accumulation",
                                      "extrapolated_full_step_seconds": flops / (fl / secs)}
            if args.sweep != "none":
                result["cpu_baseline"]["all_store"] = oracle_all_store_sample()
        print(json.dumps(result))
    iris.iris_heap_destroy(h)
    if dist_on:
        dist.barrier()
        dist.destroy_process_group()


def oracle_all_store_sample(S=4 << 20, W=8):
    """The oracle's all-store (its copy loops and flag updates on a host image of the heap) at one message size of
    the sweep, timed as it stands; GB/s counted like the GPU sweep (W*S read + W*W*S written)."""
    import oracle
    tile = 32768
    T = S // tile
    payload_off, recv_off = 0, align(S)
    flag_off = recv_off + align(W * S)
    bpr = align(flag_off + W * T * 4)
    img = oracle.HeapImage(W, bpr, fill=0)
    for r in range(W):
        img.view(r, payload_off, S)[:] = (r + 1)
    img.all_store(payload_off, recv_off, flag_off, S, tile, 1)          # first touch of the image
    t0 = time.perf_counter()
    img.all_store(payload_off, recv_off, flag_off, S, tile, 2)
    secs = time.perf_counter() - t0
    moved = float(W * S + W * W * S)
    return {"S": S, "seconds": secs, "gbs": moved / secs / 1e9, "kind": "oracle"}


def all_store_sweep(iris, pk, kind, pull=0):
    """W=8 all-store (push) or all-load (pull): message sizes 1 KiB .. (64 MiB | 1 GiB) in powers of 4.
    GB/s counts the HBM-side bytes, W*S read + W*W*S written, in both forms; the pull form also reports the bytes its
    loads request (W*W*S read + W*W*S written) as the L2-side rate."""
    import torch
    W = 8
    top = 15 if kind == "full" else 13
    out = []
    for e in range(5, top + 1):
        S = 4 ** e
        tile = min(S, 32768)
        T = -(-S // tile)
        payload_off, recv_off = 0, align(S)
        flag_off = recv_off + align(W * S)
        bpr = align(flag_off + W * T * 4)
        free, _ = torch.cuda.mem_get_info()
        if W * bpr + (2 << 30) > free:
            out.append({"S": S, "skipped": "insufficient free HBM"})
            continue
        mem = torch.empty(W * bpr, dtype=torch.uint8, device="cuda")
        mem[: 1 << 20].zero_()
        h = iris.iris_heap_create(W, bpr, external_base=mem.data_ptr())
        iris.iris_flags_fill(h, flag_off, W * T, 0)
        stream = torch.cuda.current_stream()
        iters = 20 if S <= (1 << 24) else 5
        iris.iris_all_store_bench(h, payload_off, recv_off, flag_off, S, tile, 1, 0, pull)
        iris.iris_all_store_bench(h, payload_off, recv_off, flag_off, S, tile, 2, 0, pull)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        gpu_gate(torch)
        e0.record(stream)
        for i in range(iters):
            iris.iris_all_store_bench(h, payload_off, recv_off, flag_off, S, tile, 3 + i, 0, pull)
        e1.record(stream)
        torch.cuda.synchronize()
        iris.iris_status_check(h)
        ms = e0.elapsed_time(e1) / iters
        # HBM-side bytes: every source block is fetched from DRAM once (W*S) however many ranks read it; W*W*S are written.
        # The pull form issues W*W*S of reads, of which all but W*S are served by L2: reported separately as l2_side_gbs.
        hbm_bytes = float(W * S + W * W * S)
        row = {"S": S, "ms": ms, "gbs": hbm_bytes / ms / 1e6, "frac_of_hbm_peak": hbm_bytes / ms / 1e6 / pk["hbm_gbs"],
               "l2": "warm (working set below L2)" if W * W * S < (100 << 20) else "exceeds L2"}
        if pull:
            l2_bytes = float(2 * W * W * S)
            row["l2_side_gbs"] = l2_bytes / ms / 1e6
            row["l2_side_frac_of_hbm_peak"] = l2_bytes / ms / 1e6 / pk["hbm_gbs"]
            if row["l2_side_frac_of_hbm_peak"] > 1.0:
                row["l2_side_note"] = "L2-served: W-1 of the W reads of each block hit in L2, so this figure is not an HBM rate"
        if row["frac_of_hbm_peak"] > 1.0:
            row["note"] = "L2-served (working set fits the 126 MB L2): not an HBM rate"
        out.append(row)
        iris.iris_heap_destroy(h)
        del mem
        torch.cuda.empty_cache()
    return out


def p2p_microbench(iris, pk):
    """Point-to-point put / get / copy / load / store between two emulated ranks (256 MiB) and atomic rates."""
    import torch
    nbytes = 256 << 20
    bpr = 2 * nbytes + (64 << 20)
    mem = torch.empty(3 * bpr, dtype=torch.uint8, device="cuda")
    ext = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    h = iris.iris_heap_create(3, bpr, external_base=mem.data_ptr())
    b0 = iris.iris_heap_base(h, 0)
    stream = torch.cuda.current_stream()
    rows, rb = nbytes // 65536, 65536

    def timed(fn, iters=5):
        fn(); fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        gpu_gate(torch)
        e0.record(stream)
        for _ in range(iters):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    out = {}
    ops = {"put": lambda: iris.iris_put_tile(h, b0, b0 + nbytes, rows, rb, rb, rb, 0, 1),
           "get": lambda: iris.iris_get_tile(h, b0, b0 + nbytes, rows, rb, rb, rb, 0, 1),
           "copy": lambda: iris.iris_copy_tile(h, b0, b0 + nbytes, rows, rb, rb, rb, 0, 1, 2),
           "load": lambda: iris.iris_load_tile(h, b0, ext, rows, rb, rb, rb, 0, 1),
           "store": lambda: iris.iris_store_tile(h, ext, b0, rows, rb, rb, rb, 0, 1)}
    for name, fn in ops.items():
        ms = timed(fn)
        out[name] = {"bytes": nbytes, "ms": ms, "gbs": 2.0 * nbytes / ms / 1e6, "frac_of_hbm_peak": 2.0 * nbytes / ms / 1e6 / pk["hbm_gbs"]}
    n = 1 << 24
    flag_base = b0 + 2 * nbytes
    iris.iris_flags_fill(h, 2 * nbytes, n, 0)
    for name, fn in {"atomic_add": lambda: iris.iris_atomic_add(h, flag_base, n, 4, 0, 1, 1),
                     "atomic_cas": lambda: iris.iris_atomic_cas(h, flag_base, n, 4, 0, 1, 0, 1, iris.IRIS_SEM_RELEASE),
                     "atomic_xchg": lambda: iris.iris_atomic_rmw(h, iris.IRIS_OP_XCHG, flag_base, n, 4, 0, 1, 7),
                     "atomic_add_one_word": lambda: iris.iris_atomic_add_contended(h, flag_base, n, 0, 1, 1)}.items():
        ms = timed(fn, 3)
        out[name] = {"ops": n, "ms": ms, "gops": n / ms / 1e6}
    iris.iris_heap_destroy(h)
    del mem, ext
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--mode", default="workgroup_specialized", choices=["bulk_synchronous", "fused_sequential", "workgroup_specialized"])
    ap.add_argument("--comm-ctas", type=int, default=0)
    ap.add_argument("--raster-group", type=int, default=0)
    ap.add_argument("--block-n", type=int, default=0)
    ap.add_argument("--cta-pair", type=int, default=0)
    ap.add_argument("--static-schedule", type=int, default=0)
    ap.add_argument("--fused-consumer", type=int, default=0)
    ap.add_argument("--stream-k", type=int, default=0)
    ap.add_argument("--wg-tail", type=int, default=0, help="workgroup_specialized: 0 = producers scatter the last wave themselves, -1 = never, n = last n tiles")
    ap.add_argument("--fuse-tail", type=int, default=0, help="-1 = a ragged shard's remainder columns are a tile of their own")
    ap.add_argument("--stage-k", type=int, default=0, help="pair kernel: 64 or 128 columns of K per operand stage (0 = 128)")
    ap.add_argument("--mode-iters", type=int, default=3)
    ap.add_argument("--steady-seconds", type=float, default=1.0, help="length of the back-to-back loop behind roofline.steady (0 = skip)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-strips", type=int, default=32)
    ap.add_argument("--sweep", default="short", choices=["none", "short", "full"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3                       # timing hygiene: at least three warm-up steps
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
