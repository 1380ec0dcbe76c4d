#!/usr/bin/env python
"""Benchmark of the paged-KV pack/unpack hot path on B200.

One step = one pass of the hot path over one request of the workload:
  block table -> chunk mapper -> ONE pack launch (gather the prefix into contiguous
  chunks in a staging area) -> ONE unpack launch (scatter the chunks into a second,
  independently drawn set of pool blocks).
Default workload: Llama-3.1-8B KV shape (32 layers, 8 KV heads, head dim 128, 16-token
blocks, 2-byte elements), one 80,000-token prefix = 5000 blocks scattered over a
20,000-block pool (39 GiB), 256-token chunks.  All inputs are synthetic and seeded.

`value` counts bytes read + bytes written by pack and unpack, with everything resident in
HBM.  `e2e` is the same byte count when the prefix is offloaded to pinned HOST memory and
loaded back through the bounded staging ring (device->host and host->device copies inside
the timed region).  `cpu_baseline` is the CPU oracle timed on a bounded sample.

  python bench.py [--gpus N --steps K --warmup W] [--impl reference]
For N > 1 launch under torch.distributed.run; every rank runs an independent replica
(the path needs no exchange between GPUs).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
METRIC = "pack+unpack GB/s (bytes read+written), 80k-token prefix, 8B KV shape"
# DRAM bytes of one launch of the default workload, and where the figure comes from.  The capture
# predates later edits of the kernel file; `kernel_file_sha256_at_capture` is compared with the file
# as it is now and the line says whether they still match (a mismatch means: capture again).
TRAFFIC_8B_80K = {
    "bytes": 20_920_170_000.0,
    "source": "profiles/kvc_bulk_kernel_8b_80k_dram_traffic.md",
    "kernel_file": "paper_2609_11744_b200/csrc/kvc_kernels.cu",
    "kernel_file_sha256_at_last_check": "372d51959538a4b208716ac5e245c751f5d2247fb86df750d1a596d13a7471f7",
}


def traffic_source_note():
    """Where roofline.traffic comes from, and whether the kernel source still is the file the
    figure was last checked against."""
    import hashlib
    try:
        with open(os.path.join(ROOT, TRAFFIC_8B_80K["kernel_file"]), "rb") as f:
            now = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        now = None
    same = now == TRAFFIC_8B_80K["kernel_file_sha256_at_last_check"]
    return "%s (kernel source %s since the last check of this figure)" % (
        TRAFFIC_8B_80K["source"], "unchanged" if same else "CHANGED")


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ clocks
class ClockSampler(threading.Thread):
    """Reads SM clock and clock-event (throttle) reasons through NVML every ~10 ms while the
    timed region runs; `summary(t0, t1)` keeps the samples taken inside that window."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, torch, cuda_index: int):
        super().__init__(daemon=True)
        self.samples, self._halt, self.h, self.nv = [], threading.Event(), None, None
        self.sm_max = None
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(cuda_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.nv = pynvml
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def run(self):
        if self.h is None:
            return
        nv = self.nv
        reasons_fn = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._halt.is_set():
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                rs = int(reasons_fn(self.h))
                try:
                    watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                except Exception:
                    watts = None
                self.samples.append((time.perf_counter(), float(sm), rs, watts))
            except Exception:
                pass
            time.sleep(0.01)

    def window(self, t0: float, t1: float):
        """Median SM clock, median board power and the reasons seen between two perf_counter times
        (the sampler keeps running)."""
        inside = [x for x in list(self.samples) if t0 <= x[0] <= t1]
        if not inside:
            return None
        bits = 0
        for x in inside:
            bits |= x[2]
        watts = [x[3] for x in inside if x[3] is not None]
        return {"sm_mhz": statistics.median(x[1] for x in inside),
                "watts": statistics.median(watts) if watts else None,
                "reasons": sorted(v for k, v in self.REASONS.items() if bits & k), "samples": len(inside)}

    def summary(self, t0: float, t1: float):
        self._halt.set()
        self.join(timeout=2)
        inside = [x for x in self.samples if t0 <= x[0] <= t1]
        window = "timed region"
        if len(inside) < 3:   # a very short timed region: fall back to everything sampled under load
            inside, window = self.samples, "warm-up + timed region"
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": len(inside),
               "window": window}
        if inside:
            out["sm_mhz"] = statistics.median(x[1] for x in inside)
            bits = 0
            for x in inside:
                bits |= x[2]
            out["reasons"] = sorted(v for k, v in self.REASONS.items() if bits & k)
        return out


# ------------------------------------------------------------------ CPU oracle timing
class OracleSample:
    """The CPU oracle (as it stands) on a bounded sample of the workload: `chunks_per_pass`
    chunks of the same KV geometry over a host pool that holds only as many blocks as the sample
    needs, pack then unpack, repeated until about `target_seconds` of work is done.  The work is
    split over (layer, K|V) ranges across all usable cores."""

    def __init__(self, shape: wl.KVShape, chunk_tokens: int, seed: int):
        from oracle import oracle as orc
        self.orc = orc
        self.chunk_tokens = chunk_tokens
        self.bpc = bpc = chunk_tokens // shape.B
        budget_blocks = max(2 * bpc, (1 << 30) // shape.bytes_per_block)   # about 1 GiB of pool
        self.chunks_per_pass = max(1, budget_blocks // 2 // bpc)
        self.pool_blocks = 2 * self.chunks_per_pass * bpc
        self.g = g = orc.Dims(shape.L, shape.P, self.pool_blocks, shape.B, shape.H, shape.D, shape.e)
        self.pool = wl.random_bits(seed, g.pool_bytes)
        self.src = wl.block_ids(seed + 1, self.pool_blocks, self.chunks_per_pass * bpc)
        self.dst = wl.block_ids(seed + 2, self.pool_blocks, self.chunks_per_pass * bpc)
        cores = len(os.sched_getaffinity(0))
        lp_total = g.L * g.P
        self.nthreads = max(1, min(cores, lp_total))
        cuts = np.linspace(0, lp_total, self.nthreads + 1).astype(int)
        self.ranges = [(int(a), int(b)) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]
        self.cb = orc.chunk_bytes(g, bpc)
        self.bufs = [np.zeros(self.cb, dtype=np.uint8) for _ in range(self.chunks_per_pass)]

    def _pass(self, n_chunks):
        orc, g, bpc = self.orc, self.g, self.bpc
        t0 = time.perf_counter()
        with ThreadPoolExecutor(self.nthreads) as ex:
            futs = [ex.submit(orc.pack_chunk_into, g, self.pool, self.src[c * bpc:(c + 1) * bpc],
                              self.bufs[c], r) for c in range(n_chunks) for r in self.ranges]
            for f in futs:
                f.result()
            t1 = time.perf_counter()
            futs = [ex.submit(orc.unpack_chunk, g, self.pool, self.bufs[c],
                              self.dst[c * bpc:(c + 1) * bpc], r)
                    for c in range(n_chunks) for r in self.ranges]
            for f in futs:
                f.result()
        return t1 - t0, time.perf_counter() - t1

    def single_core(self):
        """One chunk packed and unpacked by one thread: GB/s of bytes read + written."""
        orc, g, bpc = self.orc, self.g, self.bpc
        t0 = time.perf_counter()
        orc.pack_chunk_into(g, self.pool, self.src[:bpc], self.bufs[0])
        orc.unpack_chunk(g, self.pool, self.bufs[0], self.dst[:bpc])
        return 4 * self.cb / (time.perf_counter() - t0) / 1e9

    def run(self, target_seconds: float):
        p1, u1 = self._pass(1)
        want = max(1, round(target_seconds / max(p1 + u1, 1e-6)))
        tp = tu = 0.0
        done = 0
        while done < want:
            k = min(self.chunks_per_pass, want - done)
            a, b = self._pass(k)
            tp, tu, done = tp + a, tu + b, done + k
        moved = 2 * done * self.cb  # bytes read + written, per direction
        return {
            "value": 2 * moved / (tp + tu) / 1e9, "unit": "GB/s", "cores": self.nthreads,
            "kind": "oracle",
            "sample": "%d chunks of %d tokens (%d MiB each way in total) of the same KV shape, pack "
                      "then unpack, host pool of %d blocks" % (done, self.chunk_tokens,
                                                               done * self.cb >> 20, self.pool_blocks),
            "pack_gbs": moved / tp / 1e9, "unpack_gbs": moved / tu / 1e9, "seconds": tp + tu,
            "ms_per_80k_prefix_unpack_extrapolated": tu / done * (80000 / self.chunk_tokens) * 1e3,
        }


def run_reference(args, rank):
    """Reference arm: the CPU oracle on the host cores, one bounded sample per step."""
    if rank != 0:
        return
    w = wl.WORKLOADS[args.workload]
    per_step = 4.0
    vals, last = [], None
    sample = OracleSample(w.shape, args.chunk_tokens, w.seed + 100)
    for i in range(args.warmup + args.steps):
        r = sample.run(per_step)
        if i >= args.warmup:
            vals.append(r)
        last = r
    total_s = sum(v["seconds"] for v in vals)
    value = statistics.mean(v["value"] for v in vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_s / len(vals) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic",
        "config": {"workload": args.workload, "chunk_tokens": args.chunk_tokens,
                   "note": "CPU oracle on a bounded sample of the workload per step"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": last["cores"], "kind": "oracle",
                         "sample": last["sample"]},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ multi-GPU bookkeeping
def max_over_ranks(value: float, dist, world: int, device) -> float:
    """The slowest rank's time (ranks are independent replicas; there is no data-path exchange)."""
    if world <= 1:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_rank_per_step: int, steps: int, world: int, slowest_ms: float) -> float:
    """Aggregate throughput of all replicas: bytes moved by every rank over the slowest rank's time."""
    return world * bytes_per_rank_per_step * steps / (slowest_ms * 1e-3) / 1e9


# ------------------------------------------------------------------ GPU arm
def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    from paper_2609_11744_b200 import cuda_rt, kvc

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    kvc.lib()  # fail loudly if the extension is missing
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = wl.WORKLOADS[args.workload]
    s = w.shape
    NB = args.pool_blocks or w.pool_blocks
    n = args.request_blocks or w.request_blocks
    one_way = n * s.bytes_per_block
    pool = wl.random_bits_cuda(w.seed + 17 * rank, NB * s.bytes_per_block, dev)
    src = wl.block_ids(w.seed, NB, n)
    dst = wl.block_ids(w.dst_seed, NB, n)
    staging = torch.empty(one_way, dtype=torch.uint8, device=dev)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, args.chunk_tokens)
    kvc.kvc_layout_set_tuning(lay, variant=args.variant, order=args.order,
                              tile_bytes=args.tile_bytes, stages=args.stages, lag=args.lag,
                              max_ctas=args.max_ctas)
    stream = torch.cuda.current_stream()

    def step(evs=None):
        ops, keep, nbytes, on_dev = kvc.request_chunk_ops(lay, src, staging)
        if evs:
            evs[0].record(stream)
        kvc.kvc_pack_batch(lay, ops, on_dev)
        if evs:
            evs[1].record(stream)
        ops2, keep2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
        kvc.kvc_unpack_batch(lay, ops2, on_dev)
        if evs:
            evs[2].record(stream)

    sampler = ClockSampler(torch, local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    launches0 = kvc.kvc_layout_launch_count(lay)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(evs[i])
    barrier()
    t1 = time.perf_counter()
    wall = t1 - t0
    launches = kvc.kvc_layout_launch_count(lay) - launches0
    clocks = sampler.summary(t0, t1)
    total_ms = evs[0][0].elapsed_time(evs[-1][2])
    pack_ms = [e[0].elapsed_time(e[1]) for e in evs]
    unpack_ms = [e[1].elapsed_time(e[2]) for e in evs]
    skipped, expired = kvc.kvc_poll_device_status(lay)
    assert (skipped, expired) == (0, 0), "device status flags set: %r" % ((skipped, expired),)

    total_ms = max_over_ranks(total_ms, dist, world, dev)
    bytes_step = 4 * one_way  # pack: read+write; unpack: read+write
    value = whole_job_gbs(bytes_step, args.steps, world, total_ms)

    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, torch, kvc, cuda_rt, lay, s, src, dst, one_way, dev, world, dist)
    peak, peak_kind = measured_peak()
    traffic, traffic_source = args.traffic_bytes, "--traffic-bytes" if args.traffic_bytes else None
    if traffic is None and (args.workload, NB, n, args.chunk_tokens, args.variant) == \
            ("8b_80k", 20000, 5000, 256, 0):
        # dram__bytes_read.sum + dram__bytes_write.sum of one launch of this exact workload, from a
        # one-pass ncu capture (its summary is kept under profiles/): mean of the
        # pack launch (20,919,990,000) and the unpack launch (20,920,350,000)
        traffic = TRAFFIC_8B_80K["bytes"]
        traffic_source = traffic_source_note()
    launch_ms = statistics.mean(pack_ms + unpack_ms)
    achieved = 2 * one_way / (launch_ms * 1e-3) / 1e9
    roof = {
        "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "traffic": traffic, "traffic_source": traffic_source, "peak_kind": peak_kind,
        "kernel": "kvc_bulk_kernel (pack and unpack instantiations)" if args.variant != 1
                  else "kvc_vec_kernel (pack and unpack instantiations)",
        "algorithmic_bytes_per_launch": 2 * one_way,
        "avg_launch_ms": launch_ms,
        "pack": {"ms": statistics.mean(pack_ms), "min_ms": min(pack_ms),
                 "median_ms": statistics.median(pack_ms), "max_ms": max(pack_ms),
                 "gbs": 2 * one_way / statistics.mean(pack_ms) / 1e6,
                 "frac": 2 * one_way / statistics.mean(pack_ms) / 1e6 / peak},
        "unpack": {"ms": statistics.mean(unpack_ms), "min_ms": min(unpack_ms),
                   "median_ms": statistics.median(unpack_ms), "max_ms": max(unpack_ms),
                   "gbs": 2 * one_way / statistics.mean(unpack_ms) / 1e6,
                   "frac": 2 * one_way / statistics.mean(unpack_ms) / 1e6 / peak},
        "per_step_ms": {"pack": [round(x, 4) for x in pack_ms], "unpack": [round(x, 4) for x in unpack_ms]},
        "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
    }
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    overlap = None
    if world == 1 and not args.no_overlap:
        # config 5 in brief, after the timed region: chunks streamed through the ring to and from
        # the host while a bf16 matmul loop runs -- what the copies cost a compute stream
        ov = suite_ring_overlap(torch, kvc, cuda_rt, dev, 1.5, brief=True)
        overlap = {"gemm": ov["gemm"], "prefix_bytes": ov["prefix_bytes"],
                   "runs": [{"copy_blocks": "KVC_PRESET_BESIDE_COMPUTE" if r["tuning"].get("tile_bytes")
                             else "default", "direction": r["direction"],
                             "link_gbs_alone": r["link_gbs_alone"], "link_gbs_with_gemm": r["link_gbs_with_gemm"],
                             "gemm_slowdown": r["gemm_slowdown"], "overlap_efficiency": r["overlap_efficiency"],
                             "clocks": r["clocks"]}
                            for r in ov["runs"]]}
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        sample = OracleSample(s, args.chunk_tokens, w.seed + 50)
        cpu = sample.run(15.0)
        cpu["single_core_gbs"] = sample.single_core()
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.workload, "kv_shape": "L32 H8 D128 B16 2-byte", "pool_blocks": NB,
                   "request_tokens": n * s.B, "request_blocks": n,
                   "chunk_tokens": args.chunk_tokens, "bytes_each_way": one_way,
                   "launch": "one kvc_pack_batch + one kvc_unpack_batch per step",
                   "l2": "inputs larger than L2 (9.8 GiB read and 9.8 GiB written per launch)",
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "ms_to_load_80k_prefix": statistics.mean(unpack_ms),
        "pack_gbs": roof["pack"]["gbs"], "unpack_gbs": roof["unpack"]["gbs"],
        "wall_ms_per_step": wall / args.steps * 1e3,
        "clocks": clocks, "gpu_launches": int(launches), "roofline": roof,
    }
    if e2e:
        line["e2e"] = e2e
    if overlap:
        line["overlap_with_compute"] = overlap
    if cpu:
        line["cpu_baseline"] = cpu
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, torch, kvc, cuda_rt, lay, s, src, dst, one_way, dev, world, dist):
    """Offload the prefix to pinned host memory and load it back with the library's host-buffer
    entry points: chunk by chunk through a bounded ring of device staging slots
    (pack -> slot -> D2H; H2D -> slot -> unpack)."""
    cb = kvc.kvc_layout_chunk_bytes(lay, kvc.kvc_layout_blocks_per_chunk(lay))
    slot_bytes = (cb + 4095) // 4096 * 4096
    # Every rank pins a host buffer as large as the prefix.  If one of them cannot (N replicas share
    # the host's memory), all of them skip this leg together: the ranks meet in collectives below.
    ring = host = None
    problem = ""
    try:
        ring = kvc.kvc_staging_ring_create(slot_bytes, args.ring_slots, kvc.KVC_RING_DEVICE)
        host = torch.empty(one_way, dtype=torch.uint8, pin_memory=True)
    except Exception as e:  # out of pinned or device memory
        problem = "%s: %s" % (type(e).__name__, str(e)[:200])
    ok = 0.0 if problem else 1.0
    if world > 1:
        t = torch.tensor([ok], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MIN)
        ok = float(t.item())
    if ok < 1.0:
        if ring is not None:
            kvc.kvc_staging_ring_destroy(ring)
        return {"value": None, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                "unavailable": problem or "another rank could not allocate its staging memory"}
    hptr = host.data_ptr()
    s_k, s_c = torch.cuda.Stream(), torch.cuda.Stream()
    TO = 10_000_000

    def offload():
        kvc.kvc_offload_to_host(lay, ring, src, hptr, host_bytes=one_way, kernel_stream=s_k,
                                copy_stream=s_c, slot_timeout_us=TO)

    def load():
        kvc.kvc_load_from_host(lay, ring, hptr, dst, host_bytes=one_way, kernel_stream=s_k,
                               copy_stream=s_c, slot_timeout_us=TO)

    offload()
    load()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t_off, t_load = [], []
    for _ in range(args.e2e_steps):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        offload()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        load()
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        t_off.append(t1 - t0)
        t_load.append(t2 - t1)
    step_s = statistics.mean(t_off) + statistics.mean(t_load)
    step_s = max_over_ranks(step_s, dist, world, dev)
    _, acquires, stalls = kvc.kvc_staging_ring_stats(ring)
    kvc.kvc_staging_ring_destroy(ring)
    return {
        "value": world * 4 * one_way / step_s / 1e9, "unit": "GB/s",
        "h2d_bytes_per_step": one_way, "d2h_bytes_per_step": one_way,
        "ms_per_step": step_s * 1e3, "steps": args.e2e_steps,
        "offload_ms": statistics.mean(t_off) * 1e3, "load_ms": statistics.mean(t_load) * 1e3,
        "host_link_gbs_offload": one_way / statistics.mean(t_off) / 1e9,
        "host_link_gbs_load": one_way / statistics.mean(t_load) / 1e9,
        "path": "kvc_offload_to_host (kvc_pack -> %d-slot device ring -> copy engine to pinned host), then "
                "kvc_load_from_host (copy engine -> ring -> kvc_unpack): one C call each way" % args.ring_slots,
        "ring_acquires": acquires, "ring_stalls": stalls,
    }


# ------------------------------------------------------------------ suite: the other configs
def _time_ms(torch, fn, reps, warm=3, flush=None):
    """min / median of CUDA-event times of fn() on the current stream."""
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        if flush is not None:
            flush.add_(1)  # a buffer larger than L2 is rewritten between timed launches
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b))
    return min(ts), statistics.median(ts)


def _kernel_and_call_ms(torch, kvc, lay, fn, reps, warm=9):
    """(mean kernel ms, shortest kernel ms, ms per call when calls follow one another).  The kernel
    time comes from the library's own event pair around each launch, so the host work of a call
    (validating ids, building and uploading the block table) is not in it; the per-call time is
    reps back-to-back calls on one stream, first event to last, which is what a caller that keeps
    the stream fed observes (the slower of host work and kernel)."""
    kvc.kvc_layout_set_kernel_timing(lay, True)
    for _ in range(warm):   # more calls than the handle has table arenas, so none is allocated later
        fn()
    torch.cuda.synchronize()
    kvc.kvc_layout_kernel_time(lay)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    b.synchronize()
    n, total, lo, hi = kvc.kvc_layout_kernel_time(lay)
    kvc.kvc_layout_set_kernel_timing(lay, False)
    assert n == reps
    return total / n, lo, a.elapsed_time(b) / reps


def suite_chunk_sweep(torch, kvc, dev, reps):
    """8B shape, 80k-token prefix: chunk 16/256/2048 tokens, one batched launch vs one launch per
    chunk, pack and unpack timed separately."""
    w = wl.WORKLOADS["8b_80k"]
    s, NB, n = w.shape, w.pool_blocks, w.request_blocks
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    src, dst = wl.block_ids(w.seed, NB, n), wl.block_ids(w.dst_seed, NB, n)
    one_way = n * s.bytes_per_block
    staging = torch.empty(one_way, dtype=torch.uint8, device=dev)
    base = staging.data_ptr()
    out = []
    for chunk_tokens in w.chunk_tokens:
        lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, chunk_tokens)
        descs = kvc.kvc_map_request(lay, n)
        ops_p, k1, _, _ = kvc.request_chunk_ops(lay, src, staging)
        ops_u, k2, _, _ = kvc.request_chunk_ops(lay, dst, staging)

        def per_chunk(direction, ids):
            off = 0
            for (_, _, first, nb, nbytes) in descs:
                if direction == 0:
                    kvc.kvc_pack(lay, ids[first:first + nb], base + off, nbytes)
                else:
                    kvc.kvc_unpack(lay, base + off, ids[first:first + nb], nbytes)
                off += nbytes

        streams = [torch.cuda.Stream() for _ in range(4)]
        done = [torch.cuda.Event() for _ in streams]

        def per_chunk_streams(direction, ids):
            # the paper's store pipeline gives every staging slot its own stream (Sec. 6.4): here
            # the per-chunk launches rotate over four streams, so one kernel's tail overlaps the
            # next kernel's start
            cur = torch.cuda.current_stream()
            start = torch.cuda.Event()
            start.record(cur)
            for st in streams:
                st.wait_event(start)
            off = 0
            for i, (_, _, first, nb, nbytes) in enumerate(descs):
                st = streams[i % len(streams)]
                if direction == 0:
                    kvc.kvc_pack(lay, ids[first:first + nb], base + off, nbytes, stream=st)
                else:
                    kvc.kvc_unpack(lay, base + off, ids[first:first + nb], nbytes, stream=st)
                off += nbytes
            for st, ev in zip(streams, done):
                ev.record(st)
                cur.wait_event(ev)

        modes = [("batch", lambda: kvc.kvc_pack_batch(lay, ops_p, 0),
                  lambda: kvc.kvc_unpack_batch(lay, ops_u, 0))]
        modes.append(("per_chunk", lambda: per_chunk(0, src), lambda: per_chunk(1, dst)))
        modes.append(("per_chunk_4_streams", lambda: per_chunk_streams(0, src),
                      lambda: per_chunk_streams(1, dst)))
        # the same one-stream loop with the launches declared independent of one another (pdl = 3)
        modes.append(("per_chunk_independent", lambda: per_chunk(0, src), lambda: per_chunk(1, dst)))
        # ... and both one-stream loops captured once into a CUDA graph and replayed: no host work
        # per chunk at all (host ids travel in the kernel parameters, so a captured call is
        # self-contained)
        modes.append(("per_chunk_graph", None, None))
        modes.append(("per_chunk_independent_graph", None, None))
        for name, fp, fu in modes:
            kvc.kvc_layout_set_tuning(lay, pdl=3 if "independent" in name else 0, slot_memory=1)
            if name.endswith("_graph"):
                graphs = []
                for direction, ids in ((0, src), (1, dst)):
                    per_chunk(direction, ids)              # the launch shape's first use, outside capture
                    torch.cuda.synchronize()
                    gr = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gr):
                        per_chunk(direction, ids)
                    graphs.append(gr)
                fp, fu = graphs[0].replay, graphs[1].replay
            # 5000 single-chunk launches of 2 MiB are launch-bound by design: fewer repetitions
            r = reps if len(descs) <= 400 or name == "batch" else max(3, reps // 4)
            pm, pd = _time_ms(torch, fp, r)
            um, ud = _time_ms(torch, fu, r)
            out.append({"chunk_tokens": chunk_tokens, "chunks": len(descs), "mode": name,
                        "pack_ms_min": pm, "pack_ms_median": pd, "pack_gbs": 2 * one_way / pd / 1e6,
                        "unpack_ms_min": um, "unpack_ms_median": ud,
                        "unpack_gbs": 2 * one_way / ud / 1e6})
        assert kvc.kvc_poll_device_status(lay) == (0, 0)
        kvc.kvc_layout_destroy(lay)
    return out


def suite_launch_shapes(torch, kvc, dev, reps):
    """Same-process comparison of launch shapes and traversal orders on the 80k-token prefix (the
    boxes of a pool differ by a percent or so, so only numbers from one process compare)."""
    w = wl.WORKLOADS["8b_80k"]
    s, NB, n = w.shape, w.pool_blocks, w.request_blocks
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    src, dst = wl.block_ids(w.seed, NB, n), wl.block_ids(w.dst_seed, NB, n)
    one_way = n * s.bytes_per_block
    staging = torch.empty(one_way, dtype=torch.uint8, device=dev)
    other = torch.empty_like(staging)
    tm, td = _time_ms(torch, lambda: other.copy_(staging), reps)
    del other
    out = [{"name": "torch contiguous copy_ of the same bytes (context)", "pack_ms": td,
            "pack_gbs": 2 * one_way / td / 1e6, "unpack_ms": None, "unpack_gbs": None}]
    P, B, C = kvc.KVC_ORDER_PLANE_MAJOR, kvc.KVC_ORDER_BLOCK_MAJOR, kvc.KVC_ORDER_CHUNK_MAJOR
    cands = [
        ("default: bulk, streaming (2 items/block, 2 stages), chunk-major", dict()),
        ("multi-slab bulk kernel forced, one 32 KiB slab per item (A/B of the two bulk kernels)",
         dict(group=kvc.KVC_GROUP_FORCE_KERNEL)),
        ("bulk streaming, L2 evict-first hint on loads and stores", dict(l2_hint=2)),
        ("bulk streaming, L2 evict-first hint on loads only", dict(l2_hint=3)),
        ("bulk streaming, L2 evict-first hint on stores only", dict(l2_hint=4)),
        ("bulk streaming, 1 item per block", dict(items_per_cta=1)),
        ("bulk streaming, 4 items per block", dict(items_per_cta=4)),
        ("bulk streaming, 8 items per block, 3 stages", dict(items_per_cta=8, stages=3)),
        ("bulk streaming, plane-major", dict(order=P)),
        ("bulk streaming, block-major", dict(order=B)),
        ("bulk persistent 148 blocks, 4 stages, 1 load ahead, chunk-major", dict(max_ctas=148, order=C)),
        ("bulk persistent 148 blocks, 4 stages, 1 load ahead, plane-major", dict(max_ctas=148, order=P)),
        ("bulk persistent 148 blocks, 7 stages, 5 loads ahead", dict(max_ctas=148, stages=7, lag=5)),
        ("bulk persistent 148 blocks, 2 stages (serial)", dict(max_ctas=148, stages=2)),
        ("bulk persistent 148 blocks, 16 KiB tiles, 8 stages, 1 ahead", dict(max_ctas=148, tile_bytes=16384, stages=8)),
        ("bulk persistent 148 blocks, L2 evict-first hint", dict(max_ctas=148, l2_hint=2)),
        ("bulk persistent 96 blocks, 4 stages, 2 loads ahead", dict(max_ctas=96, lag=2)),
        ("vector streaming (1 item of 32 KiB per block), chunk-major", dict(variant=1)),
        ("vector persistent 444 blocks, 16 KiB tiles", dict(variant=1, max_ctas=444, tile_bytes=16384)),
        ("vector persistent 592 blocks, 16 KiB tiles", dict(variant=1, max_ctas=592, tile_bytes=16384)),
    ]
    for name, cfg in cands:
        lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
        kvc.kvc_layout_set_tuning(lay, **cfg)
        ops_p, k1, _, _ = kvc.request_chunk_ops(lay, src, staging)
        ops_u, k2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
        pm, pd = _time_ms(torch, lambda: kvc.kvc_pack_batch(lay, ops_p, 0), reps)
        um, ud = _time_ms(torch, lambda: kvc.kvc_unpack_batch(lay, ops_u, 0), reps)
        assert kvc.kvc_poll_device_status(lay) == (0, 0)
        out.append({"name": name, "tuning": cfg, "pack_ms": pd, "pack_gbs": 2 * one_way / pd / 1e6,
                    "unpack_ms": ud, "unpack_gbs": 2 * one_way / ud / 1e6})
        kvc.kvc_layout_destroy(lay)
    return out


def suite_small_slabs(torch, kvc, dev, reps, sizes=None, request_mib=2048):
    """Layouts with small slabs (tensor-parallel shards of the KV heads, 1-byte elements): 2 GiB
    requests, 32 layers x K,V, 16-token blocks, slab sizes from 32 KiB down to 256 B, 256-token
    chunks, one batched launch per direction.  Kernels: the default (bulk copies, several slabs
    per work item), the bulk kernel held to one slab per item, and the vector kernel."""
    peak = measured_peak()[0]
    L, P, B = 32, 2, 16
    out = []
    for S, H, D, e in ((32768, 8, 128, 2), (16384, 4, 128, 2), (8192, 2, 128, 2), (4096, 1, 128, 2),
                       (2048, 1, 128, 1), (1024, 1, 64, 1), (512, 1, 32, 1), (256, 1, 16, 1)):
        if sizes and S not in sizes:
            continue
        per_block = L * P * S
        n = (request_mib << 20) // per_block
        NB = 4 * n
        pool = wl.random_bits_cuda(wl.BASE_SEED + S, NB * per_block, dev)
        src, dst = wl.block_ids(wl.BASE_SEED + 1, NB, n), wl.block_ids(wl.BASE_SEED + 2, NB, n)
        staging = torch.empty(n * per_block, dtype=torch.uint8, device=dev)
        for name, cfg in (("bulk, slabs grouped per item (default)", dict()),
                          ("bulk, one slab per item", dict(group=1)),
                          ("vector kernel", dict(variant=1))):
            lay = kvc.kvc_layout_create_dense(pool, L, P, NB, B, H, D, e, 256)
            kvc.kvc_layout_set_tuning(lay, **cfg)
            ops_p, k1, nbytes, _ = kvc.request_chunk_ops(lay, src, staging)
            ops_u, k2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
            row = {"slab_bytes": S, "blocks": n, "bytes_each_way": nbytes, "kernel": name}
            for d, fn in (("pack", lambda: kvc.kvc_pack_batch(lay, ops_p, 0)),
                          ("unpack", lambda: kvc.kvc_unpack_batch(lay, ops_u, 0))):
                k_ms, k_min, call_ms = _kernel_and_call_ms(torch, kvc, lay, fn, reps)
                row.update({d + "_kernel_ms": k_ms, d + "_kernel_ms_min": k_min,
                            d + "_gbs": 2 * nbytes / k_ms / 1e6,
                            d + "_frac_of_measured_peak": 2 * nbytes / k_ms / 1e6 / peak,
                            d + "_call_ms_pipelined": call_ms,
                            d + "_call_gbs_pipelined": 2 * nbytes / call_ms / 1e6})
            assert kvc.kvc_poll_device_status(lay) == (0, 0)
            out.append(row)
            kvc.kvc_layout_destroy(lay)
        del pool, staging
        torch.cuda.empty_cache()
    return out


def suite_row_gather(torch, dev, reps):
    """Ceiling probe, independent of the library: random gather / scatter of S-byte rows by a plain
    kernel (tests/native/row_gather_probe.cu, built here with nvcc).  2 GiB of rows out of an 8 GiB
    array, best of a few launch shapes.  Context for the small_slabs part."""
    import ctypes
    import subprocess
    import tempfile
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    out = []
    with tempfile.TemporaryDirectory() as d:
        so = os.path.join(d, "librow_gather_probe.so")
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-shared",
                               "-Xcompiler", "-fPIC", "-cudart", "static", "-o", so,
                               os.path.join(ROOT, "tests", "native", "row_gather_probe.cu")])
        L = ctypes.CDLL(so)
        L.probe_rows.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 5 + [ctypes.c_void_p]
        L.probe_rows.restype = ctypes.c_int
        st = torch.cuda.current_stream().cuda_stream
        for S in (32768, 8192, 4096, 2048, 1024, 512, 256):
            total = 8 << 30
            N = total // S
            n = N // 4
            src = wl.random_bits_cuda(wl.BASE_SEED + S, total, dev)
            dst = torch.empty(n * S, dtype=torch.uint8, device=dev)
            idx = torch.from_numpy(wl.block_ids(wl.BASE_SEED + 3, N, n)).to(dev)
            best = {"gather_gbs": 0.0, "scatter_gbs": 0.0}
            for R in sorted({1, max(1, 4096 // S), max(1, 16384 // S)}):
                for grid in (148 * 8, 148 * 16):
                    def run(scatter, a, b):
                        rc = L.probe_rows(a.data_ptr(), b.data_ptr(), idx.data_ptr(), n, S, R, scatter, grid, st)
                        assert rc == 0
                    _, g = _time_ms(torch, lambda: run(0, src, dst), max(5, reps // 2))
                    _, sc = _time_ms(torch, lambda: run(1, dst, src), max(5, reps // 2))
                    best["gather_gbs"] = max(best["gather_gbs"], 2 * n * S / g / 1e6)
                    best["scatter_gbs"] = max(best["scatter_gbs"], 2 * n * S / sc / 1e6)
            out.append(dict(row_bytes=S, rows=n, **best))
            del src, dst, idx
            torch.cuda.empty_cache()
        # linear streams over 8 GiB for context: read only, write only, copy (bytes moved / time)
        L.probe_stream.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_int,
                                   ctypes.c_void_p, ctypes.c_void_p]
        L.probe_stream.restype = ctypes.c_int
        nbytes = 8 << 30
        a = wl.random_bits_cuda(wl.BASE_SEED + 5, nbytes, dev)
        b = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        sink = torch.zeros(1, dtype=torch.int32, device=dev)
        streams = {}
        for mode, name, moved in ((0, "read_only_gbs", nbytes), (1, "write_only_gbs", nbytes),
                                  (2, "copy_gbs", 2 * nbytes)):
            best = 0.0
            for grid in (148 * 4, 148 * 8, 148 * 16, 148 * 32):
                def run():
                    rc = L.probe_stream(a.data_ptr(), b.data_ptr(), nbytes, mode, grid, sink.data_ptr(), st)
                    assert rc == 0
                _, med = _time_ms(torch, run, max(5, reps // 2))
                best = max(best, moved / med / 1e6)
            streams[name] = best
        out.append({"linear_streams_8GiB": streams})
    return out


def suite_call_overhead(reps):
    """Per-call cost of the per-chunk entry points measured from C: builds and runs
    tests/native/call_overhead.c against the in-tree library (gcc and the CUDA headers needed)."""
    import subprocess
    import tempfile
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    pkg = os.path.join(ROOT, "paper_2609_11744_b200")
    with tempfile.TemporaryDirectory() as d:
        exe = os.path.join(d, "call_overhead")
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", os.path.join(ROOT, "tests", "native", "call_overhead.c"),
             "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
             "-L", pkg, "-lkvc", "-L", os.path.join(cuda, "lib64"), "-lcudart",
             "-Wl,-rpath," + pkg, "-Wl,-rpath," + os.path.join(cuda, "lib64"), "-o", exe])
        run = subprocess.run([exe, "6000", "5000", str(max(3, min(reps, 15)))], capture_output=True,
                             text=True, timeout=900)
    if run.returncode != 0:
        raise RuntimeError("call_overhead failed (%d): %s" % (run.returncode, run.stderr[-500:]))
    return [json.loads(l) for l in run.stdout.splitlines() if l.startswith("{")]


def suite_8k(torch, kvc, dev, reps):
    """Config 2: 8192-token prefix (1 GiB each way) with L2 flushed between timed launches."""
    w = wl.WORKLOADS["8b_8k"]
    s, NB, n = w.shape, w.pool_blocks, w.request_blocks
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    src, dst = wl.block_ids(w.seed, NB, n), wl.block_ids(w.dst_seed, NB, n)
    one_way = n * s.bytes_per_block
    staging = torch.empty(one_way, dtype=torch.uint8, device=dev)
    flush = torch.zeros(512 << 20, dtype=torch.uint8, device=dev)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    ops_p, k1, _, _ = kvc.request_chunk_ops(lay, src, staging)
    ops_u, k2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
    pm, pd = _time_ms(torch, lambda: kvc.kvc_pack_batch(lay, ops_p, 0), reps, flush=flush)
    um, ud = _time_ms(torch, lambda: kvc.kvc_unpack_batch(lay, ops_u, 0), reps, flush=flush)
    return {"bytes_each_way": one_way, "l2": "512 MiB scratch rewritten between timed launches",
            "pack_ms_min": pm, "pack_ms_median": pd, "pack_gbs": 2 * one_way / pd / 1e6,
            "unpack_ms_min": um, "unpack_ms_median": ud, "unpack_gbs": 2 * one_way / ud / 1e6}


def suite_batch(torch, kvc, dev, reps):
    """Config 4: 70B-class shape, 64 requests with lognormal lengths and a shared 1024-token
    prefix; every cache-hit chunk of every request unpacked by ONE call (shared chunks once)."""
    w = wl.WORKLOADS["70b_batch"]
    s = w.shape
    free, _ = torch.cuda.mem_get_info()
    scale = 1.0
    while True:
        NB, tables = wl.batch_workload(w, scale)
        uniq = len({int(b) for t in tables for b in t})
        need = NB * s.bytes_per_block + uniq * s.bytes_per_block + (4 << 30)
        if need < free or scale < 0.1:
            break
        scale *= 0.8   # not enough free device memory: shrink every length, and say so
    pool = torch.empty(NB * s.bytes_per_block, dtype=torch.uint8, device=dev)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    t0 = time.perf_counter()
    descs, uniq2 = kvc.kvc_map_requests_shared(lay, tables)
    map_ms = (time.perf_counter() - t0) * 1e3
    total = sum(d[4] for d in descs)
    staging = wl.random_bits_cuda(w.seed + 3, total, dev)
    slot, ids, nbs, off = [], [], [], 0
    for (r, c, first, nb, nbytes) in descs:
        slot.append(staging.data_ptr() + off)
        ids.append(tables[r].ctypes.data + 4 * first)
        nbs.append(nb)
        off += nbytes
    ops = kvc.make_chunk_ops(slot, ids, nbs)
    um, ud = _time_ms(torch, lambda: kvc.kvc_unpack_batch(lay, ops, 0), max(5, reps // 2))
    pm, pd = _time_ms(torch, lambda: kvc.kvc_pack_batch(lay, ops, 0), max(5, reps // 2))
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    return {"requests": len(tables), "length_scale": scale, "pool_blocks": NB,
            "table_blocks_total": int(sum(len(t) for t in tables)), "unique_blocks": int(uniq2),
            "chunks_after_dedup": len(descs), "bytes_each_way": total, "mapper_ms": map_ms,
            "launches_per_call": 1,
            "unpack_ms_min": um, "unpack_ms_median": ud, "unpack_gbs": 2 * total / ud / 1e6,
            "pack_ms_min": pm, "pack_ms_median": pd, "pack_gbs": 2 * total / pd / 1e6}


_OVERLAP_SAMPLER = None  # a running ClockSampler while an overlap suite part is measured


def _overlap_case(torch, fn, gemm_loop, s_gemm, s_k, s_c, iters, seconds, one_way, N, name,
                  direction, max_ctas):
    """Transfer alone, GEMM loop alone, both at once; see suite_ring_overlap."""
    fn()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    fn()
    torch.cuda.synchronize()
    once = time.perf_counter() - t0
    passes = max(1, int(seconds / once))
    t0 = time.perf_counter()
    for _ in range(passes):
        fn()
    torch.cuda.synchronize()
    t_xfer = time.perf_counter() - t0
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    g0.record(s_gemm)
    gemm_loop(iters)
    g1.record(s_gemm)
    torch.cuda.synchronize()
    t_gemm = time.perf_counter() - t0
    w_gemm = (t0, t0 + t_gemm)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    g0.record(s_gemm)
    gemm_loop(iters)
    g1.record(s_gemm)
    for _ in range(passes):
        fn()
    s_c.synchronize()
    s_k.synchronize()
    t_x_in_both = time.perf_counter() - t0
    torch.cuda.synchronize()
    t_both = time.perf_counter() - t0
    t_gemm_in_both = g0.elapsed_time(g1) * 1e-3
    eff = 1 - (t_both - max(t_gemm, t_xfer)) / min(t_gemm, t_xfer)
    clocks = None
    if _OVERLAP_SAMPLER is not None:
        # the GPU's clock and power while the GEMM loop runs alone and while the transfer runs beside it
        clocks = {"gemm_alone": _OVERLAP_SAMPLER.window(*w_gemm),
                  "gemm_with_transfer": _OVERLAP_SAMPLER.window(t0, t0 + min(t_x_in_both, t_gemm_in_both))}
    return {"clocks": clocks, "destination": name, "direction": direction, "max_ctas": max_ctas,
            "prefix_bytes": one_way, "passes": passes, "gemm_iters": iters,
            "once_ms": once * 1e3, "link_gbs_alone": passes * one_way / t_xfer / 1e9,
            "link_gbs_with_gemm": passes * one_way / t_x_in_both / 1e9,
            "t_xfer_s": t_xfer, "t_gemm_s": t_gemm, "t_both_s": t_both,
            "gemm_slowdown": t_gemm_in_both / t_gemm,
            "gemm_tflops_alone": 2 * N ** 3 * iters / t_gemm / 1e12,
            "overlap_efficiency": eff}


def _grouped_runs(torch, kvc, cuda_rt, pool, s, NB, n, src, dst, hptr, one_way, N, gemm_loop, s_gemm,
                  s_k, s_c, iters, seconds, GROUP, n_ring, TO):
    """Several ring slots per launch: one batched pack/unpack serves GROUP slots, so the compute
    stream is interrupted GROUP times less often."""
    out = []
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    descs = kvc.kvc_map_request(lay, n)
    cb = kvc.kvc_layout_chunk_bytes(lay, kvc.kvc_layout_blocks_per_chunk(lay))
    ring = kvc.kvc_staging_ring_create(cb, n_ring, kvc.KVC_RING_DEVICE)

    def grouped(direction):
        off = 0
        for g0 in range(0, len(descs), GROUP):
            grp = descs[g0:g0 + GROUP]
            slots = [kvc.kvc_staging_ring_acquire(ring, TO) for _ in grp]
            ops = kvc.make_chunk_ops([sl[1] for sl in slots],
                                     [(src if direction == 0 else dst).ctypes.data + 4 * d[2] for d in grp],
                                     [d[3] for d in grp])
            if direction == 0:
                kvc.kvc_pack_batch(lay, ops, 0, stream=s_k)
                for (slot, dptr, _), d in zip(slots, grp):
                    kvc.kvc_staging_ring_commit(ring, slot, s_k)
                    kvc.kvc_staging_ring_wait_filled(ring, slot, s_c)
                    cuda_rt.memcpy_async(hptr + off, dptr, d[4], cuda_rt.D2H, s_c)
                    kvc.kvc_staging_ring_release(ring, slot, s_c)
                    off += d[4]
            else:
                for (slot, dptr, _), d in zip(slots, grp):
                    cuda_rt.memcpy_async(dptr, hptr + off, d[4], cuda_rt.H2D, s_c)
                    kvc.kvc_staging_ring_commit(ring, slot, s_c)
                    kvc.kvc_staging_ring_wait_filled(ring, slot, s_k)
                    off += d[4]
                kvc.kvc_unpack_batch(lay, ops, 0, stream=s_k)
                for (slot, dptr, _) in slots:
                    kvc.kvc_staging_ring_release(ring, slot, s_k)

    for direction, name in ((0, "offload"), (1, "load")):
        out.append(_overlap_case(torch, lambda: grouped(direction), gemm_loop, s_gemm, s_k, s_c,
                                 iters, seconds, one_way, N,
                                 "device slots + cudaMemcpyAsync, %d slots per launch, %d-slot ring"
                                 % (GROUP, n_ring), name, 0))
    kvc.kvc_staging_ring_destroy(ring)
    kvc.kvc_layout_destroy(lay)
    return out


def suite_ring_overlap(torch, kvc, cuda_rt, dev, seconds, brief=False):
    """Config 5: a 32k-token prefix (8B shape, 4 GiB) streamed through an 8-slot ring of 256-token
    slots to/from pinned host memory while a bf16 GEMM loop runs on another stream.  Destinations:
    device slots drained by cudaMemcpyAsync, or slots in mapped pinned host memory that the
    kernels write/read directly.  Reports link GB/s, GEMM slowdown and overlap efficiency
    1 - (T_both - max(T_gemm, T_xfer)) / min(T_gemm, T_xfer).
    brief: device slots only, default blocks and the beside-compute preset (the part of this
    measurement that the default benchmark line carries)."""
    w = wl.WORKLOADS["8b_ring"]
    s, NB, n = w.shape, w.pool_blocks, w.request_blocks
    if brief:
        n //= 2   # a 16k-token prefix (2 GiB) per pass keeps the brief run short
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    src, dst = wl.block_ids(w.seed, NB, n), wl.block_ids(w.dst_seed, NB, n)
    one_way = n * s.bytes_per_block
    host = torch.empty(one_way, dtype=torch.uint8, pin_memory=True)
    hptr = host.data_ptr()
    lo, hi = torch.cuda.Stream.priority_range()
    s_gemm = torch.cuda.Stream(priority=lo)
    s_k, s_c = torch.cuda.Stream(priority=hi), torch.cuda.Stream(priority=hi)
    TO = 20_000_000
    N = 8192
    A = torch.randn(N, N, device=dev, dtype=torch.bfloat16)
    B = torch.randn(N, N, device=dev, dtype=torch.bfloat16)
    C = torch.empty(N, N, device=dev, dtype=torch.bfloat16)

    # The GEMM loop is replayed from a CUDA graph of GRAPH_ITERS matmuls, so that enqueueing two
    # seconds of GEMMs takes a few dozen launches and never blocks the host thread that also
    # drives the ring (thousands of queued kernel launches would fill the stream's launch queue
    # and stall the host before the transfer even starts).
    GRAPH_ITERS = 64
    with torch.cuda.stream(s_gemm):
        for _ in range(5):
            torch.matmul(A, B, out=C)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=s_gemm):
        for _ in range(GRAPH_ITERS):
            torch.matmul(A, B, out=C)

    def gemm_loop(iters):
        with torch.cuda.stream(s_gemm):
            for _ in range(iters // GRAPH_ITERS):
                graph.replay()

    # size the GEMM loop to about `seconds`
    gemm_loop(GRAPH_ITERS)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_gemm)
    gemm_loop(2 * GRAPH_ITERS)
    e1.record(s_gemm)
    torch.cuda.synchronize()
    per_iter = e0.elapsed_time(e1) / (2 * GRAPH_ITERS)
    iters = max(GRAPH_ITERS, int(seconds * 1e3 / per_iter) // GRAPH_ITERS * GRAPH_ITERS)
    results = []
    global _OVERLAP_SAMPLER
    _OVERLAP_SAMPLER = ClockSampler(torch, torch.cuda.current_device())
    _OVERLAP_SAMPLER.start()
    # small shared-memory footprints (2 stages of 8 or 4 KiB per block) are there to see whether copy
    # blocks that fit beside a resident GEMM block disturb the GEMM less than 66 KB blocks do
    preset = {k: v for k, v in kvc.kvc_tuning_preset(kvc.KVC_PRESET_BESIDE_COMPUTE).items() if v}
    assert preset == dict(max_ctas=16, tile_bytes=8192, stages=2)
    small = [dict(max_ctas=0, tile_bytes=8192, stages=2), dict(max_ctas=32, tile_bytes=8192, stages=2),
             preset, dict(max_ctas=32, tile_bytes=4096, stages=2)]
    for kind, kind_name in ((kvc.KVC_RING_DEVICE, "device slots + cudaMemcpyAsync"),
                            (kvc.KVC_RING_HOST_MAPPED, "mapped pinned host slots")):
        if brief and kind != kvc.KVC_RING_DEVICE:
            continue
        tunings = [dict(max_ctas=c) for c in ((16, 0) if kind == kvc.KVC_RING_DEVICE else (4, 16, 64))]
        if brief:
            tunings = [dict(max_ctas=0), preset]
        elif kind == kvc.KVC_RING_DEVICE:
            tunings += small
        else:   # one-warp vector blocks (about 2000 registers each): measured WORSE for the GEMM
            tunings += [dict(max_ctas=128, vec_threads=32)]
        for tuning in tunings:
            max_ctas = tuning["max_ctas"]
            lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
            kvc.kvc_layout_set_tuning(lay, **tuning)
            descs = kvc.kvc_map_request(lay, n)
            cb = kvc.kvc_layout_chunk_bytes(lay, kvc.kvc_layout_blocks_per_chunk(lay))
            ring = kvc.kvc_staging_ring_create(cb, int(w.extra["ring_slots"]), kind)

            def offload():
                off = 0
                for (_, c, first, nb, nbytes) in descs:
                    slot, dptr, hp = kvc.kvc_staging_ring_acquire(ring, TO)
                    kvc.kvc_pack(lay, src[first:first + nb], dptr, nbytes, stream=s_k)
                    kvc.kvc_staging_ring_commit(ring, slot, s_k)
                    kvc.kvc_staging_ring_wait_filled(ring, slot, s_c)
                    if kind == kvc.KVC_RING_DEVICE:
                        cuda_rt.memcpy_async(hptr + off, dptr, nbytes, cuda_rt.D2H, s_c)
                    # a mapped slot already is host memory: its consumer (file I/O in the paper)
                    # would read it here; nothing is copied
                    kvc.kvc_staging_ring_release(ring, slot, s_c)
                    off += nbytes

            def load():
                off = 0
                for (_, c, first, nb, nbytes) in descs:
                    slot, dptr, hp = kvc.kvc_staging_ring_acquire(ring, TO)
                    if kind == kvc.KVC_RING_DEVICE:
                        cuda_rt.memcpy_async(dptr, hptr + off, nbytes, cuda_rt.H2D, s_c)
                    # a mapped slot is filled by its producer (a file read) on the host side
                    kvc.kvc_staging_ring_commit(ring, slot, s_c)
                    kvc.kvc_staging_ring_wait_filled(ring, slot, s_k)
                    kvc.kvc_unpack(lay, dptr, dst[first:first + nb], nbytes, stream=s_k)
                    kvc.kvc_staging_ring_release(ring, slot, s_k)
                    off += nbytes

            for direction, fn in (("offload", offload), ("load", load)):
                results.append(_overlap_case(torch, fn, gemm_loop, s_gemm, s_k, s_c, iters, seconds,
                                             one_way, N, kind_name, direction, max_ctas))
                results[-1]["tuning"] = tuning
            kvc.kvc_staging_ring_destroy(ring)
            kvc.kvc_layout_destroy(lay)
    def stop_sampler():
        global _OVERLAP_SAMPLER
        _OVERLAP_SAMPLER._halt.set()
        _OVERLAP_SAMPLER.join(timeout=2)
        _OVERLAP_SAMPLER = None

    if brief:
        stop_sampler()
        return {"gemm": "bf16 %dx%dx%d torch.matmul loop" % (N, N, N), "ms_per_gemm": per_iter,
                "ring_slots": int(w.extra["ring_slots"]), "slot_bytes": cb, "prefix_bytes": one_way,
                "seconds_per_phase": seconds, "runs": results}
    for GROUP, n_ring in ((4, int(w.extra["ring_slots"])), (8, 16)):
        results.extend(_grouped_runs(torch, kvc, cuda_rt, pool, s, NB, n, src, dst, hptr, one_way, N,
                                     gemm_loop, s_gemm, s_k, s_c, iters, seconds, GROUP, n_ring, TO))
    # the paper's mechanism for comparison: strided DMA copies straight between the pool and
    # pinned host memory, no kernel, no staging slot
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    descs = kvc.kvc_map_request(lay, n)

    def dma_offload():
        off = 0
        for (_, c, first, nb, nbytes) in descs:
            kvc.kvc_pack_copy_engine(lay, src[first:first + nb], hptr + off, nbytes, stream=s_c)
            off += nbytes

    def dma_load():
        off = 0
        for (_, c, first, nb, nbytes) in descs:
            kvc.kvc_unpack_copy_engine(lay, hptr + off, dst[first:first + nb], nbytes, stream=s_c)
            off += nbytes

    for direction, fn in (("offload", dma_offload), ("load", dma_load)):
        results.append(_overlap_case(torch, fn, gemm_loop, s_gemm, s_c, s_c, iters, seconds, one_way, N,
                                     "copy engines, pool <-> pinned host directly", direction, 0))
    kvc.kvc_layout_destroy(lay)
    stop_sampler()
    return {"gemm": "bf16 %dx%dx%d torch.matmul loop" % (N, N, N), "ms_per_gemm": per_iter,
            "ring_slots": int(w.extra["ring_slots"]), "slot_bytes": cb, "runs": results}


def suite_duplex(torch, kvc, cuda_rt, dev, reps):
    """Sec. 6.4: loads, stores and preloads share one staging pool.  Request A (32k tokens, 8B shape,
    4 GiB) is offloaded to pinned host memory while request B (same size) is loaded from pinned host
    memory, through ONE 8-slot pool, chunk by chunk in alternation, each direction on its own kernel
    and copy stream.  Reported against the duplex ceiling of the host link measured in the same
    process (two 1 GiB cudaMemcpyAsync, one per direction, running at once)."""
    w = wl.WORKLOADS["8b_ring"]
    s, NB, n = w.shape, w.pool_blocks, w.request_blocks // 2
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    perm = wl.block_ids(w.seed, NB, NB)
    ids_a, ids_b = perm[:n], np.ascontiguousarray(perm[n:2 * n])
    one_way = n * s.bytes_per_block
    host_a = torch.empty(one_way, dtype=torch.uint8, pin_memory=True)
    host_b = torch.empty(one_way, dtype=torch.uint8, pin_memory=True)
    s_pack, s_d2h, s_h2d, s_unpack = (torch.cuda.Stream() for _ in range(4))
    # duplex ceiling
    nb1 = 1 << 30
    dbuf = torch.empty(2 * nb1, dtype=torch.uint8, device=dev)
    best = None
    for _ in range(6):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        torch.cuda.synchronize()
        e[0].record(s_d2h)
        e[2].record(s_h2d)
        cuda_rt.memcpy_async(host_a.data_ptr(), dbuf.data_ptr(), nb1, cuda_rt.D2H, s_d2h)
        cuda_rt.memcpy_async(dbuf.data_ptr() + nb1, host_b.data_ptr(), nb1, cuda_rt.H2D, s_h2d)
        e[1].record(s_d2h)
        e[3].record(s_h2d)
        torch.cuda.synchronize()
        t = max(e[0].elapsed_time(e[1]), e[2].elapsed_time(e[3]))
        cand = {"d2h_gbs": nb1 / e[0].elapsed_time(e[1]) / 1e6, "h2d_gbs": nb1 / e[2].elapsed_time(e[3]) / 1e6,
                "aggregate_gbs": 2 * nb1 / t / 1e6}
        if best is None or cand["aggregate_gbs"] > best["aggregate_gbs"]:
            best = cand
    del dbuf
    out = {"prefix_bytes_each_direction": one_way, "duplex_ceiling": best, "runs": []}
    TO = 20_000_000
    mapped = "mapped pinned host slots (kernels cross the link), %s blocks per kernel"
    for kind, kind_name, ctas in ((kvc.KVC_RING_DEVICE, "device slots + cudaMemcpyAsync", 0),
                                  (kvc.KVC_RING_HOST_MAPPED, mapped % "16 (default)", 0),
                                  (kvc.KVC_RING_HOST_MAPPED, mapped % "32", 32),
                                  (kvc.KVC_RING_HOST_MAPPED, mapped % "64", 64)):
        lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
        kvc.kvc_layout_set_tuning(lay, max_ctas=ctas)
        descs = kvc.kvc_map_request(lay, n)
        cb = kvc.kvc_layout_chunk_bytes(lay, kvc.kvc_layout_blocks_per_chunk(lay))
        ring = kvc.kvc_staging_ring_create(cb, int(w.extra["ring_slots"]), kind)
        kvc.kvc_staging_ring_set_policy(ring, 0)

        def both():
            off = 0
            for (_, c, first, nb, nbytes) in descs:
                slot, dptr, hp, _ = kvc.kvc_staging_ring_acquire_for(ring, kvc.KVC_CLASS_STORE, 2 * c, TO)
                kvc.kvc_pack(lay, ids_a[first:first + nb], dptr, nbytes, stream=s_pack)
                kvc.kvc_staging_ring_commit(ring, slot, s_pack)
                kvc.kvc_staging_ring_wait_filled(ring, slot, s_d2h)
                if kind == kvc.KVC_RING_DEVICE:
                    cuda_rt.memcpy_async(host_a.data_ptr() + off, dptr, nbytes, cuda_rt.D2H, s_d2h)
                kvc.kvc_staging_ring_release(ring, slot, s_d2h)
                slot, dptr, hp, _ = kvc.kvc_staging_ring_acquire_for(ring, kvc.KVC_CLASS_DEMAND_LOAD,
                                                                     2 * c + 1, TO)
                if kind == kvc.KVC_RING_DEVICE:
                    cuda_rt.memcpy_async(dptr, host_b.data_ptr() + off, nbytes, cuda_rt.H2D, s_h2d)
                kvc.kvc_staging_ring_commit(ring, slot, s_h2d)
                kvc.kvc_staging_ring_wait_filled(ring, slot, s_unpack)
                kvc.kvc_unpack(lay, dptr, ids_b[first:first + nb], nbytes, stream=s_unpack)
                kvc.kvc_staging_ring_release(ring, slot, s_unpack)
                off += nbytes

        both()
        torch.cuda.synchronize()
        ts = []
        for _ in range(max(3, reps // 4)):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            both()
            torch.cuda.synchronize()
            ts.append(time.perf_counter() - t0)
        t = statistics.median(ts)
        c = kvc.kvc_staging_ring_policy_counters(ring)
        out["runs"].append({"slots": kind_name, "seconds": t, "per_direction_gbs": one_way / t / 1e9,
                            "aggregate_gbs": 2 * one_way / t / 1e9,
                            "frac_of_duplex_ceiling": 2 * one_way / t / 1e9 / best["aggregate_gbs"],
                            "acquires": c["acquires"]})
        assert kvc.kvc_poll_device_status(lay) == (0, 0)
        kvc.kvc_staging_ring_destroy(ring)
        kvc.kvc_layout_destroy(lay)
    return out


def suite_host_link(torch, cuda_rt, dev):
    """Host-link ceiling of this machine: cudaMemcpyAsync of 1 GiB of pinned memory, each direction,
    best of 10."""
    nbytes = 1 << 30
    host = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    devb = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream()
    out = {}
    for name, dst, src, kind in (("d2h_gbs", host, devb, cuda_rt.D2H), ("h2d_gbs", devb, host, cuda_rt.H2D)):
        best = 1e9
        for _ in range(10):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st)
            cuda_rt.memcpy_async(dst.data_ptr(), src.data_ptr(), nbytes, kind, st)
            b.record(st)
            b.synchronize()
            best = min(best, a.elapsed_time(b))
        out[name] = nbytes / best / 1e6
    return out


def suite_file_pipeline(torch, kvc, dev, root):
    """f1: a 32k-token prefix (8B shape, 4 GiB) offloaded to chunk files and loaded back through an
    8-slot mapped-host ring, with 4 I/O threads, kernel copies and copy-engine copies.  `root` is
    where the files go (the box's scratch disk, or /dev/shm as the memory-backed upper bound)."""
    import shutil
    import tempfile
    w = wl.WORKLOADS["8b_ring"]
    s, NB, n = w.shape, w.pool_blocks, w.request_blocks
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    src, dst = wl.block_ids(w.seed, NB, n), wl.block_ids(w.dst_seed, NB, n)
    out = []
    for base in root.split(","):
        if not os.path.isdir(base):
            continue
        # (copies by the DMA engines or by kernels, I/O threads, FIFO ring or pool mode)
        M, ST = kvc.KVC_RING_HOST_MAPPED, kvc.KVC_RING_DEVICE_STAGED
        for use_ce, threads, pool_mode, kind in ((False, 4, False, M), (True, 4, False, M), (False, 8, True, M),
                                                 (False, 16, True, M), (False, 4, False, ST),
                                                 (False, 16, True, ST)):
            d = tempfile.mkdtemp(prefix="kvc_suite_", dir=base)
            try:
                lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
                if kind == ST:
                    kvc.kvc_layout_set_tuning(lay, **kvc.kvc_tuning_preset(kvc.KVC_PRESET_BESIDE_COMPUTE))
                else:
                    kvc.kvc_layout_set_tuning(lay, max_ctas=16)
                cb = kvc.kvc_layout_chunk_bytes(lay, kvc.kvc_layout_blocks_per_chunk(lay))
                ring = kvc.kvc_staging_ring_create(cb, 8 if not pool_mode else 2 * threads, kind)
                if pool_mode:
                    kvc.kvc_staging_ring_set_policy(ring, 0)
                store = kvc.kvc_store_open(d, "8b", direct_io=True)
                hashes = [kvc.kvc_fnv1a64(b"chunk%d" % c) for c in range(kvc.kvc_layout_num_chunks(lay, n))]
                st = kvc.kvc_pipeline_store(lay, ring, store, src, hashes, io_threads=threads,
                                            use_copy_engine=use_ce)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                if pool_mode:
                    ld, _ = kvc.kvc_pipeline_load_many(
                        lay, ring, store, [dict(ids=dst, hashes=hashes, cls=kvc.KVC_CLASS_DEMAND_LOAD)],
                        io_threads=threads)
                    ld["bytes"] = ld["bytes_read"]
                else:
                    ld = kvc.kvc_pipeline_load(lay, ring, store, dst, hashes, io_threads=threads,
                                               use_copy_engine=use_ce)
                torch.cuda.synchronize()
                load_s = time.perf_counter() - t0
                copies = "copy engines, pool <-> host" if use_ce else "kernels (16 CTAs) across the link"
                if kind == ST:
                    copies = "kernels (beside-compute preset) to device halves + one async copy per chunk"
                out.append({"root": base, "copies": copies,
                            "io_threads": threads,
                            "staging": (("pool mode, %d slots" % (2 * threads)) if pool_mode else "FIFO ring, 8 slots")
                            + (", device + pinned host halves" if kind == ST else ", mapped pinned"),
                            "bytes": st["bytes"], "store_s": st["seconds"],
                            "store_gbs": st["bytes"] / st["seconds"] / 1e9,
                            "load_s": load_s, "load_gbs": ld["bytes"] / load_s / 1e9,
                            "chunks": st["chunks"], "published": st["published"],
                            "direct_io_refused": kvc.kvc_store_direct_io_refused(store),
                            "ring_stalls_store": st["ring_stalls"]})
                kvc.kvc_store_close(store)
                kvc.kvc_staging_ring_destroy(ring)
                kvc.kvc_layout_destroy(lay)
            finally:
                shutil.rmtree(d, ignore_errors=True)
    return out


def suite_pipeline_beside_gemm(torch, kvc, dev, roots):
    """The paper's actual situation (Sec. 2.3, 5.1): chunks go to storage while the model computes.
    A 4 GiB request (8B shape) is offloaded to chunk files again and again while a bf16 8192^3
    matmul loop of about 3 s runs on another stream; then loaded back the same way.  Mapped pinned
    slots written / read by the kernels themselves against device + pinned-host slot pairs with the
    beside-compute kernel shape and copy-engine transfers.  Files on the memory-backed file system
    when there is one (the scratch disk would only measure the disk)."""
    import shutil
    import tempfile
    w = wl.WORKLOADS["8b_ring"]
    s, NB, n = w.shape, w.pool_blocks, w.request_blocks
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    src, dst = wl.block_ids(w.seed, NB, n), wl.block_ids(w.dst_seed, NB, n)
    lo, hi = torch.cuda.Stream.priority_range()
    s_gemm, s_io = torch.cuda.Stream(priority=lo), torch.cuda.Stream(priority=hi)
    N, GRAPH_ITERS = 8192, 64
    A = torch.randn(N, N, device=dev, dtype=torch.bfloat16)
    B = torch.randn(N, N, device=dev, dtype=torch.bfloat16)
    C = torch.empty(N, N, device=dev, dtype=torch.bfloat16)
    with torch.cuda.stream(s_gemm):
        for _ in range(5):
            torch.matmul(A, B, out=C)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=s_gemm):
        for _ in range(GRAPH_ITERS):
            torch.matmul(A, B, out=C)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def gemm_loop(replays):
        e0.record(s_gemm)
        with torch.cuda.stream(s_gemm):
            for _ in range(replays):
                graph.replay()
        e1.record(s_gemm)

    gemm_loop(4)
    torch.cuda.synchronize()
    replays = max(8, int(3000.0 / (e0.elapsed_time(e1) / 4)))
    gemm_loop(replays)
    torch.cuda.synchronize()
    t_alone = e0.elapsed_time(e1)
    roots_ok = [r for r in roots.split(",") if os.path.isdir(r)]
    base = "/dev/shm" if "/dev/shm" in roots_ok else (roots_ok[0] if roots_ok else None)
    out = {"gemm": "bf16 %d^3 matmul loop, %d launches" % (N, replays * GRAPH_ITERS), "gemm_alone_ms": t_alone,
           "files_on": base, "runs": []}
    if base is None:
        return out
    for kind, name in ((kvc.KVC_RING_HOST_MAPPED, "mapped pinned slots, kernels cross the link (16 blocks)"),
                       (kvc.KVC_RING_DEVICE_STAGED, "device + pinned-host slot pairs, beside-compute kernels, "
                                                    "copy engines cross the link")):
        d = tempfile.mkdtemp(prefix="kvc_gemm_", dir=base)
        try:
            lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
            if kind == kvc.KVC_RING_DEVICE_STAGED:
                kvc.kvc_layout_set_tuning(lay, **kvc.kvc_tuning_preset(kvc.KVC_PRESET_BESIDE_COMPUTE))
            else:
                kvc.kvc_layout_set_tuning(lay, max_ctas=16)
            cb = kvc.kvc_layout_chunk_bytes(lay, kvc.kvc_layout_blocks_per_chunk(lay))
            ring = kvc.kvc_staging_ring_create(cb, 16, kind)
            kvc.kvc_staging_ring_set_policy(ring, 0)
            n_chunks = kvc.kvc_layout_num_chunks(lay, n)
            for direction in ("store", "load"):
                stores = []

                def one_pass(k):
                    if direction == "store":
                        store = kvc.kvc_store_open(os.path.join(d, "p%d" % k), "8b", direct_io=True)
                        hashes = [kvc.kvc_fnv1a64(b"c%d" % c) for c in range(n_chunks)]
                        st = kvc.kvc_pipeline_store(lay, ring, store, src, hashes, io_threads=8, stream=s_io)
                        stores.append((store, hashes))
                        return st["bytes"]
                    store, hashes = loaded
                    st, _ = kvc.kvc_pipeline_load_many(
                        lay, ring, store, [dict(ids=dst, hashes=hashes, cls=kvc.KVC_CLASS_DEMAND_LOAD)],
                        io_threads=8, stream=s_io)
                    s_io.synchronize()
                    return st["bytes_read"]

                if direction == "load":
                    loaded = keep_store
                res = {}
                for with_gemm in (False, True):
                    os.makedirs(d, exist_ok=True)
                    torch.cuda.synchronize()
                    if with_gemm:
                        gemm_loop(replays)
                    t0 = time.perf_counter()
                    moved, k = 0, 0
                    while True:
                        moved += one_pass(k)
                        k += 1
                        elapsed = time.perf_counter() - t0
                        if (with_gemm and e1.query()) or (not with_gemm and elapsed > 1.5) or k >= 24:
                            break
                    s_io.synchronize()
                    elapsed = time.perf_counter() - t0
                    torch.cuda.synchronize()
                    res["with_gemm" if with_gemm else "alone"] = moved / elapsed / 1e9
                    if with_gemm:
                        res["gemm_slowdown"] = e0.elapsed_time(e1) / t_alone
                    if direction == "store":
                        keep_store = stores[0]
                        for st_, _h in stores[1:]:
                            kvc.kvc_store_close(st_)
                        for kk in range(1, k):
                            shutil.rmtree(os.path.join(d, "p%d" % kk), ignore_errors=True)
                        stores = []
                out["runs"].append({"slots": name, "direction": direction, "file_gbs_alone": res["alone"],
                                    "file_gbs_beside_gemm": res["with_gemm"],
                                    "gemm_slowdown": res["gemm_slowdown"]})
            assert kvc.kvc_poll_device_status(lay) == (0, 0)
            kvc.kvc_store_close(keep_store[0])
            kvc.kvc_staging_ring_destroy(ring)
            kvc.kvc_layout_destroy(lay)
        finally:
            shutil.rmtree(d, ignore_errors=True)
    return out


def suite_preload_trace(torch, kvc, dev, roots):
    """Sec. 6.5 in miniature: a queue of requests, each needing its 2048-token prefix (8 chunks of
    32 MiB, 8B shape; the first 1024 tokens are common to all) loaded from chunk files before a
    forward pass of ~40 ms (a matmul burst) can run.  Without preloading every request pays the file
    reads on its critical path.  With preloading the NEXT request's chunks are read into the staging
    pool while the current forward pass runs on the GPU, so its demand load finds them staged, claims
    them and only the unpack remains.  One staging pool of 12 slots, 4 reserved for demand work."""
    import shutil
    import tempfile
    w = wl.WORKLOADS["8b_ring"]
    s, NB = w.shape, w.pool_blocks
    n_req, n_blocks, shared_blocks = 10, 128, 64
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, dev)
    perm = wl.block_ids(w.seed, NB, NB)
    shared = perm[:shared_blocks]
    srcs, dsts, cur = [], [], shared_blocks
    for r in range(n_req):
        srcs.append(np.ascontiguousarray(np.concatenate([shared, perm[cur:cur + n_blocks - shared_blocks]])))
        cur += n_blocks - shared_blocks
    for r in range(n_req):
        dsts.append(np.ascontiguousarray(perm[cur:cur + n_blocks]))
        cur += n_blocks
    N = 8192
    A = torch.randn(N, N, device=dev, dtype=torch.bfloat16)
    B = torch.randn(N, N, device=dev, dtype=torch.bfloat16)
    C = torch.empty(N, N, device=dev, dtype=torch.bfloat16)
    s_fwd = torch.cuda.Stream()

    def forward_pass():
        with torch.cuda.stream(s_fwd):
            for _ in range(50):
                torch.matmul(A, B, out=C)

    out = []
    for base in roots.split(","):
        if not os.path.isdir(base):
            continue
        d = tempfile.mkdtemp(prefix="kvc_trace_", dir=base)
        try:
            lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
            kvc.kvc_layout_set_tuning(lay, max_ctas=16)
            cb = kvc.kvc_layout_chunk_bytes(lay, kvc.kvc_layout_blocks_per_chunk(lay))
            store = kvc.kvc_store_open(d, "8b", direct_io=True)
            hashes = []
            for r in range(n_req):
                hs, h = [], 0
                for c in range(n_blocks // 16):
                    tag = b"shared" if c < shared_blocks // 16 else b"req%d" % r
                    h = kvc.kvc_fnv1a64(tag + b".%d.%d" % (c, h))
                    hs.append(h)
                hashes.append(hs)
            fifo = kvc.kvc_staging_ring_create(cb, 8, kvc.KVC_RING_HOST_MAPPED)
            for r in range(n_req):
                kvc.kvc_pipeline_store(lay, fifo, store, srcs[r], hashes[r], io_threads=4)
            kvc.kvc_staging_ring_destroy(fifo)
            forward_pass()
            torch.cuda.synchronize()
            for preload in (False, True):
                ring = kvc.kvc_staging_ring_create(cb, 12, kvc.KVC_RING_HOST_MAPPED)
                kvc.kvc_staging_ring_set_policy(ring, foreground_reserve=4, max_speculative=8)
                reads0 = kvc.kvc_store_get_counters(store)["reads"]
                lat, joins, claims = [], 0, 0
                t_start = time.perf_counter()
                for r in range(n_req):
                    t0 = time.perf_counter()
                    st, res = kvc.kvc_pipeline_load_many(
                        lay, ring, store, [dict(ids=dsts[r], hashes=hashes[r], cls=kvc.KVC_CLASS_DEMAND_LOAD)],
                        io_threads=4)
                    torch.cuda.current_stream().synchronize()
                    lat.append(time.perf_counter() - t0)
                    joins += st["joins"]
                    claims = st["claims"]
                    forward_pass()                      # asynchronous: the GPU is busy, the host is not
                    if preload and r + 1 < n_req:
                        kvc.kvc_pipeline_load_many(
                            lay, ring, store,
                            [dict(hashes=hashes[r + 1], n_blocks=n_blocks, cls=kvc.KVC_CLASS_PRELOAD)],
                            io_threads=4)
                    s_fwd.synchronize()
                total = time.perf_counter() - t_start
                out.append({"root": base, "preloading": preload, "requests": n_req,
                            "prefix_bytes": n_blocks * s.bytes_per_block,
                            "demand_load_ms_mean": statistics.mean(lat) * 1e3,
                            "demand_load_ms_median": statistics.median(lat) * 1e3,
                            "demand_load_ms_first": lat[0] * 1e3, "total_s": total,
                            "file_reads": kvc.kvc_store_get_counters(store)["reads"] - reads0,
                            "joins": joins, "claims": claims})
                torch.cuda.synchronize()
                kvc.kvc_staging_ring_destroy(ring)
            assert kvc.kvc_poll_device_status(lay) == (0, 0)
            kvc.kvc_store_close(store)
            kvc.kvc_layout_destroy(lay)
        finally:
            shutil.rmtree(d, ignore_errors=True)
    return out


def run_suite(args):
    import torch
    from paper_2609_11744_b200 import cuda_rt, kvc
    torch.cuda.set_device(0)
    dev = "cuda:0"
    parts = args.suite.split(",")
    out = {"suite": True, "peak_hbm_gbs": measured_peak()[0], "data": "synthetic"}
    for name, fn in (("host_link", lambda: suite_host_link(torch, cuda_rt, dev)),
                     ("launch_shapes", lambda: suite_launch_shapes(torch, kvc, dev, args.steps)),
                     ("chunk_sweep", lambda: suite_chunk_sweep(torch, kvc, dev, args.steps)),
                     ("small_slabs", lambda: suite_small_slabs(
                         torch, kvc, dev, args.steps,
                         [int(x) for x in args.small_slab_sizes.split(",")] if args.small_slab_sizes else None,
                         args.small_slab_mib)),
                     ("row_gather", lambda: suite_row_gather(torch, dev, args.steps)),
                     ("call_overhead", lambda: suite_call_overhead(args.steps)),
                     ("prefix_8k", lambda: suite_8k(torch, kvc, dev, args.steps)),
                     ("batch_70b", lambda: suite_batch(torch, kvc, dev, args.steps)),
                     ("ring_overlap", lambda: suite_ring_overlap(torch, kvc, cuda_rt, dev,
                                                                 args.overlap_seconds)),
                     ("duplex", lambda: suite_duplex(torch, kvc, cuda_rt, dev, args.steps)),
                     ("file_pipeline", lambda: suite_file_pipeline(torch, kvc, dev, args.file_roots)),
                     ("preload_trace", lambda: suite_preload_trace(torch, kvc, dev, args.file_roots)),
                     ("pipeline_beside_gemm", lambda: suite_pipeline_beside_gemm(torch, kvc, dev,
                                                                                 args.file_roots))):
        if "all" in parts or name in parts:
            out[name] = fn()
            torch.cuda.synchronize()
            torch.cuda.empty_cache()
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b_80k", choices=["8b_80k", "8b_8k"])
    ap.add_argument("--chunk-tokens", type=int, default=256)
    ap.add_argument("--variant", type=int, default=0, help="0 auto, 1 vector kernel, 2 bulk-copy kernel")
    ap.add_argument("--order", type=int, default=0)
    ap.add_argument("--tile-bytes", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--lag", type=int, default=0)
    ap.add_argument("--max-ctas", type=int, default=0)
    ap.add_argument("--pool-blocks", type=int, default=0,
                    help="override the workload's pool size (small cases for profiler captures)")
    ap.add_argument("--request-blocks", type=int, default=0,
                    help="override the workload's request length in blocks")
    ap.add_argument("--ring-slots", type=int, default=8)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap", action="store_true",
                    help="skip the brief ring-streaming-beside-a-GEMM measurement after the timed region")
    ap.add_argument("--suite", default="",
                    help="run the other configs instead of the bench step: all, or a comma list of "
                         "host_link,launch_shapes,chunk_sweep,small_slabs,row_gather,call_overhead,prefix_8k,batch_70b,"
                         "ring_overlap,duplex,file_pipeline,preload_trace,pipeline_beside_gemm (1 GPU; prints "
                         "one JSON line)")
    ap.add_argument("--small-slab-sizes", default="",
                    help="small_slabs suite part: comma list of slab sizes in bytes (default: all)")
    ap.add_argument("--small-slab-mib", type=int, default=2048,
                    help="small_slabs suite part: request size in MiB (small cases for profiler captures)")
    ap.add_argument("--overlap-seconds", type=float, default=2.0)
    ap.add_argument("--file-roots", default="/tmp,/dev/shm",
                    help="comma list of directories for the file_pipeline suite part")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch from an ncu capture, copied into the roofline object "
                         "(default: the committed capture of the default workload, else null)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.suite:
        run_suite(args)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
