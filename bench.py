#!/usr/bin/env python
"""Benchmark of the demand-paging hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload CFG] [--shrink S]
                    [--impl ours|reference] [--uvm] [--no-cpu-baseline]

One step = one cold pass of the whole path over one workload: reset the page table, run the
workload kernel(s) (translation, fault coalescing, frame claim, eviction, write-back,
migration, the application arithmetic), flush dirty pages.  The default workload is the
random gather (configuration 2: 1 GiB fp32 array, 2^26 uniform indices, 64 KiB pages,
256 MiB pool); --workload 1..5 selects another configuration.

Rank 0 prints ONE JSON line.  `value` is the effective application GB/s (useful payload
bytes / CUDA-event time) with all inputs resident (paged array in pinned host memory, which
is where the method keeps it; indices in device memory).  `migration` holds page-migration
GB/s and faults/s, absolute and against the host-link peak measured in the same run.  `e2e`
is the same metric with the step's device-side operands copied from pinned host memory and
the results copied back inside the timed region.  With --gpus N>1 (under torchrun) every
rank runs an independent replica on its own GPU: the path has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "effective_app_GBps"
UNIT = "GB/s"


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML in a background thread while the timed
    region runs (falls back to one nvidia-smi query before and after when NVML is unavailable)."""

    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, index: int, period_s: float = 0.5):
        self.index, self.period = index, period_s
        self.sm, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None

    def _handle(self):
        import pynvml
        pynvml.nvmlInit()
        self._nvml = pynvml
        visible = os.environ.get("CUDA_VISIBLE_DEVICES")
        if visible and not visible.replace(",", "").isdigit():
            return pynvml.nvmlDeviceGetHandleByUUID(visible.split(",")[self.index].encode())
        phys = int(visible.split(",")[self.index]) if visible else self.index
        return pynvml.nvmlDeviceGetHandleByIndex(phys)

    def _sample(self, h):
        nv = self._nvml
        self.sm.append(float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
        mask = nv.nvmlDeviceGetCurrentClocksEventReasons(h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
            else nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
        for name, bit in self.REASONS:
            if mask & bit:
                self.reasons.add(name)

    def _run(self, h):
        while not self._stop.is_set():
            try:
                self._sample(h)
            except Exception:
                break
            self._stop.wait(self.period)

    def start(self):
        try:
            h = self._handle()
            self.max_mhz = float(self._nvml.nvmlDeviceGetMaxClockInfo(h, self._nvml.NVML_CLOCK_SM))
            self._sample(h)
            self._thread = threading.Thread(target=self._run, args=(h,), daemon=True)
            self._thread.start()
        except Exception:
            self._nvml = None
            self._smi()

    def _smi(self):
        try:
            out = subprocess.run(["nvidia-smi", f"--id={self.index}", "--query-gpu=clocks.sm,clocks.max.sm",
                                  "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=20).stdout
            a, b = [float(x) for x in out.strip().split(",")[:2]]
            self.sm.append(a)
            self.max_mhz = b
        except Exception:
            pass

    def stop(self) -> dict:
        if self._thread is not None:
            self._stop.set()
            self._thread.join(timeout=5)
        elif self._nvml is None:
            self._smi()
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "samples": len(self.sm), "reasons": sorted(self.reasons),
                "source": "nvml" if self._nvml is not None else "nvidia-smi"}


# ------------------------------------------------------------------------- link peaks

# Host-link bytes per launch that ncu counted for the full-size workloads that have a committed
# capture under profiles/ (stream_sum_kernel cfg 1: 2 097 152 sectors; gather_batch_kernel cfg 2:
# 33 554 432 sectors of 32 bytes).
NCU_LINK_BYTES = {1: 2097152 * 32, 2: 33554432 * 32}


def measure_link(torch, B, nbytes=1 << 30, reps=5) -> dict:
    """Pinned-copy peak (copy engine) and SM-issued load/store peak of the host link."""
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    devb = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    out = {}
    for name, (dst, src) in {"ce_h2d_gbs": (devb, host), "ce_d2h_gbs": (host, devb)}.items():
        best = 0.0
        for r in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            dst.copy_(src, non_blocking=True)
            e1.record()
            e1.synchronize()
            if r:
                best = max(best, nbytes / (e0.elapsed_time(e1) * 1e6))
        out[name] = best
    sm = B.gpuvm_link_peak(host.data_ptr(), devb.data_ptr(), nbytes, 3)
    out.update({"sm_h2d_gbs": sm["h2d_gbs"], "sm_d2h_gbs": sm["d2h_gbs"], "sm_duplex_gbs": sm["duplex_gbs"]})
    del host, devb
    torch.cuda.empty_cache()
    return out


def measured_peaks() -> dict:
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except OSError:
        return {}


# ------------------------------------------------------------------- CPU oracle timing

def oracle_step(cfg: int, w=None, shrink: int = 0):
    """Time the CPU oracle (as it stands, one thread) on a bounded sample of the workload.
    Returns (effective bytes, seconds, description of the sample)."""
    import numpy as np
    import oracle
    from paper_2411_05309_b200 import inputs
    if cfg == 2:
        n, n_idx = (1 << 28) >> shrink, (1 << 26) >> shrink
        if w is not None:
            x, idx = w.view("x", np.float32, w.n), w.idx_host.numpy()
        else:
            x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(2))
            idx = inputs.fill_index_i64(np.empty(n_idx, np.int64), n_idx, inputs.config_seed(2, 1), n)
        t0 = time.perf_counter()
        oracle.gather_block_sums_direct(x, idx, 1024)
        pg = oracle.Pager(x.view(np.uint8), 64 << 10, max(1, (4096 >> shrink)), oracle.CLOCK, False)
        sample = idx[: max(1, idx.size // 4)]
        pg.gather_block_sums(0, sample, 1024)
        dt = time.perf_counter() - t0
        pg.close()
        return 4 * idx.size, dt, (f"direct results for all {idx.size} indices + sequential paging replay of the first "
                                  f"{sample.size} (no byte movement)")
    if cfg == 1:
        n = (1 << 24) >> shrink
        a = w.view("a", np.int32, w.n) if w is not None else inputs.fill_i32_u20(np.empty(n, np.int32), n, inputs.config_seed(1))
        t0 = time.perf_counter()
        for _ in range(8):
            oracle.stream_sum_i32_direct(a)
        return 8 * 4 * a.size, time.perf_counter() - t0, "8 direct passes over the whole array"
    if cfg == 4:
        n = min((1 << 30) >> shrink, 1 << 27)
        a = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4))
        b = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4, 1))
        t0 = time.perf_counter()
        oracle.vadd_f32_direct(a, b)
        return 12 * n, time.perf_counter() - t0, f"direct vector add of the first {n} elements"
    if cfg in (3, 8):
        scale = min(24 - shrink, 22)
        off, col = inputs.rmat_csr(scale, 16 << scale, inputs.config_seed(3))
        t0 = time.perf_counter()
        lvl = oracle.bfs_levels_direct(off, col, 0)
        dt = time.perf_counter() - t0
        deg = np.diff(off)
        vis = lvl >= 0
        return int(16 * vis.sum() + 4 * deg[vis].sum()), dt, f"direct BFS on an RMAT graph of scale {scale}"
    if cfg in (6, 7):
        scale = min(24 - shrink, 22)
        off, col = inputs.rmat_csr(scale, 16 << scale, inputs.config_seed(3))
        if cfg == 6:
            t0 = time.perf_counter()
            oracle.cc_labels_direct(off, col)
            return 8 * off.size + 4 * col.size, time.perf_counter() - t0, f"union-find over an RMAT graph of scale {scale} (one pass over the edges)"
        w = inputs.fill_i32_range(np.empty(col.size, np.int32), col.size, inputs.config_seed(3, 2), 1, 255)
        t0 = time.perf_counter()
        d = oracle.sssp_direct(off, col, w, 0)
        dt = time.perf_counter() - t0
        reached = d != 0x7FFFFFFF
        return int(16 * reached.sum() + 8 * np.diff(off)[reached].sum()), dt, f"Dijkstra on an RMAT graph of scale {scale}"
    if cfg == 5:
        rows_n, dims, bag = 1 << 20, 128, 32
        t = inputs.fill_f32_pm1(np.empty(rows_n * dims, np.float32), rows_n * dims, inputs.config_seed(5)).reshape(rows_n, dims)
        n_lookups = 1 << 21
        rows = inputs.fill_zipf_rows(np.empty(n_lookups, np.int64), n_lookups, inputs.config_seed(5, 1), rows_n, 1.05)
        t0 = time.perf_counter()
        oracle.embag_f32_direct(t, rows, bag)
        return 4 * dims * n_lookups, time.perf_counter() - t0, f"{n_lookups} lookups into a {rows_n}-row table"
    raise ValueError(cfg)


def run_reference(args, rank: int):
    """The reference arm of this benchmark is the CPU oracle timed on the host cores."""
    if rank != 0:
        return
    times, nbytes, sample = [], 0, ""
    for i in range(args.warmup + args.steps):
        nbytes, dt, sample = oracle_step(args.workload, None, args.shrink)
        if i >= args.warmup:
            times.append(dt)
    t = sum(times) / len(times)
    value = nbytes / t / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": DTYPES[args.workload], "data": "synthetic",
            "config": {"workload": NAMES[args.workload], "shrink": args.shrink},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


NAMES = {1: "cfg1 streaming read-reduce: int64 sum over 64 MiB int32, 4 KiB pages, 16 MiB pool",
         2: "cfg2 random gather: 1 GiB fp32 array, 2^26 uniform int64 indices, sum per 1024, 64 KiB pages, 256 MiB pool",
         3: "cfg3 BFS on RMAT scale 24 (avg degree 16), CSR paged at 64 KiB, pool = half",
         4: "cfg4 vector add c=a+b over three 4 GiB fp32 arrays, 64 KiB pages, 4 GiB pool",
         5: "cfg5 Zipf(1.05) embedding bag: 64 GiB table, 2^24 lookups, bags of 32, 2 MiB pages, 16 GiB pool",
         6: "connected components on the cfg3 graph (RMAT scale 24), CSR paged at 64 KiB, pool = half",
         7: "SSSP from vertex 0 on the cfg3 graph with int32 weights in a third paged array, 64 KiB pages, pool = half",
         8: "BFS on the cfg3 graph stored as Balanced CSR (chunks of 16 Ki edges), 64 KiB pages, pool = half"}
DTYPES = {1: "int64", 2: "f32", 3: "int32", 4: "f32", 5: "f32", 6: "int32", 7: "int32", 8: "int32"}


# ---------------------------------------------------------------------- rank plumbing

def max_over_ranks(dist, values, device="cpu"):
    """Element-wise maximum of `values` over all ranks (the slowest rank sets the time)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return list(values)
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def replica_throughput(world: int, units_per_rank: float, slowest_seconds: float) -> float:
    """Whole-job throughput of `world` independent replicas: all units over the slowest time."""
    return world * units_per_rank / slowest_seconds


# ------------------------------------------------------------------------------- ours

def e2e_step(torch, B, w, cfg: int):
    """One step through the C ABI with the step's device operands coming from pinned host
    memory and the results going back to the host, all inside the timed region."""
    stream = torch.cuda.current_stream()
    h2d = d2h = 0
    B.gpuvm_reset(w.h)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    if cfg == 2:
        w.d_idx.copy_(w.idx_host, non_blocking=True)
        h2d = w.idx_host.numel() * 8
    elif cfg == 5:
        w.d_rows.copy_(w.rows_host, non_blocking=True)
        h2d = w.rows_host.numel() * 8
    w.launch(stream)
    B.gpuvm_flush(w.h, stream)
    outs = {1: ["d_sum"], 2: ["d_fsum", "d_bsum"], 3: ["d_level"], 4: [], 5: ["d_out"], 6: ["d_level"], 7: ["d_dist"], 8: ["d_level"]}[cfg]
    for name in outs:
        t = getattr(w, name)
        buf = w.__dict__.setdefault("_host_" + name, torch.empty(t.shape, dtype=t.dtype).pin_memory())
        buf.copy_(t, non_blocking=True)
        d2h += t.numel() * t.element_size()
    e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1) / 1e3, h2d, d2h


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the paged path has no CPU fallback")
    local_rank %= max(1, torch.cuda.device_count())
    torch.cuda.set_device(local_rank)
    from paper_2411_05309_b200 import binding as B
    from paper_2411_05309_b200 import configs
    B.lib()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    link = measure_link(torch, B)
    w = configs.make(args.workload, args.shrink)
    if args.scratch_limit_mib:
        B.gpuvm_set_scratch_limit(w.h, args.scratch_limit_mib << 20)
    for _ in range(args.warmup):
        w.run(check=False)
    sampler = ClockSampler(local_rank, args.clock_period)
    launches0 = B.gpuvm_launch_count()
    barrier()
    sampler.start()
    t_wall0 = time.perf_counter()
    results = [w.run(check=True) for _ in range(args.steps)]
    barrier()
    wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    launches = B.gpuvm_launch_count() - launches0
    e2e_step(torch, B, w, args.workload)                       # untimed: allocates the pinned result buffers
    e2e = [e2e_step(torch, B, w, args.workload) for _ in range(max(1, min(args.steps, 3)))]

    step_s = sum(r.seconds for r in results) / len(results)
    kern_s = sum(r.kernel_seconds for r in results) / len(results)
    e2e_s = sum(t for t, _, _ in e2e) / len(e2e)
    step_s, kern_s, e2e_s = max_over_ranks(dist, [step_s, kern_s, e2e_s], "cuda")
    eff_bytes = results[-1].effective_bytes
    st = results[-1].stats
    ck = results[-1].check
    bytes_in = sum(r.stats["bytes_in"] for r in results) / len(results)
    bytes_out = sum(r.stats["bytes_out"] for r in results) / len(results)
    faults = sum(r.stats["faults"] for r in results) / len(results)
    peaks = measured_peaks()
    hbm_peak = peaks.get("hbm_gbs", 6650.0)
    link_peak = link["ce_h2d_gbs"] if bytes_out == 0 else link["ce_h2d_gbs"] + link["ce_d2h_gbs"]
    moved = bytes_in + bytes_out

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        w.close()
        return

    line = {
        "metric": METRIC, "value": replica_throughput(world, eff_bytes, step_s) / 1e9, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPES[args.workload], "data": "synthetic",
        "config": {**w.describe(), "workload": NAMES[args.workload], "replicas": world,
                   "cache_state": "cold every step: page table reset, paged array (>= 8x L2 at full size) re-read "
                                  "from host memory; nothing of a previous step stays resident"},
        "migration": {
            "in_gbs": bytes_in / step_s / 1e9, "out_gbs": bytes_out / step_s / 1e9,
            "faults_per_s": faults / step_s, "faults": faults, "bytes_in": bytes_in, "bytes_out": bytes_out,
            "io_amplification": bytes_in / eff_bytes if eff_bytes else None,
            "frac_of_pinned_copy_peak": (moved / step_s / 1e9) / link_peak,
            "frac_of_sm_link_peak": (bytes_in / step_s / 1e9) / link["sm_h2d_gbs"] if link["sm_h2d_gbs"] else None,
            "fault_rate_ceiling_per_s": link["ce_h2d_gbs"] * 1e9 / w.page_bytes,
        },
        "link_peak": link,
        "scratch": {"bytes": B.gpuvm_scratch_bytes(w.h), "limit_bytes": args.scratch_limit_mib << 20,
                    "what": "device memory of the workload beside the pool: request tables, staged rows, queues"},
        "stats": st, "invariants": ck,
        "roofline": {
            "bound": "host_link", "achieved": moved / kern_s / 1e9, "peak": link_peak, "unit": "GB/s",
            "frac": (moved / kern_s / 1e9) / link_peak,
            "peak_source": "pinned cudaMemcpy measured in this run (H2D; H2D + D2H when pages are written back)",
            "traffic": NCU_LINK_BYTES.get(args.workload) if args.shrink == 0 and not args.scratch_limit_mib else None,
            "traffic_source": "host-link bytes of one launch counted by ncu (sysmem read sector misses x 32 B) in the "
                              "committed capture of this kernel at this size; equals the kernel's own bytes_in counter. "
                              "DRAM traffic is not the bound on this path (9.4 % of DRAM peak in the capture of cfg 2)",
            "hbm": {"achieved": (bytes_in + bytes_out + eff_bytes) / kern_s / 1e9, "peak": hbm_peak,
                    "frac": ((bytes_in + bytes_out + eff_bytes) / kern_s / 1e9) / hbm_peak,
                    "peak_source": "MEASURED_PEAKS.json" if peaks else "fallback"},
            "kernel_ms": kern_s * 1e3,
        },
        "e2e": {"value": replica_throughput(world, eff_bytes, e2e_s) / 1e9, "unit": UNIT, "h2d_bytes_per_step": e2e[-1][1],
                "d2h_bytes_per_step": e2e[-1][2], "ms_per_step": e2e_s * 1e3},
        "gpu_launches": launches, "clocks": clocks, "wall_s": wall,
        "step_ms": [r.seconds * 1e3 for r in results],
        "ms_median": statistics.median(r.seconds for r in results) * 1e3, "ms_min": min(r.seconds for r in results) * 1e3,
    }
    if args.workload == 2 and not args.scratch_limit_mib:
        # the same workload with request tables bounded to 80 MiB (4096 requests per warp in flight instead
        # of all 16 384 read from the index list in place): every page fetched about once per quarter of the list
        quarter = max(1, (80 << 20) >> args.shrink)
        B.gpuvm_set_scratch_limit(w.h, quarter)
        w.run(check=False)
        r = w.run(check=True)
        B.gpuvm_set_scratch_limit(w.h, 0)
        line["scratch"]["with_a_quarter_of_the_requests_in_flight"] = {
            "limit_bytes": quarter, "ms_per_step": r.seconds * 1e3, "value": r.effective_bytes / r.seconds / 1e9,
            "faults": r.stats["faults"], "in_gbs": r.stats["bytes_in"] / r.seconds / 1e9}
    if not args.no_cpu_baseline:
        nbytes, dt, sample = oracle_step(args.workload, w if args.workload in (1, 2) else None, args.shrink)
        line["cpu_baseline"] = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": sample, "seconds": dt}
    if args.uvm:
        from paper_2411_05309_b200 import uvm
        w.close()
        line["uvm"] = uvm.run_twin(args.workload, args.shrink, timeout_s=args.uvm_timeout)
    w.close()
    if dist is not None:
        dist.destroy_process_group()
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4, 5, 6, 7, 8])
    ap.add_argument("--shrink", type=int, default=0, help="divide all sizes by 2**shrink")
    ap.add_argument("--uvm", action="store_true", help="also run the workload over cudaMallocManaged")
    ap.add_argument("--uvm-timeout", type=float, default=120.0)
    ap.add_argument("--scratch-limit-mib", type=int, default=0,
                    help="bound of the workload's device scratch (request tables, staged rows); 0 = none. Less scratch "
                         "means fewer page requests in flight per warp and more faults")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--clock-period", type=float, default=0.1, help="seconds between NVML clock samples")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
