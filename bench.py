#!/usr/bin/env python
"""Benchmark of the demand-paging hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload CFG | --configs 1,2,3,4,5]
                    [--shrink S] [--impl ours|reference] [--no-uvm] [--no-cpu-baseline] [--no-replay]

One step = one cold pass of the whole path over one workload: reset the page table, run the
workload kernel(s) (translation, fault coalescing, frame claim, eviction, write-back,
migration, the application arithmetic), flush dirty pages.

With no --workload all five configurations are run, the largest one last: configuration 5
(Zipf embedding bag: 64 GiB table, 2 MiB pages, 16 GiB pool) is the headline record, timed
for exactly K steps after W warm-up steps, and `per_config` carries the same fields for each of
the five (configurations 1-4 with min(K, 10) steps after min(W, 3)).  --workload N runs one
workload (1-5 the configurations, 6 CC, 7 SSSP, 8 and 9 BFS and CC over Balanced CSR) as the headline.

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

DEFAULT_INPLACE_DIVISOR = 0xFFFFFFFF  # GPUVM_INPLACE_AUTO, the library's default (include/gpuvm.h, gpuvm_set_inplace_divisor)
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

# Host-link bytes of one launch of each configuration's dominant kernel as ncu counted them (sysmem read
# sector misses x 32 B inbound; for the written workload also the outbound payload) in the capture
# committed under profiles/.  Where the capture was taken on a reduced case the figure is scaled to the full
# launch by the pages moved (every page crosses the link once in these launches, so traffic grows in
# proportion).  cfg -> (bytes per launch at full size, file under profiles/, the count in that file, how scaled)
NCU_LINK_TRAFFIC = {
    1: (2097152 * 32, "stream_sum_kernel_cfg1_full_set.md", 2097152, "full size"),
    2: (33554432 * 32, "gather_batch_kernel_cfg2_full_set.md", 33554432, "full size"),
    3: (38354055 * 32, "graph_sweep_kernel_lc_cfg3_sweep1_full_set.md", 38354055,
        "full size; sweep 1 of the four sweeps of a run, 95 % of its time"),
    4: (33554432 * 32 * 8 + (4 << 30), "vadd_kernel_cfg4_eighth_full_set.md", 33554432,
        "1/8 case x 8: 8 GiB in, plus the 4 GiB of c that go out"),
    5: (60863056 * 32, "embag_direct_kernel_cfg5_default_policy.md", 60863056,
        "full size, default policy; one metric, one pass"),
    "5_always_migrate": (134217728 * 32 * 16, "embag_batch_kernel_cfg5_sixteenth_full_set.md", 134217728,
                         "1/16 case x 16, every first touch fetching its page"),
    6: (37758976 * 32, "graph_sweep_kernel_cc_cfg6_full_set.md", 37758976, "full size"),
}


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


def link_roofline(bytes_in: float, bytes_out: float, kernel_s: float, link: dict) -> dict:
    """The two directions of the link work at the same time, so the floor of a launch is the slower
    of (bytes in / inbound peak) and (bytes out / outbound peak); the fraction is that floor over
    the measured kernel time, i.e. achieved / peak in the direction that bounds the launch."""
    t_in = bytes_in / (link["ce_h2d_gbs"] * 1e9)
    t_out = bytes_out / (link["ce_d2h_gbs"] * 1e9)
    inbound = t_in >= t_out
    moved, peak = (bytes_in, link["ce_h2d_gbs"]) if inbound else (bytes_out, link["ce_d2h_gbs"])
    achieved = moved / kernel_s / 1e9 if kernel_s else 0.0
    return {"bound": "host_link", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "direction": "host_to_device" if inbound else "device_to_host",
            "floor_ms": max(t_in, t_out) * 1e3, "kernel_ms": kernel_s * 1e3,
            "other_direction_gbs": (bytes_out if inbound else bytes_in) / kernel_s / 1e9 if kernel_s else 0.0,
            "peak_source": "pinned cudaMemcpy measured in this run, in the direction that bounds the launch "
                           "(floor = max(bytes in / H2D peak, bytes out / D2H peak))",
            "frac_of_sm_issued_peak": achieved / (link["sm_h2d_gbs"] if inbound else link["sm_d2h_gbs"])}


# ------------------------------------------------------------------- CPU oracle timing

def _best_of(fn, reps=2):
    best = None
    for _ in range(reps):
        t0 = time.perf_counter()
        fn()
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best


def oracle_sample(cfg: int, w=None, shrink: int = 0):
    """The bounded sample of workload `cfg` that the CPU oracle is timed on.
    Returns (effective bytes of the sample, description, fn(impl) that runs it with `impl` = the oracle
    module or its all-core build, whether an all-core form exists)."""
    import numpy as np
    from paper_2411_05309_b200 import inputs
    if cfg == 1:
        n = (1 << 24) >> shrink
        a = w.view("a", np.int32, w.n) if w is not None else inputs.fill_i32_u20(np.empty(n, np.int32), n, inputs.config_seed(1))
        return 8 * 4 * a.size, "8 direct passes over the whole array", \
            (lambda impl: [impl.stream_sum_i32_direct(a) for _ in range(8)]), True
    if cfg == 2:
        n, n_idx = (1 << 28) >> shrink, (1 << 26) >> shrink
        if w is not None:
            x, idx = w.view("x", np.float32, w.n), w.idx_host.numpy()
        else:
            x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(2))
            idx = inputs.fill_index_i64(np.empty(n_idx, np.int64), n_idx, inputs.config_seed(2, 1), n)
        return 4 * idx.size, f"direct block sums for all {idx.size} indices", \
            (lambda impl: impl.gather_block_sums_direct(x, idx, 1024)), True
    if cfg == 4:
        n = min((1 << 30) >> shrink, 1 << 27)
        a = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4))
        b = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4, 1))
        return 12 * n, f"direct vector add of the first {n} elements", (lambda impl: impl.vadd_f32_direct(a, b)), True
    if cfg in (3, 8, 6, 7, 9):
        scale = min(24 - shrink, 22)
        off, col = inputs.rmat_csr(scale, 16 << scale, inputs.config_seed(3))
        import oracle
        if cfg in (3, 8):
            lvl = oracle.bfs_levels_direct(off, col, 0)
            vis = lvl >= 0
            nbytes = int(16 * vis.sum() + 4 * np.diff(off)[vis].sum())
            return nbytes, f"queue BFS on an RMAT graph of scale {scale} (sequential by nature: one thread)", \
                (lambda impl: impl.bfs_levels_direct(off, col, 0)), False
        if cfg in (6, 9):
            return 8 * off.size + 4 * col.size, f"union-find over an RMAT graph of scale {scale} (one pass over the edges)", \
                (lambda impl: impl.cc_labels_direct(off, col)), False
        wt = inputs.fill_i32_range(np.empty(col.size, np.int32), col.size, inputs.config_seed(3, 2), 1, 255)
        d = oracle.sssp_direct(off, col, wt, 0)
        reached = d != 0x7FFFFFFF
        return int(16 * reached.sum() + 8 * np.diff(off)[reached].sum()), f"Dijkstra on an RMAT graph of scale {scale}", \
            (lambda impl: impl.sssp_direct(off, col, wt, 0)), False
    if cfg == 5:
        rows_n, dims, bag = 1 << 25, 128, 32          # a 16 GiB table: far beyond the last-level cache, like the workload's
        t = inputs.fill_f32_pm1(np.empty(rows_n * dims, np.float32), rows_n * dims, inputs.config_seed(5)).reshape(rows_n, dims)
        n_lookups = 1 << 22
        rows = inputs.fill_zipf_rows(np.empty(n_lookups, np.int64), n_lookups, inputs.config_seed(5, 1), rows_n, 1.05)
        return 4 * dims * n_lookups, f"{n_lookups} Zipf lookups (bags of {bag}) into a {rows_n}-row table", \
            (lambda impl: impl.embag_f32_direct(t, rows, bag)), True
    raise ValueError(cfg)


def cpu_baseline(cfg: int, w=None, shrink: int = 0) -> dict:
    """The CPU oracle as it stands, timed on a bounded sample of the workload: on one thread and,
    where its outer loop splits over threads, on all host cores (the OpenMP build of the same file)."""
    import oracle
    nbytes, sample, run, splits = oracle_sample(cfg, w, shrink)
    dt1 = _best_of(lambda: run(oracle))
    out = {"value": nbytes / dt1 / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample, "seconds": dt1,
           "host_cores": os.cpu_count()}
    if splits:
        par = oracle.AllCores()
        dtn = _best_of(lambda: run(par))
        out["one_thread"] = {"value": out["value"], "seconds": dt1}
        out.update({"value": nbytes / dtn / 1e9, "cores": par.threads, "seconds": dtn,
                    "kind": "oracle (same source built with OpenMP: outer loop split over threads)"})
    return out


def replay_counts(cfg: int, w) -> dict:
    """Fault counts of the workload's canonical (sequential) page trace through the oracle's replay:
    clock, FIFO and Belady's optimum with the configuration's number of frames.  For the order-dependent
    GPU fault counts these say what a one-request-at-a-time pager would take."""
    import numpy as np
    import oracle
    t0 = time.perf_counter()
    if cfg == 3:
        pg = oracle.Pager(w.host, w.page_bytes, w.n_frames, oracle.CLOCK, False)
        pg.record_trace(1 << 28)
        pg.bfs_levels(w.off["off"], w.off["col"], w.nv, 0)
        trace = pg.trace().copy()
        pg.close()
        what = "level by level, vertices ascending, both row offsets then the edge range of each vertex"
    elif cfg == 5:
        rows = w.rows_host.numpy()
        trace = ((w.off["t"] + rows.astype(np.uint64) * np.uint64(4 * w.dims)) >> np.uint64(21)).astype(np.uint64)
        keep = np.concatenate([[True], trace[1:] != trace[:-1]])
        trace = np.ascontiguousarray(trace[keep])
        what = "lookups in list order, one page per row"
    else:
        return {}
    out = oracle.replay_counts(trace, w.n_pages, w.page_bytes, w.n_frames)
    out.update({"trace_records": int(trace.size), "order": what, "frames": w.n_frames, "seconds": time.perf_counter() - t0})
    return out


NAMES = {1: "cfg1 streaming read-reduce: int64 sum over 64 MiB int32, 4 KiB pages, 16 MiB pool",
         2: "cfg2 random gather: 1 GiB fp32 array, 2^26 uniform int64 indices, sum per 1024, 64 KiB pages, 256 MiB pool",
         3: "cfg3 BFS on RMAT scale 24 (avg degree 16), CSR paged at 64 KiB, pool = half",
         4: "cfg4 vector add c=a+b over three 4 GiB fp32 arrays, 64 KiB pages, 4 GiB pool",
         5: "cfg5 Zipf(1.05) embedding bag: 64 GiB table, 2^24 lookups, bags of 32, 2 MiB pages, 16 GiB pool",
         6: "connected components on the cfg3 graph (RMAT scale 24), CSR paged at 64 KiB, pool = half",
         7: "SSSP from vertex 0 on the cfg3 graph with int32 weights in a third paged array, 64 KiB pages, pool = half",
         8: "BFS on the cfg3 graph stored as Balanced CSR (chunks of 16 Ki edges), 64 KiB pages, pool = half",
         9: "connected components on the cfg3 graph stored as Balanced CSR, 64 KiB pages, pool = half"}
DTYPES = {1: "int64", 2: "f32", 3: "int32", 4: "f32", 5: "f32", 6: "int32", 7: "int32", 8: "int32", 9: "int32"}


def config_of(cfg: int, shrink: int) -> dict:
    """`config` of the JSON line: the same keys from both arms."""
    from paper_2411_05309_b200 import configs
    d = configs.describe(cfg, shrink)
    d["kernel"] = d["workload"]
    d["workload"] = NAMES[cfg]
    return d


def headline_of(args, world: int) -> int:
    """The workload the top-level record is quoted on: the one asked for, else the largest configuration
    (5) when its 64 GiB pinned table fits the host once per rank, else the next largest."""
    if args.workload:
        return args.workload
    order = [int(c) for c in args.configs.split(",")]
    try:
        import psutil
        ram = psutil.virtual_memory().total
    except Exception:
        ram = 1 << 62
    from paper_2411_05309_b200 import configs
    by_size = sorted(order, key=lambda c: configs.describe(c, args.shrink)["paged_bytes"], reverse=True)
    for c in by_size:
        if world * configs.describe(c, args.shrink)["paged_bytes"] <= 0.6 * ram:
            return c
    return by_size[-1]


def run_reference(args, rank: int, world: int):
    """The reference arm of this benchmark is the CPU oracle timed on the host cores."""
    if rank != 0:
        return
    import oracle
    cfg = headline_of(args, world)
    nbytes, sample, run, splits = oracle_sample(cfg, None, args.shrink)
    impl = oracle.AllCores() if splits else oracle
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        run(impl)
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    t = sum(times) / len(times)
    value = nbytes / t / 1e9
    cores = impl.threads if splits else 1
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": DTYPES[cfg], "data": "synthetic",
            "config": config_of(cfg, args.shrink),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "host_cores": os.cpu_count()},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


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

OUTPUTS = {1: ["d_sum"], 2: ["d_fsum", "d_bsum"], 3: ["d_level"], 4: [], 5: ["d_out"], 6: ["d_level"], 7: ["d_dist"],
           8: ["d_level"], 9: ["d_level"]}


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
    for name in OUTPUTS[cfg]:
        t = getattr(w, name)
        key = "_host_" + name
        if key not in w.__dict__:                           # (allocated by the untimed first call)
            w.__dict__[key] = torch.empty(t.shape, dtype=t.dtype).pin_memory()
        w.__dict__[key].copy_(t, non_blocking=True)
        d2h += t.numel() * t.element_size()
    e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1) / 1e3, h2d, d2h


def embag_policy_records(torch, B, w, args, link: dict, kern_s: float, direct: float, rec: dict) -> dict:
    """cfg 5 runs with the library's default: lookups are counted per page first, the rows of pages with fewer
    lookups than rows are read in place, page by page, the other pages are fetched once.  Reported beside it: the
    ceiling of scattered row reads over this backing store, measured here; the same policy with the rows read as
    their lookups come up (scattered: that ceiling bounds it); the online form (no count beforehand); and the same
    launch with the policy off (the paper's way: every first touch fetches the page), each with its own link
    roofline."""
    out = {}
    row_bytes = 4 * w.dims
    buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    scattered = B.gpuvm_link_peak_scattered(B.gpuvm_host_ptr(w.h), w.nbytes, row_bytes, 1 << 22, buf.data_ptr(), buf.numel())
    grouped = B.gpuvm_link_peak_scattered(B.gpuvm_host_ptr(w.h), w.nbytes, row_bytes, 1 << 22, buf.data_ptr(), buf.numel(), 2, 64)
    del buf
    out["in_place"] = {
        "bytes": direct, "gbs": direct / kern_s / 1e9 if kern_s else 0.0, "scattered_read_peak_gbs": scattered,
        "grouped_read_peak_gbs": grouped,
        "what": f"rows read in place from the backing store, page by page (bucketed by page first); "
                f"scattered_read_peak_gbs is what {1 << 22} rows of {row_bytes} B at hashed positions of the same "
                f"{w.nbytes >> 30} GiB region reach, four in flight per warp, measured in this run: the ceiling of "
                f"reading them as their lookups come up (roofline.counted_scattered); grouped_read_peak_gbs is the same "
                f"with 64 consecutive rows in the same 2 MiB of the region"}
    if args.inplace_divisor < 0 and not args.scratch_limit_mib:
        def other_policy(what, setup, restore):
            setup()
            try:
                w.run(check=False)
                rs = [w.run(check=True) for _ in range(2)]
            finally:
                restore()
            secs = sum(r.seconds for r in rs) / len(rs)
            ks = sum(r.kernel_seconds for r in rs) / len(rs)
            st = rs[-1].stats
            roof = link_roofline(st["bytes_in"] + st.get("bytes_direct", 0), st["bytes_out"], ks, link)
            return {"what": what, "ms_per_step": secs * 1e3, "value": rs[-1].effective_bytes / secs / 1e9, "unit": UNIT,
                    "steps": len(rs), "faults": st["faults"], "bytes_in": st["bytes_in"],
                    "bytes_direct": st.get("bytes_direct", 0), "in_gbs": st["bytes_in"] / secs / 1e9,
                    "invariants_status": rs[-1].check["status"], "roofline": roof}

        out["counted_scattered"] = other_policy(
            "gpuvm_set_inplace_counted(h, 1): lookups counted per page first, rows of pages with fewer lookups than a "
            "quarter of their rows read in place as their lookups come up (scattered over the table)",
            lambda: B.gpuvm_set_inplace_counted(w.h, 1), lambda: B.gpuvm_set_inplace_counted(w.h, 2))
        out["online"] = other_policy(
            "gpuvm_set_inplace_counted(h, 0): no count beforehand; the first requests that find a page absent read "
            "their rows in place, the one after them fetches the page",
            lambda: B.gpuvm_set_inplace_counted(w.h, 0), lambda: B.gpuvm_set_inplace_counted(w.h, 2))
        rec_am = other_policy(
            "gpuvm_set_inplace_divisor(h, 0): every first touch fetches the page, as in the paper",
            lambda: B.gpuvm_set_inplace_divisor(w.h, 0), lambda: B.gpuvm_set_inplace_divisor(w.h, DEFAULT_INPLACE_DIVISOR))
        traffic = NCU_LINK_TRAFFIC.get("5_always_migrate") if args.shrink == 0 else None
        rec_am["roofline"]["traffic"] = traffic[0] if traffic else None
        rec_am["roofline"]["traffic_source"] = (f"profiles/{traffic[1]} ({traffic[3]}): host-link bytes of one launch "
                                                "counted by ncu" if traffic else None)
        out["always_migrate"] = rec_am
    return out


def run_config(torch, B, configs, cfg: int, args, steps: int, warmup: int, link: dict, dist, world: int,
               local_rank: int, rank: int, barrier) -> dict:
    """All measurements of one workload: K timed cold steps, the end-to-end steps, the run under a
    scratch bound (cfg 2 and 5), and on rank 0 the CPU baseline, the oracle's replay counts and the same
    kernels over managed memory."""
    w = configs.make(cfg, args.shrink)
    try:
        if args.scratch_limit_mib:
            B.gpuvm_set_scratch_limit(w.h, args.scratch_limit_mib << 20)
        if args.inplace_divisor >= 0:
            B.gpuvm_set_inplace_divisor(w.h, args.inplace_divisor)
        for _ in range(warmup):
            w.run(check=False)
        sampler = ClockSampler(local_rank, args.clock_period)
        launches0 = B.gpuvm_launch_count()
        barrier()
        sampler.start()
        t_wall0 = time.perf_counter()
        results = [w.run(check=True) for _ in range(steps)]
        barrier()
        wall = time.perf_counter() - t_wall0
        clocks = sampler.stop()
        launches = B.gpuvm_launch_count() - launches0
        e2e_step(torch, B, w, cfg)                                # untimed: allocates the pinned result buffers
        e2e = [e2e_step(torch, B, w, cfg) for _ in range(max(1, min(steps, 3)))]

        step_s = sum(r.seconds for r in results) / len(results)
        kern_s = sum(r.kernel_seconds for r in results) / len(results)
        e2e_s = sum(t for t, _, _ in e2e) / len(e2e)
        step_s, kern_s, e2e_s = max_over_ranks(dist, [step_s, kern_s, e2e_s], "cuda")
        eff_bytes = results[-1].effective_bytes
        bytes_in = sum(r.stats["bytes_in"] for r in results) / len(results)
        bytes_out = sum(r.stats["bytes_out"] for r in results) / len(results)
        faults = sum(r.stats["faults"] for r in results) / len(results)
        direct = sum(r.stats.get("bytes_direct", 0) for r in results) / len(results)   # read in place, no page moved
        peaks = measured_peaks()
        hbm_peak = peaks.get("hbm_gbs", 6650.0)
        roof = link_roofline(bytes_in + direct, bytes_out, kern_s, link)
        traffic = (NCU_LINK_TRAFFIC.get(cfg) if args.shrink == 0 and not args.scratch_limit_mib and args.inplace_divisor < 0
                   else None)
        roof["traffic"] = traffic[0] if traffic else None
        roof["traffic_source"] = (f"profiles/{traffic[1]} ({traffic[3]}): host-link bytes of one launch counted by ncu"
                                  if traffic else None)
        roof["hbm"] = {"achieved": (bytes_in + bytes_out + eff_bytes) / kern_s / 1e9, "peak": hbm_peak,
                       "frac": ((bytes_in + bytes_out + eff_bytes) / kern_s / 1e9) / hbm_peak,
                       "peak_source": "MEASURED_PEAKS.json" if peaks else "fallback"}
        rec = {
            "value": replica_throughput(world, eff_bytes, step_s) / 1e9, "unit": UNIT, "steps": steps, "warmup": warmup,
            "ms_per_step": step_s * 1e3, "dtype": DTYPES[cfg], "config": config_of(cfg, args.shrink),
            "migration": {
                "in_gbs": bytes_in / step_s / 1e9, "out_gbs": bytes_out / step_s / 1e9,
                "direct_gbs": direct / step_s / 1e9, "bytes_direct": direct,
                "faults_per_s": faults / step_s, "faults": faults, "bytes_in": bytes_in, "bytes_out": bytes_out,
                "io_amplification": bytes_in / eff_bytes if eff_bytes else None,
                "fault_rate_ceiling_per_s": link["ce_h2d_gbs"] * 1e9 / w.page_bytes,
            },
            "scratch": {"bytes": B.gpuvm_scratch_bytes(w.h), "limit_bytes": args.scratch_limit_mib << 20,
                        "what": "device memory of the workload beside the pool: request tables, staged rows, queues"},
            "stats": results[-1].stats, "invariants": results[-1].check, "roofline": roof,
            "e2e": {"value": replica_throughput(world, eff_bytes, e2e_s) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": e2e[-1][1], "d2h_bytes_per_step": e2e[-1][2], "ms_per_step": e2e_s * 1e3},
            "gpu_launches": launches, "clocks": clocks, "wall_s": wall, "setup_s": w.setup_seconds,
            "step_ms": [r.seconds * 1e3 for r in results],
            "ms_median": statistics.median(r.seconds for r in results) * 1e3,
            "ms_min": min(r.seconds for r in results) * 1e3,
            "extra": results[-1].extra,
        }
        if cfg in (3, 8) and rank == 0:
            pages = w.compulsory_pages()
            rec["roofline"]["compulsory_pages"] = pages
            rec["roofline"]["frac_compulsory"] = pages * w.page_bytes / kern_s / 1e9 / link["ce_h2d_gbs"]
        if cfg == 5:
            rec["migration"]["inplace_divisor"] = args.inplace_divisor if args.inplace_divisor >= 0 else "auto"
        if cfg == 5 and rank == 0:
            rec["roofline"].update(embag_policy_records(torch, B, w, args, link, kern_s, direct, rec))
        if cfg in (2, 5) and not args.scratch_limit_mib:
            # the same workload with its scratch bounded to an eighth of the pool: fewer requests in flight
            # per warp, so a page serves fewer of them per visit and is fetched more often
            bound = max(w.pool_bytes // 8, 1 << 20)
            B.gpuvm_set_scratch_limit(w.h, bound)
            w.run(check=False)
            r = w.run(check=True)
            rec["scratch"]["bounded_to_an_eighth_of_the_pool"] = {
                "limit_bytes": bound, "ms_per_step": r.seconds * 1e3,
                "value": r.effective_bytes / r.seconds / 1e9, "faults": r.stats["faults"],
                "in_gbs": r.stats["bytes_in"] / r.seconds / 1e9, "invariants_status": r.check["status"]}
            B.gpuvm_set_scratch_limit(w.h, 0)
        if rank == 0:
            if not args.no_cpu_baseline:
                rec["cpu_baseline"] = cpu_baseline(cfg, w if cfg in (1, 2) else None, args.shrink)
            if not args.no_replay and cfg in (3, 5) and args.shrink >= 0:
                rec["oracle_replay_faults"] = replay_counts(cfg, w)
            if not args.no_uvm and (args.uvm or cfg in (1, 3)):
                from paper_2411_05309_b200 import uvm
                rec["uvm"] = uvm.run_twin(cfg, args.shrink, timeout_s=args.uvm_timeout, w=w if cfg in (1, 3) else None)
        return rec
    finally:
        w.close()
        torch.cuda.empty_cache()


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
    head = headline_of(args, world)
    order = [args.workload] if args.workload else [int(c) for c in args.configs.split(",")]
    order = [c for c in order if c != head] + [head]               # the headline workload runs last
    per_config = {}
    for cfg in order:
        steps, warmup = (args.steps, args.warmup) if cfg == head else (min(args.steps, 10), min(args.warmup, 3))
        per_config[str(cfg)] = run_config(torch, B, configs, cfg, args, steps, warmup, link, dist, world, local_rank,
                                          rank, barrier)
    if dist is not None:
        dist.destroy_process_group()
    if rank != 0:
        return
    h = per_config[str(head)]
    line = {"metric": METRIC, "value": h["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": h["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": h["dtype"], "data": "synthetic", "config": h["config"],
            "replicas": world,
            "cache_state": "cold every step: page table reset, the paged array (>= 8x L2 at full size) is re-read "
                           "from host memory; nothing of a previous step stays resident",
            "link_peak": link}
    for k in ("migration", "scratch", "stats", "invariants", "roofline", "e2e", "gpu_launches", "clocks", "wall_s",
              "step_ms", "ms_median", "ms_min", "cpu_baseline", "oracle_replay_faults", "uvm", "extra"):
        if k in h:
            line[k] = h[k]
    if len(per_config) > 1:
        line["per_config"] = per_config
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=0, choices=[0, 1, 2, 3, 4, 5, 6, 7, 8, 9],
                    help="run this workload only (0: all of --configs, the largest as the headline)")
    ap.add_argument("--configs", default="1,2,3,4,5", help="configurations of the default run")
    ap.add_argument("--shrink", type=int, default=0, help="divide all sizes by 2**shrink")
    ap.add_argument("--uvm", action="store_true", help="run every workload over cudaMallocManaged too (default: cfg 1 and 3)")
    ap.add_argument("--no-uvm", action="store_true")
    ap.add_argument("--uvm-timeout", type=float, default=120.0)
    ap.add_argument("--scratch-limit-mib", type=int, default=0,
                    help="bound of the workload's device scratch (request tables, staged rows); 0 = none. Less scratch "
                         "means fewer page requests in flight per warp and more faults")
    ap.add_argument("--inplace-divisor", type=int, default=-1,
                    help="rent-or-buy divisor of the batched row workloads (cfg 5): -1 = the library's default, 0 = off")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-replay", action="store_true", help="skip the oracle's sequential replay counts (cfg 3 and 5)")
    ap.add_argument("--clock-period", type=float, default=0.1, help="seconds between NVML clock samples")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
