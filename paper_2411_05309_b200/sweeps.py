"""Parameter sweeps of the paged path (the paper's transfer benchmark and its
oversubscription analysis), printed as JSON lines.

    python -m paper_2411_05309_b200.sweeps pages   [--gib 4] [--warps-per-sm 16]
    python -m paper_2411_05309_b200.sweeps warps   [--gib 2]
    python -m paper_2411_05309_b200.sweeps resident
    python -m paper_2411_05309_b200.sweeps oversub [--workload 1|2|3|4] [--shrink S]
    python -m paper_2411_05309_b200.sweeps depth   [--workload 2|5] [--shrink S]
    python -m paper_2411_05309_b200.sweeps writeback
    python -m paper_2411_05309_b200.sweeps link    [--gib 0.25]

pages   -- Section 5.1 / Fig. 7: move a fixed amount of host memory into the pool with one
           warp per page, consecutive pages, for page sizes from 4 KiB to 2 MiB; reports the
           migration bandwidth against the pinned-copy peak measured in the same run.
warps   -- Section 5.2 / Fig. 10 (sensitivity to the number of queue pairs): here the number of
           warps that migrate pages at the same time, 1 .. 32 per SM, at 4 KiB and 64 KiB pages;
           with Little's law (Section 3.2) the link saturates once warps x bytes in flight per
           warp (4 KiB) reach bandwidth x latency.
resident -- the hit path: streaming sum and random gather over an array that is entirely resident
           in the pool (no fault in the timed runs), against the same kernels on a plain device
           pointer and against the measured HBM copy bandwidth.
oversub -- Section 5.4 / Fig. 14 with Eq. 1: run a workload with the pool shrunk step by step,
           level = paged bytes / pool bytes - 1, under the clock policy and under FIFO (the
           paper's ring), reporting time relative to level 0.
depth   -- Section 3.2 (queue depth by Little's law) carried over to page requests: the batched
           workloads under a growing bound of their device scratch, i.e. with more and more page
           requests registered per warp; reports scratch bytes, faults and time.
link    -- the host link by itself: pinned-copy (copy engine) and SM-issued load / store bandwidth on a
           buffer of the given size (the kernels that every roofline of this build is measured against).
writeback -- Section 5.3 (vector add: synchronous write-back named as the weak spot) and Section 5.4
           (eviction adds to the fault latency): workloads whose victims are dirty, at pools of all,
           a quarter and a twelfth of the data: the scattered read-modify-write in its three forms and
           the vector add on a pool too small for its no-fetch path; reports time, faults, write-backs
           on and off the fault path, and both directions of the link.
"""
from __future__ import annotations

import argparse
import json
import sys


def _time(torch, fn):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fn()
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1) / 1e3


def sweep_pages(gib: float, warps_per_sm: int):
    import torch
    from . import binding as B
    nbytes = int(gib * (1 << 30))
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    devb = torch.empty(min(nbytes, 1 << 30), dtype=torch.uint8, device="cuda")
    best = 0.0
    for r in range(4):
        t = _time(torch, lambda: devb.copy_(host[:devb.numel()], non_blocking=True))
        if r:
            best = max(best, devb.numel() / t / 1e9)
    del devb
    torch.cuda.empty_cache()
    for shift in range(12, 22):
        page = 1 << shift
        h = B.gpuvm_create(host.data_ptr(), nbytes, page, nbytes)          # pool holds everything: no eviction
        try:
            times = []
            for r in range(3):
                B.gpuvm_reset(h)
                times.append(_time(torch, lambda: B.gpuvm_touch_pages(h, 0, nbytes // page, warps_per_sm)))
            st = B.gpuvm_stats(h)
            assert st["faults"] == nbytes // page and B.gpuvm_check(h)["resident"] == nbytes // page
            t = min(times[1:])
            print(json.dumps({"sweep": "pages", "page_bytes": page, "bytes": nbytes, "warps_per_sm": warps_per_sm,
                              "seconds": t, "migration_gbs": nbytes / t / 1e9, "faults_per_s": nbytes / page / t,
                              "pinned_copy_gbs": best, "frac_of_pinned_copy": nbytes / t / 1e9 / best}), flush=True)
        finally:
            B.gpuvm_destroy(h)


def sweep_warps(gib: float):
    import torch
    from . import binding as B
    nbytes = int(gib * (1 << 30))
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for page in (4096, 65536):
        h = B.gpuvm_create(host.data_ptr(), nbytes, page, nbytes)
        try:
            for warps in (1, 2, 4, 8, 16, 32, 64, sms, 4 * sms, 32 * sms):
                n_pages = min(nbytes // page, max(64, warps * (1 << 22) // page))     # a few MiB per warp
                times = []
                for r in range(3):
                    B.gpuvm_reset(h)
                    times.append(_time(torch, lambda: B.gpuvm_touch_pages_warps(h, 0, n_pages, warps)))
                t = min(times[1:])
                gbs = n_pages * page / t / 1e9
                print(json.dumps({"sweep": "warps", "page_bytes": page, "migrating_warps": warps,
                                  "bytes_in_flight": warps * 4096, "bytes": n_pages * page, "seconds": t,
                                  "migration_gbs": gbs, "gbs_per_warp": gbs / warps,
                                  "implied_latency_us": warps * 4096 / (gbs * 1e9) * 1e6}), flush=True)
        finally:
            B.gpuvm_destroy(h)


def sweep_resident():
    import torch
    from . import binding as B
    nbytes, n_idx = 1 << 30, 1 << 26
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    host.zero_()
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    dev = torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda")
    idx = torch.randint(0, nbytes // 4, (n_idx,), device="cuda", dtype=torch.int64)
    fs = torch.zeros(n_idx // 1024, dtype=torch.float32, device="cuda")
    bs = torch.zeros(n_idx // 1024, dtype=torch.int64, device="cuda")

    def best(fn, reps=4):
        fn()
        torch.cuda.synchronize()
        return min(_time(torch, fn) for _ in range(reps))

    t = best(lambda: B.gpuvm_raw_stream_sum_i32(dev.data_ptr(), nbytes // 4, out))
    print(json.dumps({"sweep": "resident", "kernel": "stream_sum on a device pointer", "gbs": nbytes / t / 1e9}), flush=True)
    t = best(lambda: B.gpuvm_raw_gather_f32(dev.data_ptr(), idx, n_idx, 1024, fs, bs))
    print(json.dumps({"sweep": "resident", "kernel": "gather on a device pointer", "g_accesses_per_s": n_idx / t / 1e9}), flush=True)
    for page in (4096, 65536, 2 << 20):
        h = B.gpuvm_create(host.data_ptr(), nbytes, page, nbytes)
        try:
            t = best(lambda: B.gpuvm_stream_sum_i32(h, 0, nbytes // 4, out))
            faults = B.gpuvm_stats(h)["faults"]
            print(json.dumps({"sweep": "resident", "kernel": "stream_sum, all pages resident", "page_bytes": page,
                              "gbs": nbytes / t / 1e9, "faults_in_warm_up_only": faults == nbytes // page}), flush=True)
            for name, fn in (("gather (batched), all pages resident", B.gpuvm_gather_f32),
                             ("gather (one request per lane), all pages resident", B.gpuvm_gather_f32_unbatched)):
                t = best(lambda: fn(h, 0, idx, n_idx, 1024, fs, bs), 3)
                print(json.dumps({"sweep": "resident", "kernel": name, "page_bytes": page,
                                  "g_accesses_per_s": n_idx / t / 1e9}), flush=True)
            assert B.gpuvm_stats(h)["faults"] == nbytes // page
        finally:
            B.gpuvm_destroy(h)


def sweep_oversub(cfg: int, shrink: int):
    from . import binding as B
    from . import configs
    levels = [0, 0.5, 1, 2, 3, 5, 7, 11]
    base = {}
    for policy, pname in ((B.POLICY_CLOCK, "clock"), (B.POLICY_FIFO, "fifo")):
        for level in levels:
            w = configs.WORKLOADS[cfg](shrink)
            w.pool_override = lambda total, level=level: int(total / (level + 1))
            w.setup()
            try:
                B.gpuvm_set_policy(w.h, policy)
                w.run(check=False)
                res = w.run()
                if level == 0:
                    base[pname] = res.seconds
                print(json.dumps({"sweep": "oversub", "workload": w.name, "policy": pname, "level": level,
                                  "level_actual": w.nbytes / w.pool_bytes - 1, "pool_bytes": w.pool_bytes,
                                  "seconds": res.seconds, "slowdown_vs_level0": res.seconds / base[pname],
                                  "faults": res.stats["faults"], "bytes_in": res.stats["bytes_in"],
                                  "bytes_out": res.stats["bytes_out"],
                                  "io_amplification": res.stats["bytes_in"] / max(1, res.effective_bytes)}), flush=True)
            finally:
                w.close()


def sweep_depth(cfg: int, shrink: int):
    from . import binding as B
    from . import configs
    limits_mib = {2: [40, 80, 150, 0], 5: [2300, 4500, 0]}[cfg]
    # the embedding bag under the paper's policy (every first touch fetches its page) and under the library's default
    # (rows of pages with few lookups are read in place)
    policies = {2: [("default", None)], 5: [("every first touch fetches", 0), ("default", None)]}[cfg]
    for policy, divisor in policies:
        for limit in limits_mib:
            w = configs.make(cfg, shrink)
            try:
                B.gpuvm_set_scratch_limit(w.h, (limit << 20) >> shrink)
                if divisor is not None:
                    B.gpuvm_set_inplace_divisor(w.h, divisor)
                w.run(check=False)
                runs = [w.run() for _ in range(3)]
                res = min(runs, key=lambda r: r.seconds)
                print(json.dumps({"sweep": "depth", "workload": w.name, "policy": policy,
                                  "scratch_limit_bytes": (limit << 20) >> shrink,
                                  "scratch_bytes": B.gpuvm_scratch_bytes(w.h), "pool_bytes": w.pool_bytes,
                                  "seconds": res.seconds, "faults": res.stats["faults"], "pages": w.nbytes // w.page_bytes,
                                  "bytes_in": res.stats["bytes_in"], "bytes_direct": res.stats["bytes_direct"],
                                  "in_gbs": res.stats["bytes_in"] / res.seconds / 1e9,
                                  "effective_gbs": res.effective_bytes / res.seconds / 1e9}), flush=True)
            finally:
                w.close()


def sweep_link(gib: float):
    import torch
    from . import binding as B
    nbytes = int(gib * (1 << 30)) // 4096 * 4096
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    devb = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    out = {"sweep": "link", "bytes": nbytes}
    for name, (dst, src) in {"ce_h2d_gbs": (devb, host), "ce_d2h_gbs": (host, devb)}.items():
        out[name] = max(nbytes / _time(torch, lambda: dst.copy_(src, non_blocking=True)) / 1e9 for _ in range(4))
    sm = B.gpuvm_link_peak(host.data_ptr(), devb.data_ptr(), nbytes, 3)
    out.update({"sm_h2d_gbs": sm["h2d_gbs"], "sm_d2h_gbs": sm["d2h_gbs"], "sm_duplex_gbs": sm["duplex_gbs"]})
    print(json.dumps(out), flush=True)
    # rows of 512 bytes at hashed positions of the first `span` bytes of the region: each at a position of its own
    # (run 1) or `run` consecutive ones in the same 2 MiB of it
    n_rows = 1 << 22
    span = 1 << 30
    while span <= nbytes:
        for run in (1, 4, 16, 64, 256):
            gbs = B.gpuvm_link_peak_scattered(host.data_ptr(), span, 512, n_rows, devb.data_ptr(), min(nbytes, 1 << 30), 2, run)
            print(json.dumps({"sweep": "link", "rows_of_512_bytes": n_rows, "span_bytes": span, "rows_per_2MiB_run": run,
                              "gbs": gbs}), flush=True)
        span *= 8


def sweep_writeback():
    import torch
    from . import binding as B
    from . import configs
    n, n_upd, page = 1 << 28, 1 << 24, 65536
    host = torch.zeros(n, dtype=torch.int32).pin_memory()
    idx = torch.randperm(n, device="cuda")[:n_upd].contiguous()
    forms = (("scatter, one access per lane", B.gpuvm_scatter_update_u32),
             ("scatter, batched, requester migrates", B.gpuvm_scatter_update_u32_batched),
             ("scatter, batched, migrator warps", B.gpuvm_scatter_update_u32_queued))

    def record(name, extra, t, st):
        print(json.dumps({"sweep": "writeback", "workload": name, **extra, "seconds": t, "faults": st["faults"],
                          "writebacks_on_fault_path": st["writebacks"], "writebacks_by_cleaners": st["cleaned"],
                          "flush_writebacks": st["flush_writebacks"], "in_gbs": st["bytes_in"] / t / 1e9,
                          "out_gbs": st["bytes_out"] / t / 1e9}), flush=True)

    for frac in (1, 4, 12):
        pool = (4 * n // frac) // page * page
        h = B.gpuvm_create(host.data_ptr(), 4 * n, page, pool)
        try:
            for name, fn in forms[1:] if frac > 1 else forms:       # (one access per lane thrashes for 15-20 s at small pools)
                for ahead in (0, None):
                    if ahead is not None:
                        B.gpuvm_set_clean_ahead(h, ahead)
                    else:
                        B.gpuvm_set_clean_ahead(h, min(pool // page // 32, 128))
                    best = None
                    for r in range(3):
                        B.gpuvm_reset(h)
                        t = _time(torch, lambda: (fn(h, 0, idx, n_upd), B.gpuvm_flush(h, torch.cuda.current_stream())))
                        st = B.gpuvm_stats(h)
                        assert B.gpuvm_check(h)["status"] == 0
                        if r and (best is None or t < best[0]):
                            best = (t, st)
                    record(name, {"pool_fraction": f"1/{frac}", "page_bytes": page,
                                  "clean_ahead": B.gpuvm_device_view(h).clean_ahead}, *best)
        finally:
            B.gpuvm_destroy(h)
    del host, idx
    torch.cuda.empty_cache()
    # vector add on small pools: out of place (the page of c is held, not fetched, and written back by its
    # producer) and in place (c = a: pages of a are read, written and left dirty: the case for the cleaners)
    for frames in (2048, 256):
        for in_place in (False, True):
            for ahead in (0, None):
                w = configs.WORKLOADS[4](2)                          # three 1 GiB arrays
                w.pool_override = frames * 65536
                w.setup()
                try:
                    if ahead is not None:
                        B.gpuvm_set_clean_ahead(w.h, ahead)
                    if in_place:
                        w.launch = lambda stream, w=w: B.gpuvm_vadd_f32(w.h, w.off["a"], w.off["b"], w.off["a"], w.n, stream)
                    w.run(check=False)
                    res = min((w.run() for _ in range(3)), key=lambda r: r.seconds)
                    record("vector add in place" if in_place else "vector add", {"frames": frames, "pool_bytes": w.pool_bytes,
                           "clean_ahead": B.gpuvm_device_view(w.h).clean_ahead}, res.seconds, res.stats)
                finally:
                    w.close()


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("which", choices=["pages", "warps", "resident", "oversub", "depth", "writeback", "link"])
    ap.add_argument("--gib", type=float, default=4.0)
    ap.add_argument("--warps-per-sm", type=int, default=16)
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--shrink", type=int, default=0)
    a = ap.parse_args(argv)
    if a.which == "pages":
        sweep_pages(a.gib, a.warps_per_sm)
    elif a.which == "resident":
        sweep_resident()
    elif a.which == "warps":
        sweep_warps(min(a.gib, 2.0))
    elif a.which == "writeback":
        sweep_writeback()
    elif a.which == "link":
        sweep_link(a.gib if a.gib != 4.0 else 0.25)
    elif a.which == "depth":
        sweep_depth(a.workload if a.workload in (2, 5) else 2, a.shrink)
    else:
        sweep_oversub(a.workload, a.shrink)


if __name__ == "__main__":
    sys.exit(main())
