"""CPU oracle for GPU-thread-driven demand paging -- TEST INFRASTRUCTURE ONLY.

A ctypes front end to ``gpuvm_oracle.c`` (plain single-threaded C, fp32 where the
workload is fp32, exact integers elsewhere).  It shares no code with the CUDA path
and must only be used by the test-suite, the smoke check and the benchmark's
CPU-baseline leg.

``*_direct`` functions are the plain definitions of what each workload computes on
the host arrays.  :class:`Pager` is the sequential paging replay (page table, frame
ring with a head cursor, FIFO or clock eviction, dirty write-back) and the
``*_paged`` functions run the same workloads element by element through it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gpuvm_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

FIFO, CLOCK = 0, 1


_LIB_OMP = os.path.join(_HERE, "liboracle_omp.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-Wall", "-Wno-unknown-pragmas", "-shared",
                               "-fPIC", _SRC, "-o", _LIB])
    return _LIB


def build_omp(force: bool = False) -> str:
    """The same source with OpenMP: the all-core CPU baseline of the benchmark."""
    if force or not os.path.exists(_LIB_OMP) or os.path.getmtime(_LIB_OMP) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-Wall", "-fopenmp", "-shared",
                               "-fPIC", _SRC, "-o", _LIB_OMP])
    return _LIB_OMP


class AllCores:
    """The four *_direct workloads whose outer loop splits over threads, from the OpenMP build."""

    def __init__(self):
        lib = ctypes.CDLL(build_omp())
        u64, vp = ctypes.c_uint64, ctypes.c_void_p
        lib.orc_stream_sum_i32_direct.restype, lib.orc_stream_sum_i32_direct.argtypes = ctypes.c_int64, [vp, u64]
        lib.orc_gather_block_sums_direct.restype, lib.orc_gather_block_sums_direct.argtypes = None, [vp, vp, u64, u64, vp, vp]
        lib.orc_vadd_f32_direct.restype, lib.orc_vadd_f32_direct.argtypes = None, [vp, vp, vp, u64]
        lib.orc_embag_f32_direct.restype, lib.orc_embag_f32_direct.argtypes = None, [vp, u64, vp, u64, u64, vp]
        lib.orc_threads.restype = ctypes.c_int
        self._lib = lib
        self.threads = int(lib.orc_threads())

    def stream_sum_i32_direct(self, a):
        return int(self._lib.orc_stream_sum_i32_direct(_p(a, np.int32), a.size))

    def gather_block_sums_direct(self, x, idx, block):
        nb = (idx.size + block - 1) // block
        fsum, bsum = np.empty(nb, dtype=np.float32), np.empty(nb, dtype=np.int64)
        self._lib.orc_gather_block_sums_direct(_p(x, np.float32), _p(idx, np.int64), idx.size, block,
                                               _p(fsum, np.float32), _p(bsum, np.int64))
        return fsum, bsum

    def vadd_f32_direct(self, a, b):
        c = np.empty_like(a)
        self._lib.orc_vadd_f32_direct(_p(a, np.float32), _p(b, np.float32), _p(c, np.float32), a.size)
        return c

    def embag_f32_direct(self, table, rows, bag):
        n_rows, dims = table.shape
        n_bags = rows.size // bag
        out = np.empty((n_bags, dims), dtype=np.float32)
        self._lib.orc_embag_f32_direct(_p(table, np.float32), dims, _p(rows, np.int64), n_bags, bag, _p(out, np.float32))
        return out


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, vp, i32, dbl = ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        sig = {
            "orc_stream_sum_i32_direct": (ctypes.c_int64, [vp, u64]),
            "orc_gather_block_sums_direct": (None, [vp, vp, u64, u64, vp, vp]),
            "orc_bfs_levels_direct": (None, [vp, vp, u64, u64, vp]),
            "orc_cc_labels_direct": (None, [vp, vp, u64, vp]),
            "orc_sssp_direct": (None, [vp, vp, vp, u64, u64, vp]),
            "orc_vadd_f32_direct": (None, [vp, vp, vp, u64]),
            "orc_embag_f32_direct": (None, [vp, u64, vp, u64, u64, vp]),
            "orc_pager_create": (vp, [vp, u64, u64, u64, i32, i32]),
            "orc_pager_destroy": (None, [vp]),
            "orc_pager_access": (u64, [vp, u64, i32]),
            "orc_pager_replay": (None, [vp, vp, vp, u64]),
            "orc_pager_flush": (None, [vp]),
            "orc_pager_counters": (None, [vp, vp]),
            "orc_pager_check": (i32, [vp]),
            "orc_pager_debug_poke": (i32, [vp, i32, u64, u64]),
            "orc_pager_trace": (None, [vp, vp, u64]),
            "orc_pager_trace_len": (u64, [vp]),
            "orc_belady_faults": (u64, [vp, u64, u64, u64]),
            "orc_stream_sum_i32_paged": (ctypes.c_int64, [vp, u64, u64]),
            "orc_gather_block_sums_paged": (None, [vp, u64, vp, u64, u64, vp, vp]),
            "orc_bfs_levels_paged": (None, [vp, u64, u64, u64, u64, vp]),
            "orc_vadd_f32_paged": (None, [vp, u64, u64, u64, u64]),
            "orc_embag_f32_paged": (None, [vp, u64, u64, vp, u64, u64, vp]),
            "orc_oversubscription_level": (dbl, [dbl, dbl]),
            "orc_queue_depth": (dbl, [dbl, dbl, dbl]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _p(a: np.ndarray, dtype) -> int:
    assert isinstance(a, np.ndarray) and a.dtype == np.dtype(dtype) and a.flags.c_contiguous, \
        (getattr(a, "dtype", None), dtype)
    return a.ctypes.data


# ---------------------------------------------------------------- results (R)

def stream_sum_i32_direct(a: np.ndarray) -> int:
    return int(_load().orc_stream_sum_i32_direct(_p(a, np.int32), a.size))


def gather_block_sums_direct(x: np.ndarray, idx: np.ndarray, block: int):
    nb = (idx.size + block - 1) // block
    fsum = np.empty(nb, dtype=np.float32)
    bsum = np.empty(nb, dtype=np.int64)
    _load().orc_gather_block_sums_direct(_p(x, np.float32), _p(idx, np.int64), idx.size, block,
                                         _p(fsum, np.float32), _p(bsum, np.int64))
    return fsum, bsum


def bfs_levels_direct(row_off: np.ndarray, col: np.ndarray, source: int) -> np.ndarray:
    nv = row_off.size - 1
    level = np.empty(nv, dtype=np.int32)
    _load().orc_bfs_levels_direct(_p(row_off, np.int64), _p(col, np.int32), nv, source,
                                  _p(level, np.int32))
    return level


def cc_labels_direct(row_off: np.ndarray, col: np.ndarray) -> np.ndarray:
    nv = row_off.size - 1
    label = np.empty(nv, dtype=np.int32)
    _load().orc_cc_labels_direct(_p(row_off, np.int64), _p(col, np.int32), nv, _p(label, np.int32))
    return label


def sssp_direct(row_off: np.ndarray, col: np.ndarray, weight: np.ndarray, source: int) -> np.ndarray:
    nv = row_off.size - 1
    dist = np.empty(nv, dtype=np.int32)
    _load().orc_sssp_direct(_p(row_off, np.int64), _p(col, np.int32), _p(weight, np.int32), nv, source,
                            _p(dist, np.int32))
    return dist


def vadd_f32_direct(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    c = np.empty_like(a)
    _load().orc_vadd_f32_direct(_p(a, np.float32), _p(b, np.float32), _p(c, np.float32), a.size)
    return c


def embag_f32_direct(table: np.ndarray, rows: np.ndarray, bag: int) -> np.ndarray:
    n_rows, dims = table.shape
    n_bags = rows.size // bag
    out = np.empty((n_bags, dims), dtype=np.float32)
    _load().orc_embag_f32_direct(_p(table, np.float32), dims, _p(rows, np.int64), n_bags, bag,
                                 _p(out, np.float32))
    return out


# ----------------------------------------------------------------- replay (P)

COUNTER_NAMES = ("accesses", "hits", "faults", "evictions", "writebacks", "bytes_in",
                 "bytes_out", "resident", "max_resident", "hand_steps")


class Pager:
    """Sequential paging replay over a host backing store held in a uint8 array."""

    def __init__(self, host: np.ndarray, page_bytes: int, n_frames: int, policy: int = CLOCK,
                 move_bytes: bool = True):
        assert host.dtype == np.uint8 and host.flags.c_contiguous
        self.host = host                      # keeps the memory alive
        self.page_bytes, self.n_frames = page_bytes, n_frames
        self._h = _load().orc_pager_create(host.ctypes.data, host.size, page_bytes, n_frames,
                                           policy, int(move_bytes))
        if not self._h:
            raise ValueError("bad pager arguments")

    def close(self):
        if self._h:
            _load().orc_pager_destroy(self._h)
            self._h = None

    __del__ = close

    def access(self, vpn: int, is_write: bool = False) -> int:
        return int(_load().orc_pager_access(self._h, vpn, int(is_write)))

    def replay(self, vpn: np.ndarray, is_write: np.ndarray | None = None):
        vpn = np.ascontiguousarray(vpn, dtype=np.uint64)
        w = None if is_write is None else np.ascontiguousarray(is_write, dtype=np.uint8)
        _load().orc_pager_replay(self._h, vpn.ctypes.data, None if w is None else w.ctypes.data,
                                 vpn.size)

    def flush(self):
        _load().orc_pager_flush(self._h)

    def counters(self) -> dict:
        out = np.zeros(10, dtype=np.uint64)
        _load().orc_pager_counters(self._h, out.ctypes.data)
        return {k: int(v) for k, v in zip(COUNTER_NAMES, out)}

    def check(self) -> int:
        return int(_load().orc_pager_check(self._h))

    def debug_poke(self, which: str, i: int, v: int) -> None:
        """Test hook: damage one word of the tables (which: 'map', 'frame_page', 'resident')."""
        rc = _load().orc_pager_debug_poke(self._h, {"map": 0, "frame_page": 1, "resident": 2}[which], i,
                                          v & 0xFFFFFFFFFFFFFFFF)
        if rc != 0:
            raise IndexError((which, i))

    def record_trace(self, capacity: int) -> np.ndarray:
        """Record the page numbers of the accesses that follow (runs of one page collapsed) into a
        new array of `capacity` entries; trace() returns the part that was filled."""
        self._trace = np.empty(capacity, dtype=np.uint64)
        _load().orc_pager_trace(self._h, self._trace.ctypes.data, capacity)
        return self._trace

    def trace(self) -> np.ndarray:
        n = int(_load().orc_pager_trace_len(self._h))
        if n > self._trace.size:
            raise OverflowError(f"trace needs {n} entries, {self._trace.size} were provided")
        return self._trace[:n]

    # workloads through the pager; offsets are byte offsets inside the backing store
    def stream_sum_i32(self, a_off: int, n: int) -> int:
        return int(_load().orc_stream_sum_i32_paged(self._h, a_off, n))

    def gather_block_sums(self, x_off: int, idx: np.ndarray, block: int):
        nb = (idx.size + block - 1) // block
        fsum = np.empty(nb, dtype=np.float32)
        bsum = np.empty(nb, dtype=np.int64)
        _load().orc_gather_block_sums_paged(self._h, x_off, _p(idx, np.int64), idx.size, block,
                                            _p(fsum, np.float32), _p(bsum, np.int64))
        return fsum, bsum

    def bfs_levels(self, off_off: int, col_off: int, nv: int, source: int) -> np.ndarray:
        level = np.empty(nv, dtype=np.int32)
        _load().orc_bfs_levels_paged(self._h, off_off, col_off, nv, source, _p(level, np.int32))
        return level

    def vadd_f32(self, a_off: int, b_off: int, c_off: int, n: int):
        _load().orc_vadd_f32_paged(self._h, a_off, b_off, c_off, n)

    def embag_f32(self, t_off: int, dims: int, rows: np.ndarray, bag: int) -> np.ndarray:
        n_bags = rows.size // bag
        out = np.empty((n_bags, dims), dtype=np.float32)
        _load().orc_embag_f32_paged(self._h, t_off, dims, _p(rows, np.int64), n_bags, bag,
                                    _p(out, np.float32))
        return out


NONE = 0xFFFFFFFFFFFFFFFF


def belady_faults(trace: np.ndarray, n_pages: int, n_frames: int) -> int:
    """Faults of Belady's optimal replacement on a trace of page numbers."""
    t = np.ascontiguousarray(trace, dtype=np.uint64)
    assert t.size == 0 or int(t.max()) < n_pages
    return int(_load().orc_belady_faults(t.ctypes.data, t.size, n_pages, n_frames))


def replay_counts(trace: np.ndarray, n_pages: int, page_bytes: int, n_frames: int, belady: bool = True) -> dict:
    """Fault counts of a read-only page trace under the sequential replay's two policies and
    under optimal replacement (what no policy can beat with this many frames)."""
    out = {}
    host = np.zeros(1, dtype=np.uint8)
    for name, policy in (("clock", CLOCK), ("fifo", FIFO)):
        h = _load().orc_pager_create(host.ctypes.data, n_pages * page_bytes, page_bytes, n_frames, policy, 0)
        t = np.ascontiguousarray(trace, dtype=np.uint64)
        _load().orc_pager_replay(h, t.ctypes.data, None, t.size)
        c = np.zeros(10, dtype=np.uint64)
        _load().orc_pager_counters(h, c.ctypes.data)
        out[name] = int(c[2])
        _load().orc_pager_destroy(h)
    if belady:
        out["belady"] = belady_faults(trace, n_pages, n_frames)
    out["distinct"] = int(np.unique(trace).size)
    return out


def oversubscription_level(workload_bytes: float, gpu_bytes: float) -> float:
    return float(_load().orc_oversubscription_level(workload_bytes, gpu_bytes))


def queue_depth(latency_s: float, bytes_per_s: float, request_bytes: float) -> float:
    return float(_load().orc_queue_depth(latency_s, bytes_per_s, request_bytes))
