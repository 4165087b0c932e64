"""ctypes binding of libgpuvm.so: same names as the C ABI, argument marshalling only.

Every step of the paged path (translation, fault coalescing, frame claim, eviction,
write-back, migration, the workloads) runs in the CUDA kernels of the library; this
module only converts Python values to pointers and sizes.  There is no fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgpuvm.so")

POLICY_FIFO, POLICY_CLOCK = 0, 1

E_ARG, E_PAGE, E_POOL, E_ALIGN, E_PIN, E_ALLOC, E_CUDA, E_TIMEOUT, E_RANGE, E_INVARIANT, E_NODEVICE, E_PINS, E_FRAMES = \
    range(-1, -14, -1)

DEBUG_POISON, DEBUG_FENCED_RELEASE = 1, 2


class GpuvmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} (status {status})")


class DevView(ctypes.Structure):
    _fields_ = [("pte", ctypes.c_void_p), ("frame_vpn", ctypes.c_void_p), ("pool", ctypes.c_void_p),
                ("host", ctypes.c_void_p), ("ctl", ctypes.c_void_p), ("bytes", ctypes.c_uint64),
                ("n_pages", ctypes.c_uint64), ("n_frames", ctypes.c_uint32), ("page_shift", ctypes.c_uint32),
                ("policy", ctypes.c_uint32), ("spin_limit_us", ctypes.c_uint32), ("debug", ctypes.c_uint32),
                ("clean_ahead", ctypes.c_uint32)]


class Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in
                ("faults", "hits", "waits", "lanes_coalesced", "evictions", "writebacks", "flush_writebacks",
                 "bytes_in", "bytes_out", "hand_steps", "retries", "resident", "cleaned", "bytes_direct", "ring_drops")] + \
               [("error", ctypes.c_int32), ("reserved", ctypes.c_uint32), ("error_page", ctypes.c_uint64)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_ if n != "reserved"}


class Check(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in
                ("resident", "frames_used", "bad_state", "bad_refcount", "bad_backref", "bad_range", "dirty")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


# name -> (restype, argtypes): every symbol declared in include/*.h
_vp, _sz, _i, _u64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64
SYMBOLS = {
    "gpuvm_create": (_i, [ctypes.POINTER(_vp), _vp, _sz, _sz, _sz]),
    "gpuvm_destroy": (_i, [_vp]),
    "gpuvm_stats": (_i, [_vp, ctypes.POINTER(Stats)]),
    "gpuvm_stats_on": (_i, [_vp, ctypes.POINTER(Stats), _vp]),
    "gpuvm_reset_on": (_i, [_vp, _vp]),
    "gpuvm_check_on": (_i, [_vp, ctypes.POINTER(Check), _vp]),
    "gpuvm_set_debug": (_i, [_vp, ctypes.c_uint]),
    "gpuvm_set_clean_ahead": (_i, [_vp, ctypes.c_uint]),
    "gpuvm_set_inplace_divisor": (_i, [_vp, ctypes.c_uint]),
    "gpuvm_advise_keep": (_i, [_vp, _sz, _sz, _i]),
    "gpuvm_set_inplace_counted": (_i, [_vp, _i]),
    "gpuvm_bcsr_build": (_i, [_vp, _sz, _sz, _vp, _sz, ctypes.POINTER(_sz)]),
    "gpuvm_device_view": (_i, [_vp, ctypes.POINTER(DevView)]),
    "gpuvm_host_ptr": (_vp, [_vp]),
    "gpuvm_flush": (_i, [_vp, _vp]),
    "gpuvm_reset": (_i, [_vp]),
    "gpuvm_check": (_i, [_vp, ctypes.POINTER(Check)]),
    "gpuvm_set_policy": (_i, [_vp, _i]),
    "gpuvm_set_spin_limit_us": (_i, [_vp, ctypes.c_uint]),
    "gpuvm_set_scratch_limit": (_i, [_vp, ctypes.c_size_t]),
    "gpuvm_scratch_bytes": (ctypes.c_size_t, [_vp]),
    "gpuvm_safe_warps": (_i, [_vp, _i]),
    "gpuvm_inflight_pages": (ctypes.c_double, [ctypes.c_double, ctypes.c_double, ctypes.c_double]),
    "gpuvm_debug_poke_pte": (_i, [_vp, _u64, _u64]),
    "gpuvm_debug_peek_pte": (_i, [_vp, _u64, ctypes.POINTER(_u64)]),
    "gpuvm_strerror": (ctypes.c_char_p, [_i]),
    "gpuvm_last_cuda_error": (_i, [_vp]),
    "gpuvm_stream_sum_i32": (_i, [_vp, _sz, _sz, _vp, _vp]),
    "gpuvm_gather_f32": (_i, [_vp, _sz, _vp, _sz, _sz, _vp, _vp, _vp]),
    "gpuvm_gather_f32_unbatched": (_i, [_vp, _sz, _vp, _sz, _sz, _vp, _vp, _vp]),
    "gpuvm_bfs_csr": (_i, [_vp, _sz, _sz, _sz, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_bfs_csr_noalloc": (_i, [_vp, _sz, _sz, _sz, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_bfs_bcsr": (_i, [_vp, _sz, _sz, _sz, _sz, _sz, _sz, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_cc_bcsr": (_i, [_vp, _sz, _sz, _sz, _sz, _sz, _sz, _vp, _vp]),
    "gpuvm_cc_csr": (_i, [_vp, _sz, _sz, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_sssp_csr": (_i, [_vp, _sz, _sz, _sz, _sz, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_raw_cc_csr": (_i, [_vp, _vp, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_raw_sssp_csr": (_i, [_vp, _vp, _vp, _sz, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_vadd_f32": (_i, [_vp, _sz, _sz, _sz, _sz, _vp]),
    "gpuvm_embag_f32": (_i, [_vp, _sz, _sz, _vp, _sz, _sz, _vp, _vp]),
    "gpuvm_embag_f32_unbatched": (_i, [_vp, _sz, _sz, _vp, _sz, _sz, _vp, _vp]),
    "gpuvm_scatter_update_u32": (_i, [_vp, _sz, _vp, _sz, _vp]),
    "gpuvm_scatter_update_u32_batched": (_i, [_vp, _sz, _vp, _sz, _vp]),
    "gpuvm_scatter_update_u32_queued": (_i, [_vp, _sz, _vp, _sz, _vp]),
    "gpuvm_touch_pages": (_i, [_vp, _sz, _sz, _i, _vp]),
    "gpuvm_touch_pages_warps": (_i, [_vp, _sz, _sz, _i, _vp]),
    "gpuvm_raw_stream_sum_i32": (_i, [_vp, _sz, _vp, _vp]),
    "gpuvm_raw_gather_f32": (_i, [_vp, _vp, _sz, _sz, _vp, _vp, _vp]),
    "gpuvm_raw_bfs_csr": (_i, [_vp, _vp, _sz, _sz, _vp, ctypes.POINTER(_i), _vp]),
    "gpuvm_raw_vadd_f32": (_i, [_vp, _vp, _vp, _sz, _vp]),
    "gpuvm_raw_embag_f32": (_i, [_vp, _sz, _vp, _sz, _sz, _vp, _vp]),
    "gpuvm_link_peak": (_i, [_vp, _vp, _sz, _i, ctypes.POINTER(ctypes.c_double)]),
    "gpuvm_link_peak_scattered": (_i, [_vp, _sz, _sz, _sz, _sz, _vp, _sz, _i, ctypes.POINTER(ctypes.c_double)]),
    "gpuvm_launch_count": (ctypes.c_ulonglong, []),
    "gpuvm_uvm_alloc": (_i, [ctypes.POINTER(_vp), _sz]),
    "gpuvm_uvm_free": (_i, [_vp]),
    "gpuvm_uvm_advise_read_mostly": (_i, [_vp, _sz, _i]),
    "gpuvm_uvm_evict_to_host": (_i, [_vp, _sz]),
    "gpuvm_mem_info": (_i, [ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "gpuvm_balloon_alloc": (_i, [ctypes.POINTER(_vp), _sz]),
    "gpuvm_balloon_free": (_i, [_vp]),
}

_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2411_05309_b200.build` "
                              "(needs nvcc); there is no fallback path")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(handle, name)          # AttributeError if the export is missing
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def strerror(status: int) -> str:
    return lib().gpuvm_strerror(status).decode()


def _check(status: int, where: str):
    if status != 0:
        raise GpuvmError(status, where)


def _ptr(x) -> int:
    """Address of a torch tensor, a numpy array, or an integer address; None -> NULL."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _stream(stream) -> int:
    if stream is None:
        return 0
    return stream if isinstance(stream, int) else stream.cuda_stream


# ------------------------------------------------------------------ handle API

def gpuvm_create(host_backing, nbytes: int, page_bytes: int, pool_bytes: int) -> int:
    h = _vp()
    _check(lib().gpuvm_create(ctypes.byref(h), _ptr(host_backing), nbytes, page_bytes, pool_bytes), "gpuvm_create")
    return h.value


def gpuvm_destroy(h):
    _check(lib().gpuvm_destroy(h), "gpuvm_destroy")


def gpuvm_stats(h, raise_on_error: bool = True) -> dict:
    s = Stats()
    rc = lib().gpuvm_stats(h, ctypes.byref(s))
    if rc != 0 and (raise_on_error or rc != s.error):
        raise GpuvmError(rc, "gpuvm_stats")
    return s.as_dict()


def gpuvm_stats_on(h, stream, raise_on_error: bool = True) -> dict:
    s = Stats()
    rc = lib().gpuvm_stats_on(h, ctypes.byref(s), _stream(stream))
    if rc != 0 and (raise_on_error or rc != s.error):
        raise GpuvmError(rc, "gpuvm_stats_on")
    return s.as_dict()


def gpuvm_reset_on(h, stream):
    _check(lib().gpuvm_reset_on(h, _stream(stream)), "gpuvm_reset_on")


def gpuvm_check_on(h, stream, raise_on_error: bool = True) -> dict:
    c = Check()
    rc = lib().gpuvm_check_on(h, ctypes.byref(c), _stream(stream))
    if rc != 0 and raise_on_error:
        raise GpuvmError(rc, f"gpuvm_check_on {c.as_dict()}")
    d = c.as_dict()
    d["status"] = rc
    return d


def gpuvm_advise_keep(h, byte_off: int, nbytes: int, keep: bool = True):
    _check(lib().gpuvm_advise_keep(h, byte_off, nbytes, int(bool(keep))), "gpuvm_advise_keep")


INPLACE_AUTO = 0xFFFFFFFF


def gpuvm_set_inplace_divisor(h, divisor: int):
    _check(lib().gpuvm_set_inplace_divisor(h, divisor), "gpuvm_set_inplace_divisor")


def gpuvm_set_inplace_counted(h, counted: int):
    """0: online; 1: lookups counted per page first; 2 (default): counted, rows in place read page by page."""
    _check(lib().gpuvm_set_inplace_counted(h, int(counted)), "gpuvm_set_inplace_counted")


def gpuvm_set_clean_ahead(h, frames: int):
    _check(lib().gpuvm_set_clean_ahead(h, frames), "gpuvm_set_clean_ahead")


def gpuvm_set_debug(h, flags: int):
    _check(lib().gpuvm_set_debug(h, flags), "gpuvm_set_debug")


def gpuvm_bcsr_build(row_off, chunk_edges: int):
    """Chunk table of Balanced CSR for int64 row offsets held in a numpy array (host side)."""
    import numpy as np
    nv = row_off.size - 1
    n = _sz(0)
    _check(lib().gpuvm_bcsr_build(_ptr(row_off), nv, chunk_edges, None, 0, ctypes.byref(n)), "gpuvm_bcsr_build")
    out = np.empty(n.value + 1, dtype=np.int32)
    _check(lib().gpuvm_bcsr_build(_ptr(row_off), nv, chunk_edges, _ptr(out), out.size, None), "gpuvm_bcsr_build")
    return out


def gpuvm_device_view(h) -> DevView:
    v = DevView()
    _check(lib().gpuvm_device_view(h, ctypes.byref(v)), "gpuvm_device_view")
    return v


def gpuvm_host_ptr(h) -> int:
    return lib().gpuvm_host_ptr(h) or 0


def gpuvm_flush(h, stream=None):
    _check(lib().gpuvm_flush(h, _stream(stream)), "gpuvm_flush")


def gpuvm_reset(h):
    _check(lib().gpuvm_reset(h), "gpuvm_reset")


def gpuvm_check(h, raise_on_error: bool = True) -> dict:
    c = Check()
    rc = lib().gpuvm_check(h, ctypes.byref(c))
    if rc != 0 and raise_on_error:
        raise GpuvmError(rc, f"gpuvm_check {c.as_dict()}")
    d = c.as_dict()
    d["status"] = rc
    return d


def gpuvm_set_policy(h, policy: int):
    _check(lib().gpuvm_set_policy(h, policy), "gpuvm_set_policy")


def gpuvm_set_scratch_limit(h, nbytes: int):
    _check(lib().gpuvm_set_scratch_limit(h, nbytes), "gpuvm_set_scratch_limit")


def gpuvm_scratch_bytes(h) -> int:
    return int(lib().gpuvm_scratch_bytes(h))


def gpuvm_set_spin_limit_us(h, us: int):
    _check(lib().gpuvm_set_spin_limit_us(h, us), "gpuvm_set_spin_limit_us")


def gpuvm_safe_warps(h, pins_per_warp: int) -> int:
    n = lib().gpuvm_safe_warps(h, pins_per_warp)
    if n < 0:
        raise GpuvmError(n, "gpuvm_safe_warps")
    return n


def gpuvm_inflight_pages(latency_s: float, bytes_per_s: float, page_bytes: float) -> float:
    return lib().gpuvm_inflight_pages(latency_s, bytes_per_s, page_bytes)


def gpuvm_debug_poke_pte(h, page: int, value: int):
    _check(lib().gpuvm_debug_poke_pte(h, page, value), "gpuvm_debug_poke_pte")


def gpuvm_debug_peek_pte(h, page: int) -> int:
    v = _u64(0)
    _check(lib().gpuvm_debug_peek_pte(h, page, ctypes.byref(v)), "gpuvm_debug_peek_pte")
    return v.value


def gpuvm_last_cuda_error(h) -> int:
    return lib().gpuvm_last_cuda_error(h)


def gpuvm_launch_count() -> int:
    return int(lib().gpuvm_launch_count())


# ---------------------------------------------------------------- workload API

def gpuvm_stream_sum_i32(h, a_off: int, n: int, d_sum, stream=None):
    _check(lib().gpuvm_stream_sum_i32(h, a_off, n, _ptr(d_sum), _stream(stream)), "gpuvm_stream_sum_i32")


def gpuvm_gather_f32(h, x_off: int, d_idx, n_idx: int, block: int, d_fsum, d_bsum, stream=None):
    _check(lib().gpuvm_gather_f32(h, x_off, _ptr(d_idx), n_idx, block, _ptr(d_fsum), _ptr(d_bsum), _stream(stream)),
           "gpuvm_gather_f32")


def gpuvm_gather_f32_unbatched(h, x_off: int, d_idx, n_idx: int, block: int, d_fsum, d_bsum, stream=None):
    _check(lib().gpuvm_gather_f32_unbatched(h, x_off, _ptr(d_idx), n_idx, block, _ptr(d_fsum), _ptr(d_bsum),
                                            _stream(stream)), "gpuvm_gather_f32_unbatched")


def gpuvm_bfs_csr(h, off_off: int, col_off: int, nv: int, source: int, d_level, stream=None) -> int:
    levels = _i(0)
    _check(lib().gpuvm_bfs_csr(h, off_off, col_off, nv, source, _ptr(d_level), ctypes.byref(levels), _stream(stream)),
           "gpuvm_bfs_csr")
    return levels.value


def gpuvm_bfs_bcsr(h, off_off: int, col_off: int, chunk_off: int, nv: int, n_edges: int, chunk_edges: int,
                   source: int, d_level, stream=None) -> int:
    levels = _i(0)
    _check(lib().gpuvm_bfs_bcsr(h, off_off, col_off, chunk_off, nv, n_edges, chunk_edges, source, _ptr(d_level),
                                ctypes.byref(levels), _stream(stream)), "gpuvm_bfs_bcsr")
    return levels.value


def gpuvm_cc_bcsr(h, off_off: int, col_off: int, chunk_off: int, nv: int, n_edges: int, chunk_edges: int, d_label,
                  stream=None):
    _check(lib().gpuvm_cc_bcsr(h, off_off, col_off, chunk_off, nv, n_edges, chunk_edges, _ptr(d_label), _stream(stream)),
           "gpuvm_cc_bcsr")


def gpuvm_cc_csr(h, off_off: int, col_off: int, nv: int, d_label, stream=None) -> int:
    sweeps = _i(0)
    _check(lib().gpuvm_cc_csr(h, off_off, col_off, nv, _ptr(d_label), ctypes.byref(sweeps), _stream(stream)),
           "gpuvm_cc_csr")
    return sweeps.value


def gpuvm_sssp_csr(h, off_off: int, col_off: int, w_off: int, nv: int, source: int, d_dist, stream=None) -> int:
    rounds = _i(0)
    _check(lib().gpuvm_sssp_csr(h, off_off, col_off, w_off, nv, source, _ptr(d_dist), ctypes.byref(rounds),
                                _stream(stream)), "gpuvm_sssp_csr")
    return rounds.value


def gpuvm_raw_cc_csr(row_off, col, nv: int, d_label, stream=None) -> int:
    sweeps = _i(0)
    _check(lib().gpuvm_raw_cc_csr(_ptr(row_off), _ptr(col), nv, _ptr(d_label), ctypes.byref(sweeps), _stream(stream)),
           "gpuvm_raw_cc_csr")
    return sweeps.value


def gpuvm_raw_sssp_csr(row_off, col, weight, nv: int, source: int, d_dist, stream=None) -> int:
    rounds = _i(0)
    _check(lib().gpuvm_raw_sssp_csr(_ptr(row_off), _ptr(col), _ptr(weight), nv, source, _ptr(d_dist),
                                    ctypes.byref(rounds), _stream(stream)), "gpuvm_raw_sssp_csr")
    return rounds.value


BFS_NOALLOC_MAX_VERTICES = 1 << 26


def gpuvm_bfs_csr_noalloc(h, off_off: int, col_off: int, nv: int, source: int, d_level, stream=None) -> int:
    """gpuvm_bfs_csr on the library's built-in scratch array: no device allocation is made.
    Calls on one device must not overlap; the first call per device belongs in set-up."""
    levels = _i(0)
    _check(lib().gpuvm_bfs_csr_noalloc(h, off_off, col_off, nv, source, _ptr(d_level), ctypes.byref(levels),
                                       _stream(stream)), "gpuvm_bfs_csr_noalloc")
    return levels.value


def gpuvm_vadd_f32(h, a_off: int, b_off: int, c_off: int, n: int, stream=None):
    _check(lib().gpuvm_vadd_f32(h, a_off, b_off, c_off, n, _stream(stream)), "gpuvm_vadd_f32")


def gpuvm_embag_f32(h, t_off: int, dims: int, d_rows, n_bags: int, bag: int, d_out, stream=None):
    _check(lib().gpuvm_embag_f32(h, t_off, dims, _ptr(d_rows), n_bags, bag, _ptr(d_out), _stream(stream)),
           "gpuvm_embag_f32")


def gpuvm_embag_f32_unbatched(h, t_off: int, dims: int, d_rows, n_bags: int, bag: int, d_out, stream=None):
    _check(lib().gpuvm_embag_f32_unbatched(h, t_off, dims, _ptr(d_rows), n_bags, bag, _ptr(d_out), _stream(stream)),
           "gpuvm_embag_f32_unbatched")


def gpuvm_scatter_update_u32(h, a_off: int, d_idx, n: int, stream=None):
    _check(lib().gpuvm_scatter_update_u32(h, a_off, _ptr(d_idx), n, _stream(stream)), "gpuvm_scatter_update_u32")


def gpuvm_scatter_update_u32_queued(h, a_off: int, d_idx, n: int, stream=None):
    _check(lib().gpuvm_scatter_update_u32_queued(h, a_off, _ptr(d_idx), n, _stream(stream)),
           "gpuvm_scatter_update_u32_queued")


def gpuvm_scatter_update_u32_batched(h, a_off: int, d_idx, n: int, stream=None):
    _check(lib().gpuvm_scatter_update_u32_batched(h, a_off, _ptr(d_idx), n, _stream(stream)),
           "gpuvm_scatter_update_u32_batched")


def gpuvm_touch_pages(h, first_page: int, n_pages: int, warps_per_sm: int, stream=None):
    _check(lib().gpuvm_touch_pages(h, first_page, n_pages, warps_per_sm, _stream(stream)), "gpuvm_touch_pages")


def gpuvm_touch_pages_warps(h, first_page: int, n_pages: int, total_warps: int, stream=None):
    _check(lib().gpuvm_touch_pages_warps(h, first_page, n_pages, total_warps, _stream(stream)),
           "gpuvm_touch_pages_warps")


def gpuvm_raw_stream_sum_i32(a, n: int, d_sum, stream=None):
    _check(lib().gpuvm_raw_stream_sum_i32(_ptr(a), n, _ptr(d_sum), _stream(stream)), "gpuvm_raw_stream_sum_i32")


def gpuvm_raw_gather_f32(x, d_idx, n_idx: int, block: int, d_fsum, d_bsum, stream=None):
    _check(lib().gpuvm_raw_gather_f32(_ptr(x), _ptr(d_idx), n_idx, block, _ptr(d_fsum), _ptr(d_bsum), _stream(stream)),
           "gpuvm_raw_gather_f32")


def gpuvm_raw_bfs_csr(row_off, col, nv: int, source: int, d_level, stream=None) -> int:
    levels = _i(0)
    _check(lib().gpuvm_raw_bfs_csr(_ptr(row_off), _ptr(col), nv, source, _ptr(d_level), ctypes.byref(levels),
                                   _stream(stream)), "gpuvm_raw_bfs_csr")
    return levels.value


def gpuvm_raw_vadd_f32(a, b, c, n: int, stream=None):
    _check(lib().gpuvm_raw_vadd_f32(_ptr(a), _ptr(b), _ptr(c), n, _stream(stream)), "gpuvm_raw_vadd_f32")


def gpuvm_raw_embag_f32(table, dims: int, d_rows, n_bags: int, bag: int, d_out, stream=None):
    _check(lib().gpuvm_raw_embag_f32(_ptr(table), dims, _ptr(d_rows), n_bags, bag, _ptr(d_out), _stream(stream)),
           "gpuvm_raw_embag_f32")


def gpuvm_link_peak(host_ptr, d_buf, nbytes: int, reps: int = 3):
    out = (ctypes.c_double * 3)()
    _check(lib().gpuvm_link_peak(_ptr(host_ptr), _ptr(d_buf), nbytes, reps, out), "gpuvm_link_peak")
    return {"h2d_gbs": out[0], "d2h_gbs": out[1], "duplex_gbs": out[2]}


def gpuvm_link_peak_scattered(host_ptr, host_bytes: int, row_bytes: int, n_rows: int, d_buf, d_bytes: int, reps: int = 2,
                              run: int = 1) -> float:
    out = (ctypes.c_double * 1)()
    _check(lib().gpuvm_link_peak_scattered(_ptr(host_ptr), host_bytes, row_bytes, n_rows, run, _ptr(d_buf), d_bytes, reps, out),
           "gpuvm_link_peak_scattered")
    return out[0]


# ------------------------------------------------------------ managed-memory helpers

def gpuvm_uvm_alloc(nbytes: int) -> int:
    p = _vp()
    _check(lib().gpuvm_uvm_alloc(ctypes.byref(p), nbytes), "gpuvm_uvm_alloc")
    return p.value


def gpuvm_uvm_free(p: int):
    _check(lib().gpuvm_uvm_free(p), "gpuvm_uvm_free")


def gpuvm_uvm_advise_read_mostly(p: int, nbytes: int, on: bool):
    _check(lib().gpuvm_uvm_advise_read_mostly(p, nbytes, int(on)), "gpuvm_uvm_advise_read_mostly")


def gpuvm_uvm_evict_to_host(p: int, nbytes: int):
    _check(lib().gpuvm_uvm_evict_to_host(p, nbytes), "gpuvm_uvm_evict_to_host")


def gpuvm_mem_info():
    f, t = _sz(0), _sz(0)
    _check(lib().gpuvm_mem_info(ctypes.byref(f), ctypes.byref(t)), "gpuvm_mem_info")
    return f.value, t.value


def gpuvm_balloon_alloc(leave_free: int) -> int:
    p = _vp()
    _check(lib().gpuvm_balloon_alloc(ctypes.byref(p), leave_free), "gpuvm_balloon_alloc")
    return p.value or 0


def gpuvm_balloon_free(p: int):
    _check(lib().gpuvm_balloon_free(p), "gpuvm_balloon_free")
