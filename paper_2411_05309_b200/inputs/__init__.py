"""Seeded synthetic inputs for the five paged-memory workloads.

Holds only data generators (``gen.c``): no paging and no workload arithmetic.  Every
array element is a pure function of ``(seed, index)`` through a counter-based 64-bit
mixer, so slices can be regenerated independently and results do not depend on the
number of threads.  Generators write into caller-provided memory (a numpy array or a
raw address such as a pinned host buffer).

The value distributions follow the workload definitions: int32 uniform in [0, 2^20)
for the streaming reduce; fp32 on the exact grid j*2^-23 - 1 in [-1, 1) for gather,
vector add and the embedding table; uniform int64 indices; an RMAT graph
(a=0.57, b=0.19, c=0.19, d=0.05) in CSR with int64 row offsets and int32 columns;
Zipf(s) row ids by rejection-inversion with row = rank - 1.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libgpuvm_inputs.so")

BASE_SEED = 0x2411053090000


def config_seed(cfg: int, stream: int = 0) -> int:
    """Seed of array ``stream`` of workload configuration ``cfg`` (1-based)."""
    return BASE_SEED + 16 * cfg + stream


def build(force: bool = False) -> str:
    """Compile ``gen.c`` with gcc + OpenMP if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-Wall", "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"])
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, vp = ctypes.c_uint64, ctypes.c_void_p
        lib.gvi_mix64.restype = u64
        lib.gvi_mix64.argtypes = [u64, u64]
        lib.gvi_fill_i32_u20.argtypes = [vp, u64, u64, u64]
        lib.gvi_fill_f32_pm1.argtypes = [vp, u64, u64, u64]
        lib.gvi_fill_index_i64.argtypes = [vp, u64, u64, u64, u64]
        lib.gvi_fill_i32_range.argtypes = [vp, u64, u64, u64, ctypes.c_int32, ctypes.c_uint32]
        lib.gvi_fill_i32_range.restype = None
        lib.gvi_rmat_csr.restype = ctypes.c_int
        lib.gvi_rmat_csr.argtypes = [ctypes.c_int, u64, u64, ctypes.c_uint32, ctypes.c_uint32,
                                     ctypes.c_uint32, vp, vp]
        lib.gvi_fill_zipf_rows.argtypes = [vp, u64, u64, u64, u64, ctypes.c_double]
        for f in (lib.gvi_fill_i32_u20, lib.gvi_fill_f32_pm1, lib.gvi_fill_index_i64,
                  lib.gvi_fill_zipf_rows):
            f.restype = None
        _lib = lib
    return _lib


def _addr(dst, dtype, n):
    """Address of the destination: a numpy array of the right dtype/size or an int."""
    if isinstance(dst, np.ndarray):
        assert dst.dtype == np.dtype(dtype) and dst.flags.c_contiguous and dst.size >= n
        return dst.ctypes.data
    return int(dst)


def mix64(seed: int, i: int) -> int:
    return int(_load().gvi_mix64(seed, i))


def fill_i32_u20(dst, n: int, seed: int, first: int = 0):
    _load().gvi_fill_i32_u20(_addr(dst, np.int32, n), first, n, seed)
    return dst


def fill_f32_pm1(dst, n: int, seed: int, first: int = 0):
    _load().gvi_fill_f32_pm1(_addr(dst, np.float32, n), first, n, seed)
    return dst


def fill_i32_range(dst, n: int, seed: int, lo: int, span: int, first: int = 0):
    """int32 values uniform in [lo, lo + span): synthetic edge weights."""
    _load().gvi_fill_i32_range(_addr(dst, np.int32, n), first, n, seed, lo, span)
    return dst


def fill_index_i64(dst, n: int, seed: int, modulo: int, first: int = 0):
    _load().gvi_fill_index_i64(_addr(dst, np.int64, n), first, n, seed, modulo)
    return dst


RMAT_T = (int(0.57 * 2 ** 32), int(0.76 * 2 ** 32), int(0.95 * 2 ** 32))


def rmat_csr(scale: int, n_edges: int, seed: int, row_off=None, col=None, thresholds=RMAT_T):
    """RMAT graph in CSR; returns (row_off int64[2^scale+1], col int32[n_edges])."""
    nv = 1 << scale
    if row_off is None:
        row_off = np.empty(nv + 1, dtype=np.int64)
    if col is None:
        col = np.empty(n_edges, dtype=np.int32)
    rc = _load().gvi_rmat_csr(scale, n_edges, seed, thresholds[0], thresholds[1], thresholds[2],
                              _addr(row_off, np.int64, nv + 1), _addr(col, np.int32, n_edges))
    if rc != 0:
        raise MemoryError("rmat_csr: temporary edge list allocation failed")
    return row_off, col


def fill_zipf_rows(dst, n: int, seed: int, n_ranks: int, s: float = 1.05, first: int = 0):
    _load().gvi_fill_zipf_rows(_addr(dst, np.int64, n), first, n, seed, n_ranks, s)
    return dst
