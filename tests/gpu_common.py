"""Helpers shared by the GPU parity tests: arena layout and handle life cycle."""
from __future__ import annotations

import contextlib

import numpy as np


def aligned_bytes(nbytes: int, align: int = 4096) -> np.ndarray:
    raw = np.zeros(nbytes + align, dtype=np.uint8)
    shift = (-raw.ctypes.data) % align
    return raw[shift:shift + nbytes]


class Arena:
    """Several arrays at page-aligned offsets of one host backing store."""

    def __init__(self, page_bytes: int, arrays: dict):
        self.page = page_bytes
        self.off, total = {}, 0
        for name, a in arrays.items():
            self.off[name] = total
            total += (a.nbytes + page_bytes - 1) // page_bytes * page_bytes
        self.nbytes = max(total, 16)
        self.host = aligned_bytes(self.nbytes)
        self.views = {}
        for name, a in arrays.items():
            v = self.host[self.off[name]:self.off[name] + a.nbytes].view(a.dtype)
            v[...] = a.reshape(-1)
            self.views[name] = v

    @property
    def n_pages(self):
        return (self.nbytes + self.page - 1) // self.page


@contextlib.contextmanager
def paged(host: np.ndarray, page_bytes: int, n_frames: int, policy=None, spin_limit_us=None):
    from paper_2411_05309_b200 import binding as B
    h = B.gpuvm_create(host, host.nbytes, page_bytes, n_frames * page_bytes)
    try:
        if policy is not None:
            B.gpuvm_set_policy(h, policy)
        if spin_limit_us is not None:
            B.gpuvm_set_spin_limit_us(h, spin_limit_us)
        yield h
    finally:
        B.gpuvm_destroy(h)


def finish(h, expect_clean=True):
    """Flush, read counters (raises on a sticky device error), run the invariant kernel."""
    from paper_2411_05309_b200 import binding as B
    B.gpuvm_flush(h)
    st = B.gpuvm_stats(h)
    ck = B.gpuvm_check(h)
    assert ck["resident"] == ck["frames_used"] == st["resident"], (ck, st)
    if expect_clean:
        assert ck["dirty"] == 0
    return st, ck
