"""The C-ABI library on a machine without a GPU: it loads, exports every function its
headers declare, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for hdr in ("gpuvm.h", "gpuvm_workloads.h", "gpuvm_uvm.h"):
        text = open(os.path.join(ROOT, "include", hdr)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(gpuvm_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def B():
    from paper_2411_05309_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def test_every_declared_symbol_is_exported_and_bound(B):
    names = declared_functions()
    assert len(names) >= 28
    handle = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(handle, n), f"{n} declared in include/ but not exported"
        assert n in B.SYMBOLS, f"{n} has no binding"
    assert set(B.SYMBOLS) <= set(names)


def test_status_strings(B):
    for code in range(0, -14, -1):
        assert B.strerror(code) and B.strerror(code) != "unknown status"
    assert B.strerror(-99) == "unknown status"


def test_create_rejects_bad_arguments_before_cuda(B):
    host = np.zeros(1 << 16, dtype=np.uint8)
    h = ctypes.c_void_p()
    L = B.lib()
    assert L.gpuvm_create(None, host.ctypes.data, 4096, 4096, 4096) == B.E_ARG
    assert L.gpuvm_create(ctypes.byref(h), host.ctypes.data, 0, 4096, 4096) == B.E_ARG
    for page in (0, 8, 24, 3000, 1 << 31):
        assert L.gpuvm_create(ctypes.byref(h), host.ctypes.data, 1 << 16, page, 1 << 16) == B.E_PAGE
    assert L.gpuvm_create(ctypes.byref(h), host.ctypes.data, 1 << 16, 4096, 0) == B.E_POOL
    assert L.gpuvm_create(ctypes.byref(h), host.ctypes.data, 1 << 16, 4096, 4096 + 512) == B.E_POOL
    assert L.gpuvm_create(ctypes.byref(h), host.ctypes.data, (1 << 16) - 8, 4096, 4096) == B.E_ALIGN
    assert L.gpuvm_create(ctypes.byref(h), host.ctypes.data + 4, 1 << 12, 4096, 4096) == B.E_ALIGN
    assert L.gpuvm_create(ctypes.byref(h), host.ctypes.data, 1 << 36, 16, 16) == B.E_PAGE    # > 2^31-2 pages
    assert h.value is None
    # NULL handles are refused everywhere
    assert L.gpuvm_destroy(None) == B.E_ARG and L.gpuvm_reset(None) == B.E_ARG
    assert L.gpuvm_flush(None, None) == B.E_ARG and L.gpuvm_safe_warps(None, 1) == B.E_ARG
    assert L.gpuvm_stream_sum_i32(None, 0, 16, None, None) == B.E_ARG
    assert L.gpuvm_bfs_csr_noalloc(None, 0, 0, 1, 0, None, None, None) == B.E_ARG
    assert L.gpuvm_set_scratch_limit(None, 1 << 20) == B.E_ARG and L.gpuvm_scratch_bytes(None) == 0
    assert L.gpuvm_gather_f32(None, 0, None, 16, 1024, None, None, None) == B.E_ARG
    assert L.gpuvm_embag_f32(None, 0, 128, None, 1, 32, None, None) == B.E_ARG
    assert L.gpuvm_scatter_update_u32_queued(None, 0, None, 1, None) == B.E_ARG


def test_no_device_no_fallback(B):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    host = np.zeros(1 << 16, dtype=np.uint8)
    with pytest.raises(B.GpuvmError) as e:
        B.gpuvm_create(host, host.nbytes, 4096, 4096)
    assert e.value.status == B.E_NODEVICE


def test_inflight_pages_is_littles_law_of_the_paper(B):
    # Section 3.2: 23 us x 12 GBps over 4 KB pages -> 72 queues, 8 KB -> 36 (binary units)
    assert abs(B.gpuvm_inflight_pages(23e-6, 12 * 2 ** 30, 4096) - 72.35) < 0.01
    assert abs(B.gpuvm_inflight_pages(23e-6, 12 * 2 ** 30, 8192) - 36.18) < 0.01
    assert B.gpuvm_inflight_pages(1.0, 1.0, 0.0) == 0.0


def test_bcsr_build_names_the_owner_of_each_chunks_first_edge(B):
    """The chunk table of Balanced CSR is built by the library on the host (no device needed)."""
    rng = np.random.default_rng(3)
    for _ in range(20):
        nv = int(rng.integers(1, 40))
        deg = rng.integers(0, 9, nv) * (rng.random(nv) < 0.6)
        off = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
        ne = int(off[-1])
        for chunk in (1, 3, 8):
            table = B.gpuvm_bcsr_build(off, chunk)
            n_chunks = (ne + chunk - 1) // chunk
            assert table.dtype == np.int32 and table.size == n_chunks + 1
            owner = np.repeat(np.arange(nv), np.diff(off))            # owner[e] by definition of CSR
            for c in range(n_chunks):
                assert table[c] == owner[c * chunk]
            assert table[-1] == (owner[-1] if ne else 0)
            assert np.all(np.diff(table) >= 0)
    # a table that is too small is refused; the size query needs no table
    off = np.array([0, 5, 5, 9], dtype=np.int64)
    n = ctypes.c_size_t(0)
    assert B.lib().gpuvm_bcsr_build(off.ctypes.data, 3, 4, None, 0, ctypes.byref(n)) == 0 and n.value == 3
    small = np.zeros(3, np.int32)
    assert B.lib().gpuvm_bcsr_build(off.ctypes.data, 3, 4, small.ctypes.data, 3, None) == B.E_RANGE
    assert B.lib().gpuvm_bcsr_build(off.ctypes.data, 3, 0, small.ctypes.data, 3, None) == B.E_ARG
    assert B.gpuvm_bcsr_build(off, 4).tolist() == [0, 0, 2, 2]
