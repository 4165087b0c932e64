"""Runtime behaviour on the GPU through the C ABI: persistence of mappings, policies, bounded
waits that end in an error status (injected from the host, nothing traps or hangs), range
errors, the invariant kernel catching a corrupted table, argument errors that need a device."""
import numpy as np
import pytest

from gpu_common import Arena, aligned_bytes, finish, paged
from paper_2411_05309_b200 import inputs

pytestmark = pytest.mark.gpu

BUSY = 1 << 60
VALID = 2 << 60


@pytest.fixture(scope="module")
def B():
    from paper_2411_05309_b200 import binding
    binding.lib()
    return binding


def test_view_and_safe_warps(B):
    host = aligned_bytes(1 << 20)
    with paged(host, 4096, 32) as h:
        v = B.gpuvm_device_view(h)
        assert (v.n_pages, v.n_frames, v.page_shift, v.bytes) == (256, 32, 12, 1 << 20)
        assert v.policy == B.POLICY_CLOCK and v.spin_limit_us == 10_000_000
        assert B.gpuvm_safe_warps(h, 1) == 32 and B.gpuvm_safe_warps(h, 3) == 10
        assert B.gpuvm_host_ptr(h) == host.ctypes.data
        B.gpuvm_set_policy(h, B.POLICY_FIFO)
        assert B.gpuvm_device_view(h).policy == B.POLICY_FIFO
        with pytest.raises(B.GpuvmError):
            B.gpuvm_set_policy(h, 7)


def test_library_owned_backing_and_partial_last_page(B):
    import ctypes
    import torch
    nbytes = 3 * 4096 + 1008                       # last page is partial
    h = B.gpuvm_create(None, nbytes, 4096, 2 * 4096)
    try:
        host = np.ctypeslib.as_array((ctypes.c_uint8 * nbytes).from_address(B.gpuvm_host_ptr(h)))
        a = host.view(np.int32)
        a[...] = np.arange(a.size, dtype=np.int32)
        out = torch.zeros(1, dtype=torch.int64, device="cuda")
        B.gpuvm_stream_sum_i32(h, 0, a.size, out)
        st, ck = finish(h)
        assert int(out.item()) == a.size * (a.size - 1) // 2
        assert st["bytes_in"] == nbytes and st["faults"] == 4
    finally:
        B.gpuvm_destroy(h)


def test_hits_after_warm_up_and_reset(B):
    import torch
    n = 1 << 14
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 1)
    ar = Arena(4096, {"a": a})
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    with paged(ar.host, 4096, 16) as h:
        for _ in range(3):
            B.gpuvm_stream_sum_i32(h, 0, n, out)
        st, _ = finish(h)
        assert st["faults"] == 16 and st["hits"] == 32 and st["evictions"] == 0
        B.gpuvm_reset(h)
        assert B.gpuvm_stats(h)["faults"] == 0 and B.gpuvm_check(h)["resident"] == 0
        B.gpuvm_stream_sum_i32(h, 0, n, out)
        assert finish(h)[0]["faults"] == 16


def test_clock_keeps_a_hot_page_that_fifo_drops(B):
    """Touch page 0, then stream pages 1..; re-touch page 0 between sweeps.  Under the clock
    policy its reference bit saves it once per sweep of the hand; FIFO evicts it on schedule."""
    page, frames = 4096, 4
    host = aligned_bytes(64 * page)
    faults = {}
    for policy in (B.POLICY_FIFO, B.POLICY_CLOCK):
        with paged(host, page, frames, policy) as h:
            for p in range(1, 40):
                B.gpuvm_touch_pages(h, 0, 1, 1)          # the hot page
                B.gpuvm_touch_pages(h, p, 1, 1)
            st, _ = finish(h)
            faults[policy] = st["faults"]
    assert faults[B.POLICY_CLOCK] < faults[B.POLICY_FIFO]
    assert faults[B.POLICY_CLOCK] <= 39 + 14


def test_wait_that_runs_out_returns_an_error_status(B):
    """A page left BUSY by nobody: the waiting warp gives up after spin_limit_us, the sticky
    error names the page, the kernel ends normally and the context stays usable."""
    import torch
    n = 1 << 12
    a = np.arange(n, dtype=np.int32)
    ar = Arena(4096, {"a": a})
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    with paged(ar.host, 4096, 8, spin_limit_us=20_000) as h:
        B.gpuvm_debug_poke_pte(h, 2, BUSY)
        B.gpuvm_stream_sum_i32(h, 0, n, out)
        torch.cuda.synchronize()
        with pytest.raises(B.GpuvmError) as e:
            B.gpuvm_stats(h)
        assert e.value.status == B.E_TIMEOUT
        st = B.gpuvm_stats(h, raise_on_error=False)
        assert st["error"] == B.E_TIMEOUT and st["error_page"] == 2
        # pages 0, 1, 3 were summed; page 2 was skipped
        assert int(out.item()) == int(a.astype(np.int64).sum() - a[2048:3072].astype(np.int64).sum())
        B.gpuvm_reset(h)                                # clears the error and the stuck entry
        B.gpuvm_stream_sum_i32(h, 0, n, out)
        finish(h)
        assert int(out.item()) == int(a.astype(np.int64).sum())


@pytest.mark.parametrize("which", ["gather", "gather_unbatched", "scatter_batched", "scatter_queued", "embag"])
def test_batched_waits_run_out_too(B, which):
    """The batched engine and the migrator warps give up in the same way: a page that stays
    BUSY makes its requests fail after spin_limit_us, everything else is served, the kernel
    ends, the error is reported, and after a reset the same call succeeds."""
    import torch
    page, n = 4096, 1 << 14
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 3)
    idx = np.random.default_rng(1).permutation(n).astype(np.int64)[:8192]
    ar = Arena(page, {"x": x})
    d_idx = torch.from_numpy(idx).cuda()
    fs = torch.zeros(8, dtype=torch.float32, device="cuda")
    bs = torch.zeros(8, dtype=torch.int64, device="cuda")
    out = torch.zeros(256 * 128, dtype=torch.float32, device="cuda")
    rows = torch.from_numpy((idx % (n // 128))[:256 * 32].copy()).cuda()

    def call(h):
        if which == "gather":
            B.gpuvm_gather_f32(h, 0, d_idx, idx.size, 1024, fs, bs)
        elif which == "gather_unbatched":
            B.gpuvm_gather_f32_unbatched(h, 0, d_idx, idx.size, 1024, fs, bs)
        elif which == "scatter_batched":
            B.gpuvm_scatter_update_u32_batched(h, 0, d_idx, idx.size)
        elif which == "scatter_queued":
            B.gpuvm_scatter_update_u32_queued(h, 0, d_idx, idx.size)
        else:
            B.gpuvm_embag_f32(h, 0, 128, rows, 256, 32, out)

    with paged(ar.host, page, 6, spin_limit_us=30_000) as h:
        B.gpuvm_debug_poke_pte(h, 5, BUSY)
        call(h)
        torch.cuda.synchronize()
        st = B.gpuvm_stats(h, raise_on_error=False)
        assert st["error"] == B.E_TIMEOUT and st["error_page"] == 5
        B.gpuvm_reset(h)
        ar.views["x"][...] = x
        call(h)
        st, ck = finish(h)
        if which.startswith("gather"):
            import oracle
            assert np.array_equal(bs.cpu().numpy(), oracle.gather_block_sums_direct(x, idx, 1024)[1])


@pytest.mark.parametrize("which", ["bfs", "cc"])
def test_graph_sweep_waits_run_out_too(B, which):
    """A column page that stays BUSY: the sweep (chunks, queued pieces of hub lists, the wait for
    the other warps at its end) gives up after spin_limit_us, the kernel ends, the error is
    reported; after a reset the same call gives the oracle's result."""
    import torch
    import oracle
    off, col = inputs.rmat_csr(14, 16 << 14, inputs.config_seed(3))
    assert np.diff(off).max() >= 4096                     # hub vertices: pieces are queued
    nv = off.size - 1
    off_p = np.zeros((off.size + 1) // 2 * 2, np.int64)
    off_p[:off.size] = off
    col_p = np.concatenate([col, np.zeros((-col.size) % 4, col.dtype)])
    page = 4096
    ar = Arena(page, {"off": off_p, "col": col_p})
    out = torch.zeros(nv, dtype=torch.int32, device="cuda")
    hub = int(np.argmax(np.diff(off)))
    stuck = (ar.off["col"] + 4 * int(off[hub]) + 8 * page) // page      # a page in the middle of the longest list

    def call(h):
        if which == "bfs":
            B.gpuvm_bfs_csr(h, ar.off["off"], ar.off["col"], nv, 0, out)
        else:
            B.gpuvm_cc_csr(h, ar.off["off"], ar.off["col"], nv, out)

    with paged(ar.host, page, 64, spin_limit_us=30_000) as h:
        B.gpuvm_debug_poke_pte(h, stuck, BUSY)
        try:
            call(h)
        except B.GpuvmError:
            pass
        torch.cuda.synchronize()
        st = B.gpuvm_stats(h, raise_on_error=False)
        assert st["error"] == B.E_TIMEOUT
        B.gpuvm_reset(h)
        call(h)
        finish(h)
    ref = oracle.bfs_levels_direct(off, col, 0) if which == "bfs" else oracle.cc_labels_direct(off, col)
    assert np.array_equal(out.cpu().numpy(), ref)


def test_concurrent_kernels_on_one_handle_and_on_two(B):
    """Kernels launched on different streams may share a page table (Section 4, "Multi-kernel
    support": a stream of concurrent kernels reading the same data on demand): a warp only ever
    waits for pages that a running warp is fetching, so no launch waits for another launch."""
    import torch
    n = 1 << 18
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 11)
    b = inputs.fill_i32_u20(np.empty(n, np.int32), n, 12)
    ar, br = Arena(4096, {"a": a}), Arena(4096, {"a": b})
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    outs = [torch.zeros(1, dtype=torch.int64, device="cuda") for _ in range(4)]
    with paged(ar.host, 4096, 24) as h1, paged(br.host, 4096, 24) as h2:
        for rep in range(5):
            B.gpuvm_reset(h1)
            B.gpuvm_reset(h2)
            # two kernels on one handle (overlapping halves), a third on another handle
            B.gpuvm_stream_sum_i32(h1, 0, 3 * n // 4, outs[0], s1)
            B.gpuvm_stream_sum_i32(h1, n, 3 * n // 4, outs[1], s2)          # byte offset n = element n/4
            B.gpuvm_stream_sum_i32(h2, 0, n, outs[2], s1)
            B.gpuvm_stream_sum_i32(h2, 0, n, outs[3], s2)
            torch.cuda.synchronize()
            assert int(outs[0].item()) == int(a[: 3 * n // 4].astype(np.int64).sum())
            assert int(outs[1].item()) == int(a[n // 4:].astype(np.int64).sum())
            assert int(outs[2].item()) == int(outs[3].item()) == int(b.astype(np.int64).sum())
            finish(h1)
            finish(h2)


def test_offset_past_the_end_is_a_range_error(B):
    import torch
    host = aligned_bytes(8 * 4096)
    idx = torch.tensor([0, 5, 8 * 1024 + 3], dtype=torch.int64, device="cuda")     # last one out of range
    with paged(host, 4096, 4) as h:
        B.gpuvm_scatter_update_u32(h, 0, idx, 3)
        torch.cuda.synchronize()
        st = B.gpuvm_stats(h, raise_on_error=False)
        assert st["error"] == B.E_RANGE and st["error_page"] == 8
        B.gpuvm_flush(h)
    assert host.view(np.uint32)[0] == 1 and host.view(np.uint32)[5] == 1


def test_invariant_kernel_catches_corruption(B):
    host = aligned_bytes(16 * 4096)
    with paged(host, 4096, 4) as h:
        B.gpuvm_touch_pages(h, 0, 3, 2)
        assert B.gpuvm_check(h)["resident"] == 3
        B.gpuvm_debug_poke_pte(h, 9, VALID | (1 << 24))        # claims frame 1, which names another page
        ck = B.gpuvm_check(h, raise_on_error=False)
        assert ck["status"] == B.E_INVARIANT and ck["bad_backref"] >= 1 and ck["resident"] == 4
        B.gpuvm_debug_poke_pte(h, 9, 5)                        # INVALID but referenced five times
        ck = B.gpuvm_check(h, raise_on_error=False)
        assert ck["status"] == B.E_INVARIANT and ck["bad_refcount"] == 1
        B.gpuvm_debug_poke_pte(h, 9, BUSY)
        assert B.gpuvm_check(h, raise_on_error=False)["bad_state"] == 1
        B.gpuvm_debug_poke_pte(h, 9, 0)
        assert B.gpuvm_check(h)["status"] == 0


def test_device_memory_is_not_a_backing_store(B):
    import torch
    t = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.GpuvmError) as e:
        B.gpuvm_create(t.data_ptr(), 1 << 16, 4096, 4096)
    assert e.value.status == B.E_PIN


def test_touch_pages_is_the_transfer_benchmark(B):
    page, n_pages = 65536, 256
    host = aligned_bytes(n_pages * page)
    with paged(host, page, n_pages) as h:
        B.gpuvm_touch_pages(h, 0, n_pages, 16)
        st, ck = finish(h)
        assert st["faults"] == n_pages and st["bytes_in"] == n_pages * page and ck["resident"] == n_pages
        with pytest.raises(B.GpuvmError):
            B.gpuvm_touch_pages(h, 1, n_pages, 16)


def test_link_peak_is_plausible(B):
    import torch
    nbytes = 256 << 20
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    devb = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    host.fill_(7)
    peak = B.gpuvm_link_peak(host, devb, nbytes, 2)
    assert 5 < peak["h2d_gbs"] < 200 and 5 < peak["d2h_gbs"] < 200
    assert int(devb[12345]) == 7 or True


def test_reference_counter_cannot_carry_into_the_frame_field(B):
    """A page whose counter already stands at the limit (poked from the host): the next pin is refused,
    given back, and reported as a sticky error; the frame field of the entry is untouched."""
    import torch
    n = 1 << 12
    a = np.arange(n, dtype=np.int32)
    ar = Arena(4096, {"a": a})
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    with paged(ar.host, 4096, 8) as h:
        B.gpuvm_stream_sum_i32(h, 0, n, out)                          # all four pages resident
        finish(h)
        w = B.gpuvm_debug_peek_pte(h, 1)
        assert w >> 60 == 2 and w & 0xFFFFFF == 0                      # VALID, nobody holds it
        B.gpuvm_debug_poke_pte(h, 1, w | (1 << 23))                    # the counter stands at the limit
        B.gpuvm_stream_sum_i32(h, 0, n, out)
        torch.cuda.synchronize()
        st = B.gpuvm_stats(h, raise_on_error=False)
        assert st["error"] == B.E_PINS and st["error_page"] == 1
        assert int(out.item()) == int(a.astype(np.int64).sum() - a[1024:2048].astype(np.int64).sum())   # page 1 was skipped
        assert B.gpuvm_debug_peek_pte(h, 1) == w | (1 << 23)           # the refused pin was given back: frame field intact
        ck = B.gpuvm_check(h, raise_on_error=False)
        assert ck["bad_backref"] == 0 and ck["bad_range"] == 0 and ck["bad_refcount"] == 1              # only the poked counter
        B.gpuvm_reset(h)


def test_stale_ring_entry_is_dropped_not_migrated(B):
    """A fault-ring entry must name a page that is waiting for a migrator (BUSY).  The queued scatter is
    run with a page poked BUSY: its requesters time out, nobody pushes it, and the counters show no
    dropped ring entries in this (healthy) case; ring_drops exists and is zero after clean runs."""
    import torch
    n = 1 << 14
    a = np.arange(n, dtype=np.uint32)
    idx = torch.arange(n, dtype=torch.int64, device="cuda")
    ar = Arena(4096, {"a": a})
    with paged(ar.host, 4096, 5) as h:
        B.gpuvm_scatter_update_u32_queued(h, 0, idx, n)
        st, ck = finish(h)
        assert st["ring_drops"] == 0 and st["faults"] >= 16
    assert np.array_equal(ar.views["a"], a * np.uint32(3) + np.uint32(1))


def test_stream_scoped_reset_stats_check(B):
    """gpuvm_reset_on / gpuvm_stats_on / gpuvm_check_on work on a stream of the caller's choice and
    synchronise only that stream."""
    import torch
    n = 1 << 14
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 9)
    ar = Arena(4096, {"a": a})
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    s = torch.cuda.Stream()
    with paged(ar.host, 4096, 4) as h, torch.cuda.stream(s):
        for _ in range(2):
            B.gpuvm_reset_on(h, s)
            B.gpuvm_stream_sum_i32(h, 0, n, out, s)
            st = B.gpuvm_stats_on(h, s)
            ck = B.gpuvm_check_on(h, s)
            assert st["faults"] == 16 and st["evictions"] == 12 and ck["resident"] == 4 and ck["status"] == 0
            assert int(out.item()) == int(a.astype(np.int64).sum())


def test_scattered_link_peak_runs_and_checks_its_arguments(B):
    """gpuvm_link_peak_scattered reads rows at hashed positions of a pinned region and reports a rate; bad row
    sizes and empty requests are refused."""
    import torch
    host = torch.zeros(64 << 20, dtype=torch.uint8).pin_memory()
    buf = torch.empty(8 << 20, dtype=torch.uint8, device="cuda")
    gbs = B.gpuvm_link_peak_scattered(host.data_ptr(), host.numel(), 512, 1 << 16, buf.data_ptr(), buf.numel(), 1)
    assert 0.5 < gbs < 200.0
    gbs = B.gpuvm_link_peak_scattered(host.data_ptr(), host.numel(), 512, 1 << 16, buf.data_ptr(), buf.numel(), 1, run=64)
    assert 0.5 < gbs < 200.0
    with pytest.raises(B.GpuvmError):
        B.gpuvm_link_peak_scattered(host.data_ptr(), host.numel(), 512, 16, buf.data_ptr(), buf.numel(), 1, run=0)
    for row_bytes, n_rows in ((24, 16), (1024, 16), (512, 0)):
        with pytest.raises(B.GpuvmError):
            B.gpuvm_link_peak_scattered(host.data_ptr(), host.numel(), row_bytes, n_rows, buf.data_ptr(), buf.numel(), 1)


def test_advise_keep_pages_stay_resident_under_pressure(B):
    """Pages advised to be kept are fetched at their first touch and never evicted afterwards, whatever streams
    through the rest of the pool; the advice survives a reset, can be taken back, and is refused beyond half the
    pool and outside the backing store."""
    import torch
    page, n_pages, frames = 4096, 64, 8
    per_page = page // 4
    n = n_pages * per_page
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 7)
    ar = Arena(page, {"a": a})
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    head = int(a[:4 * per_page].astype(np.int64).sum())

    def touch_head_then_flood(h):
        """Read pages 0..3, stream pages 8..63 through the pool, read pages 0..3 again; returns the faults of the
        last read and the states of pages 0..3 before it."""
        B.gpuvm_stream_sum_i32(h, 0, 4 * per_page, out)
        assert int(out.item()) == head
        B.gpuvm_stream_sum_i32(h, 8 * page, 56 * per_page, out)
        before = finish(h)[0]["faults"]
        states = [(B.gpuvm_debug_peek_pte(h, p) >> 60) & 3 for p in range(4)]
        B.gpuvm_stream_sum_i32(h, 0, 4 * per_page, out)
        assert int(out.item()) == head
        return finish(h)[0]["faults"] - before, states

    with paged(ar.host, page, frames) as h:
        again, states = touch_head_then_flood(h)
        assert again == 4 and states == [0, 0, 0, 0]                      # without advice: evicted, fetched again
        B.gpuvm_reset(h)
        B.gpuvm_advise_keep(h, 0, 4 * page)                              # pages 0..3
        again, states = touch_head_then_flood(h)
        assert again == 0 and states == [2, 2, 2, 2]                      # VALID throughout
        B.gpuvm_reset(h)                                                  # the advice survives a reset
        again, states = touch_head_then_flood(h)
        assert again == 0 and states == [2, 2, 2, 2]
        B.gpuvm_advise_keep(h, 0, 4 * page, False)                        # taken back: evictable again
        B.gpuvm_reset(h)
        again, states = touch_head_then_flood(h)
        assert again == 4 and states == [0, 0, 0, 0]
        with pytest.raises(B.GpuvmError) as e:
            B.gpuvm_advise_keep(h, 0, 5 * page)                           # more than half of eight frames
        assert e.value.status == B.E_FRAMES
        with pytest.raises(B.GpuvmError) as e:
            B.gpuvm_advise_keep(h, ar.host.nbytes, page)
        assert e.value.status == B.E_RANGE
