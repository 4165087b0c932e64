"""Randomised small cases, many of them: page sizes, pool sizes from one frame to everything,
both policies, all accessor styles.  Concurrency bugs in the page-table protocol (a lost
reference, a frame claimed twice, a write-back that races a re-fetch) show up as wrong
results, a failed invariant check, or a sticky error.  Every other case runs with the poison
debug mode (a frame is filled with a pattern when its page is evicted), so that a read from
the frame of a page that is no longer held cannot pass for old data."""
import os

import numpy as np
import pytest

import oracle
from gpu_common import Arena, finish, paged
from paper_2411_05309_b200 import inputs

pytestmark = pytest.mark.gpu

SOAK = int(os.environ.get("GPUVM_STRESS_SOAK", "1"))      # multiply the number of random cases


@pytest.fixture(scope="module")
def B():
    from paper_2411_05309_b200 import binding
    binding.lib()
    return binding


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_random_mix_of_workloads_on_one_handle(B):
    """Several kernels in a row on the same handle, no reset in between: gather (batched and not),
    scattered read-modify-write (both forms), streaming sum, with a shadow copy on the host."""
    import torch
    rng = np.random.default_rng(20241105)
    for case in range(40 * SOAK):
        page = int(rng.choice([64, 256, 1024, 4096, 16384]))
        n = int(rng.integers(2, 64)) * page // 4 + int(rng.integers(0, page // 16)) * 4
        n_pages = (4 * n + page - 1) // page
        frames = int(rng.choice([1, 2, 3, max(1, n_pages // 4), max(1, n_pages // 2), n_pages, n_pages + 3]))
        policy = int(rng.integers(0, 2))
        a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 1000 + case).astype(np.uint32)
        shadow = a.copy()
        ar = Arena(page, {"a": a})
        out = torch.zeros(1, dtype=torch.int64, device="cuda")
        with paged(ar.host, page, frames, policy) as h:
            if case & 1:                                               # every other case with frames poisoned on eviction
                B.gpuvm_set_debug(h, B.DEBUG_POISON)
            if case % 3 == 0:                                          # every third with write-back off the fault path
                B.gpuvm_set_clean_ahead(h, max(1, frames // 4))
            for step in range(int(rng.integers(2, 6))):
                kind = int(rng.integers(0, 5))
                if kind in (0, 1):                                     # scattered updates of distinct elements
                    m = int(rng.integers(1, n + 1))
                    idx = rng.permutation(n)[:m].astype(np.int64)
                    variant = int(rng.integers(0, 2))
                    (B.gpuvm_scatter_update_u32 if kind == 0 else
                     (B.gpuvm_scatter_update_u32_batched, B.gpuvm_scatter_update_u32_queued)[variant])(h, 0, dev(idx), m)
                    shadow[idx] = shadow[idx] * np.uint32(3) + np.uint32(1)
                elif kind in (2, 3):                                   # gather of the current contents
                    m = int(rng.integers(1, 4 * n))
                    block = int(rng.choice([32, 100, 1024, 3000]))
                    idx = rng.integers(0, n, m).astype(np.int64)
                    nb = (m + block - 1) // block
                    fs = torch.zeros(nb, dtype=torch.float32, device="cuda")
                    bs = torch.zeros(nb, dtype=torch.int64, device="cuda")
                    (B.gpuvm_gather_f32 if kind == 2 else B.gpuvm_gather_f32_unbatched)(h, 0, dev(idx), m, block, fs, bs)
                    ref = oracle.gather_block_sums_direct(shadow.view(np.float32), idx, block)[1]
                    assert np.array_equal(bs.cpu().numpy(), ref), (case, step, kind, page, frames)
                else:
                    B.gpuvm_stream_sum_i32(h, 0, n, out)
                    assert int(out.item()) == int(shadow.view(np.int32).astype(np.int64).sum()), (case, step, page, frames)
            st, ck = finish(h)
            assert ck["resident"] <= frames
        assert np.array_equal(ar.views["a"], shadow), (case, page, frames, policy)


def test_many_small_vector_adds_and_graphs(B):
    import torch
    rng = np.random.default_rng(7)
    for case in range(25 * SOAK):
        page = int(rng.choice([512, 1024, 4096]))
        n = (int(rng.integers(1, 40)) * page // 4 + int(rng.integers(0, page // 16)) * 4) // 4 * 4
        frames = int(rng.choice([1, 2, 3, 5, 9, 40, 200]))
        a = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 50 + case)
        b = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 90 + case)
        ar = Arena(page, {"a": a, "b": b, "c": np.zeros(n, np.float32)})
        with paged(ar.host, page, frames, int(rng.integers(0, 2))) as h:
            if case & 1:
                B.gpuvm_set_debug(h, B.DEBUG_POISON)
            B.gpuvm_vadd_f32(h, ar.off["a"], ar.off["b"], ar.off["c"], n)
            finish(h)
        assert np.array_equal(ar.views["c"].view(np.uint32), oracle.vadd_f32_direct(a, b).view(np.uint32)), (case, page, n, frames)
    for case in range(15 * SOAK):
        scale = int(rng.integers(6, 13))
        off, col = inputs.rmat_csr(scale, int(rng.integers(1, 24)) << scale, 300 + case)
        nv = off.size - 1
        src = int(rng.integers(0, nv))
        page = int(rng.choice([64, 1024, 4096]))
        frames = int(rng.choice([1, 2, 4, 16, 64]))
        off_p = np.zeros((off.size + 1) // 2 * 2, np.int64)
        off_p[:off.size] = off
        col_p = np.concatenate([col, np.zeros((-col.size) % 4, np.int32)])
        ar = Arena(page, {"off": off_p, "col": col_p})
        lvl = torch.zeros(nv, dtype=torch.int32, device="cuda")
        lab = torch.zeros(nv, dtype=torch.int32, device="cuda")
        with paged(ar.host, page, frames) as h:
            if case & 1:
                B.gpuvm_set_debug(h, B.DEBUG_POISON)
            B.gpuvm_bfs_csr(h, ar.off["off"], ar.off["col"], nv, src, lvl)
            B.gpuvm_cc_csr(h, ar.off["off"], ar.off["col"], nv, lab)
            finish(h)
        assert np.array_equal(lvl.cpu().numpy(), oracle.bfs_levels_direct(off, col, src)), (case, scale, page, frames)
        assert np.array_equal(lab.cpu().numpy(), oracle.cc_labels_direct(off, col)), (case, scale, page, frames)


def test_random_embedding_bags_under_every_page_policy(B):
    """Embedding bags of random shape (row size, bag length, table size, skew) over pools from one frame to the
    whole table, under the three forms of the in-place policy with random divisors (0 = every first touch
    fetches), with and without a scratch bound (a bound takes the staging slots away from the lookups, so rows in
    place are read as their lookups come up), every other case with frames poisoned on eviction.  The sums must
    have the oracle's bits, the invariants must hold, and what the counters say must add up: every lookup's row
    came from a fetched page or was read in place."""
    import torch
    rng = np.random.default_rng(20241106)
    for case in range(48 * SOAK):
        page = int(rng.choice([512, 4096, 65536]))
        dims = int(rng.choice([4, 16, 32, 128]))
        row_bytes = 4 * dims
        if row_bytes > page:
            continue
        n_rows = int(rng.integers(1, 40)) * (page // row_bytes) + int(rng.integers(0, 3))
        bag = int(rng.choice([1, 3, 8, 32, 40]))
        n_bags = int(rng.integers(1, 400))
        n_pages = (n_rows * row_bytes + page - 1) // page
        frames = int(rng.choice([1, 2, max(1, n_pages // 4), n_pages, n_pages + 2]))
        t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, 3000 + case)
        if rng.integers(0, 2):
            rows = inputs.fill_zipf_rows(np.empty(n_bags * bag, np.int64), n_bags * bag, 4000 + case, n_rows, 1.05)
        else:
            rows = rng.integers(0, n_rows, n_bags * bag).astype(np.int64)
        ref = oracle.embag_f32_direct(t.reshape(n_rows, dims), rows, bag).reshape(-1)
        ar = Arena(page, {"t": t})
        out = torch.zeros(n_bags * dims, dtype=torch.float32, device="cuda")
        counted = int(rng.integers(0, 3))
        divisor = int(rng.choice([0, 1, 2, 4, 16, B.INPLACE_AUTO]))
        bound = int(rng.choice([0, 0, 1 << 16, 1 << 20]))
        with paged(ar.host, page, frames, int(rng.integers(0, 2))) as h:
            if case & 1:
                B.gpuvm_set_debug(h, B.DEBUG_POISON)
            B.gpuvm_set_inplace_counted(h, counted)
            B.gpuvm_set_inplace_divisor(h, divisor)
            if bound:
                B.gpuvm_set_scratch_limit(h, bound)
            for _ in range(2):                                          # the second call finds pages resident
                out.zero_()
                B.gpuvm_embag_f32(h, 0, dims, dev(rows), n_bags, bag, out)
                st, ck = finish(h)
                what = (case, page, dims, n_rows, bag, n_bags, frames, counted, divisor, bound)
                assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32)), what
                assert st["bytes_direct"] % row_bytes == 0, what
                if divisor == 0:
                    assert st["bytes_direct"] == 0, what
