"""GPU parity: every workload through the C ABI against the CPU oracle, element by element,
on seeded inputs that span several pages and a ragged tail, from ample to one-frame pools.
Bit-exact for integer outputs and written-back bytes; 1e-6 relative for fp32 sums."""
import numpy as np
import pytest

import oracle
from paper_2411_05309_b200 import inputs
from gpu_common import Arena, finish, paged

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2411_05309_b200 import binding
    binding.lib()
    return binding


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


POLICIES = [0, 1]


@pytest.mark.parametrize("page,n,frames", [
    (4096, 1 << 16, 64),          # pool == data
    (4096, 1 << 16, 16),          # 4x oversubscribed
    (4096, (1 << 16) + 1000, 5),  # ragged tail, tiny pool
    (256, 5000, 1),               # one frame
    (65536, 1 << 18, 3),
    (16, 2048, 7),                # smallest page
])
@pytest.mark.parametrize("policy", POLICIES)
def test_stream_sum(B, page, n, frames, policy):
    import torch
    n4 = (n + 3) // 4 * 4
    a = inputs.fill_i32_u20(np.empty(n4, np.int32), n4, inputs.config_seed(1))
    ar = Arena(page, {"a": a})
    before = ar.host.copy()
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    with paged(ar.host, page, frames, policy) as h:
        B.gpuvm_stream_sum_i32(h, ar.off["a"], n, out)
        st, ck = finish(h)
        assert int(out.item()) == oracle.stream_sum_i32_direct(a[:n])
        touched = (4 * n + page - 1) // page
        assert st["faults"] == touched                  # each page is read in one burst by one warp
        assert st["writebacks"] == 0 and st["bytes_out"] == 0
        assert st["evictions"] == max(0, touched - frames)
        assert ck["resident"] == min(touched, frames)
        # a second pass over a pool that holds everything takes no fault (mappings persist)
        if frames >= touched:
            B.gpuvm_stream_sum_i32(h, ar.off["a"], n, out)
            st2, _ = finish(h)
            assert st2["faults"] == touched and int(out.item()) == oracle.stream_sum_i32_direct(a[:n])
    assert np.array_equal(ar.host, before)


@pytest.mark.parametrize("page,frames", [
    (256, 20000),                 # four pages per warp at a time (eight lanes each): the pool lets every warp hold four
    (256, 10000),                 # two
    (256, 4000),                  # one
    (1 << 18, 40),                # pages above 64 KiB are shared out in 64 KiB pieces, one pin per piece
])
def test_stream_sum_lane_groups(B, page, frames):
    """The streaming kernel takes as many pages per warp at a time as the pool lets every warp of its grid hold
    (4, 2 or 1), and splits large pages into 64 KiB pieces: same sum, every page fetched once when the pool holds
    them all, ragged first and last pages included."""
    import torch
    n = (1 << 20) + 4 * 37 + 3
    a = inputs.fill_i32_u20(np.empty(n + 16, np.int32), n + 16, inputs.config_seed(1))
    ar = Arena(page, {"a": a})
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    with paged(ar.host, page, frames) as h:
        for skip in (0, 12):                                                 # start off the page grid (16-byte aligned)
            B.gpuvm_reset(h)
            B.gpuvm_stream_sum_i32(h, ar.off["a"] + 4 * skip, n, out)
            st, ck = finish(h)
            assert int(out.item()) == oracle.stream_sum_i32_direct(a[skip:skip + n])
            touched = (4 * (skip + n) + page - 1) // page - (4 * skip) // page
            if frames >= touched:
                assert st["faults"] == touched and st["evictions"] == 0
                B.gpuvm_stream_sum_i32(h, ar.off["a"] + 4 * skip, n, out)     # all hits now
                st2, _ = finish(h)
                assert st2["faults"] == touched and int(out.item()) == oracle.stream_sum_i32_direct(a[skip:skip + n])
            else:
                assert st["faults"] >= touched and st["evictions"] >= touched - frames


@pytest.mark.parametrize("page,n,n_idx,block,frames", [
    (4096, 1 << 16, 1 << 14, 1024, 64),
    (4096, 1 << 16, (1 << 14) + 77, 1024, 16),     # ragged last block
    (256, 1 << 12, 5000, 100, 3),                  # block smaller than a CTA
    (65536, 1 << 20, 1 << 15, 1024, 16),
    (64, 4096, 3000, 1024, 1),                     # one frame: every warp fights for it
    (4096, 1 << 16, 9000, 3000, 5),                # blocks longer than one batch of 1024
])
@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("batched", [True, False])
def test_gather(B, page, n, n_idx, block, frames, policy, batched):
    import torch
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(2))
    idx = inputs.fill_index_i64(np.empty(n_idx, np.int64), n_idx, inputs.config_seed(2, 1), n)
    ar = Arena(page, {"x": x})
    nb = (n_idx + block - 1) // block
    fsum = torch.zeros(nb, dtype=torch.float32, device="cuda")
    bsum = torch.zeros(nb, dtype=torch.int64, device="cuda")
    with paged(ar.host, page, frames, policy) as h:
        run = B.gpuvm_gather_f32 if batched else B.gpuvm_gather_f32_unbatched
        run(h, ar.off["x"], dev(idx), n_idx, block, fsum, bsum)
        st, ck = finish(h)
    ref_f, ref_b = oracle.gather_block_sums_direct(x, idx, block)
    assert np.array_equal(bsum.cpu().numpy(), ref_b)                     # which elements: exact
    got = fsum.cpu().numpy().astype(np.float64)
    ref = ref_f.astype(np.float64)
    assert np.all(np.abs(got - ref) <= 1e-6 * np.maximum(np.abs(ref), 2.0 ** -10))
    distinct = np.unique((idx * 4) // page).size
    assert st["faults"] >= distinct and st["writebacks"] == 0
    if frames >= ar.n_pages:
        assert st["faults"] == distinct and st["evictions"] == 0        # compulsory misses only


@pytest.mark.parametrize("page,n,frames", [
    (4096, 1 << 16, 3 * 64),      # everything fits
    (4096, 1 << 16, 48),          # 4x oversubscribed: dirty victims are written back while running
    (4096, (1 << 14) + 500, 3),
    (512, 4096, 1),
    (65536, 1 << 18, 6),
])
@pytest.mark.parametrize("policy", POLICIES)
def test_vadd_writes_back_every_dirty_page(B, page, n, frames, policy):
    n = n // 4 * 4
    a = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4))
    b = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4, 1))
    ar = Arena(page, {"a": a, "b": b, "c": np.zeros(n, np.float32)})
    with paged(ar.host, page, frames, policy) as h:
        B.gpuvm_vadd_f32(h, ar.off["a"], ar.off["b"], ar.off["c"], n)
        st, ck = finish(h)
    ref = oracle.vadd_f32_direct(a, b)
    assert np.array_equal(ar.views["c"].view(np.uint32), ref.view(np.uint32))    # bit-exact
    assert np.array_equal(ar.views["a"], a) and np.array_equal(ar.views["b"], b)
    c_pages = (4 * n + page - 1) // page
    assert st["writebacks"] + st["flush_writebacks"] >= c_pages
    if frames >= ar.n_pages:                                  # every page once; c leaves eagerly or with the flush
        assert st["faults"] == ar.n_pages and st["writebacks"] + st["flush_writebacks"] == c_pages


@pytest.mark.parametrize("page,n,frames", [
    (512, 1 << 20, 10000),         # 24576 pages through 10000 frames
    (4096, (1 << 22) + 4096 + 512, 9600),   # last page of c is partial: fetched, not WRITE_ALL
    (512, 1 << 18, 20000),         # everything fits
])
def test_vadd_no_fetch_path_with_eager_write_back(B, page, n, frames):
    """With at least two frames per warp of the grid the kernel keeps the page of c pinned,
    does not fetch it (it is overwritten entirely) and writes it back as soon as it is done."""
    import torch
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert frames >= 2 * sms * 4 * 8
    a = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4))
    b = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4, 1))
    ar = Arena(page, {"a": a, "b": b, "c": np.full(n, 7.0, np.float32)})
    with paged(ar.host, page, frames) as h:
        B.gpuvm_vadd_f32(h, ar.off["a"], ar.off["b"], ar.off["c"], n)
        st, ck = finish(h)
    assert np.array_equal(ar.views["c"].view(np.uint32), oracle.vadd_f32_direct(a, b).view(np.uint32))
    assert np.array_equal(ar.views["a"], a) and np.array_equal(ar.views["b"], b)
    c_pages = (4 * n + page - 1) // page
    full_c_pages = (4 * n) // page
    assert st["writebacks"] == c_pages and st["flush_writebacks"] == 0       # every page of c left eagerly
    fetched_pages = st["bytes_in"] // page if 4 * n % page == 0 else None
    if fetched_pages is not None:
        assert fetched_pages == 2 * c_pages                                   # a and b only: c was not fetched
    assert st["faults"] >= 3 * full_c_pages


@pytest.mark.parametrize("page,n,frames", [(512, 1 << 20, 10000), (4096, 1 << 16, 3), (4096, (1 << 18) + 512, 20000)])
@pytest.mark.parametrize("target", ["a", "b"])
def test_vadd_in_place(B, page, n, frames, target):
    """c may be a or b itself: the sum replaces that input on the host, the other input stays.  A pool
    with room for the no-fetch path must not take it here (the page of c holds an operand)."""
    a = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4))
    b = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(4, 1))
    ar = Arena(page, {"a": a, "b": b})
    with paged(ar.host, page, frames) as h:
        B.gpuvm_vadd_f32(h, ar.off["a"], ar.off["b"], ar.off[target], n)
        st, ck = finish(h)
        # c overlapping an input in any other way is refused before anything runs
        for c_off in (ar.off["a"] + page, ar.off["b"] - page, ar.off["b"] + 4 * n - page):
            with pytest.raises(B.GpuvmError) as e:
                B.gpuvm_vadd_f32(h, ar.off["a"], ar.off["b"], c_off, n)
            assert e.value.status == B.E_ARG
    ref = oracle.vadd_f32_direct(a, b)
    other = "b" if target == "a" else "a"
    assert np.array_equal(ar.views[target].view(np.uint32), ref.view(np.uint32))
    assert np.array_equal(ar.views[other], {"a": a, "b": b}[other])
    assert st["bytes_in"] >= 8 * n                                          # both operands were fetched


def small_graphs():
    rng = np.random.default_rng(24)
    yield 1, [], 0
    yield 5, [(0, 0), (0, 1), (0, 1), (1, 2), (3, 4)], 0
    yield 5, [(1, 0), (2, 1)], 0
    for _ in range(3):
        nv = int(rng.integers(2, 40))
        ne = int(rng.integers(0, 200))
        yield nv, [(int(rng.integers(0, nv)), int(rng.integers(0, nv))) for _ in range(ne)], int(rng.integers(0, nv))


def csr(nv, edges):
    off = np.zeros(nv + 1, dtype=np.int64)
    for u, _ in edges:
        off[u + 1] += 1
    off = np.cumsum(off).astype(np.int64)
    col = np.zeros(max(len(edges), 4), dtype=np.int32)
    cur = off[:-1].copy()
    for u, v in edges:
        col[cur[u]] = v
        cur[u] += 1
    return off, col


def run_bfs(B, off, col, src, page, frames, policy):
    import torch
    nv = off.size - 1
    off_p = np.zeros((off.size + 1) // 2 * 2, np.int64)
    off_p[:off.size] = off
    col_p = np.zeros((col.size + 3) // 4 * 4, np.int32)
    col_p[:col.size] = col
    ar = Arena(page, {"off": off_p, "col": col_p})
    level = torch.zeros(nv, dtype=torch.int32, device="cuda")
    with paged(ar.host, page, frames, policy) as h:
        depth = B.gpuvm_bfs_csr(h, ar.off["off"], ar.off["col"], nv, src, level)
        st, ck = finish(h)
    return level.cpu().numpy(), depth, st


@pytest.mark.parametrize("policy", POLICIES)
def test_bfs_small_graphs(B, policy):
    for nv, edges, src in small_graphs():
        off, col = csr(nv, edges)
        ref = oracle.bfs_levels_direct(off, col, src)
        for page, frames in ((64, 1), (64, 4), (4096, 8)):
            got, depth, st = run_bfs(B, off, col, src, page, frames, policy)
            assert np.array_equal(got, ref)
            assert depth == ref.max() + 1


@pytest.mark.parametrize("scale,page,frames", [(12, 4096, 20), (14, 4096, 9), (14, 65536, 5)])
def test_bfs_rmat_with_hub_vertices(B, scale, page, frames):
    off, col = inputs.rmat_csr(scale, 16 << scale, inputs.config_seed(3))
    assert np.diff(off).max() >= 4096 or scale < 14          # the grid-wide path is exercised
    ref = oracle.bfs_levels_direct(off, col, 0)
    got, depth, st = run_bfs(B, off, col, 0, page, frames, 1)
    assert np.array_equal(got, ref)
    assert st["writebacks"] == 0


def graph_arena(page, off, col, weight=None):
    off_p = np.zeros((off.size + 1) // 2 * 2, np.int64)
    off_p[:off.size] = off
    pad4 = lambda a: np.concatenate([a, np.zeros((-a.size) % 4, a.dtype)])
    arrays = {"off": off_p, "col": pad4(col)}
    if weight is not None:
        arrays["w"] = pad4(weight)
    return Arena(page, arrays)


@pytest.mark.parametrize("policy", POLICIES)
def test_bfs_over_balanced_csr(B, policy):
    """Same levels as the oracle's BFS when workers take equal-size edge chunks instead of vertices."""
    import torch
    graphs = [csr(nv, edges) + (src,) for nv, edges, src in small_graphs()]
    graphs.append(inputs.rmat_csr(12, 16 << 12, inputs.config_seed(3)) + (0,))
    graphs.append(inputs.rmat_csr(14, 16 << 14, inputs.config_seed(3)) + (7,))
    for off, col, src in graphs:
        nv, ne = off.size - 1, int(off[-1])
        ref = oracle.bfs_levels_direct(off, col, src)
        for page, chunk_edges, frames in ((64, 16, 1), (64, 4, 3), (4096, 1024, 5), (4096, 256, 64)):
            chunks = B.gpuvm_bcsr_build(off, chunk_edges)
            # brute-force check of the chunk table: the owner of edge e is the vertex with off[v] <= e < off[v+1]
            for c in range(min(chunks.size - 1, 50)):
                v = int(chunks[c])
                assert off[v] <= c * chunk_edges < off[v + 1]
            off_p = np.zeros((off.size + 1) // 2 * 2, np.int64)
            off_p[:off.size] = off
            pad4 = lambda a: np.concatenate([a, np.zeros((-a.size) % 4, a.dtype)])
            ar = Arena(page, {"off": off_p, "col": pad4(col), "chunk": pad4(chunks)})
            level = torch.zeros(nv, dtype=torch.int32, device="cuda")
            label = torch.zeros(nv, dtype=torch.int32, device="cuda")
            with paged(ar.host, page, frames, policy) as h:
                depth = B.gpuvm_bfs_bcsr(h, ar.off["off"], ar.off["col"], ar.off["chunk"], nv, ne, chunk_edges, src, level)
                st, ck = finish(h)
                B.gpuvm_cc_bcsr(h, ar.off["off"], ar.off["col"], ar.off["chunk"], nv, ne, chunk_edges, label)
                finish(h)
            assert np.array_equal(level.cpu().numpy(), ref), (nv, ne, page, chunk_edges, frames)
            assert depth == ref.max() + 1
            assert np.array_equal(label.cpu().numpy(), oracle.cc_labels_direct(off, col)), (nv, ne, page)
    # a chunk that would straddle pages is refused
    with paged(ar.host, 4096, 8) as h:
        with pytest.raises(B.GpuvmError) as e:
            B.gpuvm_bfs_bcsr(h, ar.off["off"], ar.off["col"], ar.off["chunk"], nv, ne, 1536, src, level)
        assert e.value.status == B.E_ALIGN


@pytest.mark.parametrize("policy", POLICIES)
def test_cc_small_graphs_and_rmat(B, policy):
    import torch
    cases = [(nv, edges) for nv, edges, _ in small_graphs()]
    graphs = [csr(nv, edges) for nv, edges in cases]
    graphs.append(inputs.rmat_csr(12, 4 << 12, inputs.config_seed(3)))      # sparse: many components
    graphs.append(inputs.rmat_csr(14, 16 << 14, inputs.config_seed(3)))     # hub vertices: long lists are split
    for off, col in graphs:
        nv = off.size - 1
        ref = oracle.cc_labels_direct(off, col[:max(int(off[-1]), 0)] if off[-1] else col)
        for page, frames in ((64, 1), (4096, 6), (65536, 3)):
            ar = graph_arena(page, off, col)
            label = torch.zeros(nv, dtype=torch.int32, device="cuda")
            with paged(ar.host, page, frames, policy) as h:
                sweeps = B.gpuvm_cc_csr(h, ar.off["off"], ar.off["col"], nv, label)
                st, ck = finish(h)
            assert np.array_equal(label.cpu().numpy(), ref)
            assert sweeps >= 1 and st["writebacks"] == 0


@pytest.mark.parametrize("policy", POLICIES)
def test_sssp_small_graphs_and_rmat(B, policy):
    import torch
    graphs = [csr(nv, edges) + (src,) for nv, edges, src in small_graphs()]
    graphs.append(inputs.rmat_csr(12, 8 << 12, inputs.config_seed(3)) + (0,))
    graphs.append(inputs.rmat_csr(14, 16 << 14, inputs.config_seed(3)) + (0,))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    need = 2 * sms * 2 * 8                                   # two frames per warp of the grid
    for off, col, src in graphs:
        nv = off.size - 1
        weight = inputs.fill_i32_range(np.empty(col.size, np.int32), col.size, inputs.config_seed(3, 2), 1, 255)
        ref = oracle.sssp_direct(off, col, weight, src)
        for page in (64, 4096):
            ar = graph_arena(page, off, col, weight)
            dist = torch.zeros(nv, dtype=torch.int32, device="cuda")
            with paged(ar.host, page, need + 3, policy) as h:
                rounds = B.gpuvm_sssp_csr(h, ar.off["off"], ar.off["col"], ar.off["w"], nv, src, dist)
                st, ck = finish(h)
            assert np.array_equal(dist.cpu().numpy(), ref)
            assert rounds >= 1
    # a pool that cannot hold two pages per warp is refused, nothing runs
    ar = graph_arena(4096, *graphs[1][:2], np.ones(graphs[1][1].size, np.int32))
    with paged(ar.host, 4096, 8) as h:
        with pytest.raises(B.GpuvmError) as e:
            B.gpuvm_sssp_csr(h, ar.off["off"], ar.off["col"], ar.off["w"], graphs[1][0].size - 1, 0,
                             torch.zeros(8, dtype=torch.int32, device="cuda"))
        assert e.value.status == B.E_FRAMES


@pytest.mark.parametrize("page,n_rows,n_bags,frames,dims,bag", [
    (4096, 512, 64, 64, 128, 32),
    (4096, 4096, 1000, 8, 128, 32),
    (2 << 20, 1 << 14, 1 << 12, 2, 128, 32),
    (512, 100, 33, 1, 128, 32),
    (4096, 2000, 70, 16, 128, 40),                 # bags longer than one batch of 32 lookups
    (4096, 2000, 70, 16, 64, 5),                   # narrow rows, short bags
    (4096, 3000, 200, 9, 20, 7),                   # 80-byte rows straddle pages
    (4096, 1000, 200, 5, 100, 32),                 # 400-byte rows straddle pages
    (256, 300, 64, 6, 128, 32),                    # pages smaller than a row
    (256, 300, 64, 1, 128, 3),                     # ... and a single frame
])
@pytest.mark.parametrize("batched", [True, False])
def test_embag(B, page, n_rows, n_bags, frames, dims, bag, batched):
    import torch
    t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, inputs.config_seed(5))
    rows = inputs.fill_zipf_rows(np.empty(n_bags * bag, np.int64), n_bags * bag, inputs.config_seed(5, 1), n_rows, 1.05)
    ar = Arena(page, {"t": t})
    out = torch.zeros(n_bags * dims, dtype=torch.float32, device="cuda")
    with paged(ar.host, page, frames) as h:
        run = B.gpuvm_embag_f32 if batched else B.gpuvm_embag_f32_unbatched
        run(h, ar.off["t"], dims, dev(rows), n_bags, bag, out)
        st, ck = finish(h)
    ref = oracle.embag_f32_direct(t.reshape(n_rows, dims), rows, bag).reshape(-1)
    got = out.cpu().numpy()
    assert np.all(np.abs(got.astype(np.float64) - ref) <= 1e-6 * np.maximum(np.abs(ref), 2.0 ** -10))
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))     # same order of additions: same bits
    # every looked-up row crossed the link, as part of a fetched page or read in place
    touched = np.unique(rows * dims * 4 // page).size
    assert st["faults"] * page + st["bytes_direct"] >= touched * min(page, 4 * dims)
    if not batched:
        assert st["bytes_direct"] == 0 and st["faults"] >= touched


@pytest.mark.parametrize("counted", [2, 1, 0])
@pytest.mark.parametrize("frames", [1, 4, 64])
def test_embag_rent_or_buy(B, frames, counted):
    """The batched embedding bag does not fetch a page for a few rows.  Counted (default): the lookups per page are
    counted first; rows of pages below the limit (page / divisor / row size) are read in place, all of them, and the
    other pages are fetched once.  With counted = 2 (the default) the rows in place are read page by page and the
    divisor is 1 unless set otherwise; with counted = 1 they are read as their lookups come up and it is 4.  Online: the
    first `limit` requests that find a page absent read their rows in place, the next one fetches it.  Divisor 0:
    every first touch fetches, as in the paper.  Results are exact either way."""
    import torch
    page, dims, bag = 4096, 128, 4                       # 8 rows per page; a quarter of a page = 2 rows
    n_rows = 512
    t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, inputs.config_seed(5))
    ar = Arena(page, {"t": t})
    cold = np.arange(0, n_rows, 8, dtype=np.int64)[:64]                      # one row of each of 64 pages
    hot = np.full(1024, 17, dtype=np.int64)                                   # one page, over and over
    mixed = np.concatenate([cold, hot, cold + 1])
    for rows, name in ((cold, "cold"), (hot, "hot"), (mixed, "mixed")):
        n_bags = rows.size // bag
        ref = oracle.embag_f32_direct(t.reshape(n_rows, dims), rows, bag).reshape(-1)
        per_page = np.bincount(rows // 8, minlength=ar.n_pages)
        for divisor in (None, 2, 0, 8):
            out = torch.zeros(n_bags * dims, dtype=torch.float32, device="cuda")
            with paged(ar.host, page, frames) as h:
                B.gpuvm_set_inplace_counted(h, counted)
                if divisor is None:
                    divisor = 1 if counted == 2 else 4                         # the default: 1 when the rows in place are read page by page
                else:
                    B.gpuvm_set_inplace_divisor(h, divisor)
                B.gpuvm_embag_f32(h, 0, dims, dev(rows), n_bags, bag, out)
                st, ck = finish(h)
            assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32)), (name, divisor)
            limit = page // divisor // 512 if divisor else 0                  # rows of a page that are read in place
            assert st["bytes_direct"] % 512 == 0
            if divisor == 0:
                assert st["bytes_direct"] == 0 and st["faults"] >= np.count_nonzero(per_page)
            elif counted:
                bought = np.count_nonzero(per_page >= limit)
                assert st["bytes_direct"] == int(per_page[per_page < limit].sum()) * 512
                assert st["faults"] >= bought and (frames < bought or st["faults"] == bought)
            elif name == "cold":                                               # one row per page: below any limit
                assert st["faults"] == 0 and st["bytes_direct"] == rows.size * 512
            elif name == "hot":                                                # the page is bought after `limit` rows
                assert st["faults"] >= 1
                assert limit * 512 <= st["bytes_direct"] <= (limit + 31) * 512 * st["faults"]


def test_embag_direct_form_stages_only_the_rows_read_in_place(B):
    """When the pages that are fetched fit the pool twice over, the default policy holds them in their frames and
    adds their rows up from there: the scratch is the rows read in place plus a few bytes per lookup, not a staged
    copy of every row; with a pool too small for that the form with request tables runs and stages every row.
    Either way the hold bits are gone afterwards (the checker would flag one) and the sums are the oracle's."""
    import torch
    page, dims, bag, n_rows, n_bags = 4096, 128, 8, 4096, 1500
    t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, inputs.config_seed(5))
    rows = inputs.fill_zipf_rows(np.empty(n_bags * bag, np.int64), n_bags * bag, inputs.config_seed(5, 1), n_rows, 1.05)
    ref = oracle.embag_f32_direct(t.reshape(n_rows, dims), rows, bag).reshape(-1)
    per_page = np.bincount(rows // 8, minlength=n_rows // 8)
    hot, cold_rows = int(np.count_nonzero(per_page >= 8)), int(per_page[per_page < 8].sum())
    assert hot > 4 and cold_rows > 1000
    ar = Arena(page, {"t": t})
    every_row = n_bags * bag * dims * 4
    for frames, direct in ((2 * hot, True), (2 * hot - 1, False)):
        out = torch.zeros(n_bags * dims, dtype=torch.float32, device="cuda")
        with paged(ar.host, page, frames) as h:
            B.gpuvm_embag_f32(h, 0, dims, dev(rows), n_bags, bag, out)
            st, ck = finish(h)
            scratch = B.gpuvm_scratch_bytes(h)
        assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32)), frames
        assert ck["bad_state"] == 0 and st["bytes_direct"] == cold_rows * 512
        if direct:
            assert st["faults"] == hot and cold_rows * 512 <= scratch < cold_rows * 512 + every_row // 4 + (1 << 20)
        else:
            assert scratch >= every_row


def test_embag_writes_its_sums_to_pinned_host_memory(B):
    """d_out may be pinned host memory: the kernel writes the bags' sums there itself, same bits."""
    import torch
    page, dims, bag, n_rows, n_bags = 4096, 128, 8, 2048, 300
    t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, inputs.config_seed(5))
    rows = inputs.fill_zipf_rows(np.empty(n_bags * bag, np.int64), n_bags * bag, inputs.config_seed(5, 1), n_rows, 1.05)
    ref = oracle.embag_f32_direct(t.reshape(n_rows, dims), rows, bag).reshape(-1)
    ar = Arena(page, {"t": t})
    for counted in (2, 1, 0):
        out = torch.zeros(n_bags * dims, dtype=torch.float32).pin_memory()
        with paged(ar.host, page, 16) as h:
            B.gpuvm_set_inplace_counted(h, counted)
            B.gpuvm_embag_f32(h, 0, dims, dev(rows), n_bags, bag, out)
            finish(h)
        torch.cuda.synchronize()
        assert np.array_equal(out.numpy().view(np.uint32), ref.view(np.uint32)), counted


def test_embag_rows_past_the_end_and_tables_off_the_row_grid(B):
    """A row id whose row does not lie inside the backing store sets the sticky range error (batched
    and unbatched); a table that starts off the row grid of its page is still summed correctly."""
    import torch
    page, dims, bag, n_rows, n_bags = 4096, 128, 4, 64, 8
    t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, inputs.config_seed(5))
    rows = (np.arange(n_bags * bag, dtype=np.int64) * 7) % n_rows
    out = torch.zeros(n_bags * dims, dtype=torch.float32, device="cuda")
    for batched in (True, False):
        bad = rows.copy()
        bad[5] = n_rows                                                     # first row past the end
        ar = Arena(page, {"t": t})
        with paged(ar.host, page, 4) as h:
            (B.gpuvm_embag_f32 if batched else B.gpuvm_embag_f32_unbatched)(h, 0, dims, dev(bad), n_bags, bag, out)
            B.gpuvm_flush(h)
            with pytest.raises(B.GpuvmError) as e:
                B.gpuvm_stats(h)
            assert e.value.status == B.E_RANGE
            assert B.gpuvm_check(h)["status"] == 0                          # nothing left pinned or in transit
    # table at byte 16 of the arena: rows straddle pages although the row size divides the page size
    shifted = np.concatenate([np.zeros(4, np.float32), t])
    ar = Arena(page, {"t": shifted})
    with paged(ar.host, page, 3) as h:
        B.gpuvm_embag_f32(h, 16, dims, dev(rows), n_bags, bag, out)
        finish(h)
    ref = oracle.embag_f32_direct(t.reshape(n_rows, dims), rows, bag).reshape(-1)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("page,n,frames", [(4096, 1 << 16, 64), (4096, 1 << 16, 7), (64, 2048, 1), (1024, 50000, 13),
                                           (1 << 18, 1 << 22, 5)])           # 256 KiB pages: the grid-wide ring too
@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("batched", [False, True, "queued"])
def test_scatter_update_through_element_accessors(B, page, n, frames, policy, batched):
    n = n // 4 * 4
    a = (inputs.fill_i32_u20(np.empty(n, np.int32), n, 77)).astype(np.uint32)
    perm = np.random.default_rng(3).permutation(n)[: (3 * n) // 4].astype(np.int64)
    ar = Arena(page, {"a": a})
    with paged(ar.host, page, frames, policy) as h:
        run = {False: B.gpuvm_scatter_update_u32, True: B.gpuvm_scatter_update_u32_batched,
               "queued": B.gpuvm_scatter_update_u32_queued}[batched]
        run(h, ar.off["a"], dev(perm), perm.size)
        st, ck = finish(h)
    ref = a.copy()
    ref[perm] = ref[perm] * np.uint32(3) + np.uint32(1)
    assert np.array_equal(ar.views["a"], ref)                           # no dirty data lost
    assert st["faults"] >= np.unique(perm * 4 // page).size


@pytest.mark.parametrize("page,n,frames,ahead", [(4096, 1 << 18, 64, 16), (4096, 1 << 18, 7, 4), (64, 4096, 2, 1),
                                                 (1 << 16, 1 << 22, 9, 3)])
@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("form", ["single", "batched", "queued"])
def test_write_back_off_the_fault_path(B, page, n, frames, ahead, policy, form):
    """With the cleaners on (gpuvm_set_clean_ahead) idle warps write dirty pages back ahead of the head
    cursor: the host array still ends up exact (no dirty data lost, none written back stale), the
    invariants hold, and every write-back is counted on one side or the other."""
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 78).astype(np.uint32)
    perm = np.random.default_rng(5).permutation(n)[: (3 * n) // 4].astype(np.int64)
    ar = Arena(page, {"a": a})
    with paged(ar.host, page, frames, policy) as h:
        B.gpuvm_set_clean_ahead(h, ahead)
        assert B.gpuvm_device_view(h).clean_ahead == min(ahead, frames)
        run = {"single": B.gpuvm_scatter_update_u32, "batched": B.gpuvm_scatter_update_u32_batched,
               "queued": B.gpuvm_scatter_update_u32_queued}[form]
        run(h, ar.off["a"], dev(perm), perm.size)
        st, ck = finish(h)
    ref = a.copy()
    ref[perm] = ref[perm] * np.uint32(3) + np.uint32(1)
    assert np.array_equal(ar.views["a"], ref)
    dirty_pages = np.unique(perm * 4 // page).size
    assert st["writebacks"] + st["cleaned"] + st["flush_writebacks"] >= dirty_pages
    assert st["bytes_out"] == (st["writebacks"] + st["cleaned"] + st["flush_writebacks"]) * page


@pytest.mark.parametrize("frames", [1, 6, 64])
def test_fenced_release_gives_the_same_results(B, frames):
    """The batched engine normally releases the pages of read-only requests through a data dependency on
    what was read; with GPUVM_DEBUG_FENCED_RELEASE it uses a warp barrier and a fence instead (the form
    the memory model orders by itself).  Both must give the oracle's results, bit for bit."""
    import torch
    page, n, n_idx, dims, bag, n_bags = 4096, 1 << 16, 20000, 128, 8, 100
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(2))
    idx = inputs.fill_index_i64(np.empty(n_idx, np.int64), n_idx, inputs.config_seed(2, 1), n)
    rows = inputs.fill_zipf_rows(np.empty(n_bags * bag, np.int64), n_bags * bag, inputs.config_seed(5, 1), n // dims, 1.05)
    ar = Arena(page, {"x": x})
    nb = (n_idx + 1023) // 1024
    ref_f, ref_b = oracle.gather_block_sums_direct(x, idx, 1024)
    ref_e = oracle.embag_f32_direct(x.reshape(n // dims, dims), rows, bag).reshape(-1)
    for flags in (0, B.DEBUG_FENCED_RELEASE, B.DEBUG_FENCED_RELEASE | B.DEBUG_POISON):
        fs = torch.zeros(nb, dtype=torch.float32, device="cuda")
        bs = torch.zeros(nb, dtype=torch.int64, device="cuda")
        out = torch.zeros(n_bags * dims, dtype=torch.float32, device="cuda")
        with paged(ar.host, page, frames) as h:
            B.gpuvm_set_debug(h, flags)
            assert B.gpuvm_device_view(h).debug == flags
            B.gpuvm_gather_f32(h, 0, dev(idx), n_idx, 1024, fs, bs)
            B.gpuvm_embag_f32(h, 0, dims, dev(rows), n_bags, bag, out)
            finish(h)
        assert np.array_equal(bs.cpu().numpy(), ref_b), flags
        got = fs.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref_f) <= 1e-6 * np.maximum(np.abs(ref_f), 2.0 ** -10))
        assert np.array_equal(out.cpu().numpy().view(np.uint32), ref_e.view(np.uint32)), flags


@pytest.mark.parametrize("frames", [2, 64])
def test_read_n_hits_misses_and_fenced_mode(B, frames):
    """The one-request-per-lane gather issues four reads per lane together (gpuvm_read_n): a second pass over a
    pool that holds everything is served by hits alone (one per request), a pool of two frames sends almost
    every slot through the full path, and the fenced debug mode (fences instead of dependency order around the
    loads) gives the same bits."""
    import torch
    page, n, n_idx = 4096, 1 << 16, 20000 + 13
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(2))
    idx = inputs.fill_index_i64(np.empty(n_idx, np.int64), n_idx, inputs.config_seed(2, 1), n)
    ar = Arena(page, {"x": x})
    nb = (n_idx + 1023) // 1024
    ref_f, ref_b = oracle.gather_block_sums_direct(x, idx, 1024)
    for flags in (0, B.DEBUG_FENCED_RELEASE):
        fs = torch.zeros(nb, dtype=torch.float32, device="cuda")
        bs = torch.zeros(nb, dtype=torch.int64, device="cuda")
        with paged(ar.host, page, frames) as h:
            B.gpuvm_set_debug(h, flags)
            B.gpuvm_gather_f32_unbatched(h, 0, dev(idx), n_idx, 1024, fs, bs)
            st1, _ = finish(h)
            assert np.array_equal(bs.cpu().numpy(), ref_b), flags
            bs.zero_()
            B.gpuvm_gather_f32_unbatched(h, 0, dev(idx), n_idx, 1024, fs, bs)
            st2, _ = finish(h)
        assert np.array_equal(bs.cpu().numpy(), ref_b), flags
        got = fs.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref_f) <= 1e-6 * np.maximum(np.abs(ref_f), 2.0 ** -10))
        if frames >= ar.n_pages:
            assert st2["faults"] == st1["faults"] == np.unique(idx * 4 // page).size
            assert st2["hits"] - st1["hits"] == n_idx          # every request of the second pass is a hit of its own
        else:
            assert st2["faults"] > st1["faults"] > frames


def test_two_kernels_share_mappings(B):
    """Mappings persist across launches: a read-only pass after a write pass sees the
    written values without any flush in between."""
    import torch
    page, n, frames = 4096, 1 << 14, 8
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 5).astype(np.uint32)
    idx = np.arange(n, dtype=np.int64)
    ar = Arena(page, {"a": a})
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    with paged(ar.host, page, frames) as h:
        B.gpuvm_scatter_update_u32(h, 0, dev(idx), n)
        B.gpuvm_stream_sum_i32(h, 0, n, out)
        st, ck = finish(h)
    ref = (a * np.uint32(3) + np.uint32(1)).view(np.int32)
    assert int(out.item()) == int(ref.astype(np.int64).sum())
    assert np.array_equal(ar.views["a"].view(np.int32), ref)
