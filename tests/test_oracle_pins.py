"""Pins for the CPU oracle: each test checks it against something other than itself --
textbook fault counts, an independently formulated model, brute force, a closed form,
a library routine, or an invariant the paper states."""
import collections
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2411_05309_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [c.strip() for c in line.split("|")]


def make_pager(n_pages, page_bytes, n_frames, policy, move=True, fill=None):
    host = np.zeros(n_pages * page_bytes, dtype=np.uint8) if fill is None else fill
    return oracle.Pager(host, page_bytes, n_frames, policy, move)


# ------------------------------------------------------------ independent models

def belady_opt_faults(trace, frames):
    """Brute-force optimal replacement: evict the page whose next use is farthest."""
    resident, faults = set(), 0
    for i, p in enumerate(trace):
        if p in resident:
            continue
        faults += 1
        if len(resident) == frames:
            def next_use(q):
                for j in range(i + 1, len(trace)):
                    if trace[j] == q:
                        return j
                return float("inf")
            resident.remove(max(resident, key=next_use))
        resident.add(p)
    return faults


def fifo_list_model(trace, frames):
    """List-based FIFO: the oldest resident page leaves."""
    order, faults, evicted = collections.deque(), 0, []
    for p in trace:
        if p in order:
            continue
        faults += 1
        if len(order) == frames:
            evicted.append(order.popleft())
        order.append(p)
    return faults, evicted


def second_chance_queue_model(trace, frames):
    """Second chance in its queue formulation: on a fault the head of the FIFO queue is
    inspected; a referenced head loses its bit and goes to the tail, an unreferenced head
    is evicted.  New pages enter at the tail with the bit set."""
    queue, ref, faults, evicted = collections.deque(), {}, 0, []
    for p in trace:
        if p in ref:
            ref[p] = 1
            continue
        faults += 1
        if len(queue) == frames:
            while True:
                q = queue.popleft()
                if ref[q]:
                    ref[q] = 0
                    queue.append(q)
                else:
                    del ref[q]
                    evicted.append(q)
                    break
        queue.append(p)
        ref[p] = 1
    return faults, evicted


def oracle_faults(trace, frames, policy):
    n_pages = max(trace) + 1
    pg = make_pager(n_pages, 16, frames, policy)
    resident_ok = True
    for p in trace:
        pg.access(p)
        c = pg.counters()
        resident_ok &= c["resident"] <= frames and pg.check() == 0
    assert resident_ok
    return pg.counters()


# ------------------------------------------------------------------------- pins

@pytest.mark.parametrize("row", list(_rows("page_replacement_strings.txt")))
def test_textbook_reference_strings(row):
    _, frames, policy, faults, string = row
    trace = [int(t) for t in string.split()]
    frames, faults = int(frames), int(faults)
    if policy == "fifo":
        assert oracle_faults(trace, frames, oracle.FIFO)["faults"] == faults
        assert fifo_list_model(trace, frames)[0] == faults
    else:
        assert belady_opt_faults(trace, frames) == faults
        # OPT is a lower bound for both policies of the oracle
        assert oracle_faults(trace, frames, oracle.FIFO)["faults"] >= faults
        assert oracle_faults(trace, frames, oracle.CLOCK)["faults"] >= faults


@pytest.mark.parametrize("row", list(_rows("paper_closed_forms.txt")))
def test_closed_forms_printed_in_the_paper(row):
    name, args, printed = row
    a = [float(t) for t in args.split()]
    if name == "queue_depth":
        depth = oracle.queue_depth(a[0], a[1] * 2 ** 30, a[2] * 2 ** 10)
        assert int(depth) == int(printed)              # 72.35 -> 72, 36.18 -> 36
        assert abs(depth - {4: 72.35, 8: 36.18}[int(a[2])]) < 0.01
    else:
        assert oracle.oversubscription_level(a[0], a[1]) == float(printed)


def random_traces():
    rng = np.random.default_rng(2411)
    for n_pages in (1, 2, 5, 9, 17):
        for length in (1, 7, 60):
            yield list(rng.integers(0, n_pages, length))
    yield list(range(12)) * 3                       # cyclic sweep
    yield list(range(12)) + list(range(11, -1, -1))  # forward then reverse
    yield [3] * 20                                  # one page repeated
    yield list(range(0, 24, 5)) * 4                 # strided
    z = rng.zipf(1.3, 200)
    yield [int(v) % 23 for v in z]


@pytest.mark.parametrize("frames", [1, 2, 3, 4, 8, 16, 17, 18])
def test_fifo_and_clock_against_independent_models(frames):
    for trace in random_traces():
        trace = [int(t) for t in trace]
        f = oracle_faults(trace, frames, oracle.FIFO)
        c = oracle_faults(trace, frames, oracle.CLOCK)
        mf, evf = fifo_list_model(trace, frames)
        mc, evc = second_chance_queue_model(trace, frames)
        assert f["faults"] == mf and f["evictions"] == len(evf)
        assert c["faults"] == mc and c["evictions"] == len(evc)
        opt = belady_opt_faults(trace, frames)
        assert opt <= f["faults"] and opt <= c["faults"]
        distinct = len(set(trace))
        for got in (f, c):
            assert got["faults"] >= distinct
            assert got["max_resident"] <= frames
            assert got["accesses"] == len(trace) == got["hits"] + got["faults"]
            assert got["evictions"] == got["faults"] - got["resident"]
            if frames >= distinct:                   # compulsory misses only
                assert got["faults"] == distinct and got["evictions"] == 0


def test_eviction_order_matches_models():
    """Not only how many pages leave but which ones, in which order."""
    rng = np.random.default_rng(7)
    trace = [int(t) for t in rng.integers(0, 11, 300)]
    for frames in (1, 2, 3, 5, 10):
        for policy, model in ((oracle.FIFO, fifo_list_model), (oracle.CLOCK, second_chance_queue_model)):
            pg = make_pager(11, 16, frames, policy)
            owner, evicted = {}, []
            for p in trace:
                f = pg.access(p)
                assert 0 <= f < frames
                if owner.get(f) != p:              # the frame changed hands: its occupant left
                    if f in owner:
                        evicted.append(owner[f])
                    owner[f] = p
            faults, model_evicted = model(trace, frames)
            assert pg.counters()["faults"] == faults
            assert evicted == model_evicted
            pg.close()


def test_paged_workloads_equal_direct_results_and_host_is_complete():
    rng = np.random.default_rng(3)
    for page_bytes in (16, 64, 256):
        for n in (4, 64, 257 * 4):
            for frames in (1, 2, 3, 7, 1000):
                for policy in (oracle.FIFO, oracle.CLOCK):
                    pad = lambda b: (b + page_bytes - 1) // page_bytes * page_bytes
                    a = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 1)
                    b = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 2)
                    a_off, b_off, c_off = 0, pad(4 * n), 2 * pad(4 * n)
                    host = np.zeros(3 * pad(4 * n), dtype=np.uint8)
                    host[a_off:a_off + 4 * n] = np.frombuffer(a.tobytes(), np.uint8)
                    host[b_off:b_off + 4 * n] = np.frombuffer(b.tobytes(), np.uint8)
                    before = host.copy()
                    pg = oracle.Pager(host, page_bytes, frames, policy, True)
                    pg.vadd_f32(a_off, b_off, c_off, n)
                    assert pg.check() == 0
                    cnt = pg.counters()
                    pg.flush()
                    c = host[c_off:c_off + 4 * n].view(np.float32)
                    assert np.array_equal(c, a + b)                      # numpy: IEEE binary32 add
                    assert np.array_equal(c, oracle.vadd_f32_direct(a, b))
                    assert np.array_equal(host[:c_off], before[:c_off])  # a, b untouched
                    after = pg.counters()
                    c_pages = pad(4 * n) // page_bytes
                    assert after["writebacks"] >= c_pages                # every c page reached the host
                    assert after["writebacks"] <= cnt["evictions"] + min(frames, c_pages)
                    assert cnt["max_resident"] <= frames
                    pg.close()


def test_read_only_workloads_never_write_back():
    n = 3000
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 4)
    host = np.frombuffer(a.tobytes(), np.uint8).copy()
    before = host.copy()
    for frames in (1, 2, 5, 100):
        pg = oracle.Pager(host, 64, frames, oracle.CLOCK, True)
        s = pg.stream_sum_i32(0, n)
        pg.flush()
        assert s == int(a.astype(np.int64).sum()) == oracle.stream_sum_i32_direct(a)
        cnt = pg.counters()
        assert cnt["writebacks"] == 0 and cnt["bytes_out"] == 0
        assert np.array_equal(host, before)
        # a single sequential pass touches each page in one burst: one fault per page
        assert cnt["faults"] == (4 * n + 63) // 64
        pg.close()


def test_stream_sum_closed_form():
    n = 100001
    a = np.arange(n, dtype=np.int32)
    assert oracle.stream_sum_i32_direct(a) == n * (n - 1) // 2
    a = np.full(1 << 16, (1 << 20) - 1, dtype=np.int32)       # beyond 32 bits
    assert oracle.stream_sum_i32_direct(a) == (1 << 16) * ((1 << 20) - 1)
    a = np.array([-5, 3, -(1 << 31), (1 << 31) - 1], dtype=np.int32)
    assert oracle.stream_sum_i32_direct(a) == -3


def test_gather_against_numpy_and_exact_summation():
    import math
    n, m, block = 5000, 4096 + 100, 1024
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 8)
    idx = inputs.fill_index_i64(np.empty(m, np.int64), m, 9, n)
    fsum, bsum = oracle.gather_block_sums_direct(x, idx, block)
    assert fsum.size == bsum.size == 5                         # ragged last block
    g = x[idx]
    for b in range(5):
        seg = g[b * block:(b + 1) * block]
        exact = math.fsum(float(v) for v in seg)              # correctly rounded sum
        assert abs(float(fsum[b]) - exact) <= 2 ** -24 * max(abs(exact), 2 ** -10) * 1.01
        assert int(bsum[b]) == int(seg.view(np.uint32).astype(np.int64).sum())
    # a transposed operand (x[idx] vs idx[x]) or dropped element changes bsum
    host = np.frombuffer(x.tobytes(), np.uint8).copy()
    for frames in (1, 3, 1000):
        pg = oracle.Pager(host, 256, frames, oracle.CLOCK, True)
        f2, b2 = pg.gather_block_sums(0, idx, block)
        assert np.array_equal(f2, fsum) and np.array_equal(b2, bsum)
        pg.close()


def relax_levels(nv, edges, source):
    """V rounds of edge relaxation (Bellman-Ford on unit weights)."""
    INF = 10 ** 9
    d = [INF] * nv
    d[source] = 0
    for _ in range(nv):
        for u, v in edges:
            if d[u] + 1 < d[v]:
                d[v] = d[u] + 1
    return [x if x < INF else -1 for x in d]


def csr_from_edges(nv, edges):
    off = np.zeros(nv + 1, dtype=np.int64)
    for u, _ in edges:
        off[u + 1] += 1
    off = np.cumsum(off).astype(np.int64)
    col = np.zeros(max(len(edges), 1), dtype=np.int32)
    cur = off[:-1].copy()
    for u, v in edges:
        col[cur[u]] = v
        cur[u] += 1
    return off, col


def test_bfs_against_relaxation_scipy_and_paged():
    from scipy.sparse import csr_matrix
    from scipy.sparse.csgraph import shortest_path
    rng = np.random.default_rng(17)
    cases = [
        (1, [], 0),
        (4, [], 2),                                            # no edges at all
        (5, [(0, 0), (0, 1), (0, 1), (1, 2), (3, 4)], 0),      # self loop, duplicate, unreachable
        (5, [(1, 0), (2, 1)], 0),                              # source with zero out-degree
        (6, [(0, 1), (1, 2), (2, 3), (3, 4), (4, 5), (0, 5)], 0),
    ]
    for _ in range(20):
        nv = int(rng.integers(2, 17))
        ne = int(rng.integers(0, 40))
        cases.append((nv, [(int(rng.integers(0, nv)), int(rng.integers(0, nv))) for _ in range(ne)],
                      int(rng.integers(0, nv))))
    for nv, edges, src in cases:
        off, col = csr_from_edges(nv, edges)
        got = oracle.bfs_levels_direct(off, col, src)
        assert list(got) == relax_levels(nv, edges, src)
        if edges:
            m = csr_matrix((np.ones(len(edges)), ([e[0] for e in edges], [e[1] for e in edges])), shape=(nv, nv))
            sp = shortest_path(m, method="D", directed=True, unweighted=True, indices=src)
            assert list(got) == [int(x) if np.isfinite(x) else -1 for x in sp]
        # through the pager: offsets and columns in one backing store, page-aligned
        page = 32
        pad = lambda b: (b + page - 1) // page * page
        off_off, col_off = 0, pad(off.nbytes)
        host = np.zeros(col_off + pad(col.nbytes), np.uint8)
        host[:off.nbytes] = np.frombuffer(off.tobytes(), np.uint8)
        host[col_off:col_off + col.nbytes] = np.frombuffer(col.tobytes(), np.uint8)
        for frames in (1, 2, 64):
            pg = oracle.Pager(host, page, frames, oracle.CLOCK, True)
            assert np.array_equal(pg.bfs_levels(off_off, col_off, nv, src), got)
            assert pg.check() == 0 and pg.counters()["writebacks"] == 0
            pg.close()


def test_bfs_certificate_on_rmat():
    off, col = inputs.rmat_csr(12, 16 << 12, 21)
    lvl = oracle.bfs_levels_direct(off, col, 0)
    nv = off.size - 1
    src = np.repeat(np.arange(nv), np.diff(off))
    reached = lvl[src] >= 0
    assert lvl[0] == 0
    # every edge out of a reached vertex: 0 <= level[v] <= level[u] + 1
    assert np.all(lvl[col][reached] >= 0) and np.all(lvl[col][reached] <= lvl[src][reached] + 1)
    # every vertex at level k > 0 has an in-edge from level k - 1
    has_parent = np.zeros(nv, bool)
    tight = reached & (lvl[col] == lvl[src] + 1)
    has_parent[col[tight]] = True
    assert np.all(has_parent[lvl > 0])
    assert not np.any(has_parent[lvl < 0])


def test_embag_against_numpy_sequential_sum():
    n_rows, dims, bag, n_bags = 300, 128, 32, 9
    t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, 3).reshape(n_rows, dims)
    rows = inputs.fill_zipf_rows(np.empty(n_bags * bag, np.int64), n_bags * bag, 6, n_rows, 1.05)
    out = oracle.embag_f32_direct(t, rows, bag)
    for g in range(n_bags):
        acc = np.zeros(dims, np.float32)
        for r in rows[g * bag:(g + 1) * bag]:
            acc = (acc + t[r]).astype(np.float32)              # one rounding per addition
        assert np.array_equal(out[g], acc)
        # np.cumsum on float32 accumulates sequentially in float32
        assert np.array_equal(out[g], np.cumsum(t[rows[g * bag:(g + 1) * bag]], axis=0, dtype=np.float32)[-1])
    host = np.frombuffer(t.tobytes(), np.uint8).copy()
    for frames in (1, 4, 1000):
        pg = oracle.Pager(host, 2048, frames, oracle.CLOCK, True)
        assert np.array_equal(pg.embag_f32(0, dims, rows, bag), out)
        pg.close()


def test_uniform_independent_reference_hit_ratio():
    # i.i.d. uniform accesses: any non-anticipating policy hits with probability F/P
    P, F, n = 256, 64, 200000
    rng = np.random.default_rng(1)
    trace = rng.integers(0, P, n).astype(np.uint64)
    for policy in (oracle.FIFO, oracle.CLOCK):
        pg = make_pager(P, 16, F, policy, move=False)
        pg.replay(trace)
        c = pg.counters()
        assert abs(c["faults"] / n - (1 - F / P)) < 0.01
        pg.close()


def test_cc_against_scipy_and_brute_force():
    from scipy.sparse import csr_matrix
    from scipy.sparse.csgraph import connected_components
    rng = np.random.default_rng(31)
    cases = [(1, []), (4, []), (5, [(0, 0), (3, 1), (1, 3), (4, 2)]), (6, [(5, 0), (4, 5), (1, 2)])]
    for _ in range(30):
        nv = int(rng.integers(2, 30))
        cases.append((nv, [(int(rng.integers(0, nv)), int(rng.integers(0, nv))) for _ in range(int(rng.integers(0, 30)))]))
    for nv, edges in cases:
        off, col = csr_from_edges(nv, edges)
        got = oracle.cc_labels_direct(off, col)
        # brute force: repeat "every edge pulls both ends to the smaller label" until nothing changes
        lab = list(range(nv))
        changed = True
        while changed:
            changed = False
            for u, v in edges:
                m = min(lab[u], lab[v])
                if lab[u] != m or lab[v] != m:
                    lab[u] = lab[v] = m
                    changed = True
        assert list(got) == lab
        if edges:
            m = csr_matrix((np.ones(len(edges)), ([e[0] for e in edges], [e[1] for e in edges])), shape=(nv, nv))
            n_comp, part = connected_components(m, directed=True, connection="weak")
            assert len(set(got)) == n_comp
            for c in range(n_comp):                       # same partition, labelled by its smallest member
                members = np.nonzero(part == c)[0]
                assert set(got[members]) == {members.min()}


def test_sssp_against_bellman_ford_and_scipy():
    from scipy.sparse import csr_matrix
    from scipy.sparse.csgraph import dijkstra
    rng = np.random.default_rng(47)
    INF = 0x7FFFFFFF
    cases = [(1, [], 0), (3, [(0, 1, 5), (0, 1, 2), (1, 2, 0), (2, 2, 1)], 0), (4, [(1, 0, 3)], 0)]
    for _ in range(30):
        nv = int(rng.integers(2, 25))
        ne = int(rng.integers(0, 60))
        cases.append((nv, [(int(rng.integers(0, nv)), int(rng.integers(0, nv)), int(rng.integers(0, 300))) for _ in range(ne)],
                      int(rng.integers(0, nv))))
    for nv, wedges, src in cases:
        off, col = csr_from_edges(nv, [(u, v) for u, v, _ in wedges])
        w = np.zeros(col.size, dtype=np.int32)
        cur = off[:-1].copy()
        for u, v, ww in wedges:                           # same stable placement as csr_from_edges
            w[cur[u]] = ww
            cur[u] += 1
        got = oracle.sssp_direct(off, col, w, src)
        d = [INF] * nv
        d[src] = 0
        for _ in range(nv):                                # Bellman-Ford, V rounds over all edges
            for u, v, ww in wedges:
                if d[u] != INF and d[u] + ww < d[v]:
                    d[v] = d[u] + ww
        assert list(got) == d
        best = {}
        for u, v, ww in wedges:                            # scipy sums duplicate entries: keep the lightest edge
            best[(u, v)] = min(ww, best.get((u, v), 1 << 40))
        pos = {k: x for k, x in best.items() if x > 0 and k[0] != k[1]}
        if pos and all(x > 0 for x in best.values()):
            m = csr_matrix((list(pos.values()), ([k[0] for k in pos], [k[1] for k in pos])), shape=(nv, nv))
            sp = dijkstra(m, directed=True, indices=src)
            assert list(got) == [int(x) if np.isfinite(x) else INF for x in sp]


def test_pager_check_reports_each_kind_of_damage():
    """The replay's own invariant checker is only worth something if it can say no: damage its
    tables one word at a time and see each return code (a checker that always answers 0 would pass
    every other test)."""
    n_pages, frames = 12, 4

    def fresh():
        pg = make_pager(n_pages, 16, frames, oracle.CLOCK)
        for p in (0, 5, 7):                          # frames 0, 1, 2 taken; frame 3 free; pages 1.. unmapped
            pg.access(p)
        assert pg.check() == 0
        return pg

    pg = fresh(); pg.debug_poke("map", 5, frames); assert pg.check() == 1         # page table names a frame that does not exist
    pg = fresh(); pg.debug_poke("map", 3, 0); assert pg.check() == 2              # two pages claim frame 0
    pg = fresh(); pg.debug_poke("frame_page", 3, n_pages + 5); assert pg.check() == 3   # ring names a page that does not exist
    pg = fresh(); pg.debug_poke("frame_page", 3, 9); assert pg.check() == 4       # ring names a page that is not mapped there
    pg = fresh(); pg.debug_poke("resident", 0, 2); assert pg.check() == 5         # counter disagrees with the tables
    pg = fresh(); pg.debug_poke("map", 7, oracle.NONE); assert pg.check() == 4    # a mapping lost, its frame still names the page
    pg = fresh(); pg.debug_poke("frame_page", 1, oracle.NONE); assert pg.check() == 2   # a frame emptied under a mapped page
    with pytest.raises(IndexError):
        fresh().debug_poke("map", n_pages, 0)


@pytest.mark.parametrize("frames", [1, 2, 3, 4, 8, 17])
def test_belady_count_against_brute_force(frames):
    for trace in random_traces():
        trace = [int(t) for t in trace]
        n_pages = max(trace) + 1
        assert oracle.belady_faults(np.array(trace), n_pages, frames) == belady_opt_faults(trace, frames)
    assert oracle.belady_faults(np.empty(0, np.uint64), 4, frames) == 0


def test_belady_count_on_the_textbook_strings():
    for _, frames, policy, faults, string in _rows("page_replacement_strings.txt"):
        if policy != "fifo":
            trace = np.array([int(t) for t in string.split()])
            assert oracle.belady_faults(trace, int(trace.max()) + 1, int(frames)) == int(faults)


def test_recorded_trace_collapses_runs_and_keeps_the_fault_counts():
    rng = np.random.default_rng(11)
    pages = rng.integers(0, 40, 500)
    full = np.repeat(pages, rng.integers(1, 6, pages.size))           # runs of 1..5 accesses per page
    for frames in (1, 3, 8, 40):
        for policy, name in ((oracle.CLOCK, "clock"), (oracle.FIFO, "fifo")):
            pg = make_pager(40, 16, frames, policy, move=False)
            pg.record_trace(full.size)
            pg.replay(full)
            got = pg.trace()
            keep = np.concatenate([[True], full[1:] != full[:-1]])
            assert np.array_equal(got, full[keep].astype(np.uint64))   # exactly the run heads, in order
            counts = oracle.replay_counts(got, 40, 16, frames)
            assert counts[name] == pg.counters()["faults"]             # collapsed trace: same faults
            assert counts["belady"] == belady_opt_faults([int(t) for t in full], frames)
            assert counts["belady"] <= min(counts["clock"], counts["fifo"]) and counts["distinct"] == np.unique(full).size
            pg.close()
    pg = make_pager(40, 16, 4, oracle.CLOCK, move=False)
    pg.record_trace(3)
    pg.replay(full)
    with pytest.raises(OverflowError):
        pg.trace()


def test_bfs_page_trace_is_the_canonical_order():
    """Level by level, vertices ascending, per vertex its two row offsets and then its edges: on a
    hand-made graph the recorded page trace is written out and compared."""
    # 4 vertices; page = 16 bytes = 2 row offsets or 4 columns; offsets at byte 0 (5 int64 = 40 bytes -> 3 pages),
    # columns from byte 48 (page 3)
    off = np.array([0, 2, 3, 3, 6], dtype=np.int64)         # 0 -> {1, 3}; 1 -> {3}; 2 -> {}; 3 -> {0, 1, 2}
    col = np.array([1, 3, 3, 0, 1, 2], dtype=np.int32)
    host = np.zeros(48 + 32, dtype=np.uint8)
    host[:40] = np.frombuffer(off.tobytes(), np.uint8)
    host[48:48 + 24] = np.frombuffer(col.tobytes(), np.uint8)
    pg = oracle.Pager(host, 16, 2, oracle.CLOCK, True)
    pg.record_trace(64)
    lvl = pg.bfs_levels(0, 48, 4, 0)
    assert lvl.tolist() == [0, 1, 2, 1]
    # level 0: vertex 0: off[0], off[1] (page 0), edges 0..1 (page 3)
    # level 1: vertex 1: off[1] (page 0), off[2] (page 1), edge 2 (page 3); vertex 3: off[3] (page 1), off[4] (page 2),
    #          edges 3 (page 3), 4..5 (page 4)
    # level 2: vertex 2: off[2], off[3] (page 1), no edges
    assert pg.trace().tolist() == [0, 3, 0, 1, 3, 1, 2, 3, 4, 1]
    pg.close()


def test_all_core_build_gives_the_bits_of_the_one_thread_build():
    """The OpenMP build only splits outer loops: every sum, block and bag must come out bit for bit
    as from the single-threaded oracle."""
    par = oracle.AllCores()
    assert par.threads >= 1
    n = 100_003
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 5)
    assert par.stream_sum_i32_direct(a) == oracle.stream_sum_i32_direct(a) == int(a.astype(np.int64).sum())
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 6)
    idx = inputs.fill_index_i64(np.empty(5000, np.int64), 5000, 7, n)
    for block in (1, 37, 1024, 5000):
        f1, b1 = oracle.gather_block_sums_direct(x, idx, block)
        f2, b2 = par.gather_block_sums_direct(x, idx, block)
        assert np.array_equal(f1.view(np.uint32), f2.view(np.uint32)) and np.array_equal(b1, b2)
    y = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 8)
    assert np.array_equal(par.vadd_f32_direct(x, y).view(np.uint32), oracle.vadd_f32_direct(x, y).view(np.uint32))
    t = x[:100_000].reshape(1000, 100)
    rows = inputs.fill_zipf_rows(np.empty(7 * 300, np.int64), 7 * 300, 9, 1000, 1.05)
    assert np.array_equal(par.embag_f32_direct(t, rows, 7).view(np.uint32), oracle.embag_f32_direct(t, rows, 7).view(np.uint32))
