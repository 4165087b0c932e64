"""The five oversubscribed workload configurations and their runners.

Each configuration places its paged arrays at page-aligned offsets of ONE backing store
(one handle, one frame pool), fills them with the seeded generators, keeps small
operands (indices, row ids, outputs) in ordinary device memory, and runs the workload
through the C ABI.  ``shrink`` divides every size by 2**shrink (page size kept) so that
the same code serves small parity cases.

Effective bytes (numerator of "effective application GB/s"): streaming sum = bytes of the
array; gather = 4 bytes per index; BFS = 16 bytes of offsets per expanded vertex + 4 bytes
per traversed edge; vector add = bytes of a, b and c; embedding bag = bytes of the rows
looked up.
"""
from __future__ import annotations

import ctypes
import dataclasses
import time

import numpy as np

from . import binding as B
from . import inputs

KiB, MiB, GiB = 1 << 10, 1 << 20, 1 << 30


def _pad(nbytes: int, page: int) -> int:
    return (nbytes + page - 1) // page * page


def _host_view(ptr: int, nbytes: int) -> np.ndarray:
    return np.ctypeslib.as_array((ctypes.c_uint8 * nbytes).from_address(ptr))


@dataclasses.dataclass
class RunResult:
    seconds: float            # CUDA-event time: workload kernel(s) + flush, cold pool
    kernel_seconds: float     # workload kernel(s) only
    stats: dict
    check: dict
    effective_bytes: int
    extra: dict


class Workload:
    """Base: owns the handle, the host arena and the device-side operands."""

    name = "?"
    cfg = 0
    page_bytes = 0
    kernels_per_run = 1

    def __init__(self, shrink: int = 0):
        self.shrink = shrink
        self.h = None
        self.off = {}
        self.host = None
        self._layout()

    # -- layout -------------------------------------------------------------
    def sizes(self):
        """(arrays: name -> nbytes, pool_bytes or a function of the total) at this shrink; no GPU needed."""
        raise NotImplementedError

    def _layout(self):
        arrays, pool_bytes = self.sizes()
        total = 0
        for name, nbytes in arrays.items():
            self.off[name] = total
            total += _pad(nbytes, self.page_bytes)
        self.nbytes = total
        if getattr(self, "pool_override", None):
            pool_bytes = self.pool_override
        if callable(pool_bytes):
            pool_bytes = pool_bytes(total)
        self.pool_bytes = max(self.page_bytes, pool_bytes // self.page_bytes * self.page_bytes)
        self.n_pages = total // self.page_bytes
        self.n_frames = self.pool_bytes // self.page_bytes

    def _create(self):
        """The library allocates the pinned backing store."""
        self._layout()
        self.h = B.gpuvm_create(None, self.nbytes, self.page_bytes, self.pool_bytes)
        self.host = _host_view(B.gpuvm_host_ptr(self.h), self.nbytes)

    def view(self, name: str, dtype, count: int) -> np.ndarray:
        o = self.off[name]
        return self.host[o:o + count * np.dtype(dtype).itemsize].view(dtype)

    def close(self):
        if self.h:
            B.gpuvm_destroy(self.h)
            self.h = None
            self.host = None

    # -- to be provided -----------------------------------------------------
    def setup(self):
        raise NotImplementedError

    def launch(self, stream):
        raise NotImplementedError

    def effective_bytes(self) -> int:
        raise NotImplementedError

    def describe(self) -> dict:
        return {"workload": self.name, "cfg": self.cfg, "shrink": self.shrink, "page_bytes": self.page_bytes,
                "pool_bytes": self.pool_bytes, "paged_bytes": self.nbytes, "pages": self.n_pages,
                "frames": self.n_frames, "oversubscription_level": self.nbytes / self.pool_bytes - 1}

    # -- one cold run ---------------------------------------------------------
    def run(self, check: bool = True) -> RunResult:
        import torch
        stream = torch.cuda.current_stream()
        B.gpuvm_reset(self.h)                              # device-wide: nothing of an earlier step is in flight
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        extra = self.launch(stream) or {}
        e1.record(stream)
        B.gpuvm_flush(self.h, stream)
        e2.record(stream)
        e2.synchronize()
        stats = B.gpuvm_stats(self.h)
        ck = B.gpuvm_check(self.h) if check else {}
        return RunResult(e0.elapsed_time(e2) / 1e3, e0.elapsed_time(e1) / 1e3, stats, ck,
                         self.effective_bytes(), extra)


class StreamSum(Workload):
    """Streaming read-reduce: int64 sum over an int32 array, 4 KiB pages, pool = 1/4 of the data."""
    name, cfg, page_bytes = "stream_sum_i32", 1, 4 * KiB

    def sizes(self):
        self.n = (1 << 24) >> self.shrink
        return {"a": 4 * self.n}, (16 * MiB) >> self.shrink

    def setup(self):
        import torch
        self._create()
        inputs.fill_i32_u20(B.gpuvm_host_ptr(self.h) + self.off["a"], self.n, inputs.config_seed(1))
        self.d_sum = torch.zeros(1, dtype=torch.int64, device="cuda")
        return self

    def launch(self, stream):
        B.gpuvm_stream_sum_i32(self.h, self.off["a"], self.n, self.d_sum, stream)

    def effective_bytes(self):
        return 4 * self.n


class Gather(Workload):
    """Random gather: fp32 array, uniform int64 indices, one sum per 1024 indices, 64 KiB pages, pool 1/4."""
    name, cfg, page_bytes = "random_gather_f32", 2, 64 * KiB
    block = 1024

    def sizes(self):
        self.n = (1 << 28) >> self.shrink
        self.n_idx = (1 << 26) >> self.shrink
        return {"x": 4 * self.n}, (256 * MiB) >> self.shrink

    def setup(self):
        import torch
        self._create()
        inputs.fill_f32_pm1(B.gpuvm_host_ptr(self.h) + self.off["x"], self.n, inputs.config_seed(2))
        self.idx_host = torch.empty(self.n_idx, dtype=torch.int64).pin_memory()
        inputs.fill_index_i64(self.idx_host.data_ptr(), self.n_idx, inputs.config_seed(2, 1), self.n)
        self.d_idx = self.idx_host.cuda()
        nb = (self.n_idx + self.block - 1) // self.block
        self.d_fsum = torch.zeros(nb, dtype=torch.float32, device="cuda")
        self.d_bsum = torch.zeros(nb, dtype=torch.int64, device="cuda")
        return self

    def launch(self, stream):
        B.gpuvm_gather_f32(self.h, self.off["x"], self.d_idx, self.n_idx, self.block, self.d_fsum, self.d_bsum, stream)

    def effective_bytes(self):
        return 4 * self.n_idx


class Bfs(Workload):
    """BFS from vertex 0 on an RMAT graph; row offsets and column indices paged at 64 KiB, pool = half."""
    name, cfg, page_bytes = "bfs_rmat_csr", 3, 64 * KiB
    kernels_per_run = None        # 1 + 2 per level

    def sizes(self):
        self.scale = 24 - self.shrink
        self.nv = 1 << self.scale
        self.ne = 16 << self.scale
        return {"off": _pad(8 * (self.nv + 1), 16), "col": 4 * self.ne}, lambda total: total // 2   # pool = half their size

    def setup(self):
        import torch
        self._create()
        base = B.gpuvm_host_ptr(self.h)
        inputs.rmat_csr(self.scale, self.ne, inputs.config_seed(3), base + self.off["off"], base + self.off["col"])
        self.d_level = torch.zeros(self.nv, dtype=torch.int32, device="cuda")
        self.levels = 0
        return self

    def launch(self, stream):
        self.levels = B.gpuvm_bfs_csr(self.h, self.off["off"], self.off["col"], self.nv, 0, self.d_level, stream)
        return {"levels": self.levels}

    def effective_bytes(self):
        lvl = self.d_level.cpu().numpy()
        off = self.view("off", np.int64, self.nv + 1)
        deg = np.diff(off)
        visited = lvl >= 0
        self.traversed_edges = int(deg[visited].sum())
        return int(16 * visited.sum() + 4 * self.traversed_edges)

    def compulsory_pages(self) -> int:
        """Distinct pages any BFS must touch: the two row offsets and the whole edge range of every
        vertex it reaches (from the levels the last run produced)."""
        reached = np.flatnonzero(self.d_level.cpu().numpy() >= 0)
        off = self.view("off", np.int64, self.nv + 1)
        mark = np.zeros(self.n_pages + 1, np.int64)
        for lo, hi in ((self.off["off"] + 8 * reached, self.off["off"] + 8 * reached + 15),
                       (self.off["col"] + 4 * off[reached], self.off["col"] + 4 * off[reached + 1] - 1)):
            keep = hi >= lo
            np.add.at(mark, lo[keep] // self.page_bytes, 1)
            np.add.at(mark, hi[keep] // self.page_bytes + 1, -1)
        return int(np.count_nonzero(np.cumsum(mark[:-1]) > 0))


class BfsBalanced(Bfs):
    """BFS on the cfg 3 graph stored as Balanced CSR: chunks of one page of edges (16 Ki edges), the chunk
    table paged with the other two arrays; pool = half."""
    name, cfg = "bfs_rmat_balanced_csr", 8

    def sizes(self):
        self.scale = 24 - self.shrink
        self.nv = 1 << self.scale
        self.ne = 16 << self.scale
        self.chunk_edges = self.page_bytes // 4
        n_chunks = (self.ne + self.chunk_edges - 1) // self.chunk_edges
        return ({"off": _pad(8 * (self.nv + 1), 16), "col": 4 * self.ne, "chunk": _pad(4 * (n_chunks + 1), 16)},
                lambda total: total // 2)

    def setup(self):
        import torch
        self._create()
        base = B.gpuvm_host_ptr(self.h)
        inputs.rmat_csr(self.scale, self.ne, inputs.config_seed(3), base + self.off["off"], base + self.off["col"])
        chunks = B.gpuvm_bcsr_build(self.view("off", np.int64, self.nv + 1), self.chunk_edges)
        self.view("chunk", np.int32, chunks.size)[...] = chunks
        self.d_level = torch.zeros(self.nv, dtype=torch.int32, device="cuda")
        self.levels = 0
        return self

    def launch(self, stream):
        self.levels = B.gpuvm_bfs_bcsr(self.h, self.off["off"], self.off["col"], self.off["chunk"], self.nv, self.ne,
                                       self.chunk_edges, 0, self.d_level, stream)
        return {"levels": self.levels}


class CcBalanced(BfsBalanced):
    """Connected components on the cfg 3 graph stored as Balanced CSR."""
    name, cfg = "cc_rmat_balanced_csr", 9

    def launch(self, stream):
        B.gpuvm_cc_bcsr(self.h, self.off["off"], self.off["col"], self.off["chunk"], self.nv, self.ne, self.chunk_edges,
                        self.d_level, stream)
        return {"sweeps": 1}

    def effective_bytes(self):
        return int(8 * (self.nv + 1) + 4 * self.ne)

    def compulsory_pages(self):
        return self.n_pages


class Cc(Bfs):
    """Connected components on the BFS configuration's graph and pool (the paper's second graph workload)."""
    name, cfg = "cc_rmat_csr", 6

    def launch(self, stream):
        self.sweeps = B.gpuvm_cc_csr(self.h, self.off["off"], self.off["col"], self.nv, self.d_level, stream)
        return {"sweeps": self.sweeps}

    def effective_bytes(self):
        # every sweep reads every row offset and every edge
        return int(self.sweeps * (8 * (self.nv + 1) + 4 * self.ne))


class Sssp(Workload):
    """SSSP from vertex 0 on the same RMAT graph with int32 weights in [1, 255] in a third paged array;
    pool = half of the three arrays; the row offsets are advised to be kept."""
    name, cfg, page_bytes = "sssp_rmat_csr", 7, 64 * KiB

    def sizes(self):
        self.scale = 24 - self.shrink
        self.nv = 1 << self.scale
        self.ne = 16 << self.scale
        return {"off": _pad(8 * (self.nv + 1), 16), "col": 4 * self.ne, "w": 4 * self.ne}, lambda total: total // 2

    def setup(self):
        import torch
        self._create()
        base = B.gpuvm_host_ptr(self.h)
        inputs.rmat_csr(self.scale, self.ne, inputs.config_seed(3), base + self.off["off"], base + self.off["col"])
        inputs.fill_i32_range(base + self.off["w"], self.ne, inputs.config_seed(3, 2), 1, 255)
        # the row offsets (6 % of the data) stay in the pool once fetched: vertices that are lowered behind the
        # sweep find theirs there instead of reading them over the link (86 -> 80 ms)
        B.gpuvm_advise_keep(self.h, self.off["off"], 8 * (self.nv + 1))
        self.d_dist = torch.zeros(self.nv, dtype=torch.int32, device="cuda")
        self.rounds = 0
        return self

    def launch(self, stream):
        self.rounds = B.gpuvm_sssp_csr(self.h, self.off["off"], self.off["col"], self.off["w"], self.nv, 0, self.d_dist,
                                       stream)
        return {"rounds": self.rounds}

    def effective_bytes(self):
        d = self.d_dist.cpu().numpy()
        off = self.view("off", np.int64, self.nv + 1)
        reached = d != 0x7FFFFFFF
        return int(16 * reached.sum() + 8 * np.diff(off)[reached].sum())     # offsets + (column, weight) per edge, once


class VAdd(Workload):
    """c = a + b over three fp32 arrays, 64 KiB pages, pool = one array (3x oversubscribed)."""
    name, cfg, page_bytes = "vector_add_f32", 4, 64 * KiB

    def sizes(self):
        self.n = (1 << 30) >> self.shrink
        return {"a": 4 * self.n, "b": 4 * self.n, "c": 4 * self.n}, (4 * GiB) >> self.shrink

    def setup(self):
        self._create()
        base = B.gpuvm_host_ptr(self.h)
        inputs.fill_f32_pm1(base + self.off["a"], self.n, inputs.config_seed(4))
        inputs.fill_f32_pm1(base + self.off["b"], self.n, inputs.config_seed(4, 1))
        self.view("c", np.float32, self.n)[...] = 0
        return self

    def launch(self, stream):
        B.gpuvm_vadd_f32(self.h, self.off["a"], self.off["b"], self.off["c"], self.n, stream)

    def effective_bytes(self):
        return 12 * self.n


class EmbeddingBag(Workload):
    """Zipf-skewed embedding gather: rows x 128 fp32 table, bags of 32 rows, 2 MiB pages, pool 1/4."""
    name, cfg, page_bytes = "zipf_embedding_bag_f32", 5, 2 * MiB
    dims, bag, s = 128, 32, 1.05

    def sizes(self):
        self.n_rows = (1 << 27) >> self.shrink
        self.n_lookups = (1 << 24) >> self.shrink
        self.n_bags = self.n_lookups // self.bag
        return {"t": 4 * self.dims * self.n_rows}, (16 * GiB) >> self.shrink

    def setup(self):
        import torch
        self._create()
        inputs.fill_f32_pm1(B.gpuvm_host_ptr(self.h) + self.off["t"], self.dims * self.n_rows, inputs.config_seed(5))
        self.rows_host = torch.empty(self.n_lookups, dtype=torch.int64).pin_memory()
        inputs.fill_zipf_rows(self.rows_host.data_ptr(), self.n_lookups, inputs.config_seed(5, 1), self.n_rows, self.s)
        self.d_rows = self.rows_host.cuda()
        self.d_out = torch.zeros(self.n_bags * self.dims, dtype=torch.float32, device="cuda")
        return self

    def launch(self, stream):
        B.gpuvm_embag_f32(self.h, self.off["t"], self.dims, self.d_rows, self.n_bags, self.bag, self.d_out, stream)

    def effective_bytes(self):
        return 4 * self.dims * self.n_lookups


WORKLOADS = {1: StreamSum, 2: Gather, 3: Bfs, 4: VAdd, 5: EmbeddingBag, 6: Cc, 7: Sssp, 8: BfsBalanced, 9: CcBalanced}


def make(cfg: int, shrink: int = 0) -> Workload:
    t0 = time.time()
    w = WORKLOADS[cfg](shrink).setup()
    w.setup_seconds = time.time() - t0
    return w


def describe(cfg: int, shrink: int = 0) -> dict:
    """The configuration's sizes without creating anything (no GPU needed)."""
    return WORKLOADS[cfg](shrink).describe()
