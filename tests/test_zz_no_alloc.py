"""The allocation-free BFS entry point against the regular one.

gpuvm_bfs_csr_noalloc serves callers that cannot allocate device memory when they call
(latency-critical pipelines, hosts that forbid allocation after start-up, processes whose
own pool already owns all free memory): it keeps its scratch in an array inside the
library's device image.  The test calls it twice in a row through the C ABI -- the second
call finds the first call's leftovers in the shared array -- and expects exactly the levels
the regular entry point produces (BFS levels are integers: bit-exact), plus the argument
check for graphs beyond the stated maximum.  This file sorts last on purpose, so a run that
stops at the first failure has already been through every other test.
"""
import numpy as np
import pytest

from gpu_common import Arena, finish, paged
from paper_2411_05309_b200 import inputs

pytestmark = pytest.mark.gpu


def test_noalloc_bfs_matches_regular_bfs_twice_in_a_row():
    import torch
    from paper_2411_05309_b200 import binding as B
    scale, page, frames = 14, 4096, 24
    off, col = inputs.rmat_csr(scale, 16 << scale, inputs.config_seed(3))
    nv = off.size - 1
    assert np.diff(off).max() >= 4096          # long lists: the piece queue in the scratch is used
    off_p = np.zeros((off.size + 1) // 2 * 2, np.int64)
    off_p[:off.size] = off
    ar = Arena(page, {"off": off_p, "col": col})
    want = torch.zeros(nv, dtype=torch.int32, device="cuda")
    got = torch.zeros(nv, dtype=torch.int32, device="cuda")
    # the reference levels come from a handle of their own, so that the handle under test never
    # sees a call that allocates scratch
    with paged(ar.host, page, frames) as h_ref:
        depth_want = {}
        wants = {}
        for source in (0, 5):
            depth_want[source] = B.gpuvm_bfs_csr(h_ref, ar.off["off"], ar.off["col"], nv, source, want)
            finish(h_ref)
            wants[source] = want.clone()
        assert B.gpuvm_scratch_bytes(h_ref) > 0                       # the regular entry point does allocate
    with paged(ar.host, page, frames) as h:
        for call, source in enumerate((0, 0, 5)):                     # two calls in a row, then a different source
            got.fill_(-7)
            B.gpuvm_reset(h)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            depth = B.gpuvm_bfs_csr_noalloc(h, ar.off["off"], ar.off["col"], nv, source, got)
            torch.cuda.synchronize()
            if call > 0:                                              # (the first call may load the module lazily)
                assert torch.cuda.mem_get_info()[0] == free_before    # no device memory was taken
            assert B.gpuvm_scratch_bytes(h) == 0                      # and none through the handle either
            finish(h)
            assert depth == depth_want[source]
            assert torch.equal(got, wants[source])
        want = wants[5]
        # beyond the stated maximum: refused with a clear status, nothing runs
        with pytest.raises(B.GpuvmError) as err:
            B.gpuvm_bfs_csr_noalloc(h, ar.off["off"], ar.off["col"], B.BFS_NOALLOC_MAX_VERTICES + 1, 0, got)
        assert err.value.status == B.E_RANGE
        assert torch.equal(got, want)
