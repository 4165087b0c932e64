"""Batched workloads with long request tables: many requests per warp, several mask words,
the scratch bound, the grid-wide fault ring of large pages.  Same oracle, same tolerances as
the parity tests."""
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


def _gather(B, h, ar, idx, block):
    import torch
    nb = (idx.size + block - 1) // block
    fsum = torch.zeros(nb, dtype=torch.float32, device="cuda")
    bsum = torch.zeros(nb, dtype=torch.int64, device="cuda")
    B.gpuvm_gather_f32(h, ar.off["x"], dev(idx), idx.size, block, fsum, bsum)
    st, _ = finish(h)
    return fsum.cpu().numpy(), bsum.cpu().numpy(), st


@pytest.mark.parametrize("page,n,n_idx,block,frames", [
    (16384, 1 << 21, (1 << 24) + 12345, 1024, 64),      # 4096 requests per warp: two mask words
    (4096, 1 << 20, (1 << 25) + 4321, 1024, 256),       # 8192+ per warp, ragged tail
    (65536, 1 << 22, (1 << 26) - 999, 1000, 64),        # 16384 per warp: every request in flight at once
    (4096, 1 << 20, (1 << 24) + 5, 256, 64),            # smallest index block that is summed without a table
    (4096, 1 << 20, (1 << 24) + 5, 1 << 15, 64),        # index blocks longer than a warp's piece: carried over
])
def test_gather_with_long_tables(B, page, n, n_idx, block, frames):
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, inputs.config_seed(2))
    idx = inputs.fill_index_i64(np.empty(n_idx, np.int64), n_idx, inputs.config_seed(2, 3), n)
    ar = Arena(page, {"x": x})
    ref_f, ref_b = oracle.gather_block_sums_direct(x, idx, block)
    with paged(ar.host, page, frames) as h:
        fsum, bsum, st = _gather(B, h, ar, idx, block)
        deep_faults, deep_scratch = st["faults"], B.gpuvm_scratch_bytes(h)
    assert np.array_equal(bsum, ref_b)
    assert np.all(np.abs(fsum.astype(np.float64) - ref_f) <= 1e-6 * np.maximum(np.abs(ref_f), 2.0 ** -10))
    assert deep_faults >= ar.n_pages or deep_faults >= np.unique(idx * 4 // page).size
    assert deep_scratch <= 1 << 20              # no request tables: the index list is read in place
    # the same call under a scratch bound: request tables that fit the bound, same sums, not fewer faults
    with paged(ar.host, page, frames) as h:
        B.gpuvm_set_scratch_limit(h, 40 << 20)
        fsum2, bsum2, st2 = _gather(B, h, ar, idx, block)
        assert (1 << 20) < B.gpuvm_scratch_bytes(h) <= max(40 << 20, 148 * 28 * 2048 * 4 + (1 << 20))
    assert np.array_equal(bsum2, ref_b)
    assert np.all(np.abs(fsum2.astype(np.float64) - ref_f) <= 1e-6 * np.maximum(np.abs(ref_f), 2.0 ** -10))
    assert st2["faults"] >= deep_faults


@pytest.mark.parametrize("page,n_rows,n_bags,frames,dims,bag", [
    (1 << 20, 1 << 16, 1 << 18, 8, 128, 8),      # 1 MiB pages: grid-wide ring; two groups of 32 bags per warp
    (4096, 1 << 14, (1 << 19) + (1 << 14) + 77, 64, 32, 4),  # eight groups per warp, ragged tail, block rings only
    (1 << 18, 1 << 15, 1 << 17, 4, 128, 40),     # bags longer than one batch of lookups: tables follow one another
])
def test_embag_with_several_groups_per_warp(B, page, n_rows, n_bags, frames, dims, bag):
    import torch
    t = inputs.fill_f32_pm1(np.empty(n_rows * dims, np.float32), n_rows * dims, inputs.config_seed(5))
    rows = inputs.fill_zipf_rows(np.empty(n_bags * bag, np.int64), n_bags * bag, inputs.config_seed(5, 7), n_rows, 1.05)
    ar = Arena(page, {"t": t})
    ref = oracle.embag_f32_direct(t.reshape(n_rows, dims), rows, bag).reshape(-1)
    results = []
    for limit in (0, 64 << 20):
        out = torch.zeros(n_bags * dims, dtype=torch.float32, device="cuda")
        with paged(ar.host, page, frames) as h:
            if limit:
                B.gpuvm_set_scratch_limit(h, limit)
            B.gpuvm_embag_f32(h, ar.off["t"], dims, dev(rows), n_bags, bag, out)
            st, _ = finish(h)
            results.append((out.cpu().numpy(), st["faults"], B.gpuvm_scratch_bytes(h)))
    for got, faults, _ in results:
        assert np.array_equal(got.view(np.uint32), ref.astype(np.float32).view(np.uint32))   # list-order fp32 sums: same bits
        assert faults >= np.unique(rows * dims * 4 // page).size
    assert results[1][2] <= results[0][2]


def test_scratch_limit_arguments(B):
    ar = Arena(4096, {"x": np.zeros(4096, np.float32)})
    with paged(ar.host, 4096, 2) as h:
        assert B.gpuvm_scratch_bytes(h) == 0
        B.gpuvm_set_scratch_limit(h, 1 << 20)
        B.gpuvm_set_scratch_limit(h, 0)
    with pytest.raises(B.GpuvmError):
        B.gpuvm_set_scratch_limit(None, 1)
    assert B.gpuvm_scratch_bytes(None) == 0
