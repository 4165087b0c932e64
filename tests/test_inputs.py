"""The seeded generators: reproducible, slice-independent, right distributions."""
import math

import numpy as np

from paper_2411_05309_b200 import inputs

M64 = (1 << 64) - 1


def py_mix64(seed, i):
    z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def test_mixer_matches_python_restatement():
    for seed in (0, 1, inputs.config_seed(1), M64):
        for i in (0, 1, 2, 12345, 1 << 40):
            assert inputs.mix64(seed, i) == py_mix64(seed, i)


def test_fills_are_pure_functions_of_seed_and_index():
    seed = inputs.config_seed(2)
    n = 5000
    whole = inputs.fill_f32_pm1(np.empty(n, np.float32), n, seed)
    part = inputs.fill_f32_pm1(np.empty(100, np.float32), 100, seed, first=1234)
    assert np.array_equal(whole[1234:1334], part)
    exp = np.array([np.float32(py_mix64(seed, i) >> 40) * np.float32(2.0 ** -23) - np.float32(1)
                    for i in range(64)], dtype=np.float32)
    assert np.array_equal(whole[:64], exp)
    assert whole.min() >= -1.0 and whole.max() < 1.0
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, seed)
    assert a.min() >= 0 and a.max() < (1 << 20)
    assert a[7] == py_mix64(seed, 7) & 0xFFFFF
    idx = inputs.fill_index_i64(np.empty(n, np.int64), n, seed, 1000)
    assert idx.min() >= 0 and idx.max() < 1000 and idx[3] == py_mix64(seed, 3) % 1000


def test_uniform_moments():
    n = 1 << 20
    a = inputs.fill_i32_u20(np.empty(n, np.int32), n, 99)
    mean = a.astype(np.float64).mean()
    sigma = (2 ** 20) / math.sqrt(12 * n)
    assert abs(mean - (2 ** 20 - 1) / 2) < 6 * sigma
    x = inputs.fill_f32_pm1(np.empty(n, np.float32), n, 7).astype(np.float64)
    assert abs(x.mean()) < 6 * (2 / math.sqrt(12 * n))


def test_rmat_csr_is_a_valid_stable_csr():
    scale, ne = 10, 16 << 10
    off, col = inputs.rmat_csr(scale, ne, 5)
    nv = 1 << scale
    assert off[0] == 0 and off[-1] == ne and np.all(np.diff(off) >= 0)
    assert col.min() >= 0 and col.max() < nv
    # quadrant a dominates: vertex 0 has the largest expected out-degree ne*0.76^scale
    deg = np.diff(off)
    expect0 = ne * 0.76 ** scale
    assert abs(deg[0] - expect0) < 6 * math.sqrt(expect0) + 1
    # source marginal: P(source bit = 1) = c + d = 0.24 at every level
    mean_src_bits = sum(bin(v).count("1") * int(d) for v, d in enumerate(deg)) / ne
    assert abs(mean_src_bits - 0.24 * scale) < 0.05
    # destination marginal: P(dest bit = 1) = b + d = 0.24
    mean_dst_bits = np.mean([bin(int(v)).count("1") for v in col[:4000]])
    assert abs(mean_dst_bits - 0.24 * scale) < 0.15
    off2, col2 = inputs.rmat_csr(scale, ne, 5)
    assert np.array_equal(off, off2) and np.array_equal(col, col2)


def test_zipf_matches_its_probability_mass_function():
    n_ranks, s, n = 1 << 27, 1.05, 1 << 20
    rows = inputs.fill_zipf_rows(np.empty(n, np.int64), n, 11, n_ranks, s)
    assert rows.min() >= 0 and rows.max() < n_ranks
    # generalised harmonic number by direct summation of the head + Euler-Maclaurin tail
    head = 1 << 16
    k = np.arange(1, head + 1, dtype=np.float64)
    H = (k ** -s).sum()
    a, b = head + 0.5, n_ranks + 0.5
    H += (b ** (1 - s) - a ** (1 - s)) / (1 - s)
    assert abs(H - 12.7350) < 2e-3
    for upto, expect in ((1, 1 / H), (32, (k[:32] ** -s).sum() / H), (4096, (k[:4096] ** -s).sum() / H)):
        got = np.mean(rows < upto)
        assert abs(got - expect) < 5 * math.sqrt(expect * (1 - expect) / n), (upto, got, expect)
    part = inputs.fill_zipf_rows(np.empty(50, np.int64), 50, 11, n_ranks, s, first=777)
    assert np.array_equal(rows[777:827], part)
