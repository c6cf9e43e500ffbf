"""The input generator against its written definition (pure-Python restatement of
the hash) and against the distributions it promises."""
import math

import numpy as np

import datagen

M64 = (1 << 64) - 1
GOLD = 0x9E3779B97F4A7C15


def mix64(z):
    z &= M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def key(seed, stream):
    return mix64(mix64(seed + GOLD) ^ ((stream * 0xD1B54A32D192ED03 + 1) & M64))


def draw(k, i):
    return mix64(k + GOLD * (i + 1))


def test_uniform_matches_definition():
    k = key(5, 2)
    got = datagen.uniform(5, 2, 16, lo=-1.0, hi=3.0, offset=7)
    ref = [-1.0 + 4.0 * ((draw(k, 7 + i) >> 11) * 2.0 ** -53) for i in range(16)]
    assert got.tolist() == ref


def test_normal_matches_box_muller():
    k = key(1, 0)
    got = datagen.normal(1, 0, 10, mean=0.5, std=2.0, offset=3)
    for i in range(10):
        e = 3 + i
        p = e >> 1
        u1 = ((draw(k, 2 * p) >> 11) + 1) * 2.0 ** -53
        u2 = (draw(k, 2 * p + 1) >> 11) * 2.0 ** -53
        r = math.sqrt(-2.0 * math.log(u1))
        a = 2.0 * math.pi * u2
        ref = 0.5 + 2.0 * r * (math.sin(a) if e & 1 else math.cos(a))
        assert abs(got[i] - ref) <= 1e-14 * max(1.0, abs(ref))


def test_slices_are_consistent():
    a = datagen.normal(9, 1, 1000)
    assert np.array_equal(datagen.normal(9, 1, 100, offset=333), a[333:433])
    rp, ci, va = datagen.csr_bernoulli(3, 0, 200, 50, 0.1)
    rp2, ci2, va2 = datagen.csr_bernoulli(3, 0, 20, 50, 0.1, row0=60)
    assert np.array_equal(ci2, ci[rp[60]:rp[80]]) and np.array_equal(va2, va[rp[60]:rp[80]])
    assert np.array_equal(rp2, rp[60:81] - rp[60])


def test_distributions():
    u = datagen.uniform(0, 0, 200_000)
    assert 0.0 <= u.min() and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 5e-3 and abs(u.var() - 1 / 12) < 2e-3
    z = datagen.normal(1, 0, 200_000)
    assert abs(z.mean()) < 1e-2 and abs(z.std() - 1.0) < 1e-2
    assert abs(np.mean(z ** 3)) < 5e-2 and abs(np.mean(z ** 4) - 3.0) < 0.1
    # independent streams
    z2 = datagen.normal(1, 2, 200_000)
    assert abs(np.corrcoef(z, z2)[0, 1]) < 1e-2


def test_csr_structure_and_density():
    rows, cols, p = 20_000, 1000, 0.01
    rp, ci, va = datagen.csr_bernoulli(3, 0, rows, cols, p, 1.0, 5.0)
    assert rp.dtype == np.int32 and ci.dtype == np.int32 and va.dtype == np.float64
    assert rp[0] == 0 and rp[-1] == len(ci) == len(va)
    lens = np.diff(rp)
    assert abs(lens.mean() - cols * p) < 0.1
    assert abs(lens.var() - cols * p * (1 - p)) < 0.5          # Binomial row lengths
    assert ci.min() >= 0 and ci.max() < cols
    # strictly ascending columns inside every row
    inner = np.ones(len(ci), dtype=bool)
    inner[rp[:-1][lens > 0]] = False
    assert np.all(np.diff(ci.astype(np.int64))[inner[1:]] > 0)
    # uniform column positions, value range
    hist = np.bincount(ci, minlength=cols)
    assert hist.min() > 0.5 * rows * p and hist.max() < 1.6 * rows * p
    assert va.min() >= 1.0 and va.max() < 5.0
    assert (lens == 0).sum() >= 0


def test_csr_edge_densities():
    rp, ci, va = datagen.csr_bernoulli(3, 0, 4, 6, 1.0)
    assert rp.tolist() == [0, 6, 12, 18, 24] and ci.tolist() == list(range(6)) * 4
    rp, ci, va = datagen.csr_bernoulli(3, 0, 4, 6, 0.0)
    assert rp.tolist() == [0] * 5 and len(ci) == 0


def test_workload_shapes():
    w = datagen.row_dense_workload(30, 20)
    assert w["X"].shape == (30, 20) and w["v"].shape == (20,) and w["w"].shape == (30,)
    assert 0 <= w["w"].min() and w["w"].max() < 1
    o = datagen.outer_workload(300, 200, 10, 0.05)
    assert o["U"].shape == (300, 10) and o["V"].shape == (200, 10)
    assert abs(o["U"].std() - 0.1) < 0.01
    assert o["vals"].min() >= 1.0 and o["vals"].max() < 5.0
