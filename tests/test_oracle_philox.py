"""Pins for oracle/philox.py: published known answers, exactness of the uniform map,
and the distribution of the Box-Muller output against library routines."""
import os

import numpy as np
from scipy import stats

from oracle import philox


def _kat(golden_dir):
    rows = []
    for line in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_known_answers(golden_dir):
    rows = _kat(golden_dir)
    assert len(rows) == 3
    for ctr, key, out in rows:
        got = philox.philox4x32_10(np.array([ctr], dtype=np.uint64), key)[0]
        assert [int(x) for x in got] == out


def test_vectorised_equals_one_by_one():
    rng = np.random.default_rng(0)
    ctr = rng.integers(0, 2 ** 32, size=(64, 4), dtype=np.uint64)
    key = (0x12345678, 0x9ABCDEF0)
    batch = philox.philox4x32_10(ctr, key)
    for i in range(64):
        assert np.array_equal(batch[i], philox.philox4x32_10(ctr[i:i + 1], key)[0])


def test_uniform_is_exact_in_float32_and_open():
    w = np.array([0, 1, 511, 512, 2 ** 31, 2 ** 32 - 1], dtype=np.uint32)
    u = philox.uniform_open(w)
    assert np.all(u > 0) and np.all(u < 1)
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)
    assert u[0] == 2.0 ** -24 and u[-1] == 1.0 - 2.0 ** -24
    # the map is monotone in the top 23 bits and ignores the low 9
    assert u[0] == u[1] == u[2] and u[3] > u[2]


def test_uniform_distribution():
    w = philox.noise_words(7, 3, 2, philox.TAG_INNOV, 1 << 20).reshape(-1)
    u = philox.uniform_open(w)
    assert stats.kstest(u, "uniform").pvalue > 1e-3
    # every bit of the words is fair
    bits = ((w[:, None] >> np.arange(32, dtype=np.uint32)) & 1).mean(axis=0)
    assert np.all(np.abs(bits - 0.5) < 5 * 0.5 / np.sqrt(len(w)))


def test_box_muller_identity_and_extremes():
    w = np.array([[0, 0, 2 ** 32 - 1, 2 ** 31]], dtype=np.uint32)
    z = philox.box_muller(w)[0]
    u = philox.uniform_open(w[0])
    assert np.isclose(z[0] ** 2 + z[1] ** 2, -2 * np.log(u[0]), rtol=1e-14)
    assert np.isclose(z[2] ** 2 + z[3] ** 2, -2 * np.log(u[2]), rtol=1e-12)
    # angle of the first pair is 2*pi*u_b
    assert np.isclose(np.arctan2(z[1], z[0]) % (2 * np.pi), 2 * np.pi * u[1], rtol=1e-12)
    assert abs(z[0]) < 5.8 and np.hypot(z[0], z[1]) <= np.sqrt(2 * 24 * np.log(2)) + 1e-12


def test_normals_match_library_distribution():
    x = philox.node_noise(1223627, 5, 3, philox.TAG_INNOV, 1 << 21)
    n = len(x)
    assert abs(x.mean()) < 4 / np.sqrt(n)
    assert abs(x.var() - 1) < 4 * np.sqrt(2 / n)
    assert abs(stats.kurtosis(x)) < 4 * np.sqrt(24 / n)
    assert abs(stats.skew(x)) < 4 * np.sqrt(6 / n)
    assert stats.kstest(x, "norm").pvalue > 1e-3
    # the four lanes of a block and neighbouring blocks are uncorrelated
    q = x.reshape(-1, 4)
    c = np.corrcoef(q.T)
    assert np.all(np.abs(c - np.eye(4)) < 5 / np.sqrt(len(q)))
    assert abs(np.corrcoef(x[:-4], x[4:])[0, 1]) < 5 / np.sqrt(n)


def test_streams_are_distinct_and_sliceable():
    a = philox.node_noise(9, 1, 0, philox.TAG_INNOV, 4096)
    for other in (philox.node_noise(9, 2, 0, philox.TAG_INNOV, 4096),
                  philox.node_noise(9, 1, 1, philox.TAG_INNOV, 4096),
                  philox.node_noise(9, 1, 0, philox.TAG_SHARED, 4096),
                  philox.node_noise(10, 1, 0, philox.TAG_INNOV, 4096),
                  philox.node_noise(9 + (1 << 32), 1, 0, philox.TAG_INNOV, 4096)):
        assert abs(np.corrcoef(a, other)[0, 1]) < 0.08
        assert not np.array_equal(a, other)
    assert np.array_equal(philox.node_noise(9, 1, 0, philox.TAG_INNOV, 100, elem_start=1000), a[1000:1100])
    assert np.array_equal(philox.node_noise(9, 1, 0, philox.TAG_INNOV, 4090), a[:4090])
