"""Pins for the oracle's counter-based generator."""
import os

import numpy as np
from scipy import stats

from oracle import philox

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_known_answer_vectors():
    rows = [l.split() for l in open(GOLD) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r if x != "->"]
        out = philox.philox4x32_10(*v[:6])
        assert [int(o) for o in out] == v[6:]


def test_unit_interval_is_open_and_fp32_exact():
    n = np.array([0, 1, 511, 512, 0xFFFFFFFF, 0x80000000], dtype=np.uint64)
    u = philox.bits_to_unit(n)
    assert u.min() > 0.0 and u.max() < 1.0
    assert np.all(u.astype(np.float32).astype(np.float64) == u)
    assert u[0] == 2.0 ** -24 and u[4] == 1.0 - 2.0 ** -24


def test_streams_are_functions_of_their_coordinates_only():
    a = philox.xi(3, 5, 17, 64)
    assert np.array_equal(a, philox.xi(3, 5, 17, 64))
    assert np.array_equal(a[:10], philox.xi(3, 5, 17, 10))          # prefix property
    for other in (philox.xi(4, 5, 17, 64), philox.xi(3, 6, 17, 64), philox.xi(3, 5, 18, 64),
                  philox.x_init(3, 5, 64)):
        assert not np.array_equal(a, other)
    tab = philox.normals_table(3, [5, 6], philox.STREAM_XI, range(20), 7)
    assert np.array_equal(tab[0, 17], a[:7])
    assert philox.uniform_table(3, [5, 6], 20)[1, 9] == philox.uniform(3, 6, 9)


def test_normals_and_uniforms_have_the_right_law():
    z = philox.normals(11, 0, philox.STREAM_XI, 3, 200_000)
    assert stats.kstest(z, "norm").pvalue > 0.01
    assert abs(np.corrcoef(z[0::2], z[1::2])[0, 1]) < 0.01        # the two Box-Muller branches
    u = philox.uniform_table(11, range(2000), 100).reshape(-1)
    assert stats.kstest(u, "uniform").pvalue > 0.01
