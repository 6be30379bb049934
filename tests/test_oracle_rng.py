"""Pins for the oracle's random numbers: published Philox4x32-10 vectors and the uniform grid."""
import os

import numpy as np

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox_kat.txt")


def kat_rows():
    rows = []
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers():
    rows = kat_rows()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = oracle.philox(ctr, key)
        assert [int(x) for x in got] == want


def test_uniform_words_and_grid():
    # counter = (t, s, b, 0), key = (seed low, seed high); words 0..2 -> u_draft, u_acc, u_res
    seed, b, s, t = 0x0123456789ABCDEF, 7, 5, 3
    w = oracle.philox([t, s, b, 0], [seed & 0xFFFFFFFF, seed >> 32])
    u = oracle.uniforms(seed, b, s, t)
    for i in range(3):
        assert u[i] == (int(w[i]) >> 8) / 2.0 ** 24
        assert 0.0 <= u[i] < 1.0
        assert np.float32(u[i]) == u[i]  # exact in fp32


def test_uniforms_are_uniform():
    # 3 x 20000 draws, 20 bins: chi-square against the flat law
    from scipy.stats import chi2
    n = 20000
    u = np.array([oracle.uniforms(11, b, 0, 0) for b in range(n)])
    for i in range(3):
        h, _ = np.histogram(u[:, i], bins=20, range=(0, 1))
        stat = ((h - n / 20) ** 2 / (n / 20)).sum()
        assert chi2.sf(stat, 19) > 1e-4
    # distinct counters give distinct streams
    assert not np.allclose(oracle.uniforms(11, 0, 0, 0), oracle.uniforms(11, 0, 0, 1))
    assert not np.allclose(oracle.uniforms(11, 0, 0, 0), oracle.uniforms(11, 0, 1, 0))
    assert not np.allclose(oracle.uniforms(11, 0, 0, 0), oracle.uniforms(12, 0, 0, 0))
