"""Pins for the oracle's counter-based generator (Philox4x32-10 reading)."""
import numpy as np
from scipy import stats

import oracle


def test_known_answer_vectors(golden):
    kat = golden("philox_kat.txt")
    assert len(kat) == 3
    for words in kat.values():
        w = [int(x, 16) for x in words]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


def test_uniform_mapping_and_range():
    # word 0 -> accept uniform, word 1 -> resample uniform; counter (j, 0, r, 0); 24-bit grid in [0,1)
    seed = 0x1234567890ABCDEF
    for r, j in [(0, 0), (5, 3), (1023, 31), (2**20, 7)]:
        w = oracle.philox4x32_10((j, 0, r, 0), (seed & 0xFFFFFFFF, seed >> 32))
        ua, ur = oracle.uniforms(seed, r, j)
        assert ua == (int(w[0]) >> 8) / 2.0**24
        assert ur == (int(w[1]) >> 8) / 2.0**24
        assert 0.0 <= ua < 1.0 and 0.0 <= ur < 1.0


def test_uniformity_chi_square():
    n, bins = 40000, 64
    u = np.array([oracle.uniforms(7, r, j) for r in range(n // 8) for j in range(8)])
    for col in (0, 1):
        counts = np.bincount((u[:, col] * bins).astype(int), minlength=bins)
        p = stats.chisquare(counts).pvalue
        assert p > 1e-4
    # accept and resample streams are not the same numbers
    assert abs(np.corrcoef(u[:, 0], u[:, 1])[0, 1]) < 0.03


def test_distinct_counters_and_seeds_differ():
    assert oracle.uniforms(1, 0, 0) != oracle.uniforms(2, 0, 0)
    assert oracle.uniforms(1, 0, 0) != oracle.uniforms(1, 1, 0)
    assert oracle.uniforms(1, 0, 0) != oracle.uniforms(1, 0, 1)
    assert oracle.uniforms(1, 2, 3) != oracle.uniforms(1, 3, 2)
