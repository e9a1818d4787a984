"""Pins of the oracle's Sequential Temperature Scaling (Section 3.2.1, post-hoc calibration).

The oracle is checked against things other than itself: a case worked by hand, a numpy restatement of
the ECE built from library routines (digitize / bincount), the closed-form behaviour of temperature
scaling (order preservation, T = 1 is the identity), and a recovery experiment whose answer is known by
construction (confidences made overconfident by a known factor must be given that factor back).
"""
import numpy as np
from scipy.special import expit, logit

import oracle


def _ece_numpy(a, y, n_bins):
    b = np.minimum(np.floor(a * n_bins).astype(np.int64), n_bins - 1)
    sa = np.bincount(b, weights=a, minlength=n_bins)
    sy = np.bincount(b, weights=y.astype(np.float64), minlength=n_bins)
    return np.abs(sy - sa).sum() / len(a)


def test_hand_worked_case():
    # four blocks, one position, two bins.  Confidences 0.2, 0.4 fall in bin 0 (labels 0, 1), 0.6, 0.9 in
    # bin 1 (labels 1, 1): ECE = (|1 - 0.6| + |2 - 1.5|) / 4 = 0.225 at T = 1.
    conf = np.array([[0.2], [0.4], [0.6], [0.9]], dtype=np.float32)
    acc = np.array([0, 1, 1, 3], dtype=np.int32)
    T, eb, ea, eg = oracle.sts_calibrate(conf, acc, [1.0], n_bins=2)
    assert T[0] == 1.0
    c = conf[:, 0].astype(np.float64)
    want = (abs(1 - (c[0] + c[1])) + abs(2 - (c[2] + c[3]))) / 4
    assert abs(eb[0] - want) < 1e-15 and abs(ea[0] - want) < 1e-15 and abs(eg[0, 0] - want) < 1e-15
    assert abs(want - 0.225) < 1e-7          # float32 inputs: 0.2f etc. are not exactly the decimals


def test_ece_and_products_against_numpy():
    rng = np.random.default_rng(3)
    N, gamma, nb = 5000, 6, 15
    conf = rng.uniform(0.05, 0.99, (N, gamma)).astype(np.float32)
    acc = rng.integers(0, gamma + 1, N).astype(np.int32)
    ver = rng.integers(1, gamma + 1, N).astype(np.int32)
    grid = np.array([0.5, 1.0, 2.0], dtype=np.float32)
    T, eb, ea, eg = oracle.sts_calibrate(conf, acc, grid, n_bins=nb, verified_len=ver)
    c64 = conf.astype(np.float64)
    a_raw = np.cumprod(c64, axis=1)
    a_cal = np.ones(N)
    for k in range(gamma):
        use = ver > k
        y = (acc > k)[use]
        assert abs(eb[k] - _ece_numpy(a_raw[use, k], y, nb)) < 1e-12
        e = [_ece_numpy((a_cal * expit(logit(c64[:, k]) / t))[use], y, nb) for t in grid.astype(np.float64)]
        np.testing.assert_allclose(eg[k], e, atol=1e-12)
        g = int(np.argmin(e))                 # first minimum, as the oracle
        assert T[k] == grid[g]
        a_cal = a_cal * expit(logit(c64[:, k]) / float(grid[g]))
        assert abs(ea[k] - e[g]) < 1e-12


def test_recovers_a_known_overconfidence_factor():
    rng = np.random.default_rng(11)
    N, gamma, s = 200_000, 4, 2.0
    z_true = rng.normal(1.2, 1.0, (N, gamma))
    p_true = expit(z_true)
    # block outcome: position k is accepted with its true conditional probability, first failure ends it
    ok = rng.uniform(size=(N, gamma)) < p_true
    acc = np.where(ok.all(1), gamma, np.argmin(ok, axis=1)).astype(np.int32)
    conf = expit(s * z_true).astype(np.float32)          # overconfident by a factor s on the logit
    grid = np.geomspace(0.5, 4.0, 49).astype(np.float32)  # contains 2.0 up to rounding
    T, eb, ea, _ = oracle.sts_calibrate(conf, acc, grid, n_bins=15)
    assert np.all(np.abs(T - s) <= 0.2), T
    assert np.all(ea < 0.25 * eb), (eb, ea)
    assert np.all(ea < 0.01)
    # calibrated confidences keep the ranking inside every position (temperature scaling is monotone)
    cal = oracle.sts_apply(conf, T)
    for k in range(gamma):
        o = np.argsort(conf[:2000, k], kind="stable")
        assert np.all(np.diff(cal[:2000, k][o]) >= 0)
    np.testing.assert_allclose(cal, expit(logit(conf.astype(np.float64)) / T.astype(np.float64)), rtol=1e-12)


def test_identity_and_edge_values():
    conf = np.array([[0.0, 0.5], [1.0, 0.25], [np.nan, 0.75], [1.5, 0.5]], dtype=np.float32)
    out = oracle.sts_apply(conf, [3.0, 1.0])
    np.testing.assert_array_equal(out[:, 0], [0.0, 1.0, 0.0, 1.0])        # clamped, never rescaled
    np.testing.assert_allclose(out[:, 1], [0.5, 0.25, 0.75, 0.5], rtol=1e-15)  # T = 1 is the identity
    # a position nobody verified keeps T = 1 and reports ECE 0
    T, eb, ea, eg = oracle.sts_calibrate(conf, np.zeros(4, np.int32), [0.5, 2.0], verified_len=np.ones(4, np.int32))
    assert T[1] == 1.0 and eb[1] == 0.0 and ea[1] == 0.0 and np.all(eg[1] == 0.0)
