"""Pins for the oracle's scheduler: the paper's worked example (Appendix A), brute
force on tiny batches, monotonicity, library routines and closed-form special cases."""
import itertools

import numpy as np
import pytest

import oracle

TWO40 = 2.0**40


def _f(golden_vals):
    return [float(x) for x in golden_vals]


def _appendix_table(g):
    sps = _f(g["sps"])
    # dense table over B = 0..3 (B = 0 is never looked up)
    return np.array([sps[0], sps[0], sps[1], sps[2]])


@pytest.mark.parametrize("case", ["case1", "case2"])
def test_appendix_a_worked_example(golden, case):
    g = golden("appendix_a.txt")
    table = _appendix_table(g)
    a1 = _f(g["a1"])[0]
    c2 = _f(g[f"{case}_c2"])[0]
    conf = np.array([[a1, c2]], dtype=np.float32)
    early = oracle.schedule(conf, table, budget_tokens=3, mode=oracle.MODE_EARLY_STOP)
    glob = oracle.schedule(conf, table, budget_tokens=3, mode=oracle.MODE_GLOBAL)
    # survival products a1, a2 = a1 * c2
    assert early.survival[0, 0] == pytest.approx(a1, rel=1e-7)
    assert early.survival[0, 1] == pytest.approx(_f(g[f"{case}_a2"])[0], rel=1e-6, abs=0)
    # Theta path: Theta_0, Theta_1 (and Theta_2 when a2 > 0 is a candidate)
    path = glob.theta_path / TWO40
    assert path[0] == pytest.approx(_f(g["theta0"])[0], rel=1e-9)
    assert path[1] == pytest.approx(_f(g["theta1"])[0], rel=1e-7)
    if c2 > 0:
        assert path[2] == pytest.approx(_f(g[f"{case}_theta2"])[0], rel=1e-7)
    else:
        assert glob.n_candidates == 1      # a2 = 0 is not in the candidate space
    assert int(early.lengths[0]) == int(g[f"{case}_len_early"][0])
    assert int(glob.lengths[0]) == int(g[f"{case}_len_global"][0])
    # early stop never evaluated Theta_2
    assert np.isnan(early.theta_path[2])
    assert early.theta == pytest.approx(_f(g["theta0"])[0], rel=1e-12)


def test_initial_state_is_R_times_SPS_R():
    rng = np.random.default_rng(0)
    table = np.linspace(50.0, 1.0, 200)
    for R in (1, 3, 17):
        conf = rng.uniform(0.1, 0.9, size=(R, 4)).astype(np.float32)
        res = oracle.schedule(conf, table, budget_tokens=R, mode=oracle.MODE_GLOBAL)  # cap 0
        assert res.n_admitted == 0 and res.B == R
        assert (res.lengths == 0).all()
        assert res.tau == R
        assert res.theta == R * table[R]


def test_survival_matches_cumprod_and_is_monotone():
    rng = np.random.default_rng(1)
    conf = rng.uniform(0.0, 1.0, size=(64, 16)).astype(np.float32)
    res = oracle.schedule(conf, np.ones(2000), budget_tokens=2000)
    ref = np.cumprod(conf, axis=1, dtype=np.float32)
    np.testing.assert_array_equal(res.survival, ref)
    assert (np.diff(res.survival, axis=1) <= 0).all()


def test_sps_table_against_interp_and_breakpoints():
    bp_t = np.array([1, 128, 256, 384, 512, 640, 768, 1024])
    bp_s = np.array([120.0, 118, 112, 104, 92, 84, 70, 50])
    tab = oracle.sps_table(bp_t, bp_s, 1500)
    for t, s in zip(bp_t, bp_s):
        assert tab[t] == s                      # passes through every breakpoint exactly
    assert tab[0] == bp_s[0]                    # constant below the first
    assert (tab[1024:] == bp_s[-1]).all()       # constant beyond the last
    np.testing.assert_allclose(tab, np.interp(np.arange(1501), bp_t, bp_s), rtol=1e-14)
    # second differences vanish inside a segment (linear)
    seg = tab[129:256]
    assert np.abs(np.diff(seg, 2)).max() < 1e-12
    with pytest.raises(ValueError):
        oracle.sps_table([4, 4], [1.0, 2.0], 10)


def _random_tables(rng, n, size):
    for _ in range(n):
        kind = rng.integers(0, 3)
        if kind == 0:       # smooth decreasing
            yield np.sort(rng.uniform(1, 100, size))[::-1].copy()
        elif kind == 1:     # jagged
            yield rng.uniform(1, 100, size)
        else:               # step-wise cliffs
            yield np.repeat(np.sort(rng.uniform(1, 100, (size + 3) // 4))[::-1], 4)[:size].copy()


def test_global_equals_bruteforce_on_tiny_batches():
    rng = np.random.default_rng(2)
    n_checked = 0
    for R, gamma in [(1, 2), (2, 3), (3, 3), (4, 4), (3, 4)]:
        for table in _random_tables(rng, 12, R * (gamma + 1) + 2):
            conf = rng.uniform(0.2, 1.0, size=(R, gamma)).astype(np.float32)
            if rng.random() < 0.3:
                conf[rng.integers(0, R), rng.integers(0, gamma)] = 0.0
            budget = int(rng.integers(R, R * (gamma + 1) + 1))
            res = oracle.schedule(conf, table, budget, mode=oracle.MODE_GLOBAL)
            best, best_B, _ = oracle.schedule_bruteforce(conf, table, budget)
            assert res.theta * TWO40 == best
            assert res.B == best_B        # first maximiser on the path = smallest batch among optima
            assert res.B <= max(budget, R)
            n_checked += 1
    assert n_checked == 60


def test_bruteforce_itself_against_python_enumeration():
    # the exhaustive companion is pinned too: plain Python enumeration in exact rationals
    from fractions import Fraction
    rng = np.random.default_rng(3)
    R, gamma = 3, 3
    conf = rng.uniform(0.3, 1.0, size=(R, gamma)).astype(np.float32)
    table = rng.uniform(1, 10, R * (gamma + 1) + 1)
    surv = np.cumprod(conf, axis=1, dtype=np.float32)
    best = None
    for lens in itertools.product(range(gamma + 1), repeat=R):
        tau = Fraction(R) + sum(Fraction(int(float(surv[r, j]) * TWO40), 2**40)
                                for r in range(R) for j in range(lens[r]))
        theta = tau * Fraction(float(table[R + sum(lens)]))
        best = theta if best is None or theta > best else best
    got, _, _ = oracle.schedule_bruteforce(conf, table, R * (gamma + 1))
    assert got / TWO40 == pytest.approx(float(best), rel=1e-15)


def test_early_stop_equals_global_when_theta_is_unimodal():
    rng = np.random.default_rng(4)
    for _ in range(20):
        R, gamma = 16, 8
        conf = rng.uniform(0.3, 0.99, size=(R, gamma)).astype(np.float32)
        B = np.arange(R * (gamma + 1) + 1)
        table = 100.0 - 0.002 * B.astype(float) ** 2        # concave decreasing capacity curve
        e = oracle.schedule(conf, table, 10**6, mode=oracle.MODE_EARLY_STOP)
        g = oracle.schedule(conf, table, 10**6, mode=oracle.MODE_GLOBAL)
        path = g.theta_path[: g.n_candidates + 1]
        peak = int(np.argmax(path))
        assert (np.diff(path[: peak + 1]) > 0).all() and (np.diff(path[peak:]) <= 0).all()
        np.testing.assert_array_equal(e.lengths, g.lengths)
        assert e.n_admitted == g.n_admitted == peak


def test_early_stop_halts_at_first_non_improvement_even_if_later_is_better():
    # a cliff then a plateau: Theta dips, then recovers beyond the dip
    conf = np.full((1, 4), 0.9, dtype=np.float32)
    table = np.array([1.0, 1.0, 0.4, 0.4, 0.4, 0.4])
    e = oracle.schedule(conf, table, 10, mode=oracle.MODE_EARLY_STOP)
    g = oracle.schedule(conf, table, 10, mode=oracle.MODE_GLOBAL)
    assert e.lengths[0] == 0
    assert g.lengths[0] == 4          # (1+.9+.81+.729+.6561)*0.4 = 1.638 > 1
    # equality is not an improvement (strict '>'): flat Theta never admits
    flat = np.array([[1.0, 1.0]], dtype=np.float32)
    table = np.array([6.0, 6.0, 3.0, 2.0])      # Theta_i = (1+i) * 6/(1+i) = 6
    assert oracle.schedule(flat, table, 10, mode=oracle.MODE_EARLY_STOP).lengths[0] == 0
    assert oracle.schedule(flat, table, 10, mode=oracle.MODE_GLOBAL).lengths[0] == 0


def test_budget_constant_and_steep_profiles():
    rng = np.random.default_rng(5)
    R, gamma = 32, 8
    conf = rng.uniform(0.5, 1.0, size=(R, gamma)).astype(np.float32)
    const = np.ones(R * (gamma + 1) + 1)
    for budget in (R, R + 1, R + 57, R * (gamma + 1), 10**5):
        res = oracle.schedule(conf, const, budget)
        cap = min(budget - R, R * gamma)
        assert res.n_admitted == cap                       # SPS const: admit up to the cap
        assert int((res.lengths + 1).sum()) == res.B <= max(budget, R)
        # the admitted set is the top-cap survival values
        surv = np.sort(res.survival.ravel())[::-1]
        admitted = np.concatenate([res.survival[r, : res.lengths[r]] for r in range(R)])
        np.testing.assert_array_equal(np.sort(admitted)[::-1], surv[:cap])
    steep = 1.0 / np.arange(1, R * (gamma + 1) + 2) ** 2
    res = oracle.schedule(conf, steep, 10**5)
    assert (res.lengths == 0).all()
    low = oracle.schedule(conf, const, R - 5)
    assert (low.lengths == 0).all() and low.status & oracle.ST_BUDGET_LT_R


def test_lengths_are_prefixes_of_the_sorted_order():
    rng = np.random.default_rng(6)
    R, gamma = 8, 6
    conf = rng.uniform(0.4, 1.0, size=(R, gamma)).astype(np.float32)
    conf[:, 2] = 1.0                       # ties inside a request
    conf[3] = conf[4]                      # ties across requests
    table = np.linspace(10, 9, R * (gamma + 1) + 1)
    for K in range(0, R * gamma + 1, 5):
        res = oracle.schedule(conf, table, 10**5, mode=oracle.MODE_TOPK, topk_K=K)
        assert res.n_admitted == K
        # independent ordering: (a desc, j asc, r asc) via a stable lexsort
        surv = res.survival
        rr, jj = np.meshgrid(np.arange(R), np.arange(gamma), indexing="ij")
        order = np.lexsort((rr.ravel(), jj.ravel(), -surv.ravel().astype(np.float64)))
        want = np.bincount(rr.ravel()[order[:K]], minlength=R)
        np.testing.assert_array_equal(res.lengths, want)


def test_draft_len_and_confidence_sanitising():
    conf = np.array([[0.9, 0.9, 0.9, 0.9], [0.8, np.nan, 0.9, 0.9], [1.5, -0.2, 0.5, 0.5]], dtype=np.float32)
    table = np.ones(20)
    res = oracle.schedule(conf, table, 100, draft_len=[2, 4, 4])
    np.testing.assert_array_equal(res.lengths, [2, 1, 1])
    assert res.status & oracle.ST_CONF_CLAMPED
    assert res.survival[2, 0] == 1.0 and res.survival[2, 1] == 0.0
    assert res.survival[0, 2] == 0.0
    np.testing.assert_allclose(res.expected_len, [1 + 0.9 + 0.81, 1.8, 2.0], rtol=1e-6)
    # tau counts one token per request plus the admitted survival mass
    assert res.tau == pytest.approx(3 + 0.9 + 0.81 + 0.8 + 1.0, rel=1e-6)


def test_async_topk_uses_the_capacity_of_two_steps_earlier():
    # Section 5.2: K at step t comes from the no-break search on the confidences of step t-2,
    # the ranking from the current confidences.  Tiny batches: the capacity is checked against the
    # exhaustive optimum, the admitted set against an independent top-K by sorting.
    rng = np.random.default_rng(21)
    R, gamma, budget = 3, 4, 12
    table = np.array([0, 9.0, 8.8, 8.5, 8.0, 7.2, 6.5, 5.0, 4.9, 4.8, 3.0, 2.0, 1.0, 0.5])
    K0 = 2
    state = np.array([0, K0, K0], dtype=np.int32)
    confs = [rng.uniform(0.3, 1.0, size=(R, gamma)).astype(np.float32) for _ in range(7)]
    optimal_counts = []
    for t, conf in enumerate(confs):
        _, best_B, _ = oracle.schedule_bruteforce(conf, table, budget)
        optimal_counts.append(best_B - R)
        res = oracle.schedule_async(conf, table, budget, state)
        K_expected = K0 if t < 2 else optimal_counts[t - 2]
        assert res.n_admitted == min(K_expected, budget - R, R * gamma)
        surv = np.cumprod(conf, axis=1, dtype=np.float32)
        rr, jj = np.meshgrid(np.arange(R), np.arange(gamma), indexing="ij")
        order = np.lexsort((rr.ravel(), jj.ravel(), -surv.ravel().astype(np.float64)))
        want = np.bincount(rr.ravel()[order[: res.n_admitted]], minlength=R)
        np.testing.assert_array_equal(res.lengths, want)
        assert state[0] == t + 1
    # after the loop the two slots hold the capacities found on the last two steps
    assert sorted(state[1:3].tolist()) == sorted(optimal_counts[-2:])
