"""Pins for the oracle's verifier: library routines (argmax, log-sum-exp), the paper's
Appendix A distributions, the closed-form acceptance rate 1 - TV, chi-square checks of
the lossless-sampling invariant on small vocabularies, and the degenerate cases."""
import numpy as np
import pytest
import torch
from scipy import special, stats

import oracle


def _bf16_bits(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


# ------------------------------------------------------------------ greedy ----
def test_row_argmax_is_numpy_argmax_with_ties_and_bf16():
    rng = np.random.default_rng(0)
    x = rng.normal(0, 4, size=(12, 1000)).astype(np.float32)
    x[3, [10, 500, 900]] = x[3].max() + 1.0          # ties: lowest index must win
    x[4, 77] = np.inf
    x[5] = -np.abs(x[5]) - 1.0; x[5, 2] = -0.0; x[5, 5] = 0.0      # -0.0 == +0.0 is a tie
    x[6, 0] = np.nan                                    # NaN never wins
    ro = np.arange(13, dtype=np.int32)                  # 12 requests, no draft tokens
    res = oracle.verify_greedy(x, ro, np.zeros(12, np.int32))
    want = np.argmax(np.where(np.isnan(x), -np.inf, x), axis=1)
    np.testing.assert_array_equal(res.row_argmax, want)
    assert res.row_argmax[3] == 10 and res.row_argmax[5] == 2
    np.testing.assert_array_equal(res.out_tokens, want)     # l = 0: bonus token = argmax(row 0)
    assert (res.accepted_len == 0).all()
    bits = _bf16_bits(x[:3])
    resb = oracle.verify_greedy(bits, np.arange(4, dtype=np.int32), np.zeros(3, np.int32))
    np.testing.assert_array_equal(resb.row_argmax, np.argmax(_bf16_to_f64(bits), axis=1))


def test_greedy_accept_logic():
    rng = np.random.default_rng(1)
    V = 50
    ro = np.array([0, 4, 5, 9, 12], dtype=np.int32)     # l = 3, 0, 3, 2
    x = rng.normal(size=(12, V)).astype(np.float32)
    am = x.argmax(1).astype(np.int32)
    d = am.copy()
    d[6] = (am[6] + 1) % V          # request 2 mismatches at j = 1
    d[9] = (am[9] + 3) % V          # request 3 mismatches at j = 0
    res = oracle.verify_greedy(x, ro, d)
    np.testing.assert_array_equal(res.accepted_len, [3, 0, 1, 0])
    np.testing.assert_array_equal(res.out_tokens,
                                  [am[0], am[1], am[2], am[3], am[4], am[5], am[6], -1, -1, am[9], -1, -1])
    # all -inf row: index 0 plus a status bit
    x[4] = -np.inf
    res = oracle.verify_greedy(x, ro, d)
    assert res.out_tokens[4] == 0 and res.status[1] & oracle.ST_ALL_NEG_INF
    # invalid token id: nothing emitted for that request
    d[0] = V
    res = oracle.verify_greedy(x, ro, d)
    assert res.status[0] & oracle.ST_BAD_TOKEN and res.accepted_len[0] == 0
    assert (res.out_tokens[0:4] == -1).all()


# ----------------------------------------------------------------- softmax ----
@pytest.mark.parametrize("T", [1.0, 0.7, 2.5])
def test_softmax_stats_against_scipy(T):
    rng = np.random.default_rng(2)
    x = rng.normal(0, 3, size=(3, 4097)).astype(np.float32)
    x[1, 5] = -np.inf
    for row in range(3):
        probs, m, Z, bad = oracle.softmax_row(x, row, T)
        assert not bad
        xs = x[row].astype(np.float64) / T
        assert m + np.log(Z) == pytest.approx(special.logsumexp(xs), rel=1e-13)
        np.testing.assert_allclose(probs, special.softmax(xs), rtol=1e-12, atol=0)
    bits = _bf16_bits(x)
    probs, m, Z, bad = oracle.softmax_row(bits, 0, T)
    np.testing.assert_allclose(probs, special.softmax(_bf16_to_f64(bits)[0] / T), rtol=1e-12)
    x[2, 9] = np.nan
    assert oracle.softmax_row(x, 2, T)[3]
    assert oracle.softmax_row(np.full((1, 8), -np.inf, np.float32), 0, T)[3]


# --------------------------------------------------- acceptance / sampling ----
def _single_position_batch(p, q, n, rng):
    """n independent requests, each with one draft position (rows: position 0 and bonus)."""
    V = len(p)
    tl = np.log(np.asarray(p, dtype=np.float64)).astype(np.float32)
    ql = np.log(np.asarray(q, dtype=np.float64)).astype(np.float32)
    target = np.broadcast_to(tl, (2 * n, V))
    draft = np.broadcast_to(ql, (n, V))
    ro = (2 * np.arange(n + 1)).astype(np.int32)
    qn = np.exp(ql.astype(np.float64)); qn /= qn.sum()
    d = rng.choice(V, size=n, p=qn).astype(np.int32)
    toks = np.zeros(2 * n, np.int32)
    toks[0::2] = d
    return target, draft, ro, toks


def _probs_of(logits_row):
    e = np.exp(logits_row.astype(np.float64))
    return e / e.sum()


def test_appendix_a_distributions(golden):
    g = golden("appendix_a.txt")
    p = [float(x) for x in g["p_target"]]
    q = [float(x) for x in g["p_draft"]]
    n = 200_000
    rng = np.random.default_rng(3)
    target, draft, ro, toks = _single_position_batch(p, q, n, rng)
    res = oracle.verify(target, draft, ro, toks, 1.0, seed=11)
    # acceptance probability sum_x min(p, q) = 0.8
    rate = res.accepted_len.mean()
    want = float(g["accept_prob"][0])
    assert abs(rate - want) < 4 * np.sqrt(want * (1 - want) / n)
    # token A is accepted with probability min(1, 0.7/0.5) = 1
    assert float(g["accept_ratio_A"][0]) == 1.0
    assert (res.accepted_len[toks[0::2] == 0] == 1).all()
    # the residual norm(max(0, p - q)) = (1, 0): every rejection emits A
    rejected = res.accepted_len == 0
    assert (res.out_tokens[0::2][rejected] == 0).all()
    # lossless: first emitted token ~ (0.7, 0.3), and it is NOT the biased (0.85, 0.15)
    first = res.out_tokens[0::2]
    counts = np.bincount(first, minlength=2)
    lossless = np.array([float(x) for x in g["lossless_output"]])
    biased = np.array([float(x) for x in g["biased_output"]])
    assert stats.chisquare(counts, lossless * n).pvalue > 1e-3
    assert stats.chisquare(counts, biased * n).pvalue < 1e-12
    # bonus token after an acceptance ~ p as well
    bonus = res.out_tokens[1::2][~rejected]
    assert stats.chisquare(np.bincount(bonus, minlength=2), lossless * len(bonus)).pvalue > 1e-3


@pytest.mark.parametrize("V,seed", [(3, 0), (8, 1), (16, 2)])
def test_accept_rate_is_one_minus_tv_and_output_is_p(V, seed):
    rng = np.random.default_rng(100 + seed)
    p = rng.dirichlet(np.ones(V) * 0.7)
    q = rng.dirichlet(np.ones(V) * 0.7)
    n = 250_000
    target, draft, ro, toks = _single_position_batch(p, q, n, rng)
    res = oracle.verify(target, draft, ro, toks, 1.0, seed=seed)
    pp, qq = _probs_of(target[0]), _probs_of(draft[0])
    want = 1.0 - 0.5 * np.abs(pp - qq).sum()          # per-step acceptance rate, Eq. (accept_rate)
    rate = res.accepted_len.mean()
    assert abs(rate - want) < 4 * np.sqrt(want * (1 - want) / n)
    first = res.out_tokens[0::2]
    assert stats.chisquare(np.bincount(first, minlength=V), pp * n).pvalue > 1e-3
    # residual support is inside {p > q}
    rej_tok = first[res.accepted_len == 0]
    assert (pp[rej_tok] > qq[rej_tok]).all()
    # and it follows norm(max(0, p - q))
    w = np.maximum(pp - qq, 0); w /= w.sum()
    keep = w > 0
    cnt = np.bincount(rej_tok, minlength=V)
    assert cnt[~keep].sum() == 0
    assert stats.chisquare(cnt[keep], w[keep] * len(rej_tok)).pvalue > 1e-3
    # reported p(d), q(d)
    np.testing.assert_allclose(res.p_tok[0::2], pp[toks[0::2]], rtol=1e-12)
    np.testing.assert_allclose(res.q_tok[0::2], qq[toks[0::2]], rtol=1e-12)


def test_every_position_emits_from_its_own_target_distribution():
    # 3 draft positions with different (p_j, q_j); the token emitted at position j, over the
    # requests that reach j, must follow p_j (accepted draft or residual), the bonus p_3
    rng = np.random.default_rng(7)
    V, L, n = 6, 3, 120_000
    P = rng.dirichlet(np.ones(V), size=L + 1)
    Q = rng.dirichlet(np.ones(V), size=L)
    tl = np.log(P).astype(np.float32)
    ql = np.log(Q).astype(np.float32)
    target = np.broadcast_to(tl[None], (n, L + 1, V)).reshape(n * (L + 1), V)
    draft = np.broadcast_to(ql[None], (n, L, V)).reshape(n * L, V)
    ro = ((L + 1) * np.arange(n + 1)).astype(np.int32)
    toks = np.zeros((n, L + 1), np.int32)
    for j in range(L):
        toks[:, j] = rng.choice(V, size=n, p=_probs_of(ql[j]))
    res = oracle.verify(target, draft, ro, toks.ravel(), 1.0, seed=5)
    out = res.out_tokens.reshape(n, L + 1)
    for j in range(L + 1):
        reached = res.accepted_len >= j
        pj = _probs_of(tl[j])
        cnt = np.bincount(out[reached, j], minlength=V)
        assert stats.chisquare(cnt, pj * reached.sum()).pvalue > 1e-3
        assert (out[~reached, j] == -1).all()
    # expected accepted length = sum_j prod_{i<=j} (1 - TV_i)
    acc = np.array([1 - 0.5 * np.abs(_probs_of(tl[j]) - _probs_of(ql[j])).sum() for j in range(L)])
    assert res.accepted_len.mean() == pytest.approx(np.cumprod(acc).sum(), abs=0.02)


def test_temperature_applies_to_both_distributions():
    rng = np.random.default_rng(8)
    V, n, T = 5, 150_000, 0.7
    tl = rng.normal(0, 1.5, V).astype(np.float32)
    ql = rng.normal(0, 1.5, V).astype(np.float32)
    pT = special.softmax(tl.astype(np.float64) / T)
    qT = special.softmax(ql.astype(np.float64) / T)
    target = np.broadcast_to(tl, (2 * n, V)); draft = np.broadcast_to(ql, (n, V))
    ro = (2 * np.arange(n + 1)).astype(np.int32)
    toks = np.zeros(2 * n, np.int32); toks[0::2] = rng.choice(V, size=n, p=qT)
    res = oracle.verify(target, draft, ro, toks, T, seed=9)
    want = 1 - 0.5 * np.abs(pT - qT).sum()
    assert abs(res.accepted_len.mean() - want) < 4 * np.sqrt(want * (1 - want) / n)
    assert stats.chisquare(np.bincount(res.out_tokens[0::2], minlength=V), pT * n).pvalue > 1e-3


def test_degenerate_cases():
    rng = np.random.default_rng(9)
    V, n = 7, 5000
    p = rng.dirichlet(np.ones(V))
    # q == p: always accept (u < 1), bonus ~ p
    target, draft, ro, toks = _single_position_batch(p, p, n, rng)
    res = oracle.verify(target, draft, ro, toks, 1.0, seed=1)
    assert (res.accepted_len == 1).all() and (res.status == 0).all()
    # p(d) = 0 (target -inf at the draft token): always reject, residual never returns d
    tl = np.log(p).astype(np.float32); tl[2] = -np.inf
    target = np.broadcast_to(tl, (2 * n, V))
    toks2 = toks.copy(); toks2[0::2] = 2
    res = oracle.verify(target, draft, ro, toks2, 1.0, seed=1)
    assert (res.accepted_len == 0).all() and (res.out_tokens[0::2] != 2).all()
    assert (res.p_tok[0::2] == 0).all()
    # l = 0 for every request: one bonus token each, drawn from p
    ro0 = np.arange(n + 1, dtype=np.int32)
    res = oracle.verify(np.broadcast_to(np.log(p).astype(np.float32), (n, V)),
                        np.zeros((1, V), np.float32), ro0, np.zeros(n, np.int32), 1.0, seed=2)
    assert (res.accepted_len == 0).all()
    assert stats.chisquare(np.bincount(res.out_tokens, minlength=V), _probs_of(np.log(p).astype(np.float32)) * n).pvalue > 1e-3
    # NaN row / invalid token / bad offsets -> status, nothing emitted
    bad = np.log(p).astype(np.float32).reshape(1, V).repeat(2, 0); bad[0, 1] = np.nan
    r = oracle.verify(bad, bad[:1], [0, 2], [1, 0], 1.0, seed=3)
    assert r.status[0] & oracle.ST_BAD_ROW and r.accepted_len[0] == 0 and (r.out_tokens == -1).all()
    ok = np.log(p).astype(np.float32).reshape(1, V).repeat(2, 0)
    r = oracle.verify(ok, ok[:1], [0, 2], [V, 0], 1.0, seed=3)
    assert r.status[0] & oracle.ST_BAD_TOKEN and (r.out_tokens == -1).all()
    # a request without a row of its own: reported; in the compact layout the draft rows of the next request would
    # start before the array (off[1] - 1 = -1), so it is reported too and nothing is read; with explicit draft row
    # starts the next request is verified as usual
    r = oracle.verify(ok, ok[:1], [0, 0, 2], [0, 0], 1.0, seed=3)
    assert r.status[0] & oracle.ST_BAD_OFFSETS and r.status[1] & oracle.ST_BAD_OFFSETS and (r.out_tokens == -1).all()
    r = oracle.verify(ok, ok[:1], [0, 0, 2], [0, 0], 1.0, seed=3, draft_row_start=np.array([0, 0], dtype=np.int64))
    assert r.status[0] & oracle.ST_BAD_OFFSETS and r.status[1] == 0 and r.out_tokens[1] >= 0


def test_inverse_cdf_against_cumsum_searchsorted():
    rng = np.random.default_rng(10)
    V, R = 2000, 300
    x = rng.normal(0, 3, size=(R, V)).astype(np.float32)
    ro = np.arange(R + 1, dtype=np.int32)
    res = oracle.verify(x, np.zeros((1, V), np.float32), ro, np.zeros(R, np.int32), 1.0, seed=21)
    for r in range(R):
        _, ur = oracle.uniforms(21, r, 0)
        cdf = np.cumsum(special.softmax(x[r].astype(np.float64)))
        want = int(np.searchsorted(cdf, ur, side="right"))       # smallest v with cdf[v] > u
        if res.token_margin[r] > 1e-12:
            assert res.out_tokens[r] == want
    # residual draw against an explicit cumulative sum
    y = (x + rng.normal(0, 1, size=x.shape)).astype(np.float32)
    ro2 = (2 * np.arange(R // 2 + 1)).astype(np.int32)
    toks = np.zeros(R, np.int32)
    toks[0::2] = [int(np.argmin(x[2 * r] - y[r])) for r in range(R // 2)]   # p/q smallest: mostly rejected
    res = oracle.verify(x, y[: R // 2], ro2, toks, 1.0, seed=22)
    n_rej = 0
    for r in range(R // 2):
        if res.accepted_len[r] == 0:
            n_rej += 1
            _, ur = oracle.uniforms(22, r, 0)
            w = np.maximum(special.softmax(x[2 * r].astype(np.float64)) - special.softmax(y[r].astype(np.float64)), 0)
            cdf = np.cumsum(w)
            want = int(np.searchsorted(cdf, ur * cdf[-1], side="right"))
            # margins against an independent statement: the CDF of the residual distribution itself,
            # cumsum(max(0, p - q) / W); the absolute margin is that distance times W
            W = cdf[-1]
            ncdf = np.cumsum(w / W)
            prev_n = ncdf[want - 1] if want else 0.0
            norm = min(ur - prev_n, ncdf[want] - ur)
            if norm > 1e-9:
                assert res.out_tokens[2 * r] == want
                assert abs(res.token_margin[r] - norm) < 1e-9
                assert abs(res.token_margin_abs[r] - norm * W) < 1e-9 * W + 1e-15
                assert abs(res.resid_mass[r] - W) < 1e-12
    assert n_rej > 50


def test_threads_and_eval_all_do_not_change_results():
    rng = np.random.default_rng(11)
    V, R, L = 300, 40, 4
    ro = ((L + 1) * np.arange(R + 1)).astype(np.int32)
    x = rng.normal(0, 3, size=(R * (L + 1), V)).astype(np.float32)
    y = rng.normal(0, 3, size=(R * L, V)).astype(np.float32)
    toks = rng.integers(0, V, size=R * (L + 1)).astype(np.int32)
    a = oracle.verify(x, y, ro, toks, 0.9, seed=4, eval_all=True, n_threads=1)
    b = oracle.verify(x, y, ro, toks, 0.9, seed=4, eval_all=False, n_threads=3)
    np.testing.assert_array_equal(a.accepted_len, b.accepted_len)
    np.testing.assert_array_equal(a.out_tokens, b.out_tokens)
    # non-compact draft layout: rows of request r start at r * L
    c = oracle.verify(x, y, ro, toks, 0.9, seed=4, draft_row_start=np.arange(R) * L)
    np.testing.assert_array_equal(a.out_tokens, c.out_tokens)


def test_per_request_temperatures():
    # every request carries its own temperature: each one's first emitted token must follow
    # softmax(target / T_r), and the acceptance rate 1 - TV at that temperature
    rng = np.random.default_rng(12)
    V, n = 6, 90_000
    temps = np.array([0.6, 1.0, 1.7], dtype=np.float32)
    tl = rng.normal(0, 1.5, V).astype(np.float32)
    ql = rng.normal(0, 1.5, V).astype(np.float32)
    R = 3 * n
    Tr = np.tile(temps, n)
    target = np.broadcast_to(tl, (2 * R, V)); draft = np.broadcast_to(ql, (R, V))
    ro = (2 * np.arange(R + 1)).astype(np.int32)
    toks = np.zeros(2 * R, np.int32)
    for k, T in enumerate(temps):
        qT = special.softmax(ql.astype(np.float64) / T)
        toks[0::2][k::3] = rng.choice(V, size=n, p=qT)
    res = oracle.verify(target, draft, ro, toks, 1.0, seed=31, temperatures=Tr, n_threads=4)
    for k, T in enumerate(temps):
        pT = special.softmax(tl.astype(np.float64) / T); qT = special.softmax(ql.astype(np.float64) / T)
        first = res.out_tokens[0::2][k::3]
        assert stats.chisquare(np.bincount(first, minlength=V), pT * n).pvalue > 1e-3
        want = 1 - 0.5 * np.abs(pT - qT).sum()
        assert abs(res.accepted_len[k::3].mean() - want) < 4 * np.sqrt(want * (1 - want) / n)
    # a uniform array gives exactly the scalar result; a bad temperature kills only its request
    a = oracle.verify(target[:40], draft[:20], ro[:21], toks[:40], 0.8, seed=5)
    b = oracle.verify(target[:40], draft[:20], ro[:21], toks[:40], 123.0, seed=5, temperatures=np.full(20, 0.8, np.float32))
    np.testing.assert_array_equal(a.out_tokens, b.out_tokens)
    bad = np.full(20, 0.8, np.float32); bad[3] = 0.0; bad[7] = np.nan
    c = oracle.verify(target[:40], draft[:20], ro[:21], toks[:40], 1.0, seed=5, temperatures=bad)
    assert c.status[3] & oracle.ST_BAD_TEMPERATURE and c.status[7] & oracle.ST_BAD_TEMPERATURE
    assert (c.out_tokens[6:8] == -1).all() and c.accepted_len[3] == 0
    keep = np.ones(40, bool); keep[6:8] = False; keep[14:16] = False
    np.testing.assert_array_equal(c.out_tokens[keep], a.out_tokens[keep])


def test_accept_rate_label(golden):
    # Eq. (accept_rate): c* = 1 - 1/2 ||p_d - p_t||_1.  Appendix A pair: 0.8.
    g = golden("appendix_a.txt")
    p = np.array([float(x) for x in g["p_target"]]); q = np.array([float(x) for x in g["p_draft"]])
    tl = np.log(p).astype(np.float32).reshape(1, 2).repeat(2, 0); ql = np.log(q).astype(np.float32).reshape(1, 2)
    c, st = oracle.accept_rate(tl, ql, [0, 2], 1.0)
    assert c[0] == pytest.approx(float(g["accept_prob"][0]), abs=1e-7) and np.isnan(c[1]) and st[0] == 0
    # against numpy on random rows, several temperatures, ragged batch, block layout of the draft rows
    rng = np.random.default_rng(13)
    V, lens = 700, np.array([2, 0, 3, 1])
    ro = np.concatenate([[0], np.cumsum(lens + 1)]).astype(np.int32)
    x = rng.normal(0, 3, size=(ro[-1], V)).astype(np.float32)
    y = rng.normal(0, 3, size=(4 * 3, V)).astype(np.float32)              # block layout: request r starts at 3 r
    for T in (0.7, 1.0, 1.9):
        c, st = oracle.accept_rate(x, y, ro, T, draft_row_start=np.arange(4) * 3)
        for r in range(4):
            for j in range(lens[r]):
                pp = special.softmax(x[ro[r] + j].astype(np.float64) / T)
                qq = special.softmax(y[3 * r + j].astype(np.float64) / T)
                assert c[ro[r] + j] == pytest.approx(1 - 0.5 * np.abs(pp - qq).sum(), abs=1e-12)
            assert np.isnan(c[ro[r + 1] - 1])
    # identical distributions: c* = 1; the empirical acceptance frequency of the verifier converges to c*
    c, _ = oracle.accept_rate(x[:2], x[:1], [0, 2], 1.3)
    assert c[0] == pytest.approx(1.0, abs=1e-12)
    n = 100_000
    pq = rng.dirichlet(np.ones(5), size=2)
    tl = np.log(pq[0]).astype(np.float32); ql = np.log(pq[1]).astype(np.float32)
    target = np.broadcast_to(tl, (2 * n, 5)); draft = np.broadcast_to(ql, (n, 5))
    ro = (2 * np.arange(n + 1)).astype(np.int32)
    toks = np.zeros(2 * n, np.int32); toks[0::2] = rng.choice(5, size=n, p=_probs_of(ql))
    res = oracle.verify(target, draft, ro, toks, 1.0, seed=77, n_threads=4)
    c, _ = oracle.accept_rate(target[:2], draft[:1], [0, 2], 1.0)
    assert abs(res.accepted_len.mean() - c[0]) < 4 * np.sqrt(c[0] * (1 - c[0]) / n)


def test_threaded_greedy_oracle_equals_the_sequential_one():
    # the threaded variant (what the benchmark times as the CPU baseline) against the sequential one on a ragged
    # batch with ties, a token out of range and a row without any element above -inf
    rng = np.random.default_rng(77)
    V = 513
    lengths = rng.integers(0, 7, size=37)
    ro = np.concatenate([[0], np.cumsum(lengths + 1)]).astype(np.int32)
    n_rows = int(ro[-1])
    x = np.round(rng.normal(0, 2, size=(n_rows, V))).astype(np.float32)      # rounded: many exact ties
    x[int(ro[2]), :] = -np.inf                                               # first row of a request: always looked at
    x[9, 100:] = -np.inf
    toks = np.argmax(x, axis=1).astype(np.int32)
    flip = rng.random(n_rows) < 0.3
    toks[flip] = rng.integers(0, V, size=int(flip.sum()))
    bad_req = int(np.nonzero(lengths >= 1)[0][3])
    toks[int(ro[bad_req])] = V + 3                                           # a draft token outside the vocabulary
    want = oracle.verify_greedy(x, ro, toks)
    assert want.status[bad_req] & oracle.ST_BAD_TOKEN and (want.accepted_len > 0).any()
    assert (want.status & oracle.ST_ALL_NEG_INF).any()
    for threads in (1, 3, 8, 64):
        acc, out, st = oracle.verify_greedy_mt(x, ro, toks, threads)
        np.testing.assert_array_equal(acc, want.accepted_len)
        np.testing.assert_array_equal(out, want.out_tokens)
        np.testing.assert_array_equal(st, want.status)
    xb = (x.view(np.uint32) >> 16).astype(np.uint16)                         # the same rows as bf16 patterns
    wb = oracle.verify_greedy(xb, ro, toks)
    acc, out, st = oracle.verify_greedy_mt(xb, ro, toks, 5)
    np.testing.assert_array_equal(acc, wb.accepted_len)
    np.testing.assert_array_equal(out, wb.out_tokens)
    np.testing.assert_array_equal(st, wb.status)
