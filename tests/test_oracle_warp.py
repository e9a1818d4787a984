"""Pins of the oracle's top-k / top-p truncation of the target rows (per-request sampling parameters).

Checked against library routines (torch.topk, torch.sort + cumsum of a softmax) on rows without ties, a
brute-force statement of the value-cut definition on tiny rows with ties, and invariants (the kept set
is closed upwards in value, never empty, masked entries are exactly -inf, rows that switch the
truncation off or cannot be normalised are left alone).
"""
import numpy as np
import torch

import oracle


def _rows(n, V, seed, scale=3.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(n, V, generator=g) * scale).float()


def test_top_k_matches_torch_topk_without_ties():
    t = _rows(6, 500, 1)
    off = np.arange(7, dtype=np.int32)
    ks = np.array([1, 5, 50, 499, 0, 700], dtype=np.int32)
    out, tau, kept, _ = oracle.warp_target(t.numpy(), off, top_k=ks)
    for r in range(6):
        k = int(ks[r])
        if k <= 0 or k >= 500:
            np.testing.assert_array_equal(out[r], t[r].numpy()); assert kept[r] == 500 and tau[r] == -np.inf
            continue
        idx = torch.topk(t[r], k).indices.numpy()
        keep = np.zeros(500, bool); keep[idx] = True
        np.testing.assert_array_equal(np.isneginf(out[r]), ~keep)
        np.testing.assert_array_equal(out[r][keep], t[r].numpy()[keep])
        assert kept[r] == k and tau[r] == float(torch.topk(t[r], k).values[-1])


def test_top_p_matches_sorted_cumsum_without_ties():
    t = _rows(8, 400, 2)
    off = np.arange(9, dtype=np.int32)
    ps = np.array([0.1, 0.5, 0.9, 0.99, 1.0, 0.0, 0.75, 0.3], dtype=np.float32)
    Ts = np.array([1.0, 0.7, 1.3, 1.0, 1.0, 1.0, 2.0, 0.5], dtype=np.float32)
    out, tau, kept, margin = oracle.warp_target(t.numpy(), off, top_p=ps, temperatures=Ts)
    for r in range(8):
        p, T = float(ps[r]), float(Ts[r])
        if p >= 1.0:
            np.testing.assert_array_equal(out[r], t[r].numpy()); continue
        probs = torch.softmax(t[r].double() / T, 0)
        sp, si = torch.sort(probs, descending=True)
        n = 1 if p <= 0 else int(torch.searchsorted(torch.cumsum(sp, 0), torch.tensor(p, dtype=torch.float64)).item()) + 1
        keep = np.zeros(400, bool); keep[si[:n].numpy()] = True
        assert margin[r] > 1e-9 or p <= 0          # the decision was not a coin flip
        np.testing.assert_array_equal(np.isneginf(out[r]), ~keep)
        assert kept[r] == n


def _brute(vals, T, k, p):
    """Value-cut definition written out: candidates for tau are the distinct values."""
    V = len(vals)
    m = vals.max()
    w = np.exp((vals - m) / T)
    distinct = np.sort(np.unique(vals))[::-1]
    tau_k = -np.inf
    if 0 < k < V:
        tau_k = next(t for t in distinct if (vals >= t).sum() >= k)          # largest tau keeping >= k tokens
    in_k = vals >= tau_k
    tau_p = -np.inf
    if p < 1.0:
        Zk = w[in_k].sum()
        if p <= 0:
            tau_p = m
        else:
            tau_p = next(t for t in distinct if w[in_k & (vals >= t)].sum() >= p * Zk)
    return max(tau_k, tau_p)


def test_ties_follow_the_value_cut_definition():
    rng = np.random.default_rng(5)
    for case in range(300):
        V = int(rng.integers(2, 10))
        vals = rng.integers(-3, 4, V).astype(np.float32) * 0.5        # few distinct values: many ties
        k = int(rng.integers(0, V + 2))
        p = float(rng.choice([0.0, 0.2, 0.5, 0.8, 0.95, 1.0]))
        T = float(rng.choice([0.5, 1.0, 2.0]))
        out, tau, kept, margin = oracle.warp_target(vals[None, :], [0, 1], top_k=[k], top_p=[p], temperature=T)
        if not (0 < k < V) and p >= 1.0:
            assert tau[0] == -np.inf and kept[0] == V
            continue
        if p < 1.0 and margin[0] < 1e-12:
            continue                                                  # exact tie of cumulative mass and threshold
        want = _brute(vals.astype(np.float64), T, k, p)
        assert tau[0] == want, (vals, k, p, T, tau[0], want)
        np.testing.assert_array_equal(np.isneginf(out[0]), vals < want)
        assert kept[0] == (vals >= want).sum() >= 1


def test_top_k_then_top_p_renormalises_over_the_top_k_set():
    # probabilities 0.5, 0.25, 0.125, 0.125: top-k = 2 leaves (2/3, 1/3); top-p = 0.6 then keeps one token,
    # whereas top-p = 0.6 on the full row would keep two.
    x = np.log(np.array([[0.5, 0.25, 0.125, 0.125]])).astype(np.float32)
    out, _, kept, _ = oracle.warp_target(x, [0, 1], top_k=[2], top_p=[0.6])
    assert kept[0] == 1 and np.isneginf(out[0]).tolist() == [False, True, True, True]
    out, _, kept, _ = oracle.warp_target(x, [0, 1], top_p=[0.6])
    assert kept[0] == 2


def test_bf16_rows_request_parameters_and_untouched_rows():
    t = (_rows(7, 300, 9) * 1.0).to(torch.bfloat16)
    bits = t.view(torch.int16).numpy().view(np.uint16).copy()
    bits[5, 17] = 0x7FC0                                              # NaN: that row is left alone
    off = np.array([0, 3, 4, 7], dtype=np.int32)                      # three requests: rows 0-2, 3, 4-6
    out, tau, kept, _ = oracle.warp_target(bits, off, top_k=[10, 0, 4], top_p=[1.0, 1.0, 0.9])
    f = lambda b: (b.astype(np.uint32) << 16).view(np.float32)
    for row in (0, 1, 2):
        assert kept[row] >= 10 and (f(out[row]) >= tau[row]).sum() == kept[row]
        assert (out[row][f(bits[row]) < tau[row]] == 0xFF80).all()
        assert kept[row] == (f(bits[row]) >= np.sort(f(bits[row]))[-10]).sum()      # ties with the 10th value kept
    np.testing.assert_array_equal(out[3], bits[3])
    np.testing.assert_array_equal(out[5], bits[5])                    # NaN row untouched
    for row in (4, 6):
        assert 1 <= kept[row] <= (f(bits[row]) >= np.sort(f(bits[row]))[-4]).sum()


def test_verifier_on_masked_rows_never_emits_a_masked_token():
    t = _rows(12, 200, 4, scale=1.0)
    off = np.arange(13, dtype=np.int32)
    masked, tau, kept, _ = oracle.warp_target(t.numpy(), off, top_k=np.full(12, 5, np.int32))
    for seed in range(40):
        o = oracle.verify(masked, masked, off, np.zeros(12, np.int32), 1.0, seed)
        assert (o.status == 0).all()
        tok = o.out_tokens[:12]
        assert all(masked[r, tok[r]] >= tau[r] for r in range(12))
