"""Pins for the oracle's Markov-head draft step and confidence head: library matmul in fp64,
torch's own bf16 rounding, and special cases."""
import numpy as np
import torch

import oracle


def _bits(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _f64(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


def test_logits_are_base_plus_low_rank_bias():
    rng = np.random.default_rng(0)
    R, V, rank = 5, 300, 16
    U = _bits(rng.normal(0, 3, (R, V))); W1 = _bits(rng.normal(0, 0.3, (V, rank))); W2 = _bits(rng.normal(0, 0.3, (rank, V)))
    xp = rng.integers(0, V, R)
    f64, b16 = oracle.markov_logits(U, W1, W2, xp)
    want = _f64(U) + _f64(W1)[xp] @ _f64(W2)                      # library matmul, fp64
    np.testing.assert_allclose(f64, want, rtol=1e-13, atol=1e-13)
    # the stored pattern is torch's round-to-nearest-even bf16 of the same number
    np.testing.assert_array_equal(b16, _bits(want))
    # zero projection: logits are the base logits, bit for bit
    _, b0 = oracle.markov_logits(U, W1, np.zeros_like(W2), xp)
    np.testing.assert_array_equal(b0, U)
    # the bias depends only on the previous token: same token, same bias row
    f2, _ = oracle.markov_logits(np.zeros_like(U), W1, W2, np.full(R, 7))
    assert np.ptp(f2, axis=0).max() == 0.0
    # one-hot embedding row i picks row i of W2
    W1h = np.zeros((V, rank), np.float32); W1h[:, 3] = 1.0
    f3, _ = oracle.markov_logits(np.zeros_like(U), _bits(W1h), W2, xp)
    np.testing.assert_array_equal(f3, np.broadcast_to(_f64(W2)[3], (R, V)))


def test_confidence_head():
    rng = np.random.default_rng(1)
    R, d, V, rank = 9, 40, 100, 16
    H = _bits(rng.normal(0, 1, (R, d))); W1 = _bits(rng.normal(0, 1, (V, rank)))
    w = rng.normal(0, 0.2, d + rank).astype(np.float32)
    xp = rng.integers(0, V, R)
    c = oracle.confidence(H, W1, w, xp)
    z = _f64(H) @ w[:d].astype(np.float64) + _f64(W1)[xp] @ w[d:].astype(np.float64)
    np.testing.assert_allclose(c, 1 / (1 + np.exp(-z)), rtol=1e-13)
    assert ((c > 0) & (c < 1)).all()
    assert oracle.confidence(H, W1, np.zeros_like(w), xp).tolist() == [0.5] * R
