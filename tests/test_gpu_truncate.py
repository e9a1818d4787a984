"""GPU top-k / top-p truncation of the target rows vs the oracle.

The top-k part is integer work on the 16-bit keys: bit-exact.  The top-p threshold compares sums of
exponentials with top_p * Z; the oracle reports how close that comparison was (margin, relative to Z), and
a row may differ from the oracle only when the margin is below 1e-5 -- then the GPU's cut must be the
neighbouring value group.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu
MARGIN = 1e-5


def _f(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


def _run(target, off, top_k=None, top_p=None, temperature=1.0, temperatures=None):
    t = target.clone()
    n_rows = t.shape[0]
    tau = torch.full((n_rows,), 7.0, device="cuda")
    kept = torch.full((n_rows,), -7, dtype=torch.int32, device="cuda")
    dev = lambda a, dt: None if a is None else torch.as_tensor(np.asarray(a), dtype=dt, device="cuda")
    B.dspark_truncate_target(t, off, top_k=dev(top_k, torch.int32), top_p=dev(top_p, torch.float32), temperature=temperature,
                             temperatures=dev(temperatures, torch.float32), out_tau=tau, out_kept=kept)
    torch.cuda.synchronize()
    return t, tau.cpu().numpy(), kept.cpu().numpy()


def _check(target, off, top_k=None, top_p=None, temperature=1.0, temperatures=None):
    got, tau, kept = _run(target, off, top_k, top_p, temperature, temperatures)
    bits = W.bf16_bits(target)
    want, otau, okept, margin = oracle.warp_target(bits, off.cpu().numpy(), top_k=top_k, top_p=top_p, temperature=temperature,
                                                   temperatures=temperatures)
    gb = W.bf16_bits(got)
    close = 0
    for row in range(int(off[-1].item())):
        if np.array_equal(gb[row], want[row]):
            assert kept[row] == okept[row]
            assert tau[row] == np.float32(otau[row]) or (np.isneginf(otau[row]) and np.isneginf(tau[row]))
            continue
        # a different cut: only where the oracle's own decision was within MARGIN, and then the kept set is
        # still a value cut of the original row at a neighbouring distinct value
        assert margin[row] < MARGIN, (row, margin[row], kept[row], okept[row])
        x = _f(bits[row])
        np.testing.assert_array_equal(np.isneginf(_f(gb[row])), x < tau[row])
        vals = np.unique(x)
        assert abs(int(np.searchsorted(vals, tau[row])) - int(np.searchsorted(vals, otau[row]))) <= 1
        close += 1
    assert close <= max(1, int(off[-1].item()) // 20)
    return got, tau, kept, close


def test_full_vocabulary_rows_top_k_and_top_p():
    lengths = torch.tensor([2, 0, 3, 1, 4, 0, 2, 1])
    b = W.sampling_batch(lengths, W.V_FULL, 17, "cuda", temperature=0.8)
    R = len(lengths)
    ks = np.array([1, 50, 0, 1000, 20, 129280, 5, 40000], dtype=np.int32)
    ps = np.array([1.0, 0.9, 0.95, 0.5, 1.0, 0.99, 0.0, 0.8], dtype=np.float32)
    Ts = np.array([0.8, 1.0, 0.6, 1.5, 1.0, 0.7, 1.0, 1.2], dtype=np.float32)
    got, tau, kept, close = _check(b.target, b.row_offsets, ks, ps, temperatures=Ts)
    assert kept[0] >= 1 and kept.min() >= 1
    print(f"[truncate] kept sizes {kept.tolist()}, {close} near-boundary rows")


@pytest.mark.parametrize("V", [1000, 4097, 70000])
def test_unaligned_rows_ties_and_flat_rows(V):
    g = torch.Generator(device="cuda").manual_seed(V)
    n = 12
    t = torch.empty(n, V, device="cuda")
    t[0:3] = torch.randn(3, V, generator=g, device="cuda") * 3
    t[3:5] = torch.randint(-3, 4, (2, V), generator=g, device="cuda").float() * 0.5          # few distinct values
    t[5] = 1.25                                                                              # one value only
    t[6:8] = torch.rand(2, V, generator=g, device="cuda") * 2 - 1                            # flat, both signs
    t[8] = -torch.rand(V, generator=g, device="cuda") * 40                                   # all negative
    t[9] = torch.randn(V, generator=g, device="cuda") * 1e-3                                 # tiny values, -0/+0
    t[9, ::7] = -0.0
    t[10:12] = torch.randn(2, V, generator=g, device="cuda") * 8
    t = t.to(torch.bfloat16)
    off = torch.arange(n + 1, dtype=torch.int32, device="cuda")
    ks = np.array([3, 0, V - 1, 10, 0, 5, V // 2, 0, 7, 100, 0, 1], dtype=np.int32)
    ps = np.array([1.0, 0.7, 0.999, 0.6, 0.5, 0.3, 0.9, 0.999, 0.9, 0.5, 0.0, 0.2], dtype=np.float32)
    _check(t, off, ks, ps, temperature=1.3)
    _check(t, off, ks, None, temperature=1.0)
    _check(t, off, None, ps, temperature=0.7)


def test_rows_that_are_left_alone():
    V = 3000
    t = (torch.randn(6, V, device="cuda") * 2).to(torch.bfloat16)
    t[1, 5] = float("nan")
    t[2, 9] = float("inf")
    t[3, :] = float("-inf")
    off = torch.tensor([0, 2, 4, 6], dtype=torch.int32, device="cuda")
    got, tau, kept = _run(t, off, top_k=[4, 4, 0], top_p=[0.9, 0.9, 1.0])
    for row in (1, 2, 3, 4, 5):
        assert torch.equal(got[row].view(torch.int16), t[row].view(torch.int16)) and np.isneginf(tau[row]) and kept[row] == V
    assert kept[0] <= 4 + 5 and not torch.equal(got[0].view(torch.int16), t[0].view(torch.int16))


def test_verifier_on_truncated_rows_matches_the_oracle_pipeline():
    lengths = torch.tensor([3, 1, 0, 4, 2, 5, 0, 1, 2, 3])
    b = W.sampling_batch(lengths, 50_000, 23, "cuda", temperature=1.0, draft_noise=1.0, verify_seed=5)
    R = len(lengths)
    ks = np.full(R, 30, dtype=np.int32)
    ps = np.full(R, 0.9, dtype=np.float32)
    got, tau, kept, close = _check(b.target, b.row_offsets, ks, ps, temperature=1.0)
    assert close == 0
    import sys, os
    sys.path.insert(0, os.path.dirname(__file__))
    import helpers as H
    masked = W.VerifyBatch(got, b.draft, b.row_offsets, b.draft_tokens, b.draft_row_start, b.temperature, b.seed, b.meta)
    g, o, mism = H.check_sampling(masked)
    # every emitted correction / bonus token lies in the kept set of its row
    ro = b.row_offsets.cpu().numpy()
    x = _f(W.bf16_bits(b.target))
    for r in range(R):
        n = int(g["acc"][r]); row = ro[r] + n
        assert x[row, g["out"][row]] >= tau[row]
    print(f"[truncate] verifier on masked rows: accepted {g['acc'].tolist()}, {mism} boundary mismatches")
