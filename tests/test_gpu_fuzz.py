"""Randomised small cases: many shapes, strides, dtypes, temperatures and schedules, each compared
with the oracle under the same bars as the configuration tests."""
import numpy as np
import pytest
import torch

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _pad_rows(t, rng):
    """Same values in a buffer with a random row stride and a random element offset."""
    pad = int(rng.integers(0, 9))
    shift = int(rng.integers(0, 5))
    buf = torch.zeros(t.shape[0], t.shape[1] + pad + shift, dtype=t.dtype, device=t.device)
    buf[:, shift:shift + t.shape[1]] = t
    return buf[:, shift:shift + t.shape[1]]


@pytest.mark.parametrize("seed", range(12))
def test_sampling_fuzz(seed):
    rng = np.random.default_rng(1000 + seed)
    total_mism = 0
    for _ in range(6):
        R = int(rng.integers(1, 30))
        V = int(rng.choice([1, 2, 3, 17, 255, 1024, 2049, 5000, 12345]))
        lengths = torch.from_numpy(rng.integers(0, 10, size=R))
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        block = int(lengths.max()) + int(rng.integers(0, 3)) if rng.random() < 0.5 and int(lengths.max()) > 0 else None
        b = W.sampling_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", dtype=dtype,
                             sigma=float(rng.uniform(0.5, 4)), draft_noise=float(rng.uniform(0.0, 2.5)),
                             temperature=float(rng.uniform(0.3, 2.0)), verify_seed=int(rng.integers(0, 2**40)),
                             block=block)
        if rng.random() < 0.5:
            b = W.VerifyBatch(_pad_rows(b.target, rng), _pad_rows(b.draft, rng), b.row_offsets, b.draft_tokens,
                              b.draft_row_start, b.temperature, b.seed, b.meta)
        temps = None
        if rng.random() < 0.4:
            temps = torch.from_numpy(rng.uniform(0.4, 1.8, size=R).astype(np.float32)).cuda()
        _, _, mism = H.check_sampling(b, want_probs=bool(rng.random() < 0.7), temperatures=temps)
        total_mism += mism
    assert total_mism <= 1


@pytest.mark.parametrize("seed", range(6))
def test_greedy_fuzz(seed):
    rng = np.random.default_rng(2000 + seed)
    for _ in range(8):
        R = int(rng.integers(1, 60))
        V = int(rng.choice([1, 2, 5, 33, 1000, 1025, 4096, 30001]))
        lengths = torch.from_numpy(rng.integers(0, 12, size=R))
        dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        b = W.greedy_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", sigma=float(rng.uniform(0.1, 5)),
                           tie_frac=float(rng.choice([0.0, 0.1, 0.9])) if V > 4 else 0.0,
                           perturb=float(rng.uniform(0, 0.6)), dtype=dtype)
        if rng.random() < 0.5:
            b = W.VerifyBatch(_pad_rows(b.target, rng), None, b.row_offsets, b.draft_tokens)
        H.check_greedy(b)


@pytest.mark.parametrize("seed", range(8))
def test_schedule_fuzz(seed):
    rng = np.random.default_rng(3000 + seed)
    for _ in range(6):
        R = int(rng.integers(1, 400))
        gamma = int(rng.choice([0, 1, 2, 3, 5, 8, 16, 31, 32, 33, 48]))
        if R * max(gamma, 1) > 20000:
            R = 20000 // max(gamma, 1)
        conf = rng.uniform(0.0, 1.0, size=(R, gamma)).astype(np.float32) ** float(rng.choice([0.2, 1.0, 3.0]))
        if gamma:
            conf[rng.random((R, gamma)) < 0.05] = 1.0
        n_bp = int(rng.integers(1, 9))
        hi = R * (gamma + 1) + 5
        toks = np.sort(rng.choice(np.arange(1, hi), size=min(n_bp, hi - 1), replace=False)).tolist()
        sps = rng.uniform(1, 100, len(toks)).tolist()
        budget = int(rng.integers(max(0, R - 3), hi + 10))
        s = W.ScheduleInput(torch.from_numpy(conf).reshape(R, gamma), toks, sps, budget, max_tokens=int(rng.integers(1, hi + 1)))
        mode = int(rng.choice([B.DSPARK_SCHED_EARLY_STOP, B.DSPARK_SCHED_GLOBAL, B.DSPARK_SCHED_TOPK]))
        dl = rng.integers(0, gamma + 2, size=R).astype(np.int32) if rng.random() < 0.3 else None
        H.check_schedule(s, mode, topk=int(rng.integers(0, R * gamma + 2)), draft_len=dl)
