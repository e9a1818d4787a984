"""GPU greedy verifier vs the CPU oracle: bit-exact token ids and accepted lengths."""
import numpy as np
import pytest
import torch

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_config_1_fixed_and_scheduled():
    sched, batch = W.config_1("cuda")
    H.check_greedy(batch)
    # the scheduled prefix rows: schedule on the GPU, then verify the first l*_r + 1 rows of each block
    g, _ = H.check_schedule(sched, B.DSPARK_SCHED_EARLY_STOP)
    lens = torch.from_numpy(g["lengths"]).cuda()
    rows = torch.cat([torch.arange(5 * r, 5 * r + int(lens[r]) + 1) for r in range(4)]).cuda()
    sub = W.VerifyBatch(batch.target[rows].contiguous(), None, torch.from_numpy(g["offsets"]).cuda(),
                        batch.draft_tokens[rows].contiguous())
    H.check_greedy(sub)


@pytest.mark.parametrize("R", [64, 1024])
def test_config_4(R):
    batch = W.config_4("cuda", R=R)               # R = 1024 is the full 2.65 GB configuration
    acc, out, o = H.check_greedy(batch)
    lens = batch.meta["lengths"].cpu().numpy()
    assert (acc <= lens).all() and (lens == 0).any()
    # ties were injected: the emitted argmax must be the lowest index among equal maxima
    t = batch.target
    rows_with_ties = ((t == t.max(dim=1, keepdim=True).values).sum(dim=1) > 1).nonzero().squeeze(1)
    assert rows_with_ties.numel() > 0
    am = o.row_argmax
    for i in rows_with_ties[:20].tolist():
        if am[i] >= 0:
            assert am[i] == int((t[i] == t[i].max()).nonzero()[0])


@pytest.mark.parametrize("V", [1, 7, 512, 1000, 4097, 129281])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_odd_vocabularies_and_dtypes(V, dtype):
    lengths = torch.tensor([0, 3, 1, 8, 2, 0, 5])
    batch = W.greedy_batch(lengths, V, 40 + V, "cuda", tie_frac=0.2 if V > 8 else 0.0, perturb=0.3, dtype=dtype)
    H.check_greedy(batch)
    B.dspark_set_stream_path(1)                  # same through the direct-load path
    try:
        H.check_greedy(batch)
    finally:
        B.dspark_set_stream_path(0)


def test_very_large_vocabulary_and_many_requests():
    H.check_greedy(W.greedy_batch(torch.tensor([1, 0, 2]), 1_000_003, 8, "cuda", tie_frac=0.5, perturb=0.3))
    # thousands of requests that verify only their bonus token
    H.check_greedy(W.greedy_batch(torch.zeros(5000, dtype=torch.int64), 4096, 9, "cuda", perturb=0.0))


def test_padded_rows_and_unaligned_views():
    lengths = torch.tensor([2, 4, 0, 1])
    base = W.greedy_batch(lengths, 3000, 5, "cuda", perturb=0.2)
    padded = torch.zeros(base.n_rows, 3072, device="cuda")
    padded[:, :3000] = base.target
    H.check_greedy(W.VerifyBatch(padded[:, :3000], None, base.row_offsets, base.draft_tokens))
    shifted = torch.zeros(base.n_rows, 3001, device="cuda")
    shifted[:, 1:] = base.target                       # rows start 4 bytes off a 16-byte boundary
    H.check_greedy(W.VerifyBatch(shifted[:, 1:], None, base.row_offsets, base.draft_tokens))


def test_special_values_and_device_errors():
    lengths = torch.tensor([1, 1, 1, 1, 0])
    b = W.greedy_batch(lengths, 5000, 9, "cuda", perturb=0.0)
    t = b.target
    t[0, 7] = float("nan"); t[1, :] = float("-inf"); t[2, 100] = float("inf")
    i4 = int(b.row_offsets[4])
    t[i4] = -1.0; t[i4, 4000] = 0.0; t[i4, 3000] = -0.0         # -0.0 ties +0.0: lowest index wins
    acc, out, o = H.check_greedy(b)
    assert out[i4] == 3000
    b.draft_tokens[0] = 5000                                     # token id out of range
    acc, out, _ = H.check_greedy(b)
    assert acc[0] == 0 and out[0] == -1
    # offsets that do not advance: flagged, other requests still verified
    off = b.row_offsets.clone(); off[2] = off[1]
    bad = W.VerifyBatch(b.target, None, off, b.draft_tokens)
    acc2, out2, st = H.gpu_verify_greedy(bad)
    assert st & B.DEV_BAD_OFFSETS and acc2[1] == 0
    assert acc2[3] == acc[3]


def test_capacity_larger_than_row_count():
    lengths = torch.tensor([2, 0, 3])
    b = W.greedy_batch(lengths, 2048, 3, "cuda", perturb=0.4)
    big = torch.zeros(b.n_rows + 5, 2048, device="cuda"); big[: b.n_rows] = b.target
    toks = torch.zeros(b.n_rows + 5, dtype=torch.int32, device="cuda"); toks[: b.n_rows] = b.draft_tokens
    acc, out, st = H.gpu_verify_greedy(W.VerifyBatch(big, None, b.row_offsets, toks))
    acc0, out0, _ = H.check_greedy(b)
    np.testing.assert_array_equal(acc, acc0)
    np.testing.assert_array_equal(out[: b.n_rows], out0[: b.n_rows])
    assert (out[b.n_rows:] == -7).all() and st == 0


def test_host_side_errors():
    b = W.greedy_batch(torch.tensor([1, 1]), 256, 1, "cuda")
    acc = torch.zeros(2, dtype=torch.int32, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DsparkError, match="workspace"):
        B.dspark_verify_greedy(b.target, b.row_offsets, b.draft_tokens, accepted_len=acc, out_tokens=out,
                               dev_status=None, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    with pytest.raises(B.DsparkError):
        B.dspark_verify_greedy(b.target.double(), b.row_offsets, b.draft_tokens, accepted_len=acc, out_tokens=out,
                               dev_status=None, workspace=B.workspace(1 << 20))
