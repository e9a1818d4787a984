"""Batches whose logits reach beyond 4 GiB from the base pointer (and beyond 2^31 elements): every
row address has to be formed in 64 bits.  The strided cases compare against the same batch stored
densely, which the other tests check against the oracle; the dense greedy case goes to the oracle."""
import numpy as np
import pytest
import torch

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_greedy_on_more_than_4_gib_of_dense_rows():
    V = W.V_FULL
    g = torch.Generator().manual_seed(5)
    lengths = torch.randint(0, 9, (3400,), generator=g)            # about 17 000 rows of 258 560 B
    batch = W.greedy_batch(lengths, V, 77, "cuda", tie_frac=0.05, perturb=0.3)
    assert batch.n_rows * V > 2 ** 31 and batch.target.is_contiguous()
    acc, out, o = H.check_greedy(batch)
    assert (acc < lengths.numpy()).any() and (acc == lengths.numpy()).any()


@pytest.mark.parametrize("path", [0, 1])
def test_sampling_with_a_row_pitch_that_puts_rows_beyond_4_gib(path):
    V = W.V_FULL
    lengths = torch.tensor([3, 0, 8, 1, 5, 2, 8, 4] * 12)          # 96 requests, 468 target and 372 draft rows
    b = W.sampling_batch(lengths, V, 31, "cuda", verify_seed=17)
    pitch = 48 * V                                                 # elements; row 346 starts beyond 4 GiB
    tp = torch.zeros(b.n_rows, pitch, dtype=torch.bfloat16, device="cuda")
    dp = torch.zeros(b.draft.shape[0], pitch, dtype=torch.bfloat16, device="cuda")
    tp[:, :V] = b.target
    dp[:, :V] = b.draft
    assert (b.n_rows - 1) * pitch * 2 > 2 ** 32 and (b.draft.shape[0] - 1) * pitch > 2 ** 31
    wide = W.VerifyBatch(tp[:, :V], dp[:, :V], b.row_offsets, b.draft_tokens, None, b.temperature, b.seed, b.meta)
    g0, _, mism = H.check_sampling(b)
    B.dspark_set_stream_path(path)
    try:
        g1 = H.gpu_verify(wide)
    finally:
        B.dspark_set_stream_path(0)
    assert g1["status"] == g0["status"] == 0
    np.testing.assert_array_equal(g0["acc"], g1["acc"])
    np.testing.assert_array_equal(g0["out"], g1["out"])
    np.testing.assert_array_equal(g0["p"], g1["p"])
    np.testing.assert_array_equal(g0["q"], g1["q"])
    assert (g0["acc"] < lengths.numpy()).sum() > 10               # the residual pass ran on far rows too


def test_truncated_verification_and_in_place_truncation_with_a_far_row_pitch():
    import test_gpu_verify_truncated as TV

    V = W.V_FULL
    lengths = torch.tensor([3, 0, 8, 1, 5, 2, 8, 4] * 12)
    b = W.sampling_batch(lengths, V, 32, "cuda", verify_seed=18)
    pitch = 48 * V
    tp = torch.zeros(b.n_rows, pitch, dtype=torch.bfloat16, device="cuda")
    dp = torch.zeros(b.draft.shape[0], pitch, dtype=torch.bfloat16, device="cuda")
    tp[:, :V] = b.target
    dp[:, :V] = b.draft
    wide = W.VerifyBatch(tp[:, :V], dp[:, :V], b.row_offsets, b.draft_tokens, None, b.temperature, b.seed, b.meta)
    rng = np.random.default_rng(3)
    ks = rng.choice([0, 1, 20, 50, 400], b.R).astype(np.int32)
    ps = rng.choice([0.0, 0.5, 0.9, 0.95], b.R).astype(np.float32)
    g0 = TV._gpu_truncated(b, ks, ps, None)
    g1 = TV._gpu_truncated(wide, ks, ps, None)
    assert g0["status"] == g1["status"] == 0
    for key in ("acc", "out", "p", "q"):
        np.testing.assert_array_equal(g0[key], g1[key])
    # in place on the wide rows: same masks as on the dense rows, the padding between rows untouched
    dev = lambda a, dt: torch.as_tensor(a, dtype=dt, device="cuda")
    dense = b.target.clone()
    B.dspark_truncate_target(dense, b.row_offsets, top_k=dev(ks, torch.int32), top_p=dev(ps, torch.float32), temperature=b.temperature)
    B.dspark_truncate_target(tp[:, :V], b.row_offsets, top_k=dev(ks, torch.int32), top_p=dev(ps, torch.float32), temperature=b.temperature)
    torch.cuda.synchronize()
    assert torch.equal(dense.view(torch.int16), tp[:, :V].view(torch.int16))
    assert torch.isneginf(dense).any()
    assert int(torch.count_nonzero(tp[:, V:2 * V])) == 0 and int(torch.count_nonzero(tp[-1, V:])) == 0
