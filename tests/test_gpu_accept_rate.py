"""GPU c* = 1 - TV(p, q) per draft position vs the oracle (absolute 1e-5, the probability bar)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu
TOL = 1e-5


def _gpu(batch, T):
    c = torch.full((batch.n_rows,), -7.0, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_accept_rate_workspace_bytes(batch.R, batch.n_rows, batch.V)).fill_(0xFF)
    B.dspark_accept_rate(batch.target, batch.draft, batch.row_offsets, T, draft_row_start=batch.draft_row_start,
                         out_cstar=c, dev_status=st, workspace=ws)
    torch.cuda.synchronize()
    return c.cpu().numpy().astype(np.float64), int(st.item())


def _check(batch, T):
    got, st = _gpu(batch, T)
    drs = None if batch.draft_row_start is None else batch.draft_row_start.cpu().numpy()
    want, ost = oracle.accept_rate(W.bf16_bits(batch.target), W.bf16_bits(batch.draft), batch.row_offsets.cpu().numpy(),
                                   T, draft_row_start=drs)
    assert st == int(np.bitwise_or.reduce(ost))
    np.testing.assert_array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.abs(got[ok] - want[ok]).max() <= TOL if ok.any() else True
    return got, want


@pytest.mark.parametrize("dtype,V,block", [(torch.bfloat16, W.V_FULL, None), (torch.bfloat16, W.V_FULL, 8),
                                           (torch.float32, 50_001, None), (torch.bfloat16, 1000, 8)])
def test_against_oracle(dtype, V, block):
    g = torch.Generator(device="cpu"); g.manual_seed(V)
    lengths = torch.randint(0, 8, (24,), generator=g)
    for T, noise in ((1.0, 1.0), (0.7, 2.0)):
        batch = W.sampling_batch(lengths, V, 31, "cuda", dtype=dtype, temperature=T, draft_noise=noise, block=block)
        got, want = _check(batch, T)
        ok = ~np.isnan(want)
        assert 0.0 < want[ok].min() and want[ok].max() < 1.0
        print(f"[c*] V={V} T={T}: mean c* = {want[ok].mean():.3f}, max |gpu - oracle| = {np.abs(got[ok] - want[ok]).max():.2e}")


def test_special_cases():
    lengths = torch.tensor([2, 0, 3, 1])
    b = W.sampling_batch(lengths, 4096, 3, "cuda", temperature=1.0)
    # identical distributions: c* = 1
    same = W.VerifyBatch(b.target, b.target[[0, 1, 4, 5, 6, 8]].contiguous(), b.row_offsets, b.draft_tokens, None, 1.0, 0, b.meta)
    got, _ = _check(same, 1.0)
    assert np.allclose(got[[0, 1, 4, 5, 6, 8]], 1.0, atol=2e-6)
    # a NaN row: that position is NaN and flagged, the others are unaffected
    t = b.target.clone(); t[4, 100] = float("nan")
    bad = W.VerifyBatch(t, b.draft, b.row_offsets, b.draft_tokens, None, 1.0, 0, b.meta)
    got_bad, _ = _check(bad, 1.0)
    got_ok, _ = _check(b, 1.0)
    assert np.isnan(got_bad[4]) and np.allclose(np.delete(got_bad, [2, 3, 4, 7, 9]), np.delete(got_ok, [2, 3, 4, 7, 9]), atol=0)
    # only bonus rows (no draft position at all)
    none = W.sampling_batch(torch.zeros(5, dtype=torch.int64), 2048, 1, "cuda")
    got, _ = _check(none, 1.0)
    assert np.isnan(got).all()
    # the accepted fraction of the sampling verifier follows c*: mean over many requests with one position
    n = 4000
    one = W.sampling_batch(torch.ones(n, dtype=torch.int64), 512, 9, "cuda", draft_noise=1.5, verify_seed=5)
    cs, _ = _check(one, 1.0)
    acc = torch.zeros(n, dtype=torch.int32, device="cuda"); out = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(n, 2 * n, 512))
    B.dspark_verify(one.target, one.draft, one.row_offsets, one.draft_tokens, 1.0, 5, accepted_len=acc, out_tokens=out,
                    dev_status=None, workspace=ws)
    mean_c = np.nanmean(cs)
    assert abs(acc.float().mean().item() - mean_c) < 4 * np.sqrt(0.25 / n)
