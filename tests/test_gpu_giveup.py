"""The give-up path of the streamed passes, reached without hanging anything: with the diagnostic poll limit set
to "no poll at all" every entry wait of the bulk-copy pipeline (a consumer waiting for data, the producer
waiting for a free stage) runs out at once, the kernels set DSPARK_DEV_TIMEOUT and leave after the copies they
had issued have landed, and the device, the stream and the workspace stay usable: the next call with the normal
limit gives the oracle's answer."""
import numpy as np
import pytest
import torch

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run(batch, ws, greedy):
    acc = torch.full((batch.R,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((batch.n_rows,), -7, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    if greedy:
        B.dspark_verify_greedy(batch.target, batch.row_offsets, batch.draft_tokens, accepted_len=acc, out_tokens=out,
                               dev_status=st, workspace=ws)
    else:
        B.dspark_verify(batch.target, batch.draft, batch.row_offsets, batch.draft_tokens, batch.temperature, batch.seed,
                        accepted_len=acc, out_tokens=out, dev_status=st, workspace=ws)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), out.cpu().numpy(), int(st.item())


@pytest.mark.parametrize("greedy", [False, True])
def test_entry_waits_that_run_out_set_the_status_and_leave_the_workspace_usable(greedy):
    lengths = torch.tensor([3, 0, 2, 4])
    V = 4096
    batch = (W.greedy_batch(lengths, V, 5, "cuda", dtype=torch.bfloat16, perturb=0.3) if greedy
             else W.sampling_batch(lengths, V, 5, "cuda", temperature=0.9, verify_seed=3))
    ws = B.workspace(B.dspark_verify_workspace_bytes(batch.R, batch.n_rows, V))
    B.dspark_set_wait_poll_limit(1)
    try:
        _, _, status = _run(batch, ws, greedy)
    finally:
        B.dspark_set_wait_poll_limit(0)
    assert status & B.DEV_TIMEOUT                       # outputs of that call are unspecified
    # the same workspace, the normal limit: the oracle's answer
    if greedy:
        acc, out, status = _run(batch, ws, True)
        import oracle
        o = oracle.verify_greedy(W.bf16_bits(batch.target), batch.row_offsets.cpu().numpy(), batch.draft_tokens.cpu().numpy())
        np.testing.assert_array_equal(acc, o.accepted_len)
        np.testing.assert_array_equal(out, o.out_tokens)
        assert status == 0
    else:
        acc, out, status = _run(batch, ws, False)
        o = H.oracle_verify(batch, eval_all=False)
        g = dict(acc=acc, out=out, status=status, p=None, q=None)
        assert H.compare_sampling(g, o, batch.row_offsets.cpu().numpy(), check_probs=False) == 0


def test_the_histogram_pass_of_the_truncated_verifier_gives_up_the_same_way():
    # the streamed threshold search adds one more kind of wait (the consumer warps of a unit wait for one another's
    # counts before they move them to the row); it is bounded like the others
    import oracle
    lengths = torch.tensor([2, 0, 3, 1])
    V = 4096
    batch = W.sampling_batch(lengths, V, 6, "cuda", temperature=0.9, verify_seed=4)
    R = batch.R
    ks = torch.tensor([5, 0, 40, 0], dtype=torch.int32, device="cuda")
    ps = torch.tensor([1.0, 0.9, 0.8, 0.97], dtype=torch.float32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, batch.n_rows, V))

    def run():
        acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
        out = torch.full((batch.n_rows,), -7, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.dspark_verify_truncated(batch.target, batch.draft, batch.row_offsets, batch.draft_tokens, batch.seed,
                                  temperature=batch.temperature, temperatures=None, top_k=ks, top_p=ps,
                                  draft_row_start=batch.draft_row_start, accepted_len=acc, out_tokens=out,
                                  out_p_tok=None, out_q_tok=None, dev_status=st, workspace=ws)
        torch.cuda.synchronize()
        return dict(acc=acc.cpu().numpy(), out=out.cpu().numpy()), int(st.item())

    B.dspark_set_wait_poll_limit(1)
    try:
        _, status = run()
    finally:
        B.dspark_set_wait_poll_limit(0)
    assert status & B.DEV_TIMEOUT
    g, status = run()
    assert status == 0
    off = batch.row_offsets.cpu().numpy()
    masked, tau, kept, margin = oracle.warp_target(W.bf16_bits(batch.target), off, top_k=ks.cpu().numpy(),
                                                   top_p=ps.cpu().numpy(), temperature=batch.temperature)
    o = oracle.verify(masked, W.bf16_bits(batch.draft), off, batch.draft_tokens.cpu().numpy(), batch.temperature,
                      batch.seed, eval_all=False, n_threads=H.THREADS)
    skipped, mism = H.compare_away_from_top_p_boundaries(g, o, margin, off)
    assert skipped == 0 and mism == 0
