"""The per-kernel timers of the library (dspark_ktimer_*), which bench.py's roofline figures rest on: what they record
for a call, that they record nothing when detached or full, and that their sum fits inside the time of the calls."""
import numpy as np
import pytest
import torch

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _sampling_call(b, ws, acc, out, st):
    B.dspark_verify(b.target, b.draft, b.row_offsets, b.draft_tokens, b.temperature, b.seed,
                    accepted_len=acc, out_tokens=out, dev_status=st, workspace=ws)


def test_what_the_timers_record_for_the_verifiers():
    lengths = torch.tensor([3, 0, 2, 5, 1, 4, 0, 2])
    V = 40_000
    b = W.sampling_batch(lengths, V, 12, "cuda", temperature=0.9, verify_seed=4)
    gb = W.greedy_batch(lengths, V, 13, "cuda", dtype=torch.bfloat16, perturb=0.3)
    R = b.R
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, b.n_rows, V))
    acc = torch.zeros(R, dtype=torch.int32, device="cuda")
    out = torch.zeros(b.n_rows, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    _sampling_call(b, ws, acc, out, st)                    # warm-up, not recorded
    torch.cuda.synchronize()

    n_calls = 3
    timer = B.KernelTimer(64)
    try:
        timer.attach()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(n_calls):
            _sampling_call(b, ws, acc, out, st)
        t1.record()
        timer.detach()
        _sampling_call(b, ws, acc, out, st)                # detached: leaves no record
        torch.cuda.synchronize()
        got = timer.read()
        assert set(got) == {"stream_stats", "decide", "residual_stream", "finalize"}, got
        for name, rec in got.items():
            assert rec["launches"] == n_calls and rec["ms"] > 0.0, (name, rec)
        # the timed kernels ran inside the bracket of the three calls
        assert sum(rec["ms"] for rec in got.values()) <= t0.elapsed_time(t1) * 1.05

        # the greedy verifier, recorded after a reset
        timer.attach()
        B.dspark_verify_greedy(gb.target, gb.row_offsets, gb.draft_tokens, accepted_len=acc, out_tokens=out,
                               dev_status=st, workspace=ws)
        timer.detach()
        torch.cuda.synchronize()
        got = timer.read()
        assert set(got) == {"greedy_stream", "greedy_decide"}, got
        assert all(rec["launches"] == 1 for rec in got.values())
    finally:
        timer.close()

    # a timer that is full records no further launch and disturbs nothing
    small = B.KernelTimer(2)
    try:
        small.attach()
        _sampling_call(b, ws, acc, out, st)
        small.detach()
        torch.cuda.synchronize()
        got = small.read()
        assert sum(rec["launches"] for rec in got.values()) == 2
        assert int(st.item()) == 0
        o = H.oracle_verify(b, eval_all=False)
        g = dict(acc=acc.cpu().numpy(), out=out.cpu().numpy(), status=0, p=None, q=None)
        assert H.compare_sampling(g, o, b.row_offsets.cpu().numpy(), check_probs=False) == 0
    finally:
        small.close()
    with pytest.raises(B.DsparkError):
        B.KernelTimer(0)
