"""The allocation-free greedy entry point.

Some callers cannot hand the library a workspace because they cannot allocate one: an engine in
its steady-state loop has given all of HBM away already, and a cudaMalloc would stall the device
in the middle of a step.  For them `dspark_verify_greedy_static` keeps its scratch in a fixed array
inside the library.  This file checks, through the C ABI, that it returns exactly what
`dspark_verify_greedy` returns -- twice in a row on different batches, so that whatever the
first call left in the shared array is shown not to leak into the second -- and that a batch too
large for the array is refused.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run_workspace(batch):
    R = batch.R
    acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((batch.n_rows,), -7, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, batch.n_rows, batch.V))
    B.dspark_verify_greedy(batch.target, batch.row_offsets, batch.draft_tokens, accepted_len=acc, out_tokens=out,
                           dev_status=st, workspace=ws)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), out.cpu().numpy(), int(st.item())


def _run_static(batch):
    R = batch.R
    acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((batch.n_rows,), -7, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.dspark_verify_greedy_static(batch.target, batch.row_offsets, batch.draft_tokens, accepted_len=acc,
                                  out_tokens=out, dev_status=st)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), out.cpu().numpy(), int(st.item())


def test_static_entry_point_matches_workspace_entry_point_twice_in_a_row():
    # first a larger fp32 batch, then a smaller bf16 one with other data: the second call runs over
    # the leftovers of the first
    first = W.greedy_batch(torch.randint(0, 9, (96,)), 50_000, 77, "cuda", tie_frac=0.05, perturb=0.25)
    second = W.greedy_batch(torch.randint(0, 5, (40,)), 20_011, 78, "cuda", tie_frac=0.05, perturb=0.4,
                            dtype=torch.bfloat16)
    for batch in (first, second):
        want = _run_workspace(batch)
        got = _run_static(batch)
        np.testing.assert_array_equal(got[0], want[0])       # accepted lengths, bit-exact
        np.testing.assert_array_equal(got[1], want[1])       # token ids, bit-exact
        assert got[2] == want[2] == 0
    # and once more on the first batch: same answer as before
    np.testing.assert_array_equal(_run_static(first)[1], _run_workspace(first)[1])


def test_static_entry_point_takes_batches_the_sampling_workspace_would_not_fit():
    # the array has to hold only what greedy verification uses (header + 8 bytes per 4 KB block of a row), not the
    # sampling verifier's workspace: 3 000 rows at V = 20 000 need 0.5 MB of it, while a sampling workspace for
    # the same shape is larger than the whole array
    cap = B.dspark_verify_greedy_static_capacity()
    lengths = torch.randint(0, 6, (1000,))
    batch = W.greedy_batch(lengths, 20_000, 79, "cuda", tie_frac=0.05, perturb=0.3)
    assert batch.n_rows >= 3000
    assert B.dspark_verify_workspace_bytes(batch.R, batch.n_rows, batch.V) > cap
    assert B.dspark_verify_greedy_static_bytes(batch.R, batch.n_rows, batch.V, torch.float32) < cap // 8
    want, got = _run_workspace(batch), _run_static(batch)
    np.testing.assert_array_equal(got[0], want[0])
    np.testing.assert_array_equal(got[1], want[1])
    assert got[2] == want[2] == 0


def test_static_entry_point_capacity_is_what_the_header_says():
    # "about 8 000 fp32 rows or 16 000 bf16 rows at V = 129 280"
    cap = B.dspark_verify_greedy_static_capacity()
    V = 129_280
    assert B.dspark_verify_greedy_static_bytes(1000, 8000, V, torch.float32) <= cap
    assert B.dspark_verify_greedy_static_bytes(1000, 16000, V, torch.bfloat16) <= cap
    # the last batch that fits runs and agrees with the workspace entry point; one more row is refused
    lo, hi = 1, 20_000                                        # largest row count that fits, by bisection
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if B.dspark_verify_greedy_static_bytes(8, mid, V, torch.float32) <= cap:
            lo = mid
        else:
            hi = mid
    rows = lo
    assert 8000 <= rows < 8500
    assert B.dspark_verify_greedy_static_bytes(8, rows, V, torch.float32) <= cap < B.dspark_verify_greedy_static_bytes(8, rows + 1, V, torch.float32)
    R = rows // 8
    lengths = torch.full((R,), 7)
    lengths[: rows - 8 * R] += 1                              # exactly `rows` target rows
    batch = W.greedy_batch(lengths, V, 80, "cuda", tie_frac=0.01, perturb=0.2)
    assert batch.n_rows == rows
    want, got = _run_workspace(batch), _run_static(batch)
    np.testing.assert_array_equal(got[0], want[0])
    np.testing.assert_array_equal(got[1], want[1])
    acc = torch.zeros(R, dtype=torch.int32, device="cuda")
    out = torch.zeros(rows + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DsparkError, match="built-in scratch"):
        B.dspark_verify_greedy_static(batch.target, batch.row_offsets, batch.draft_tokens, accepted_len=acc,
                                      out_tokens=out, dev_status=None, n_rows=rows + 1)
    del batch
    torch.cuda.empty_cache()


def test_static_entry_point_refuses_batches_beyond_its_array():
    cap = B.dspark_verify_greedy_static_capacity()
    assert cap == 8 << 20
    R, V = 4, 129_280
    n_rows = 20_000
    assert B.dspark_verify_greedy_static_bytes(R, n_rows, V, torch.float32) > cap
    # only the sizes matter for the refusal: nothing is launched, the small tensors are never read
    dummy = torch.zeros(8, V, device="cuda")
    off = torch.tensor([0, 2, 4, 6, 8], dtype=torch.int32, device="cuda")
    toks = torch.zeros(n_rows, dtype=torch.int32, device="cuda")
    acc = torch.zeros(R, dtype=torch.int32, device="cuda")
    out = torch.zeros(n_rows, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DsparkError, match="built-in scratch"):
        B.dspark_verify_greedy_static(dummy, off, toks, accepted_len=acc, out_tokens=out, dev_status=None,
                                      n_rows=n_rows)
