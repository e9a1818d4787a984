"""Shared plumbing for the GPU parity tests: run a batch through the C ABI and through
the CPU oracle, and compare under the stated bars."""
from __future__ import annotations

import os

import numpy as np
import torch

import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

P_REL_TOL = 1e-5        # p(x), q(x): relative agreement with the fp64 oracle
MARGIN_TOL = 1e-6       # a decision may differ only if the oracle's margin is below this
# A residual draw is a draw from max(0, p - q) / W.  Its margin is measured on that CDF (normalised), as for
# every other draw -- except where W itself is below what fp32 resolves: p(v) and q(v) are fp32 numbers with
# about 1e-7 relative error, so the running sum of max(0, p - q) carries an ABSOLUTE error of about 1e-7
# whatever W is, and for W < 1e-3 a normalised 1e-6 would ask for 1e-9 absolute.  There (and only there) the
# margin is taken in probability units.
SMALL_RESIDUAL_MASS = 1e-3
MISMATCH_COUNTS = {"accept": 0, "token_normalised": 0, "token_small_mass": 0}   # running totals, printed by the config tests


def token_mismatch_allowed(o, r):
    """Which rule (if any) allows the emitted token of request r to differ from the oracle's."""
    if o.token_margin[r] < MARGIN_TOL:
        return "token_normalised"
    w = o.resid_mass[r]
    if w == w and w < SMALL_RESIDUAL_MASS and o.token_margin_abs[r] < MARGIN_TOL:
        return "token_small_mass"
    return None
THREADS = max(1, min(32, os.cpu_count() or 1))


def gpu_schedule(sched: W.ScheduleInput, mode: int, topk: int = 0, draft_len=None, want_all=True):
    conf = sched.conf.cuda().contiguous()
    R, gamma = conf.shape
    prof = B.Profile(sched.bp_tokens, sched.bp_sps, sched.max_tokens)
    out_len = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    off = torch.full((R + 1,), -7, dtype=torch.int32, device="cuda")
    surv = torch.full((R, gamma), -1.0, dtype=torch.float32, device="cuda") if want_all else None
    exp = torch.full((R,), -1.0, dtype=torch.float32, device="cuda") if want_all else None
    info = torch.zeros(32, dtype=torch.uint8, device="cuda")
    ws = B.workspace(B.dspark_schedule_workspace_bytes(R, gamma)).fill_(0xFF)     # results must not depend on its content
    dl = None if draft_len is None else torch.as_tensor(draft_len, dtype=torch.int32).cuda()
    B.dspark_schedule(prof, conf, sched.budget_tokens, mode, topk, dl, out_len=out_len, out_row_offsets=off,
                      out_survival=surv, out_expected_len=exp, out_info=info, workspace=ws)
    torch.cuda.synchronize()
    table = prof.table().numpy()
    prof.close()
    return dict(lengths=out_len.cpu().numpy(), offsets=off.cpu().numpy(),
                survival=None if surv is None else surv.cpu().numpy(),
                expected=None if exp is None else exp.cpu().numpy(),
                info=B.read_sched_info(info), table=table)


def check_schedule(sched: W.ScheduleInput, mode: int, topk: int = 0, draft_len=None):
    g = gpu_schedule(sched, mode, topk, draft_len)
    tab = oracle.sps_table(sched.bp_tokens, sched.bp_sps, sched.max_tokens)
    np.testing.assert_array_equal(g["table"], tab)                       # bit-exact fp64 table
    o = oracle.schedule(sched.conf.cpu().numpy(), tab, sched.budget_tokens, mode, topk, draft_len)
    np.testing.assert_array_equal(g["lengths"], o.lengths)               # bit-exact lengths
    np.testing.assert_array_equal(g["survival"], o.survival)             # fp32 products, same order
    np.testing.assert_array_equal(g["expected"], o.expected_len)
    want_off = np.concatenate([[0], np.cumsum(o.lengths + 1)]).astype(np.int32)
    np.testing.assert_array_equal(g["offsets"], want_off)
    i = g["info"]
    assert (i.B, i.n_admitted, i.n_candidates, i.status) == (o.B, o.n_admitted, o.n_candidates, o.status)
    assert i.tau == o.tau and i.theta == o.theta
    return g, o


def gpu_verify_greedy(batch: W.VerifyBatch, n_rows_cap=None):
    R = batch.R
    cap = batch.n_rows if n_rows_cap is None else n_rows_cap
    acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, cap, batch.V)).fill_(0xFF)
    B.dspark_verify_greedy(batch.target, batch.row_offsets, batch.draft_tokens, accepted_len=acc,
                           out_tokens=out, dev_status=st, workspace=ws, n_rows=cap)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), out.cpu().numpy(), int(st.item())


def check_greedy(batch: W.VerifyBatch, expect_status=None):
    acc, out, st = gpu_verify_greedy(batch)
    o = oracle.verify_greedy(W.bf16_bits(batch.target), batch.row_offsets.cpu().numpy(),
                             batch.draft_tokens.cpu().numpy())
    np.testing.assert_array_equal(acc, o.accepted_len)
    np.testing.assert_array_equal(out[: batch.n_rows], o.out_tokens)
    want_st = int(np.bitwise_or.reduce(o.status)) if expect_status is None else expect_status
    assert st == want_st
    return acc, out, o


def gpu_verify(batch: W.VerifyBatch, want_probs=True, n_rows_cap=None, temperatures=None):
    R = batch.R
    cap = batch.n_rows if n_rows_cap is None else n_rows_cap
    acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
    p = torch.full((cap,), float("nan"), dtype=torch.float32, device="cuda") if want_probs else None
    q = torch.full((cap,), float("nan"), dtype=torch.float32, device="cuda") if want_probs else None
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, cap, batch.V)).fill_(0xFF)     # poisoned: NaN patterns everywhere
    if temperatures is None:
        B.dspark_verify(batch.target, batch.draft, batch.row_offsets, batch.draft_tokens, batch.temperature,
                        batch.seed, draft_row_start=batch.draft_row_start, accepted_len=acc, out_tokens=out,
                        out_p_tok=p, out_q_tok=q, dev_status=st, workspace=ws, n_rows=cap)
    else:
        B.dspark_verify_per_request(batch.target, batch.draft, batch.row_offsets, batch.draft_tokens,
                                    temperatures, batch.seed, draft_row_start=batch.draft_row_start,
                                    accepted_len=acc, out_tokens=out, out_p_tok=p, out_q_tok=q, dev_status=st,
                                    workspace=ws, n_rows=cap)
    torch.cuda.synchronize()
    return dict(acc=acc.cpu().numpy(), out=out.cpu().numpy(), status=int(st.item()),
                p=None if p is None else p.cpu().numpy(), q=None if q is None else q.cpu().numpy())


def oracle_verify(batch: W.VerifyBatch, eval_all=True, temperatures=None):
    drs = None if batch.draft_row_start is None else batch.draft_row_start.cpu().numpy()
    return oracle.verify(W.bf16_bits(batch.target), W.bf16_bits(batch.draft), batch.row_offsets.cpu().numpy(),
                         batch.draft_tokens.cpu().numpy(), batch.temperature, batch.seed,
                         draft_row_start=drs, eval_all=eval_all, n_threads=THREADS,
                         temperatures=None if temperatures is None else temperatures.cpu().numpy())


def compare_sampling(g: dict, o, row_offsets: np.ndarray, check_probs=True):
    """Bit-exact accepted lengths and tokens, except where the oracle's own margin says the
    decision sat within MARGIN_TOL of a boundary.  Returns the number of such mismatches."""
    R = len(row_offsets) - 1
    n_rows = int(row_offsets[-1])
    assert g["status"] == int(np.bitwise_or.reduce(o.status))
    mismatches = 0
    for r in range(R):
        lo, hi = int(row_offsets[r]), int(row_offsets[r + 1])
        if o.status[r]:
            assert g["acc"][r] == 0 and (g["out"][lo:hi] == -1).all()
            continue
        ng, no = int(g["acc"][r]), int(o.accepted_len[r])
        if ng != no:
            j = min(ng, no)
            assert o.accept_margin[lo + j] < MARGIN_TOL, (r, j, ng, no, o.accept_margin[lo + j])
            mismatches += 1
            MISMATCH_COUNTS["accept"] += 1
            continue
        if not (g["out"][lo:hi] == o.out_tokens[lo:hi]).all():
            assert (g["out"][lo:lo + no] == o.out_tokens[lo:lo + no]).all()
            assert (g["out"][lo + no + 1:hi] == -1).all()
            rule = token_mismatch_allowed(o, r)
            assert rule is not None, (r, no, g["out"][lo + no], o.out_tokens[lo + no], o.token_margin[r],
                                      o.token_margin_abs[r], o.resid_mass[r])
            MISMATCH_COUNTS[rule] += 1
            mismatches += 1
    if check_probs and g["p"] is not None:
        have = ~np.isnan(o.p_tok[:n_rows])
        gp, gq = g["p"][:n_rows][have].astype(np.float64), g["q"][:n_rows][have].astype(np.float64)
        op, oq = o.p_tok[:n_rows][have], o.q_tok[:n_rows][have]
        # relative agreement; probabilities below fp32's normal range are compared absolutely
        np.testing.assert_allclose(gp, op, rtol=P_REL_TOL, atol=1e-37)
        np.testing.assert_allclose(gq, oq, rtol=P_REL_TOL, atol=1e-37)
    return mismatches


def check_sampling(batch: W.VerifyBatch, want_probs=True, temperatures=None):
    g = gpu_verify(batch, want_probs, temperatures=temperatures)
    o = oracle_verify(batch, eval_all=want_probs, temperatures=temperatures)
    mism = compare_sampling(g, o, batch.row_offsets.cpu().numpy(), check_probs=want_probs)
    return g, o, mism


def compare_away_from_top_p_boundaries(g, o, margin, off):
    """Requests with a row whose top-p decision sits on its boundary (margin < 1e-5 of Z) may see a neighbouring cut;
    all others must agree with the oracle under the usual margin rule.  Returns (skipped, boundary mismatches)."""
    R = len(off) - 1
    near_req = {r for r in range(R) if (margin[off[r]:off[r + 1]] < 1e-5).any()}
    mism = 0
    for r in range(R):
        if r in near_req:
            continue
        lo, hi = int(off[r]), int(off[r + 1])
        ng, no = int(g["acc"][r]), int(o.accepted_len[r])
        if ng != no:
            assert o.accept_margin[lo + min(ng, no)] < MARGIN_TOL, (r, ng, no)
            mism += 1
            continue
        if not (g["out"][lo:hi] == o.out_tokens[lo:hi]).all():
            assert (g["out"][lo:lo + no] == o.out_tokens[lo:lo + no]).all()
            assert token_mismatch_allowed(o, r), (r, g["out"][lo + no], o.out_tokens[lo + no], o.token_margin[r])
            mism += 1
    return len(near_req), mism
