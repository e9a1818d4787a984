"""The pieces chained the way a serving step uses them (Sections 3.1 - 3.2, 2.1): a block of Markov-head draft
positions (each position's previous token is the one just drawn), the confidences of the head calibrated by
Sequential Temperature Scaling, the scheduler's verification lengths, and the lossless verifier reading the
drafter's logits in place through `draft_row_start` -- every step on the GPU, device-resident between the
calls, and every step checked against the oracle on the same tensors."""
import numpy as np
import pytest
import torch

import helpers as H
import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _draft_block(R, V, gamma, seed, T):
    """gamma sequential draft positions; logits land in the block layout [R * gamma, V] (row r * gamma + k)."""
    m = W.markov_input(R, V, seed, "cuda", d=64)
    g = torch.Generator(device="cuda").manual_seed(seed + 1)
    U = (torch.randn(gamma, R, V, generator=g, device="cuda") * 3).to(torch.bfloat16)
    Hs = torch.randn(gamma, R, 64, generator=g, device="cuda").to(torch.bfloat16)
    packed = torch.empty(B.dspark_markov_w2_packed_bytes(V), dtype=torch.uint8, device="cuda")
    B.dspark_markov_pack_w2(m.W2, packed)
    draft = torch.zeros(R * gamma, V, dtype=torch.bfloat16, device="cuda")
    toks = torch.zeros(gamma, R, dtype=torch.int32, device="cuda")
    conf = torch.zeros(gamma, R, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_markov_workspace_bytes(R, V))
    x_prev = m.x_prev                                   # anchor tokens
    for k in range(gamma):
        out_k = draft.view(R, gamma, V)[:, k, :]        # rows r * gamma + k, row stride gamma * V
        B.dspark_markov_draft_step(U[k], m.W1, packed, x_prev, T, 1000 + k, H=Hs[k], w_conf=m.w_conf,
                                   out_logits=out_k, out_tokens=toks[k], out_conf=conf[k], dev_status=st, workspace=ws)
        x_prev = toks[k]
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return m, U, Hs, draft, toks, conf


def test_draft_block_schedule_verify():
    R, V, gamma, T = 48, 8192, 6, 1.0
    m, U, Hs, draft, toks, conf = _draft_block(R, V, gamma, 5, T)
    # each position against the oracle: logits from the previous position's token, draw from the stored logits
    x_prev = m.x_prev.cpu().numpy()
    for k in range(gamma):
        exact, bits = oracle.markov_logits(W.bf16_bits(U[k]), W.bf16_bits(m.W1), W.bf16_bits(m.W2), x_prev)
        got = W.bf16_bits(draft.view(R, gamma, V)[:, k, :].contiguous())
        assert float((got != bits).mean()) < 2e-3
        o = oracle.verify(got, got, np.arange(R + 1, dtype=np.int32), np.zeros(R, np.int32), T, 1000 + k)
        tk = toks[k].cpu().numpy()
        for r in np.nonzero(tk != o.out_tokens[:R])[0]:
            assert o.token_margin[r] < 1e-6
        want_c = oracle.confidence(W.bf16_bits(Hs[k]), W.bf16_bits(m.W1), m.w_conf.cpu().numpy(), x_prev)
        assert np.abs(conf[k].cpu().numpy() - want_c).max() < 1e-6
        x_prev = tk                                      # the chain continues from the GPU's own tokens

    # confidences [R, gamma] -> calibration temperatures from (synthetic) held-out blocks -> calibrated confidences
    conf_rg = conf.t().contiguous()
    held, acc_h, ver_h = W.sts_input(20_000, gamma, 9, "cuda", overconfidence=1.5)
    grid = torch.tensor(np.geomspace(0.5, 3.0, 21), dtype=torch.float32, device="cuda")
    Tk = torch.empty(gamma, device="cuda")
    B.dspark_sts_calibrate(held, acc_h, grid, 15, verified_len=ver_h, out_T=Tk,
                           workspace=B.workspace(B.dspark_sts_workspace_bytes(20_000, gamma, 21, 15)))
    cal = torch.empty_like(conf_rg)
    B.dspark_sts_apply(conf_rg, Tk, cal)
    torch.cuda.synchronize()
    np.testing.assert_allclose(cal.cpu().numpy(), oracle.sts_apply(conf_rg.cpu().numpy(), Tk.cpu().numpy()), atol=2e-6)

    # scheduler on the calibrated confidences; its offsets stay on the device for the verifier
    sched = W.ScheduleInput(cal, *W.PROFILE_P3, budget_tokens=160, max_tokens=1024)
    prof = B.Profile(sched.bp_tokens, sched.bp_sps, sched.max_tokens)
    out_len = torch.empty(R, dtype=torch.int32, device="cuda")
    offsets = torch.empty(R + 1, dtype=torch.int32, device="cuda")
    B.dspark_schedule(prof, cal, sched.budget_tokens, B.DSPARK_SCHED_EARLY_STOP, out_len=out_len, out_row_offsets=offsets,
                      workspace=B.workspace(B.dspark_schedule_workspace_bytes(R, gamma)))
    torch.cuda.synchronize()
    tab = prof.table().numpy()
    o_s = oracle.schedule(cal.cpu().numpy(), tab, sched.budget_tokens, oracle.MODE_EARLY_STOP)
    np.testing.assert_array_equal(out_len.cpu().numpy(), o_s.lengths)
    lengths = out_len.cpu().numpy()
    assert 0 < lengths.sum() <= sched.budget_tokens - R and lengths.max() <= gamma
    off = offsets.cpu().numpy()
    n_rows = int(off[-1])

    # target rows for the scheduled prefixes (+ bonus rows): the drafter's rows plus noise; draft tokens in the
    # flat layout; the verifier reads the draft logits in place (row r * gamma + j)
    g = torch.Generator(device="cuda").manual_seed(77)
    target = torch.empty(n_rows, V, dtype=torch.bfloat16, device="cuda")
    flat_tok = torch.zeros(n_rows, dtype=torch.int32, device="cuda")
    for r in range(R):
        for j in range(lengths[r] + 1):
            src = draft[r * gamma + min(j, gamma - 1)].float()
            target[off[r] + j] = (src + 0.7 * torch.randn(V, generator=g, device="cuda")).to(torch.bfloat16)
            if j < lengths[r]:
                flat_tok[off[r] + j] = toks[j, r]
    drs = (torch.arange(R, dtype=torch.int64, device="cuda") * gamma)
    batch = W.VerifyBatch(target, draft, offsets, flat_tok, drs, T, 4242)
    gv, ov, mism = H.check_sampling(batch)
    assert (gv["acc"] <= lengths).all()
    print(f"[pipeline] lengths {lengths.tolist()} accepted {gv['acc'].tolist()} ({mism} boundary mismatches)")

    # a target that IS the draft distribution accepts every scheduled token (p = q: u q < p for every u < 1)
    same = target.clone()
    for r in range(R):
        for j in range(lengths[r]):
            same[off[r] + j] = draft[r * gamma + j]
    g2 = H.gpu_verify(W.VerifyBatch(same, draft, offsets, flat_tok, drs, T, 4242))
    np.testing.assert_array_equal(g2["acc"], lengths)
