"""The drafter hands the verifier the softmax statistics of the rows it wrote (dspark_verify_draft_stats).

The accept test needs of a draft row only q(x) = 2^(x s - c) / Z at the draft token, so a drafter that kept (c, Z)
saves the verifier the pass over the draft rows.  Checked here: dspark_row_stats gives the pairs the verifier itself
would compute; the verifier fed with them agrees with the plain verifier and, under the margin rule, with the oracle
(which knows nothing of the shortcut: it computes q from the draft logits); the Markov draft step's own pairs equal
dspark_row_stats of the logits it stored; unusable rows and wrong statistics behave as documented.
"""
import numpy as np
import pytest
import torch

import helpers as H
import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _stats(logits, T=1.0, row_T=None):
    out = torch.full((logits.shape[0], 2), 7.0, device="cuda")
    B.dspark_row_stats(logits, T, row_temperatures=row_T, out_row_stats=out)
    torch.cuda.synchronize()
    return out


def _verify_with_stats(b, stats, temperatures=None, want_probs=True, n_rows_cap=None):
    R = b.R
    cap = b.n_rows if n_rows_cap is None else n_rows_cap
    acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
    p = torch.full((cap,), float("nan"), device="cuda") if want_probs else None
    q = torch.full((cap,), float("nan"), device="cuda") if want_probs else None
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, cap, b.V)).fill_(0xFF)
    B.dspark_verify_draft_stats(b.target, b.draft, b.row_offsets, b.draft_tokens, stats, b.seed, temperature=b.temperature,
                                temperatures=temperatures, draft_row_start=b.draft_row_start, accepted_len=acc,
                                out_tokens=out, out_p_tok=p, out_q_tok=q, dev_status=st, workspace=ws, n_rows=cap)
    torch.cuda.synchronize()
    return dict(acc=acc.cpu().numpy(), out=out.cpu().numpy(), status=int(st.item()),
                p=None if p is None else p.cpu().numpy(), q=None if q is None else q.cpu().numpy())


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("V", [1000, 4097, 40_000, W.V_FULL])
def test_row_stats_are_the_softmax_statistics(V, dtype):
    g = torch.Generator(device="cuda").manual_seed(V)
    x = (torch.randn(9, V + 5, generator=g, device="cuda") * 3).to(dtype)[:, :V]          # strided rows
    x[3, 7] = float("-inf")
    T = 0.8
    got = _stats(x, T).cpu().numpy().astype(np.float64)
    xs = x.double().cpu().numpy() * (1.4426950408889634 / T)
    c = xs.max(axis=1)
    z = np.exp2(xs - c[:, None]).sum(axis=1)
    np.testing.assert_allclose(got[:, 0], c, rtol=2e-7)
    np.testing.assert_allclose(got[:, 1], z, rtol=2e-6)
    # per-row temperatures; rows that cannot be normalised; an unusable temperature
    bad = x.clone()
    bad[1, 3] = float("nan"); bad[2, :] = float("-inf"); bad[4, 0] = float("inf")
    rowT = torch.tensor([0.5, 1.0, 1.0, 2.0, 1.0, 0.0, 1.3, 0.9, 1.1], device="cuda")
    s = _stats(bad, row_T=rowT).cpu().numpy()
    assert np.isnan(s[1]).any() or not (s[1, 1] > 0)
    assert not (s[2, 1] > 0) or np.isneginf(s[2, 0])
    assert np.isnan(s[5]).all()
    xs0 = bad[0].double().cpu().numpy() * (1.4426950408889634 / 0.5)
    np.testing.assert_allclose(s[0, 1], np.exp2(xs0 - xs0.max()).sum(), rtol=2e-6)


@pytest.mark.parametrize("V,block,dtype", [(W.V_FULL, None, torch.bfloat16), (W.V_FULL, 8, torch.bfloat16),
                                           (50_000, None, torch.float32), (4097, 6, torch.bfloat16), (1000, None, torch.float32)])
def test_verifier_with_supplied_draft_statistics(V, block, dtype):
    g0 = torch.Generator().manual_seed(V + 3)
    R = 28
    lengths = torch.randint(0, 7, (R,), generator=g0)
    b = W.sampling_batch(lengths, V, 61, "cuda", temperature=0.9, draft_noise=1.0, verify_seed=99, block=block, dtype=dtype)
    stats = _stats(b.draft, b.temperature)
    for want_probs in (True, False):
        g = _verify_with_stats(b, stats, want_probs=want_probs)
        o = H.oracle_verify(b, eval_all=want_probs)
        mism = H.compare_sampling(g, o, b.row_offsets.cpu().numpy(), check_probs=want_probs)
        plain = H.gpu_verify(b, want_probs=want_probs)
        # Z travels as fp32: a decision can differ from the plain verifier's only where it was within rounding
        assert int((g["acc"] != plain["acc"]).sum()) <= 1
        print(f"[draft stats] V={V} block={block} probs={want_probs}: accepted {g['acc'].tolist()}, {mism} boundary mismatches")
    # per-request temperatures: the statistics carry each row's own temperature
    rng = np.random.default_rng(V)
    temps = torch.tensor(rng.choice([0.7, 1.0, 1.3], size=R), dtype=torch.float32, device="cuda")
    off = b.row_offsets.cpu().numpy()
    n_phys = b.draft.shape[0]
    rowT = torch.ones(n_phys, device="cuda")
    for r in range(R):
        d0 = int(b.draft_row_start[r]) if b.draft_row_start is not None else int(off[r]) - r
        for j in range(int(lengths[r])):
            rowT[d0 + j] = temps[r]
    stats_t = _stats(b.draft, row_T=rowT)
    g = _verify_with_stats(b, stats_t, temperatures=temps)
    o = H.oracle_verify(b, eval_all=True, temperatures=temps)
    H.compare_sampling(g, o, off)


def test_markov_step_hands_out_the_statistics_of_the_rows_it_wrote():
    R, V, gamma, T = 40, 20_000, 4, 0.9
    m = W.markov_input(R, V, 7, "cuda", d=64)
    g = torch.Generator(device="cuda").manual_seed(8)
    U = (torch.randn(gamma, R, V, generator=g, device="cuda") * 3).to(torch.bfloat16)
    packed = torch.empty(B.dspark_markov_w2_packed_bytes(V), dtype=torch.uint8, device="cuda")
    B.dspark_markov_pack_w2(m.W2, packed)
    draft = torch.zeros(R * gamma, V, dtype=torch.bfloat16, device="cuda")
    toks = torch.zeros(gamma, R, dtype=torch.int32, device="cuda")
    stats = torch.full((R * gamma, 2), 7.0, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_markov_workspace_bytes(R, V))
    x_prev = m.x_prev
    for k in range(gamma):
        out_k = draft.view(R, gamma, V)[:, k, :]                    # rows r * gamma + k
        B.dspark_markov_draft_step_stats(U[k], m.W1, packed, x_prev, T, 1000 + k, out_logits=out_k, out_tokens=toks[k],
                                         out_row_stats=stats.view(-1)[2 * k:], row_stats_stride=gamma,
                                         dev_status=st, workspace=ws)
        x_prev = toks[k]
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    want = _stats(draft, T).cpu().numpy()
    got = stats.cpu().numpy()
    np.testing.assert_array_equal(got[:, 0], want[:, 0])            # the reference is max * scale on both sides
    np.testing.assert_allclose(got[:, 1], want[:, 1], rtol=3e-6)    # the sums run over other tiles in another order
    # the verifier on the drafter's rows, tokens and statistics, against the oracle that only sees the logits
    lengths = torch.randint(0, gamma + 1, (R,), generator=torch.Generator().manual_seed(3))
    off = W.offsets_from_lengths(lengths.to("cuda", torch.int32))
    n_rows = int(off[-1])
    offc = off.cpu().numpy()
    target = torch.empty(n_rows, V, dtype=torch.bfloat16, device="cuda")
    flat_tok = torch.zeros(n_rows, dtype=torch.int32, device="cuda")
    for r in range(R):
        for j in range(int(lengths[r]) + 1):
            src = draft[r * gamma + min(j, gamma - 1)].float()
            target[offc[r] + j] = (src + 0.7 * torch.randn(V, generator=g, device="cuda")).to(torch.bfloat16)
            if j < int(lengths[r]):
                flat_tok[offc[r] + j] = toks[j, r]
    drs = torch.arange(R, dtype=torch.int64, device="cuda") * gamma
    b = W.VerifyBatch(target, draft, off, flat_tok, drs, T, 515)
    gv = _verify_with_stats(b, stats)
    ov = H.oracle_verify(b, eval_all=True)
    mism = H.compare_sampling(gv, ov, offc)
    print(f"[draft stats] markov block: accepted {gv['acc'].tolist()}, {mism} boundary mismatches")


def test_unusable_statistics_void_the_request_that_looks_at_them():
    lengths = torch.tensor([2, 3, 0, 1, 4])
    b = W.sampling_batch(lengths, 3000, 5, "cuda", temperature=1.0, verify_seed=1)
    stats = _stats(b.draft, 1.0)
    off = b.row_offsets.cpu().numpy()
    stats[int(off[1]) - 1 + 0] = float("nan")                       # request 1, position 0 (compact draft index lo - r)
    stats[int(off[4]) - 4 + 1, 1] = 0.0                             # request 4, position 1: Z = 0
    g = _verify_with_stats(b, stats)
    assert g["status"] & B.DEV_BAD_ROW
    assert g["acc"][1] == 0 and (g["out"][off[1]:off[2]] == -1).all()
    assert g["acc"][4] == 0 and (g["out"][off[4]:off[5]] == -1).all()
    plain = H.gpu_verify(b)
    for r in (0, 2, 3):
        assert g["acc"][r] == plain["acc"][r]
        np.testing.assert_array_equal(g["out"][off[r]:off[r + 1]], plain["out"][off[r]:off[r + 1]])
    with pytest.raises(B.DsparkError):
        B.dspark_verify_draft_stats(b.target, b.draft, b.row_offsets, b.draft_tokens, stats.view(-1)[1:], b.seed,
                                    accepted_len=torch.zeros(5, dtype=torch.int32, device="cuda"),
                                    out_tokens=torch.zeros(b.n_rows, dtype=torch.int32, device="cuda"), dev_status=None,
                                    workspace=B.workspace(B.dspark_verify_workspace_bytes(5, b.n_rows, b.V)))
