"""dspark_verify_truncated (top-k / top-p inside the verifier, target rows untouched) vs the oracle pipeline
`warp_target` -> `verify` on the masked rows, and vs the GPU's own two-step pipeline
(dspark_truncate_target + dspark_verify_per_request).  Same bars as the sampling verifier: accepted lengths
and tokens equal unless the oracle's margin is below 1e-6, probabilities within 1e-5 relative."""
import numpy as np
import pytest
import torch

import helpers as H
import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _gpu_truncated(batch, ks, ps, temps, want_probs=True):
    R, cap = batch.R, batch.n_rows
    acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
    p = torch.full((cap,), float("nan"), device="cuda") if want_probs else None
    q = torch.full((cap,), float("nan"), device="cuda") if want_probs else None
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, cap, batch.V)).fill_(0xFF)
    before = batch.target.clone()
    dev = lambda a, dt: None if a is None else torch.as_tensor(np.asarray(a), dtype=dt, device="cuda")
    B.dspark_verify_truncated(batch.target, batch.draft, batch.row_offsets, batch.draft_tokens, batch.seed,
                              temperature=batch.temperature, temperatures=dev(temps, torch.float32),
                              top_k=dev(ks, torch.int32), top_p=dev(ps, torch.float32),
                              draft_row_start=batch.draft_row_start, accepted_len=acc, out_tokens=out,
                              out_p_tok=p, out_q_tok=q, dev_status=st, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(before.view(torch.uint8), batch.target.view(torch.uint8)), "the target rows were modified"
    return dict(acc=acc.cpu().numpy(), out=out.cpu().numpy(), status=int(st.item()),
                p=None if p is None else p.cpu().numpy(), q=None if q is None else q.cpu().numpy())


def _oracle_pipeline(batch, ks, ps, temps):
    off = batch.row_offsets.cpu().numpy()
    masked, tau, kept, margin = oracle.warp_target(W.bf16_bits(batch.target), off, top_k=ks, top_p=ps,
                                                   temperature=batch.temperature, temperatures=temps)
    drs = None if batch.draft_row_start is None else batch.draft_row_start.cpu().numpy()
    o = oracle.verify(masked, W.bf16_bits(batch.draft), off, batch.draft_tokens.cpu().numpy(), batch.temperature,
                      batch.seed, draft_row_start=drs, eval_all=True, n_threads=H.THREADS, temperatures=temps)
    return o, margin


@pytest.mark.parametrize("V,block", [(W.V_FULL, None), (W.V_FULL, 8), (50_000, None), (4097, 6), (1000, None)])
def test_against_the_oracle_pipeline(V, block):
    g0 = torch.Generator().manual_seed(V)
    R = 24
    lengths = torch.randint(0, 7, (R,), generator=g0)
    b = W.sampling_batch(lengths, V, 41, "cuda", temperature=0.9, draft_noise=1.0, verify_seed=77, block=block)
    rng = np.random.default_rng(V)
    ks = rng.choice([0, 1, 5, 40, 500], size=R).astype(np.int32)
    ps = rng.choice([1.0, 0.95, 0.8, 0.5], size=R).astype(np.float32)
    temps = rng.choice([0.7, 1.0, 1.3], size=R).astype(np.float32)
    for use_temps in (False, True):
        t = temps if use_temps else None
        g = _gpu_truncated(b, ks, ps, t)
        o, margin = _oracle_pipeline(b, ks, ps, t)
        if (margin < 1e-5).any():
            pytest.skip("a top-p decision sits on its boundary for this seed")
        mism = H.compare_sampling(g, o, b.row_offsets.cpu().numpy())
        print(f"[verify_truncated] V={V} per-request T={use_temps}: accepted {g['acc'].tolist()}, {mism} boundary mismatches")


def test_matches_the_two_step_gpu_pipeline_and_plain_verify_when_off():
    lengths = torch.tensor([3, 0, 5, 2, 1, 4, 2, 0, 6, 3])
    b = W.sampling_batch(lengths, 30_000, 43, "cuda", temperature=1.0, draft_noise=1.0, verify_seed=9)
    R = b.R
    ks = np.full(R, 20, dtype=np.int32); ps = np.full(R, 0.9, dtype=np.float32); temps = np.full(R, 1.0, dtype=np.float32)
    g = _gpu_truncated(b, ks, ps, temps)
    masked = b.target.clone()
    B.dspark_truncate_target(masked, b.row_offsets, top_k=torch.from_numpy(ks).cuda(), top_p=torch.from_numpy(ps).cuda(),
                             temperatures=torch.from_numpy(temps).cuda())
    mb = W.VerifyBatch(masked, b.draft, b.row_offsets, b.draft_tokens, b.draft_row_start, b.temperature, b.seed, b.meta)
    g2 = H.gpu_verify(mb, temperatures=torch.from_numpy(temps).cuda())
    np.testing.assert_array_equal(g["acc"], g2["acc"])
    np.testing.assert_array_equal(g["out"][:b.n_rows], g2["out"][:b.n_rows])
    have = ~np.isnan(g2["p"][:b.n_rows])
    np.testing.assert_allclose(g["p"][:b.n_rows][have], g2["p"][:b.n_rows][have], rtol=1e-5, atol=1e-37)
    # truncation switched off for everybody: identical to dspark_verify
    off = _gpu_truncated(b, np.zeros(R, np.int32), np.ones(R, np.float32), None)
    plain = H.gpu_verify(b)
    np.testing.assert_array_equal(off["acc"], plain["acc"])
    np.testing.assert_array_equal(off["out"], plain["out"])
    np.testing.assert_array_equal(off["p"][:b.n_rows][have], plain["p"][:b.n_rows][have])


def test_emitted_tokens_follow_the_truncated_distribution():
    # one position, many requests sharing the same rows: corrections and bonus tokens must all lie in the kept set
    R, V = 600, 300
    g0 = torch.Generator().manual_seed(1)
    trow = (torch.randn(1, V, generator=g0) * 2).to(torch.bfloat16)
    drow = (trow.float() + torch.randn(1, V, generator=g0)).to(torch.bfloat16)
    target = trow.repeat(2 * R, 1).contiguous().cuda()
    draft = drow.repeat(R, 1).contiguous().cuda()
    off = torch.arange(0, 2 * R + 1, 2, dtype=torch.int32, device="cuda")
    qd = torch.softmax(drow.float()[0], 0)
    toks = torch.multinomial(qd, R, replacement=True, generator=g0).to(torch.int32)
    dt = torch.zeros(2 * R, dtype=torch.int32); dt[0::2] = toks
    b = W.VerifyBatch(target, draft, off, dt.cuda(), None, 1.0, 5)
    ks = np.full(R, 12, dtype=np.int32)
    g = _gpu_truncated(b, ks, None, None)
    kept = set(torch.topk(trow.float()[0], 12).indices.tolist())
    x = trow.float()[0]
    kept |= {int(v) for v in torch.nonzero(x >= torch.topk(x, 12).values[-1]).flatten()}
    emitted = [int(g["out"][2 * r + g["acc"][r]]) for r in range(R)]
    assert set(emitted) <= kept
    # accepted draft tokens are in the kept set too (p = 0 outside it)
    for r in range(R):
        if g["acc"][r] == 1:
            assert int(toks[r]) in kept
    # frequencies of the emitted tokens at rejected / accepted+bonus positions follow the truncated target:
    # the token finally standing at position 0 is distributed as p~ (losslessness), chi-square over the kept set
    first = np.array([int(toks[r]) if g["acc"][r] == 1 else emitted[r] for r in range(R)])
    p = torch.zeros(V, dtype=torch.float64)
    idx = torch.tensor(sorted(kept))
    p[idx] = torch.softmax(x.double()[idx], 0)
    counts = np.bincount(first, minlength=V).astype(np.float64)
    e = p.numpy() * R
    big = e >= 5
    chi = ((counts[big] - e[big]) ** 2 / e[big]).sum() + ((counts[~big].sum() - e[~big].sum()) ** 2 / max(e[~big].sum(), 1e-9) if e[~big].sum() > 0 else 0.0)
    dof = int(big.sum())
    assert chi < dof + 6 * (2 * dof) ** 0.5, (chi, dof)


def test_flat_rows_take_the_per_row_search():
    # rows without a peak: the top-k threshold and the nucleus lie far below the maximum, beyond the window of
    # the streamed search, so every row goes through the per-row fallback; results must not change
    R, V = 12, 20_000
    g0 = torch.Generator().manual_seed(8)
    lengths = torch.randint(0, 4, (R,), generator=g0)
    off = torch.cat([torch.zeros(1, dtype=torch.int64), torch.cumsum(lengths + 1, 0)]).to(torch.int32)
    n_rows = int(off[-1])
    target = (torch.rand(n_rows, V, generator=g0) * 2 - 1).to(torch.bfloat16)            # flat, both signs
    target[1] = (torch.randn(V, generator=g0) * 30).to(torch.bfloat16)                   # very wide
    draft = (target[: n_rows - R].float() + 0.3 * torch.randn(n_rows - R, V, generator=g0)).to(torch.bfloat16)
    toks = torch.randint(0, V, (n_rows,), generator=g0, dtype=torch.int32)
    b = W.VerifyBatch(target.cuda(), draft.cuda(), off.cuda(), toks.cuda(), None, 1.0, 11)
    ks = np.array([5000, 0, 19000, 200, 0, 70, 3, 0, 12000, 1, 0, 400], dtype=np.int32)
    # top-k is integer work and exact; on a flat row every top-p decision sits within 1e-5 of a value boundary
    # (each value carries 1/V of the mass), so only the decisive cases are given a top-p
    ps = np.array([1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 0.0, 1.0], dtype=np.float32)
    g = _gpu_truncated(b, ks, ps, None)
    o, margin = _oracle_pipeline(b, ks, ps, None)
    mism = H.compare_sampling(g, o, b.row_offsets.cpu().numpy())
    print(f"[verify_truncated] flat rows: accepted {g['acc'].tolist()}, {mism} boundary mismatches")


@pytest.mark.parametrize("temperature", [1.0, 0.7])
def test_a_nucleus_below_the_first_window_gets_a_second_look(temperature):
    # top-p alone on rows with a wide bulk: the nucleus of most rows ends below m - 8 T, where the first window of
    # the streamed search stops; those rows are counted a second time down to the bound on their nucleus (p = 0.9 to
    # 0.99), the others (p = 0.3, 0.5) are resolved by the first look; top-k of more tokens than a row has blocks
    # takes every key of the histogram at once.  Full-vocabulary rows, so that units of several rows interleave.
    R, V = 20, W.V_FULL
    g0 = torch.Generator().manual_seed(31)
    lengths = torch.randint(0, 5, (R,), generator=g0)
    b = W.sampling_batch(lengths, V, 53, "cuda", temperature=temperature, draft_noise=1.0, verify_seed=5)
    ps = np.array([0.9, 0.97, 0.99, 0.5, 0.3, 0.95, 0.9, 1.0, 0.999, 0.9] * 2, dtype=np.float32)
    ks = np.array([0, 0, 0, 0, 0, 0, 0, 300, 0, 2000] * 2, dtype=np.int32)
    off = b.row_offsets.cpu().numpy()
    for want_probs in (True, False):
        g = _gpu_truncated(b, ks, ps, None, want_probs=want_probs)
        assert g["status"] == 0
        o, margin = _oracle_pipeline(b, ks, ps, None)
        skipped, mism = H.compare_away_from_top_p_boundaries(g, o, margin, off)
        if want_probs:
            have = ~np.isnan(g["p"][:b.n_rows]) & (np.asarray(o.p_tok)[:b.n_rows] > 0)
            np.testing.assert_allclose(g["p"][:b.n_rows][have], np.asarray(o.p_tok)[:b.n_rows][have], rtol=1e-5)
        print(f"[verify_truncated] second look, T={temperature}: accepted {g['acc'].tolist()}, {skipped} requests on a "
              f"boundary, {mism} boundary mismatches")
        # a nucleus that ends in the bulk has many tokens of little mass each next to its boundary: some rows are near
        assert skipped <= R // 4 and mism <= 1
    # the two-step pipeline (rows masked in place by the per-row search, then the plain verifier) decides the same
    masked = b.target.clone()
    B.dspark_truncate_target(masked, b.row_offsets, temperature=b.temperature,
                             top_k=torch.as_tensor(ks, device="cuda"), top_p=torch.as_tensor(ps, device="cuda"))
    b2 = W.VerifyBatch(masked, b.draft, b.row_offsets, b.draft_tokens, b.draft_row_start, b.temperature, b.seed)
    g2 = H.gpu_verify(b2)
    g = _gpu_truncated(b, ks, ps, None)
    assert int((g["acc"] != g2["acc"]).sum()) <= 1           # the kept mass comes from the key counts: equal up to rounding


@pytest.mark.parametrize("top_k,top_p", [(50, 0.9), (0, 0.9), (200, 1.0)])
def test_config_3_full_size_with_truncation(top_k, top_p):
    # the batch and launch configuration that `bench.py --top-k 50 --top-p 0.9` times; with top-p alone some rows
    # take the second look of the threshold search, with top-k 200 every row is counted over the widest window
    sched = W.config_3_schedule("cuda")
    gs, _ = H.check_schedule(sched, B.DSPARK_SCHED_EARLY_STOP)
    b = W.config_3_batch(torch.from_numpy(gs["lengths"]), "cuda")
    R = b.R
    ks = np.full(R, top_k, dtype=np.int32); ps = np.full(R, top_p, dtype=np.float32)
    g = _gpu_truncated(b, ks, ps, None, want_probs=False)
    assert g["status"] == 0
    o, margin = _oracle_pipeline(b, ks, ps, None)
    # requests with a row whose top-p decision sits on its boundary (margin < 1e-5 of Z) may legitimately see a
    # neighbouring cut; all others must agree under the usual rule
    skipped, mism = H.compare_away_from_top_p_boundaries(g, o, margin, b.row_offsets.cpu().numpy())
    print(f"[verify_truncated] cfg3 top_k={top_k} top_p={top_p}: {b.n_rows} rows, mean accepted {g['acc'].mean():.2f}, "
          f"{skipped} requests skipped (top-p decision on its boundary), {mism} boundary mismatches")
    assert skipped <= R // 20 and mism <= 2
