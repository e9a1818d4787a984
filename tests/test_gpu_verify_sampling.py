"""GPU sampling verifier vs the CPU oracle.  Bars: accepted lengths and tokens bit-exact except
where the oracle's margin to a decision boundary is below 1e-6 (counted and printed);
p(x), q(x) within 1e-5 relative."""
import numpy as np
import pytest
import torch
from scipy import stats

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _report(name, batch, g, mism):
    lens = batch.meta["lengths"].cpu().numpy()
    print(f"[{name}] requests={batch.R} rows={batch.n_rows} mean_len={lens.mean():.2f} "
          f"mean_accepted={g['acc'].mean():.2f} rejected={(g['acc'] < lens).mean():.2f} "
          f"boundary_mismatches={mism} ({mism / batch.R:.2e} per request); running totals by rule: {H.MISMATCH_COUNTS}")


def test_config_2_reduced():
    batch = W.config_2("cuda", R=16)
    g, o, mism = H.check_sampling(batch)
    _report("cfg2/R=16", batch, g, mism)


def test_config_2_full_size():
    batch = W.config_2("cuda")
    g, o, mism = H.check_sampling(batch)
    _report("cfg2", batch, g, mism)
    assert mism <= 1
    # the run without probability outputs (stops at the first rejection) gives the same tokens
    g2 = H.gpu_verify(batch, want_probs=False)
    np.testing.assert_array_equal(g2["acc"], g["acc"])
    np.testing.assert_array_equal(g2["out"], g["out"])


def test_config_3_full_size_scheduled_then_verified():
    sched = W.config_3_schedule("cuda")
    gs, _ = H.check_schedule(sched, B.DSPARK_SCHED_EARLY_STOP)
    batch = W.config_3_batch(torch.from_numpy(gs["lengths"]), "cuda")
    assert torch.equal(batch.row_offsets.cpu(), torch.from_numpy(gs["offsets"]))
    g, o, mism = H.check_sampling(batch)
    _report("cfg3", batch, g, mism)
    assert mism <= 2


def test_config_5_full_size_scheduled_then_verified():
    sched = W.config_5_schedule("cuda")
    gs, _ = H.check_schedule(sched, B.DSPARK_SCHED_EARLY_STOP)
    batch = W.config_5_batch(torch.from_numpy(gs["lengths"]), "cuda")
    g, o, mism = H.check_sampling(batch)
    _report("cfg5", batch, g, mism)
    assert mism <= 3
    lens = gs["lengths"]
    assert (g["acc"] < lens).mean() > 0.3          # high rejection rate: the residual pass is exercised


@pytest.mark.parametrize("V", [2, 16, 1000, 4097, 129281])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_odd_vocabularies_dtypes_and_paths(V, dtype):
    lengths = torch.tensor([3, 0, 1, 6, 2, 0, 4, 8, 1])
    batch = W.sampling_batch(lengths, V, 70 + V, "cuda", dtype=dtype, temperature=0.9, verify_seed=V)
    g, o, mism = H.check_sampling(batch)
    B.dspark_set_stream_path(1)
    try:
        g1, o1, mism1 = H.check_sampling(batch)
    finally:
        B.dspark_set_stream_path(0)
    assert mism + mism1 <= 1
    np.testing.assert_array_equal(g["acc"], g1["acc"])


@pytest.mark.parametrize("V,dtype,block", [(W.V_FULL, torch.bfloat16, 8), (50_000, torch.float32, None), (4097, torch.bfloat16, None)])
def test_bonus_rows_in_the_second_pass_change_nothing(V, dtype, block):
    # the verifier leaves the bonus rows out of its statistics pass and streams them in the second pass for the requests
    # that accepted every draft token; the earlier order (every bonus row in the statistics pass) stays behind the
    # diagnostic switch: same accepted lengths, tokens and probabilities, bit for bit -- also with the draft rows'
    # statistics handed over, with per-request temperatures, and for requests without a draft token
    g0 = torch.Generator().manual_seed(V)
    R = 40
    lengths = torch.randint(0, 7, (R,), generator=g0)
    lengths[:4] = 0
    b = W.sampling_batch(lengths, V, 90, "cuda", dtype=dtype, temperature=0.8, draft_noise=0.5, verify_seed=17, block=block)
    temps = torch.tensor(np.random.default_rng(V).choice([0.6, 1.0, 1.4], size=R), dtype=torch.float32, device="cuda")
    stats = torch.empty(b.draft.shape[0], 2, device="cuda")
    B.dspark_row_stats(b.draft, b.temperature, out_row_stats=stats)

    def run_all():
        res = [H.gpu_verify(b), H.gpu_verify(b, temperatures=temps)]
        acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
        out = torch.full((b.n_rows,), -7, dtype=torch.int32, device="cuda")
        p = torch.full((b.n_rows,), float("nan"), device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = B.workspace(B.dspark_verify_workspace_bytes(R, b.n_rows, V))
        B.dspark_verify_draft_stats(b.target, b.draft, b.row_offsets, b.draft_tokens, stats, b.seed, temperature=b.temperature,
                                    draft_row_start=b.draft_row_start, accepted_len=acc, out_tokens=out, out_p_tok=p,
                                    out_q_tok=None, dev_status=st, workspace=ws)
        torch.cuda.synchronize()
        res.append(dict(acc=acc.cpu().numpy(), out=out.cpu().numpy(), p=p.cpu().numpy(), status=int(st.item())))
        return res

    new = run_all()
    B.dspark_set_stream_path(16)
    try:
        old = run_all()
    finally:
        B.dspark_set_stream_path(0)
    assert (new[0]["acc"] == lengths.numpy()).any() and (new[0]["acc"] < lengths.numpy()).any()    # both kinds of request
    for a, c in zip(new, old):
        assert a["status"] == 0 and c["status"] == 0
        np.testing.assert_array_equal(a["acc"], c["acc"])
        np.testing.assert_array_equal(a["out"], c["out"])
        np.testing.assert_array_equal(a["p"], c["p"])          # NaN where not evaluated, on both sides


# 256 is the number of block values the finalize kernel keeps in registers; rows of 131 072 / 262 144 / 524 288
# logits sit exactly at 256 residual or statistics blocks for one of the dtypes
_BLOCK_COUNT_EDGES = [(dt, V + d) for dt in (torch.bfloat16, torch.float32)
                      for V in (131_072, 262_144, 524_288) for d in (0, 1)]


@pytest.mark.parametrize("dtype,V", [(torch.bfloat16, 600_011), (torch.float32, 300_000), (torch.bfloat16, 1_100_000),
                                     (torch.float32, 200_000), (torch.bfloat16, 400_000)] + _BLOCK_COUNT_EDGES)
def test_very_large_vocabularies(dtype, V):
    # more than 256 statistics / residual blocks per row: the inverse CDF walks memory instead of registers.
    # The last two: at most 256 statistics blocks but more than 256 residual blocks per row, so a bonus draw
    # still runs from registers while a residual draw walks memory
    lengths = torch.tensor([2, 0, 3, 1, 0, 2])
    batch = W.sampling_batch(lengths, V, 5, "cuda", dtype=dtype, temperature=1.1, draft_noise=1.5, verify_seed=V % 97)
    g, o, mism = H.check_sampling(batch)
    assert mism == 0
    assert (g["acc"] < lengths.numpy()).any() and (g["acc"] == lengths.numpy()).any()   # both kinds of draw


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_per_request_temperatures(dtype):
    g = torch.Generator(device="cpu"); g.manual_seed(4)
    lengths = torch.randint(0, 7, (48,), generator=g)
    batch = W.sampling_batch(lengths, W.V_FULL if dtype == torch.bfloat16 else 40_000, 17, "cuda", dtype=dtype,
                             draft_noise=1.2, verify_seed=6, block=8)
    temps = (0.5 + 1.2 * torch.rand(48, generator=g)).float().cuda()
    gp, o, mism = H.check_sampling(batch, temperatures=temps)
    assert mism == 0
    # a uniform temperature array reproduces the scalar entry point bit for bit
    uni = torch.full((48,), 0.8, device="cuda")
    a = H.gpu_verify(W.VerifyBatch(batch.target, batch.draft, batch.row_offsets, batch.draft_tokens,
                                   batch.draft_row_start, 0.8, batch.seed, batch.meta))
    b = H.gpu_verify(batch, temperatures=uni)
    for k in ("acc", "out", "p", "q"):
        np.testing.assert_array_equal(a[k], b[k])
    # invalid temperatures void only their own requests
    bad = temps.clone(); bad[5] = 0.0; bad[9] = float("nan"); bad[11] = float("inf")
    gb, ob, _ = H.check_sampling(batch, temperatures=bad)
    assert gb["status"] & B.DEV_BAD_TEMPERATURE and (gb["acc"][[5, 9, 11]] == 0).all()
    keep = np.ones(48, bool); keep[[5, 9, 11]] = False
    np.testing.assert_array_equal(gb["acc"][keep], gp["acc"][keep])


def test_compact_and_block_layouts_agree():
    lengths = torch.tensor([2, 5, 0, 3, 1, 7])
    a = W.sampling_batch(lengths, 20000, 3, "cuda", verify_seed=5)
    b = W.sampling_batch(lengths, 20000, 3, "cuda", verify_seed=5, block=8)
    ga, _, _ = H.check_sampling(a)
    gb, _, _ = H.check_sampling(b)
    np.testing.assert_array_equal(ga["acc"], gb["acc"])
    np.testing.assert_array_equal(ga["out"], gb["out"])


def test_padded_strides_and_capacity():
    lengths = torch.tensor([2, 0, 4, 1])
    b = W.sampling_batch(lengths, 3000, 8, "cuda", verify_seed=3)
    tp = torch.zeros(b.n_rows + 3, 3080, dtype=torch.bfloat16, device="cuda"); tp[: b.n_rows, :3000] = b.target
    dp = torch.zeros(b.draft.shape[0], 3008, dtype=torch.bfloat16, device="cuda"); dp[:, :3000] = b.draft
    toks = torch.zeros(b.n_rows + 3, dtype=torch.int32, device="cuda"); toks[: b.n_rows] = b.draft_tokens
    padded = W.VerifyBatch(tp[:, :3000], dp[:, :3000], b.row_offsets, toks, None, b.temperature, b.seed, b.meta)
    g0, _, _ = H.check_sampling(b)
    g1 = H.gpu_verify(padded)
    np.testing.assert_array_equal(g0["acc"], g1["acc"])
    np.testing.assert_array_equal(g0["out"][: b.n_rows], g1["out"][: b.n_rows])
    assert (g1["out"][b.n_rows:] == -7).all()


def test_degenerate_batches():
    V = 5000
    lengths = torch.tensor([4, 4, 4, 0, 0])
    b = W.sampling_batch(lengths, V, 21, "cuda", verify_seed=9)
    # draft == target: every token accepted (u < 1), bonus from p
    same = W.VerifyBatch(b.target, b.target[[0, 1, 2, 3, 5, 6, 7, 8, 10, 11, 12, 13]].contiguous(), b.row_offsets,
                         b.draft_tokens, None, 1.0, 9, b.meta)
    g, o, _ = H.check_sampling(same)
    assert (g["acc"] == lengths.numpy()).all()
    # target -inf at the draft token: p(x) = 0, always rejected, residual never returns x
    t = b.target.clone()
    off = b.row_offsets.cpu().numpy()
    for r in range(3):
        t[off[r], b.draft_tokens[off[r]].item()] = float("-inf")
    rej = W.VerifyBatch(t, b.draft, b.row_offsets, b.draft_tokens, None, 1.0, 9, b.meta)
    g, o, _ = H.check_sampling(rej)
    assert (g["acc"][:3] == 0).all()
    for r in range(3):
        assert g["out"][off[r]] != b.draft_tokens[off[r]].item()
    # NaN row, +inf row, all -inf row, bad token: flagged, nothing emitted, others unaffected
    t2 = b.target.clone(); t2[off[0] + 1, 17] = float("nan"); t2[off[1], :] = float("-inf"); t2[off[2], 5] = float("inf")
    toks = b.draft_tokens.clone(); toks[off[4] - 1] = 0
    bad = W.VerifyBatch(t2, b.draft, b.row_offsets, toks, None, 1.0, 9, b.meta)
    g, o, _ = H.check_sampling(bad)
    assert g["status"] & B.DEV_BAD_ROW and (g["acc"][:3] == 0).all() and g["out"][off[3]] >= 0
    toks[off[0]] = V
    g, o, _ = H.check_sampling(W.VerifyBatch(b.target, b.draft, b.row_offsets, toks, None, 1.0, 9, b.meta))
    assert g["status"] & B.DEV_BAD_TOKEN


def test_which_rows_void_a_request_and_hidden_nan():
    V = 6000                                        # three 4 KB blocks of bf16 per row
    lengths = torch.tensor([5, 5, 0, 2])
    b = W.sampling_batch(lengths, V, 33, "cuda", verify_seed=12, draft_noise=2.0)
    off = b.row_offsets.cpu().numpy()
    # (1) a NaN in a block whose other elements are all -inf: the block maximum does not see it
    t = b.target.clone()
    t[off[2], :] = float("-inf"); t[off[2], 100] = 3.0; t[off[2], 5000] = float("nan")
    g, o, _ = H.check_sampling(W.VerifyBatch(t, b.draft, b.row_offsets, b.draft_tokens, None, 1.0, 12, b.meta))
    assert o.status[2] & B.DEV_BAD_ROW and g["status"] & B.DEV_BAD_ROW and g["out"][off[2]] == -1
    # (2) an unusable row behind the first rejection: looked at only when the probabilities are asked for
    base = H.gpu_verify(b, want_probs=False)
    r = next(r for r in (0, 1) if base["acc"][r] < 4)        # rejected with at least one position behind it
    t = b.target.clone()
    t[off[r] + int(base["acc"][r]) + 1, 7] = float("nan")
    bad = W.VerifyBatch(t, b.draft, b.row_offsets, b.draft_tokens, None, 1.0, 12, b.meta)
    g0, o0, _ = H.check_sampling(bad, want_probs=False)
    assert g0["status"] == 0 and g0["acc"][r] == base["acc"][r] and g0["out"][off[r] + g0["acc"][r]] >= 0
    g1, o1, _ = H.check_sampling(bad, want_probs=True)
    assert g1["status"] & B.DEV_BAD_ROW and (g1["out"][off[r]:off[r + 1]] == -1).all()
    # (3) a request with a token out of range AND an invalid temperature reports both
    toks = b.draft_tokens.clone(); toks[off[0]] = V
    temps = torch.tensor([float("nan"), 1.0, 1.0, 0.9], device="cuda")
    g, o, _ = H.check_sampling(W.VerifyBatch(b.target, b.draft, b.row_offsets, toks, None, 1.0, 12, b.meta), temperatures=temps)
    assert g["status"] == B.DEV_BAD_TOKEN | B.DEV_BAD_TEMPERATURE


def test_lossless_invariant_on_the_gpu():
    # first emitted token ~ p whatever q is (chi-square, V = 16, 60k single-position requests)
    rng = np.random.default_rng(5)
    V, n = 16, 60_000
    p = rng.dirichlet(np.ones(V) * 0.6); q = rng.dirichlet(np.ones(V) * 0.6)
    tl = torch.tensor(np.log(p), dtype=torch.float32); ql = torch.tensor(np.log(q), dtype=torch.float32)
    target = tl.repeat(2 * n, 1).cuda(); draft = ql.repeat(n, 1).cuda()
    pp = torch.softmax(tl.double(), 0).numpy(); qq = torch.softmax(ql.double(), 0).numpy()
    toks = torch.zeros(2 * n, dtype=torch.int32); toks[0::2] = torch.from_numpy(rng.choice(V, size=n, p=qq)).int()
    off = (2 * torch.arange(n + 1)).int()
    batch = W.VerifyBatch(target, draft, off.cuda(), toks.cuda(), None, 1.0, 123, {"lengths": torch.ones(n)})
    g = H.gpu_verify(batch, want_probs=False)
    first = g["out"][0::2]
    assert stats.chisquare(np.bincount(first, minlength=V), pp * n).pvalue > 1e-3
    want = 1 - 0.5 * np.abs(pp - qq).sum()
    assert abs(g["acc"].mean() - want) < 4 * np.sqrt(want * (1 - want) / n)
    bonus = g["out"][1::2][g["acc"] == 1]
    assert stats.chisquare(np.bincount(bonus, minlength=V), pp * len(bonus)).pvalue > 1e-3


def test_results_are_reproducible_run_to_run():
    batch = W.config_2("cuda", R=24)
    a = H.gpu_verify(batch)
    for _ in range(3):
        b = H.gpu_verify(batch)
        for k in ("acc", "out", "p", "q"):
            np.testing.assert_array_equal(a[k], b[k])


def test_one_workspace_serves_calls_of_different_kinds_and_sizes():
    # the unit counters of the streamed passes live in the workspace: whatever an earlier call (greedy or
    # sampling, larger or smaller, many back to back without a host sync) left there must not matter
    big = W.config_2("cuda", R=24)
    small = W.sampling_batch(torch.tensor([2, 0, 5]), 40_000, 8, "cuda", verify_seed=4)
    greedy = W.greedy_batch(torch.tensor([3, 1, 0, 6]), 50_000, 3, "cuda", perturb=0.3)
    want_big, want_small = H.gpu_verify(big), H.gpu_verify(small)
    want_greedy = H.gpu_verify_greedy(greedy)
    nbytes = max(B.dspark_verify_workspace_bytes(b.R, b.n_rows, b.V) for b in (big, small, greedy))
    ws = B.workspace(nbytes).fill_(0xA5)

    def sampling(b):
        acc = torch.full((b.R,), -7, dtype=torch.int32, device="cuda")
        out = torch.full((b.n_rows,), -7, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.dspark_verify(b.target, b.draft, b.row_offsets, b.draft_tokens, b.temperature, b.seed,
                        draft_row_start=b.draft_row_start, accepted_len=acc, out_tokens=out, dev_status=st,
                        workspace=ws, n_rows=b.n_rows)
        return acc, out, st

    def greedy_call(b):
        acc = torch.full((b.R,), -7, dtype=torch.int32, device="cuda")
        out = torch.full((b.n_rows,), -7, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.dspark_verify_greedy(b.target, b.row_offsets, b.draft_tokens, accepted_len=acc, out_tokens=out,
                               dev_status=st, workspace=ws, n_rows=b.n_rows)
        return acc, out, st

    results = []
    for rep in range(4):                         # all enqueued before the first result is read
        results.append(("big", sampling(big)))
        results.append(("greedy", greedy_call(greedy)))
        results.append(("small", sampling(small)))
        results.append(("small", sampling(small)))
    torch.cuda.synchronize()
    for kind, (acc, out, st) in results:
        assert int(st.item()) == 0
        if kind == "greedy":
            np.testing.assert_array_equal(acc.cpu().numpy(), want_greedy[0])
            np.testing.assert_array_equal(out.cpu().numpy(), want_greedy[1])
        else:
            want = want_big if kind == "big" else want_small
            np.testing.assert_array_equal(acc.cpu().numpy(), want["acc"])
            np.testing.assert_array_equal(out.cpu().numpy(), want["out"])


def test_calls_on_several_streams_at_once():
    # every call has its own workspace; the kernels of different calls share the SMs (so the CTAs of one grid are
    # not all resident at once) and nothing in the library is shared between them
    rng = np.random.default_rng(5)
    jobs = []
    for i in range(4):
        R, V = int(rng.integers(20, 200)), int(rng.choice([5000, 40_000, W.V_FULL]))
        b = W.sampling_batch(torch.from_numpy(rng.integers(0, 8, size=R)), V, 100 + i, "cuda", verify_seed=50 + i, draft_noise=1.5)
        jobs.append(dict(b=b, ref=H.gpu_verify(b, want_probs=False), stream=torch.cuda.Stream(),
                         ws=B.workspace(B.dspark_verify_workspace_bytes(b.R, b.n_rows, b.V)).fill_(0xFF),
                         acc=torch.zeros(b.R, dtype=torch.int32, device="cuda"),
                         out=torch.zeros(b.n_rows, dtype=torch.int32, device="cuda"),
                         st=torch.zeros(1, dtype=torch.int32, device="cuda")))
    torch.cuda.synchronize()
    for it in range(12):
        for j in jobs:
            with torch.cuda.stream(j["stream"]):
                j["acc"].fill_(-3); j["out"].fill_(-3)
                b = j["b"]
                B.dspark_verify(b.target, b.draft, b.row_offsets, b.draft_tokens, b.temperature, b.seed,
                                draft_row_start=b.draft_row_start, accepted_len=j["acc"], out_tokens=j["out"],
                                dev_status=j["st"], workspace=j["ws"], n_rows=b.n_rows)
        torch.cuda.synchronize()
        for j in jobs:
            assert int(j["st"].item()) == 0
            np.testing.assert_array_equal(j["acc"].cpu().numpy(), j["ref"]["acc"])
            np.testing.assert_array_equal(j["out"].cpu().numpy(), j["ref"]["out"])


def test_host_side_errors():
    b = W.sampling_batch(torch.tensor([1, 2]), 512, 1, "cuda")
    acc = torch.zeros(2, dtype=torch.int32, device="cuda"); out = torch.zeros(5, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(2, 5, 512))
    for T in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(B.DsparkError, match="invalid"):
            B.dspark_verify(b.target, b.draft, b.row_offsets, b.draft_tokens, T, 1, accepted_len=acc,
                            out_tokens=out, dev_status=None, workspace=ws)
    with pytest.raises(B.DsparkError, match="workspace"):
        B.dspark_verify(b.target, b.draft, b.row_offsets, b.draft_tokens, 1.0, 1, accepted_len=acc,
                        out_tokens=out, dev_status=None, workspace=torch.empty(512, dtype=torch.uint8, device="cuda"))
