"""top-k / top-p truncation of fp32 target rows (in place and inside the verifier) vs the oracle.

An fp32 logit is a 32-bit pattern, so the threshold is found by a descent (a histogram linear in the distance to
the row maximum, then 11 bits of the key at a time) instead of the key window of the bf16 path.  The bars are the
same: the top-k part is integer work and must be exact; the top-p threshold compares sums of exponentials with
top_p * Z, the oracle reports how close that comparison was (margin, relative to Z), and a row may differ from the
oracle only when the margin is below 1e-5 -- then the GPU's cut must be the neighbouring value group.
"""
import numpy as np
import pytest
import torch

import helpers as H
import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu
MARGIN = 1e-5


def _run(target, off, top_k=None, top_p=None, temperature=1.0, temperatures=None):
    t = target.clone()
    n_rows = t.shape[0]
    tau = torch.full((n_rows,), 7.0, device="cuda")
    kept = torch.full((n_rows,), -7, dtype=torch.int32, device="cuda")
    dev = lambda a, dt: None if a is None else torch.as_tensor(np.asarray(a), dtype=dt, device="cuda")
    B.dspark_truncate_target(t, off, top_k=dev(top_k, torch.int32), top_p=dev(top_p, torch.float32), temperature=temperature,
                             temperatures=dev(temperatures, torch.float32), out_tau=tau, out_kept=kept)
    torch.cuda.synchronize()
    return t, tau.cpu().numpy(), kept.cpu().numpy()


def _check(target, off, top_k=None, top_p=None, temperature=1.0, temperatures=None, max_close=None):
    assert target.dtype == torch.float32
    got, tau, kept = _run(target, off, top_k, top_p, temperature, temperatures)
    x_all = target.cpu().numpy()
    want, otau, okept, margin = oracle.warp_target(x_all, off.cpu().numpy(), top_k=top_k, top_p=top_p, temperature=temperature,
                                                   temperatures=temperatures)
    g = got.cpu().numpy()
    close = 0
    n = int(off[-1].item())
    for row in range(n):
        # bit patterns: kept logits untouched (including -0.0), excluded ones -inf
        if np.array_equal(g[row].view(np.uint32), want[row].view(np.uint32)):
            assert kept[row] == okept[row], (row, kept[row], okept[row])
            assert tau[row] == np.float32(otau[row]) or (np.isneginf(otau[row]) and np.isneginf(tau[row]))
            continue
        # a different cut: only where the oracle's own decision was within MARGIN, and then the kept set is
        # still a value cut of the original row at a neighbouring distinct value
        assert margin[row] < MARGIN, (row, margin[row], kept[row], okept[row], tau[row], otau[row])
        x = x_all[row]
        np.testing.assert_array_equal(np.isneginf(g[row]), x < tau[row])
        vals = np.unique(x)
        assert abs(int(np.searchsorted(vals, tau[row])) - int(np.searchsorted(vals, otau[row]))) <= 1
        close += 1
    assert close <= (max(1, n // 20) if max_close is None else max_close)
    return got, tau, kept, close


def test_full_vocabulary_rows_top_k_and_top_p():
    lengths = torch.tensor([2, 0, 3, 1, 4, 0, 2, 1])
    b = W.sampling_batch(lengths, W.V_FULL, 17, "cuda", temperature=0.8, dtype=torch.float32)
    ks = np.array([1, 50, 0, 1000, 20, 129280, 5, 40000], dtype=np.int32)
    ps = np.array([1.0, 0.9, 0.95, 0.5, 1.0, 0.99, 0.0, 0.8], dtype=np.float32)
    Ts = np.array([0.8, 1.0, 0.6, 1.5, 1.0, 0.7, 1.0, 1.2], dtype=np.float32)
    got, tau, kept, close = _check(b.target, b.row_offsets, ks, ps, temperatures=Ts)
    assert kept.min() >= 1
    print(f"[truncate fp32] kept sizes {kept.tolist()}, {close} near-boundary rows")


@pytest.mark.parametrize("V", [1000, 4097, 70000])
def test_ties_flat_rows_and_values_that_differ_in_the_last_bits(V):
    g = torch.Generator(device="cuda").manual_seed(V)
    n = 14
    t = torch.empty(n, V, device="cuda")
    t[0:3] = torch.randn(3, V, generator=g, device="cuda") * 3
    t[3:5] = torch.randint(-3, 4, (2, V), generator=g, device="cuda").float() * 0.5          # few distinct values
    t[5] = 1.25                                                                              # one value only
    t[6:8] = torch.rand(2, V, generator=g, device="cuda") * 2 - 1                            # flat, both signs
    t[8] = -torch.rand(V, generator=g, device="cuda") * 40                                   # all negative, far apart
    t[9] = torch.randn(V, generator=g, device="cuda") * 1e-3                                 # tiny values, -0/+0
    t[9, ::7] = -0.0
    t[9, 3::7] = 0.0
    t[10:12] = torch.randn(2, V, generator=g, device="cuda") * 8
    # neighbouring bit patterns: the descent has to go down to single keys
    base = torch.tensor(np.float32(2.5)).view(torch.int32).item()
    t[12] = (torch.randint(0, 37, (V,), generator=g, device="cuda", dtype=torch.int32) + base).view(torch.float32)
    t[13] = (torch.randint(0, 5000, (V,), generator=g, device="cuda", dtype=torch.int32) * 4097 + base).view(torch.float32)
    off = torch.arange(n + 1, dtype=torch.int32, device="cuda")
    ks = np.array([3, 0, V - 1, 10, 0, 5, V // 2, 0, 7, 100, 0, 1, 40, 333], dtype=np.int32)
    ps = np.array([1.0, 0.7, 0.999, 0.6, 0.5, 0.3, 0.9, 0.999, 0.9, 0.5, 0.0, 0.2, 0.5, 0.9], dtype=np.float32)
    _check(t, off, ks, ps, temperature=1.3)
    _check(t, off, ks, None, temperature=1.0, max_close=0)            # counts only: exact
    _check(t, off, None, ps, temperature=0.7)


def test_strided_rows_and_requests_of_several_rows():
    V = 5003
    g = torch.Generator(device="cuda").manual_seed(5)
    orig = torch.randn(9, V + 13, generator=g, device="cuda") * 2.5
    buf = orig.clone()
    t = buf[:, :V]                                                     # row stride V + 13
    off = torch.tensor([0, 3, 3, 7, 9], dtype=torch.int32, device="cuda")
    ks = np.array([4, 9, 0, 60], dtype=np.int32)
    ps = np.array([0.9, 0.5, 0.8, 1.0], dtype=np.float32)
    Ts = np.array([1.0, 0.5, 2.0, 0.9], dtype=np.float32)
    kept = torch.full((9,), -7, dtype=torch.int32, device="cuda")
    B.dspark_truncate_target(t, off, top_k=torch.from_numpy(ks).cuda(), top_p=torch.from_numpy(ps).cuda(),
                             temperatures=torch.from_numpy(Ts).cuda(), out_kept=kept)
    torch.cuda.synchronize()
    want, otau, okept, margin = oracle.warp_target(np.ascontiguousarray(orig[:, :V].cpu().numpy()), off.cpu().numpy(), top_k=ks,
                                                   top_p=ps, temperatures=Ts)
    assert (margin > MARGIN).all()
    np.testing.assert_array_equal(np.ascontiguousarray(t.cpu().numpy()).view(np.uint32), want.view(np.uint32))
    np.testing.assert_array_equal(kept.cpu().numpy(), okept)
    assert torch.equal(buf[:, V:], orig[:, V:])                        # nothing outside the rows is touched


def test_rows_that_are_left_alone():
    V = 3000
    t = torch.randn(6, V, device="cuda") * 2
    t[1, 5] = float("nan")
    t[2, 9] = float("inf")
    t[3, :] = float("-inf")
    off = torch.tensor([0, 2, 4, 6], dtype=torch.int32, device="cuda")
    got, tau, kept = _run(t, off, top_k=[4, 4, 0], top_p=[0.9, 0.9, 1.0])
    for row in (1, 2, 3, 4, 5):
        assert torch.equal(got[row].view(torch.int32), t[row].view(torch.int32)) and np.isneginf(tau[row]) and kept[row] == V
    assert kept[0] <= 4 and not torch.equal(got[0].view(torch.int32), t[0].view(torch.int32))


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
    assert torch.equal(before.view(torch.int32), batch.target.view(torch.int32)), "the target rows were modified"
    return dict(acc=acc.cpu().numpy(), out=out.cpu().numpy(), status=int(st.item()),
                p=None if p is None else p.cpu().numpy(), q=None if q is None else q.cpu().numpy())


@pytest.mark.parametrize("V,block", [(W.V_FULL, None), (50_000, 8), (4097, None), (1000, 6)])
def test_verifier_on_the_truncated_fp32_target_against_the_oracle_pipeline(V, block):
    g0 = torch.Generator().manual_seed(V + 1)
    R = 20
    lengths = torch.randint(0, 7, (R,), generator=g0)
    rng = np.random.default_rng(V + 1)
    ks = rng.choice([0, 1, 5, 40, 500], size=R).astype(np.int32)
    ps = rng.choice([1.0, 0.95, 0.8, 0.5], size=R).astype(np.float32)
    temps = rng.choice([0.7, 1.0, 1.3], size=R).astype(np.float32)
    for use_temps in (False, True):
        t = temps if use_temps else None
        b = W.sampling_batch(lengths, V, 47, "cuda", temperature=0.9, draft_noise=1.0, verify_seed=78, block=block,
                             dtype=torch.float32)
        off = b.row_offsets.cpu().numpy()
        # Where a top-p decision of the oracle sits on its boundary either neighbour is right and the comparison of
        # the verifier's outputs would say nothing (on a flat full-vocabulary row a single token carries about 1e-5
        # of the mass, so this is common): those requests run without top-p here.
        ps_run = ps.copy()
        for _ in range(3):
            masked, tau, kept, margin = oracle.warp_target(W.bf16_bits(b.target), off, top_k=ks, top_p=ps_run,
                                                           temperature=b.temperature, temperatures=t)
            on_boundary = [r for r in range(R) if (margin[off[r]:off[r + 1]] < 1e-5).any()]
            if not on_boundary:
                break
            ps_run[on_boundary] = 1.0
        assert not on_boundary and (ps_run < 1.0).sum() >= 3
        g = _gpu_truncated(b, ks, ps_run, t)
        drs = None if b.draft_row_start is None else b.draft_row_start.cpu().numpy()
        o = oracle.verify(masked, W.bf16_bits(b.draft), off, b.draft_tokens.cpu().numpy(), b.temperature, b.seed,
                          draft_row_start=drs, eval_all=True, n_threads=H.THREADS, temperatures=t)
        mism = H.compare_sampling(g, o, off)
        print(f"[verify_truncated fp32] V={V} per-request T={use_temps}, top-p on {int((ps_run < 1.0).sum())} requests: accepted {g['acc'].tolist()}, {mism} boundary mismatches")


def test_matches_the_two_step_gpu_pipeline_on_fp32_rows():
    lengths = torch.tensor([3, 0, 5, 2, 1, 4, 2, 0, 6, 3])
    b = W.sampling_batch(lengths, 30_000, 43, "cuda", temperature=1.0, draft_noise=1.0, verify_seed=9, dtype=torch.float32)
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


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_truncated_verifier_replayed_from_a_cuda_graph(dtype):
    # the call captured once and replayed on other logits in the same buffers gives what the eager call gives
    lengths = torch.tensor([2, 0, 4, 1, 3, 2, 0, 5])
    V = 20_000
    batches = [W.sampling_batch(lengths, V, 300 + i, "cuda", temperature=0.8, draft_noise=1.0, verify_seed=11, dtype=dtype)
               for i in range(3)]
    b0 = batches[0]
    R, cap = b0.R, b0.n_rows
    ks = torch.full((R,), 30, dtype=torch.int32, device="cuda")
    ps = torch.full((R,), 0.9, dtype=torch.float32, device="cuda")
    target = b0.target.clone(); draft = b0.draft.clone()
    acc = torch.zeros(R, dtype=torch.int32, device="cuda")
    out = torch.zeros(cap, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_verify_workspace_bytes(R, cap, V))

    def call():
        B.dspark_verify_truncated(target, draft, b0.row_offsets, b0.draft_tokens, b0.seed, temperature=b0.temperature,
                                  top_k=ks, top_p=ps, accepted_len=acc, out_tokens=out, dev_status=st, workspace=ws)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call()                                                # eager pass first: sets the kernel attributes
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        call()
    torch.cuda.synchronize()
    for b in batches[::-1]:
        target.copy_(b.target); draft.copy_(b.draft)
        call()
        torch.cuda.synchronize()
        want = (acc.cpu().numpy().copy(), out.cpu().numpy().copy(), int(st.item()))
        acc.fill_(-5); out.fill_(-5)
        graph.replay()
        torch.cuda.synchronize()
        np.testing.assert_array_equal(acc.cpu().numpy(), want[0])
        np.testing.assert_array_equal(out.cpu().numpy(), want[1])
        assert int(st.item()) == want[2] == 0
