"""Markov-head draft step on the GPU vs the oracle (Section 3.1, Eq. markov; Section 3.2.1, Eq. confidence).

Logits: the GPU accumulates the 256 products in fp32 on the tensor cores, adds the base logit in fp32
and rounds once to bf16; the oracle sums in fp64 and rounds once.  Both are a correct rounding of a
sum whose fp32 error is far below half a bf16 ulp, so the two agree bit for bit except where the
exact value sits within that fp32 error of a bf16 rounding boundary: there they differ by one ulp.
The test bounds the distance to the exact value, the size of a difference (one ulp unless the sum
cancels to nearly zero) and the share of differing elements.
Draw: the GPU's stored logits are handed to the oracle's sampler, which must pick the same tokens.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _run(m: W.MarkovInput, temperature=None, seed=0, out_stride=None, want_conf=True):
    R, V = m.U.shape
    packed = torch.empty(B.dspark_markov_w2_packed_bytes(V), dtype=torch.uint8, device="cuda").fill_(0xFF)
    B.dspark_markov_pack_w2(m.W2, packed)
    stride = V if out_stride is None else out_stride
    out_full = torch.full((R, stride), float("nan"), dtype=torch.bfloat16, device="cuda")
    out = out_full[:, :V]
    conf = torch.full((R,), -7.0, dtype=torch.float32, device="cuda") if want_conf else None
    toks = torch.full((R,), -5, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.workspace(B.dspark_markov_workspace_bytes(R, V)).fill_(0xFF)
    kw = dict(H=m.H if want_conf else None, w_conf=m.w_conf if want_conf else None, out_logits=out, out_conf=conf,
              dev_status=st, workspace=ws)
    if temperature is None:
        B.dspark_markov_logits(m.U, m.W1, packed, m.x_prev, **kw)
    else:
        B.dspark_markov_draft_step(m.U, m.W1, packed, m.x_prev, temperature, seed, out_tokens=toks, **kw)
    torch.cuda.synchronize()
    if out_stride is not None and stride > V:
        assert torch.isnan(out_full[:, V:].float()).all(), "columns past V were written"
    return out, conf, toks, int(st.item())


def _check_logits(m: W.MarkovInput, out: torch.Tensor):
    exact, want_bits = oracle.markov_logits(W.bf16_bits(m.U), W.bf16_bits(m.W1), W.bf16_bits(m.W2), m.x_prev.cpu().numpy())
    got_bits = W.bf16_bits(out)
    got = _bf16_to_f64(got_bits)
    assert np.isfinite(got).all()
    # a correct rounding is within half a bf16 ulp (2^-9 relative, 2^-8 after binade effects) of the
    # exact sum; fp32 accumulation of 257 terms of magnitude <= ~20 adds at most ~1e-4
    assert (np.abs(got - exact) <= np.abs(exact) * 2.0 ** -8 + 2e-4).all()
    diff = got_bits.astype(np.int32) - want_bits.astype(np.int32)
    # near zero the sum cancels, a bf16 ulp shrinks below the fp32 error of the accumulation and the bit
    # patterns may be several ulps apart; there only the absolute bound above applies
    sizeable = np.abs(exact) >= 2.0 ** -4
    assert np.abs(diff[sizeable]).max(initial=0) <= 1
    share = float((diff != 0).mean())
    assert share <= 2e-3, share
    return share


@pytest.mark.parametrize("R,V", [(8, 256), (128, 1024), (130, 4097), (300, 2000), (1, 129), (600, 4097), (700, 8192), (16, W.V_FULL)])
def test_logits_and_confidence(R, V):
    m = W.markov_input(R, V, 100 + R, "cuda", d=96 if V < 10_000 else 1024)
    out, conf, _, st = _run(m)
    assert st == 0
    share = _check_logits(m, out)
    want_c = oracle.confidence(W.bf16_bits(m.H), W.bf16_bits(m.W1), m.w_conf.cpu().numpy(), m.x_prev.cpu().numpy())
    err = np.abs(conf.cpu().numpy().astype(np.float64) - want_c).max()
    assert err <= 1e-6
    print(f"[markov] R={R} V={V}: one-ulp share {share:.2e}, confidence max err {err:.1e}")


def test_padded_output_rows_and_no_confidence():
    m = W.markov_input(40, 3000, 7, "cuda", d=64)
    out, conf, _, st = _run(m, out_stride=3008, want_conf=False)
    assert st == 0 and conf is None
    _check_logits(m, out)


@pytest.mark.parametrize("path,V", [(1, 2048), (1, 3000)])
def test_epilogue_paths_give_the_same_logits(path, V):
    m = W.markov_input(150, V, 11, "cuda", d=64)
    a, _, _, st_a = _run(m, out_stride=3008 if V == 3000 else None)
    B.dspark_markov_set_epilogue_path(path)
    try:
        b, _, _, st_b = _run(m, out_stride=3008 if V == 3000 else None)
    finally:
        B.dspark_markov_set_epilogue_path(0)
    assert st_a == 0 and st_b == 0
    assert torch.equal(a, b)
    _check_logits(m, a)


def test_bad_previous_token_is_flagged():
    m = W.markov_input(5, 512, 9, "cuda", d=32)
    m.x_prev[3] = 512
    out, _, _, st = _run(m)
    assert st & B.DEV_BAD_TOKEN
    # the flagged request gets a zero embedding: its logits are the base logits
    assert torch.equal(out[3], m.U[3])


@pytest.mark.parametrize("R,V,T", [(64, 4097, 1.0), (200, 1500, 0.6), (12, W.V_FULL, 1.0), (33, 5000, 0.0)])
def test_draft_step_draws_like_the_oracle(R, V, T):
    m = W.markov_input(R, V, 300 + R, "cuda", d=64)
    seed = 0xD5A9 + R
    out, conf, toks, st = _run(m, temperature=T, seed=seed)
    assert st == 0
    _check_logits(m, out)
    bits = W.bf16_bits(out)
    off = np.arange(R + 1, dtype=np.int32)
    got = toks.cpu().numpy()
    if T == 0.0:
        o = oracle.verify_greedy(bits, off, np.zeros(R, dtype=np.int32))
        np.testing.assert_array_equal(got, o.out_tokens[:R])
        return
    o = oracle.verify(bits, bits, off, np.zeros(R, dtype=np.int32), T, seed)
    assert (o.accepted_len == 0).all()
    differ = np.nonzero(got != o.out_tokens[:R])[0]
    for r in differ:
        assert o.token_margin[r] < 1e-6, (r, got[r], o.out_tokens[r], o.token_margin[r])
    assert len(differ) <= max(1, R // 50)
    assert ((got >= 0) & (got < V)).all()


def test_degenerate_rows_in_the_draw():
    R, V = 6, 1500
    m = W.markov_input(R, V, 21, "cuda", d=32)
    m.U[1, 700] = float("nan")
    m.U[3, :] = float("-inf")
    m.U[4, 5] = float("inf")
    for T in (1.0, 0.0):
        out, _, toks, st = _run(m, temperature=T, seed=5, want_conf=False)
        bits = W.bf16_bits(out)
        off = np.arange(R + 1, dtype=np.int32)
        got = toks.cpu().numpy()
        if T == 0.0:
            o = oracle.verify_greedy(bits, off, np.zeros(R, dtype=np.int32))
            np.testing.assert_array_equal(got, o.out_tokens[:R])
            assert st == int(np.bitwise_or.reduce(o.status)) == B.DEV_ALL_NEG_INF
        else:
            o = oracle.verify(bits, bits, off, np.zeros(R, dtype=np.int32), T, 5)
            assert st == int(np.bitwise_or.reduce(o.status)) == B.DEV_BAD_ROW
            for r in range(R):
                if o.status[r]:
                    assert got[r] == -1 and r in (1, 3, 4)
                else:
                    assert got[r] == o.out_tokens[r] or o.token_margin[r] < 1e-6


@pytest.mark.parametrize("T", [0.3, 1.0, 2.5])
def test_draw_frequencies_follow_the_softmax(T):
    # many requests share one previous token and one base row: their draws are i.i.d. from one softmax
    R, V = 2048, 300
    m = W.markov_input(R, V, 31, "cuda", d=32, sigma=1.5)
    m.U[:] = m.U[0:1].clone()
    m.x_prev[:] = m.x_prev[0]
    out, _, toks, st = _run(m, temperature=T, seed=99, want_conf=False)
    assert st == 0
    p = torch.softmax(out[0].double() / T, 0).cpu().numpy()
    counts = np.bincount(toks.cpu().numpy(), minlength=V).astype(np.float64)
    # chi-square against the exact probabilities, cells with expectation >= 5 (others pooled)
    exp = p * R
    big = exp >= 5
    chi = ((counts[big] - exp[big]) ** 2 / exp[big]).sum()
    rest_e, rest_c = exp[~big].sum(), counts[~big].sum()
    if rest_e > 0:
        chi += (rest_c - rest_e) ** 2 / rest_e
    dof = int(big.sum())
    assert chi < dof + 6 * (2 * dof) ** 0.5, (chi, dof)


@pytest.mark.parametrize("R", [256, 1024, 17000])
def test_bench_configuration_on_sampled_rows(R):
    # the launch configuration of `bench.py --markov-draft` (V = 129 280); the oracle recomputes a sample of rows
    # that spans the row tiles (first / last row of a tile, a few in between).  R = 17 000: 17 launches, the last
    # one ragged, and the logits of the last rows lie beyond 4 GiB from the base pointer (64-bit addressing)
    V = W.V_FULL
    m = W.markov_input(R, V, 4242, "cuda")
    seed = 77
    out, conf, toks, st = _run(m, temperature=1.0, seed=seed)
    assert st == 0
    rows = sorted({0, 127, 128, R // 2 + 3, R - 129, R - 128, R - 1} | {int(x) for x in np.random.default_rng(R).integers(0, R, 5)})
    idx = torch.tensor(rows, device="cuda")
    sub = W.MarkovInput(m.U[idx].contiguous(), m.W1, m.W2, m.x_prev[idx].contiguous(), m.H[idx].contiguous(), m.w_conf)
    share = _check_logits(sub, out[idx].contiguous())
    want_c = oracle.confidence(W.bf16_bits(sub.H), W.bf16_bits(m.W1), m.w_conf.cpu().numpy(), sub.x_prev.cpu().numpy())
    assert np.abs(conf[idx].cpu().numpy() - want_c).max() <= 1e-6
    # the draw of request r uses the uniform of (seed, r, 0): the oracle verifies one request at a time in place r
    bits = W.bf16_bits(out[idx].contiguous())
    got = toks[idx].cpu().numpy()
    for i, r in enumerate(rows):
        u = oracle.uniforms(seed, r, 0)[1]
        p, _, _, bad = oracle.softmax_row(bits, i, 1.0)
        assert not bad
        cum = np.cumsum(p)
        want = int(np.searchsorted(cum, u, side="right"))
        if got[i] != want:
            assert min(abs(cum[want] - u), abs(u - (cum[want - 1] if want else 0.0))) < 1e-6, (r, got[i], want)
    print(f"[markov] R={R} V={V}: {len(rows)} sampled rows, one-ulp share {share:.2e}")


def test_one_workspace_many_calls_and_graph_replay():
    # calls of different sizes (one with two launches, R > 1024) back to back on one workspace without a host
    # sync in between, then a captured call replayed several times: all must give the results of a fresh call
    V = 9000
    small, big = W.markov_input(200, V, 11, "cuda"), W.markov_input(1300, V, 12, "cuda")
    want = {}
    for name, m in (("small", small), ("big", big)):
        out, conf, toks, st = _run(m, temperature=0.8, seed=5)
        assert st == 0
        want[name] = (out.clone(), toks.clone())
    ws = B.workspace(max(B.dspark_markov_workspace_bytes(m.U.shape[0], V) for m in (small, big))).fill_(0x5A)
    packed = {}
    for name, m in (("small", small), ("big", big)):
        packed[name] = torch.empty(B.dspark_markov_w2_packed_bytes(V), dtype=torch.uint8, device="cuda")
        B.dspark_markov_pack_w2(m.W2, packed[name])
    st = torch.zeros(1, dtype=torch.int32, device="cuda")

    def call(name, m, out, toks):
        B.dspark_markov_draft_step(m.U, m.W1, packed[name], m.x_prev, 0.8, 5, out_logits=out, out_tokens=toks,
                                   dev_status=st, workspace=ws)

    results = []
    for rep in range(3):
        for name, m in (("big", big), ("small", small), ("small", small)):
            out = torch.zeros_like(m.U); toks = torch.full((m.U.shape[0],), -9, dtype=torch.int32, device="cuda")
            call(name, m, out, toks)
            results.append((name, out, toks))
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    for name, out, toks in results:
        assert torch.equal(out.view(torch.int16), want[name][0].view(torch.int16))
        assert torch.equal(toks, want[name][1])
    # graph replay
    out = torch.zeros_like(small.U); toks = torch.full((200,), -9, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        call("small", small, out, toks)                       # warm-up on the capture stream
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            call("small", small, out, toks)
        for rep in range(4):
            out.zero_(); toks.fill_(-9)
            g.replay()
            side.synchronize()
            assert int(st.item()) == 0
            assert torch.equal(out.view(torch.int16), want["small"][0].view(torch.int16))
            assert torch.equal(toks, want["small"][1])
