"""Randomised small cases: many shapes, strides, dtypes, temperatures and schedules, each compared
with the oracle under the same bars as the configuration tests."""
import numpy as np
import pytest
import torch

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _pad_rows(t, rng):
    """Same values in a buffer with a random row stride and a random element offset."""
    pad = int(rng.integers(0, 9))
    shift = int(rng.integers(0, 5))
    buf = torch.zeros(t.shape[0], t.shape[1] + pad + shift, dtype=t.dtype, device=t.device)
    buf[:, shift:shift + t.shape[1]] = t
    return buf[:, shift:shift + t.shape[1]]


# seed 1416: a request whose target and draft rows agree to about 1e-10 in total variation (temperature 0.43,
# one token holds almost all the mass) and that is rejected all the same: the residual's total mass is far
# below what fp32 resolves, the emitted token is decided by rounding (oracle margin 1e-11 in probability)
@pytest.mark.parametrize("seed", list(range(12)) + [1416])
def test_sampling_fuzz(seed):
    rng = np.random.default_rng(1000 + seed)
    total_mism = 0
    for _ in range(6):
        R = int(rng.integers(1, 30))
        V = int(rng.choice([1, 2, 3, 17, 255, 1024, 2049, 5000, 12345]))
        lengths = torch.from_numpy(rng.integers(0, 10, size=R))
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        block = int(lengths.max()) + int(rng.integers(0, 3)) if rng.random() < 0.5 and int(lengths.max()) > 0 else None
        b = W.sampling_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", dtype=dtype,
                             sigma=float(rng.uniform(0.5, 4)), draft_noise=float(rng.uniform(0.0, 2.5)),
                             temperature=float(rng.uniform(0.3, 2.0)), verify_seed=int(rng.integers(0, 2**40)),
                             block=block)
        if rng.random() < 0.5:
            b = W.VerifyBatch(_pad_rows(b.target, rng), _pad_rows(b.draft, rng), b.row_offsets, b.draft_tokens,
                              b.draft_row_start, b.temperature, b.seed, b.meta)
        temps = None
        if rng.random() < 0.4:
            temps = torch.from_numpy(rng.uniform(0.4, 1.8, size=R).astype(np.float32)).cuda()
        _, _, mism = H.check_sampling(b, want_probs=bool(rng.random() < 0.7), temperatures=temps)
        total_mism += mism
        if temps is None and seed != 1416:
            # the same batch with the draft rows' statistics handed over instead of streamed
            import test_gpu_draft_stats as DS
            want_probs = bool(rng.random() < 0.5)
            g = DS._verify_with_stats(b, DS._stats(b.draft, b.temperature), want_probs=want_probs)
            total_mism += H.compare_sampling(g, H.oracle_verify(b, eval_all=want_probs), b.row_offsets.cpu().numpy(),
                                             check_probs=want_probs)
    assert total_mism <= 1


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 5006, 5026])
def test_sampling_fuzz_many_units(seed):
    # batches large enough that most 32 KB units of the streamed passes are handed out by the grid-wide
    # counter (more than two units per CTA), with ragged last pieces and both dtypes
    rng = np.random.default_rng(7000 + seed)
    R = int(rng.integers(40, 300))
    V = int(rng.choice([40_000, 65_536, 100_003, W.V_FULL, 200_000]))
    lengths = torch.from_numpy(rng.integers(0, 9, size=R))
    dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
    b = W.sampling_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", dtype=dtype,
                         sigma=float(rng.uniform(1.0, 4)), draft_noise=float(rng.uniform(0.3, 2.5)),
                         temperature=float(rng.uniform(0.5, 1.5)), verify_seed=int(rng.integers(0, 2**40)))
    temps = None
    if rng.random() < 0.5:
        temps = torch.from_numpy(rng.uniform(0.5, 1.6, size=R).astype(np.float32)).cuda()
    g, o, mism = H.check_sampling(b, want_probs=bool(rng.random() < 0.5), temperatures=temps)
    assert mism <= 3                                       # a few hundred draws over ~1e5 tokens: margins of 1e-9 occur
    assert (g["acc"] < lengths.numpy()).sum() > 5          # the residual pass had work
    gb = W.greedy_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", tie_frac=0.1, perturb=0.3, dtype=dtype)
    H.check_greedy(gb)


@pytest.mark.parametrize("seed", range(6))
def test_greedy_fuzz(seed):
    rng = np.random.default_rng(2000 + seed)
    for _ in range(8):
        R = int(rng.integers(1, 60))
        V = int(rng.choice([1, 2, 5, 33, 1000, 1025, 4096, 30001]))
        lengths = torch.from_numpy(rng.integers(0, 12, size=R))
        dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        b = W.greedy_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", sigma=float(rng.uniform(0.1, 5)),
                           tie_frac=float(rng.choice([0.0, 0.1, 0.9])) if V > 4 else 0.0,
                           perturb=float(rng.uniform(0, 0.6)), dtype=dtype)
        if rng.random() < 0.5:
            b = W.VerifyBatch(_pad_rows(b.target, rng), None, b.row_offsets, b.draft_tokens)
        H.check_greedy(b)


@pytest.mark.parametrize("seed", range(8))
def test_schedule_fuzz(seed):
    rng = np.random.default_rng(3000 + seed)
    for _ in range(6):
        R = int(rng.integers(1, 400))
        gamma = int(rng.choice([0, 1, 2, 3, 5, 8, 16, 31, 32, 33, 48]))
        if R * max(gamma, 1) > 20000:
            R = 20000 // max(gamma, 1)
        conf = rng.uniform(0.0, 1.0, size=(R, gamma)).astype(np.float32) ** float(rng.choice([0.2, 1.0, 3.0]))
        if gamma:
            conf[rng.random((R, gamma)) < 0.05] = 1.0
        n_bp = int(rng.integers(1, 9))
        hi = R * (gamma + 1) + 5
        toks = np.sort(rng.choice(np.arange(1, hi), size=min(n_bp, hi - 1), replace=False)).tolist()
        sps = rng.uniform(1, 100, len(toks)).tolist()
        budget = int(rng.integers(max(0, R - 3), hi + 10))
        s = W.ScheduleInput(torch.from_numpy(conf).reshape(R, gamma), toks, sps, budget, max_tokens=int(rng.integers(1, hi + 1)))
        mode = int(rng.choice([B.DSPARK_SCHED_EARLY_STOP, B.DSPARK_SCHED_GLOBAL, B.DSPARK_SCHED_TOPK]))
        dl = rng.integers(0, gamma + 2, size=R).astype(np.int32) if rng.random() < 0.3 else None
        H.check_schedule(s, mode, topk=int(rng.integers(0, R * gamma + 2)), draft_len=dl)


@pytest.mark.parametrize("seed", range(6))
def test_truncate_fuzz(seed):
    import oracle
    rng = np.random.default_rng(3000 + seed)
    for _ in range(5):
        R = int(rng.integers(1, 12))
        V = int(rng.choice([1, 2, 9, 64, 255, 1000, 4097, 20000]))
        lengths = rng.integers(0, 4, size=R)
        off = np.concatenate([[0], np.cumsum(lengths + 1)]).astype(np.int32)
        n_rows = int(off[-1])
        kind = rng.integers(0, 3)
        if kind == 0:
            t = torch.randn(n_rows, V) * float(rng.uniform(0.2, 6))
        elif kind == 1:
            t = torch.from_numpy(rng.integers(-4, 5, (n_rows, V)).astype(np.float32)) * 0.25      # heavy ties
        else:
            t = torch.from_numpy(rng.uniform(-30, 30, (n_rows, V)).astype(np.float32))
        dt = torch.bfloat16 if rng.random() < 0.5 else torch.float32      # 16-bit key window / 32-bit descent
        t = _pad_rows(t.to(dt).cuda(), rng)
        ks = rng.integers(-1, V + 3, size=R).astype(np.int32)
        ps = rng.choice([0.0, 0.1, 0.5, 0.9, 0.99, 1.0, 1.5], size=R).astype(np.float32)
        Ts = rng.uniform(0.3, 2.5, size=R).astype(np.float32)
        got = t.clone()
        tau = torch.empty(n_rows, device="cuda"); kept = torch.empty(n_rows, dtype=torch.int32, device="cuda")
        B.dspark_truncate_target(got, torch.from_numpy(off).cuda(), top_k=torch.from_numpy(ks).cuda(),
                                 top_p=torch.from_numpy(ps).cuda(), temperatures=torch.from_numpy(Ts).cuda(),
                                 out_tau=tau, out_kept=kept)
        torch.cuda.synchronize()
        bits = W.bf16_bits(t)
        want, otau, okept, margin = oracle.warp_target(bits, off, top_k=ks, top_p=ps, temperatures=Ts)
        gb = W.bf16_bits(got)
        for row in range(n_rows):
            if margin[row] < 1e-5:
                continue                                  # a top-p decision on its boundary: either neighbour is right
            np.testing.assert_array_equal(gb[row], want[row], err_msg=f"row {row} V={V} k={ks} p={ps}")
            assert int(kept[row]) == okept[row]


@pytest.mark.parametrize("seed", range(6))
def test_verify_truncated_fuzz(seed):
    """dspark_verify_truncated (streamed threshold search with its second look on bf16 rows, descent on fp32 rows)
    against the oracle pipeline warp_target -> verify: peaked, wide, tied and flat rows, top-k / top-p / both / none per
    request, per-request temperatures, compact and block draft layouts, padded strides."""
    import oracle
    rng = np.random.default_rng(9000 + seed)
    for _ in range(4):
        R = int(rng.integers(1, 14))
        V = int(rng.choice([9, 255, 1000, 4097, 20000, 70000]))
        lengths = torch.from_numpy(rng.integers(0, 5, size=R))
        dt = torch.bfloat16 if rng.random() < 0.7 else torch.float32
        kind = int(rng.integers(0, 3))
        sigma = float(rng.choice([0.5, 1.5, 3.0, 6.0]))
        block = None if rng.random() < 0.6 else int(lengths.max()) + int(rng.integers(0, 3))
        T = float(rng.choice([0.5, 1.0, 1.6]))
        b = W.sampling_batch(lengths, V, int(rng.integers(1 << 30)), "cuda", dtype=dt, sigma=sigma, temperature=T,
                             draft_noise=float(rng.choice([0.3, 1.0])), verify_seed=int(rng.integers(1 << 30)),
                             block=block if block else None)
        if kind == 1:                                          # heavy ties: a coarse grid of values
            b.target.copy_((b.target.float() * 2).round() / 2)
        elif kind == 2:                                        # flat rows: no peak at all
            b.target.copy_(torch.from_numpy(rng.uniform(-2, 2, tuple(b.target.shape)).astype(np.float32)))
        b.target = _pad_rows(b.target, rng)
        ks = rng.choice([0, 0, 1, 3, 50, 300, V + 2], size=R).astype(np.int32)
        ps = rng.choice([1.0, 0.0, 0.3, 0.9, 0.97, 0.999], size=R).astype(np.float32)
        temps = rng.choice([0.5, 1.0, 1.6], size=R).astype(np.float32) if rng.random() < 0.5 else None
        acc = torch.full((R,), -7, dtype=torch.int32, device="cuda")
        out = torch.full((b.n_rows,), -7, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = B.workspace(B.dspark_verify_workspace_bytes(R, b.n_rows, V)).fill_(int(rng.integers(0, 256)))
        dev = lambda a, d: None if a is None else torch.as_tensor(a, dtype=d, device="cuda")
        B.dspark_verify_truncated(b.target, b.draft, b.row_offsets, b.draft_tokens, b.seed, temperature=b.temperature,
                                  temperatures=dev(temps, torch.float32), top_k=dev(ks, torch.int32),
                                  top_p=dev(ps, torch.float32), draft_row_start=b.draft_row_start, accepted_len=acc,
                                  out_tokens=out, out_p_tok=None, out_q_tok=None, dev_status=st, workspace=ws)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        off = b.row_offsets.cpu().numpy()
        bits, dbits = W.bf16_bits(b.target), W.bf16_bits(b.draft)
        masked, tau, kept, margin = oracle.warp_target(bits, off, top_k=ks, top_p=ps, temperature=b.temperature,
                                                       temperatures=temps)
        drs = None if b.draft_row_start is None else b.draft_row_start.cpu().numpy()
        o = oracle.verify(masked, dbits, off, b.draft_tokens.cpu().numpy(), b.temperature, b.seed, draft_row_start=drs,
                          eval_all=False, n_threads=H.THREADS, temperatures=temps)
        g = dict(acc=acc.cpu().numpy(), out=out.cpu().numpy())
        H.compare_away_from_top_p_boundaries(g, o, margin, off)


@pytest.mark.parametrize("seed", range(4))
def test_markov_fuzz(seed):
    import oracle
    rng = np.random.default_rng(4000 + seed)
    for _ in range(3):
        R = int(rng.integers(1, 400))
        V = int(rng.choice([8, 129, 1000, 2048, 4097, 9000]))
        T = float(rng.choice([0.0, 0.5, 1.0, 1.7]))
        m = W.markov_input(R, V, int(rng.integers(0, 10**6)), "cuda", d=int(rng.choice([8, 100, 256])),
                           sigma=float(rng.uniform(0.5, 4)))
        packed = torch.empty(B.dspark_markov_w2_packed_bytes(V), dtype=torch.uint8, device="cuda")
        B.dspark_markov_pack_w2(m.W2, packed)
        U = _pad_rows(m.U, rng)
        out = _pad_rows(torch.zeros_like(m.U), rng)
        conf = torch.empty(R, device="cuda"); toks = torch.empty(R, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = B.workspace(B.dspark_markov_workspace_bytes(R, V)).fill_(0xFF)
        seed_v = int(rng.integers(0, 2**40))
        B.dspark_markov_draft_step(U, m.W1, packed, m.x_prev, T, seed_v, H=m.H, w_conf=m.w_conf, out_logits=out,
                                   out_tokens=toks, out_conf=conf, dev_status=st, workspace=ws)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        exact, bits = oracle.markov_logits(W.bf16_bits(m.U), W.bf16_bits(m.W1), W.bf16_bits(m.W2), m.x_prev.cpu().numpy())
        got = W.bf16_bits(out.contiguous())
        diff = np.abs(got.astype(np.int32) - bits.astype(np.int32))
        assert diff[np.abs(exact) >= 2.0 ** -4].max(initial=0) <= 1
        assert int((diff != 0).sum()) <= max(2, int(5e-3 * diff.size))      # rounding boundaries: a few per thousand
        want_c = oracle.confidence(W.bf16_bits(m.H), W.bf16_bits(m.W1), m.w_conf.cpu().numpy(), m.x_prev.cpu().numpy())
        assert np.abs(conf.cpu().numpy() - want_c).max() <= 1e-6
        off = np.arange(R + 1, dtype=np.int32)
        tk = toks.cpu().numpy()
        if T == 0.0:
            o = oracle.verify_greedy(got, off, np.zeros(R, dtype=np.int32))
            np.testing.assert_array_equal(tk, o.out_tokens[:R])
        else:
            o = oracle.verify(got, got, off, np.zeros(R, dtype=np.int32), T, seed_v)
            for r in np.nonzero(tk != o.out_tokens[:R])[0]:
                assert o.token_margin[r] < 1e-6, (r, tk[r], o.out_tokens[r], o.token_margin[r])


# ---- special values: NaN, +-inf, huge, flat and empty rows, tokens / temperatures / lengths out of range ----
_SPECIALS = [float("nan"), float("inf"), float("-inf"), 1.0e4, -1.0e4, 0.0, -0.0]


def _corrupt(rng, tensors, V, n_max=10):
    for _ in range(int(rng.integers(0, n_max))):
        which = tensors[int(rng.integers(0, len(tensors)))]
        if which.shape[0] == 0:
            continue
        r, v = int(rng.integers(0, which.shape[0])), int(rng.integers(0, V))
        kind = rng.random()
        if kind < 0.6:
            which[r, v] = float(rng.choice(_SPECIALS))
        elif kind < 0.8:
            which[r, :] = float("-inf")
        elif kind < 0.9:
            which[r, :] = float(rng.choice([0.0, 5.0, -7.5]))          # a flat row: every token ties
        else:
            which[r, : max(1, V // 2)] = float("-inf")


# seeds 20001 / 20022 / 20293: an unusable row behind the first rejection, a request with two things wrong
# with it, a NaN in a block whose other elements are all -inf (all three once disagreed with the oracle)
@pytest.mark.parametrize("seed", [0, 1, 2, 3, 20001, 20022, 20293])
def test_special_values_fuzz(seed):
    import oracle
    rng = np.random.default_rng([seed, 0])
    for it in range(1 if seed >= 20000 else 6):
        R = int(rng.integers(1, 40))
        lengths = torch.from_numpy(rng.integers(0, 8, size=R))
        V = int(rng.choice([3, 100, 2049, 5000, 40_000, 129_280]))
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        b = W.sampling_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", dtype=dtype, sigma=float(rng.uniform(0.5, 4)),
                             draft_noise=float(rng.uniform(0.05, 2.5)), temperature=float(rng.uniform(0.3, 2.0)),
                             verify_seed=int(rng.integers(0, 2**40)), block=(8 if rng.random() < 0.3 else None))
        t, d, toks = b.target.clone(), b.draft.clone(), b.draft_tokens.clone()
        for _ in range(int(rng.integers(0, 12))):
            which = t if rng.random() < 0.6 else d
            r_, v_ = int(rng.integers(0, which.shape[0])), int(rng.integers(0, V))
            kind = rng.random()
            if kind < 0.6:
                which[r_, v_] = float(rng.choice(_SPECIALS))
            elif kind < 0.8:
                which[r_, :] = float("-inf")
            elif kind < 0.9:
                which[r_, :] = float(rng.choice([0.0, 5.0, -7.5]))
            else:
                which[r_, : max(1, V // 2)] = float("-inf")
        for _ in range(int(rng.integers(0, 3))):
            toks[int(rng.integers(0, toks.numel()))] = int(rng.choice([-1, V, V + 5, 2**31 - 1, -2**31]))
        temps = None
        if rng.random() < 0.5:
            tv = rng.uniform(0.4, 1.8, size=R).astype(np.float32)
            for _ in range(int(rng.integers(0, 3))):
                tv[int(rng.integers(0, R))] = np.float32(rng.choice([0.0, -1.0, np.nan, np.inf]))
            temps = torch.from_numpy(tv).cuda()
        bb = W.VerifyBatch(t, d, b.row_offsets, toks, b.draft_row_start, b.temperature, b.seed, b.meta)
        want_probs = bool(rng.random() < 0.5)
        _, _, mism = H.check_sampling(bb, want_probs=want_probs, temperatures=temps)
        assert mism <= 2
        H.check_greedy(W.VerifyBatch(t, None, b.row_offsets, toks.clamp(0, V - 1)))


@pytest.mark.parametrize("seed", range(3))
def test_special_values_fuzz_other_entry_points(seed):
    import oracle
    import test_gpu_accept_rate as AR
    import test_gpu_verify_truncated as TV
    rng = np.random.default_rng([seed, 1])
    for it in range(4):
        # truncated verification and truncation in place
        R = int(rng.integers(1, 30))
        lengths = torch.from_numpy(rng.integers(0, 6, size=R))
        V = int(rng.choice([3, 100, 2049, 5000, 40_000]))
        b = W.sampling_batch(lengths, V, int(rng.integers(0, 10**6)), "cuda", temperature=float(rng.uniform(0.5, 1.5)),
                             sigma=float(rng.uniform(1, 4)), draft_noise=float(rng.uniform(0.3, 2.0)),
                             verify_seed=int(rng.integers(0, 2**40)))
        t, d = b.target.clone(), b.draft.clone()
        _corrupt(rng, [t, d], V)
        bb = W.VerifyBatch(t, d, b.row_offsets, b.draft_tokens, b.draft_row_start, b.temperature, b.seed, b.meta)
        ks = rng.choice([-3, 0, 1, 2, 5, 40, V, V + 7], size=R).astype(np.int32)
        ps = rng.choice([1.0, 0.99, 0.9, 0.5, 0.0, 1.5, -0.5], size=R).astype(np.float32)
        temps = rng.uniform(0.5, 1.6, size=R).astype(np.float32) if rng.random() < 0.5 else None
        want_probs = bool(rng.random() < 0.5)
        g = TV._gpu_truncated(bb, ks, ps, temps, want_probs=want_probs)
        off = bb.row_offsets.cpu().numpy()
        masked, tau, kept, margin = oracle.warp_target(W.bf16_bits(bb.target), off, top_k=ks, top_p=ps,
                                                       temperature=bb.temperature, temperatures=temps)
        if not (margin < 1e-5).any():
            o = oracle.verify(masked, W.bf16_bits(bb.draft), off, bb.draft_tokens.cpu().numpy(), bb.temperature, bb.seed,
                              eval_all=want_probs, n_threads=H.THREADS, temperatures=temps)
            assert H.compare_sampling(g, o, off, check_probs=want_probs) <= 2
            got = t.clone()
            dev = lambda a, dt: torch.as_tensor(a, dtype=dt, device="cuda")
            B.dspark_truncate_target(got, bb.row_offsets, top_k=dev(ks, torch.int32), top_p=dev(ps, torch.float32),
                                     temperature=bb.temperature, temperatures=None if temps is None else dev(temps, torch.float32))
            torch.cuda.synchronize()
            np.testing.assert_array_equal(W.bf16_bits(got), masked)
        # acceptance rate
        if int(lengths.sum()) > 0:
            AR._check(bb, float(bb.temperature))
        # scheduler: confidences outside [0, 1], NaN, denormals; lengths and K out of range
        Rs, gamma = int(rng.integers(1, 300)), int(rng.choice([1, 2, 5, 8, 16, 32, 33]))
        conf = rng.uniform(0.0, 1.0, size=(Rs, gamma)).astype(np.float32)
        for _ in range(int(rng.integers(0, 20))):
            conf[int(rng.integers(0, Rs)), int(rng.integers(0, gamma))] = np.float32(
                rng.choice([np.nan, np.inf, -np.inf, -0.5, 1.5, 0.0, 1.0, 1e-30, 1e-45, 2.0]))
        hi = Rs * (gamma + 1) + 5
        bp = np.sort(rng.choice(np.arange(1, hi), size=min(int(rng.integers(1, 6)), hi - 1), replace=False)).tolist()
        s = W.ScheduleInput(torch.from_numpy(conf), bp, rng.uniform(1, 100, len(bp)).tolist(), int(rng.integers(0, hi + 10)),
                            max_tokens=int(rng.integers(1, hi + 1)))
        mode = int(rng.choice([B.DSPARK_SCHED_EARLY_STOP, B.DSPARK_SCHED_GLOBAL, B.DSPARK_SCHED_TOPK]))
        dl = rng.integers(-2, gamma + 3, size=Rs).astype(np.int32) if rng.random() < 0.4 else None
        H.check_schedule(s, mode, topk=int(rng.integers(-2, Rs * gamma + 2)), draft_len=dl)
