"""Seeded synthetic inputs shaped like the paper's serving workloads.

This module only draws random tensors (torch generators).  It holds none of the
method's arithmetic and imports neither the CUDA binding nor the CPU oracle, so
both sides can be fed the very same tensors.  The paper evaluates on public
benchmark suites and live traffic; these tensors stand in for them with the same
shapes and regimes (vocabulary 129 280, draft blocks of 4..32, 64..1024
concurrent requests, per-position acceptance 0.5..0.95).

Each ``config_N`` follows one of the five benchmark configurations; ``scale_*``
arguments shrink a configuration so the CPU oracle finishes in seconds while
keeping its structure (ragged lengths, tie injection, boosts, noise).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import torch

V_FULL = 129_280

# Engine throughput profiles (steps/s at a number of batch tokens).  The paper prints no
# capacity curve beyond the three toy values of its appendix, so these are invented here.
PROFILE_P1 = ([1, 4, 6, 8, 10, 12, 14, 16], [100.0, 99.0, 96.0, 90.0, 80.0, 66.0, 50.0, 36.0])
PROFILE_P3 = ([1, 128, 256, 384, 512, 640, 768, 1024], [120.0, 118.0, 112.0, 104.0, 92.0, 84.0, 70.0, 50.0])
PROFILE_P5 = ([1, 512, 1024, 1536, 2048, 2560, 3072, 4096], [60.0, 56.0, 48.0, 38.0, 31.0, 24.0, 21.0, 14.0])


@dataclass
class VerifyBatch:
    """One ragged verification batch (flat target rows + per-request offsets)."""
    target: torch.Tensor                  # [n_rows, V] fp32 or bf16
    draft: Optional[torch.Tensor]         # [n_draft_rows, V] same dtype, or None (greedy)
    row_offsets: torch.Tensor             # [R+1] int32; request r owns rows [off[r], off[r+1])
    draft_tokens: torch.Tensor            # [n_rows] int32; entry off[r]+j for j < l_r
    draft_row_start: Optional[torch.Tensor] = None   # [R] int64 or None (compact layout)
    temperature: float = 1.0
    seed: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def R(self) -> int:
        return self.row_offsets.numel() - 1

    @property
    def n_rows(self) -> int:
        return self.target.shape[0]

    @property
    def V(self) -> int:
        return self.target.shape[1]


@dataclass
class ScheduleInput:
    conf: torch.Tensor                    # [R, gamma] fp32
    bp_tokens: list
    bp_sps: list
    budget_tokens: int
    max_tokens: int


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def offsets_from_lengths(lengths: torch.Tensor) -> torch.Tensor:
    """row_offsets[R+1] for verify lengths l_r (each request owns l_r + 1 target rows)."""
    off = torch.zeros(lengths.numel() + 1, dtype=torch.int32, device=lengths.device)
    off[1:] = torch.cumsum(lengths.to(torch.int64) + 1, 0).to(torch.int32)
    return off


def _rows_of_requests(lengths: torch.Tensor):
    """For flat target rows: owning request and position inside it."""
    R = lengths.numel()
    counts = lengths.to(torch.int64) + 1
    req = torch.repeat_interleave(torch.arange(R, device=lengths.device), counts)
    start = torch.cumsum(counts, 0) - counts
    pos = torch.arange(int(counts.sum()), device=lengths.device) - start[req]
    return req, pos


def _boosted_logits(n_rows, V, sigma, g, device, n_boost=64, beta=14.0, zipf=1.1, chunk=256):
    """fp32 rows sigma*N(0,1) plus Zipf-ranked peaks: n_boost random ids per row get
    beta - zipf*ln(rank) added (ids are drawn with replacement; a repeated id gets both)."""
    out = torch.empty(n_rows, V, dtype=torch.float32, device=device)
    k = min(n_boost, V)
    boost = beta - zipf * torch.log(torch.arange(1, k + 1, device=device, dtype=torch.float32))
    for s in range(0, n_rows, chunk):
        e = min(n_rows, s + chunk)
        blk = torch.randn(e - s, V, generator=g, device=device) * sigma
        ids = torch.randint(0, V, (e - s, k), generator=g, device=device)
        blk.scatter_add_(1, ids, boost.expand(e - s, k).contiguous())
        out[s:e] = blk
    return out


def _sample_tokens(logits_f32_rows, T, g, chunk=256):
    """One token per row from softmax(row / T) by the Gumbel-max trick (input generation only)."""
    n, V = logits_f32_rows.shape
    out = torch.empty(n, dtype=torch.int32, device=logits_f32_rows.device)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        u = torch.rand(e - s, V, generator=g, device=logits_f32_rows.device).clamp_(1e-12, 1.0)
        gum = -torch.log((-torch.log(u)).clamp_min_(1e-20))
        out[s:e] = torch.argmax(logits_f32_rows[s:e].float() / T + gum, dim=1).to(torch.int32)
    return out


def sampling_batch(lengths: torch.Tensor, V: int, seed: int, device, *, dtype=torch.bfloat16,
                   sigma=3.0, draft_noise=1.0, temperature=1.0, verify_seed=None,
                   block: Optional[int] = None) -> VerifyBatch:
    """Target rows = boosted noise; draft rows = target + N(0, draft_noise^2); draft tokens ~
    softmax(draft / T).  ``block`` given: draft rows are laid out [R, block, V] (the drafter's
    whole block) and ``draft_row_start[r] = r * block``; otherwise the compact ragged layout."""
    g = _gen(seed, device)
    lengths = lengths.to(device=device, dtype=torch.int32)
    R = lengths.numel()
    off = offsets_from_lengths(lengths)
    n_rows = int(off[-1])
    req, pos = _rows_of_requests(lengths)
    target = _boosted_logits(n_rows, V, sigma, g, device).to(dtype)
    is_draft_pos = pos < lengths[req]
    t_rows = torch.nonzero(is_draft_pos).squeeze(1)          # target rows that have a draft row
    n_draft = t_rows.numel()
    if block is None:
        draft = torch.empty(max(n_draft, 1), V, dtype=dtype, device=device)
        d_rows = torch.arange(n_draft, device=device)
        drs = None
    else:
        draft = torch.zeros(R * block, V, dtype=dtype, device=device)
        d_rows = req[t_rows] * block + pos[t_rows]
        drs = (torch.arange(R, device=device, dtype=torch.int64) * block)
    tokens = torch.zeros(n_rows, dtype=torch.int32, device=device)
    chunk = 256
    for s in range(0, n_draft, chunk):
        e = min(n_draft, s + chunk)
        noise = torch.randn(e - s, V, generator=g, device=device) * draft_noise
        drow = (target[t_rows[s:e]].float() + noise).to(dtype)
        draft[d_rows[s:e]] = drow
        tokens[t_rows[s:e]] = _sample_tokens(drow, temperature, g)
    return VerifyBatch(target, draft, off, tokens, drs, temperature,
                       seed if verify_seed is None else verify_seed,
                       {"lengths": lengths, "n_draft": n_draft})


def greedy_batch(lengths: torch.Tensor, V: int, seed: int, device, *, sigma=4.0, boost=None,
                 tie_frac=0.0, match_prob=None, perturb=None, dtype=torch.float32) -> VerifyBatch:
    """fp32 target rows sigma*N(0,1) (optionally one id per row boosted); ties injected in a
    fraction of rows (row max copied to 1..3 other random ids); draft token = row argmax with
    probability match_prob[j] (or 1 - perturb), otherwise a different random id."""
    g = _gen(seed, device)
    lengths = lengths.to(device=device, dtype=torch.int32)
    off = offsets_from_lengths(lengths)
    n_rows = int(off[-1])
    req, pos = _rows_of_requests(lengths)
    target = torch.empty(n_rows, V, dtype=torch.float32, device=device)
    for s in range(0, n_rows, 512):
        e = min(n_rows, s + 512)
        target[s:e] = torch.randn(e - s, V, generator=g, device=device) * sigma
    if boost is not None:
        ids = torch.randint(0, V, (n_rows,), generator=g, device=device)
        target[torch.arange(n_rows, device=device), ids] += boost
    if tie_frac > 0:
        n_tie = max(1, int(round(tie_frac * n_rows)))
        rows = torch.randperm(n_rows, generator=g, device=device)[:n_tie]
        mx = target[rows].max(dim=1).values
        ncopies = torch.randint(1, 4, (n_tie,), generator=g, device=device)
        ids = torch.randint(0, V, (n_tie, 3), generator=g, device=device)
        for c in range(3):
            sel = ncopies > c
            target[rows[sel], ids[sel, c]] = mx[sel]
    target = target.to(dtype)
    am = torch.argmax(target.float(), dim=1).to(torch.int32)    # draft construction only
    u = torch.rand(n_rows, generator=g, device=device)
    if match_prob is not None:
        keep = u < torch.as_tensor(match_prob, device=device, dtype=torch.float32)[pos.clamp_max(len(match_prob) - 1)]
    else:
        keep = u >= (perturb or 0.0)
    other = (am.to(torch.int64) + torch.randint(1, max(V, 2), (n_rows,), generator=g, device=device)) % V
    tokens = torch.where(keep, am, other.to(torch.int32))
    tokens[pos == lengths[req]] = 0                             # bonus-row entries are ignored
    return VerifyBatch(target, None, off, tokens.contiguous(), None, 1.0, seed, {"lengths": lengths})


# --------------------------------------------------------------------------- configs ----
def config_1(device="cpu"):
    """Tiny greedy: 4 requests, V = 1024, block 4, budget 16, profile P1; seed 0."""
    g = _gen(0, device)
    conf = 0.5 + 0.5 * torch.rand(4, 4, generator=g, device=device)
    sched = ScheduleInput(conf.float(), *PROFILE_P1, budget_tokens=16, max_tokens=16)
    batch = greedy_batch(torch.full((4,), 4), 1024, 0, device, sigma=3.0, boost=8.0, perturb=0.3)
    return sched, batch


def config_2(device="cpu", R=64, V=V_FULL):
    """Sampling, moderate batch: ragged k_r ~ U{1..8}, bf16, T = 1, Philox seed 1."""
    g = _gen(1, device)
    lengths = torch.randint(1, 9, (R,), generator=g, device=device)
    return sampling_batch(lengths, V, 1001, device, temperature=1.0, draft_noise=1.0, verify_seed=1)


def config_3_schedule(device="cpu", R=256, gamma=16, budget=1024):
    """Confidence-scheduled: c_{r,i} = sigmoid(N(2.0 - 0.25 i, 1)), i = 1..gamma; profile P3."""
    g = _gen(2, device)
    i = torch.arange(1, gamma + 1, device=device, dtype=torch.float32)
    conf = torch.sigmoid(torch.randn(R, gamma, generator=g, device=device) + (2.0 - 0.25 * i))
    return ScheduleInput(conf.float().contiguous(), *PROFILE_P3, budget_tokens=budget, max_tokens=budget)


def config_3_batch(lengths, device="cpu", V=V_FULL, block=16, seed=1002):
    """bf16 sampling verification of the scheduled ragged blocks (drafter block layout)."""
    return sampling_batch(lengths, V, seed, device, temperature=1.0, draft_noise=1.0,
                          verify_seed=2, block=block)


def config_4(device="cpu", R=1024, V=V_FULL):
    """Large batch greedy: k_r ~ U{0..8}, fp32 4*N(0,1), ties in 1 % of rows, match prob 0.85^(j+1)."""
    g = _gen(3, device)
    lengths = torch.randint(0, 9, (R,), generator=g, device=device)
    mp = [0.85 ** (j + 1) for j in range(8)]
    return greedy_batch(lengths, V, 1003, device, sigma=4.0, tie_frac=0.01, match_prob=mp)


def config_5_schedule(device="cpu", R=512, gamma=32, budget=4096):
    """Long-block stress: c_{r,i} = 0.95^i * U(0.8, 1); profile P5 (convex kink)."""
    g = _gen(4, device)
    i = torch.arange(1, gamma + 1, device=device, dtype=torch.float32)
    conf = (0.95 ** i) * (0.8 + 0.2 * torch.rand(R, gamma, generator=g, device=device))
    return ScheduleInput(conf.float().contiguous(), *PROFILE_P5, budget_tokens=budget, max_tokens=budget)


def config_5_batch(lengths, device="cpu", V=V_FULL, block=32, seed=1004):
    """bf16 sampling at T = 0.7 with draft = target + N(0, 2^2): high rejection rate."""
    return sampling_batch(lengths, V, seed, device, temperature=0.7, draft_noise=2.0,
                          verify_seed=4, block=block)



@dataclass
class MarkovInput:
    """Inputs of one Markov-head draft step (Section 3.1): base logits of the block position, the
    two low-rank factors, previous tokens, hidden states and confidence weights."""
    U: torch.Tensor        # bf16 [R, V]
    W1: torch.Tensor       # bf16 [V, 256]
    W2: torch.Tensor       # bf16 [256, V]
    x_prev: torch.Tensor   # int32 [R]
    H: torch.Tensor        # bf16 [R, d]
    w_conf: torch.Tensor   # fp32 [d + 256]


def markov_input(R: int, V: int, seed: int, device, d: int = 1024, sigma: float = 3.0, chunk: int = 8192) -> MarkovInput:
    """Seeded synthetic head: logit-like base scores (normal, std sigma), embedding rows of std 0.5 and
    output factors of std 0.12 (a bias of about unit scale after 256 terms), unit hidden states."""
    g = _gen(seed, device)
    U = (torch.randn(R, V, generator=g, device=device) * sigma).to(torch.bfloat16)
    W1 = torch.empty(V, 256, dtype=torch.bfloat16, device=device)
    for lo in range(0, V, chunk):
        hi = min(V, lo + chunk)
        W1[lo:hi] = (torch.randn(hi - lo, 256, generator=g, device=device) * 0.5).to(torch.bfloat16)
    W2 = (torch.randn(256, V, generator=g, device=device) * 0.12).to(torch.bfloat16)
    x_prev = torch.randint(0, V, (R,), generator=g, device=device, dtype=torch.int32)
    H = torch.randn(R, d, generator=g, device=device).to(torch.bfloat16)
    w_conf = torch.randn(d + 256, generator=g, device=device) / float(d + 256) ** 0.5
    return MarkovInput(U, W1, W2, x_prev, H, w_conf)



def sts_input(N: int, gamma: int, seed: int, device, overconfidence: float = 2.0, partial: bool = True):
    """Held-out blocks for the calibration of the confidence head: true conditional acceptance
    probabilities sigmoid(z), z ~ N(1.2 - 0.05 k, 1); the head reports sigmoid(overconfidence * z); a
    block is verified up to a random length (partial) and accepted up to the first failed draw.
    Returns (conf [N, gamma] fp32, accepted_len [N] int32, verified_len [N] int32)."""
    g = _gen(seed, device)
    k = torch.arange(gamma, device=device, dtype=torch.float32)
    z = torch.randn(N, gamma, generator=g, device=device) + (1.2 - 0.05 * k)
    ok = torch.rand(N, gamma, generator=g, device=device) < torch.sigmoid(z)
    if partial:
        ver = torch.randint(1, gamma + 1, (N,), generator=g, device=device, dtype=torch.int32)
    else:
        ver = torch.full((N,), gamma, device=device, dtype=torch.int32)
    ok = ok & (k[None, :] < ver[:, None])
    fail = (~ok).to(torch.int32)
    acc = torch.where(fail.any(1), fail.argmax(1).to(torch.int32), torch.full((N,), gamma, device=device, dtype=torch.int32))
    acc = torch.minimum(acc, ver)
    conf = torch.sigmoid(overconfidence * z).to(torch.float32)
    return conf.contiguous(), acc.contiguous(), ver.contiguous()


def bf16_bits(t: torch.Tensor):
    """Host numpy view of a tensor for the oracle: fp32 as is, bf16 as raw uint16 patterns."""
    import numpy as np
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
