"""ctypes access to the CPU oracle (``dspark_oracle.c``) -- test infrastructure only.

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs
may import this package.  It never imports the CUDA package and the CUDA
package never imports it.  Arrays are numpy; bf16 logits are passed as their
raw 16-bit patterns (``uint16``).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dspark_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

F32, BF16 = 0, 1
MODE_EARLY_STOP, MODE_GLOBAL, MODE_TOPK = 0, 1, 2
ST_BAD_OFFSETS, ST_BAD_TOKEN, ST_BAD_ROW = 1, 2, 4
ST_CONF_CLAMPED, ST_BUDGET_LT_R, ST_ALL_NEG_INF = 16, 32, 64
ST_BAD_TEMPERATURE = 128


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no contraction, no fast-math) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-Wall", "-shared", "-fPIC",
             "-pthread", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


class _SchedInfo(C.Structure):
    _fields_ = [("B", C.c_int32), ("n_admitted", C.c_int32), ("status", C.c_int32),
                ("n_candidates", C.c_int32), ("tau", C.c_double), ("theta", C.c_double)]


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def _p(a, ctype=C.c_void_p):
    return None if a is None else a.ctypes.data_as(ctype)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"logits must be float32 or uint16 (bf16 bits), got {a.dtype}")


def philox4x32_10(ctr, key) -> np.ndarray:
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return np.array(list(o), dtype=np.uint32)


def uniforms(seed: int, r: int, j: int):
    ua, ur = C.c_float(), C.c_float()
    lib().orc_uniforms(C.c_uint64(seed), C.c_uint32(r), C.c_uint32(j), C.byref(ua), C.byref(ur))
    return ua.value, ur.value


def sps_table(bp_tokens, bp_sps, max_tokens: int) -> np.ndarray:
    bt = np.ascontiguousarray(bp_tokens, dtype=np.int32)
    bs = np.ascontiguousarray(bp_sps, dtype=np.float64)
    out = np.empty(max_tokens + 1, dtype=np.float64)
    rc = lib().orc_sps_table(_p(bt), _p(bs), C.c_int(len(bt)), C.c_int(max_tokens), _p(out))
    if rc != 0:
        raise ValueError("invalid breakpoints")
    return out


@dataclass
class ScheduleResult:
    lengths: np.ndarray
    survival: np.ndarray
    expected_len: np.ndarray
    B: int
    n_admitted: int
    n_candidates: int
    status: int
    tau: float
    theta: float
    theta_path: np.ndarray


def schedule(conf, table, budget_tokens: int, mode: int = MODE_EARLY_STOP, topk_K: int = 0,
             draft_len=None) -> ScheduleResult:
    conf = np.ascontiguousarray(conf, dtype=np.float32)
    R, gamma = conf.shape
    table = np.ascontiguousarray(table, dtype=np.float64)
    dl = None if draft_len is None else np.ascontiguousarray(draft_len, dtype=np.int32)
    out_len = np.zeros(R, dtype=np.int32)
    surv = np.zeros((R, max(gamma, 1)), dtype=np.float32)[:, :gamma].copy()
    exp_len = np.zeros(R, dtype=np.float32)
    path = np.full(R * gamma + 1, np.nan, dtype=np.float64)
    info = _SchedInfo()
    rc = lib().orc_schedule(_p(conf), _p(dl), C.c_int(R), C.c_int(gamma), C.c_int(budget_tokens),
                            C.c_int(mode), C.c_int(topk_K), _p(table), C.c_int(len(table) - 1),
                            _p(out_len), _p(surv), _p(exp_len), C.byref(info), _p(path))
    if rc != 0:
        raise ValueError(f"orc_schedule failed ({rc})")
    return ScheduleResult(out_len, surv, exp_len, info.B, info.n_admitted, info.n_candidates,
                          info.status, info.tau, info.theta, path)


def schedule_async(conf, table, budget_tokens: int, state: np.ndarray, draft_len=None) -> ScheduleResult:
    """One step of the asynchronous top-K scheduler; `state` (int32[3] = step, K slot 0, K slot 1)
    is updated in place."""
    conf = np.ascontiguousarray(conf, dtype=np.float32)
    R, gamma = conf.shape
    table = np.ascontiguousarray(table, dtype=np.float64)
    dl = None if draft_len is None else np.ascontiguousarray(draft_len, dtype=np.int32)
    assert state.dtype == np.int32 and state.size >= 3 and state.flags.c_contiguous
    out_len = np.zeros(R, dtype=np.int32)
    surv = np.zeros((R, max(gamma, 1)), dtype=np.float32)[:, :gamma].copy()
    exp_len = np.zeros(R, dtype=np.float32)
    info = _SchedInfo()
    rc = lib().orc_schedule_async(_p(conf), _p(dl), C.c_int(R), C.c_int(gamma), C.c_int(budget_tokens),
                                  _p(table), C.c_int(len(table) - 1), _p(state), _p(out_len), _p(surv),
                                  _p(exp_len), C.byref(info))
    if rc != 0:
        raise ValueError(f"orc_schedule_async failed ({rc})")
    return ScheduleResult(out_len, surv, exp_len, info.B, info.n_admitted, info.n_candidates,
                          info.status, info.tau, info.theta, np.empty(0))


def schedule_bruteforce(conf, table, budget_tokens: int, draft_len=None):
    conf = np.ascontiguousarray(conf, dtype=np.float32)
    R, gamma = conf.shape
    table = np.ascontiguousarray(table, dtype=np.float64)
    dl = None if draft_len is None else np.ascontiguousarray(draft_len, dtype=np.int32)
    best = C.c_double()
    best_B = C.c_int32()
    best_len = np.zeros(R, dtype=np.int32)
    rc = lib().orc_schedule_bruteforce(_p(conf), _p(dl), C.c_int(R), C.c_int(gamma),
                                       C.c_int(budget_tokens), _p(table), C.c_int(len(table) - 1),
                                       C.byref(best), C.byref(best_B), _p(best_len))
    if rc != 0:
        raise ValueError("brute force limited to R <= 8, gamma <= 8")
    return best.value, best_B.value, best_len


def _logits(a):
    a = np.asarray(a)
    if a.ndim != 2 or a.strides[1] != a.itemsize:
        raise ValueError("logits must be 2-D with unit inner stride")
    return a, a.strides[0] // a.itemsize


def softmax_row(logits, row: int, temperature: float = 1.0):
    a, stride = _logits(logits)
    V = a.shape[1]
    probs = np.empty(V, dtype=np.float64)
    m, Z = C.c_double(), C.c_double()
    bad = lib().orc_softmax_row(_p(a), C.c_int(_dtype_code(a)), C.c_int64(row), C.c_int64(stride),
                                C.c_int(V), C.c_double(temperature), _p(probs), C.byref(m), C.byref(Z))
    return probs, m.value, Z.value, bool(bad)


@dataclass
class GreedyResult:
    accepted_len: np.ndarray
    out_tokens: np.ndarray
    row_argmax: np.ndarray
    status: np.ndarray


def verify_greedy(target, row_offsets, draft_tokens) -> GreedyResult:
    t, stride = _logits(target)
    ro = np.ascontiguousarray(row_offsets, dtype=np.int32)
    dt = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    R = len(ro) - 1
    n_rows = t.shape[0]
    acc = np.zeros(R, dtype=np.int32)
    out = np.full(n_rows, -1, dtype=np.int32)
    am = np.full(n_rows, -1, dtype=np.int32)
    st = np.zeros(R, dtype=np.int32)
    rc = lib().orc_verify_greedy(_p(t), C.c_int(_dtype_code(t)), C.c_int64(stride), C.c_int(t.shape[1]),
                                 _p(ro), _p(dt), C.c_int(R), _p(acc), _p(out), _p(am), _p(st))
    if rc != 0:
        raise ValueError("orc_verify_greedy failed")
    return GreedyResult(acc, out, am, st)


def verify_greedy_mt(target, row_offsets, draft_tokens, n_threads: int):
    t, stride = _logits(target)
    ro = np.ascontiguousarray(row_offsets, dtype=np.int32)
    dt = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    R = len(ro) - 1
    acc = np.zeros(R, dtype=np.int32)
    out = np.full(t.shape[0], -1, dtype=np.int32)
    st = np.zeros(R, dtype=np.int32)
    rc = lib().orc_verify_greedy_mt(_p(t), C.c_int(_dtype_code(t)), C.c_int64(stride), C.c_int(t.shape[1]),
                                    _p(ro), _p(dt), C.c_int(R), C.c_int(n_threads), _p(acc), _p(out), _p(st))
    if rc != 0:
        raise ValueError("orc_verify_greedy_mt failed")
    return acc, out, st


@dataclass
class VerifyResult:
    accepted_len: np.ndarray
    out_tokens: np.ndarray
    p_tok: np.ndarray
    q_tok: np.ndarray
    accept_margin: np.ndarray
    token_margin: np.ndarray          # per request: distance of the draw to the nearer CDF boundary of the distribution drawn from
    status: np.ndarray
    token_margin_abs: np.ndarray = None   # the same distance in probability units (residual draws: times W)
    resid_mass: np.ndarray = None         # W = sum max(0, p - q) of a residual draw, NaN for a draw from p


def verify(target, draft, row_offsets, draft_tokens, temperature: float, seed: int,
           draft_row_start=None, eval_all: bool = True, n_threads: int = 1, temperatures=None) -> VerifyResult:
    """temperatures: optional float32[R], one temperature per request (overrides `temperature`)."""
    t, ts = _logits(target)
    d, ds = _logits(draft)
    if t.dtype != d.dtype:
        raise TypeError("target and draft logits must share a dtype")
    ro = np.ascontiguousarray(row_offsets, dtype=np.int32)
    dt = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    drs = None if draft_row_start is None else np.ascontiguousarray(draft_row_start, dtype=np.int64)
    R = len(ro) - 1
    n_rows = t.shape[0]
    acc = np.zeros(R, dtype=np.int32)
    out = np.full(n_rows, -1, dtype=np.int32)
    p = np.full(n_rows, np.nan)
    q = np.full(n_rows, np.nan)
    am = np.full(n_rows, np.nan)
    tm = np.full(R, np.nan)
    tma = np.full(R, np.nan)
    rw = np.full(R, np.nan)
    st = np.zeros(R, dtype=np.int32)
    temps = None if temperatures is None else np.ascontiguousarray(temperatures, dtype=np.float32)
    rc = lib().orc_verify(_p(t), _p(d), C.c_int(_dtype_code(t)), C.c_int64(ts), C.c_int64(ds),
                          C.c_int(t.shape[1]), _p(ro), _p(drs), _p(dt), C.c_int(R),
                          C.c_double(temperature), _p(temps), C.c_uint64(seed), C.c_int(int(eval_all)),
                          C.c_int(n_threads), _p(acc), _p(out), _p(p), _p(q), _p(am), _p(tm), _p(tma), _p(rw), _p(st))
    if rc != 0:
        raise ValueError("orc_verify rejected its arguments")
    return VerifyResult(acc, out, p, q, am, tm, st, tma, rw)


def accept_rate(target, draft, row_offsets, temperature: float, draft_row_start=None):
    """c*_{r,j} = 1 - TV(p, q) at every draft position (NaN at bonus rows); returns (cstar, status)."""
    t, ts = _logits(target)
    d, ds = _logits(draft)
    ro = np.ascontiguousarray(row_offsets, dtype=np.int32)
    drs = None if draft_row_start is None else np.ascontiguousarray(draft_row_start, dtype=np.int64)
    R = len(ro) - 1
    cstar = np.full(t.shape[0], np.nan)
    st = np.zeros(R, dtype=np.int32)
    rc = lib().orc_accept_rate(_p(t), _p(d), C.c_int(_dtype_code(t)), C.c_int64(ts), C.c_int64(ds),
                               C.c_int(t.shape[1]), _p(ro), _p(drs), C.c_int(R), C.c_double(temperature),
                               _p(cstar), _p(st))
    if rc != 0:
        raise ValueError("orc_accept_rate rejected its arguments")
    return cstar, st


def markov_logits(U, W1, W2, x_prev):
    """Draft logits U + W1[x_prev] @ W2 from bf16 bit patterns (uint16).  Returns (fp64, bf16 bits)."""
    U = np.asarray(U); W1 = np.ascontiguousarray(W1); W2 = np.ascontiguousarray(W2)
    assert U.dtype == W1.dtype == W2.dtype == np.uint16 and U.strides[1] == 2
    R, V = U.shape
    rank = W1.shape[1]
    assert W1.shape[0] == V and W2.shape == (rank, V)
    xp = np.ascontiguousarray(x_prev, dtype=np.int32)
    f64 = np.empty((R, V), dtype=np.float64)
    b16 = np.empty((R, V), dtype=np.uint16)
    rc = lib().orc_markov_logits(_p(U), C.c_int64(U.strides[0] // 2), _p(W1), _p(W2), _p(xp), C.c_int(R), C.c_int(V),
                                 C.c_int(rank), _p(f64), _p(b16))
    if rc != 0:
        raise ValueError(f"orc_markov_logits failed ({rc})")
    return f64, b16


def confidence(H, W1, w, x_prev):
    """c = sigmoid(w . [h ; W1[x_prev]]): H bf16 bits [R, d], W1 bf16 bits [V, rank], w float32 [d + rank]."""
    H = np.asarray(H); W1 = np.ascontiguousarray(W1)
    w = np.ascontiguousarray(w, dtype=np.float32)
    R, d = H.shape
    V, rank = W1.shape
    assert w.size == d + rank
    xp = np.ascontiguousarray(x_prev, dtype=np.int32)
    out = np.empty(R, dtype=np.float64)
    rc = lib().orc_confidence(_p(H), C.c_int64(H.strides[0] // 2), C.c_int(d), _p(W1), C.c_int(rank), C.c_int(V),
                              _p(w), _p(xp), C.c_int(R), _p(out))
    if rc != 0:
        raise ValueError(f"orc_confidence failed ({rc})")
    return out


def sts_calibrate(conf, accepted_len, grid, n_bins: int = 15, verified_len=None):
    """Sequential Temperature Scaling.  conf float32 [N, gamma]; returns (T[gamma] float32, ece_before, ece_after,
    ece_grid[gamma, G]) with the ECE values in fp64."""
    c = np.ascontiguousarray(conf, dtype=np.float32)
    N, gamma = c.shape
    acc = np.ascontiguousarray(accepted_len, dtype=np.int32)
    ver = None if verified_len is None else np.ascontiguousarray(verified_len, dtype=np.int32)
    g = np.ascontiguousarray(grid, dtype=np.float32)
    T = np.empty(gamma, dtype=np.float32)
    eb = np.empty(gamma); ea = np.empty(gamma); eg = np.empty((gamma, len(g)))
    rc = lib().orc_sts_calibrate(_p(c), C.c_int(N), C.c_int(gamma), _p(acc), _p(ver), _p(g), C.c_int(len(g)),
                                 C.c_int(n_bins), _p(T), _p(eb), _p(ea), _p(eg))
    if rc != 0:
        raise ValueError(f"orc_sts_calibrate failed ({rc})")
    return T, eb, ea, eg


def sts_apply(conf, T):
    c = np.ascontiguousarray(conf, dtype=np.float32)
    t = np.ascontiguousarray(T, dtype=np.float32)
    out = np.empty(c.shape)
    lib().orc_sts_apply(_p(c), C.c_int(c.shape[0]), C.c_int(c.shape[1]), _p(t), _p(out))
    return out


def warp_target(target, row_offsets, top_k=None, top_p=None, temperature: float = 1.0, temperatures=None):
    """Top-k / top-p truncation of the target rows of a ragged batch: returns (masked copy, tau[n_rows],
    kept[n_rows], margin[n_rows]).  target: float32 or bf16 bit patterns (uint16), [n_rows, V]."""
    t = np.array(target, copy=True)
    tt, stride = _logits(t)
    ro = np.ascontiguousarray(row_offsets, dtype=np.int32)
    R = len(ro) - 1
    k = None if top_k is None else np.ascontiguousarray(top_k, dtype=np.int32)
    p = None if top_p is None else np.ascontiguousarray(top_p, dtype=np.float32)
    temps = None if temperatures is None else np.ascontiguousarray(temperatures, dtype=np.float32)
    n_rows = t.shape[0]
    tau = np.full(n_rows, -np.inf); kept = np.full(n_rows, t.shape[1], dtype=np.int32); margin = np.full(n_rows, np.inf)
    rc = lib().orc_warp_target(_p(tt), C.c_int(_dtype_code(tt)), C.c_int64(stride), C.c_int(t.shape[1]), _p(ro), C.c_int(R),
                               _p(k), _p(p), C.c_double(temperature), _p(temps), _p(tau), _p(kept), _p(margin))
    if rc != 0:
        raise ValueError(f"orc_warp_target failed ({rc})")
    return tt, tau, kept, margin
