"""Thin ctypes binding over ``libdspark.so`` (declared in ``include/dspark.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels.  The
functions keep the C names and take torch CUDA tensors (device memory and streams
are PyTorch's), returning the library's status code turned into an exception.
There is no CPU fallback: a missing library or a CPU tensor raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdspark.so")
_lib: Optional[C.CDLL] = None

DSPARK_F32, DSPARK_BF16 = 0, 1
DSPARK_SCHED_EARLY_STOP, DSPARK_SCHED_GLOBAL, DSPARK_SCHED_TOPK = 0, 1, 2
DEV_BAD_OFFSETS, DEV_BAD_TOKEN, DEV_BAD_ROW, DEV_TIMEOUT = 1, 2, 4, 8
DEV_CONF_CLAMPED, DEV_BUDGET_LT_R, DEV_ALL_NEG_INF, DEV_BAD_TEMPERATURE = 16, 32, 64, 128
(K_SCHEDULE, K_OFFSETS, K_STREAM, K_DECIDE, K_RESIDUAL, K_FINALIZE, K_GREEDY_STREAM, K_GREEDY_DECIDE,
 K_ROW_SCALE, K_MARKOV_GEMM, K_MARKOV_DRAW, K_TRUNCATE, K_COUNT) = range(13)

EXPORTS = [
    "dspark_profile_create", "dspark_profile_destroy", "dspark_profile_table",
    "dspark_schedule_workspace_bytes", "dspark_schedule", "dspark_build_offsets",
    "dspark_schedule_async", "dspark_async_state_init",
    "dspark_verify_workspace_bytes", "dspark_verify_greedy", "dspark_verify", "dspark_uniforms",
    "dspark_verify_greedy_static", "dspark_verify_greedy_static_capacity", "dspark_verify_greedy_static_bytes",
    "dspark_verify_per_request", "dspark_verify_draft_stats", "dspark_row_stats",
    "dspark_accept_rate", "dspark_accept_rate_workspace_bytes",
    "dspark_markov_w2_packed_bytes", "dspark_markov_pack_w2", "dspark_markov_workspace_bytes",
    "dspark_markov_logits", "dspark_markov_draft_step", "dspark_markov_draft_step_stats", "dspark_markov_set_epilogue_path",
    "dspark_truncate_target", "dspark_verify_truncated",
    "dspark_sts_workspace_bytes", "dspark_sts_calibrate", "dspark_sts_apply",
    "dspark_ktimer_create", "dspark_ktimer_destroy", "dspark_ktimer_attach", "dspark_ktimer_reset",
    "dspark_ktimer_read", "dspark_set_stream_path", "dspark_set_wait_poll_limit", "dspark_status_string", "dspark_kernel_name",
    "dspark_version",
]


class DsparkError(RuntimeError):
    pass


class SchedInfo(C.Structure):
    _fields_ = [("B", C.c_int32), ("n_admitted", C.c_int32), ("status", C.c_int32),
                ("n_candidates", C.c_int32), ("tau", C.c_double), ("theta", C.c_double)]


def lib() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise DsparkError(f"{_LIB_PATH} is missing: run `python -m paper_2607_05147_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(_LIB_PATH)
        vp, i32, i64, u64, sz = C.c_void_p, C.c_int, C.c_int64, C.c_uint64, C.c_size_t
        L.dspark_profile_create.argtypes = [vp, vp, i32, i32, C.POINTER(vp)]
        L.dspark_profile_destroy.argtypes = [vp]
        L.dspark_profile_table.argtypes = [vp, C.POINTER(C.c_int)]
        L.dspark_profile_table.restype = vp
        L.dspark_schedule_workspace_bytes.argtypes = [i32, i32]
        L.dspark_schedule_workspace_bytes.restype = sz
        L.dspark_schedule.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.dspark_build_offsets.argtypes = [vp, i32, vp, vp]
        L.dspark_async_state_init.argtypes = [vp, i32, vp]
        L.dspark_schedule_async.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.dspark_verify_workspace_bytes.argtypes = [i32, i32, i32]
        L.dspark_verify_workspace_bytes.restype = sz
        L.dspark_verify_greedy.argtypes = [vp, i32, i64, i32, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp]
        L.dspark_verify_greedy_static.argtypes = [vp, i32, i64, i32, vp, vp, i32, i32, vp, vp, vp, vp]
        L.dspark_verify_greedy_static_capacity.argtypes = []
        L.dspark_verify_greedy_static_capacity.restype = sz
        L.dspark_verify_greedy_static_bytes.argtypes = [i32, i32, i32, i32]
        L.dspark_verify_greedy_static_bytes.restype = sz
        L.dspark_verify.argtypes = [vp, vp, i32, i64, i64, i32, vp, vp, vp, i32, i32, C.c_float, u64,
                                    vp, vp, vp, vp, vp, vp, sz, vp]
        L.dspark_verify_per_request.argtypes = [vp, vp, i32, i64, i64, i32, vp, vp, vp, i32, i32, vp, u64,
                                                vp, vp, vp, vp, vp, vp, sz, vp]
        L.dspark_verify_draft_stats.argtypes = [vp, vp, i32, i64, i64, i32, vp, vp, vp, vp, i32, i32, C.c_float, vp, u64,
                                                vp, vp, vp, vp, vp, vp, sz, vp]
        L.dspark_row_stats.argtypes = [vp, i32, i64, i32, i32, C.c_float, vp, vp, vp]
        L.dspark_accept_rate_workspace_bytes.argtypes = [i32, i32, i32]
        L.dspark_accept_rate_workspace_bytes.restype = sz
        L.dspark_accept_rate.argtypes = [vp, vp, i32, i64, i64, i32, vp, vp, i32, i32, C.c_float, vp, vp, vp, sz, vp]
        L.dspark_markov_set_epilogue_path.argtypes = [i32]
        L.dspark_markov_w2_packed_bytes.argtypes = [i32]
        L.dspark_markov_w2_packed_bytes.restype = sz
        L.dspark_markov_pack_w2.argtypes = [vp, i32, vp, vp]
        L.dspark_markov_workspace_bytes.argtypes = [i32, i32]
        L.dspark_markov_workspace_bytes.restype = sz
        L.dspark_markov_logits.argtypes = [vp, i64, vp, vp, vp, i32, i32, vp, i64, i32, vp, vp, i64, vp, vp, vp, sz, vp]
        L.dspark_markov_draft_step.argtypes = [vp, i64, vp, vp, vp, i32, i32, vp, i64, i32, vp, C.c_float, u64,
                                               vp, i64, vp, vp, vp, vp, sz, vp]
        L.dspark_markov_draft_step_stats.argtypes = [vp, i64, vp, vp, vp, i32, i32, vp, i64, i32, vp, C.c_float, u64,
                                                     vp, i64, vp, vp, vp, i64, vp, vp, sz, vp]
        L.dspark_verify_truncated.argtypes = [vp, vp, i32, i64, i64, i32, vp, vp, vp, i32, i32, C.c_float, vp, vp, vp, u64,
                                              vp, vp, vp, vp, vp, vp, sz, vp]
        L.dspark_truncate_target.argtypes = [vp, i32, i64, i32, vp, i32, i32, vp, vp, C.c_float, vp, vp, vp, vp, vp]
        L.dspark_sts_workspace_bytes.argtypes = [i32, i32, i32, i32]
        L.dspark_sts_workspace_bytes.restype = sz
        L.dspark_sts_calibrate.argtypes = [vp, i32, i32, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.dspark_sts_apply.argtypes = [vp, i32, i32, vp, vp, vp]
        L.dspark_uniforms.argtypes = [u64, C.c_uint32, C.c_uint32, C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.dspark_uniforms.restype = None
        L.dspark_ktimer_create.argtypes = [i32, C.POINTER(vp)]
        L.dspark_ktimer_destroy.argtypes = [vp]
        L.dspark_ktimer_attach.argtypes = [vp]
        L.dspark_ktimer_reset.argtypes = [vp]
        L.dspark_ktimer_read.argtypes = [vp, i32, C.POINTER(C.c_float), C.POINTER(C.c_int)]
        L.dspark_set_stream_path.argtypes = [i32]
        L.dspark_set_wait_poll_limit.argtypes = [C.c_uint]
        L.dspark_status_string.argtypes = [i32]
        L.dspark_status_string.restype = C.c_char_p
        L.dspark_kernel_name.argtypes = [i32]
        L.dspark_kernel_name.restype = C.c_char_p
        _lib = L
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise DsparkError(f"{what}: {lib().dspark_status_string(rc).decode()} ({rc})")


def _dev(t: Optional[torch.Tensor], name: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise DsparkError(f"{name} must be a CUDA tensor (no CPU path exists)")
    if dtype is not None and t.dtype != dtype:
        raise DsparkError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous() and t.dim() <= 1:
        raise DsparkError(f"{name} must be contiguous")
    return t.data_ptr()


def _logits(t: torch.Tensor, name: str):
    if t.dim() != 2 or t.stride(1) != 1:
        raise DsparkError(f"{name} must be 2-D with unit inner stride")
    if t.dtype == torch.float32:
        code = DSPARK_F32
    elif t.dtype == torch.bfloat16:
        code = DSPARK_BF16
    else:
        raise DsparkError(f"{name} must be float32 or bfloat16")
    return _dev(t, name), code, t.stride(0)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


# ------------------------------------------------------------------------------- profile ----
class Profile:
    """Owner of a ``dspark_profile_t`` (device SPS table)."""

    def __init__(self, bp_tokens, bp_sps, max_tokens: int):
        n = len(bp_tokens)
        bt = (C.c_int32 * n)(*[int(x) for x in bp_tokens])
        bs = (C.c_double * n)(*[float(x) for x in bp_sps])
        h = C.c_void_p()
        _check(lib().dspark_profile_create(bt, bs, n, int(max_tokens), C.byref(h)), "dspark_profile_create")
        self.handle = h
        self.max_tokens = int(max_tokens)

    def table(self) -> torch.Tensor:
        """Copy of the device table as a host fp64 tensor (tests)."""
        mt = C.c_int()
        ptr = lib().dspark_profile_table(self.handle, C.byref(mt))

        class _Raw:   # view of the library-owned device table through the CUDA array interface
            __cuda_array_interface__ = {"shape": (mt.value + 1,), "typestr": "<f8", "data": (ptr, False), "version": 2}
        return torch.as_tensor(_Raw(), device="cuda").clone().cpu()

    def close(self):
        if self.handle:
            lib().dspark_profile_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def dspark_schedule_workspace_bytes(R: int, gamma: int) -> int:
    return int(lib().dspark_schedule_workspace_bytes(R, gamma))


def dspark_schedule(prof: Profile, conf: torch.Tensor, budget_tokens: int, mode: int = DSPARK_SCHED_EARLY_STOP,
                    topk_K: int = 0, draft_len: Optional[torch.Tensor] = None, *, out_len: torch.Tensor,
                    out_row_offsets: Optional[torch.Tensor] = None, out_survival: Optional[torch.Tensor] = None,
                    out_expected_len: Optional[torch.Tensor] = None, out_info: Optional[torch.Tensor] = None,
                    workspace: torch.Tensor) -> None:
    """out_info: a 32-byte CUDA uint8 tensor receiving dspark_sched_info_t."""
    if conf.dim() != 2 or not conf.is_contiguous():
        raise DsparkError("conf must be a contiguous [R, gamma] tensor")
    R, gamma = conf.shape
    rc = lib().dspark_schedule(prof.handle, _dev(conf, "conf", torch.float32), _dev(draft_len, "draft_len", torch.int32),
                               R, gamma, int(budget_tokens), int(mode), int(topk_K),
                               _dev(out_len, "out_len", torch.int32), _dev(out_row_offsets, "out_row_offsets", torch.int32),
                               _dev(out_survival, "out_survival", torch.float32),
                               _dev(out_expected_len, "out_expected_len", torch.float32),
                               _dev(out_info, "out_info", torch.uint8), _dev(workspace, "workspace"),
                               workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_schedule")


def dspark_async_state_init(state: torch.Tensor, initial_K: int) -> None:
    """state: CUDA int32[4] kept by the caller between steps."""
    if state.numel() < 4:
        raise DsparkError("state must hold 4 int32")
    _check(lib().dspark_async_state_init(_dev(state, "state", torch.int32), int(initial_K), _stream()),
           "dspark_async_state_init")


def dspark_schedule_async(prof: Profile, conf: torch.Tensor, budget_tokens: int, state: torch.Tensor,
                          draft_len: Optional[torch.Tensor] = None, *, out_len: torch.Tensor,
                          out_row_offsets: Optional[torch.Tensor] = None, out_survival: Optional[torch.Tensor] = None,
                          out_expected_len: Optional[torch.Tensor] = None, out_info: Optional[torch.Tensor] = None,
                          workspace: torch.Tensor) -> None:
    if conf.dim() != 2 or not conf.is_contiguous():
        raise DsparkError("conf must be a contiguous [R, gamma] tensor")
    R, gamma = conf.shape
    rc = lib().dspark_schedule_async(prof.handle, _dev(conf, "conf", torch.float32),
                                     _dev(draft_len, "draft_len", torch.int32), R, gamma, int(budget_tokens),
                                     _dev(state, "state", torch.int32), _dev(out_len, "out_len", torch.int32),
                                     _dev(out_row_offsets, "out_row_offsets", torch.int32),
                                     _dev(out_survival, "out_survival", torch.float32),
                                     _dev(out_expected_len, "out_expected_len", torch.float32),
                                     _dev(out_info, "out_info", torch.uint8), _dev(workspace, "workspace"),
                                     workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_schedule_async")


def read_sched_info(out_info: torch.Tensor) -> SchedInfo:
    raw = bytes(out_info.cpu().numpy().tobytes())
    return SchedInfo.from_buffer_copy(raw)


def dspark_build_offsets(lengths: torch.Tensor, row_offsets: torch.Tensor) -> None:
    _check(lib().dspark_build_offsets(_dev(lengths, "lengths", torch.int32), lengths.numel(),
                                      _dev(row_offsets, "row_offsets", torch.int32), _stream()), "dspark_build_offsets")


def dspark_verify_workspace_bytes(R: int, n_rows: int, V: int) -> int:
    return int(lib().dspark_verify_workspace_bytes(R, n_rows, V))


def dspark_verify_greedy(target: torch.Tensor, row_offsets: torch.Tensor, draft_tokens: torch.Tensor, *,
                         accepted_len: torch.Tensor, out_tokens: torch.Tensor,
                         dev_status: Optional[torch.Tensor], workspace: torch.Tensor,
                         n_rows: Optional[int] = None) -> None:
    tp, code, ts = _logits(target, "target")
    R = row_offsets.numel() - 1
    n_rows = target.shape[0] if n_rows is None else n_rows
    rc = lib().dspark_verify_greedy(tp, code, ts, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32),
                                    _dev(draft_tokens, "draft_tokens", torch.int32), R, n_rows,
                                    _dev(accepted_len, "accepted_len", torch.int32),
                                    _dev(out_tokens, "out_tokens", torch.int32),
                                    _dev(dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
                                    workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_verify_greedy")


def dspark_verify_greedy_static_capacity() -> int:
    return int(lib().dspark_verify_greedy_static_capacity())


def dspark_verify_greedy_static_bytes(R: int, n_rows: int, V: int, dtype: torch.dtype) -> int:
    """Bytes of the built-in array a batch of this shape would use (0: invalid shape)."""
    code = DSPARK_BF16 if dtype == torch.bfloat16 else DSPARK_F32
    return int(lib().dspark_verify_greedy_static_bytes(R, n_rows, V, code))


def dspark_verify_greedy_static(target: torch.Tensor, row_offsets: torch.Tensor, draft_tokens: torch.Tensor, *,
                                accepted_len: torch.Tensor, out_tokens: torch.Tensor,
                                dev_status: Optional[torch.Tensor], n_rows: Optional[int] = None) -> None:
    """Greedy verification without a caller workspace, for callers that may not allocate device
    memory: the scratch is a fixed array inside the library.  Raises when the batch is larger than
    that array (see dspark_verify_greedy_static_capacity)."""
    tp, code, ts = _logits(target, "target")
    R = row_offsets.numel() - 1
    n_rows = target.shape[0] if n_rows is None else n_rows
    rc = lib().dspark_verify_greedy_static(tp, code, ts, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32),
                                           _dev(draft_tokens, "draft_tokens", torch.int32), R, n_rows,
                                           _dev(accepted_len, "accepted_len", torch.int32),
                                           _dev(out_tokens, "out_tokens", torch.int32),
                                           _dev(dev_status, "dev_status", torch.int32), _stream())
    _check(rc, "dspark_verify_greedy_static")


def dspark_verify(target: torch.Tensor, draft: torch.Tensor, row_offsets: torch.Tensor,
                  draft_tokens: torch.Tensor, temperature: float, seed: int, *,
                  draft_row_start: Optional[torch.Tensor] = None,
                  accepted_len: torch.Tensor, out_tokens: torch.Tensor,
                  out_p_tok: Optional[torch.Tensor] = None, out_q_tok: Optional[torch.Tensor] = None,
                  dev_status: Optional[torch.Tensor], workspace: torch.Tensor,
                  n_rows: Optional[int] = None) -> None:
    tp, code, ts = _logits(target, "target")
    dp, dcode, ds = _logits(draft, "draft")
    if code != dcode or target.shape[1] != draft.shape[1]:
        raise DsparkError("target and draft logits must share dtype and vocabulary size")
    R = row_offsets.numel() - 1
    n_rows = target.shape[0] if n_rows is None else n_rows
    rc = lib().dspark_verify(tp, dp, code, ts, ds, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32),
                             _dev(draft_row_start, "draft_row_start", torch.int64),
                             _dev(draft_tokens, "draft_tokens", torch.int32), R, n_rows,
                             float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF,
                             _dev(accepted_len, "accepted_len", torch.int32), _dev(out_tokens, "out_tokens", torch.int32),
                             _dev(out_p_tok, "out_p_tok", torch.float32), _dev(out_q_tok, "out_q_tok", torch.float32),
                             _dev(dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
                             workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_verify")


def dspark_verify_per_request(target: torch.Tensor, draft: torch.Tensor, row_offsets: torch.Tensor,
                              draft_tokens: torch.Tensor, temperatures: torch.Tensor, seed: int, *,
                              draft_row_start: Optional[torch.Tensor] = None,
                              accepted_len: torch.Tensor, out_tokens: torch.Tensor,
                              out_p_tok: Optional[torch.Tensor] = None, out_q_tok: Optional[torch.Tensor] = None,
                              dev_status: Optional[torch.Tensor], workspace: torch.Tensor,
                              n_rows: Optional[int] = None) -> None:
    """dspark_verify with a CUDA float32[R] of per-request temperatures."""
    tp, code, ts = _logits(target, "target")
    dp, dcode, ds = _logits(draft, "draft")
    if code != dcode or target.shape[1] != draft.shape[1]:
        raise DsparkError("target and draft logits must share dtype and vocabulary size")
    R = row_offsets.numel() - 1
    if temperatures.numel() != R:
        raise DsparkError("temperatures must have one entry per request")
    n_rows = target.shape[0] if n_rows is None else n_rows
    rc = lib().dspark_verify_per_request(
        tp, dp, code, ts, ds, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32),
        _dev(draft_row_start, "draft_row_start", torch.int64), _dev(draft_tokens, "draft_tokens", torch.int32),
        R, n_rows, _dev(temperatures, "temperatures", torch.float32), int(seed) & 0xFFFFFFFFFFFFFFFF,
        _dev(accepted_len, "accepted_len", torch.int32), _dev(out_tokens, "out_tokens", torch.int32),
        _dev(out_p_tok, "out_p_tok", torch.float32), _dev(out_q_tok, "out_q_tok", torch.float32),
        _dev(dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_verify_per_request")


def dspark_verify_truncated(target: torch.Tensor, draft: torch.Tensor, row_offsets: torch.Tensor,
                            draft_tokens: torch.Tensor, seed: int, *, temperature: float = 1.0,
                            temperatures: Optional[torch.Tensor] = None, top_k: Optional[torch.Tensor] = None,
                            top_p: Optional[torch.Tensor] = None, draft_row_start: Optional[torch.Tensor] = None,
                            accepted_len: torch.Tensor, out_tokens: torch.Tensor,
                            out_p_tok: Optional[torch.Tensor] = None, out_q_tok: Optional[torch.Tensor] = None,
                            dev_status: Optional[torch.Tensor], workspace: torch.Tensor,
                            n_rows: Optional[int] = None) -> None:
    """Sampling verification against the top-k / top-p truncated target distribution (rows not modified)."""
    tp, code, ts = _logits(target, "target")
    dp, dcode, ds = _logits(draft, "draft")
    if code != dcode or target.shape[1] != draft.shape[1]:
        raise DsparkError("target and draft logits must share dtype and vocabulary size")
    R = row_offsets.numel() - 1
    for t, name in ((temperatures, "temperatures"), (top_k, "top_k"), (top_p, "top_p")):
        if t is not None and t.numel() != R:
            raise DsparkError(f"{name} must have one entry per request")
    n_rows = target.shape[0] if n_rows is None else n_rows
    rc = lib().dspark_verify_truncated(
        tp, dp, code, ts, ds, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32),
        _dev(draft_row_start, "draft_row_start", torch.int64), _dev(draft_tokens, "draft_tokens", torch.int32),
        R, n_rows, float(temperature), _dev(temperatures, "temperatures", torch.float32),
        _dev(top_k, "top_k", torch.int32), _dev(top_p, "top_p", torch.float32), int(seed) & 0xFFFFFFFFFFFFFFFF,
        _dev(accepted_len, "accepted_len", torch.int32), _dev(out_tokens, "out_tokens", torch.int32),
        _dev(out_p_tok, "out_p_tok", torch.float32), _dev(out_q_tok, "out_q_tok", torch.float32),
        _dev(dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_verify_truncated")


def dspark_accept_rate_workspace_bytes(R: int, n_rows: int, V: int) -> int:
    return int(lib().dspark_accept_rate_workspace_bytes(R, n_rows, V))


def dspark_accept_rate(target: torch.Tensor, draft: torch.Tensor, row_offsets: torch.Tensor, temperature: float, *,
                       draft_row_start: Optional[torch.Tensor] = None, out_cstar: torch.Tensor,
                       dev_status: Optional[torch.Tensor], workspace: torch.Tensor,
                       n_rows: Optional[int] = None) -> None:
    """c* = 1 - TV(p, q) at every draft position (the confidence head's analytical label)."""
    tp, code, ts = _logits(target, "target")
    dp, dcode, ds = _logits(draft, "draft")
    if code != dcode or target.shape[1] != draft.shape[1]:
        raise DsparkError("target and draft logits must share dtype and vocabulary size")
    R = row_offsets.numel() - 1
    n_rows = target.shape[0] if n_rows is None else n_rows
    rc = lib().dspark_accept_rate(tp, dp, code, ts, ds, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32),
                                  _dev(draft_row_start, "draft_row_start", torch.int64), R, n_rows, float(temperature),
                                  _dev(out_cstar, "out_cstar", torch.float32), _dev(dev_status, "dev_status", torch.int32),
                                  _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_accept_rate")


def dspark_markov_set_epilogue_path(path: int) -> None:
    _check(lib().dspark_markov_set_epilogue_path(int(path)), "dspark_markov_set_epilogue_path")


def dspark_markov_w2_packed_bytes(V: int) -> int:
    return int(lib().dspark_markov_w2_packed_bytes(V))


def dspark_markov_pack_w2(W2: torch.Tensor, W2_packed: torch.Tensor) -> None:
    """W2: CUDA bf16 [256, V] contiguous; W2_packed: CUDA uint8 of dspark_markov_w2_packed_bytes(V)."""
    if W2.dim() != 2 or W2.shape[0] != 256 or not W2.is_contiguous():
        raise DsparkError("W2 must be a contiguous [256, V] tensor")
    if W2_packed.numel() * W2_packed.element_size() < dspark_markov_w2_packed_bytes(W2.shape[1]):
        raise DsparkError("W2_packed is too small")
    _check(lib().dspark_markov_pack_w2(_dev(W2, "W2", torch.bfloat16), W2.shape[1], _dev(W2_packed, "W2_packed"),
                                       _stream()), "dspark_markov_pack_w2")


def dspark_markov_workspace_bytes(R: int, V: int) -> int:
    return int(lib().dspark_markov_workspace_bytes(R, V))


def _markov_args(U, W1, W2_packed, x_prev, H, w_conf, out_logits, out_conf):
    if U.dim() != 2 or U.stride(1) != 1 or out_logits.dim() != 2 or out_logits.stride(1) != 1:
        raise DsparkError("U and out_logits must be 2-D with unit inner stride")
    R, V = U.shape
    if W1.shape != (V, 256) or not W1.is_contiguous():
        raise DsparkError("W1 must be a contiguous [V, 256] tensor")
    if out_logits.shape[0] < R or out_logits.shape[1] < V or x_prev.numel() < R:
        raise DsparkError("out_logits / x_prev are too small")
    d = 0
    if out_conf is not None:
        if H is None or w_conf is None or H.dim() != 2 or H.stride(1) != 1 or H.shape[0] < R:
            raise DsparkError("out_conf needs H [R, d] and w_conf [d + 256]")
        d = H.shape[1]
        if w_conf.numel() != d + 256 or out_conf.numel() < R:
            raise DsparkError("w_conf must hold d + 256 weights, out_conf R values")
    return (_dev(U, "U", torch.bfloat16), U.stride(0), _dev(W1, "W1", torch.bfloat16), _dev(W2_packed, "W2_packed"),
            _dev(x_prev, "x_prev", torch.int32), R, V, _dev(H, "H", torch.bfloat16) if out_conf is not None else None,
            H.stride(0) if out_conf is not None else 0, d,
            _dev(w_conf, "w_conf", torch.float32) if out_conf is not None else None)


def dspark_markov_logits(U: torch.Tensor, W1: torch.Tensor, W2_packed: torch.Tensor, x_prev: torch.Tensor, *,
                         H: Optional[torch.Tensor] = None, w_conf: Optional[torch.Tensor] = None,
                         out_logits: torch.Tensor, out_conf: Optional[torch.Tensor] = None,
                         dev_status: torch.Tensor, workspace: torch.Tensor) -> None:
    head = _markov_args(U, W1, W2_packed, x_prev, H, w_conf, out_logits, out_conf)
    rc = lib().dspark_markov_logits(*head, _dev(out_logits, "out_logits", torch.bfloat16), out_logits.stride(0),
                                    _dev(out_conf, "out_conf", torch.float32), _dev(dev_status, "dev_status", torch.int32),
                                    _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_markov_logits")


def dspark_markov_draft_step(U: torch.Tensor, W1: torch.Tensor, W2_packed: torch.Tensor, x_prev: torch.Tensor,
                             temperature: float, seed: int, *,
                             H: Optional[torch.Tensor] = None, w_conf: Optional[torch.Tensor] = None,
                             out_logits: torch.Tensor, out_tokens: torch.Tensor,
                             out_conf: Optional[torch.Tensor] = None,
                             dev_status: torch.Tensor, workspace: torch.Tensor) -> None:
    head = _markov_args(U, W1, W2_packed, x_prev, H, w_conf, out_logits, out_conf)
    if out_tokens.numel() < head[5]:
        raise DsparkError("out_tokens is too small")
    rc = lib().dspark_markov_draft_step(*head, float(temperature), int(seed) & (2**64 - 1),
                                        _dev(out_logits, "out_logits", torch.bfloat16), out_logits.stride(0),
                                        _dev(out_tokens, "out_tokens", torch.int32),
                                        _dev(out_conf, "out_conf", torch.float32),
                                        _dev(dev_status, "dev_status", torch.int32),
                                        _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_markov_draft_step")


def dspark_markov_draft_step_stats(U: torch.Tensor, W1: torch.Tensor, W2_packed: torch.Tensor, x_prev: torch.Tensor,
                                   temperature: float, seed: int, *,
                                   H: Optional[torch.Tensor] = None, w_conf: Optional[torch.Tensor] = None,
                                   out_logits: torch.Tensor, out_tokens: torch.Tensor,
                                   out_conf: Optional[torch.Tensor] = None,
                                   out_row_stats: torch.Tensor, row_stats_stride: int = 1,
                                   dev_status: torch.Tensor, workspace: torch.Tensor) -> None:
    """The draft step that also writes (c, Z) of request r's draft row to out_row_stats[r * row_stats_stride] (fp32 pairs)."""
    head = _markov_args(U, W1, W2_packed, x_prev, H, w_conf, out_logits, out_conf)
    R = head[5]
    if out_tokens.numel() < R:
        raise DsparkError("out_tokens is too small")
    if out_row_stats.numel() < 2 * ((R - 1) * int(row_stats_stride) + 1):
        raise DsparkError("out_row_stats is too small")
    rc = lib().dspark_markov_draft_step_stats(*head, float(temperature), int(seed) & (2**64 - 1),
                                              _dev(out_logits, "out_logits", torch.bfloat16), out_logits.stride(0),
                                              _dev(out_tokens, "out_tokens", torch.int32),
                                              _dev(out_conf, "out_conf", torch.float32),
                                              _dev(out_row_stats, "out_row_stats", torch.float32), int(row_stats_stride),
                                              _dev(dev_status, "dev_status", torch.int32),
                                              _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_markov_draft_step_stats")


def dspark_row_stats(logits: torch.Tensor, temperature: float = 1.0, *, row_temperatures: Optional[torch.Tensor] = None,
                     out_row_stats: torch.Tensor) -> None:
    """(c, Z) of every row of `logits` as the verifier computes them: out_row_stats is CUDA float32 [n_rows, 2]."""
    lp, code, ls = _logits(logits, "logits")
    n_rows = logits.shape[0]
    if out_row_stats.numel() < 2 * n_rows or (row_temperatures is not None and row_temperatures.numel() < n_rows):
        raise DsparkError("out_row_stats needs two floats per row, row_temperatures one")
    rc = lib().dspark_row_stats(lp, code, ls, logits.shape[1], n_rows, float(temperature),
                                _dev(row_temperatures, "row_temperatures", torch.float32),
                                _dev(out_row_stats, "out_row_stats", torch.float32), _stream())
    _check(rc, "dspark_row_stats")


def dspark_verify_draft_stats(target: torch.Tensor, draft: torch.Tensor, row_offsets: torch.Tensor,
                              draft_tokens: torch.Tensor, draft_row_stats: torch.Tensor, seed: int, *,
                              temperature: float = 1.0, temperatures: Optional[torch.Tensor] = None,
                              draft_row_start: Optional[torch.Tensor] = None,
                              accepted_len: torch.Tensor, out_tokens: torch.Tensor,
                              out_p_tok: Optional[torch.Tensor] = None, out_q_tok: Optional[torch.Tensor] = None,
                              dev_status: Optional[torch.Tensor], workspace: torch.Tensor,
                              n_rows: Optional[int] = None) -> None:
    """Sampling verification with the draft rows' statistics supplied (CUDA float32 [physical draft rows, 2])."""
    tp, code, ts = _logits(target, "target")
    dp, dcode, ds = _logits(draft, "draft")
    if code != dcode or target.shape[1] != draft.shape[1]:
        raise DsparkError("target and draft logits must share dtype and vocabulary size")
    R = row_offsets.numel() - 1
    if temperatures is not None and temperatures.numel() != R:
        raise DsparkError("temperatures must have one entry per request")
    if draft_row_stats.numel() < 2 * draft.shape[0]:
        raise DsparkError("draft_row_stats needs two floats per draft row")
    n_rows = target.shape[0] if n_rows is None else n_rows
    rc = lib().dspark_verify_draft_stats(
        tp, dp, code, ts, ds, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32),
        _dev(draft_row_start, "draft_row_start", torch.int64), _dev(draft_tokens, "draft_tokens", torch.int32),
        _dev(draft_row_stats, "draft_row_stats", torch.float32), R, n_rows, float(temperature),
        _dev(temperatures, "temperatures", torch.float32), int(seed) & 0xFFFFFFFFFFFFFFFF,
        _dev(accepted_len, "accepted_len", torch.int32), _dev(out_tokens, "out_tokens", torch.int32),
        _dev(out_p_tok, "out_p_tok", torch.float32), _dev(out_q_tok, "out_q_tok", torch.float32),
        _dev(dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_verify_draft_stats")


def dspark_truncate_target(target: torch.Tensor, row_offsets: torch.Tensor, *, top_k: Optional[torch.Tensor] = None,
                           top_p: Optional[torch.Tensor] = None, temperature: float = 1.0,
                           temperatures: Optional[torch.Tensor] = None, out_tau: Optional[torch.Tensor] = None,
                           out_kept: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None) -> None:
    """Masks the excluded tokens of every target row to -inf in place (bf16 or fp32 rows)."""
    tp, code, ts = _logits(target, "target")
    R = row_offsets.numel() - 1
    n_rows = target.shape[0]
    for t, n, name in ((top_k, R, "top_k"), (top_p, R, "top_p"), (temperatures, R, "temperatures"),
                       (out_tau, n_rows, "out_tau"), (out_kept, n_rows, "out_kept")):
        if t is not None and t.numel() < n:
            raise DsparkError(f"{name} is too small")
    rc = lib().dspark_truncate_target(tp, code, ts, target.shape[1], _dev(row_offsets, "row_offsets", torch.int32), R, n_rows,
                                      _dev(top_k, "top_k", torch.int32), _dev(top_p, "top_p", torch.float32),
                                      float(temperature), _dev(temperatures, "temperatures", torch.float32),
                                      _dev(out_tau, "out_tau", torch.float32), _dev(out_kept, "out_kept", torch.int32),
                                      _dev(dev_status, "dev_status", torch.int32), _stream())
    _check(rc, "dspark_truncate_target")


def dspark_sts_workspace_bytes(N: int, gamma: int, G: int, n_bins: int) -> int:
    return int(lib().dspark_sts_workspace_bytes(N, gamma, G, n_bins))


def dspark_sts_calibrate(conf: torch.Tensor, accepted_len: torch.Tensor, grid: torch.Tensor, n_bins: int = 15, *,
                         verified_len: Optional[torch.Tensor] = None, out_T: torch.Tensor,
                         out_ece_before: Optional[torch.Tensor] = None, out_ece_after: Optional[torch.Tensor] = None,
                         out_ece_grid: Optional[torch.Tensor] = None, workspace: torch.Tensor) -> None:
    if conf.dim() != 2 or not conf.is_contiguous():
        raise DsparkError("conf must be a contiguous [N, gamma] tensor")
    N, gamma = conf.shape
    G = grid.numel()
    if accepted_len.numel() < N or out_T.numel() < gamma or (verified_len is not None and verified_len.numel() < N):
        raise DsparkError("accepted_len / verified_len need N entries, out_T gamma")
    for t, n, name in ((out_ece_before, gamma, "out_ece_before"), (out_ece_after, gamma, "out_ece_after"),
                       (out_ece_grid, gamma * G, "out_ece_grid")):
        if t is not None and (t.numel() < n or not t.is_contiguous()):
            raise DsparkError(f"{name} is too small")
    rc = lib().dspark_sts_calibrate(_dev(conf, "conf", torch.float32), N, gamma,
                                    _dev(accepted_len, "accepted_len", torch.int32),
                                    _dev(verified_len, "verified_len", torch.int32), _dev(grid, "grid", torch.float32), G,
                                    int(n_bins), _dev(out_T, "out_T", torch.float32),
                                    _dev(out_ece_before, "out_ece_before", torch.float64),
                                    _dev(out_ece_after, "out_ece_after", torch.float64),
                                    _dev(out_ece_grid, "out_ece_grid", torch.float64), _dev(workspace, "workspace"),
                                    workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "dspark_sts_calibrate")


def dspark_sts_apply(conf: torch.Tensor, T: torch.Tensor, out: torch.Tensor) -> None:
    if conf.dim() != 2 or not conf.is_contiguous() or out.shape != conf.shape or not out.is_contiguous():
        raise DsparkError("conf and out must be contiguous [N, gamma] tensors of one shape")
    if T.numel() < conf.shape[1]:
        raise DsparkError("T needs gamma entries")
    _check(lib().dspark_sts_apply(_dev(conf, "conf", torch.float32), conf.shape[0], conf.shape[1],
                                  _dev(T, "T", torch.float32), _dev(out, "out", torch.float32), _stream()), "dspark_sts_apply")


def dspark_uniforms(seed: int, request: int, position: int):
    a, b = C.c_float(), C.c_float()
    lib().dspark_uniforms(int(seed) & 0xFFFFFFFFFFFFFFFF, request, position, C.byref(a), C.byref(b))
    return a.value, b.value


def dspark_set_stream_path(path: int) -> None:
    _check(lib().dspark_set_stream_path(path), "dspark_set_stream_path")


def dspark_set_wait_poll_limit(polls: int) -> None:
    """Diagnostic: poll limit of the streamed passes' entry waits (0: default, 1: give up at once)."""
    _check(lib().dspark_set_wait_poll_limit(polls), "dspark_set_wait_poll_limit")


class KernelTimer:
    """Per-kernel CUDA-event timing of the library's launches (measurement aid)."""

    def __init__(self, capacity: int):
        h = C.c_void_p()
        _check(lib().dspark_ktimer_create(capacity, C.byref(h)), "dspark_ktimer_create")
        self.handle = h

    def attach(self):
        lib().dspark_ktimer_reset(self.handle)
        lib().dspark_ktimer_attach(self.handle)

    def detach(self):
        lib().dspark_ktimer_attach(None)

    def read(self) -> dict:
        out = {}
        for k in range(K_COUNT):
            ms, n = C.c_float(), C.c_int()
            _check(lib().dspark_ktimer_read(self.handle, k, C.byref(ms), C.byref(n)), "dspark_ktimer_read")
            if n.value:
                out[lib().dspark_kernel_name(k).decode()] = {"ms": ms.value, "launches": n.value}
        return out

    def close(self):
        if self.handle:
            self.detach()
            lib().dspark_ktimer_destroy(self.handle)
            self.handle = None


def workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned scratch buffer (torch allocations are 512-byte aligned)."""
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
