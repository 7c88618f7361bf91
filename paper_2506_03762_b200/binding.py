"""Thin ctypes binding of libahakv.so: same names as the C ABI, argument marshalling only.

Every step of the eviction path runs in the library's CUDA kernels; PyTorch is
used here for device memory and streams.  There is no CPU fallback: if the
shared library is missing, loading fails with an error that says how to build it.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libahakv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, F16, BF16 = 0, 1, 2
SCALE_FIXED, SCALE_ADAPTIVE_ROW, SCALE_ADAPTIVE_CALL = 0, 1, 2
FLAG_VALUE_PRIOR, FLAG_POOL_ZERO_PAD, FLAG_GROUP_MAX = 1, 2, 4

DTYPE_CODE = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}
CODE_DTYPE = {v: k for k, v in DTYPE_CODE.items()}


class AhakvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class CParams(ctypes.Structure):
    """Mirror of ``ahakv_params``."""
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("n_ctx", ctypes.c_int32), ("n_total", ctypes.c_int64),
        ("obs_window", ctypes.c_int32), ("recent_window", ctypes.c_int32), ("budget", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("scale_mode", ctypes.c_int32), ("scale", ctypes.c_float),
        ("pool_kernel", ctypes.c_int32), ("flags", ctypes.c_uint32),
        ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3), ("v_stride", ctypes.c_int64 * 3),
    ]


class CSeq(ctypes.Structure):
    """Mirror of ``ahakv_seq``."""
    _fields_ = [("n_ctx", ctypes.c_int32), ("budget", ctypes.c_int32), ("n_total", ctypes.c_int64)]


@dataclass
class Params:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_ctx: int
    obs_window: int
    recent_window: int
    budget: int
    dtype: int = F16
    n_total: int | None = None           # None: prefill, n_total = n_ctx
    scale_mode: int = SCALE_ADAPTIVE_ROW
    scale: float = 0.0
    pool_kernel: int = 7
    flags: int = FLAG_VALUE_PRIOR
    q_stride: tuple = field(default=(0, 0, 0))
    k_stride: tuple = field(default=(0, 0, 0))
    v_stride: tuple = field(default=(0, 0, 0))

    def c(self) -> CParams:
        nt = self.n_ctx if self.n_total is None else self.n_total
        return CParams(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.n_ctx, nt,
                       self.obs_window, self.recent_window, self.budget, self.dtype, self.scale_mode,
                       float(self.scale), self.pool_kernel, self.flags,
                       (ctypes.c_int64 * 3)(*self.q_stride), (ctypes.c_int64 * 3)(*self.k_stride),
                       (ctypes.c_int64 * 3)(*self.v_stride))

    @property
    def n_keep(self) -> int:
        return min(self.n_ctx, self.budget)


_lib = None
_vp, _sz = ctypes.c_void_p, ctypes.c_size_t
_PP = ctypes.POINTER(CParams)

SIGNATURES = {
    "ahakv_workspace_bytes": (_sz, [_PP]),
    "ahakv_lambda": (ctypes.c_double, [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]),
    "ahakv_score": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_score_rows": (ctypes.c_int, [_PP, ctypes.POINTER(ctypes.c_int64), _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_score_full_causal": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_score_step": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp]),
    "ahakv_compact_inplace": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp]),
    "ahakv_step_slots": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "ahakv_entropy_workspace_bytes": (_sz, [_PP]),
    "ahakv_row_entropy": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_select": (ctypes.c_int, [_PP, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_compact": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "ahakv_evict": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_evict_head_budgets": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_evict_ragged": (ctypes.c_int, [_PP, ctypes.POINTER(CSeq), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "ahakv_score_static": (ctypes.c_int, [_PP, _vp, _vp, _vp, _vp, _vp, _vp]),
    "ahakv_static_workspace_bytes": (_sz, []),
    "ahakv_static_last_device_status": (ctypes.c_int, [_vp]),
    "ahakv_last_device_status": (ctypes.c_int, [_vp, _vp]),
    "ahakv_test_set_wait": (None, [ctypes.c_int32, ctypes.c_int32]),
    "ahakv_launch_count": (ctypes.c_int64, []),
    "ahakv_profile_enable": (ctypes.c_int, [ctypes.c_int]),
    "ahakv_profile_read": (ctypes.c_int64, [ctypes.POINTER(ctypes.c_double)]),
    "ahakv_stage_name": (ctypes.c_char_p, [ctypes.c_int]),
    "ahakv_status_string": (ctypes.c_char_p, [ctypes.c_int]),
}


def lib():
    """The loaded C library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_03762_b200.build` "
                "(needs nvcc). This package has no CPU fallback.")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().ahakv_status_string(int(status)).decode()


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _raise(status: int, where: str):
    if status != OK:
        raise AhakvError(status, where)


def ahakv_workspace_bytes(p: Params) -> int:
    cp = p.c()
    return int(lib().ahakv_workspace_bytes(ctypes.byref(cp)))


def ahakv_lambda(n_total: int, budget: int, head_dim: int) -> float:
    return float(lib().ahakv_lambda(n_total, budget, head_dim))


def ahakv_test_set_wait(wait_ms: int, withhold_first_partial: bool) -> None:
    lib().ahakv_test_set_wait(int(wait_ms), 1 if withhold_first_partial else 0)


def ahakv_launch_count() -> int:
    return int(lib().ahakv_launch_count())


def ahakv_score(p: Params, q_obs, k, v, score_prev, score, ws, ws_bytes: int | None = None, stream=None,
                check: bool = True) -> int:
    cp = p.c()
    nbytes = ws.numel() * ws.element_size() if ws_bytes is None else ws_bytes
    st = lib().ahakv_score(ctypes.byref(cp), _ptr(q_obs), _ptr(k), _ptr(v), _ptr(score_prev), _ptr(score),
                           _ptr(ws), nbytes, _stream(stream))
    if check:
        _raise(st, "ahakv_score")
    return st


def ahakv_score_rows(p: Params, obs_pos, q_obs, k, v, score_prev, score, ws, ws_bytes: int | None = None,
                     stream=None, check: bool = True) -> int:
    """``ahakv_score`` with the observation rows at the given logical positions (a host sequence of r ints)."""
    cp = p.c()
    pos = None if obs_pos is None else (ctypes.c_int64 * len(obs_pos))(*[int(x) for x in obs_pos])
    nbytes = ws.numel() * ws.element_size() if ws_bytes is None else ws_bytes
    st = lib().ahakv_score_rows(ctypes.byref(cp), pos, _ptr(q_obs), _ptr(k), _ptr(v), _ptr(score_prev),
                                _ptr(score), _ptr(ws), nbytes, _stream(stream))
    if check:
        _raise(st, "ahakv_score_rows")
    return st


def ahakv_score_full_causal(p: Params, q_all, k, v, score_prev, score, ws, ws_bytes: int | None = None,
                            stream=None, check: bool = True) -> int:
    """Accumulation over all query rows (Eq. 2-3); ``p.obs_window`` rows per pass."""
    cp = p.c()
    nbytes = ws.numel() * ws.element_size() if ws_bytes is None else ws_bytes
    st = lib().ahakv_score_full_causal(ctypes.byref(cp), _ptr(q_all), _ptr(k), _ptr(v), _ptr(score_prev),
                                       _ptr(score), _ptr(ws), nbytes, _stream(stream))
    if check:
        _raise(st, "ahakv_score_full_causal")
    return st


def ahakv_score_step(p: Params, q_t, k, score_prev, score, stream=None, check: bool = True) -> int:
    cp = p.c()
    st = lib().ahakv_score_step(ctypes.byref(cp), _ptr(q_t), _ptr(k), _ptr(score_prev), _ptr(score), _stream(stream))
    if check:
        _raise(st, "ahakv_score_step")
    return st


def ahakv_compact_inplace(p: Params, k, v, score, kept_idx, stream=None, check: bool = True) -> int:
    cp = p.c()
    st = lib().ahakv_compact_inplace(ctypes.byref(cp), _ptr(k), _ptr(v), _ptr(score), _ptr(kept_idx), _stream(stream))
    if check:
        _raise(st, "ahakv_compact_inplace")
    return st


def ahakv_step_slots(p: Params, q_t, k_t, v_t, k, v, score, pos, free_slot, stream=None, check: bool = True) -> int:
    cp = p.c()
    st = lib().ahakv_step_slots(ctypes.byref(cp), _ptr(q_t), _ptr(k_t), _ptr(v_t), _ptr(k), _ptr(v), _ptr(score),
                                _ptr(pos), _ptr(free_slot), _stream(stream))
    if check:
        _raise(st, "ahakv_step_slots")
    return st


def ahakv_row_entropy(p: Params, q_obs, k, entropy=None, stream=None):
    """Eq. 6 entropy [B,Hq,r] (float32) of every observation row; allocates its scratch and, if not given, the output."""
    cp = p.c()
    nbytes = int(lib().ahakv_entropy_workspace_bytes(ctypes.byref(cp)))
    if nbytes == 0:
        raise AhakvError(ERR_INVALID_ARG, "ahakv_entropy_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=k.device)
    if entropy is None:
        entropy = torch.empty((p.batch, p.n_q_heads, p.obs_window), dtype=torch.float32, device=k.device)
    _raise(lib().ahakv_row_entropy(ctypes.byref(cp), _ptr(q_obs), _ptr(k), _ptr(entropy), _ptr(ws), nbytes,
                                   _stream(stream)), "ahakv_row_entropy")
    return entropy


def ahakv_static_workspace_bytes() -> int:
    return int(lib().ahakv_static_workspace_bytes())


def ahakv_static_last_device_status(stream=None) -> int:
    return int(lib().ahakv_static_last_device_status(_stream(stream)))


def ahakv_score_static(p: Params, q_obs, k, v, score_prev, score, stream=None, check: bool = True) -> int:
    """``ahakv_score`` on the library's own fixed scratch array: no workspace argument, no allocation."""
    cp = p.c()
    st = lib().ahakv_score_static(ctypes.byref(cp), _ptr(q_obs), _ptr(k), _ptr(v), _ptr(score_prev),
                                  _ptr(score), _stream(stream))
    if check:
        _raise(st, "ahakv_score_static")
    return st


def ahakv_select(p: Params, score, kept_idx, ws=None, ws_bytes: int | None = None, stream=None,
                 check: bool = True) -> int:
    cp = p.c()
    nbytes = (0 if ws is None else ws.numel() * ws.element_size()) if ws_bytes is None else ws_bytes
    st = lib().ahakv_select(ctypes.byref(cp), _ptr(score), _ptr(kept_idx), _ptr(ws), nbytes, _stream(stream))
    if check:
        _raise(st, "ahakv_select")
    return st


def ahakv_compact(p: Params, k, v, score, kept_idx, k_out, v_out, score_out, stream=None,
                  check: bool = True) -> int:
    cp = p.c()
    st = lib().ahakv_compact(ctypes.byref(cp), _ptr(k), _ptr(v), _ptr(score), _ptr(kept_idx), _ptr(k_out),
                             _ptr(v_out), _ptr(score_out), _stream(stream))
    if check:
        _raise(st, "ahakv_compact")
    return st


def ahakv_evict(p: Params, q_obs, k, v, score_prev, k_out, v_out, score_out, kept_idx, ws,
                ws_bytes: int | None = None, stream=None, check: bool = True) -> int:
    cp = p.c()
    nbytes = ws.numel() * ws.element_size() if ws_bytes is None else ws_bytes
    st = lib().ahakv_evict(ctypes.byref(cp), _ptr(q_obs), _ptr(k), _ptr(v), _ptr(score_prev), _ptr(k_out),
                           _ptr(v_out), _ptr(score_out), _ptr(kept_idx), _ptr(ws), nbytes, _stream(stream))
    if check:
        _raise(st, "ahakv_evict")
    return st


def ahakv_evict_head_budgets(p: Params, head_budget, q_obs, k, v, score_prev, k_out, v_out, score_out, kept_idx, ws,
                             ws_bytes: int | None = None, stream=None, check: bool = True) -> int:
    """``ahakv_evict`` with ``head_budget`` [B,Hkv] int32 on the device: a budget per (sequence, KV head)."""
    cp = p.c()
    nbytes = ws.numel() * ws.element_size() if ws_bytes is None else ws_bytes
    st = lib().ahakv_evict_head_budgets(ctypes.byref(cp), _ptr(head_budget), _ptr(q_obs), _ptr(k), _ptr(v),
                                        _ptr(score_prev), _ptr(k_out), _ptr(v_out), _ptr(score_out), _ptr(kept_idx),
                                        _ptr(ws), nbytes, _stream(stream))
    if check:
        _raise(st, "ahakv_evict_head_budgets")
    return st


def ahakv_evict_ragged(p: Params, seqs, q_obs, k, v, score_prev, k_out, v_out, score_out, kept_idx, ws,
                       ws_bytes: int | None = None, stream=None, check: bool = True) -> int:
    """``seqs``: one (n_ctx, budget, n_total) triple per sequence."""
    cp = p.c()
    arr = (CSeq * len(seqs))(*[CSeq(int(a), int(b), int(c)) for a, b, c in seqs])
    nbytes = ws.numel() * ws.element_size() if ws_bytes is None else ws_bytes
    st = lib().ahakv_evict_ragged(ctypes.byref(cp), arr, _ptr(q_obs), _ptr(k), _ptr(v), _ptr(score_prev), _ptr(k_out),
                                  _ptr(v_out), _ptr(score_out), _ptr(kept_idx), _ptr(ws), nbytes, _stream(stream))
    if check:
        _raise(st, "ahakv_evict_ragged")
    return st


def ahakv_last_device_status(ws, stream=None) -> int:
    return int(lib().ahakv_last_device_status(_ptr(ws), _stream(stream)))


N_STAGES = 5


def ahakv_profile_enable(on: bool) -> None:
    _raise(lib().ahakv_profile_enable(1 if on else 0), "ahakv_profile_enable")


def ahakv_profile_read():
    """(calls, {stage name: total milliseconds}) since the last read; synchronises the device."""
    ms = (ctypes.c_double * N_STAGES)()
    calls = int(lib().ahakv_profile_read(ms))
    return calls, {lib().ahakv_stage_name(t).decode(): ms[t] for t in range(N_STAGES)}


# ---- convenience for callers that hold torch tensors -------------------------------------------

def params_for(q_obs: torch.Tensor, k: torch.Tensor, *, recent_window: int, budget: int,
               n_total: int | None = None, **kw) -> Params:
    """Params for dense q_obs [B,Hq,r,d] and k [B,Hkv,n,d]."""
    B, Hq, r, d = q_obs.shape
    _, Hkv, n, _ = k.shape
    return Params(B, Hq, Hkv, d, n, r, recent_window, budget, dtype=DTYPE_CODE[k.dtype], n_total=n_total, **kw)


def alloc_workspace(p: Params, device="cuda") -> torch.Tensor:
    nbytes = ahakv_workspace_bytes(p)
    if nbytes == 0:
        raise AhakvError(ERR_INVALID_ARG, "ahakv_workspace_bytes")
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def alloc_outputs(p: Params, device="cuda"):
    """(k_out, v_out, score_out, kept_idx) with the shapes the C ABI writes."""
    dt = CODE_DTYPE[p.dtype]
    shape = (p.batch, p.n_kv_heads, p.n_keep)
    return (torch.empty(shape + (p.head_dim,), dtype=dt, device=device),
            torch.empty(shape + (p.head_dim,), dtype=dt, device=device),
            torch.empty(shape, dtype=torch.float32, device=device),
            torch.empty(shape, dtype=torch.int32, device=device))
