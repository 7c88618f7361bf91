"""ctypes front end of the AhaKV eviction oracle -- TEST INFRASTRUCTURE.

The arithmetic lives in ``ahakv_oracle.cpp`` (plain double-precision C++ that
follows the paper's Eq. 1, 5, 9, 12-15 and Algorithm 1 step by step).  This
module only marshals numpy arrays into it.  Nothing in the product package may
import this file; it imports nothing from the product package either.

Arrays: ``q_obs [B,Hq,r,d]``, ``k, v [B,Hkv,n,d]`` as numpy float32, float16 or
uint16 holding bfloat16 bits (``dtype='bf16'``).  Scores are float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ahakv_oracle.cpp")
_LIB = os.path.join(_HERE, "libahakv_oracle.so")

F32, F16, BF16 = 0, 1, 2
SCALE_FIXED, SCALE_ADAPTIVE_ROW, SCALE_ADAPTIVE_CALL = 0, 1, 2
FLAG_VALUE_PRIOR, FLAG_POOL_ZERO_PAD, FLAG_GROUP_MAX = 1, 2, 4


def build(force: bool = False) -> str:
    """Compile the oracle with g++ when the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", _LIB, _SRC])
    return _LIB


class _Params(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("n_ctx", ctypes.c_int32), ("n_total", ctypes.c_int64),
        ("obs_window", ctypes.c_int32), ("recent_window", ctypes.c_int32), ("budget", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("scale_mode", ctypes.c_int32), ("scale", ctypes.c_double),
        ("pool_kernel", ctypes.c_int32), ("flags", ctypes.c_uint32),
        ("obs_pos", ctypes.POINTER(ctypes.c_int64)),
    ]


@dataclass
class OracleParams:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_ctx: int
    obs_window: int
    recent_window: int
    budget: int
    dtype: int = F32
    n_total: int | None = None          # None: prefill, n_total = n_ctx
    scale_mode: int = SCALE_ADAPTIVE_ROW
    scale: float = 0.0
    pool_kernel: int = 7
    flags: int = FLAG_VALUE_PRIOR
    obs_pos: object = None              # None: the last r positions; else r ascending logical positions

    def c(self) -> _Params:
        nt = self.n_ctx if self.n_total is None else self.n_total
        pos = None
        if self.obs_pos is not None:
            arr = np.ascontiguousarray(self.obs_pos, np.int64)
            if arr.shape != (self.obs_window,):
                raise ValueError("obs_pos must hold obs_window positions")
            self._pos_keepalive = arr               # the C struct only borrows the pointer
            pos = arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))
        return _Params(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.n_ctx, nt,
                       self.obs_window, self.recent_window, self.budget, self.dtype, self.scale_mode,
                       float(self.scale), self.pool_kernel, self.flags, pos)

    @property
    def n_keep(self) -> int:
        return min(self.n_ctx, self.budget)


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.ahakv_oracle_lambda.restype = ctypes.c_double
        _lib.ahakv_oracle_lambda.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_inputs(p: OracleParams, q_obs, k, v):
    want = {F32: np.float32, F16: np.float16, BF16: np.uint16}[p.dtype]
    for name, a, shape in (("q_obs", q_obs, (p.batch, p.n_q_heads, p.obs_window, p.head_dim)),
                           ("k", k, (p.batch, p.n_kv_heads, p.n_ctx, p.head_dim)),
                           ("v", v, (p.batch, p.n_kv_heads, p.n_ctx, p.head_dim))):
        if a is None:
            continue
        if a.dtype != want or tuple(a.shape) != shape or not a.flags.c_contiguous:
            raise ValueError(f"{name}: want contiguous {want.__name__}{shape}, got {a.dtype}{a.shape}")


def _rc(rc: int):
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (code {rc})")


def eq12_lambda(n_total: int, budget: int, head_dim: int) -> float:
    """Eq. 12: sqrt(2 ln(i/k) / d)."""
    return lib().ahakv_oracle_lambda(n_total, budget, head_dim)


def attention(p: OracleParams, q_obs, k, b: int, hq: int) -> np.ndarray:
    """SG-softmax matrix [r, n] of query head (b, hq); masked columns are 0."""
    _check_inputs(p, q_obs, k, None)
    out = np.empty((p.obs_window, p.n_ctx), np.float64)
    cp = p.c()
    _rc(lib().ahakv_oracle_attention(ctypes.byref(cp), _ptr(q_obs), _ptr(k), b, hq, _ptr(out)))
    return out


def row_entropy(p: OracleParams, q_obs, k, b: int, hq: int) -> np.ndarray:
    """Eq. 6 entropy of each observation row of query head (b, hq)."""
    _check_inputs(p, q_obs, k, None)
    out = np.empty((p.obs_window,), np.float64)
    cp = p.c()
    _rc(lib().ahakv_oracle_row_entropy(ctypes.byref(cp), _ptr(q_obs), _ptr(k), b, hq, _ptr(out)))
    return out


def score(p: OracleParams, q_obs, k, v, score_prev=None, nthreads: int = 0, return_raw: bool = False):
    """Refined eviction score [B,Hkv,n] (float64); optionally also the score before Eq. 15."""
    _check_inputs(p, q_obs, k, v)
    shape = (p.batch, p.n_kv_heads, p.n_ctx)
    if score_prev is not None:
        score_prev = np.ascontiguousarray(score_prev, np.float64).reshape(shape)
    out = np.empty(shape, np.float64)
    raw = np.empty(shape, np.float64) if return_raw else None
    cp = p.c()
    _rc(lib().ahakv_oracle_score(ctypes.byref(cp), _ptr(q_obs), _ptr(k), _ptr(v), _ptr(score_prev),
                                 _ptr(raw), _ptr(out), nthreads))
    return (out, raw) if return_raw else out


def select(p: OracleParams, score_arr) -> np.ndarray:
    """Kept indices [B,Hkv,n_keep] int32, ascending: recent window plus TopK of the rest."""
    s = np.ascontiguousarray(score_arr, np.float64).reshape(p.batch, p.n_kv_heads, p.n_ctx)
    out = np.empty((p.batch, p.n_kv_heads, p.n_keep), np.int32)
    cp = p.c()
    _rc(lib().ahakv_oracle_select(ctypes.byref(cp), _ptr(s), _ptr(out)))
    return out


def compact(p: OracleParams, k, v, kept_idx, score_arr=None):
    """Gather rows kept_idx of K and V (and of the score): returns (k_out, v_out, score_out)."""
    _check_inputs(p, None, k, v)
    idx = np.ascontiguousarray(kept_idx, np.int32).reshape(p.batch, p.n_kv_heads, p.n_keep)
    k_out = np.empty((p.batch, p.n_kv_heads, p.n_keep, p.head_dim), k.dtype)
    v_out = np.empty_like(k_out)
    s = s_out = None
    if score_arr is not None:
        s = np.ascontiguousarray(score_arr, np.float64).reshape(p.batch, p.n_kv_heads, p.n_ctx)
        s_out = np.empty((p.batch, p.n_kv_heads, p.n_keep), np.float64)
    cp = p.c()
    _rc(lib().ahakv_oracle_compact(ctypes.byref(cp), _ptr(k), _ptr(v), _ptr(s), _ptr(idx), _ptr(k_out),
                                   _ptr(v_out), _ptr(s_out)))
    return k_out, v_out, s_out


def evict(p: OracleParams, q_obs, k, v, score_prev=None, nthreads: int = 0):
    """score -> select -> compact.  Returns dict(k_out, v_out, score_out, kept_idx, score)."""
    _check_inputs(p, q_obs, k, v)
    shape = (p.batch, p.n_kv_heads, p.n_ctx)
    if score_prev is not None:
        score_prev = np.ascontiguousarray(score_prev, np.float64).reshape(shape)
    k_out = np.empty((p.batch, p.n_kv_heads, p.n_keep, p.head_dim), k.dtype)
    v_out = np.empty_like(k_out)
    s_out = np.empty((p.batch, p.n_kv_heads, p.n_keep), np.float64)
    idx = np.empty((p.batch, p.n_kv_heads, p.n_keep), np.int32)
    full = np.empty(shape, np.float64)
    cp = p.c()
    _rc(lib().ahakv_oracle_evict(ctypes.byref(cp), _ptr(q_obs), _ptr(k), _ptr(v), _ptr(score_prev),
                                 _ptr(k_out), _ptr(v_out), _ptr(s_out), _ptr(idx), _ptr(full), nthreads))
    return dict(k_out=k_out, v_out=v_out, score_out=s_out, kept_idx=idx, score=full)
