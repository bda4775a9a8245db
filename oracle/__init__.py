"""ctypes access to the CPU oracle (``sjd_oracle.cpp``).

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg import this package.  It never imports the CUDA library's binding and the
CUDA library never imports it.  The shared object is compiled on first use with g++.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sjd_oracle.cpp")
_HDR = os.path.join(_HERE, "sjd_oracle.h")
_SO = os.path.join(_HERE, "libsjd_oracle.so")

F32, BF16, F16 = 0, 1, 2
FLAG_REUSE, FLAG_DRAFT_ALL = 1, 2
PURPOSE_ACCEPT, PURPOSE_RESIDUAL, PURPOSE_REDRAFT, PURPOSE_INIT = 0, 1, 2, 3
OUT_INVALID, OUT_ACCEPTED, OUT_RESIDUAL, OUT_REUSED, OUT_RESAMPLED = 0, 1, 2, 3, 4
STATUS_QTOK_NONPOSITIVE, STATUS_EMPTY_RESIDUAL, STATUS_DEGENERATE_ROW = 1, 2, 4
Q_UNIFORM = -1


def build(force: bool = False) -> str:
    """Compile the oracle's shared object when it is missing or older than its sources."""
    stale = force or not os.path.exists(_SO) or os.path.getmtime(_SO) < max(
        os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if stale:
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC",
                               _SRC, "-o", tmp, "-lpthread"])
        os.replace(tmp, _SO)
    return _SO


class _Probs(C.Structure):
    _fields_ = [("tok_prob", C.c_void_p), ("ids", C.c_void_p), ("vals", C.c_void_p), ("cnt", C.c_void_p)]


class _Params(C.Structure):
    _fields_ = [("B", C.c_int32), ("W", C.c_int32), ("V", C.c_int32), ("logits_dtype", C.c_int32),
                ("stride_b", C.c_int64), ("stride_w", C.c_int64), ("cfg_scale", C.c_float),
                ("inv_temperature", C.c_float), ("top_k", C.c_int32), ("reuse_tau", C.c_float),
                ("flags", C.c_int32), ("win_len", C.c_void_p), ("pos_base", C.c_void_p),
                ("iteration", C.c_void_p), ("iteration0", C.c_int32), ("n_threads", C.c_int32), ("seq_base", C.c_int32)]


class _Diag(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("u", "ratio", "accept_margin", "reuse_margin", "pot_ok", "pot_reuse",
                                          "pot_redraft", "redraft_margin", "pot_residual", "residual_margin")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_philox4x32_10.restype = None
        L.orc_uniform24.argtypes = [C.c_uint32]
        L.orc_uniform24.restype = C.c_float
        L.orc_half_to_float.argtypes = [C.c_uint16]
        L.orc_half_to_float.restype = C.c_float
        L.orc_row_probs.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_float,
                                    C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_row_probs.restype = C.c_int32
        L.orc_accept.argtypes = [C.c_float, C.c_float, C.c_float, C.c_void_p]
        L.orc_accept.restype = C.c_int32
        L.orc_first_reject.argtypes = [C.c_void_p, C.c_int32]
        L.orc_first_reject.restype = C.c_int32
        L.orc_icdf.argtypes = [C.c_void_p, C.c_int32, C.c_uint64, C.c_void_p]
        L.orc_icdf.restype = C.c_int32
        L.orc_residual_weights.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                           C.c_int32, C.c_void_p]
        L.orc_residual_weights.restype = None
        L.orc_sjd_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_sjd_step.restype = C.c_int32
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


def half_to_float(bits: int) -> float:
    return float(lib().orc_half_to_float(int(bits) & 0xFFFF))


def uniform24(x: int) -> float:
    return float(lib().orc_uniform24(int(x) & 0xFFFFFFFF))


def _logits_view(a, dtype):
    """Raw host array the oracle reads: float32, or the uint16 patterns of bf16."""
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if dtype in (BF16, F16):
        assert a.dtype == np.uint16, "16-bit logits are passed as their uint16 bit patterns"
    else:
        assert a.dtype == np.float32
    return a


def row_probs(cond, uncond, dtype, cfg_scale, inv_temperature, top_k):
    """Distribution of one row.  Returns (ids int32[kcap], vals float32[kcap], degenerate)."""
    cond = _logits_view(cond, dtype)
    uncond = _logits_view(uncond, dtype)
    V = cond.shape[-1]
    kcap = min(top_k, V)
    ids = np.zeros(kcap, dtype=np.int32)
    vals = np.zeros(kcap, dtype=np.float32)
    dg = np.zeros(1, dtype=np.int32)
    n = lib().orc_row_probs(_ptr(cond), _ptr(uncond), dtype, V, cfg_scale, inv_temperature, top_k, ids.ctypes.data,
                            vals.ctypes.data, dg.ctypes.data)
    assert n == kcap, n
    return ids, vals, int(dg[0])


def accept(p_tok, q_tok, u):
    r = np.zeros(1, dtype=np.float32)
    ok = lib().orc_accept(p_tok, q_tok, u, r.ctypes.data)
    return int(ok), float(r[0])


def first_reject(ok) -> int:
    ok = np.ascontiguousarray(ok, dtype=np.int32)
    return int(lib().orc_first_reject(ok.ctypes.data, ok.shape[0]))


def icdf(w, R):
    w = np.ascontiguousarray(w, dtype=np.float32)
    m = np.zeros(1, dtype=np.float32)
    k = lib().orc_icdf(w.ctypes.data, w.shape[0], int(R) & 0xFFFFFFFFFFFFFFFF, m.ctypes.data)
    return int(k), float(m[0])


def residual_weights(p_ids, p_vals, q_ids, q_vals, q_cnt, V):
    p_ids = np.ascontiguousarray(p_ids, dtype=np.int32)
    p_vals = np.ascontiguousarray(p_vals, dtype=np.float32)
    q_ids = np.ascontiguousarray(q_ids, dtype=np.int32)
    q_vals = np.ascontiguousarray(q_vals, dtype=np.float32)
    w = np.zeros(p_ids.shape[0], dtype=np.float32)
    lib().orc_residual_weights(p_ids.ctypes.data, p_vals.ctypes.data, p_ids.shape[0], q_ids.ctypes.data,
                               q_vals.ctypes.data, q_cnt, V, w.ctypes.data)
    return w


@dataclass
class Probs:
    """A set of per-position sparse distributions on the host (numpy)."""
    tok_prob: np.ndarray  # [B,W] float32
    ids: np.ndarray       # [B,W,kcap] int32
    vals: np.ndarray      # [B,W,kcap] float32
    cnt: np.ndarray       # [B,W] int32

    @staticmethod
    def empty(B, W, kcap):
        return Probs(np.zeros((B, W), np.float32), np.zeros((B, W, kcap), np.int32),
                     np.zeros((B, W, kcap), np.float32), np.zeros((B, W), np.int32))

    @staticmethod
    def uniform(B, W, kcap, V):
        p = Probs.empty(B, W, kcap)
        p.cnt[:] = Q_UNIFORM
        p.tok_prob[:] = np.float32(1.0) / np.float32(V)
        return p

    def _c(self):
        for a in (self.tok_prob, self.ids, self.vals, self.cnt):
            assert a.flags["C_CONTIGUOUS"]
        return _Probs(self.tok_prob.ctypes.data, self.ids.ctypes.data, self.vals.ctypes.data, self.cnt.ctypes.data)


@dataclass
class StepResult:
    accept_len: np.ndarray
    tokens: np.ndarray
    probs: Probs
    flags: np.ndarray
    status: np.ndarray
    diag: dict = field(default_factory=dict)


_DIAG_F = ("u", "ratio", "accept_margin", "reuse_margin", "redraft_margin", "residual_margin")
_DIAG_I = ("pot_ok", "pot_reuse", "pot_redraft", "pot_residual")


def sjd_step(logits_cond, logits_uncond, drafts, draft_probs, *, dtype, V, cfg_scale=1.0, inv_temperature=1.0,
             top_k, reuse_tau=0.5, flags=FLAG_REUSE, win_len=None, pos_base=None, iteration=None, iteration0=0,
             seed=0, n_threads=1, diag=False, seq_base=0) -> StepResult:
    """One verify-and-redraft step on host arrays shaped [B,W,V] (contiguous)."""
    cond = _logits_view(logits_cond, dtype)
    unc = _logits_view(logits_uncond, dtype)
    B, W = cond.shape[0], cond.shape[1]
    assert cond.shape[2] == V
    kcap = min(top_k, V)
    out = Probs.empty(B, W, kcap)
    acc = np.zeros(B, np.int32)
    toks = np.zeros((B, W), np.int32)
    oflags = np.zeros((B, W), np.int32)
    status = np.zeros(B, np.int32)
    keep = []

    def opt_i32(a):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=np.int32)
        keep.append(a)
        return a.ctypes.data

    P = _Params(B, W, V, dtype, W * V, V, cfg_scale, inv_temperature, top_k, reuse_tau, flags, opt_i32(win_len),
                opt_i32(pos_base), opt_i32(iteration), iteration0, n_threads, seq_base)
    d = {}
    dstruct = None
    if diag:
        for n in _DIAG_F:
            d[n] = np.full((B, W), np.inf, np.float32)
        for n in _DIAG_I:
            d[n] = np.full((B, W), -1, np.int32)
        dstruct = _Diag(*[d[n].ctypes.data for n, _ in _Diag._fields_])
    if drafts is not None:
        drafts = np.ascontiguousarray(drafts, dtype=np.int32)
    qs = draft_probs._c() if draft_probs is not None else None
    os_ = out._c()
    rc = lib().orc_sjd_step(_ptr(cond), _ptr(unc), _ptr(drafts), C.byref(qs) if qs is not None else None, C.byref(P),
                            int(seed) & 0xFFFFFFFFFFFFFFFF, acc.ctypes.data, toks.ctypes.data, C.byref(os_),
                            oflags.ctypes.data, status.ctypes.data, C.byref(dstruct) if dstruct is not None else None)
    if rc != 0:
        raise ValueError(f"orc_sjd_step failed with {rc}")
    return StepResult(acc, toks, out, oflags, status, d)
