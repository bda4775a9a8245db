"""Thin ctypes binding of the C ABI in ``include/sjd.h``.

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch is used
for device memory and streams.  There is no CPU fallback: if the shared library cannot be built or
loaded, importing a symbol from it raises.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

SJD_F32, SJD_BF16, SJD_F16 = 0, 1, 2
SJD_FLAG_REUSE, SJD_FLAG_DRAFT_ALL, SJD_FLAG_FORCE_GENERIC, SJD_FLAG_FORCE_TILES, SJD_FLAG_NO_REFINE = 1, 2, 4, 8, 16
SJD_Q_UNIFORM = -1
SJD_INIT_RANDOM, SJD_INIT_REPEAT_LEFT, SJD_INIT_REPEAT_ABOVE, SJD_INIT_SAMPLE_LEFT, SJD_INIT_SAMPLE_ABOVE = 0, 1, 2, 3, 4
SJD_OUT_INVALID, SJD_OUT_ACCEPTED, SJD_OUT_RESIDUAL, SJD_OUT_REUSED, SJD_OUT_RESAMPLED = 0, 1, 2, 3, 4
SJD_STATUS_QTOK_NONPOSITIVE, SJD_STATUS_EMPTY_RESIDUAL, SJD_STATUS_DEGENERATE_ROW = 1, 2, 4
SJD_STATUS_INTERNAL_TIMEOUT, SJD_STATUS_ROW_REDONE = 8, 16
SJD_W_MAX = 512


class sjd_probs(C.Structure):
    _fields_ = [("tok_prob", C.c_void_p), ("ids", C.c_void_p), ("vals", C.c_void_p), ("cnt", C.c_void_p)]


class sjd_params(C.Structure):
    _fields_ = [("struct_size", C.c_int32), ("B", C.c_int32), ("W", C.c_int32), ("V", C.c_int32),
                ("logits_dtype", C.c_int32), ("stride_b", C.c_int64), ("stride_w", C.c_int64),
                ("cfg_scale", C.c_float), ("inv_temperature", C.c_float), ("top_k", C.c_int32),
                ("reuse_tau", C.c_float), ("flags", C.c_int32), ("iteration0", C.c_int32), ("seq_base", C.c_int32),
                ("win_len", C.c_void_p), ("pos_base", C.c_void_p), ("iteration", C.c_void_p),
                ("out_flags", C.c_void_p), ("status", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p), ("ev_rows_begin", C.c_void_p),
                ("ev_rows_end", C.c_void_p), ("init_mode", C.c_int32), ("grid_width", C.c_int32)]


class SjdError(RuntimeError):
    pass


_lib = None


def lib() -> C.CDLL:
    """The loaded CUDA library; built in-tree with nvcc when missing or stale.  Raises when that fails."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.sjd_version.restype = C.c_int
        L.sjd_status_string.argtypes = [C.c_int]
        L.sjd_status_string.restype = C.c_char_p
        L.sjd_last_cuda_error.restype = C.c_char_p
        L.sjd_launch_count.restype = C.c_uint64
        L.sjd_workspace_bytes.argtypes = [C.POINTER(sjd_params)]
        L.sjd_workspace_bytes.restype = C.c_size_t
        L.sjd_row_kernel.argtypes = [C.POINTER(sjd_params)]
        L.sjd_row_kernel.restype = C.c_int
        L.sjd_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(sjd_probs), C.POINTER(sjd_params),
                               C.c_uint64, C.c_void_p, C.c_void_p, C.POINTER(sjd_probs)]
        L.sjd_step.restype = C.c_int
        L.sjd_step_static.argtypes = L.sjd_step.argtypes
        L.sjd_step_static.restype = C.c_int
        L.sjd_window_init.argtypes = [C.POINTER(sjd_params), C.c_int32, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.POINTER(sjd_probs)]
        L.sjd_window_init.restype = C.c_int
        L.sjd_window_advance.argtypes = [C.POINTER(sjd_params), C.c_int32, C.c_uint64, C.c_void_p, C.c_void_p,
                                         C.POINTER(sjd_probs), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.POINTER(sjd_probs), C.c_void_p, C.c_void_p]
        L.sjd_window_advance.restype = C.c_int
        _lib = L
    return _lib


def sjd_version() -> int:
    return int(lib().sjd_version())


def sjd_launch_count() -> int:
    return int(lib().sjd_launch_count())


def sjd_status_string(code: int) -> str:
    return lib().sjd_status_string(int(code)).decode()


def _check(code: int) -> None:
    if code != 0:
        extra = lib().sjd_last_cuda_error().decode()
        raise SjdError(f"sjd error {code}: {sjd_status_string(code)}" + (f" ({extra})" if extra else ""))


@dataclass
class DeviceProbs:
    """Device arrays of one ``sjd_probs``: tok_prob [B,W] f32, ids [B,W,kcap] i32, vals [B,W,kcap] f32, cnt [B,W] i32."""
    tok_prob: torch.Tensor
    ids: torch.Tensor
    vals: torch.Tensor
    cnt: torch.Tensor

    @staticmethod
    def empty(B: int, W: int, kcap: int, device) -> "DeviceProbs":
        return DeviceProbs(torch.zeros(B, W, dtype=torch.float32, device=device),
                           torch.zeros(B, W, kcap, dtype=torch.int32, device=device),
                           torch.zeros(B, W, kcap, dtype=torch.float32, device=device),
                           torch.zeros(B, W, dtype=torch.int32, device=device))

    @staticmethod
    def uniform(B: int, W: int, kcap: int, V: int, device) -> "DeviceProbs":
        p = DeviceProbs.empty(B, W, kcap, device)
        p.cnt.fill_(SJD_Q_UNIFORM)
        p.tok_prob.fill_(1.0 / V)
        return p

    def c_struct(self) -> sjd_probs:
        for t, dt in ((self.tok_prob, torch.float32), (self.ids, torch.int32), (self.vals, torch.float32),
                      (self.cnt, torch.int32)):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == dt):
                raise SjdError("sjd_probs arrays must be contiguous CUDA tensors of the documented dtypes")
        return sjd_probs(self.tok_prob.data_ptr(), self.ids.data_ptr(), self.vals.data_ptr(), self.cnt.data_ptr())


def _opt_ptr(t: Optional[torch.Tensor], dtype=torch.int32) -> Optional[int]:
    if t is None:
        return None
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise SjdError("optional arrays must be contiguous CUDA tensors of the documented dtype")
    return t.data_ptr()


SJD_ROWS_GENERIC, SJD_ROWS_TILES, SJD_ROWS_RANGES = 0, 1, 2


def sjd_row_kernel(params: "sjd_params") -> int:
    """Which row kernel sjd_step() takes for these parameters (SJD_ROWS_*)."""
    code = lib().sjd_row_kernel(C.byref(params))
    if code < 0:
        _check(code)
    return code


def make_params(logits: torch.Tensor, *, top_k: int, cfg_scale: float = 1.0, inv_temperature: float = 1.0,
                reuse_tau: float = 0.5, flags: int = SJD_FLAG_REUSE, iteration0: int = 0,
                win_len: Optional[torch.Tensor] = None, pos_base: Optional[torch.Tensor] = None,
                iteration: Optional[torch.Tensor] = None, out_flags: Optional[torch.Tensor] = None,
                status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                stream: Optional[torch.cuda.Stream] = None, seq_base: int = 0, init_mode: int = 0,
                grid_width: int = 1) -> sjd_params:
    """Fill an ``sjd_params`` from a [B,W,V] logits tensor (fp32, bf16 or fp16, vocabulary axis contiguous)."""
    if logits.dim() != 3 or logits.stride(2) != 1:
        raise SjdError("logits must be [B,W,V] with a contiguous vocabulary axis")
    if logits.dtype == torch.float32:
        dt = SJD_F32
    elif logits.dtype == torch.bfloat16:
        dt = SJD_BF16
    elif logits.dtype == torch.float16:
        dt = SJD_F16
    else:
        raise SjdError("logits must be float32, bfloat16 or float16")
    B, W, V = logits.shape
    p = sjd_params()
    p.struct_size = C.sizeof(sjd_params)
    p.B, p.W, p.V = B, W, V
    p.logits_dtype = dt
    p.stride_b, p.stride_w = logits.stride(0), logits.stride(1)
    p.cfg_scale = cfg_scale
    p.inv_temperature = inv_temperature
    p.top_k = top_k
    p.reuse_tau = reuse_tau
    p.flags = flags
    p.iteration0 = iteration0
    p.seq_base = seq_base
    p.init_mode = init_mode
    p.grid_width = grid_width
    p.win_len = _opt_ptr(win_len)
    p.pos_base = _opt_ptr(pos_base)
    p.iteration = _opt_ptr(iteration)
    p.out_flags = _opt_ptr(out_flags)
    p.status = _opt_ptr(status)
    if workspace is not None:
        p.workspace = workspace.data_ptr()
        p.workspace_bytes = workspace.numel() * workspace.element_size()
    s = stream if stream is not None else torch.cuda.current_stream(logits.device)
    p.stream = s.cuda_stream
    # the struct only holds raw addresses: keep the tensors alive as long as the struct lives
    p._keepalive = (win_len, pos_base, iteration, out_flags, status, workspace, s)
    return p


def sjd_workspace_bytes(params: sjd_params) -> int:
    return int(lib().sjd_workspace_bytes(C.byref(params)))


def _check_logits(logits_cond: torch.Tensor, logits_uncond: Optional[torch.Tensor]) -> None:
    """What both device entry points ask of the two logits tensors (the C side sees only pointers)."""
    if not logits_cond.is_cuda:
        raise SjdError("logits must live on a CUDA device")
    if logits_uncond is not None and (logits_uncond.shape != logits_cond.shape or
                                      logits_uncond.stride() != logits_cond.stride() or
                                      logits_uncond.dtype != logits_cond.dtype or
                                      logits_uncond.device != logits_cond.device):
        raise SjdError("cond and uncond logits must share shape, strides, dtype and device")


def sjd_step(logits_cond: torch.Tensor, logits_uncond: Optional[torch.Tensor], drafts: Optional[torch.Tensor],
             draft_probs: Optional[DeviceProbs], params: sjd_params, philox_seed: int, out_accept_len: torch.Tensor,
             out_tokens: torch.Tensor, out_probs: DeviceProbs) -> None:
    """Enqueue one verify-and-redraft step on ``params.stream``.  Same arguments as the C entry point."""
    _check_logits(logits_cond, logits_uncond)
    q = draft_probs.c_struct() if draft_probs is not None else None
    o = out_probs.c_struct()
    with torch.cuda.device(logits_cond.device):
        code = lib().sjd_step(logits_cond.data_ptr(), None if logits_uncond is None else logits_uncond.data_ptr(),
                              _opt_ptr(drafts), C.byref(q) if q is not None else None, C.byref(params),
                              int(philox_seed) & 0xFFFFFFFFFFFFFFFF, _opt_ptr(out_accept_len), _opt_ptr(out_tokens),
                              C.byref(o))
    _check(code)


def sjd_window_init(params: sjd_params, n_total: int, philox_seed: int, win_len: torch.Tensor, pos_base: torch.Tensor,
                    iteration: torch.Tensor, drafts: torch.Tensor, draft_probs: DeviceProbs) -> None:
    """Fill the first window with randomly initialised drafts (uniform reference distribution)."""
    q = draft_probs.c_struct()
    with torch.cuda.device(drafts.device):
        code = lib().sjd_window_init(C.byref(params), int(n_total), int(philox_seed) & 0xFFFFFFFFFFFFFFFF,
                                     _opt_ptr(win_len), _opt_ptr(pos_base), _opt_ptr(iteration), _opt_ptr(drafts),
                                     C.byref(q))
    _check(code)


def sjd_window_advance(params: sjd_params, n_total: int, philox_seed: int, accept_len: torch.Tensor,
                       step_tokens: torch.Tensor, step_probs: DeviceProbs, win_len: torch.Tensor, pos_base: torch.Tensor,
                       iteration: torch.Tensor, next_drafts: torch.Tensor, next_probs: DeviceProbs,
                       committed: torch.Tensor, n_committed: Optional[torch.Tensor] = None) -> None:
    """Commit the accepted prefix and the residual token, shift the window and refill it (same arguments as
    the C entry point)."""
    sp, nq = step_probs.c_struct(), next_probs.c_struct()
    with torch.cuda.device(step_tokens.device):
        code = lib().sjd_window_advance(C.byref(params), int(n_total), int(philox_seed) & 0xFFFFFFFFFFFFFFFF,
                                        _opt_ptr(accept_len), _opt_ptr(step_tokens), C.byref(sp), _opt_ptr(win_len),
                                        _opt_ptr(pos_base), _opt_ptr(iteration), _opt_ptr(next_drafts), C.byref(nq),
                                        _opt_ptr(committed), _opt_ptr(n_committed))
    _check(code)


SJD_STATIC_MAX_ROWS = 16384


def sjd_step_static(logits_cond: torch.Tensor, logits_uncond: Optional[torch.Tensor], drafts: Optional[torch.Tensor],
                    draft_probs: Optional[DeviceProbs], params: sjd_params, philox_seed: int,
                    out_accept_len: torch.Tensor, out_tokens: torch.Tensor, out_probs: DeviceProbs) -> None:
    """``sjd_step`` without a caller-supplied workspace, for hosts that may not allocate device memory where
    they call the library (a frozen allocator, a pool they do not own).  The scratch is a fixed array inside
    the library, good for B*W <= SJD_STATIC_MAX_ROWS; larger problems raise.  ``params.workspace`` is ignored.
    Calls on one device share that array: do not let two of them overlap on the GPU."""
    _check_logits(logits_cond, logits_uncond)
    q = draft_probs.c_struct() if draft_probs is not None else None
    o = out_probs.c_struct()
    with torch.cuda.device(logits_cond.device):
        code = lib().sjd_step_static(logits_cond.data_ptr(),
                                     None if logits_uncond is None else logits_uncond.data_ptr(), _opt_ptr(drafts),
                                     C.byref(q) if q is not None else None, C.byref(params),
                                     int(philox_seed) & 0xFFFFFFFFFFFFFFFF, _opt_ptr(out_accept_len),
                                     _opt_ptr(out_tokens), C.byref(o))
    _check(code)


# ----------------------------------------------------------------------------------------------------
# host-buffer variant
# ----------------------------------------------------------------------------------------------------
@dataclass
class HostProbs:
    """Host (CPU, ideally pinned) arrays of one ``sjd_probs``."""
    tok_prob: torch.Tensor
    ids: torch.Tensor
    vals: torch.Tensor
    cnt: torch.Tensor

    @staticmethod
    def empty(B: int, W: int, kcap: int, pin: bool = True) -> "HostProbs":
        mk = lambda shape, dt: torch.zeros(shape, dtype=dt, pin_memory=pin)
        return HostProbs(mk((B, W), torch.float32), mk((B, W, kcap), torch.int32), mk((B, W, kcap), torch.float32),
                         mk((B, W), torch.int32))

    def c_struct(self) -> sjd_probs:
        for t in (self.tok_prob, self.ids, self.vals, self.cnt):
            if t.is_cuda or not t.is_contiguous():
                raise SjdError("host sjd_probs arrays must be contiguous CPU tensors")
        return sjd_probs(self.tok_prob.data_ptr(), self.ids.data_ptr(), self.vals.data_ptr(), self.cnt.data_ptr())

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.tok_prob, self.ids, self.vals, self.cnt))


def _host_ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise SjdError("host arrays must be contiguous CPU tensors")
    return t.data_ptr()


class HostContext:
    """Owner of an ``sjd_host_ctx`` (device mirrors for one shape on the current device)."""

    def __init__(self, B: int, W: int, V: int, logits_dtype: int, top_k: int, device=None):
        L = lib()
        L.sjd_host_ctx_create.argtypes = [C.POINTER(sjd_params), C.POINTER(C.c_void_p)]
        L.sjd_host_ctx_create.restype = C.c_int
        L.sjd_step_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(sjd_probs),
                                    C.POINTER(sjd_params), C.c_uint64, C.c_void_p, C.c_void_p, C.POINTER(sjd_probs)]
        L.sjd_step_host.restype = C.c_int
        L.sjd_host_ctx_destroy.argtypes = [C.c_void_p]
        L.sjd_host_ctx_destroy.restype = None
        self.shape = (B, W, V, logits_dtype, top_k)
        self.device = torch.device(device if device is not None else "cuda:0")
        p = sjd_params()
        p.struct_size = C.sizeof(sjd_params)
        p.B, p.W, p.V, p.logits_dtype, p.top_k = B, W, V, logits_dtype, top_k
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(L.sjd_host_ctx_create(C.byref(p), C.byref(h)))
        self._h = h

    def close(self) -> None:
        if getattr(self, "_h", None):
            with torch.cuda.device(self.device):
                lib().sjd_host_ctx_destroy(self._h)
            self._h = None

    __del__ = close

    def params(self, *, cfg_scale=1.0, inv_temperature=1.0, reuse_tau=0.5, flags=SJD_FLAG_REUSE, iteration0=0,
               win_len=None, pos_base=None, iteration=None, out_flags=None, status=None, seq_base=0) -> sjd_params:
        B, W, V, dt, top_k = self.shape
        p = sjd_params()
        p.struct_size = C.sizeof(sjd_params)
        p.B, p.W, p.V, p.logits_dtype, p.top_k = B, W, V, dt, top_k
        p.stride_b, p.stride_w = W * V, V
        p.cfg_scale, p.inv_temperature, p.reuse_tau, p.flags, p.iteration0 = (cfg_scale, inv_temperature, reuse_tau,
                                                                               flags, iteration0)
        p.seq_base = seq_base
        p.win_len, p.pos_base, p.iteration = _host_ptr(win_len), _host_ptr(pos_base), _host_ptr(iteration)
        p.out_flags, p.status = _host_ptr(out_flags), _host_ptr(status)
        return p


def sjd_step_host(ctx: HostContext, logits_cond: torch.Tensor, logits_uncond: Optional[torch.Tensor],
                  drafts: Optional[torch.Tensor], draft_probs: Optional[HostProbs], params: sjd_params,
                  philox_seed: int, out_accept_len: torch.Tensor, out_tokens: torch.Tensor,
                  out_probs: HostProbs) -> None:
    """Host-buffer step: copies in, runs the kernels, copies out; the host arrays are ready on return."""
    q = draft_probs.c_struct() if draft_probs is not None else None
    o = out_probs.c_struct()
    with torch.cuda.device(ctx.device):
        code = lib().sjd_step_host(ctx._h, _host_ptr(logits_cond), _host_ptr(logits_uncond), _host_ptr(drafts),
                                   C.byref(q) if q is not None else None, C.byref(params),
                                   int(philox_seed) & 0xFFFFFFFFFFFFFFFF, _host_ptr(out_accept_len),
                                   _host_ptr(out_tokens), C.byref(o))
    _check(code)
