"""Decode loop on the device: sjd_step + sjd_window_advance per Jacobi iteration, with every buffer
allocated once.  The model's forward pass is a callable that maps the current window to cond / uncond
logits on the device.  Marshalling only: all arithmetic runs in the library's kernels.

With ``use_graphs=True`` the four kernels of an iteration are captured once per buffer parity into a CUDA
graph and replayed, which removes the host's launch work from the critical path of small windows; the
logits then have to sit in the loop's own buffers (``cond_buf`` / ``uncond_buf``; other tensors are copied
there)."""
from __future__ import annotations

from typing import Callable, Optional, Tuple

import torch

from . import binding as B


class DecodeLoop:
    def __init__(self, *, batch: int, window: int, vocab: int, n_total: int, logits_dtype: torch.dtype, top_k: int,
                 cfg_scale: float = 1.0, inv_temperature: float = 1.0, reuse_tau: float = 0.5, reuse: bool = True,
                 seed: int = 0, seq_base: int = 0, init_mode: int = B.SJD_INIT_RANDOM, grid_width: int = 1,
                 use_graphs: bool = False, guidance: bool = True, refine: bool = True, device="cuda:0"):
        self.B, self.W, self.V, self.N = batch, window, vocab, n_total
        self.kcap = min(top_k, vocab)
        self.seed, self.device = seed, torch.device(device)
        dev = self.device
        i32 = dict(dtype=torch.int32, device=dev)
        self.win_len = torch.full((batch,), min(window, n_total), **i32)
        self.pos_base = torch.zeros(batch, **i32)
        self.iteration = torch.zeros(batch, **i32)
        self.committed = torch.full((batch, n_total), -1, **i32)
        self.n_committed = torch.zeros(batch, **i32)
        self.drafts = [torch.zeros(batch, window, **i32) for _ in range(2)]
        self.q = [B.DeviceProbs.empty(batch, window, self.kcap, dev) for _ in range(2)]
        self.out = B.DeviceProbs.empty(batch, window, self.kcap, dev)
        self.acc = torch.zeros(batch, **i32)
        self.toks = torch.zeros(batch, window, **i32)
        self.status = torch.zeros(batch, **i32)
        self.cur = 0
        proto = torch.empty(batch, window, vocab, dtype=logits_dtype, device=dev)
        self.params = B.make_params(proto, top_k=top_k, cfg_scale=cfg_scale, inv_temperature=inv_temperature,
                                    reuse_tau=reuse_tau,
                                    flags=(B.SJD_FLAG_REUSE if reuse else 0) | (0 if refine else B.SJD_FLAG_NO_REFINE),
                                    win_len=self.win_len,
                                    pos_base=self.pos_base, iteration=self.iteration, status=self.status,
                                    seq_base=seq_base, init_mode=init_mode, grid_width=grid_width)
        del proto
        self.use_graphs = use_graphs
        self.graphs = [None, None]   # one per buffer parity
        self.eager_done = [False, False]
        if use_graphs:
            self.cond_buf = torch.empty(batch, window, vocab, dtype=logits_dtype, device=dev)
            self.uncond_buf = torch.empty_like(self.cond_buf) if guidance else None
        self.ws = torch.empty(B.sjd_workspace_bytes(self.params), dtype=torch.uint8, device=dev)
        self.params.workspace, self.params.workspace_bytes = self.ws.data_ptr(), self.ws.numel()
        B.sjd_window_init(self.params, n_total, seed, self.win_len, self.pos_base, self.iteration, self.drafts[0], self.q[0])
        self.steps = 0

    @property
    def window_tokens(self) -> torch.Tensor:
        return self.drafts[self.cur]

    def _launch(self, cond, uncond, c: int) -> None:
        n = c ^ 1
        p = self.params
        p.stride_b, p.stride_w = cond.stride(0), cond.stride(1)
        p.stream = torch.cuda.current_stream(self.device).cuda_stream
        B.sjd_step(cond, uncond, self.drafts[c], self.q[c], p, self.seed, self.acc, self.toks, self.out)
        B.sjd_window_advance(p, self.N, self.seed, self.acc, self.toks, self.out, self.win_len, self.pos_base,
                             self.iteration, self.drafts[n], self.q[n], self.committed, self.n_committed)

    def step(self, cond: torch.Tensor, uncond: Optional[torch.Tensor]) -> None:
        """One Jacobi iteration on logits [B,W,V] for the current window (asynchronous)."""
        c = self.cur
        if not self.use_graphs:
            self._launch(cond, uncond, c)
        else:
            if (uncond is None) != (self.uncond_buf is None):
                raise B.SjdError("guidance must match the loop's `guidance` setting when graphs are used")
            if cond.data_ptr() != self.cond_buf.data_ptr():
                self.cond_buf.copy_(cond)
            if uncond is not None and uncond.data_ptr() != self.uncond_buf.data_ptr():
                self.uncond_buf.copy_(uncond)
            if not self.eager_done[c]:
                # first use of this parity: an ordinary launch (it also performs the one-time kernel set-up)
                self._launch(self.cond_buf, self.uncond_buf, c)
                self.eager_done[c] = True
            else:
                if self.graphs[c] is None:
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        self._launch(self.cond_buf, self.uncond_buf, c)
                    self.graphs[c] = g
                self.graphs[c].replay()
        self.cur = c ^ 1
        self.steps += 1

    def done(self) -> bool:
        """True when every sequence is complete.  This is the loop's one synchronisation point per iteration: the
        status words of the last step come back with it, and a step whose on-chip wait gave up (its outputs are
        invalid, and the window was advanced on them) raises here instead of passing unnoticed."""
        state = torch.stack([(self.win_len != 0).any().to(torch.int32),
                             (self.status & B.SJD_STATUS_INTERNAL_TIMEOUT).any().to(torch.int32)]).cpu()
        if int(state[1]) != 0:
            raise B.SjdError("a step reported SJD_STATUS_INTERNAL_TIMEOUT: its outputs are invalid")
        return int(state[0]) == 0

    def run(self, logit_source: Callable[["DecodeLoop"], Tuple[torch.Tensor, Optional[torch.Tensor]]],
            max_steps: Optional[int] = None):
        """Iterate until every sequence is complete.  Returns (committed tokens, steps, committed counts per step)."""
        history = []
        while not self.done():
            if max_steps is not None and self.steps >= max_steps:
                break
            cond, uncond = logit_source(self)
            self.step(cond, uncond)
            history.append(self.n_committed.clone())
        counts = torch.stack(history).cpu() if history else torch.zeros(0, self.B, dtype=torch.int32)
        return self.committed.cpu(), self.steps, counts
