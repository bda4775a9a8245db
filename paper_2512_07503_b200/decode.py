"""Decode loop on the device: sjd_step + sjd_window_advance per Jacobi iteration, with every buffer
allocated once.  The model's forward pass is a callable that maps the current window to cond / uncond
logits on the device.  Marshalling only: all arithmetic runs in the library's kernels."""
from __future__ import annotations

from typing import Callable, Optional, Tuple

import torch

from . import binding as B


class DecodeLoop:
    def __init__(self, *, batch: int, window: int, vocab: int, n_total: int, logits_dtype: torch.dtype, top_k: int,
                 cfg_scale: float = 1.0, inv_temperature: float = 1.0, reuse_tau: float = 0.5, reuse: bool = True,
                 seed: int = 0, seq_base: int = 0, init_mode: int = B.SJD_INIT_RANDOM, grid_width: int = 1,
                 device="cuda:0"):
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
                                    reuse_tau=reuse_tau, flags=(B.SJD_FLAG_REUSE if reuse else 0), win_len=self.win_len,
                                    pos_base=self.pos_base, iteration=self.iteration, status=self.status,
                                    seq_base=seq_base, init_mode=init_mode, grid_width=grid_width)
        del proto
        self.ws = torch.empty(B.sjd_workspace_bytes(self.params), dtype=torch.uint8, device=dev)
        self.params.workspace, self.params.workspace_bytes = self.ws.data_ptr(), self.ws.numel()
        B.sjd_window_init(self.params, n_total, seed, self.win_len, self.pos_base, self.iteration, self.drafts[0], self.q[0])
        self.steps = 0

    @property
    def window_tokens(self) -> torch.Tensor:
        return self.drafts[self.cur]

    def step(self, cond: torch.Tensor, uncond: Optional[torch.Tensor]) -> None:
        """One Jacobi iteration on logits [B,W,V] for the current window (asynchronous)."""
        c, n = self.cur, self.cur ^ 1
        p = self.params
        p.stride_b, p.stride_w = cond.stride(0), cond.stride(1)
        B.sjd_step(cond, uncond, self.drafts[c], self.q[c], p, self.seed, self.acc, self.toks, self.out)
        B.sjd_window_advance(p, self.N, self.seed, self.acc, self.toks, self.out, self.win_len, self.pos_base,
                             self.iteration, self.drafts[n], self.q[n], self.committed, self.n_committed)
        self.cur = n
        self.steps += 1

    def done(self) -> bool:
        return bool((self.win_len == 0).all().item())

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
