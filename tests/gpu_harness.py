"""Helpers for the GPU parity tests: move host inputs to the device, call the CUDA library through its
binding, bring the outputs back as numpy arrays, and run the oracle on the same inputs."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import compare
import paper_2512_07503_b200 as sjd
from paper_2512_07503_b200 import workloads as wk

DEV = "cuda:0"


def to_device_logits(a: np.ndarray, dtype: int) -> torch.Tensor:
    if a is None:
        return None
    if dtype == wk.BF16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
    if dtype == wk.F16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.float16)
    return torch.from_numpy(a).to(DEV)


def probs_to_device(p: oracle.Probs) -> sjd.DeviceProbs:
    return sjd.DeviceProbs(torch.from_numpy(p.tok_prob).to(DEV), torch.from_numpy(p.ids).to(DEV),
                           torch.from_numpy(p.vals).to(DEV), torch.from_numpy(p.cnt).to(DEV))


class GpuOut:
    def __init__(self, accept_len, tokens, probs: sjd.DeviceProbs, flags, status):
        torch.cuda.synchronize()
        self.accept_len = accept_len.cpu().numpy()
        self.tokens = tokens.cpu().numpy()
        self.tok_prob = probs.tok_prob.cpu().numpy()
        self.ids = probs.ids.cpu().numpy()
        self.vals = probs.vals.cpu().numpy()
        self.cnt = probs.cnt.cpu().numpy()
        self.flags = flags.cpu().numpy()
        self.status = status.cpu().numpy()

    def same_as(self, other: "GpuOut") -> bool:
        # byte comparison: rows beyond win_len keep their (NaN) poison
        return all(getattr(self, n).tobytes() == getattr(other, n).tobytes()
                   for n in ("accept_len", "tokens", "tok_prob", "ids", "vals", "cnt", "flags", "status"))


def gpu_step(cond, uncond, drafts, qprobs, *, dtype, top_k, cfg_scale=1.0, inv_temperature=1.0, reuse_tau=0.5,
             flags=sjd.binding.SJD_FLAG_REUSE, win_len=None, pos_base=None, iteration=None, iteration0=0, seed=0,
             poison=True) -> GpuOut:
    """One sjd_step through the binding on host inputs.  Outputs start poisoned so that anything the
    kernels fail to write shows up."""
    c = to_device_logits(cond, dtype)
    u = to_device_logits(uncond, dtype)
    B, W, V = c.shape
    kcap = min(top_k, V)
    out = sjd.DeviceProbs.empty(B, W, kcap, DEV)
    acc = torch.zeros(B, dtype=torch.int32, device=DEV)
    toks = torch.zeros(B, W, dtype=torch.int32, device=DEV)
    oflags = torch.zeros(B, W, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    if poison:
        for t in (out.ids, out.cnt, acc, toks, oflags, status):
            t.fill_(-7)
        out.vals.fill_(float("nan"))
        out.tok_prob.fill_(float("nan"))
    dev_i32 = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)
    wl_, pb_, it_ = dev_i32(win_len), dev_i32(pos_base), dev_i32(iteration)
    params = sjd.make_params(c, top_k=top_k, cfg_scale=cfg_scale, inv_temperature=float(inv_temperature),
                             reuse_tau=reuse_tau, flags=flags, iteration0=iteration0, win_len=wl_, pos_base=pb_,
                             iteration=it_, out_flags=oflags, status=status)
    ws = torch.empty(sjd.sjd_workspace_bytes(params), dtype=torch.uint8, device=DEV)
    params.workspace = ws.data_ptr()
    params.workspace_bytes = ws.numel()
    d = dev_i32(drafts)
    q = probs_to_device(qprobs) if qprobs is not None else None
    sjd.sjd_step(c, u, d, q, params, seed, acc, toks, out)
    return GpuOut(acc, toks, out, oflags, status)


def step_kwargs(inp: wk.StepInputs, **over):
    wl = inp.wl
    kw = dict(dtype=wl.dtype, top_k=wl.top_k, cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature),
              reuse_tau=wl.reuse_tau, flags=(oracle.FLAG_REUSE if wl.reuse else 0), win_len=inp.win_len,
              pos_base=inp.pos_base, iteration0=inp.iteration, seed=wl.seed)
    kw.update(over)
    return kw


def oracle_prime(inp: wk.StepInputs, n_threads=8) -> oracle.StepResult:
    kw = step_kwargs(inp, flags=oracle.FLAG_DRAFT_ALL, iteration0=inp.iteration - 1)
    return oracle.sjd_step(inp.prev_cond, inp.prev_uncond, None, None, V=inp.wl.V, n_threads=n_threads, diag=True, **kw)


def check_parity(cond, uncond, drafts, qprobs, kw, win_len, *, expect_flagged_below=2e-3, n_threads=8):
    """Run both sides on the same inputs, compare, and return (report, gpu_out, oracle_result)."""
    V = cond.shape[-1]
    ref = oracle.sjd_step(cond, uncond, drafts, qprobs, V=V, n_threads=n_threads, diag=True, **kw)
    got = gpu_step(cond, uncond, drafts, qprobs, **kw)
    again = gpu_step(cond, uncond, drafts, qprobs, **kw)
    assert got.same_as(again), "two runs on the same inputs differ: a race in the kernels"
    rep = compare.compare_step(got.accept_len, got.tokens, got.tok_prob, got.flags, got.ids, got.vals, got.cnt, ref,
                               drafts, win_len, kw["flags"])
    assert rep.ok(), rep.summary() + "\n" + "\n".join(rep.errors)
    # bit 16 only says that a row took the any-shape path inside the library: no counterpart in the oracle
    assert np.array_equal(got.status & ~16, ref.status), (got.status, ref.status)
    # decisions within 1e-6 of their boundary may fall on either side; they are rare, and rare in every category
    allowed = max(2, int(expect_flagged_below * rep.positions))
    for what, n in (("accept", rep.flagged_accept), ("reuse", rep.flagged_reuse), ("sample", rep.flagged_sample)):
        assert n <= allowed, (what, rep.summary())
    return rep, got, ref
