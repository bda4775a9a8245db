"""The allocation-free entry point against the ordinary one.

``sjd_step_static`` exists for hosts that may not allocate device memory where they call the library (an
allocator frozen after start-up, a memory pool owned by someone else): it takes its scratch from a fixed
array inside the library instead of a caller-supplied workspace.  It runs the same kernels, so every
output must equal ``sjd_step``'s bit for bit (and, like it, agree with the CPU oracle); two calls in a row
check that what the first call left in the shared array does not leak into the second.  This file sorts
last on purpose: a run that stops at
the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare
import paper_2512_07503_b200 as sjd
from paper_2512_07503_b200 import workloads as wk

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _device_inputs(wl):
    inp = wk.make_step_inputs(wl)
    kw = dict(dtype=wl.dtype, V=wl.V, cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature),
              top_k=wl.top_k, win_len=inp.win_len, pos_base=inp.pos_base, seed=wl.seed, n_threads=8)
    prev = oracle.sjd_step(inp.prev_cond, inp.prev_uncond, None, None, flags=oracle.FLAG_DRAFT_ALL, iteration0=0, **kw)

    def up(a):
        if wl.dtype == wk.BF16:
            return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
        return torch.from_numpy(a).to(DEV)

    q = sjd.DeviceProbs(*(torch.from_numpy(a).to(DEV) for a in (prev.probs.tok_prob, prev.probs.ids, prev.probs.vals,
                                                                prev.probs.cnt)))
    # what the oracle makes of the same step, for the comparison with the allocation-free entry point
    ref = oracle.sjd_step(inp.cond, inp.uncond, prev.tokens, prev.probs, flags=oracle.FLAG_REUSE, iteration0=1,
                          reuse_tau=wl.reuse_tau, diag=True, **kw)
    return dict(cond=up(inp.cond), uncond=up(inp.uncond), drafts=torch.from_numpy(prev.tokens).to(DEV), q=q,
                win_len=torch.from_numpy(inp.win_len).to(DEV), pos_base=torch.from_numpy(inp.pos_base).to(DEV),
                ref=ref, host_drafts=prev.tokens, host_win_len=inp.win_len)


def _run(entry, wl, d, with_workspace):
    out = sjd.DeviceProbs.empty(wl.B, wl.W, wl.kcap, DEV)
    acc = torch.full((wl.B,), -7, dtype=torch.int32, device=DEV)
    toks = torch.full((wl.B, wl.W), -7, dtype=torch.int32, device=DEV)
    flags = torch.full((wl.B, wl.W), -7, dtype=torch.int32, device=DEV)
    status = torch.full((wl.B,), -7, dtype=torch.int32, device=DEV)
    p = sjd.make_params(d["cond"], top_k=wl.top_k, cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature),
                        reuse_tau=wl.reuse_tau, flags=sjd.binding.SJD_FLAG_REUSE, iteration0=1, win_len=d["win_len"],
                        pos_base=d["pos_base"], out_flags=flags, status=status)
    ws = None
    if with_workspace:
        ws = torch.empty(sjd.sjd_workspace_bytes(p), dtype=torch.uint8, device=DEV)
        p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel()
    entry(d["cond"], d["uncond"], d["drafts"], d["q"], p, wl.seed, acc, toks, out)
    torch.cuda.synchronize()
    return [t.cpu().numpy() for t in (acc, toks, flags, status, out.tok_prob, out.ids, out.vals, out.cnt)]


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    # first call: fp32, ragged windows; second call: bf16, larger vocabulary, other row count
    first = wk.CONFIGS["cfg3"].scaled(B=6, V=4096, top_k=200)
    second = wk.CONFIGS["cfg2"].scaled(B=2, W=5, V=8192, top_k=500)
    for wl in (first, second, first):
        d = _device_inputs(wl)
        want = _run(sjd.sjd_step, wl, d, with_workspace=True)
        got = _run(sjd.sjd_step_static, wl, d, with_workspace=False)
        for a, b in zip(got, want):
            assert a.tobytes() == b.tobytes()
        assert (got[0] >= 0).all() and (got[0] <= wl.W).all()
        acc, toks, flags, status, tok_prob, ids, vals, cnt = got
        rep = compare.compare_step(acc, toks, tok_prob, flags, ids, vals, cnt, d["ref"], d["host_drafts"],
                                   d["host_win_len"], oracle.FLAG_REUSE)
        assert rep.ok(), rep.summary() + "\n" + "\n".join(rep.errors)


def test_static_scratch_refuses_what_does_not_fit():
    rows_over = sjd.binding.SJD_STATIC_MAX_ROWS // 512 + 1   # B * 512 rows: one sequence too many
    logits = torch.zeros(rows_over, 512, 8, device=DEV)
    out = sjd.DeviceProbs.empty(rows_over, 512, 8, DEV)
    acc = torch.zeros(rows_over, dtype=torch.int32, device=DEV)
    toks = torch.zeros(rows_over, 512, dtype=torch.int32, device=DEV)
    p = sjd.make_params(logits, top_k=8, flags=sjd.binding.SJD_FLAG_DRAFT_ALL)
    with pytest.raises(sjd.SjdError, match="sjd error -8"):
        sjd.sjd_step_static(logits, None, None, None, p, 0, acc, toks, out)
    torch.cuda.synchronize()
