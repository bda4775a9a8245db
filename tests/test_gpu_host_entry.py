"""The host-buffer entry point (sjd_step_host: copies in, kernels, copies out) against the CPU oracle, on
pageable and on pinned host arrays: every output, including the per-position flags and the status words."""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare
import paper_2512_07503_b200 as sjd
from paper_2512_07503_b200 import workloads as wk

pytestmark = pytest.mark.gpu


def _host(a, pin):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return t.pin_memory() if pin else t


def _logits(a, dtype, pin):
    if dtype == wk.F32:
        return _host(a, pin)
    t = _host(a.view(np.int16), pin)
    return t.view(torch.bfloat16 if dtype == wk.BF16 else torch.float16)


@pytest.mark.parametrize("pin", [False, True], ids=["pageable", "pinned"])
@pytest.mark.parametrize("name,B", [("cfg1", None), ("cfg2", None), ("cfg3", 8)])
def test_host_entry_point_matches_the_oracle(name, B, pin):
    from gpu_harness import oracle_prime, step_kwargs
    wl = wk.CONFIGS[name] if B is None else wk.CONFIGS[name].scaled(B=B)
    inp = wk.make_step_inputs(wl)
    prev = oracle_prime(inp, n_threads=8)
    kw = step_kwargs(inp)
    ref = oracle.sjd_step(inp.cond, inp.uncond, prev.tokens, prev.probs, V=wl.V, n_threads=8, diag=True, **kw)

    Bn, W, kcap = wl.B, wl.W, wl.kcap
    ctx = sjd.HostContext(Bn, W, wl.V, wl.dtype, wl.top_k, device="cuda:0")
    h_cond, h_unc = _logits(inp.cond, wl.dtype, pin), _logits(inp.uncond, wl.dtype, pin)
    h_drafts = _host(prev.tokens.astype(np.int32), pin)
    h_q = sjd.HostProbs(_host(prev.probs.tok_prob, pin), _host(prev.probs.ids, pin), _host(prev.probs.vals, pin),
                        _host(prev.probs.cnt, pin))
    h_out = sjd.HostProbs.empty(Bn, W, kcap, pin=pin)
    mk = lambda shape: (torch.full(shape, -7, dtype=torch.int32).pin_memory() if pin
                        else torch.full(shape, -7, dtype=torch.int32))
    h_acc, h_tok, h_flags, h_status = mk((Bn,)), mk((Bn, W)), mk((Bn, W)), mk((Bn,))
    h_out.ids.fill_(-7)
    h_out.cnt.fill_(-7)
    h_out.vals.fill_(float("nan"))
    h_out.tok_prob.fill_(float("nan"))
    h_win, h_pos = _host(inp.win_len.astype(np.int32), pin), _host(inp.pos_base.astype(np.int32), pin)
    p = ctx.params(cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature), reuse_tau=wl.reuse_tau,
                   flags=kw["flags"], iteration0=inp.iteration, win_len=h_win, pos_base=h_pos, out_flags=h_flags,
                   status=h_status)
    sjd.sjd_step_host(ctx, h_cond, h_unc, h_drafts, h_q, p, wl.seed, h_acc, h_tok, h_out)
    ctx.close()

    rep = compare.compare_step(h_acc.numpy(), h_tok.numpy(), h_out.tok_prob.numpy(), h_flags.numpy(), h_out.ids.numpy(),
                               h_out.vals.numpy(), h_out.cnt.numpy(), ref, prev.tokens, inp.win_len, kw["flags"])
    assert rep.ok(), rep.summary() + "\n" + "\n".join(rep.errors)
    assert rep.positions == int(inp.win_len.sum())
    # bit 16 only says that a row took the any-shape path inside the library: no counterpart in the oracle
    assert np.array_equal(h_status.numpy() & ~16, ref.status), (h_status.numpy(), ref.status)
