"""GPU parity on the wider shapes around the headline configuration: the paper's window sizes (16 to 512), the
top-K values of its sampling ablation and the vocabularies of the models it accelerates.  Same checks as
the full-size tests, at a reduced batch so that the oracle stays within seconds per case."""
import numpy as np
import pytest

from paper_2512_07503_b200 import workloads as wk

pytestmark = pytest.mark.gpu

CASES = [("w16", 6), ("w32", 4), ("w96", 2), ("w250", 1), ("w512", 1), ("k1", 2), ("k10", 2), ("k100", 2), ("k500", 2),
         ("k1000", 2), ("k8192", 1), ("v32k", 3), ("v16k", 4), ("v16k_f32", 4), ("f16", 3), ("hetero", 4)]


@pytest.mark.parametrize("name,B", CASES)
def test_sweep_shape_matches_the_oracle(name, B):
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = wk.SWEEP[name].scaled(B=B)
    inp = wk.make_step_inputs(wl)
    prev = oracle_prime(inp, n_threads=16)
    rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len, n_threads=16)
    print(name, rep.summary(), "mean accept_len", float(got.accept_len.mean()))
    assert rep.positions == B * wl.W
    s = got.vals.reshape(-1, got.vals.shape[-1]).astype(np.float64).sum(axis=1)
    assert np.all(np.abs(s - 1.0) < 1e-5)
