"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (one sjd_step on
the whole batch): every output of every row against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from paper_2512_07503_b200 import workloads as wk

pytestmark = pytest.mark.gpu


def _full(name, flags=None):
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = wk.CONFIGS[name]
    inp = wk.make_step_inputs(wl)
    prev = oracle_prime(inp, n_threads=16)
    kw = step_kwargs(inp)
    if flags is not None:
        kw["flags"] = flags
    rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, kw, inp.win_len, n_threads=16)
    print(name, rep.summary(), "mean accept_len", float(got.accept_len.mean()))
    assert rep.positions == int(inp.win_len.sum())
    assert np.all(got.accept_len <= inp.win_len) and np.all(got.accept_len >= 0)
    return rep, got, ref


def test_cfg2_full():
    _full("cfg2")


def test_cfg3_full_ragged_batch():
    rep, got, ref = _full("cfg3")
    assert len(set(got.accept_len.tolist())) > 1  # ragged accept lengths, as the workload intends


def test_cfg4_full_headline_workload():
    rep, got, ref = _full("cfg4")
    # probabilities of every row sum to one within fp32 rounding
    s = got.vals.reshape(-1, got.vals.shape[-1]).astype(np.float64).sum(axis=1)
    assert np.all(np.abs(s - 1.0) < 1e-5)


def test_cfg4_full_plain_sjd():
    _full("cfg4", flags=0)
