"""Whole-step pins for the oracle: special cases with a known answer and invariants of
Section 4.1 (Steps 3-4), the reuse rule (Eq. reuse) and plain SJD (Eq. refine-sjd)."""
import numpy as np
import pytest

import oracle
from paper_2512_07503_b200 import workloads as wk


def _prime(inp, **kw):
    """Previous-iteration distributions and drafts: sample every row from the perturbed logits."""
    wl = inp.wl
    return oracle.sjd_step(inp.prev_cond, inp.prev_uncond, None, None, dtype=wl.dtype, V=wl.V, cfg_scale=wl.cfg_scale,
                           inv_temperature=float(wl.inv_temperature), top_k=wl.top_k, flags=oracle.FLAG_DRAFT_ALL,
                           win_len=inp.win_len, pos_base=inp.pos_base, iteration0=inp.iteration - 1, seed=wl.seed, **kw)


def _step(inp, prev, flags=None, **kw):
    wl = inp.wl
    if flags is None:
        flags = oracle.FLAG_REUSE if wl.reuse else 0
    args = dict(dtype=wl.dtype, V=wl.V, cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature),
                top_k=wl.top_k, reuse_tau=wl.reuse_tau, flags=flags, win_len=inp.win_len, pos_base=inp.pos_base,
                iteration0=inp.iteration, seed=wl.seed, diag=True)
    args.update(kw)
    return oracle.sjd_step(inp.cond, inp.uncond, prev.tokens, prev.probs, **args)


SMALL = wk.CONFIGS["cfg1"].scaled(B=3, W=12, V=512, top_k=32)


def test_draft_all_samples_inside_support():
    inp = wk.make_step_inputs(SMALL)
    prev = _prime(inp)
    assert np.all(prev.accept_len == 0)
    for b in range(SMALL.B):
        for i in range(SMALL.W):
            ids, vals = prev.probs.ids[b, i], prev.probs.vals[b, i]
            k = np.searchsorted(ids, prev.tokens[b, i])
            assert ids[k] == prev.tokens[b, i]
            assert prev.probs.tok_prob[b, i] == vals[k] > 0
    assert np.all(prev.flags == oracle.OUT_RESAMPLED)


def test_identical_distributions_accept_everything():
    # p == q on every row: the ratio is exactly 1, r < 1 always, so the whole window is accepted
    inp = wk.make_step_inputs(SMALL)
    inp.prev_cond, inp.prev_uncond = inp.cond, inp.uncond
    prev = _prime(inp)
    r = _step(inp, prev)
    assert np.all(r.accept_len == SMALL.W)
    assert np.array_equal(r.tokens, prev.tokens)
    assert np.all(r.flags == oracle.OUT_ACCEPTED)
    assert np.array_equal(r.probs.tok_prob, prev.probs.tok_prob)
    assert np.all(r.status == 0)


def test_top1_reduces_to_deterministic_jacobi():
    # K = 1: every distribution is one-hot at the arg max, so the step is the Jacobi update x <- argmax
    # (Eq. 1) with the deterministic stop rule "token unchanged"
    wl = SMALL.scaled(top_k=1)
    inp = wk.make_step_inputs(wl)
    prev = _prime(inp)
    c = inp.cond.astype(np.float64)
    u = inp.uncond.astype(np.float64)
    amax = np.argmax(u + wl.cfg_scale * (c - u), axis=-1)
    r = _step(inp, prev)
    for b in range(wl.B):
        same = prev.tokens[b] == amax[b]
        a = int(np.argmin(same)) if not same.all() else wl.W
        assert r.accept_len[b] == a
        assert np.array_equal(r.tokens[b], amax[b])
    assert np.all(r.probs.tok_prob == 1.0)


def test_drafts_outside_support_are_rejected_at_row_zero():
    inp = wk.make_step_inputs(SMALL)
    prev = _prime(inp)
    r0 = _step(inp, prev)
    # replace every draft by a token that is not in the current support
    for b in range(SMALL.B):
        for i in range(SMALL.W):
            sup = set(r0.probs.ids[b, i].tolist())
            prev.tokens[b, i] = next(t for t in range(SMALL.V) if t not in sup)
    r = _step(inp, prev)
    assert np.all(r.accept_len == 0)
    assert np.all(r.flags[:, 0] == oracle.OUT_RESIDUAL)
    assert np.all(r.flags[:, 1:] == oracle.OUT_RESAMPLED)  # p(x_i) = 0 is never reused


def test_window_of_one_and_empty_window():
    wl = SMALL.scaled(W=1)
    inp = wk.make_step_inputs(wl)
    prev = _prime(inp)
    r = _step(inp, prev)
    assert np.all((r.accept_len == 0) | (r.accept_len == 1))
    inp2 = wk.make_step_inputs(SMALL)
    inp2.win_len[:] = [0, 5, SMALL.W]
    prev2 = _prime(inp2)
    r2 = _step(inp2, prev2)
    assert r2.accept_len[0] == 0 and np.all(r2.tokens[0] == -1) and np.all(r2.flags[0] == oracle.OUT_INVALID)
    assert r2.accept_len[1] <= 5 and np.all(r2.tokens[1, 5:] == -1) and np.all(r2.tokens[1, :5] >= 0)
    assert np.all(r2.probs.cnt[1, 5:] == 0) and np.all(r2.probs.tok_prob[1, 5:] == 0)


@pytest.mark.parametrize("name", ["cfg1", "mid"])
def test_step_invariants(name):
    wl = wk.CONFIGS["cfg1"] if name == "cfg1" else wk.CONFIGS["cfg3"].scaled(B=6, V=2048, top_k=100)
    inp = wk.make_step_inputs(wl)
    prev = _prime(inp)
    r = _step(inp, prev)
    sjd = _step(inp, prev, flags=0)
    inf_tau = _step(inp, prev, reuse_tau=np.inf)
    neg_tau = _step(inp, prev, reuse_tau=-1.0)
    d = r.diag
    for b in range(wl.B):
        L = int(inp.win_len[b])
        a = int(r.accept_len[b])
        assert 0 <= a <= L <= wl.W
        # accepted prefix: unchanged drafts whose tests all passed; row a failed its test
        assert np.all(d["pot_ok"][b, :a] == 1)
        assert np.array_equal(r.tokens[b, :a], prev.tokens[b, :a])
        if a < L:
            assert d["pot_ok"][b, a] == 0
            assert r.flags[b, a] == oracle.OUT_RESIDUAL and r.tokens[b, a] == d["pot_residual"][b, a]
            # residual support is {p > q}
            ids, vals = r.probs.ids[b, a], r.probs.vals[b, a]
            k = np.searchsorted(ids, r.tokens[b, a])
            qrow = dict(zip(prev.probs.ids[b, a].tolist(), prev.probs.vals[b, a].tolist()))
            assert vals[k] > qrow.get(int(ids[k]), 0.0)
        for i in range(a + 1, L):
            tok, fl = r.tokens[b, i], r.flags[b, i]
            ids, vals = r.probs.ids[b, i], r.probs.vals[b, i]
            k = int(np.searchsorted(ids, tok))
            assert k < len(ids) and ids[k] == tok, "every emitted token lies in the top-K support"
            assert r.probs.tok_prob[b, i] == vals[k]
            if fl == oracle.OUT_REUSED:
                assert tok == prev.tokens[b, i] and d["ratio"][b, i] > wl.reuse_tau and vals[k] > 0
            else:
                assert fl == oracle.OUT_RESAMPLED and tok == d["pot_redraft"][b, i]
                assert not (d["ratio"][b, i] > wl.reuse_tau)
        # the accept length does not depend on the redraft rule, and tau = +inf is plain SJD
        assert sjd.accept_len[b] == a == inf_tau.accept_len[b] == neg_tau.accept_len[b]
        assert np.all(sjd.flags[b, a + 1:L] == oracle.OUT_RESAMPLED)
        assert np.array_equal(sjd.tokens[b], inf_tau.tokens[b])
        # tau < 0 keeps every draft that is still in the support
        for i in range(a + 1, L):
            in_sup = prev.tokens[b, i] in set(r.probs.ids[b, i].tolist())
            assert (neg_tau.flags[b, i] == oracle.OUT_REUSED) == in_sup
        assert np.all(r.tokens[b, L:] == -1)
    # the distributions do not depend on the decisions
    assert np.array_equal(r.probs.vals, sjd.probs.vals) and np.array_equal(r.probs.ids, sjd.probs.ids)
    for b in range(wl.B):
        for i in range(int(inp.win_len[b])):
            assert abs(float(r.probs.vals[b, i].astype(np.float64).sum()) - 1) < 1e-6


def test_randomness_is_keyed_by_seed_batch_position_iteration():
    inp = wk.make_step_inputs(SMALL)
    prev = _prime(inp)
    r = _step(inp, prev)
    again = _step(inp, prev)
    assert np.array_equal(r.diag["u"], again.diag["u"]) and np.array_equal(r.tokens, again.tokens)
    other_seed = _step(inp, prev, seed=SMALL.seed + 1)
    other_iter = _step(inp, prev, iteration0=inp.iteration + 1)
    assert not np.array_equal(r.diag["u"], other_seed.diag["u"])
    assert not np.array_equal(r.diag["u"], other_iter.diag["u"])
    # window shifted by one absolute position: row i now draws what row i+1 drew
    shifted = _step(inp, prev, pos_base=inp.pos_base + 1)
    assert np.array_equal(shifted.diag["u"][:, :-1], r.diag["u"][:, 1:])
    # per-sequence iteration array overrides the scalar
    per_seq = _step(inp, prev, iteration=np.full(SMALL.B, inp.iteration + 1, np.int32))
    assert np.array_equal(per_seq.diag["u"], other_iter.diag["u"])
    # sequences draw from independent streams
    assert len({r.diag["u"][b].tobytes() for b in range(SMALL.B)}) == SMALL.B


def test_threads_do_not_change_the_result():
    wl = wk.CONFIGS["cfg3"].scaled(B=5, V=1024, top_k=50)
    inp = wk.make_step_inputs(wl)
    prev = _prime(inp)
    r1 = _step(inp, prev, n_threads=1)
    r4 = _step(inp, prev, n_threads=4)
    for a, b in [(r1.accept_len, r4.accept_len), (r1.tokens, r4.tokens), (r1.probs.vals, r4.probs.vals),
                 (r1.probs.ids, r4.probs.ids), (r1.probs.tok_prob, r4.probs.tok_prob), (r1.flags, r4.flags)]:
        assert np.array_equal(a, b)


def test_uniform_previous_distribution():
    # newly initialised slots: q is uniform over V (cnt = Q_UNIFORM); ratio = p(x) * V
    wl = SMALL
    inp = wk.make_step_inputs(wl)
    rng = np.random.default_rng(0)
    drafts = rng.integers(0, wl.V, size=(wl.B, wl.W)).astype(np.int32)
    q = oracle.Probs.uniform(wl.B, wl.W, wl.kcap, wl.V)
    r = oracle.sjd_step(inp.cond, inp.uncond, drafts, q, dtype=wl.dtype, V=wl.V, cfg_scale=wl.cfg_scale, top_k=wl.top_k,
                        flags=oracle.FLAG_REUSE, seed=5, diag=True)
    for b in range(wl.B):
        for i in range(wl.W):
            ids, vals = r.probs.ids[b, i], r.probs.vals[b, i]
            k = np.searchsorted(ids, drafts[b, i])
            p = vals[k] if k < len(ids) and ids[k] == drafts[b, i] else 0.0
            assert r.diag["ratio"][b, i] == np.float32(p) / (np.float32(1) / np.float32(wl.V))
        a = r.accept_len[b]
        if a < wl.W:
            ids, vals = r.probs.ids[b, a], r.probs.vals[b, a]
            k = np.searchsorted(ids, r.tokens[b, a])
            assert vals[k] > 1.0 / wl.V


def test_bad_arguments_are_refused():
    inp = wk.make_step_inputs(SMALL)
    with pytest.raises(ValueError):
        oracle.sjd_step(inp.cond, inp.uncond, None, None, dtype=SMALL.dtype, V=SMALL.V, top_k=8, flags=0)
    with pytest.raises(ValueError):
        oracle.sjd_step(inp.cond, inp.uncond, None, None, dtype=SMALL.dtype, V=SMALL.V, top_k=0,
                        flags=oracle.FLAG_DRAFT_ALL)
