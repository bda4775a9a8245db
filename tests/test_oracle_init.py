"""Spatial-prior token initialisation in the oracle's decode loop (paper Section 4.2): invariants of the four
strategies and the qualitative result of the paper's initialisation ablation."""
import numpy as np
import pytest

import oracle
from oracle import loop
from paper_2512_07503_b200 import workloads as wk

MODES = [loop.INIT_RANDOM, loop.INIT_REPEAT_LEFT, loop.INIT_REPEAT_ABOVE, loop.INIT_SAMPLE_LEFT, loop.INIT_SAMPLE_ABOVE]


def _markov(V, N, states=8):
    src = wk.MarkovSource(V, N, wk.F32, states=states)
    return src, (lambda w: src.logits(w.drafts, w.win_len, w.pos_base, w.committed))


def _sequence(w, b):
    """Committed tokens followed by the window's drafts: the token at every position decided or drafted so far."""
    p0, L = int(w.pos_base[b]), int(w.win_len[b])
    return np.concatenate([w.committed[b, :p0], w.drafts[b, :L]])


def _new_slots(prev_w, prev_r, b):
    L, a = int(prev_w.win_len[b]), int(prev_r.accept_len[b])
    c = a + 1 if a < L else L
    return L - c        # first row of the next window that is newly initialised


def test_greedy_result_does_not_depend_on_the_initialisation():
    # K = 1: the loop is deterministic Jacobi decoding, whose fixed point is the greedy sequence whatever
    # the initial guesses are
    V, N, G = 128, 30, 6
    results = []
    for mode in MODES:
        src, source = _markov(V, N)
        committed, steps, _ = loop.decode(source, B=1, W=8, V=V, n_total=N, dtype=oracle.F32, top_k=1, cfg_scale=3.0, seed=2,
                                          init_mode=mode, grid_width=G)
        results.append(committed[0].tolist())
        assert steps <= N
    assert all(r == results[0] for r in results)


@pytest.mark.parametrize("mode,G", [(loop.INIT_REPEAT_LEFT, 5), (loop.INIT_REPEAT_ABOVE, 5), (loop.INIT_REPEAT_ABOVE, 3)])
def test_repeat_strategies_copy_the_neighbour_and_use_a_point_mass(mode, G):
    V, N, W = 200, 40, 7
    src, source = _markov(V, N)
    trace = []
    loop.decode(source, B=2, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=16, cfg_scale=3.0, seed=5, trace=trace,
                init_mode=mode, grid_width=G)
    checked = 0
    for n, (w, r) in enumerate(trace):
        for b in range(2):
            first_new = 0 if n == 0 else _new_slots(*trace[n - 1], b)
            seq = _sequence(w, b)
            p0 = int(w.pos_base[b])
            for i in range(first_new, int(w.win_len[b])):
                p = p0 + i
                if p == 0:
                    assert w.probs.cnt[b, i] == oracle.Q_UNIFORM
                    continue
                back = G if (mode == loop.INIT_REPEAT_ABOVE and p >= G) else 1
                assert w.drafts[b, i] == seq[p - back]
                assert w.probs.cnt[b, i] == 1 and w.probs.ids[b, i, 0] == w.drafts[b, i]
                assert w.probs.vals[b, i, 0] == 1.0 and w.probs.tok_prob[b, i] == 1.0
                checked += 1
    assert checked > 40


@pytest.mark.parametrize("mode,G", [(loop.INIT_SAMPLE_LEFT, 5), (loop.INIT_SAMPLE_ABOVE, 5), (loop.INIT_SAMPLE_ABOVE, 3),
                                    (loop.INIT_SAMPLE_ABOVE, 12)])
def test_sample_strategies_draw_from_the_neighbours_prediction(mode, G):
    V, N, W, K = 200, 48, 9, 16
    src, source = _markov(V, N)
    trace = []
    loop.decode(source, B=2, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=K, cfg_scale=3.0, seed=6, trace=trace,
                init_mode=mode, grid_width=G)
    drawn = repeated = 0
    for n in range(1, len(trace)):
        (pw, pr), (w, _) = trace[n - 1], trace[n]
        for b in range(2):
            p0_prev, L_prev, p0 = int(pw.pos_base[b]), int(pw.win_len[b]), int(w.pos_base[b])
            for i in range(_new_slots(pw, pr, b), int(w.win_len[b])):
                p = p0 + i
                r = p - 1
                if mode == loop.INIT_SAMPLE_ABOVE and p >= G:
                    r = p - G
                    while r >= p0_prev + L_prev:
                        r -= G
                else:
                    r = p0_prev + L_prev - 1           # the last position the step predicted
                if r >= p0_prev:
                    row = r - p0_prev
                    assert w.probs.cnt[b, i] == K
                    assert np.array_equal(w.probs.ids[b, i], pr.probs.ids[b, row])
                    assert np.array_equal(w.probs.vals[b, i], pr.probs.vals[b, row])
                    k = int(np.searchsorted(w.probs.ids[b, i], w.drafts[b, i]))
                    assert w.probs.ids[b, i, k] == w.drafts[b, i] and w.probs.tok_prob[b, i] == w.probs.vals[b, i, k] > 0
                    drawn += 1
                else:
                    assert r >= 0
                    assert w.drafts[b, i] == w.committed[b, r] and w.probs.cnt[b, i] == 1
                    repeated += 1
    assert drawn > 20
    if G > W:          # the position above can lie before the verified window: its prediction is gone
        assert repeated > 0


def test_draws_follow_the_source_distribution():
    V, K, n = 64, 8, 6000
    src = oracle.Probs.empty(1, 1, K)
    src.ids[0, 0] = np.arange(K) * 7
    vals = np.array([0.4, 0.2, 0.15, 0.1, 0.08, 0.04, 0.02, 0.01], np.float32)
    src.vals[0, 0] = vals
    src.cnt[0, 0] = K
    dst = oracle.Probs.empty(1, 1, K)
    counts = np.zeros(K)
    for pos in range(n):
        tok = loop._draw_from_row(dst, 0, 0, src, 0, 0, seed=9, pos=pos, seq=3, iteration=1)
        assert tok % 7 == 0 and dst.tok_prob[0, 0] == vals[tok // 7]
        counts[tok // 7] += 1
    expect = vals.astype(np.float64) / vals.sum() * n
    assert np.all(np.abs(counts - expect) < 5 * np.sqrt(expect) + 1)


def _pattern_source(V, W, G, axis, sharp=9.0, seed=0):
    """Logits of a flat image: the prediction at every position is peaked on one fixed token (axis 'left': a
    single colour) or on a token that depends on the column only (axis 'above': vertical stripes)."""
    rng = np.random.default_rng(seed)
    colours = rng.permutation(V)[:G]

    def source(w):
        B = w.drafts.shape[0]
        cond = (0.3 * rng.standard_normal((B, W, V))).astype(np.float32)
        for b in range(B):
            for i in range(int(w.win_len[b])):
                p = int(w.pos_base[b]) + i
                cond[b, i, colours[0] if axis == "left" else colours[p % G]] += sharp
        return cond, None
    return source


@pytest.mark.parametrize("axis,mode", [("left", loop.INIT_REPEAT_LEFT), ("above", loop.INIT_REPEAT_ABOVE),
                                       ("left", loop.INIT_SAMPLE_LEFT), ("above", loop.INIT_SAMPLE_ABOVE)])
def test_spatial_prior_needs_fewer_steps_than_random_on_a_repetitive_image(axis, mode):
    # the paper's initialisation ablation: on an image of simple repeated patterns the spatially aware
    # strategies compress the step count more than random initialisation
    V, W, G, N = 512, 12, 8, 96
    steps = {}
    for m in (loop.INIT_RANDOM, mode):
        total = 0
        for seed in range(4):
            _, s, _ = loop.decode(_pattern_source(V, W, G, axis, seed=seed), B=1, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=64,
                                  seed=seed, init_mode=m, grid_width=G)
            total += s
        steps[m] = total
    assert steps[mode] < 0.8 * steps[loop.INIT_RANDOM], steps


# ---- the "no refinement" ablation: unaccepted tokens are replaced by newly initialised ones ----

def test_without_refinement_every_slot_behind_the_commit_is_new():
    V, N, W = 200, 40, 7
    src, source = _markov(V, N)
    trace = []
    loop.decode(source, B=2, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=16, cfg_scale=3.0, seed=5, trace=trace, refine=False)
    for w, _ in trace:
        for b in range(2):
            assert np.all(w.probs.cnt[b, :int(w.win_len[b])] == oracle.Q_UNIFORM)
    trace = []
    loop.decode(source, B=2, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=16, cfg_scale=3.0, seed=5, trace=trace, refine=False,
                init_mode=loop.INIT_REPEAT_LEFT, grid_width=5)
    for n, (w, _) in enumerate(trace[1:]):
        for b in range(2):
            L, p0 = int(w.win_len[b]), int(w.pos_base[b])
            assert np.all(w.drafts[b, :L] == w.committed[b, p0 - 1])      # the last committed token, repeated
            assert np.all(w.probs.cnt[b, :L] == 1)


def test_without_refinement_greedy_decoding_still_reaches_the_greedy_sequence():
    V, N = 128, 30
    out = []
    for refine in (True, False):
        src, source = _markov(V, N)
        committed, steps, _ = loop.decode(source, B=1, W=8, V=V, n_total=N, dtype=oracle.F32, top_k=1, cfg_scale=3.0, seed=2,
                                          refine=refine)
        out.append(committed[0].tolist())
    assert out[0] == out[1]


def test_without_refinement_there_is_almost_no_acceleration():
    # the paper's refinement ablation: replacing unaccepted tokens by new ones needs about one forward pass
    # per token, refinement about half as many; a spatial prior helps a little when the image is flat
    V, W, N = 512, 12, 96
    src, source = _markov(V, N, states=16)
    kw = dict(B=1, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=64, cfg_scale=3.0, seed=3)
    _, with_ref, _ = loop.decode(source, **kw)
    _, without, _ = loop.decode(source, refine=False, **kw)
    assert without >= 0.9 * N and without > 1.1 * with_ref, (with_ref, without)
    flat = lambda seed: _pattern_source(V, W, 8, "left", seed=seed)
    kw = dict(B=1, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=64, seed=1)
    _, rnd, _ = loop.decode(flat(1), refine=False, **kw)
    _, rep, _ = loop.decode(flat(1), refine=False, init_mode=loop.INIT_REPEAT_LEFT, grid_width=8, **kw)
    assert rnd >= 0.9 * N and rep < 0.5 * rnd, (rnd, rep)
