"""The oracle's decode loop: invariants the paper's schedule fixes (no implementation to compare against)."""
import numpy as np

import oracle
from oracle import loop
from paper_2512_07503_b200 import workloads as wk


def _run(B=2, W=6, V=256, N=40, top_k=32, flags=oracle.FLAG_REUSE, seed=11, trace=None, **kw):
    src = wk.MarkovSource(V, N, wk.F32, states=16)
    source = lambda w: src.logits(w.drafts, w.win_len, w.pos_base, w.committed)
    return loop.decode(source, B=B, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=top_k, cfg_scale=3.0, flags=flags, seed=seed,
                       trace=trace, **kw)


def test_every_step_commits_at_least_one_token_and_the_grid_is_filled():
    committed, steps, counts = _run()
    assert counts.shape == (steps, 2)
    active = np.cumsum(counts, axis=0) - counts < 40          # sequence still running before the step
    assert np.all(counts[active] >= 1) and np.all(counts <= 6)
    assert np.all(counts.sum(axis=0) == 40)
    assert steps <= 40
    assert np.all((committed >= 0) & (committed < 256))


def test_random_initialisation_is_uniform_and_keyed_by_position():
    toks = [loop.random_token(3, p, 0, 0, 1000) for p in range(4000)]
    assert min(toks) >= 0 and max(toks) < 1000
    hist = np.bincount(np.array(toks) // 100, minlength=10)
    assert np.all(np.abs(hist - 400) < 5 * np.sqrt(400 * 0.9))
    assert loop.random_token(3, 5, 0, 0, 1000) == toks[5]
    assert loop.random_token(3, 5, 1, 0, 1000) != toks[5] or loop.random_token(3, 6, 1, 0, 1000) != toks[6]


def test_k1_is_deterministic_jacobi_decoding_and_reaches_the_greedy_sequence():
    # With K = 1 every distribution is one-hot: a draft is accepted iff it equals the arg max given its
    # prefix (Eq. 1 of the paper), so the committed sequence is the greedy autoregressive one.
    V, N = 128, 24
    src = wk.MarkovSource(V, N, wk.F32, states=8)
    source = lambda w: src.logits(w.drafts, w.win_len, w.pos_base, w.committed)
    committed, steps, counts = loop.decode(source, B=1, W=5, V=V, n_total=N, dtype=oracle.F32, top_k=1, cfg_scale=3.0, seed=2)
    greedy, prev = [], 0
    for p in range(N):
        c = src.table[prev % 8] + src.noise_c[p]
        u = c + src.noise_u[p]
        y = (u + np.float32(3.0) * (c - u)).astype(np.float32)
        prev = int(np.argmax(y))
        greedy.append(prev)
    assert committed[0].tolist() == greedy
    assert steps <= N


def test_a_source_that_ignores_the_prefix_converges_in_two_iterations_per_window():
    # logits independent of the drafts: after one iteration every row's reference distribution equals the
    # next iteration's distribution, so everything still in the window is accepted (ratio 1)
    V, N, W = 64, 30, 10
    rng = np.random.default_rng(0)
    fixed = rng.standard_normal((N, V)).astype(np.float32)

    def source(w):
        cond = np.zeros((1, W, V), np.float32)
        for i in range(int(w.win_len[0])):
            cond[0, i] = fixed[int(w.pos_base[0]) + i]
        return cond, None

    trace = []
    committed, steps, counts = loop.decode(source, B=1, W=W, V=V, n_total=N, dtype=oracle.F32, top_k=16, seed=4, trace=trace)
    for (w, r) in trace:
        moved = w.probs.cnt[0, :int(w.win_len[0])] != oracle.Q_UNIFORM     # rows that were drafted by an earlier step
        n_moved = int(moved.sum())
        assert np.all(moved[:n_moved])                                        # they sit at the front
        assert int(r.accept_len[0]) >= n_moved                                # and are all accepted
    assert counts.sum() == N


def test_resume_from_a_dumped_window_reproduces_the_trajectory():
    trace = []
    committed, steps, counts = _run(trace=trace)
    # restart from the window before step 3 and replay: counter-based randomness makes it identical
    w3, _ = trace[3]
    src = wk.MarkovSource(256, 40, wk.F32, states=16)
    w = loop.Window(w3.drafts.copy(), oracle.Probs(w3.probs.tok_prob.copy(), w3.probs.ids.copy(), w3.probs.vals.copy(),
                                                    w3.probs.cnt.copy()), w3.win_len.copy(), w3.pos_base.copy(),
                    w3.iteration.copy(), w3.committed.copy())
    while np.any(w.win_len > 0):
        cond, unc = src.logits(w.drafts, w.win_len, w.pos_base, w.committed)
        r = oracle.sjd_step(cond, unc, w.drafts, w.probs, dtype=oracle.F32, V=256, cfg_scale=3.0, top_k=32,
                            flags=oracle.FLAG_REUSE, win_len=w.win_len, pos_base=w.pos_base, iteration=w.iteration, seed=11)
        w, _ = loop.window_advance(w, r.accept_len, r.tokens, r.probs, 256, 40, 11)
    assert np.array_equal(w.committed, committed)
