"""Decode loop on the GPU (sjd_step + sjd_window_advance through the C ABI) in lock-step with the oracle's
loop on the same synthetic Markov logit source: same committed tokens, same number of iterations, same
tokens committed per iteration."""
import numpy as np
import pytest
import torch

import oracle
from oracle import loop
from paper_2512_07503_b200 import workloads as wk

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(B, W, V, N, top_k, dtype, reuse=True, seed=21, states=64, init_mode=0, grid_width=1, windows=False,
          use_graphs=False, refine=True, lazy=False):
    from paper_2512_07503_b200.decode import DecodeLoop
    src = wk.MarkovSource(V, N, dtype, states=states, lazy=lazy)
    flags = oracle.FLAG_REUSE if reuse else 0
    trace = []
    ref_committed, ref_steps, ref_counts = loop.decode(
        lambda w: src.logits(w.drafts, w.win_len, w.pos_base, w.committed), B=B, W=W, V=V, n_total=N, dtype=dtype,
        top_k=top_k, cfg_scale=3.0, flags=flags, seed=seed, n_threads=8, init_mode=init_mode, grid_width=grid_width,
        trace=trace, refine=refine)

    tdt = torch.bfloat16 if dtype == wk.BF16 else torch.float32
    dl = DecodeLoop(batch=B, window=W, vocab=V, n_total=N, logits_dtype=tdt, top_k=top_k, cfg_scale=3.0, reuse=reuse,
                    seed=seed, init_mode=init_mode, grid_width=grid_width, use_graphs=use_graphs, refine=refine, device=DEV)

    def up(a):
        if dtype == wk.BF16:
            return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
        return torch.from_numpy(a).to(DEV)

    def source(d):
        if windows:
            _same_window(d, trace[d.steps][0])
        c, u = src.logits(d.window_tokens.cpu().numpy(), d.win_len.cpu().numpy(), d.pos_base.cpu().numpy(),
                          d.committed.cpu().numpy())
        return up(c), up(u)

    committed, steps, counts = dl.run(source, max_steps=4 * N)
    assert int(dl.status.max().item()) & 8 == 0
    return (committed.numpy(), steps, counts.numpy()), (ref_committed, ref_steps, ref_counts)


def _same_window(d, w):
    """The device loop's current window against the oracle's: drafts, reference distributions, state."""
    L = w.win_len
    assert np.array_equal(d.win_len.cpu().numpy(), L) and np.array_equal(d.pos_base.cpu().numpy(), w.pos_base)
    q = d.q[d.cur]
    drafts, cnt, tp = d.window_tokens.cpu().numpy(), q.cnt.cpu().numpy(), q.tok_prob.cpu().numpy()
    ids, vals = q.ids.cpu().numpy(), q.vals.cpu().numpy()
    for b in range(L.shape[0]):
        n = int(L[b])
        assert np.array_equal(drafts[b, :n], w.drafts[b, :n]), (b, drafts[b, :n], w.drafts[b, :n])
        assert np.array_equal(cnt[b, :n], w.probs.cnt[b, :n])
        np.testing.assert_allclose(tp[b, :n], w.probs.tok_prob[b, :n], rtol=1e-5, atol=0)
        for i in range(n):
            k = max(int(cnt[b, i]), 0)
            assert np.array_equal(ids[b, i, :k], w.probs.ids[b, i, :k])
            np.testing.assert_allclose(vals[b, i, :k], w.probs.vals[b, i, :k], rtol=1e-5, atol=1e-30)


@pytest.mark.parametrize("mode", [1, 2, 3, 4])
@pytest.mark.parametrize("B,W,V,N,K,dtype,G", [(2, 8, 4096, 60, 64, wk.F32, 5), (2, 12, 8192, 70, 300, wk.BF16, 16),
                                               (1, 6, 512, 30, 40, wk.F32, 2)])
def test_spatial_prior_initialisation_matches_the_oracle(B, W, V, N, K, dtype, G, mode):
    # Section 4.2's four strategies, window by window: new slots' tokens and their reference distributions
    got, ref = _both(B, W, V, N, K, dtype, init_mode=mode, grid_width=G, windows=True)
    assert got[1] == ref[1], (got[1], ref[1])
    assert np.array_equal(got[2], ref[2])
    assert np.array_equal(got[0], ref[0])


@pytest.mark.parametrize("mode", [0, 4])
def test_graph_replay_gives_the_same_trajectory(mode):
    # every iteration after the first two replays a captured CUDA graph of the four kernels
    got, ref = _both(2, 12, 8192, 70, 300, wk.BF16, init_mode=mode, grid_width=16, windows=True, use_graphs=True)
    assert got[1] == ref[1] and np.array_equal(got[2], ref[2]) and np.array_equal(got[0], ref[0])
    assert got[1] > 6


@pytest.mark.parametrize("mode", [0, 1, 2, 3, 4])
def test_no_refinement_ablation_matches_the_oracle(mode):
    # nothing is carried over: every slot behind the committed tokens is newly initialised
    got, ref = _both(2, 10, 4096, 40, 64, wk.F32, init_mode=mode, grid_width=4, windows=True, refine=False)
    assert got[1] == ref[1] and np.array_equal(got[2], ref[2]) and np.array_equal(got[0], ref[0])


def test_random_initialisation_windows_match_the_oracle():
    got, ref = _both(2, 8, 4096, 50, 64, wk.F32, windows=True)
    assert np.array_equal(got[0], ref[0]) and got[1] == ref[1]


@pytest.mark.parametrize("B,W,V,N,K,dtype,reuse", [(3, 8, 4096, 50, 64, wk.F32, True), (2, 16, 8192, 70, 300, wk.BF16, True),
                                                   (2, 5, 512, 23, 40, wk.F32, False), (1, 32, 16384, 96, 1000, wk.BF16, True)])
def test_loop_matches_the_oracle(B, W, V, N, K, dtype, reuse):
    got, ref = _both(B, W, V, N, K, dtype, reuse)
    assert got[1] == ref[1], (got[1], ref[1])
    assert np.array_equal(got[2], ref[2])
    assert np.array_equal(got[0], ref[0])
    assert np.all(got[2].sum(axis=0) == N)
    print("steps", got[1], "tokens per step", N * B / max(1, got[2].shape[0] * B))


def test_decode_loop_workload_at_full_size_matches_the_oracle():
    # the decode-loop configuration as benchmarked: one 48 x 48 grid of 2,304 tokens, V = 65,536, W = 32,
    # bf16 logits, guidance 3.0, top-K 2,000, random initialisation - every iteration in lock-step with the oracle
    N = 2304
    got, ref = _both(1, 32, 65536, N, 2000, wk.BF16, seed=5, states=1024, lazy=True)
    assert got[1] == ref[1], (got[1], ref[1])
    assert np.array_equal(got[2], ref[2])
    assert np.array_equal(got[0], ref[0])
    assert int(got[2].sum()) == N and np.all(got[0] >= 0)
    print("cfg5 full size: steps", got[1], "step compression", round(N / got[1], 3))
