"""CPU oracle of the decode loop around the step (paper Section 4.1, Steps 1-4 iterated; the token
initialisation strategies of Section 4.2: random and the four spatial-prior ones).

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Plain numpy bookkeeping around ``oracle.sjd_step``; shares no code
with the CUDA library.

Per iteration and sequence: the step reports a = number of leading accepted rows and puts the residual
draw at row a.  The loop commits c = a + 1 tokens (the accepted prefix and the residual token, which is an
exact sample because its prefix is final), or the whole window when every row was accepted; rows beyond
the committed ones move to the front of the window and keep this iteration's distributions as their
verification reference (Step 1); freed slots get a token drawn uniformly from [0, V) whose reference is
the uniform distribution, or, with a spatial-prior strategy, the token (or a draw from the distribution) of
the left or above neighbour on a raster grid.  Parity of the loop beyond the step it calls is pinned by
invariants only.

Spatial-prior initialisation of a new slot at absolute position p, grid width G (the paper names the four
strategies and fixes nothing else; the choices below are this implementation's):
  * the token of an earlier position r < p is the committed token when r lies before the window that was
    just verified, that step's output token when r lies inside it, and otherwise (r is itself a new slot)
    the token that slot was initialised with;
  * "repeat left" copies the token of p-1, "repeat above" the token of p-G (of p-1 when p < G); the draft
    is deterministic, so its reference distribution is the point mass on that token (one entry of
    probability 1), which keeps the accept test and the residual exact;
  * "sample left" / "sample above" draw from a sparse distribution the step just produced: for "left" the
    one predicted for position p-1, or the last window row's when p-1 lies behind the verified window (with
    refinement every new slot does); for "above" the row of position p-G, stepping a further G back while
    that position lies behind the verified window; the draw is the fixed-point inverse CDF on one Philox block (purpose 5) and the
    reference distribution is the one drawn from.  When position p-G was verified before this step, its
    distribution no longer exists and the slot falls back to "repeat above"; when p < G it falls back to
    "sample left";
  * the first window has no predictions and nothing to its left: its slot 0 is random with a uniform
    reference, and the sampling strategies act as their repeating counterparts inside that window.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import FLAG_REUSE, Probs, Q_UNIFORM, icdf, philox4x32_10, sjd_step

PURPOSE_TOKEN_INIT = 4
PURPOSE_PRIOR_INIT = 5

INIT_RANDOM, INIT_REPEAT_LEFT, INIT_REPEAT_ABOVE, INIT_SAMPLE_LEFT, INIT_SAMPLE_ABOVE = 0, 1, 2, 3, 4


def random_token(seed: int, pos: int, seq: int, iteration: int, V: int) -> int:
    """Uniform token for absolute position `pos`: floor(x0 * V / 2^32) of one Philox block."""
    x = philox4x32_10([pos, seq, iteration, PURPOSE_TOKEN_INIT], [seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF])
    return (int(x[0]) * V) >> 32


@dataclass
class Window:
    drafts: np.ndarray      # [B,W] int32
    probs: Probs            # reference distributions of the drafts
    win_len: np.ndarray     # [B]
    pos_base: np.ndarray    # [B]
    iteration: np.ndarray   # [B]
    committed: np.ndarray   # [B,N] int32, -1 where not yet decided


def _set_uniform(probs: Probs, b, i, V):
    probs.tok_prob[b, i] = np.float32(1.0) / np.float32(V)
    probs.cnt[b, i] = Q_UNIFORM


def _set_point_mass(probs: Probs, b, i, tok):
    probs.ids[b, i, 0] = tok
    probs.vals[b, i, 0] = np.float32(1.0)
    probs.cnt[b, i] = 1
    probs.tok_prob[b, i] = np.float32(1.0)


def _draw_from_row(probs: Probs, b, i, src: Probs, sb, si, seed, pos, seq, iteration):
    """Slot (b,i) gets a draw from row (sb,si) of `src` and that row as its reference distribution."""
    n = int(src.cnt[sb, si])
    x = philox4x32_10([pos, seq, iteration, PURPOSE_PRIOR_INIT], [seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF])
    R = int(x[0]) | (int(x[1]) << 32)
    k, _ = icdf(src.vals[sb, si, :n], R)
    k = max(k, 0)
    probs.ids[b, i, :n] = src.ids[sb, si, :n]
    probs.vals[b, i, :n] = src.vals[sb, si, :n]
    probs.cnt[b, i] = n
    probs.tok_prob[b, i] = src.vals[sb, si, k]
    return int(src.ids[sb, si, k])


def window_init(B, W, V, kcap, n_total, seed, seq_base=0, iteration0=0, init_mode=INIT_RANDOM, grid_width=0) -> Window:
    w = Window(np.full((B, W), -1, np.int32), Probs.empty(B, W, kcap), np.zeros(B, np.int32), np.zeros(B, np.int32),
               np.full(B, iteration0, np.int32), np.full((B, n_total), -1, np.int32))
    for b in range(B):
        w.win_len[b] = min(W, n_total)
        for i in range(int(w.win_len[b])):
            back = 0
            if init_mode in (INIT_REPEAT_LEFT, INIT_SAMPLE_LEFT):
                back = 1
            elif init_mode in (INIT_REPEAT_ABOVE, INIT_SAMPLE_ABOVE):
                back = grid_width if i >= grid_width else 1
            if back == 0 or i - back < 0:
                w.drafts[b, i] = random_token(seed, i, seq_base + b, iteration0, V)
                _set_uniform(w.probs, b, i, V)
            else:
                w.drafts[b, i] = w.drafts[b, i - back]
                _set_point_mass(w.probs, b, i, w.drafts[b, i])
    return w


def window_advance(w: Window, accept_len, step_tokens, step_probs: Probs, V, n_total, seed, seq_base=0,
                   init_mode=INIT_RANDOM, grid_width=0, refine=True):
    """Commit, shift and refill.  Returns (next window, committed counts).  With refine=False (the paper's
    "no refinement" ablation) nothing is shifted: every slot behind the committed tokens is newly initialised."""
    B, W = w.drafts.shape
    kcap = w.probs.ids.shape[-1]
    nxt = Window(np.full((B, W), -1, np.int32), Probs.empty(B, W, kcap), np.zeros(B, np.int32), np.zeros(B, np.int32),
                 w.iteration + 1, w.committed.copy())
    counts = np.zeros(B, np.int32)
    for b in range(B):
        L, a, p0, it = int(w.win_len[b]), int(accept_len[b]), int(w.pos_base[b]), int(w.iteration[b])
        c = a + 1 if a < L else L
        counts[b] = c
        nxt.committed[b, p0:p0 + c] = step_tokens[b, :c]
        p1 = p0 + c
        L1 = max(0, min(W, n_total - p1))
        nxt.pos_base[b], nxt.win_len[b] = p1, L1
        for i in range(L1):
            src = i + c
            if refine and src < L:
                nxt.drafts[b, i] = step_tokens[b, src]
                nxt.probs.tok_prob[b, i] = step_probs.tok_prob[b, src]
                n = int(step_probs.cnt[b, src])
                nxt.probs.ids[b, i, :n] = step_probs.ids[b, src, :n]
                nxt.probs.vals[b, i, :n] = step_probs.vals[b, src, :n]
                nxt.probs.cnt[b, i] = n
                continue
            p = p1 + i
            if init_mode == INIT_RANDOM:
                nxt.drafts[b, i] = random_token(seed, p, seq_base + b, it, V)
                _set_uniform(nxt.probs, b, i, V)
                continue

            known = L if refine else c        # window rows whose token survives into the next iteration

            def token_at(r):
                # r < p; new slots before p are already filled in nxt
                if r < p0:
                    return int(w.committed[b, r])
                if r < p0 + known:
                    return int(step_tokens[b, r - p0])
                return int(nxt.drafts[b, r - p1])

            above = init_mode in (INIT_REPEAT_ABOVE, INIT_SAMPLE_ABOVE) and p >= grid_width
            sample = init_mode in (INIT_SAMPLE_LEFT, INIT_SAMPLE_ABOVE)
            if not sample:
                nxt.drafts[b, i] = token_at(p - grid_width if above else p - 1)
                _set_point_mass(nxt.probs, b, i, nxt.drafts[b, i])
            elif not above:
                left = min(p - 1 - p0, L - 1)   # the prediction made for position p-1, else the last one made
                nxt.drafts[b, i] = _draw_from_row(nxt.probs, b, i, step_probs, b, left, seed, p, seq_base + b, it)
            else:
                r = p - grid_width
                while r >= p0 + L:
                    r -= grid_width
                if r >= p0:
                    nxt.drafts[b, i] = _draw_from_row(nxt.probs, b, i, step_probs, b, r - p0, seed, p, seq_base + b, it)
                elif r >= 0:
                    nxt.drafts[b, i] = int(w.committed[b, r])
                    _set_point_mass(nxt.probs, b, i, nxt.drafts[b, i])
                else:
                    left = min(p - 1 - p0, L - 1)
                    nxt.drafts[b, i] = _draw_from_row(nxt.probs, b, i, step_probs, b, left, seed, p, seq_base + b, it)
    return nxt, counts


def decode(logit_source, *, B, W, V, n_total, dtype, top_k, cfg_scale=1.0, inv_temperature=1.0, reuse_tau=0.5,
           flags=FLAG_REUSE, seed=0, seq_base=0, max_steps=None, n_threads=1, trace=None, init_mode=INIT_RANDOM,
           grid_width=0, refine=True):
    """Run the loop to the end.  `logit_source(window) -> (cond, uncond)` plays the model's forward pass.
    Returns (committed [B,n_total], steps, committed counts per step [steps,B])."""
    kcap = min(top_k, V)
    w = window_init(B, W, V, kcap, n_total, seed, seq_base, 0, init_mode, grid_width)
    history = []
    steps = 0
    while np.any(w.win_len > 0):
        if max_steps is not None and steps >= max_steps:
            break
        cond, uncond = logit_source(w)
        r = sjd_step(cond, uncond, w.drafts, w.probs, dtype=dtype, V=V, cfg_scale=cfg_scale,
                     inv_temperature=inv_temperature, top_k=top_k, reuse_tau=reuse_tau, flags=flags, win_len=w.win_len,
                     pos_base=w.pos_base, iteration=w.iteration, seed=seed, seq_base=seq_base, n_threads=n_threads)
        if trace is not None:
            trace.append((w, r))
        w, counts = window_advance(w, r.accept_len, r.tokens, r.probs, V, n_total, seed, seq_base, init_mode, grid_width, refine)
        history.append(counts)
        steps += 1
    return w.committed, steps, np.array(history, np.int32).reshape(steps, B)
