"""CPU oracle of the decode loop around the step (paper Section 4.1, Steps 1-4 iterated; random token
initialisation of Section 4.2).

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Plain numpy bookkeeping around ``oracle.sjd_step``; shares no code
with the CUDA library.

Per iteration and sequence: the step reports a = number of leading accepted rows and puts the residual
draw at row a.  The loop commits c = a + 1 tokens (the accepted prefix and the residual token, which is an
exact sample because its prefix is final), or the whole window when every row was accepted; rows beyond
the committed ones move to the front of the window and keep this iteration's distributions as their
verification reference (Step 1); freed slots get a token drawn uniformly from [0, V) whose reference is
the uniform distribution.  Parity of the loop beyond the step it calls is pinned by invariants only.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import FLAG_REUSE, Probs, Q_UNIFORM, philox4x32_10, sjd_step

PURPOSE_TOKEN_INIT = 4


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


def window_init(B, W, V, kcap, n_total, seed, seq_base=0, iteration0=0) -> Window:
    w = Window(np.full((B, W), -1, np.int32), Probs.empty(B, W, kcap), np.zeros(B, np.int32), np.zeros(B, np.int32),
               np.full(B, iteration0, np.int32), np.full((B, n_total), -1, np.int32))
    for b in range(B):
        w.win_len[b] = min(W, n_total)
        for i in range(int(w.win_len[b])):
            w.drafts[b, i] = random_token(seed, i, seq_base + b, iteration0, V)
            w.probs.tok_prob[b, i] = np.float32(1.0) / np.float32(V)
            w.probs.cnt[b, i] = Q_UNIFORM
    return w


def window_advance(w: Window, accept_len, step_tokens, step_probs: Probs, V, n_total, seed, seq_base=0):
    """Commit, shift and refill.  Returns (next window, committed counts)."""
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
            if src < L:
                nxt.drafts[b, i] = step_tokens[b, src]
                nxt.probs.tok_prob[b, i] = step_probs.tok_prob[b, src]
                n = int(step_probs.cnt[b, src])
                nxt.probs.ids[b, i, :n] = step_probs.ids[b, src, :n]
                nxt.probs.vals[b, i, :n] = step_probs.vals[b, src, :n]
                nxt.probs.cnt[b, i] = n
            else:
                nxt.drafts[b, i] = random_token(seed, p1 + i, seq_base + b, it, V)
                nxt.probs.tok_prob[b, i] = np.float32(1.0) / np.float32(V)
                nxt.probs.cnt[b, i] = Q_UNIFORM
    return nxt, counts


def decode(logit_source, *, B, W, V, n_total, dtype, top_k, cfg_scale=1.0, inv_temperature=1.0, reuse_tau=0.5,
           flags=FLAG_REUSE, seed=0, seq_base=0, max_steps=None, n_threads=1, trace=None):
    """Run the loop to the end.  `logit_source(window) -> (cond, uncond)` plays the model's forward pass.
    Returns (committed [B,n_total], steps, committed counts per step [steps,B])."""
    kcap = min(top_k, V)
    w = window_init(B, W, V, kcap, n_total, seed, seq_base)
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
        w, counts = window_advance(w, r.accept_len, r.tokens, r.probs, V, n_total, seed, seq_base)
        history.append(counts)
        steps += 1
    return w.committed, steps, np.array(history, np.int32).reshape(steps, B)
