"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds NONE of the method's arithmetic: it only draws Gaussian logits, rounds them to
the storage type and lays out the window bookkeeping.  Both the CUDA path and the CPU oracle consume
what it returns, so that the two see the same bits.

The workloads are the benchmark's configurations (top-K 2000 and guidance weight 3.0
are the paper's Section 5.1 settings; window sizes 16-64 lie in the range of the paper's window
ablation; 576 tokens is the 24x24 grid the paper quotes for Janus-Pro).  They stand in for the
paper's prompt sets and models, none of which can be used offline.

Logits are drawn on the host with numpy's Philox bit generator; bf16 storage is produced by
round-to-nearest-even on the fp32 value and handed around as uint16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

F32, BF16, F16 = 0, 1, 2


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    W: int
    V: int
    dtype: int            # F32, BF16 or F16
    sigma: float          # std of the conditional logits
    peaks: int            # tokens per row boosted by `boost`
    boost: float
    uncond_iid: bool      # True: uncond drawn independently; False: uncond = cond + N(0, 1)
    cfg_scale: float
    temperature: float
    top_k: int
    reuse: bool
    reuse_tau: float
    seed: int
    ragged_total: int = 0  # >0: window starts staggered uniformly in [0, ragged_total)
    prev_sigma: float = 0.5
    row_spread: float = 0.0  # >0: row (b,i) is scaled by exp(row_spread * U(-1,1)): flat and peaked rows side by side

    @property
    def kcap(self) -> int:
        return min(self.top_k, self.V)

    @property
    def inv_temperature(self) -> np.float32:
        return np.float32(1.0) / np.float32(self.temperature)

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


CONFIGS = {
    # small case the oracle finishes in well under a second
    "cfg1": Workload("cfg1", B=1, W=16, V=4096, dtype=F32, sigma=2.0, peaks=0, boost=0.0, uncond_iid=True,
                     cfg_scale=3.0, temperature=1.0, top_k=64, reuse=True, reuse_tau=0.5, seed=0),
    "cfg2": Workload("cfg2", B=1, W=32, V=65536, dtype=BF16, sigma=3.0, peaks=20, boost=8.0, uncond_iid=False,
                     cfg_scale=3.0, temperature=1.0, top_k=2000, reuse=True, reuse_tau=0.5, seed=2),
    "cfg3": Workload("cfg3", B=64, W=16, V=16384, dtype=F32, sigma=2.5, peaks=10, boost=6.0, uncond_iid=False,
                     cfg_scale=4.0, temperature=0.9, top_k=1000, reuse=True, reuse_tau=0.5, seed=3,
                     ragged_total=576),
    # the configuration the headline metric is quoted on
    "cfg4": Workload("cfg4", B=16, W=64, V=65536, dtype=BF16, sigma=3.0, peaks=20, boost=8.0, uncond_iid=False,
                     cfg_scale=3.0, temperature=1.0, top_k=2000, reuse=True, reuse_tau=0.5, seed=4),
}


def _sweep():
    """Wider shapes around the headline configuration, same recipe: the window sizes of the paper's window
    ablation (16 to 512), the top-K values of its sampling ablation, and the vocabularies of the models it
    accelerates (16,384, 32,768 and 65,536 entries).  Batches keep the row count near the headline's 1,024."""
    base = CONFIGS["cfg4"]
    out = {}
    for W, B in ((16, 64), (32, 32), (96, 11), (250, 4), (512, 2)):
        out[f"w{W}"] = base.scaled(name=f"w{W}", B=B, W=W, seed=100 + W)
    for K in (1, 10, 100, 500, 1000, 8192):
        out[f"k{K}"] = base.scaled(name=f"k{K}", top_k=K, seed=200 + K % 97)
    out["v32k"] = base.scaled(name="v32k", V=32768, seed=301)
    out["v16k"] = base.scaled(name="v16k", V=16384, seed=302)
    out["v16k_f32"] = base.scaled(name="v16k_f32", V=16384, dtype=F32, seed=303)
    out["f16"] = base.scaled(name="f16", dtype=F16, seed=304)
    # rows of very different sharpness in one batch (scale factors from 1/e to e), as a model's rows are
    out["hetero"] = base.scaled(name="hetero", row_spread=1.0, seed=305)
    return out


SWEEP = _sweep()


def workload(name: str) -> Workload:
    """A benchmark configuration or a sweep shape by name."""
    return CONFIGS[name] if name in CONFIGS else SWEEP[name]


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even) and return the uint16 patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(x: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == F16:   # IEEE half precision, round to nearest even; kept as uint16 patterns like bf16
        return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)
    return to_bf16_bits(x) if dtype == BF16 else np.ascontiguousarray(x, dtype=np.float32)


def _as_f32(x: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == F16:
        return x.view(np.float16).astype(np.float32)
    return bf16_bits_to_f32(x) if dtype == BF16 else x


@dataclass
class StepInputs:
    wl: Workload
    cond: np.ndarray        # [B,W,V] float32, or uint16 bf16 patterns
    uncond: np.ndarray
    prev_cond: np.ndarray   # previous-iteration logits: cond/uncond + N(0, prev_sigma^2) each
    prev_uncond: np.ndarray
    win_len: np.ndarray     # [B] int32
    pos_base: np.ndarray    # [B] int32
    iteration: int          # Jacobi iteration index of the step under test (the priming call uses iteration-1)


def make_step_inputs(wl: Workload) -> StepInputs:
    """Logits of the current and of the previous Jacobi iteration for one step of `wl`."""
    rng = np.random.Generator(np.random.Philox(wl.seed))
    shape = (wl.B, wl.W, wl.V)
    cond = rng.standard_normal(shape, dtype=np.float32) * np.float32(wl.sigma)
    if wl.row_spread > 0:
        cond *= np.exp(wl.row_spread * rng.uniform(-1.0, 1.0, size=(wl.B, wl.W, 1))).astype(np.float32)
    if wl.peaks > 0:
        # `peaks` distinct ids per row, uniformly chosen, boosted by `boost`
        for b in range(wl.B):
            for i in range(wl.W):
                ids = rng.choice(wl.V, size=wl.peaks, replace=False)
                cond[b, i, ids] += np.float32(wl.boost)
    if wl.uncond_iid:
        uncond = rng.standard_normal(shape, dtype=np.float32) * np.float32(wl.sigma)
    else:
        uncond = cond + rng.standard_normal(shape, dtype=np.float32)
    cond_s, uncond_s = _store(cond, wl.dtype), _store(uncond, wl.dtype)
    ps = np.float32(wl.prev_sigma)
    prev_c = _store(_as_f32(cond_s, wl.dtype) + rng.standard_normal(shape, dtype=np.float32) * ps, wl.dtype)
    prev_u = _store(_as_f32(uncond_s, wl.dtype) + rng.standard_normal(shape, dtype=np.float32) * ps, wl.dtype)
    if wl.ragged_total > 0:
        start = rng.integers(0, wl.ragged_total, size=wl.B).astype(np.int32)
        win_len = np.minimum(wl.W, wl.ragged_total - start).astype(np.int32)
    else:
        start = np.zeros(wl.B, np.int32)
        win_len = np.full(wl.B, wl.W, np.int32)
    return StepInputs(wl, cond_s, uncond_s, prev_c, prev_u, win_len, start, iteration=1)


def markov_table(V: int, states: int = 1024, sigma: float = 3.0, seed: int = 7) -> np.ndarray:
    """Fixed [states, V] fp32 table of N(0, sigma^2) logits for the synthetic first-order Markov
    logit source of the decode-loop workload (logits[pos] = table[prev_token mod states] + noise)."""
    rng = np.random.Generator(np.random.Philox(seed))
    return rng.standard_normal((states, V), dtype=np.float32) * np.float32(sigma)


def markov_noise(V: int, pos: int, seed: int) -> np.ndarray:
    """N(0,1) noise row keyed by (seed, position) only, so that an unchanged prefix reproduces the
    same logits in every Jacobi iteration."""
    rng = np.random.Generator(np.random.Philox(key=[seed, pos]))
    return rng.standard_normal(V, dtype=np.float32)


class MarkovSource:
    """Synthetic first-order Markov "model" of the decode-loop workload, on the host:
    cond[pos] = table[prev_token mod states] + noise(seed_c, pos), uncond = cond + noise(seed_u, pos), where
    prev_token of window row i is the window's own draft at i-1 (the last committed token for row 0, token 0 at
    the very start), so that a rejection invalidates the later rows' logits.  The noise depends on the position
    only: an unchanged prefix reproduces the same logits in every iteration.  No method arithmetic here."""

    def __init__(self, V: int, n_total: int, dtype: int, states: int = 1024, sigma: float = 3.0, seed_table: int = 7,
                 seed_c: int = 5, seed_u: int = 6, lazy: bool = False):
        self.V, self.N, self.dtype, self.states = V, n_total, dtype, states
        self.table = markov_table(V, states, sigma, seed_table)
        self.seed_c, self.seed_u = seed_c, seed_u
        # the noise rows: all at once for small problems; drawn when first asked for, and kept while the window
        # is near, at the decode-loop workload's full size (2 x 2,304 x 65,536 floats would be 1.2 GB)
        self._rows = {} if lazy else None
        if not lazy:
            self.noise_c = np.stack([markov_noise(V, p, seed_c) for p in range(n_total)])
            self.noise_u = np.stack([markov_noise(V, p, seed_u) for p in range(n_total)])
        self._last_key, self._last = None, None

    def _noise(self, pos: int):
        if self._rows is None:
            return self.noise_c[pos], self.noise_u[pos]
        hit = self._rows.get(pos)
        if hit is None:
            hit = (markov_noise(self.V, pos, self.seed_c), markov_noise(self.V, pos, self.seed_u))
            self._rows[pos] = hit
            for old in [q for q in self._rows if q < pos - 256]:  # the window only moves forward
                del self._rows[old]
        return hit

    def logits(self, drafts: np.ndarray, win_len: np.ndarray, pos_base: np.ndarray, committed: np.ndarray):
        """cond, uncond of shape [B,W,V] in the storage type, for the given window state."""
        B, W = drafts.shape
        # the same window asked for twice in a row (two decoders in lock-step) is answered from memory
        key = (drafts.tobytes(), win_len.tobytes(), pos_base.tobytes(),
               tuple(int(committed[b, int(pos_base[b]) - 1]) if int(pos_base[b]) > 0 else 0 for b in range(B)))
        if key == self._last_key:
            return self._last
        cond = np.zeros((B, W, self.V), np.float32)
        unc = np.zeros((B, W, self.V), np.float32)
        for b in range(B):
            p0 = int(pos_base[b])
            for i in range(int(win_len[b])):
                prev = int(drafts[b, i - 1]) if i > 0 else (int(committed[b, p0 - 1]) if p0 > 0 else 0)
                nc, nu = self._noise(p0 + i)
                c = self.table[prev % self.states] + nc
                cond[b, i] = c
                unc[b, i] = c + nu
        self._last_key, self._last = key, (_store(cond, self.dtype), _store(unc, self.dtype))
        return self._last
