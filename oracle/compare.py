"""Parity protocol: compare the outputs of a step produced elsewhere (numpy arrays) with the oracle's.

TEST INFRASTRUCTURE.  Works on host arrays only and imports nothing from the CUDA side.

Bar: token ids, supports and accept lengths bit-exact; probabilities within 1e-5 relative.  A decision
whose oracle margin is below 1e-6 (|u - p/q| for the accept test, |C - tau| for the reuse test, distance
of the sampler's t to the nearest CDF step in units of probability mass) may legitimately fall on either
side, because the two sides' probabilities differ in the last bits; such positions are followed along the
branch the other side took, counted and reported, never silently ignored.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import OUT_ACCEPTED, OUT_INVALID, OUT_REUSED, OUT_RESAMPLED, OUT_RESIDUAL, FLAG_DRAFT_ALL, StepResult

MARGIN = 1e-6
REL_TOL = 1e-5
ABS_TOL = 1e-37  # below the normal range a float has no relative precision left


@dataclass
class ParityReport:
    positions: int = 0
    flagged_accept: int = 0
    flagged_reuse: int = 0
    flagged_sample: int = 0
    max_rel_err: float = 0.0
    errors: list = field(default_factory=list)

    @property
    def flagged(self) -> int:
        return self.flagged_accept + self.flagged_reuse + self.flagged_sample

    def ok(self) -> bool:
        return not self.errors

    def summary(self) -> str:
        return (f"positions={self.positions} flagged(accept/reuse/sample)={self.flagged_accept}/"
                f"{self.flagged_reuse}/{self.flagged_sample} max_rel_err={self.max_rel_err:.3g} "
                f"errors={len(self.errors)}")


def _err(rep, msg):
    if len(rep.errors) < 20:
        rep.errors.append(msg)
    else:
        rep.errors.append("...") if rep.errors[-1] != "..." else None


def compare_probs(rep: ParityReport, got_ids, got_vals, got_cnt, ref, win_len) -> None:
    """Supports bit-exact, probabilities within tolerance, for every valid row."""
    B, W = ref.probs.cnt.shape
    if not np.array_equal(got_cnt, ref.probs.cnt):
        _err(rep, f"cnt differs at {np.argwhere(got_cnt != ref.probs.cnt)[:5].tolist()}")
        return
    for b in range(B):
        L = int(win_len[b])
        if L == 0:
            continue
        gi, ri = got_ids[b, :L], ref.probs.ids[b, :L]
        if not np.array_equal(gi, ri):
            bad = np.argwhere((gi != ri).any(axis=-1)).ravel()[:5].tolist()
            _err(rep, f"support differs: sequence {b} rows {bad}")
            continue
        g = got_vals[b, :L].astype(np.float64)
        r = ref.probs.vals[b, :L].astype(np.float64)
        err = np.abs(g - r)
        bound = REL_TOL * np.abs(r) + ABS_TOL
        if np.any(err > bound):
            k = np.unravel_index(np.argmax(err - bound), err.shape)
            _err(rep, f"probability out of tolerance: sequence {b} row {k[0]} entry {k[1]}: {g[k]} vs {r[k]}")
        with np.errstate(divide="ignore", invalid="ignore"):
            rel = np.where(r > 1e-30, err / r, 0.0)
        rep.max_rel_err = max(rep.max_rel_err, float(rel.max()))


def _p_of(ids_row, vals_row, tok):
    k = int(np.searchsorted(ids_row, tok))
    if k < len(ids_row) and ids_row[k] == tok:
        return float(vals_row[k])
    return 0.0


def compare_step(got_accept_len, got_tokens, got_tok_prob, got_flags, got_ids, got_vals, got_cnt, ref: StepResult,
                 drafts, win_len, flags) -> ParityReport:
    """Full comparison of one step.  `ref` must have been computed with diag=True on the same inputs."""
    rep = ParityReport()
    B, W = got_tokens.shape
    win_len = np.asarray(win_len)
    compare_probs(rep, got_ids, got_vals, got_cnt, ref, win_len)
    d = ref.diag
    draft_all = bool(flags & FLAG_DRAFT_ALL)
    for b in range(B):
        L = int(win_len[b])
        rep.positions += L
        a = int(got_accept_len[b])
        if not (0 <= a <= L):
            _err(rep, f"sequence {b}: accept_len {a} outside [0, {L}]")
            continue
        if np.any(got_tokens[b, L:] != -1) or np.any(got_flags[b, L:] != OUT_INVALID) or np.any(got_tok_prob[b, L:] != 0):
            _err(rep, f"sequence {b}: rows beyond win_len are not blank")
        for i in range(L):
            tok, fl = int(got_tokens[b, i]), int(got_flags[b, i])
            if draft_all:
                expect_fl = OUT_RESAMPLED
            elif i < a:
                expect_fl = OUT_ACCEPTED
            elif i == a:
                expect_fl = OUT_RESIDUAL
            else:
                expect_fl = None  # reused or resampled
            if expect_fl is not None and fl != expect_fl:
                _err(rep, f"({b},{i}): flag {fl}, expected {expect_fl}")
                continue
            if not draft_all and i <= a:
                # the accept decision the other side took at this row
                took_ok = 1 if i < a else 0
                if int(d["pot_ok"][b, i]) != took_ok:
                    if d["accept_margin"][b, i] < MARGIN:
                        rep.flagged_accept += 1
                    else:
                        _err(rep, f"({b},{i}): accept decision {took_ok} vs oracle {int(d['pot_ok'][b, i])}, "
                                  f"margin {d['accept_margin'][b, i]:.3g}")
                        continue
            if fl == OUT_ACCEPTED:
                if tok != int(drafts[b, i]):
                    _err(rep, f"({b},{i}): accepted token is not the draft")
            elif fl == OUT_RESIDUAL:
                if tok != int(d["pot_residual"][b, i]):
                    if d["residual_margin"][b, i] < MARGIN:
                        rep.flagged_sample += 1
                    else:
                        _err(rep, f"({b},{i}): residual token {tok} vs oracle {int(d['pot_residual'][b, i])}, "
                                  f"margin {d['residual_margin'][b, i]:.3g}")
            elif fl in (OUT_REUSED, OUT_RESAMPLED):
                if not draft_all:
                    took_reuse = 1 if fl == OUT_REUSED else 0
                    if int(d["pot_reuse"][b, i]) != took_reuse:
                        if d["reuse_margin"][b, i] < MARGIN:
                            rep.flagged_reuse += 1
                        else:
                            _err(rep, f"({b},{i}): reuse decision {took_reuse} vs oracle {int(d['pot_reuse'][b, i])}, "
                                      f"margin {d['reuse_margin'][b, i]:.3g}")
                            continue
                if fl == OUT_REUSED:
                    if tok != int(drafts[b, i]):
                        _err(rep, f"({b},{i}): reused token is not the draft")
                elif tok != int(d["pot_redraft"][b, i]):
                    if d["redraft_margin"][b, i] < MARGIN:
                        rep.flagged_sample += 1
                    else:
                        _err(rep, f"({b},{i}): redraft token {tok} vs oracle {int(d['pot_redraft'][b, i])}, "
                                  f"margin {d['redraft_margin'][b, i]:.3g}")
            else:
                _err(rep, f"({b},{i}): unexpected flag {fl}")
            # the reported probability is the other side's own p of the emitted token, bit for bit, and
            # agrees with the oracle's p of that token
            own = _p_of(got_ids[b, i], got_vals[b, i], tok)
            if np.float32(own) != np.float32(got_tok_prob[b, i]):
                _err(rep, f"({b},{i}): tok_prob {got_tok_prob[b, i]} is not p(token) = {own}")
            refp = _p_of(ref.probs.ids[b, i], ref.probs.vals[b, i], tok)
            if abs(own - refp) > REL_TOL * abs(refp) + ABS_TOL:
                _err(rep, f"({b},{i}): tok_prob {own} vs oracle {refp}")
    return rep
