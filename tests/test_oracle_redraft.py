"""Pins of the oracle's redraft draw: rows behind the first rejection, when they are not kept, are drawn from
this call's own distribution p_i of that row (Eq. reuse second case; Eq. refine-sjd for plain SJD), and so
is every row of a call that drafts all rows.

The expected distributions are written out here with numpy in double precision (top-K of the row's logits,
renormalised) and never come from the oracle.  The cases are built so that a plausible mistake - drawing the
later row from the residual max(0, p - q), from another row's distribution, or from the reference q - moves
the chi-square statistic by more than a thousand.
"""
import numpy as np
import pytest
from scipy.stats import chi2 as chi2_dist

import oracle

V, K, N = 6, 5, 1_000_000

# row distributions before top-K (each row drops its smallest entry and renormalises)
ROW_P = np.array([[0.30, 0.05, 0.25, 0.10, 0.20, 0.10],
                  [0.08, 0.32, 0.04, 0.26, 0.12, 0.18],
                  [0.22, 0.11, 0.33, 0.03, 0.09, 0.22]], dtype=np.float64)
# reference of row 1: far from p_1, so that the residual of row 1 is far from p_1 as well.  Five entries, like
# every sparse row of a call with top-K = 5.
Q1 = np.array([0.40, 0.05, 0.35, 0.0, 0.10, 0.10], dtype=np.float64)
Q1_IDS = np.flatnonzero(Q1).astype(np.int32)


def _reference(drafts):
    """Row 0: uniform over the vocabulary; row 1: Q1 as a sparse row."""
    qp = oracle.Probs.empty(N, 2, K)
    qp.cnt[:, 0] = oracle.Q_UNIFORM
    qp.tok_prob[:, 0] = np.float32(1.0) / np.float32(V)
    qp.ids[:, 1] = Q1_IDS
    qp.vals[:, 1] = Q1[Q1_IDS].astype(np.float32)
    qp.cnt[:, 1] = K
    qp.tok_prob[:, 1] = Q1.astype(np.float32)[drafts[:, 1]]
    return qp


def _top_k_renormalised(p, k):
    keep = np.sort(np.argsort(-p, kind="stable")[:k])
    out = np.zeros_like(p)
    out[keep] = p[keep] / p[keep].sum()
    return out


def _chi2(obs, expected_p):
    sup = expected_p > 0
    assert obs[~sup].sum() == 0, "a token outside the expected support was drawn"
    exp = expected_p[sup] * obs.sum()
    return float(((obs[sup] - exp) ** 2 / exp).sum()), int(sup.sum()) - 1


def _chi2_any(obs, expected_p):
    """Statistic against a candidate law that may have zeros where tokens were observed (then it is infinite)."""
    sup = expected_p > 0
    if obs[~sup].sum() > 0:
        return np.inf
    exp = expected_p[sup] * obs.sum()
    return float(((obs[sup] - exp) ** 2 / exp).sum())


def _logits(W):
    return np.broadcast_to(np.log(ROW_P[:W]).astype(np.float32), (N, W, V)).copy()


def test_rows_behind_the_rejection_are_drawn_from_their_own_distribution():
    W = 2
    p0, p1 = _top_k_renormalised(ROW_P[0], K), _top_k_renormalised(ROW_P[1], K)
    out0 = int(np.argmin(ROW_P[0]))  # the token top-K drops at row 0: a draft there has p = 0 and is rejected
    rng = np.random.default_rng(5)
    drafts = np.empty((N, W), np.int32)
    drafts[:, 0] = out0
    drafts[:, 1] = rng.choice(V, size=N, p=Q1)
    qp = _reference(drafts)
    r = oracle.sjd_step(_logits(W), None, drafts, qp, dtype=oracle.F32, V=V, top_k=K, flags=0, seed=99, n_threads=8)
    assert np.all(r.accept_len == 0)
    assert np.all(r.flags[:, 0] == oracle.OUT_RESIDUAL) and np.all(r.flags[:, 1] == oracle.OUT_RESAMPLED)
    obs = np.bincount(r.tokens[:, 1], minlength=V)
    stat, dof = _chi2(obs, p1)
    assert stat < chi2_dist.ppf(1 - 1e-5, dof), stat
    # the same counts refute the plausible mistakes
    resid1 = np.maximum(0.0, p1 - Q1)
    resid1 /= resid1.sum()
    for name, wrong in (("residual of row 1", resid1), ("row 0's distribution", p0), ("reference q of row 1", Q1),
                        ("row 1 without top-K", ROW_P[1])):
        assert _chi2_any(obs, wrong) > 1000, name
    # row 0 itself: the residual of p_0 against the uniform reference (Eq. rej-sjd)
    resid0 = np.maximum(0.0, p0 - 1.0 / V)
    resid0 /= resid0.sum()
    stat, dof = _chi2(np.bincount(r.tokens[:, 0], minlength=V), resid0)
    assert stat < chi2_dist.ppf(1 - 1e-5, dof), stat
    # the probability reported with a token is this call's p_i of that token
    np.testing.assert_allclose(r.probs.tok_prob[:, 1], p1[r.tokens[:, 1]], rtol=2e-6)


def test_a_kept_row_is_not_redrawn_and_a_dropped_one_is():
    # with reuse on, row 1 keeps its draft exactly when p_1(x) / q_1(x) > tau; the others are drawn from p_1
    W, tau = 2, 0.9
    p1 = _top_k_renormalised(ROW_P[1], K)
    out0 = int(np.argmin(ROW_P[0]))
    rng = np.random.default_rng(6)
    drafts = np.empty((N, W), np.int32)
    drafts[:, 0] = out0
    drafts[:, 1] = rng.choice(V, size=N, p=Q1)
    qp = _reference(drafts)
    r = oracle.sjd_step(_logits(W), None, drafts, qp, dtype=oracle.F32, V=V, top_k=K, reuse_tau=tau,
                        flags=oracle.FLAG_REUSE, seed=7, n_threads=8)
    keep_token = p1 > tau * Q1  # p / q > tau; a token the reference never proposes does not occur as a draft
    kept = keep_token[drafts[:, 1]]
    assert np.all(r.flags[kept, 1] == oracle.OUT_REUSED) and np.all(r.tokens[kept, 1] == drafts[kept, 1])
    assert np.all(r.flags[~kept, 1] == oracle.OUT_RESAMPLED)
    obs = np.bincount(r.tokens[~kept, 1], minlength=V)
    stat, dof = _chi2(obs, p1)
    assert stat < chi2_dist.ppf(1 - 1e-5, dof), stat
    assert _chi2_any(obs, Q1) > 1000


def test_drafting_every_row_draws_each_from_its_own_distribution():
    W = 3
    r = oracle.sjd_step(_logits(W), None, None, None, dtype=oracle.F32, V=V, top_k=K, flags=oracle.FLAG_DRAFT_ALL,
                        seed=123, n_threads=8)
    rows = [_top_k_renormalised(ROW_P[i], K) for i in range(W)]
    for i in range(W):
        obs = np.bincount(r.tokens[:, i], minlength=V)
        stat, dof = _chi2(obs, rows[i])
        assert stat < chi2_dist.ppf(1 - 1e-5, dof), (i, stat)
        for j in range(W):
            if j != i:
                assert _chi2_any(obs, rows[j]) > 1000, (i, j)
    # rows of one sequence are drawn independently of one another: the joint counts of rows 0 and 1 factorise
    joint = np.zeros((V, V))
    np.add.at(joint, (r.tokens[:, 0], r.tokens[:, 1]), 1)
    exp = np.outer(rows[0], rows[1]) * N
    sup = exp > 0
    stat = float(((joint[sup] - exp[sup]) ** 2 / exp[sup]).sum())
    assert stat < chi2_dist.ppf(1 - 1e-5, int(sup.sum()) - 1), stat
