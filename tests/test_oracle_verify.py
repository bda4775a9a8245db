"""Pins for the oracle's verification rule (accept test, prefix, residual, inverse CDF) against the
closed forms of the paper's appendix proof, brute force and exhaustive sweeps."""
import itertools
import os

import numpy as np
import pytest
from scipy.stats import chi2 as chi2_dist

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "speculative_closed_forms.txt")


def _cases():
    out = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, p, q, acc, tot, res = [x.strip() for x in line.split("|")]
        f = lambda s: np.array([float(x) for x in s.split()], np.float64)
        out.append((name, f(p), f(q), f(acc), float(tot), f(res)))
    return out


CASES = _cases()


def _accept_threshold_count(p, q):
    """Exact number of 24-bit uniforms the oracle accepts for (p, q), by bisection on its own decision
    (the decision is monotone in u)."""
    lo, hi = 0, 1 << 24  # smallest n whose u = n/2^24 is rejected
    while lo < hi:
        mid = (lo + hi) // 2
        ok, _ = oracle.accept(np.float32(p), np.float32(q), np.float32(mid * 2.0 ** -24))
        if ok:
            lo = mid + 1
        else:
            hi = mid
    return lo


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_accept_probability_closed_form(case):
    _, p, q, acc, tot, _ = case
    probs = np.array([_accept_threshold_count(pi, qi) / 2.0 ** 24 for pi, qi in zip(p, q)])
    np.testing.assert_allclose(probs, acc, atol=2e-7)
    assert abs(float((q * probs).sum()) - tot) < 1e-6  # Eq. joint-ac summed over tokens


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_residual_weights_closed_form(case):
    _, p, q, _, tot, res = case
    V = len(p)
    ids = np.arange(V, dtype=np.int32)
    w = oracle.residual_weights(ids, p.astype(np.float32), ids, q.astype(np.float32), V, V).astype(np.float64)
    assert abs(w.sum() - (1.0 - tot)) < 1e-6  # Eq. demon-rej
    np.testing.assert_allclose(w / w.sum(), res, atol=1e-6)
    assert np.all(w[p <= q] == 0)


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_exact_marginal_preservation_by_enumeration(case):
    # sum_d q(d) [acc(d) 1{x=d} + (1-acc(d)) res(x)] = p(x), with the oracle's own acc and res
    _, p, q, _, _, _ = case
    V = len(p)
    ids = np.arange(V, dtype=np.int32)
    acc = np.array([_accept_threshold_count(pi, qi) / 2.0 ** 24 for pi, qi in zip(p, q)])
    w = oracle.residual_weights(ids, p.astype(np.float32), ids, q.astype(np.float32), V, V).astype(np.float64)
    res = w / w.sum()
    out = q * acc + float((q * (1 - acc)).sum()) * res
    np.testing.assert_allclose(out, p, atol=1e-6)


def test_residual_with_sparse_and_uniform_q():
    p_ids = np.array([1, 4, 6, 9], np.int32)
    p_vals = np.array([0.4, 0.3, 0.2, 0.1], np.float32)
    q_ids = np.array([0, 4, 9, 11], np.int32)
    q_vals = np.array([0.5, 0.1, 0.3, 0.1], np.float32)
    w = oracle.residual_weights(p_ids, p_vals, q_ids, q_vals, 4, 16)
    np.testing.assert_allclose(w, [0.4, 0.2, 0.2, 0.0], atol=1e-7)
    w = oracle.residual_weights(p_ids, p_vals, q_ids, q_vals, oracle.Q_UNIFORM, 16)
    np.testing.assert_allclose(w, np.maximum(0, p_vals - np.float32(1 / 16)), atol=1e-7)


def test_first_reject_brute_force_all_masks():
    for W in range(0, 13):
        for bits in itertools.product([0, 1], repeat=W) if W <= 10 else []:
            m = sum(b << i for i, b in enumerate(bits))
            expect = ((~m & (m + 1)).bit_length() - 1) if W else 0
            expect = min(expect, W)
            assert oracle.first_reject(np.array(bits, np.int32)) == expect
    # all masks for W = 11, 12 through integers (faster than itertools)
    for W in (11, 12):
        for m in range(1 << W):
            bits = np.array([(m >> i) & 1 for i in range(W)], np.int32)
            expect = min(((~m & (m + 1)).bit_length() - 1), W)
            assert oracle.first_reject(bits) == expect


def test_icdf_exhaustive_sweep_of_t():
    # weights that are exact multiples of 2^-40: the fixed-point weights are the multipliers
    n = np.array([3, 0, 5, 1, 0, 7, 2, 6], np.int64)
    w = (n.astype(np.float64) * 2.0 ** -40).astype(np.float32)
    T = int(n.sum())
    counts = np.zeros(len(n), np.int64)
    prev = -1
    for t in range(T):
        R = -(-(t << 64) // T)  # smallest R with floor(R T / 2^64) = t
        k, margin = oracle.icdf(w, R)
        lo, hi = int(n[:k].sum()), int(n[: k + 1].sum())
        assert lo <= t < hi
        assert abs(margin - min(t - lo, hi - t) * 2.0 ** -40) < 1e-18
        assert k >= prev
        prev = k
        counts[k] += 1
        # the last R that still maps to t gives the same answer
        R2 = min(((t + 1) << 64) // T - (0 if ((t + 1) << 64) % T else 1), (1 << 64) - 1)
        assert oracle.icdf(w, R2)[0] == k
    assert counts.tolist() == n.tolist()


def test_icdf_edge_cases():
    assert oracle.icdf(np.zeros(4, np.float32), 12345)[0] == -1
    assert oracle.icdf(np.array([0, 0, 1.0, 0], np.float32), 0)[0] == 2
    assert oracle.icdf(np.array([0, 0, 1.0, 0], np.float32), (1 << 64) - 1)[0] == 2
    assert oracle.icdf(np.array([0.5, 0.5], np.float32), (1 << 63) - 1)[0] == 0
    assert oracle.icdf(np.array([0.5, 0.5], np.float32), 1 << 63)[0] == 1
    # negative weights count as zero, weights below 2^-40 vanish
    assert oracle.icdf(np.array([-1.0, 2.0 ** -41, 0.25], np.float32), 0)[0] == 2


def _one_position_trials(p, q, n_trials, seed, flags):
    """n_trials independent one-row steps (B = n_trials, W = 1) with drafts drawn from q."""
    V = len(p)
    rng = np.random.default_rng(seed)
    drafts = rng.choice(V, size=(n_trials, 1), p=q / q.sum()).astype(np.int32)
    logits = np.broadcast_to(np.log(p).astype(np.float32), (n_trials, 1, V)).copy()
    qp = oracle.Probs.empty(n_trials, 1, V)
    qp.ids[:] = np.arange(V, dtype=np.int32)
    qp.vals[:] = q.astype(np.float32)
    qp.cnt[:] = V
    qp.tok_prob[:, 0] = q.astype(np.float32)[drafts[:, 0]]
    res = oracle.sjd_step(logits, None, drafts, qp, dtype=oracle.F32, V=V, top_k=V, flags=flags, seed=seed + 1000,
                          diag=True)
    return drafts[:, 0], res


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_million_trials_match_closed_forms(case):
    _, p, q, acc, tot, resd = case
    V = len(p)
    N = 1_000_000
    drafts, r = _one_position_trials(p, q, N, seed=17, flags=0)
    accepted = r.accept_len == 1
    # acceptance rate per drafted token: min(1, p/q)  (Eq. ac-prob), 4.5 sigma
    for d in range(V):
        sel = drafts == d
        n = int(sel.sum())
        rate = float(accepted[sel].mean())
        sigma = max(np.sqrt(acc[d] * (1 - acc[d]) / n), 1e-9)
        assert abs(rate - acc[d]) <= 4.5 * sigma + 1e-6, (d, rate, acc[d])
    # total acceptance: sum min(p, q)
    assert abs(float(accepted.mean()) - tot) < 4.5 * np.sqrt(tot * (1 - tot) / N)
    # accepted rows emit the draft, rejected rows emit a token with p > q
    out = r.tokens[:, 0]
    assert np.all(out[accepted] == drafts[accepted])
    assert np.all((p > q)[out[~accepted]])
    assert np.all(r.flags[accepted, 0] == oracle.OUT_ACCEPTED) and np.all(r.flags[~accepted, 0] == oracle.OUT_RESIDUAL)
    # residual distribution: chi-square against max(0, p-q) / sum  (Eq. resample-prob)
    sup = resd > 0
    obs = np.bincount(out[~accepted], minlength=V)[sup]
    if sup.sum() > 1:
        exp = resd[sup] * obs.sum()
        stat = float(((obs - exp) ** 2 / exp).sum())
        assert stat < chi2_dist.ppf(1 - 1e-5, int(sup.sum()) - 1), stat
    # Theorem 1: the emitted token is distributed as p
    obs = np.bincount(out, minlength=V)
    exp = p * N
    stat = float(((obs - exp) ** 2 / exp).sum())
    assert stat < chi2_dist.ppf(1 - 1e-5, V - 1), stat
    # emitted probability is p of the emitted token
    pf = r.probs.vals[0, 0]
    np.testing.assert_allclose(pf, p, rtol=1e-6)
    assert np.all(r.probs.tok_prob[:, 0] == pf[out])


def test_wrong_rules_would_fail_the_marginal_check():
    # the chi-square above has the power to catch a plausible mistake: emitting the draft
    # unconditionally (marginal q) or resampling from p instead of the residual
    _, p, q, _, _, _ = CASES[0]
    N = 200_000
    rng = np.random.default_rng(3)
    bad = rng.choice(len(p), size=N, p=q)
    obs = np.bincount(bad, minlength=len(p))
    assert float(((obs - p * N) ** 2 / (p * N)).sum()) > 1000
    acc = np.minimum(1, p / q)
    d = rng.choice(len(p), size=N, p=q)
    rej = rng.random(N) >= acc[d]
    d[rej] = rng.choice(len(p), size=int(rej.sum()), p=p)
    obs = np.bincount(d, minlength=len(p))
    assert float(((obs - p * N) ** 2 / (p * N)).sum()) > 1000
