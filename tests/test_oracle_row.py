"""Pins for the oracle's sampling head (guidance merge, temperature, top-K, softmax)."""
import math

import numpy as np
import pytest
import torch
from scipy.special import softmax as scipy_softmax

import oracle
from paper_2512_07503_b200 import workloads as wk


def _dense(ids, vals, V):
    d = np.zeros(V, np.float64)
    d[ids] = vals
    return d


def test_matches_fp64_library_topk_softmax():
    rng = np.random.default_rng(1)
    V, K = 4096, 64
    x = (rng.standard_normal(V) * 2).astype(np.float32)
    ids, vals, dg = oracle.row_probs(x, None, oracle.F32, 1.0, 1.0, K)
    t = torch.from_numpy(x).double()
    tv, ti = torch.topk(t, K)
    ref = torch.zeros(V, dtype=torch.float64)
    ref[ti] = torch.softmax(tv, dim=0)
    assert dg == 0
    assert sorted(ti.tolist()) == ids.tolist()
    np.testing.assert_allclose(_dense(ids, vals, V), ref.numpy(), rtol=2e-7, atol=0)


def test_k_geq_v_is_plain_softmax():
    rng = np.random.default_rng(2)
    V = 257
    x = rng.standard_normal(V).astype(np.float32) * 3
    for K in (V, V + 5, 10 * V):
        ids, vals, _ = oracle.row_probs(x, None, oracle.F32, 1.0, 1.0, K)
        assert ids.tolist() == list(range(V))
        np.testing.assert_allclose(vals, scipy_softmax(x.astype(np.float64)), rtol=2e-7)


def test_k1_is_one_hot_at_lowest_argmax():
    x = np.array([0.5, 3.0, -1.0, 3.0, 2.0, 3.0], np.float32)
    ids, vals, _ = oracle.row_probs(x, None, oracle.F32, 1.0, 1.0, 1)
    assert ids.tolist() == [1] and vals.tolist() == [1.0]


def test_guidance_direction_and_scale_exact_small_integers():
    # integer logits: every fp32 operation is exact, so the merged logits are exactly
    # u + s (c - u) and the expected distribution is a closed form
    c = np.array([2, -1, 0, 3, 1, -2, 0, 1], np.float32)
    u = np.array([1, 0, 0, 1, 2, -1, -3, 1], np.float32)
    s = 3.0
    g = [float(ui + s * (ci - ui)) for ci, ui in zip(c, u)]
    m = max(g)
    e = [math.exp(x - m) for x in g]
    ref = np.array(e) / sum(e)
    ids, vals, _ = oracle.row_probs(c, u, oracle.F32, s, 1.0, 8)
    assert ids.tolist() == list(range(8))
    np.testing.assert_allclose(vals, ref, rtol=2e-7)
    # swapping the operands must give something else (guards against a transposed merge)
    _, swapped, _ = oracle.row_probs(u, c, oracle.F32, s, 1.0, 8)
    assert np.abs(swapped - ref).max() > 1e-2
    # s = 0 returns the unconditional distribution, s with c == u changes nothing
    _, v0, _ = oracle.row_probs(c, u, oracle.F32, 0.0, 1.0, 8)
    np.testing.assert_allclose(v0, scipy_softmax(u.astype(np.float64)), rtol=2e-7)
    _, vs, _ = oracle.row_probs(c, c, oracle.F32, 7.0, 1.0, 8)
    np.testing.assert_allclose(vs, scipy_softmax(c.astype(np.float64)), rtol=2e-7)


def test_temperature_scales_logits_before_softmax():
    c = np.array([0, 1, 2, 3, -1, 0.5, 1.5, 2.5], np.float32)
    # inv_T = 2 and 0.5 are exact in fp32
    for inv_t in (2.0, 0.5):
        ids, vals, _ = oracle.row_probs(c, None, oracle.F32, 1.0, inv_t, 8)
        np.testing.assert_allclose(vals, scipy_softmax(c.astype(np.float64) * inv_t), rtol=2e-7)
    # with top-K: the kept set is the K largest of the scaled logits, renormalised
    ids, vals, _ = oracle.row_probs(c, None, oracle.F32, 1.0, 2.0, 3)
    assert ids.tolist() == [2, 3, 7]
    np.testing.assert_allclose(vals, scipy_softmax(np.array([2, 3, 2.5]) * 2.0), rtol=2e-7)


def test_ties_break_to_lower_id_with_bf16_logits():
    rng = np.random.default_rng(5)
    V, K = 8192, 500
    x = wk.to_bf16_bits((rng.standard_normal(V) * 1.5).astype(np.float32))
    xf = wk.bf16_bits_to_f32(x)
    ids, vals, _ = oracle.row_probs(x, None, oracle.BF16, 1.0, 1.0, K)
    order = np.lexsort((np.arange(V), -xf.astype(np.float64)))  # by value descending, then id ascending
    expect = np.sort(order[:K])
    assert ids.tolist() == expect.tolist()
    thr = xf[order[K - 1]]
    assert (xf == thr).sum() > 1, "the case must contain a tie at the threshold to mean anything"
    assert xf[order[K]] == thr, "the tie must straddle the cut"
    # bf16 storage is read exactly
    ref = scipy_softmax(xf[expect].astype(np.float64))
    np.testing.assert_allclose(vals, ref, rtol=2e-7)


def test_invariants_on_benchmark_like_rows():
    wl = wk.CONFIGS["cfg2"].scaled(B=1, W=3)
    inp = wk.make_step_inputs(wl)
    for i in range(wl.W):
        ids, vals, dg = oracle.row_probs(inp.cond[0, i], inp.uncond[0, i], wl.dtype, wl.cfg_scale,
                                         float(wl.inv_temperature), wl.top_k)
        assert dg == 0
        assert len(ids) == wl.top_k and np.all(np.diff(ids) > 0) and ids[0] >= 0 and ids[-1] < wl.V
        assert np.all(vals > 0)
        assert abs(float(vals.astype(np.float64).sum()) - 1.0) < 1e-6
        # kept logits dominate dropped ones (merge recomputed in float64; exact for bf16 inputs up to the
        # fp32 roundings, hence the small slack)
        c = wk.bf16_bits_to_f32(inp.cond[0, i]).astype(np.float64)
        u = wk.bf16_bits_to_f32(inp.uncond[0, i]).astype(np.float64)
        g = u + wl.cfg_scale * (c - u)
        mask = np.zeros(wl.V, bool)
        mask[ids] = True
        assert g[mask].min() >= g[~mask].max() - 1e-5
        # probabilities are ordered like the merged logits
        np.testing.assert_allclose(vals, scipy_softmax(g[ids]), rtol=3e-6)


def test_masked_and_degenerate_rows():
    ninf = -np.inf
    x = np.array([ninf, 1.0, ninf, 0.0, ninf, ninf], np.float32)
    ids, vals, dg = oracle.row_probs(x, None, oracle.F32, 1.0, 1.0, 4)
    assert dg == 0
    assert ids.tolist() == [0, 1, 2, 3]  # two finite, then the lowest-id masked entries
    np.testing.assert_allclose(vals, [0.0, math.e / (1 + math.e), 0.0, 1 / (1 + math.e)], rtol=2e-7)
    x[:] = ninf
    ids, vals, dg = oracle.row_probs(x, None, oracle.F32, 1.0, 1.0, 3)
    assert dg == 1 and ids.tolist() == [0, 1, 2] and vals.tolist() == [0, 0, 0]
    # masked in both branches: (-inf) - (-inf) is NaN, which ranks as masked
    c = np.array([ninf, 2.0, 1.0], np.float32)
    u = np.array([ninf, 1.0, 1.0], np.float32)
    ids, vals, dg = oracle.row_probs(c, u, oracle.F32, 3.0, 1.0, 2)
    assert ids.tolist() == [1, 2] and dg == 0
    np.testing.assert_allclose(vals, scipy_softmax(np.array([4.0, 1.0])), rtol=2e-7)


@pytest.mark.parametrize("V,K", [(8, 3), (33, 33), (1000, 1), (4096, 4095)])
def test_sum_and_count(V, K):
    rng = np.random.default_rng(V * 7 + K)
    c = rng.standard_normal(V).astype(np.float32) * 2
    u = rng.standard_normal(V).astype(np.float32) * 2
    ids, vals, _ = oracle.row_probs(c, u, oracle.F32, 3.0, np.float32(1 / 0.9), K)
    assert len(ids) == min(K, V)
    assert abs(float(vals.astype(np.float64).sum()) - 1.0) < 1e-6


def test_half_precision_patterns_decode_like_numpy_for_all_65536_values():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))   # bit for bit, signed zeros included


def test_fp16_rows_equal_the_same_values_given_as_fp32():
    rng = np.random.default_rng(5)
    V = 1024
    c16 = (rng.standard_normal(V) * 3).astype(np.float16)
    u16 = (c16.astype(np.float32) + rng.standard_normal(V).astype(np.float32)).astype(np.float16)
    a = oracle.row_probs(c16.view(np.uint16), u16.view(np.uint16), oracle.F16, 3.0, 1.0, 50)
    b = oracle.row_probs(c16.astype(np.float32), u16.astype(np.float32), oracle.F32, 3.0, 1.0, 50)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
