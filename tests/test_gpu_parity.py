"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2512_07503_b200 import workloads as wk

pytestmark = pytest.mark.gpu


def _run(wl, flags=None, **over):
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    inp = wk.make_step_inputs(wl)
    prev = oracle_prime(inp)
    kw = step_kwargs(inp, **over)
    if flags is not None:
        kw["flags"] = flags
    rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, kw, inp.win_len)
    print(wl.name, rep.summary(), "accept_len", got.accept_len[:8])
    return rep, got, ref, inp, prev


def test_draft_all_cfg1():
    from gpu_harness import check_parity, step_kwargs
    wl = wk.CONFIGS["cfg1"]
    inp = wk.make_step_inputs(wl)
    kw = step_kwargs(inp, flags=oracle.FLAG_DRAFT_ALL, iteration0=0)
    rep, got, ref = check_parity(inp.prev_cond, inp.prev_uncond, None, None, kw, inp.win_len)
    assert np.all(got.accept_len == 0)


def test_cfg1_full_step():
    _run(wk.CONFIGS["cfg1"])


def test_cfg1_plain_sjd():
    _run(wk.CONFIGS["cfg1"], flags=0)


def test_cfg2_bf16_reduced_window():
    _run(wk.CONFIGS["cfg2"].scaled(W=8))


def test_cfg3_ragged_reduced_batch():
    _run(wk.CONFIGS["cfg3"].scaled(B=12))


@pytest.mark.parametrize("V,K,W", [(8, 3, 1), (40, 40, 5), (264, 1, 33), (4096, 4095, 4), (1032, 7, 64),
                                   (8200, 2000, 3), (2048, 5000, 2)])
def test_shapes_spanning_tiles_and_tails(V, K, W):
    _run(wk.CONFIGS["cfg1"].scaled(B=3, W=W, V=V, top_k=K, seed=V + K))


def test_bf16_ties_at_the_threshold():
    # few distinct values: most of the row ties with the K-th largest
    wl = wk.CONFIGS["cfg2"].scaled(B=2, W=4, V=4096, top_k=300, sigma=0.05, peaks=0)
    rep, got, ref, inp, prev = _run(wl)
    xf = wk.bf16_bits_to_f32(inp.cond[0, 0])
    assert len(np.unique(xf)) < 2000


def test_all_equal_logits():
    from gpu_harness import check_parity, step_kwargs
    wl = wk.CONFIGS["cfg1"].scaled(B=2, W=3, V=1024, top_k=100)
    inp = wk.make_step_inputs(wl)
    inp.cond[:] = 1.5
    inp.uncond[:] = 1.5
    q = oracle.Probs.uniform(wl.B, wl.W, wl.kcap, wl.V)
    drafts = np.arange(wl.B * wl.W, dtype=np.int32).reshape(wl.B, wl.W) * 37 % wl.V
    rep, got, ref = check_parity(inp.cond, inp.uncond, drafts, q, step_kwargs(inp), inp.win_len)
    assert np.array_equal(got.ids[0, 0], np.arange(100))


def test_masked_and_degenerate_rows():
    from gpu_harness import check_parity, step_kwargs
    wl = wk.CONFIGS["cfg1"].scaled(B=2, W=4, V=512, top_k=64)
    inp = wk.make_step_inputs(wl)
    inp.cond[0, 0, 100:] = -np.inf          # fewer finite logits than K
    inp.uncond[0, 0, 100:] = -np.inf        # masked in both branches: NaN after the merge
    inp.cond[0, 1, :] = -np.inf             # nothing finite
    inp.cond[1, 2, ::2] = -np.inf
    q = oracle.Probs.uniform(wl.B, wl.W, wl.kcap, wl.V)
    drafts = np.full((wl.B, wl.W), 5, np.int32)
    rep, got, ref = check_parity(inp.cond, inp.uncond, drafts, q, step_kwargs(inp), inp.win_len)
    assert got.status[0] & oracle.STATUS_DEGENERATE_ROW


def test_no_guidance_and_temperature():
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = wk.CONFIGS["cfg3"].scaled(B=4, V=2048, top_k=200, temperature=0.7)
    inp = wk.make_step_inputs(wl)
    prev = oracle_prime(inp)
    check_parity(inp.cond, None, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len)


def test_identical_distributions_accept_everything():
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = wk.CONFIGS["cfg1"].scaled(B=4, W=20)
    inp = wk.make_step_inputs(wl)
    inp.prev_cond, inp.prev_uncond = inp.cond, inp.uncond
    prev = oracle_prime(inp)
    rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len)
    assert np.all(ref.accept_len == wl.W)


def test_empty_and_ragged_windows_and_iterations():
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = wk.CONFIGS["cfg1"].scaled(B=5, W=9, V=512, top_k=40)
    inp = wk.make_step_inputs(wl)
    inp.win_len[:] = [0, 1, 9, 4, 0]
    inp.pos_base[:] = [0, 575, 3, 100, 7]
    prev = oracle_prime(inp)
    kw = step_kwargs(inp, iteration=np.array([3, 1, 4, 1, 5], np.int32))
    check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, kw, inp.win_len)


def test_reuse_thresholds():
    for tau in (-1.0, 0.0, 0.5, 2.0, np.inf):
        _run(wk.CONFIGS["cfg1"].scaled(B=4, reuse_tau=tau))


def test_bad_arguments_are_refused_on_the_host():
    import torch
    import paper_2512_07503_b200 as sjd
    dev = "cuda:0"
    logits = torch.zeros(1, 2, 64, device=dev)
    out = sjd.DeviceProbs.empty(1, 2, 8, dev)
    acc = torch.zeros(1, dtype=torch.int32, device=dev)
    toks = torch.zeros(1, 2, dtype=torch.int32, device=dev)
    ws = torch.empty(4096, dtype=torch.uint8, device=dev)
    flags = sjd.binding.SJD_FLAG_DRAFT_ALL
    p = sjd.make_params(logits, top_k=8, flags=flags, workspace=ws)
    sjd.sjd_step(logits, None, None, None, p, 0, acc, toks, out)  # fine
    for mutate, code in [(lambda p: setattr(p, "top_k", 0), -2), (lambda p: setattr(p, "V", 60), -2),
                         (lambda p: setattr(p, "W", 513), -2), (lambda p: setattr(p, "logits_dtype", 9), -4),
                         (lambda p: setattr(p, "workspace_bytes", 8), -5), (lambda p: setattr(p, "struct_size", 4), -6),
                         (lambda p: setattr(p, "stride_w", 65), -3), (lambda p: setattr(p, "flags", 0), -1)]:
        p = sjd.make_params(logits, top_k=8, flags=flags, workspace=ws)
        mutate(p)
        with pytest.raises(sjd.SjdError, match=f"sjd error {code}"):
            sjd.sjd_step(logits, None, None, None, p, 0, acc, toks, out)
    torch.cuda.synchronize()


# ---- shapes the single-pass pipelined kernel takes, driven into its rare paths ----
def _pipeline_case(V=8192, K=200, B=2, W=6, dtype_cfg="cfg1", **scaled):
    return wk.CONFIGS[dtype_cfg].scaled(B=B, W=W, V=V, top_k=K, **scaled)


def test_pipeline_rows_with_few_finite_logits_and_an_infinite_logit():
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = _pipeline_case()
    inp = wk.make_step_inputs(wl)
    inp.cond[0, 0, 150:] = -np.inf           # fewer finite logits than K: the candidates cannot hold the top-K
    inp.uncond[0, 0, 150:] = -np.inf
    inp.cond[0, 1, :] = -np.inf              # nothing finite
    inp.cond[0, 2, 77] = np.inf              # an infinite logit: no finite maximum
    inp.cond[1, 3, ::3] = -np.inf
    prev = oracle_prime(inp)
    rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len)
    assert got.status[0] & oracle.STATUS_DEGENERATE_ROW


def test_pipeline_all_equal_logits_overflow_the_candidate_lists():
    from gpu_harness import check_parity, step_kwargs
    wl = _pipeline_case(V=4096, K=64, B=1, W=3)
    inp = wk.make_step_inputs(wl)
    inp.cond[:] = 0.25
    inp.uncond[:] = 0.25
    q = oracle.Probs.uniform(wl.B, wl.W, wl.kcap, wl.V)
    drafts = np.array([[3, 70, 4000]], np.int32)
    rep, got, ref = check_parity(inp.cond, inp.uncond, drafts, q, step_kwargs(inp), inp.win_len)
    assert np.array_equal(got.ids[0, 0], np.arange(64))
    assert got.status[0] & 16          # SJD_STATUS_ROW_REDONE: the rows went through the any-shape path


def test_pipeline_bf16_ties_at_the_threshold():
    # few distinct values: the threshold bin holds more members than the on-chip ranking takes
    wl = wk.CONFIGS["cfg2"].scaled(B=2, W=3, V=16384, top_k=500, sigma=0.05, peaks=0)
    rep, got, ref, inp, prev = _run(wl)
    assert len(np.unique(wk.bf16_bits_to_f32(inp.cond[0, 0]))) < 2000


def test_pipeline_k1_no_guidance_and_temperature():
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    _run(_pipeline_case(V=4096, K=1, B=2, W=5))
    wl = wk.CONFIGS["cfg3"].scaled(B=3, V=16384, top_k=700, temperature=0.7)
    inp = wk.make_step_inputs(wl)
    prev = oracle_prime(inp)
    check_parity(inp.cond, None, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len)


def test_pipeline_structured_row_defeats_the_sample():
    # every sample tile (every 8th tile of 256) is very negative: the sampled threshold is far too low,
    # the lists overflow and the row is redone exactly
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = _pipeline_case(V=8192, K=100, B=1, W=2)
    inp = wk.make_step_inputs(wl)
    for t in range(0, 32, 8):
        inp.cond[:, :, t * 256:(t + 1) * 256] -= 50.0
        inp.uncond[:, :, t * 256:(t + 1) * 256] -= 50.0
    prev = oracle_prime(inp)
    rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, step_kwargs(inp, flags=oracle.FLAG_REUSE | 8),
                                 inp.win_len)
    assert got.status[0] & 16
    # and the opposite: the sample tiles hold the largest values, so the threshold is too high
    inp2 = wk.make_step_inputs(wl)
    for t in range(0, 32, 8):
        inp2.cond[:, :, t * 256:(t + 1) * 256] += 50.0
        inp2.uncond[:, :, t * 256:(t + 1) * 256] += 50.0
    prev2 = oracle_prime(inp2)
    rep, got, ref = check_parity(inp2.cond, inp2.uncond, prev2.tokens, prev2.probs,
                                 step_kwargs(inp2, flags=oracle.FLAG_REUSE | 8), inp2.win_len)
    assert got.status[0] & 16


@pytest.mark.parametrize("dtype,V,K", [(wk.BF16, 16384, 500), (wk.F32, 16384, 300), (wk.BF16, 16384, 2000)])
def test_range_kernel_structured_row_defeats_the_sample(dtype, V, K):
    # the range kernel samples the first 64 bytes of each of the 256 id ranges of a row: make exactly those
    # entries very small (threshold far too low, lists overflow) or very large (too few candidates); both
    # ways the row is redone by the any-shape path and stays exact
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = wk.CONFIGS["cfg2"].scaled(B=1, W=3, V=V, top_k=K, dtype=dtype)
    R, bw = V // 256, 64 // (2 if dtype == wk.BF16 else 4)
    sample = (np.arange(V) % R) < bw
    for shift in (-50.0, 50.0):
        inp = wk.make_step_inputs(wl)
        for arr in (inp.cond, inp.uncond):
            if dtype == wk.BF16:
                f = wk.bf16_bits_to_f32(arr)
                f[:, :, sample] += np.float32(shift)
                arr[:] = wk.to_bf16_bits(f)
            else:
                arr[:, :, sample] += np.float32(shift)
        prev = oracle_prime(inp)
        rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len)
        assert got.status[0] & 16, shift


def test_ordinary_rows_are_not_redone():
    rep, got, ref, inp, prev = _run(wk.CONFIGS["cfg2"].scaled(W=8))
    assert not (got.status[0] & 16)
    rep, got, ref, inp, prev = _run(wk.SWEEP["v16k"].scaled(B=2, W=8))
    assert not np.any(got.status & 16)


@pytest.mark.parametrize("force", [4, 8])  # SJD_FLAG_FORCE_GENERIC, SJD_FLAG_FORCE_TILES
def test_every_row_kernel_gives_the_same_answer(force):
    # the same shapes through the any-shape kernel and the tile-dealing kernel instead of the range kernel
    _run(wk.CONFIGS["cfg2"].scaled(W=6), flags=oracle.FLAG_REUSE | force)
    _run(wk.CONFIGS["cfg2"].scaled(W=6, top_k=1000), flags=oracle.FLAG_REUSE | force)   # a shape the tile kernel takes
    _run(wk.CONFIGS["cfg3"].scaled(B=6), flags=oracle.FLAG_REUSE | force)


@pytest.mark.parametrize("V,K", [(16384, 300), (4096, 64), (1032, 7)])
def test_fp16_all_classes_of_bit_patterns(V, K):
    # logits taken from random 16-bit patterns: normal, subnormal, zero of both signs, infinities, NaNs
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = wk.CONFIGS["cfg2"].scaled(B=2, W=4, V=V, top_k=K, dtype=wk.F16, seed=77)
    inp = wk.make_step_inputs(wl)
    rng = np.random.default_rng(V)
    for arr in (inp.cond, inp.prev_cond):
        raw = rng.integers(0, 65536, size=arr.shape, dtype=np.uint32).astype(np.uint16)
        pick = rng.random(arr.shape) < 0.3
        arr[pick] = raw[pick]
        if V == 1032:
            arr[..., 5] = 0x7C00      # one +inf per row in the smallest case
    prev = oracle_prime(inp)
    check_parity(inp.cond, None, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len)
    wl2 = wk.CONFIGS["cfg2"].scaled(B=2, W=4, V=V, top_k=K, dtype=wk.F16, seed=78)
    inp2 = wk.make_step_inputs(wl2)
    prev2 = oracle_prime(inp2)
    check_parity(inp2.cond, inp2.uncond, prev2.tokens, prev2.probs, step_kwargs(inp2), inp2.win_len)
