"""GPU parity on seeded random shapes and settings: vocabulary, top-K, window, batch, storage type, guidance
scale, temperature, reuse threshold, ragged windows.  Every case goes through whichever row kernel the
library selects for it and is compared with the oracle element by element."""
import numpy as np
import pytest

import oracle
from paper_2512_07503_b200 import workloads as wk

pytestmark = pytest.mark.gpu


def _case(seed):
    rng = np.random.default_rng(1000 + seed)
    kind = seed % 3
    if kind == 0:      # vocabularies the range kernel takes (multiples of 256 ranges x 64-byte slices)
        V = int(rng.choice([8192, 12288, 16384, 24576, 32768, 49152, 65536]))
    elif kind == 1:    # multiples of 2,048 and of 8 only
        V = int(rng.choice([2048, 4096, 6144, 10240, 18432])) if rng.random() < 0.5 else 8 * int(rng.integers(1, 1500))
    else:
        V = 256 * int(rng.integers(8, 200))
    dtype = [wk.BF16, wk.F32, wk.F16][int(rng.choice(3, p=[0.45, 0.3, 0.25]))]
    K = int(min(V, rng.choice([1, 2, 7, 50, 64, 300, 777, 1000, 2000, 2048, 2500])))
    W = int(rng.integers(1, 20))
    B = int(rng.integers(1, 4))
    base = wk.CONFIGS["cfg2"]
    return base.scaled(name=f"rand{seed}", B=B, W=W, V=V, dtype=dtype, top_k=K, seed=5000 + seed,
                       sigma=float(rng.choice([0.5, 2.0, 3.0, 6.0])), peaks=int(rng.integers(0, 30)),
                       boost=float(rng.choice([2.0, 8.0, 15.0])), cfg_scale=float(rng.choice([1.0, 1.5, 3.0, 7.5])),
                       temperature=float(rng.choice([1.0, 0.7, 1.3])), reuse=bool(rng.random() < 0.7),
                       reuse_tau=float(rng.choice([0.5, 0.1, 0.9])), ragged_total=int(rng.choice([0, 0, 40])))


@pytest.mark.parametrize("seed", range(36))
def test_random_case_matches_the_oracle(seed):
    from gpu_harness import check_parity, oracle_prime, step_kwargs
    wl = _case(seed)
    inp = wk.make_step_inputs(wl)
    prev = oracle_prime(inp)
    rep, got, ref = check_parity(inp.cond, inp.uncond, prev.tokens, prev.probs, step_kwargs(inp), inp.win_len)
    print(wl.name, wl.V, wl.top_k, wl.W, wl.B, ("f32", "bf16", "f16")[wl.dtype], rep.summary())
