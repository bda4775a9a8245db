"""The time-out path of the single-pass row kernel: every wait on the chip is bounded, and a wait that runs out
becomes a status word, not a hang.  A test build of the library (short limit; one copy of the producer is
never issued, so the wait for it cannot end) runs in a process of its own; the call must return, report
SJD_STATUS_INTERNAL_TIMEOUT for the sequence, leave the rows empty, and leave the context usable."""
import os
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = textwrap.dedent("""
    import sys, time
    sys.path.insert(0, %r); sys.path.insert(0, %r)
    import numpy as np, torch
    import paper_2512_07503_b200 as sjd
    from paper_2512_07503_b200 import workloads as wk
    from gpu_harness import gpu_step, step_kwargs
    import oracle
    wl = wk.CONFIGS["cfg2"].scaled(W=4)
    inp = wk.make_step_inputs(wl)
    kw = step_kwargs(inp, flags=oracle.FLAG_DRAFT_ALL, iteration0=0)
    assert sjd.sjd_row_kernel(sjd.make_params(torch.empty(1, 4, wl.V, dtype=torch.bfloat16, device="cuda:0"),
                                              top_k=wl.top_k)) == 2, "the shape must take the single-pass range kernel"
    t0 = time.time()
    for _ in range(2):   # twice: the context must still be usable after the first time-out
        got = gpu_step(inp.cond, inp.uncond, None, None, **kw)
        assert got.status[0] & 8, got.status
        assert np.all(got.cnt[0, :4] == 0), got.cnt
    x = torch.arange(10, device="cuda:0").sum().item()
    assert x == 45
    print("TIMEOUT_PATH_OK", round(time.time() - t0, 2))
""")


def test_a_wait_that_cannot_end_becomes_a_status_word(tmp_path):
    from paper_2512_07503_b200 import build
    lib = build.build_variant(str(tmp_path / "libsjd_timeout_test.so"),
                              ["SJD_TEST_SPIN_CYCLES=2000000", "SJD_TEST_DROP_COPY=3"])
    env = dict(os.environ, SJD_LIBRARY=lib)
    out = subprocess.run([sys.executable, "-c", SCRIPT % (ROOT, os.path.join(ROOT, "tests"))], env=env,
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "TIMEOUT_PATH_OK" in out.stdout
