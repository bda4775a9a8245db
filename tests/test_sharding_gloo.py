"""Multi-rank host logic on CPU (gloo, world size 2): the batch shards over ranks with no exchange of
data, a sharded run reproduces the unsharded one bit for bit (the generator's sequence word is the global
sequence index), and the timing reduction takes the max over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2512_07503_b200 import sharding
from paper_2512_07503_b200 import workloads as wk


def test_shard_range_partitions_the_batch():
    for B in (0, 1, 5, 16, 17):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_range(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(spans[r][1] == spans[r + 1][0] for r in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_range(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _step(inp, prev_tokens, prev_probs, lo, hi, seq_base):
    wl = inp.wl
    sl = slice(lo, hi)
    q = oracle.Probs(prev_probs.tok_prob[sl].copy(), prev_probs.ids[sl].copy(), prev_probs.vals[sl].copy(),
                     prev_probs.cnt[sl].copy())
    return oracle.sjd_step(inp.cond[sl].copy(), inp.uncond[sl].copy(), prev_tokens[sl].copy(), q, dtype=wl.dtype, V=wl.V,
                           cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature), top_k=wl.top_k,
                           reuse_tau=wl.reuse_tau, flags=oracle.FLAG_REUSE, win_len=inp.win_len[sl],
                           pos_base=inp.pos_base[sl], iteration0=1, seed=wl.seed, seq_base=seq_base)


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = wk.CONFIGS["cfg1"].scaled(B=5, W=6, V=512, top_k=32)
        inp = wk.make_step_inputs(wl)
        prev = oracle.sjd_step(inp.prev_cond, inp.prev_uncond, None, None, dtype=wl.dtype, V=wl.V, cfg_scale=wl.cfg_scale,
                               inv_temperature=float(wl.inv_temperature), top_k=wl.top_k, flags=oracle.FLAG_DRAFT_ALL,
                               win_len=inp.win_len, pos_base=inp.pos_base, iteration0=0, seed=wl.seed)
        lo, hi = sharding.shard_range(wl.B, rank, world)
        mine = _step(inp, prev.tokens, prev.probs, lo, hi, seq_base=lo)
        parts = [None] * world
        dist.all_gather_object(parts, (lo, hi, mine.accept_len, mine.tokens, mine.probs.vals, mine.probs.ids))
        slowest = sharding.max_over_ranks(10.0 + rank)
        total = sharding.sum_over_ranks(float(hi - lo))
        dist.barrier()
        if rank == 0:
            whole = _step(inp, prev.tokens, prev.probs, 0, wl.B, seq_base=0)
            parts.sort(key=lambda p: p[0])
            ok = (np.array_equal(np.concatenate([p[2] for p in parts]), whole.accept_len)
                  and np.array_equal(np.concatenate([p[3] for p in parts]), whole.tokens)
                  and np.array_equal(np.concatenate([p[4] for p in parts]), whole.probs.vals)
                  and np.array_equal(np.concatenate([p[5] for p in parts]), whole.probs.ids))
            # without the global sequence index the second shard would reuse the first shard's random numbers
            wrong = _step(inp, prev.tokens, prev.probs, parts[1][0], parts[1][1], seq_base=0)
            differs = not np.array_equal(wrong.tokens, parts[1][3])
            with open(os.path.join(out_dir, "result.txt"), "w") as f:
                f.write(f"{int(ok)} {int(differs)} {slowest} {total}")
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_step(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    ok, differs, slowest, total = open(tmp_path / "result.txt").read().split()
    assert ok == "1", "sharded and unsharded results differ"
    assert differs == "1", "the sequence word of the generator does not reach the draws"
    assert float(slowest) == 11.0 and float(total) == 5.0
