#!/usr/bin/env python
"""Benchmark of the SJD++ verify-and-redraft step (sjd_step) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg4]

A step is one pass of the whole hot path (sampling head, accept test, prefix scan, residual draw, reuse /
redraft) over one batch of synthetic logits.  Default workload: B=16, W=64, V=65,536, bf16, CFG 3.0,
top-K 2000, reuse threshold 0.5.  With N > 1 (launched by torch.distributed.run, one rank per GPU) every
rank runs the same per-GPU workload on its own data (weak scaling, no data-path collective).

Prints ONE JSON line: verified window tokens/s with the inputs resident in HBM (`value`), the same
through the host-buffer entry point (`e2e`), the HBM roofline of the dominant kernel (`roofline`) and the
CPU oracle timed on a bounded sample (`cpu_baseline`).  `--impl reference` times the CPU oracle alone.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified window tokens/sec per sjd_step"
UNIT = "tokens/s"
NBUF = 3  # independent input sets rotated through the timed loop


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--init-mode", type=int, default=0, choices=[0, 1, 2, 3, 4],
                    help="--loop only: token initialisation (0 random, 1 repeat left, 2 repeat above, 3 sample left, 4 sample above)")
    ap.add_argument("--loop-source", default="markov", choices=["markov", "stripes"],
                    help="--loop only: synthetic logit source (first-order Markov chain, or an image of vertical stripes)")
    ap.add_argument("--no-refine", action="store_true",
                    help="--loop only: the no-refinement ablation (unaccepted slots are re-initialised, not carried over)")
    ap.add_argument("--graphs", action="store_true", help="--loop only: replay each iteration's kernels from a CUDA graph")
    ap.add_argument("--check", action="store_true",
                    help="--loop only: run the loop on host-generated logits in lock-step with the CPU oracle's loop and "
                         "report whether committed tokens, iterations and tokens per iteration are identical")
    ap.add_argument("--loop", action="store_true",
                    help="run the full decode loop of the 48x48 grid workload (cfg5) instead of the single-step benchmark")
    return ap.parse_args()


def workload_config(wl, n_gpus):
    return {"workload": f"{wl.name}: B={wl.B} W={wl.W} V={wl.V} {('fp32', 'bf16', 'fp16')[wl.dtype]} logits, "
                        f"CFG {wl.cfg_scale}, T {wl.temperature}, top-K {wl.top_k}, reuse tau {wl.reuse_tau}",
            "B_per_gpu": wl.B, "W": wl.W, "V": wl.V, "top_k": wl.top_k, "global_batch": wl.B * n_gpus,
            "parallelism": f"replicas over B x{n_gpus}, no collective",
            "l2": f"inputs larger than L2 ({NBUF} rotated input sets)"}


def algorithmic_bytes(wl) -> int:
    """Bytes the method itself must move per step: both logits tensors read, the sparse distributions and
    per-position results written, one previous-iteration sparse row per sequence read."""
    esize = 4 if wl.dtype == 0 else 2
    rows = wl.B * wl.W
    return rows * (2 * wl.V * esize + 8 * wl.kcap + 16) + wl.B * 8 * wl.kcap


# ------------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=5)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # the loop keeps the GPU busy; take the upper half of the samples as "under load"
        sm_sorted = sorted(sm)
        under = sm_sorted[len(sm_sorted) // 2:]
        return {"sm_mhz": statistics.median(under), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------------
# synthetic data on the device (same recipe as paper_2512_07503_b200.workloads, drawn with torch)
# ------------------------------------------------------------------------------------------------------
def device_inputs(wl, device, seed):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    dt = {0: torch.float32, 1: torch.bfloat16, 2: torch.float16}[wl.dtype]
    shape = (wl.B, wl.W, wl.V)
    cond = torch.randn(shape, generator=g, device=device, dtype=torch.float32) * wl.sigma
    if wl.row_spread > 0:
        cond *= torch.exp(wl.row_spread * (2 * torch.rand(wl.B, wl.W, 1, generator=g, device=device) - 1))
    if wl.peaks > 0:
        idx = torch.rand(wl.B, wl.W, wl.V, generator=g, device=device).topk(wl.peaks, dim=-1).indices
        cond.scatter_add_(2, idx, torch.full(idx.shape, wl.boost, device=device))
        del idx
    if wl.uncond_iid:
        uncond = torch.randn(shape, generator=g, device=device, dtype=torch.float32) * wl.sigma
    else:
        uncond = cond + torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    cond_s, uncond_s = cond.to(dt), uncond.to(dt)
    del cond, uncond
    prev_c = (cond_s.float() + torch.randn(shape, generator=g, device=device) * wl.prev_sigma).to(dt)
    prev_u = (uncond_s.float() + torch.randn(shape, generator=g, device=device) * wl.prev_sigma).to(dt)
    if wl.ragged_total > 0:
        start = torch.randint(0, wl.ragged_total, (wl.B,), generator=g, device=device, dtype=torch.int32)
        win_len = torch.minimum(torch.full_like(start, wl.W), wl.ragged_total - start).to(torch.int32)
    else:
        start = torch.zeros(wl.B, dtype=torch.int32, device=device)
        win_len = torch.full((wl.B,), wl.W, dtype=torch.int32, device=device)
    return cond_s, uncond_s, prev_c, prev_u, win_len, start


class DeviceSet:
    """One input set on the device with its outputs and parameters."""

    def __init__(self, sjd, wl, device, seed, seq_base=0):
        import torch
        self.wl = wl
        cond, uncond, prev_c, prev_u, self.win_len, self.pos_base = device_inputs(wl, device, seed)
        self.cond, self.uncond = cond, uncond
        B, W, kcap = wl.B, wl.W, wl.kcap
        mk = lambda: sjd.DeviceProbs.empty(B, W, kcap, device)
        self.q, self.out = mk(), mk()
        self.drafts = torch.zeros(B, W, dtype=torch.int32, device=device)
        self.acc = torch.zeros(B, dtype=torch.int32, device=device)
        self.toks = torch.zeros(B, W, dtype=torch.int32, device=device)
        self.flags = torch.zeros(B, W, dtype=torch.int32, device=device)
        self.status = torch.zeros(B, dtype=torch.int32, device=device)
        common = dict(top_k=wl.top_k, cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature),
                      reuse_tau=wl.reuse_tau, win_len=self.win_len, pos_base=self.pos_base, out_flags=self.flags,
                      status=self.status, seq_base=seq_base)
        p0 = sjd.make_params(cond, flags=sjd.binding.SJD_FLAG_DRAFT_ALL, iteration0=0, **common)
        self.ws = torch.empty(sjd.sjd_workspace_bytes(p0), dtype=torch.uint8, device=device)
        p0.workspace, p0.workspace_bytes = self.ws.data_ptr(), self.ws.numel()
        # previous iteration: draw every row from the perturbed logits (the library's own draft mode)
        sjd.sjd_step(prev_c, prev_u, None, None, p0, seed, self.acc, self.drafts, self.q)
        torch.cuda.synchronize(device)
        del prev_c, prev_u
        self.params = sjd.make_params(cond, flags=(sjd.binding.SJD_FLAG_REUSE if wl.reuse else 0), iteration0=1,
                                      **common)
        self.params.workspace, self.params.workspace_bytes = self.ws.data_ptr(), self.ws.numel()
        self.seed = seed

    def step(self, sjd):
        sjd.sjd_step(self.cond, self.uncond, self.drafts, self.q, self.params, self.seed, self.acc, self.toks, self.out)


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2512_07503_b200 as sjd
    from paper_2512_07503_b200 import sharding
    from paper_2512_07503_b200 import workloads as wk

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    wl = wk.workload(args.workload)
    K, Wm = args.steps, max(args.warmup, 3)

    # every rank owns wl.B sequences of a global batch of world * wl.B (weak scaling over sequences)
    seq_lo, _ = sharding.shard_range(world * wl.B, rank, world)
    sets = [DeviceSet(sjd, wl, device, wl.seed + 1000 * rank + j, seq_base=seq_lo) for j in range(NBUF)]
    tokens_per_step = int(sum(int(s.win_len.sum().item()) for s in sets) / NBUF)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    stream = torch.cuda.current_stream(device)
    for i in range(Wm):
        sets[i % NBUF].step(sjd)
    barrier()

    # ---- timed region: K steps, inputs resident in HBM ----
    clocks = None
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    # the K-step region is timed REPS times (barrier and synchronisation on both sides of each); the median
    # is reported, so that a short --steps still gives a steady number, with the spread beside it
    REPS = 5
    rep_ms = []
    launches = 0
    for r in range(REPS):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = sjd.sjd_launch_count()
        barrier()
        ev0.record(stream)
        for i in range(K):
            sets[i % NBUF].step(sjd)
        ev1.record(stream)
        barrier()
        launches = sjd.sjd_launch_count() - launches0
        rep_ms.append(sharding.max_over_ranks(ev0.elapsed_time(ev1), device))
    elapsed_ms = statistics.median(rep_ms)

    # ---- same loop with the row stage bracketed by events: duration of the dominant kernel ----
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in pairs:  # create the underlying events
        a.record(stream)
        b.record(stream)
    torch.cuda.synchronize(device)
    for i, (a, b) in enumerate(pairs):
        s = sets[i % NBUF]
        s.params.ev_rows_begin, s.params.ev_rows_end = a.cuda_event, b.cuda_event
        s.step(sjd)
    torch.cuda.synchronize(device)
    for s in sets:
        s.params.ev_rows_begin = s.params.ev_rows_end = None
    # The GPU's event clock ticks every 2.048 us here: a single launch of ~85 us reads 41, 42 or 43 ticks and the
    # median of many launches snaps to a tick.  The mean over the steps (lowest and highest tenth dropped) does
    # not: launches start at every phase of the tick.
    samples = sorted(a.elapsed_time(b) for a, b in pairs)
    trim = len(samples) // 10
    kept = samples[trim:len(samples) - trim] if len(samples) > 2 * trim else samples
    row_ms = sum(kept) / len(kept)
    if sampler:
        clocks = sampler.stop()

    ms_per_step = elapsed_ms / K
    value = world * tokens_per_step * K / (elapsed_ms * 1e-3)

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(sjd, wl, sets[0], device, min(K, 10), world, tokens_per_step, barrier)

    # ---- roofline of the dominant kernel ----
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"
    abytes = algorithmic_bytes(wl)
    achieved = abytes / (row_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "row stage (sampling head)", "achieved": round(achieved, 1), "peak": peak,
                "unit": "GB/s", "frac": round(achieved / peak, 4), "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                "traffic_source": (NCU_TRAFFIC_SOURCE if args.workload in NCU_TRAFFIC_BYTES else None),
                "algorithmic_bytes": abytes, "kernel_ms": round(row_ms, 5), "kernel_ms_is": "mean over the steps, lowest and highest tenth dropped (the event clock ticks every 2.048 us)",
                "peak_source": peak_src, "frac_of_nominal_8TBs": round(achieved / 8000.0, 4)}
    if clocks and clocks.get("sm_mhz"):
        # duration in SM cycles at the clock seen under load: comparable between runs whose clocks differ
        roofline["kernel_mcycles_at_sampled_clock"] = round(row_ms * 1e-3 * clocks["sm_mhz"], 2)

    cpu, parity = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu, parity = run_cpu_baseline(wl, sets[0])

    # status words of the last step of every input set: sequences with a row the single-pass kernel handed to
    # the any-shape path (exact, but many times slower), and the selected row kernel
    redone = sum(int(((d.status & 16) != 0).sum().item()) for d in sets)
    row_kernel = ["generic", "tiles", "ranges"][sjd.sjd_row_kernel(sets[0].params)]
    if rank == 0:
        line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
                "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak",
                "ms_per_step_is": f"median of {REPS} timed regions of {K} steps",
                "ms_per_step_min_max": [round(min(rep_ms) / K, 5), round(max(rep_ms) / K, 5)],
                "vs_baseline": None, "dtype": "f32", "logits_dtype": ("f32", "bf16", "f16")[wl.dtype], "data": "synthetic",
                "config": workload_config(wl, world),
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
                "cpu_baseline": cpu, "parity": parity,
                "hbm_gbs_whole_step": round(abytes / (ms_per_step * 1e-3) / 1e9, 1),
                "row_kernel": row_kernel, "sequences_with_a_redone_row": redone}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (read + write) of one launch of the dominant kernel from an ncu capture, per workload;
# the capture is summarised under profiles/.  None = not captured yet.
NCU_TRAFFIC_BYTES = {"cfg4": 281_000_000}
NCU_TRAFFIC_SOURCE = ("stored figure, not measured by this run: dram__bytes_read.sum + dram__bytes_write.sum of one launch, "
                      "from the ncu capture summarised in profiles/rows_ranges_cfg4.md")


def run_e2e(sjd, wl, dset, device, n, world, tokens_per_step, barrier):
    import torch
    import torch.distributed as dist
    B, W, kcap = wl.B, wl.W, wl.kcap
    ctx = sjd.HostContext(B, W, wl.V, wl.dtype, wl.top_k, device=device)
    pin = lambda t: t.detach().cpu().pin_memory()
    h_cond, h_unc, h_drafts = pin(dset.cond), pin(dset.uncond), pin(dset.drafts)
    h_q = sjd.HostProbs(pin(dset.q.tok_prob), pin(dset.q.ids), pin(dset.q.vals), pin(dset.q.cnt))
    h_out = sjd.HostProbs.empty(B, W, kcap)
    h_acc = torch.zeros(B, dtype=torch.int32).pin_memory()
    h_tok = torch.zeros(B, W, dtype=torch.int32).pin_memory()
    h_win, h_pos = pin(dset.win_len), pin(dset.pos_base)
    p = ctx.params(cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature), reuse_tau=wl.reuse_tau,
                   flags=(sjd.binding.SJD_FLAG_REUSE if wl.reuse else 0), iteration0=1, win_len=h_win, pos_base=h_pos)
    call = lambda: sjd.sjd_step_host(ctx, h_cond, h_unc, h_drafts, h_q, p, dset.seed, h_acc, h_tok, h_out)
    for _ in range(3):
        call()
    barrier()
    t0 = time.perf_counter()
    for _ in range(n):
        call()  # returns after the outputs are in host memory
    dt = time.perf_counter() - t0
    t = torch.tensor([dt], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dt = float(t.item())
    # the host results of the last call must equal the device-resident path's
    torch.cuda.synchronize(device)
    same = bool((h_acc == dset.acc.cpu()).all()) and bool((h_tok == dset.toks.cpu()).all())
    for host, dev_t in ((h_out.cnt, dset.out.cnt), (h_out.ids, dset.out.ids), (h_out.vals, dset.out.vals),
                        (h_out.tok_prob, dset.out.tok_prob)):
        live = (dset.win_len.cpu().view(B, 1) > torch.arange(W).view(1, W))  # rows inside their window
        a, b = host[live], dev_t.cpu()[live]
        same = same and bool((a == b).all())
    nb = lambda t: t.numel() * t.element_size()
    h2d = nb(h_cond) + nb(h_unc) + nb(h_drafts) + h_q.nbytes() + nb(h_win) + nb(h_pos)
    d2h = nb(h_acc) + nb(h_tok) + h_out.nbytes()
    ctx.close()
    return {"value": round(world * tokens_per_step * n / dt, 1), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "steps": n, "ms_per_step": round(dt / n * 1e3, 3),
            "api": "sjd_step_host (pinned host buffers, copies inside the timed region)",
            "matches_device_path": same}


def host_arrays(dset):
    """Host copies of one device input set in the layout the oracle reads."""
    import numpy as np
    import torch
    import oracle
    wl = dset.wl

    def logits(t):
        if wl.dtype != 0:
            return t.view(torch.int16).cpu().numpy().view(np.uint16)
        return t.cpu().numpy()

    q = oracle.Probs(dset.q.tok_prob.cpu().numpy(), dset.q.ids.cpu().numpy(), dset.q.vals.cpu().numpy(),
                     dset.q.cnt.cpu().numpy())
    return logits(dset.cond), logits(dset.uncond), dset.drafts.cpu().numpy(), q


def run_cpu_baseline(wl, dset):
    """The oracle, as it stands, on the host cores, on a bounded sample of the same workload."""
    import oracle
    cores = os.cpu_count() or 1
    cond, unc, drafts, q = host_arrays(dset)
    Bs = min(wl.B, 4)  # sample: the first Bs sequences of the step's batch
    sl = slice(0, Bs)
    qs = oracle.Probs(q.tok_prob[sl].copy(), q.ids[sl].copy(), q.vals[sl].copy(), q.cnt[sl].copy())
    kw = dict(dtype=wl.dtype, V=wl.V, cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature),
              top_k=wl.top_k, reuse_tau=wl.reuse_tau, flags=(oracle.FLAG_REUSE if wl.reuse else 0),
              win_len=dset.win_len.cpu().numpy()[sl], pos_base=dset.pos_base.cpu().numpy()[sl], iteration0=1,
              seed=dset.seed, n_threads=cores)
    c, u, d = cond[sl].copy(), unc[sl].copy(), drafts[sl].copy()
    ref = oracle.sjd_step(c, u, d, qs, diag=True, **kw)  # warm-up (page in, build) - and the parity check's reference
    # the device results of the last step on this input set, against the oracle, on the sampled sequences
    from oracle import compare
    host = lambda t: t.cpu().numpy()[sl]
    rep = compare.compare_step(host(dset.acc), host(dset.toks), host(dset.out.tok_prob), host(dset.flags),
                               host(dset.out.ids), host(dset.out.vals), host(dset.out.cnt), ref, d, kw["win_len"],
                               kw["flags"])
    parity = {"sample": f"first {Bs} of {wl.B} sequences of the last timed step, every output against the oracle",
              "positions": rep.positions, "mismatches": len(rep.errors), "max_rel_err_probabilities": float(rep.max_rel_err),
              "decisions_within_1e-6_of_their_boundary": {"accept": rep.flagged_accept, "reuse": rep.flagged_reuse,
                                                          "sample": rep.flagged_sample},
              "rule": "ids, counts, accept lengths and tokens bit-exact except at the counted near-boundary decisions; "
                      "probabilities within 1e-5 relative"}
    reps, t_total = 0, 0.0
    while reps < 3 or (t_total < 3.0 and reps < 50):
        t0 = time.perf_counter()
        oracle.sjd_step(c, u, d, qs, **kw)
        t_total += time.perf_counter() - t0
        reps += 1
    toks = int(kw["win_len"].sum())
    return {"value": round(toks * reps / t_total, 1), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {Bs} of {wl.B} sequences of the step ({toks} window tokens), {reps} repetitions, "
                      f"{cores} threads", "ms_per_sample_step": round(t_total / reps * 1e3, 2)}, parity


def run_reference(args):
    """Reference arm: the CPU oracle timed on the host cores on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2512_07503_b200 import workloads as wk
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl_full = wk.workload(args.workload)
    Bs = min(wl_full.B, 2)
    wl = wl_full.scaled(B=Bs)
    cores = os.cpu_count() or 1
    inp = wk.make_step_inputs(wl)
    base = dict(dtype=wl.dtype, V=wl.V, cfg_scale=wl.cfg_scale, inv_temperature=float(wl.inv_temperature),
                top_k=wl.top_k, reuse_tau=wl.reuse_tau, win_len=inp.win_len, pos_base=inp.pos_base, seed=wl.seed,
                n_threads=cores)
    prev = oracle.sjd_step(inp.prev_cond, inp.prev_uncond, None, None, flags=oracle.FLAG_DRAFT_ALL, iteration0=0, **base)
    step = lambda: oracle.sjd_step(inp.cond, inp.uncond, prev.tokens, prev.probs,
                                   flags=(oracle.FLAG_REUSE if wl.reuse else 0), iteration0=1, **base)
    K, Wm = args.steps, max(args.warmup, 1)
    # keep the whole run within a few minutes: time one step, then cap the repetitions
    t0 = time.perf_counter()
    step()
    one = time.perf_counter() - t0
    Wm = min(Wm, max(1, int(20.0 / max(one, 1e-6))))
    K_run = min(K, max(3, int(150.0 / max(one, 1e-6))))
    for _ in range(Wm):
        step()
    t0 = time.perf_counter()
    for _ in range(K_run):
        step()
    dt = time.perf_counter() - t0
    toks = int(inp.win_len.sum())
    value = toks * K_run / dt
    sample = (f"{Bs} of {wl_full.B} sequences per step ({toks} window tokens), {K_run} timed steps, {cores} threads; "
              "host arrays, no device involved")
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
            "steps": K_run, "warmup": Wm, "ms_per_step": round(dt / K_run * 1e3, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl_full, world),
            "cpu_baseline": {"value": round(value, 1), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_loop(args):
    """Decode loop workload: one 48x48 = 2,304-token grid, V=65,536, W=32, bf16, CFG 3.0, top-K 2000, logits
    from a synthetic first-order Markov source on the device (table row of the previous token + per-position
    noise).  Reports iterations, mean committed tokens per iteration and the time spent in the library."""
    import torch
    import paper_2512_07503_b200 as sjd
    from paper_2512_07503_b200.decode import DecodeLoop
    dev = torch.device("cuda", 0)
    V, N, W, K, states = 65536, 2304, 32, 2000, 1024
    g = torch.Generator(device=dev)
    g.manual_seed(7)
    table = torch.randn(states, V, generator=g, device=dev) * 3.0
    g.manual_seed(5)
    noise_c = torch.randn(N, V, generator=g, device=dev).to(torch.bfloat16)
    g.manual_seed(6)
    noise_u = torch.randn(N, V, generator=g, device=dev).to(torch.bfloat16)
    G = 48
    dl = DecodeLoop(batch=1, window=W, vocab=V, n_total=N, logits_dtype=torch.bfloat16, top_k=K, cfg_scale=3.0, seed=5,
                    init_mode=args.init_mode, grid_width=G, use_graphs=args.graphs, refine=not args.no_refine, device=dev)
    ar = torch.arange(W, device=dev)
    g.manual_seed(8)
    colours = torch.randperm(V, generator=g, device=dev)[:G]

    def stripes(d):
        # every column of the grid has its own colour: the prediction is peaked on it whatever the prefix is
        pos = (d.pos_base[0] + ar).clamp(max=N - 1)
        cond = 0.3 * noise_c[pos].float()
        cond[ar, colours[pos % G]] += 16.0
        cond_s = cond.to(torch.bfloat16)
        unc_s = (cond_s.float() + 0.3 * noise_u[pos].float()).to(torch.bfloat16)
        return cond_s.view(1, W, V), unc_s.view(1, W, V)

    def source(d):
        p0 = int(d.pos_base[0].item())
        L = int(d.win_len[0].item())
        toks = d.window_tokens[0].long()
        first = d.committed[0, p0 - 1].long().clamp(min=0) if p0 > 0 else torch.zeros((), dtype=torch.long, device=dev)
        prev = torch.cat([first.view(1), toks[:W - 1].clamp(min=0)])
        pos = (p0 + ar).clamp(max=N - 1)
        cond = table[prev % states] + noise_c[pos].float()
        cond_s = cond.to(torch.bfloat16)
        unc_s = (cond_s.float() + noise_u[pos].float()).to(torch.bfloat16)
        return cond_s.view(1, W, V), unc_s.view(1, W, V)

    ev = []
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    lib_ms = 0.0
    while not dl.done():
        cond, unc = stripes(dl) if args.loop_source == "stripes" else source(dl)
        if args.graphs:  # the model would write its logits straight into the loop's buffers
            dl.cond_buf.copy_(cond)
            dl.uncond_buf.copy_(unc)
            cond, unc = dl.cond_buf, dl.uncond_buf
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        dl.step(cond, unc)
        b.record()
        ev.append((a, b))
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    lib_ms = sum(a.elapsed_time(b) for a, b in ev)
    print(json.dumps({"workload": "cfg5: decode loop, 2304 tokens, V=65536, W=32, bf16, CFG 3.0, top-K 2000, "
                                  + ("Markov source" if args.loop_source == "markov" else "vertical-stripes source"),
                      "init_mode": args.init_mode, "grid_width": G, "cuda_graphs": bool(args.graphs), "refinement": not args.no_refine, "steps": dl.steps, "tokens": N, "mean_committed_per_step": round(N / dl.steps, 4),
                      "step_compression_S": round(N / dl.steps, 4), "library_ms_total": round(lib_ms, 3),
                      "library_us_per_step": round(1e3 * lib_ms / dl.steps, 2), "wall_s_including_logit_source": round(wall, 3),
                      "complete": bool((dl.committed >= 0).all().item())}), flush=True)


def run_loop_check(args):
    """The decode-loop workload at its full size against the CPU oracle's loop: both take their logits from the
    same host-side Markov source, so that committed tokens, iterations and tokens per iteration must be equal."""
    import numpy as np
    import torch
    import oracle
    from oracle import loop as oracle_loop
    from paper_2512_07503_b200 import workloads as wk
    from paper_2512_07503_b200.decode import DecodeLoop
    dev = torch.device("cuda", 0)
    V, N, W, K, states, seed = 65536, 2304, 32, 2000, 1024, 5
    src = wk.MarkovSource(V, N, wk.BF16, states=states, lazy=True)
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    ref_committed, ref_steps, ref_counts = oracle_loop.decode(
        lambda w: src.logits(w.drafts, w.win_len, w.pos_base, w.committed), B=1, W=W, V=V, n_total=N, dtype=wk.BF16,
        top_k=K, cfg_scale=3.0, flags=oracle.FLAG_REUSE, seed=seed, n_threads=cores, init_mode=args.init_mode,
        grid_width=48, refine=not args.no_refine)
    oracle_wall = time.perf_counter() - t0
    src = wk.MarkovSource(V, N, wk.BF16, states=states, lazy=True)
    dl = DecodeLoop(batch=1, window=W, vocab=V, n_total=N, logits_dtype=torch.bfloat16, top_k=K, cfg_scale=3.0, seed=seed,
                    init_mode=args.init_mode, grid_width=48, use_graphs=False, refine=not args.no_refine, device=dev)
    ev = []
    while not dl.done():
        c, u = src.logits(dl.window_tokens.cpu().numpy(), dl.win_len.cpu().numpy(), dl.pos_base.cpu().numpy(),
                          dl.committed.cpu().numpy())
        cond = torch.from_numpy(c.view(np.int16)).to(dev).view(torch.bfloat16)
        unc = torch.from_numpy(u.view(np.int16)).to(dev).view(torch.bfloat16)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        dl.step(cond, unc)
        b.record()
        ev.append((a, b))
    torch.cuda.synchronize()
    lib_ms = sum(a.elapsed_time(b) for a, b in ev)
    committed = dl.committed.cpu().numpy()
    same_tokens = bool(np.array_equal(committed, ref_committed))
    same_steps = dl.steps == ref_steps
    print(json.dumps({"workload": "cfg5: decode loop, 2304 tokens, V=65536, W=32, bf16, CFG 3.0, top-K 2000, host Markov source, "
                                  "in lock-step with the CPU oracle", "steps": dl.steps, "oracle_steps": int(ref_steps),
                      "tokens": N, "step_compression_S": round(N / dl.steps, 4), "library_ms_total": round(lib_ms, 3),
                      "library_us_per_step": round(1e3 * lib_ms / dl.steps, 2), "oracle_wall_s": round(oracle_wall, 2),
                      "oracle_cores": cores, "committed_tokens_identical": same_tokens, "iterations_identical": same_steps,
                      "status_bits": int(dl.status.max().item())}), flush=True)
    return 0 if (same_tokens and same_steps) else 1


if __name__ == "__main__":
    a = parse_args()
    if a.loop and a.check:
        sys.exit(run_loop_check(a))
    elif a.loop:
        run_loop(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
