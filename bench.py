#!/usr/bin/env python
"""Benchmark of the arithmetic-sampling decode step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c5|c4] [--impl reference]

A step is one pass of the decode hot path over one batch of synthetic input: a fresh
shifted lattice of codes and one decode step for every lane, in one launch (as_step_lattice
forms the codes in the step kernel; the two-call form is timed beside it).
The default workload is the 256-lane x 32000-token bf16 step (temperature 0.7, top_k 40).
Rank 0 prints ONE JSON line.  With N > 1 (torchrun) every
rank decodes its own batch (lanes never communicate), so scaling is weak and there is no
data-path collective: only the timing is reduced (max over ranks).

`--impl reference` times the CPU oracle (oracle/, test infrastructure) on host cores for
the same workload; it is a deliberately plain program and serves as a reported baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2210_15458_b200 import synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the step kernel on the default
# workload, from the ncu capture summarised in profiles/as_step_stream_c2.md
NCU_TRAFFIC_BYTES = {"c2": 16472576}
RING_BYTES = 3 * L2_BYTES          # rotating input buffers: each launch reads from HBM


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value_ms: float, world: int, device=None) -> float:
    """Slowest rank's time (the job is done when the last rank is)."""
    if world == 1:
        return value_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([value_ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def to_dev(arr, dtype):
    import torch
    if dtype == synth.BF16:
        return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).cuda()


# ----------------------------------------------------------------------------- step workloads
def step_workload(name: str, lanes=None):
    if name == "c2":
        return synth.c2()
    if name == "c3":
        return synth.c3() if lanes is None else synth.c3(lanes)
    if name == "c5":
        return synth.c5(1024 if lanes is None else lanes)
    raise ValueError(name)


def step_bytes(w) -> int:
    """Algorithmic bytes of one step: each row read once, code in, code out, token out."""
    return w.lanes * (w.V * w.elem_bytes + 8 + 8 + 4)


class StepBench:
    """Device-resident inputs for a step workload: a ring of distinct logits buffers larger
    than 3x L2, so that consecutive launches never find their rows in cache."""

    def __init__(self, w, rank: int, base_lanes=None):
        import torch
        from paper_2210_15458_b200 import binding as B
        self.B, self.w, self.torch = B, w, torch
        # host generation is the slow part: for many-lane workloads the first base_lanes rows are
        # generated and repeated with a per-copy rotation of the lanes
        gen = w.lanes if base_lanes is None else min(w.lanes, base_lanes)
        base = w.logits(gen, seed_offset=rank)
        first = to_dev(base, w.dtype)
        if gen < w.lanes:
            first = torch.cat([torch.roll(first, shifts=i, dims=0) for i in range(w.lanes // gen)], dim=0)
        total = first.numel() * first.element_size()
        nbuf = 1 if total > 4 * L2_BYTES else max(2, -(-RING_BYTES // total))
        self.ring = [first] + [torch.roll(first, shifts=i, dims=0) for i in range(1, nbuf)]
        self.host_base = base
        self.ring_bytes = nbuf * total
        self.shifts = np.random.default_rng(1234 + rank).random(4096)
        self.codes = B.as_lattice_codes(w.N, float(self.shifts[0]))      # for the calls that read stored codes
        self.tokens = torch.empty(w.lanes, dtype=torch.int32, device="cuda")
        self.codes_out = torch.empty(w.lanes, dtype=torch.float64, device="cuda")
        self.i = 0

    def step(self):
        """One pass of the hot path: the lattice codes of a fresh shift, formed in the step kernel
        (as_step_lattice: the same values as_lattice_codes would write), and the decode step."""
        B, w = self.B, self.w
        B.as_step_lattice(self.ring[self.i % len(self.ring)], w.N, float(self.shifts[self.i % 4096]), 0,
                          w.temp, w.top_k, w.top_p, tokens=self.tokens, codes_out=self.codes_out)
        self.i += 1

    def step_two_calls(self):
        """The same pass as two launches: as_lattice_codes, then as_step on the stored codes."""
        B, w = self.B, self.w
        B.as_lattice_codes(w.N, float(self.shifts[self.i % 4096]), out=self.codes)
        B.as_step(self.ring[self.i % len(self.ring)], self.codes[: w.lanes], w.temp, w.top_k, w.top_p,
                  tokens=self.tokens, codes_out=self.codes_out)
        self.i += 1

    def step_kernel_only(self):
        """as_step on stored codes (every step after the first in a decode loop)."""
        B, w = self.B, self.w
        B.as_step(self.ring[self.i % len(self.ring)], self.codes[: w.lanes], w.temp, w.top_k, w.top_p,
                  tokens=self.tokens, codes_out=self.codes_out)
        self.i += 1

    def timed(self, fn, n: int) -> float:
        """Device time of n calls of fn.  The calls are captured once into a CUDA graph (the step
        is launch-bound from Python: a ctypes call costs more than the kernel) and the graph
        is replayed; the inputs still rotate through the ring inside the graph."""
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(n):
                    fn()
        torch.cuda.current_stream().wait_stream(side)
        self.last_graph = g
        for _ in range(3):              # untimed: the first replay uploads the graph
            g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)


def e2e_step(w, steps: int, warmup: int):
    """Same metric through the host-buffer entry point: every step copies the logits and codes
    from pinned host memory, runs the step and copies tokens and codes back."""
    import torch
    from paper_2210_15458_b200 import binding as B
    base = w.logits()
    view = base.view(np.int16) if w.dtype == synth.BF16 else base
    nslots = 4
    h_logits = [torch.from_numpy(np.roll(view, i, axis=0).copy()).pin_memory() for i in range(nslots)]
    if w.dtype == synth.BF16:
        h_logits = [h.view(torch.bfloat16) for h in h_logits]
    codes = np.random.default_rng(99).random(w.lanes)
    h_codes = torch.from_numpy(codes).pin_memory()
    h_tok = torch.empty(w.lanes, dtype=torch.int32).pin_memory()
    h_out = torch.empty(w.lanes, dtype=torch.float64).pin_memory()
    h_st = torch.empty(w.lanes, dtype=torch.int32).pin_memory()
    work = torch.empty(B.as_step_host_work_bytes(w.dtype, w.lanes, w.V) + 256, dtype=torch.uint8, device="cuda")

    def one(i):
        B.as_step_host(h_logits[i % nslots], h_codes, w.temp, w.top_k, w.top_p, h_tok, h_out, h_st, work)
    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(steps):
        one(i)                       # synchronises: results are in host memory on return
    ms = (time.perf_counter() - t0) * 1e3
    assert int((h_st != 0).sum()) == 0
    h2d = w.lanes * w.V * w.elem_bytes + w.lanes * 8
    d2h = w.lanes * (4 + 8 + 4)
    return ms, h2d, d2h


def cpu_baseline_step(w, budget_s: float = 12.0):
    """The oracle as it stands, on host cores, on a bounded sample of the same workload."""
    from oracle import oracle
    cores = os.cpu_count() or 1
    lanes = min(w.lanes, 256)
    arr = w.logits(lanes)
    codes = oracle.lattice_codes(w.N, w.shift())[:lanes]
    threads = min(cores, lanes)
    oracle.step(arr[: min(lanes, threads)], w.dtype, codes[: min(lanes, threads)], w.temp, w.top_k, w.top_p,
                threads=threads)
    t0 = time.perf_counter()
    reps = 0
    while True:
        oracle.step(arr, w.dtype, codes, w.temp, w.top_k, w.top_p, threads=threads)
        reps += 1
        dt = time.perf_counter() - t0
        if dt > budget_s or reps >= 20:
            break
    return {"value": reps * lanes * w.V / dt, "unit": "logits/s", "cores": threads, "kind": "oracle",
            "sample": "%d x the first %d lanes of %s (V=%d), %.1f s" % (reps, lanes, w.name, w.V, dt)}


# ----------------------------------------------------------------------------- bigram workload (c4)
def bench_bigram(steps: int, warmup: int, S: int = 64, T: int = 128):
    """tokens/s of the full decode loop over the 32128 x 32128 bf16 bigram table, lattice
    codes versus iid codes (ordinary ancestral sampling through the same kernel)."""
    import torch
    from paper_2210_15458_b200 import binding as B
    w = synth.c4(S=S, T=T)
    table = to_dev(w.table(), w.dtype)
    starts = torch.from_numpy(w.starts()).cuda()
    out = {}
    seq = torch.empty((w.lanes, w.T), dtype=torch.int32, device="cuda")
    ln = torch.empty(w.lanes, dtype=torch.int32, device="cuda")
    prev = starts.repeat_interleave(w.N).contiguous()
    iid = torch.from_numpy(synth.iid_codes(w.lanes, 77)).cuda()

    def run_lattice():
        B.as_decode_bigram(table, starts, w.N, w.shift(), w.T, w.eos, w.temp, w.top_k, w.top_p, seq=seq, length=ln)

    def run_iid():
        B.as_decode_bigram_codes(table, prev, iid, w.T, w.eos, w.temp, w.top_k, w.top_p, seq=seq, length=ln)

    def dup_rates(s):
        s = s.cpu().numpy().reshape(w.S, w.N, w.T)
        res = {}
        for L in (1, 2, 4, 8, 128):
            r = [1.0 - len({tuple(x[:L]) for x in grp}) / w.N for grp in s]
            res[str(L)] = float(np.mean(r))
        return res

    for name, fn in (("lattice", run_lattice), ("iid", run_iid)):
        for _ in range(max(1, warmup)):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / steps
        tokens = int(ln.sum().item())
        out[name] = {"ms_per_decode": ms, "tokens": tokens, "tokens_per_s": tokens / ms * 1e3,
                     "mean_len": tokens / w.lanes,
                     "row_gbs_upper": tokens * w.V * w.elem_bytes / ms / 1e6,
                     "duplicate_prefix_rate": dup_rates(seq)}
    # the same loop with a cut (Sec. 5.1 "Top-k sampling": k = 2 and 10; a nucleus): one launch of
    # the streaming step kernel per step, rows gathered from the table
    cf = torch.empty(w.lanes, dtype=torch.float64, device="cuda")
    for name, k, p in (("top_k_2", 2, 1.0), ("top_k_10", 10, 1.0), ("top_p_0.9", 0, 0.9)):
        fn = lambda: B.as_decode_bigram(table, starts, w.N, w.shift(), w.T, w.eos, w.temp, k, p, seq=seq, length=ln,
                                        codes_final=cf)
        for _ in range(max(1, warmup)):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / steps
        tokens = int(ln.sum().item())
        out["lattice_" + name] = {"ms_per_decode": ms, "tokens": tokens, "tokens_per_s": tokens / ms * 1e3,
                                  "launches_per_decode": w.T + 2}
    # the other direction on the sequences just decoded: sequence -> interval, same tokens
    run_iid()
    fn = lambda: B.as_encode_bigram(table, prev, seq, ln, w.temp, w.top_k, w.top_p)
    for _ in range(max(1, warmup)):
        fn()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    tokens = int(ln.sum().item())
    out["encode"] = {"ms_per_encode": ms, "tokens": tokens, "tokens_per_s": tokens / ms * 1e3}
    # what is computed from the decoded groups: n-gram diversity (Sec. 5.1) and the sample-mean
    # estimator of an additive synthetic reward (Sec. 4.2 / 5.2), lattice codes against iid codes
    r = torch.from_numpy(synth.reward_table(w.V, 78)).cuda()

    def timed_call(fn, reps=20):
        fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    K = 16
    fits = w.N * w.T <= B.NGRAM_MAX_ITEMS          # one group's tokens and hash table in shared memory
    shifts = np.random.default_rng(79).random(K)
    stats = {}
    for name in ("lattice", "iid"):
        means, divs = [], []
        for k in range(K):
            if name == "lattice":
                B.as_decode_bigram(table, starts, w.N, float(shifts[k]), w.T, w.eos, w.temp, w.top_k, w.top_p,
                                   seq=seq, length=ln)
            else:
                codes = torch.from_numpy(synth.iid_codes(w.lanes, 1000 + k)).cuda()
                B.as_decode_bigram_codes(table, prev, codes, w.T, w.eos, w.temp, w.top_k, w.top_p, seq=seq, length=ln)
            means.append(B.as_reward_mean(seq, ln, w.N, r)[1])
            if fits:
                divs.append(B.as_ngram_diversity(seq, ln, w.N)[2])
        means = torch.stack(means)
        stats[name] = {"estimator_sd_over_%d_runs_mean_over_groups" % K: float(means.std(dim=0).mean().item()),
                       "ngram_diversity_mean": float(torch.stack(divs).mean().item()) if fits else None}
    stats["ms_ngram_diversity"] = timed_call(lambda: B.as_ngram_diversity(seq, ln, w.N)) if fits else None
    stats["ms_reward_mean"] = timed_call(lambda: B.as_reward_mean(seq, ln, w.N, r))
    out["groups"] = stats
    out["workload"] = "c4: bf16 bigram table 32128x32128, %d starts x 32 codes, T<=%d, temp 0.8, EOS 1" % (S, T)
    return out


# ----------------------------------------------------------------------------- arms
def run_ours(args):
    import torch
    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2210_15458_b200 import binding as B
    B.lib()
    w = step_workload(args.workload, args.lanes)
    sb = StepBench(w, rank)
    for _ in range(args.warmup):
        sb.step()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier(world)
    ms = sb.timed(sb.step, args.steps)
    barrier(world)
    if rank == 0:
        # the timed replay lasts a few tens of ms; keep the same graph running for ~0.5 s so that
        # nvidia-smi (100 ms period) sees the clocks under this load
        t_end = time.perf_counter() + 0.5
        while time.perf_counter() < t_end:
            sb.last_graph.replay()
        torch.cuda.synchronize()
    ms = max_over_ranks(ms, world, torch.device("cuda", local_rank))
    # the step is a single launch of the step kernel: its duration is the step's; the same kernel
    # on stored codes (as_step) and the two-launch form are timed beside it
    for _ in range(3):
        sb.step_kernel_only()
    kern_launches = max(args.steps, 200)
    kms = sb.timed(sb.step, kern_launches) / kern_launches
    kms_stored = sb.timed(sb.step_kernel_only, kern_launches) / kern_launches
    ms2 = sb.timed(sb.step_two_calls, kern_launches) / kern_launches
    clocks = sampler.stop() if rank == 0 else None
    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return
    peak, peak_kind = measured_peaks()
    logits_per_step = w.lanes * w.V * world
    value = logits_per_step * args.steps / (ms / 1e3)
    lattice_step_bytes = step_bytes(w) - 8 * w.lanes          # the codes are not read from memory
    achieved = lattice_step_bytes / (kms / 1e3) / 1e9
    line = {
        "metric": "logits decoded/s", "value": value, "unit": "logits/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s: %d lanes x V=%d %s logits, temp %g, top_k %d, top_p %g, fp64 lattice codes"
                               % (w.name, w.lanes, w.V, "bf16" if w.dtype else "f32", w.temp, w.top_k, w.top_p),
                   "lanes_per_gpu": w.lanes, "V": w.V, "l2": "inputs rotate through %d buffers (%.0f MB > 3x L2)"
                                                             % (len(sb.ring), sb.ring_bytes / 1e6),
                   "step": "one as_step_lattice launch: lattice codes of a fresh shift formed in the step kernel",
                   "timing": "K steps captured in one CUDA graph, replayed once between events",
                   "parallelism": "lanes sharded, no collective"},
        "lane_steps_per_s": w.lanes * world * args.steps / (ms / 1e3),
        "gpu_launches": args.steps,
        "ms_per_step_two_calls": ms2,          # as_lattice_codes + as_step on the stored codes
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "step_stream_kernel (as_step_lattice)", "achieved": achieved,
                     "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": peak_kind, "frac_of_8TBs_nominal": achieved / 8000.0,
                     "us_per_launch": kms * 1e3, "bytes_per_launch": lattice_step_bytes,
                     "us_per_launch_stored_codes": kms_stored * 1e3,
                     "traffic": NCU_TRAFFIC_BYTES.get(w.name)},
    }
    if world == 1:
        e_ms, h2d, d2h = e2e_step(w, args.steps, args.warmup)
        line["e2e"] = {"value": w.lanes * w.V * args.steps / (e_ms / 1e3), "unit": "logits/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e_ms / args.steps}
        line["cpu_baseline"] = cpu_baseline_step(w)
        if not args.no_extras:
            extras = {}
            for name, lanes in (("c3", None), ("c5", 1024), ("c5", 4096), ("c5", 8192)):
                if name == w.name:
                    continue
                del sb
                torch.cuda.empty_cache()
                ww = step_workload(name, lanes)
                sb = StepBench(ww, 0, base_lanes=1024)
                for _ in range(3):
                    sb.step_kernel_only()
                n = 2 * len(sb.ring) if len(sb.ring) > 1 else 6
                k = sb.timed(sb.step_kernel_only, n) / n
                gbs = step_bytes(ww) / (k / 1e3) / 1e9
                key = name if lanes in (None, 1024) else "%s_%d" % (name, lanes)
                extras[key] = {"lanes": ww.lanes, "V": ww.V, "us_per_launch": k * 1e3, "GBs": gbs,
                               "frac_of_peak": gbs / peak, "logits_per_s": ww.lanes * ww.V / (k / 1e3)}
            del sb
            torch.cuda.empty_cache()
            extras["bigram_decode"] = bench_bigram(2, 1)
            line["other_workloads"] = extras
    else:
        line["e2e"] = None
        torch.distributed.destroy_process_group()
    print(json.dumps(line))


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from oracle import oracle
    w = step_workload(args.workload, args.lanes)
    cores = os.cpu_count() or 1
    lanes = min(w.lanes, 256)
    arr = w.logits(lanes)
    threads = min(cores, lanes)
    shifts = np.random.default_rng(1234).random(4096)

    def one(i):
        codes = oracle.lattice_codes(w.N, float(shifts[i % 4096]))[:lanes]
        oracle.step(arr, w.dtype, codes, w.temp, w.top_k, w.top_p, threads=threads)
    for i in range(args.warmup):
        one(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        one(i)
    dt = time.perf_counter() - t0
    value = lanes * w.V * args.steps / dt
    sample = "each step = the first %d lanes of %s on %d host threads" % (lanes, w.name, threads)
    print(json.dumps({
        "impl": "reference", "metric": "logits decoded/s", "value": value, "unit": "logits/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s: %d lanes x V=%d %s logits, temp %g, top_k %d, top_p %g (CPU oracle, %s)"
                               % (w.name, lanes, w.V, "bf16" if w.dtype else "f32", w.temp, w.top_k, w.top_p, sample)},
        "cpu_baseline": {"value": value, "unit": "logits/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "logits/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c5", "c4"],
                    help="c4 prints the bigram decode / encode loop's own line (a side measurement)")
    ap.add_argument("--lanes", type=int, default=None,
                    help="lanes for c3 / c5 / c4 (default: the configured size; c4: a multiple of 32)")
    ap.add_argument("--T", type=int, default=128, help="c4 only: maximum steps per lane (512-1024: summarisation-sized outputs)")
    ap.add_argument("--no-extras", action="store_true", help="skip the other workloads' short measurements")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)
    if args.workload == "c4":
        if args.impl == "reference" or dist_env()[2] > 1:
            raise SystemExit("--workload c4 is a single-GPU side measurement of the CUDA path")
        print(json.dumps(bench_bigram(min(args.steps, 20), min(args.warmup, 3), S=(args.lanes or 2048) // 32,
                                      T=args.T)))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
