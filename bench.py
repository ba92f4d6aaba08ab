#!/usr/bin/env python
"""Benchmark of the arithmetic-sampling decode step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5|c2|c3|c4] [--lanes L]
                  [--impl reference] [--no-extras]

A step is one pass of the decode hot path over one batch of synthetic input: a fresh shifted
lattice of codes and one decode step for every lane, in one launch (as_step_lattice forms the
codes in the step kernel).  The default workload is the largest single-GPU step configuration:
8192 lanes x 256000 bf16 logits, temperature 0.8, top_k 64 and top_p 0.95 together.  Rank 0
prints ONE JSON line; `rooflines` in it holds one block per configuration (bytes per launch,
median and minimum time per launch over >= 20 graph replays, fraction of the measured copy
bandwidth and of the nominal 8 TB/s).  With N > 1 every rank decodes its own batch (lanes never
communicate), so scaling is weak and there is no data-path collective: only the timing is
reduced (max over ranks).  `--gpus N` without a torchrun environment starts the N ranks itself.

`--impl reference` times the CPU oracle (oracle/, test infrastructure) on host cores for the
same workload; it is a deliberately plain program and serves as a reported baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import socket
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
RING_BYTES = 3 * L2_BYTES          # small inputs rotate through this much memory
REPLAYS = 20                       # graph replays behind every median / minimum
NOMINAL_GBS = 8000.0


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def captured_traffic(kernel_file: str, key: str):
    """DRAM bytes per lane of a kernel from its ncu summary under profiles/ (a line
    `traffic_bytes_per_lane[<key>]: <number>` written with the capture), or None."""
    path = os.path.join(ROOT, "profiles", kernel_file)
    try:
        with open(path) as f:
            m = re.search(r"traffic_bytes_per_lane\[%s\]:\s*([0-9.eE+]+)" % re.escape(key), f.read())
        return float(m.group(1)) if m else None
    except OSError:
        return None


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


def check_world(gpus: int, world: int) -> None:
    """--gpus must agree with the ranks that were actually started."""
    if gpus != world:
        raise SystemExit("bench.py: --gpus %d but WORLD_SIZE is %d: start it as `python bench.py --gpus %d` "
                         "(it spawns the ranks) or under torchrun with --nproc-per-node %d" % (gpus, world, gpus, gpus))


def spawn_ranks(gpus: int) -> int:
    """`python bench.py --gpus N` outside torchrun: start the N ranks (one per GPU) on this node."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def to_dev(arr, dtype):
    import torch
    if dtype == synth.BF16:
        return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).cuda()


def device_rows(rows: int, V: int, sigma: float, dtype: int, seed: int, bias):
    """rows x V logits ~ N(0, sigma^2) + bias, drawn on the device (torch's seeded generator) in the
    workload's distribution and rounded to its storage type: the host recipe of synth.py yields the
    same distribution but takes minutes for gigabytes of rows."""
    import torch
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    tdt = torch.bfloat16 if dtype == synth.BF16 else torch.float32
    out = torch.empty((rows, V), dtype=tdt, device="cuda")
    b = torch.from_numpy(bias).cuda() if bias is not None else None
    step = max(1, (64 << 20) // V)
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        x = torch.randn((r1 - r0, V), generator=g, device="cuda", dtype=torch.float32) * sigma
        if b is not None:
            x += b[None, :]
        out[r0:r1] = x.to(tdt)
    return out


def median_min(xs):
    return float(np.median(xs)), float(np.min(xs))


# ----------------------------------------------------------------------------- step workloads
def step_workload(name: str, lanes=None):
    if name == "c2":
        return synth.c2()
    if name == "c3":
        return synth.c3() if lanes is None else synth.c3(lanes)
    if name == "c5":
        return synth.c5(8192 if lanes is None else lanes)
    raise ValueError(name)


def step_key(w) -> str:
    return "c5_%d" % w.lanes if w.name == "c5" else w.name


def step_bytes(w, stored_codes: bool = True) -> int:
    """Algorithmic bytes of one step: each row read once, code in (unless formed in the kernel),
    code out, token out."""
    return w.lanes * (w.V * w.elem_bytes + (8 if stored_codes else 0) + 8 + 4)


def workload_text(w, lanes=None) -> str:
    return "%s: %d lanes x V=%d %s logits, temp %g, top_k %d, top_p %g, fp64 lattice codes" % (
        w.name, w.lanes if lanes is None else lanes, w.V, "bf16" if w.dtype else "f32", w.temp, w.top_k, w.top_p)


class StepBench:
    """Device-resident inputs of a step workload.  Inputs smaller than 4x L2 rotate through a ring
    of distinct buffers larger than 3x L2, so that no launch finds its rows in cache; larger ones
    are their own flush."""

    def __init__(self, w, rank: int):
        import torch
        from paper_2210_15458_b200 import binding as B
        self.B, self.w, self.torch = B, w, torch
        bias = synth.zipf_bias(w.V, w.seed_perm)
        total = w.lanes * w.V * w.elem_bytes
        nbuf = 1 if total > 4 * L2_BYTES else max(2, -(-RING_BYTES // total))
        self.ring = [device_rows(w.lanes, w.V, w.sigma, w.dtype, w.seed_logits + 1000 * rank + 7 * i, bias)
                     for i in range(nbuf)]
        self.ring_bytes = nbuf * total
        self.shifts = np.random.default_rng(1234 + rank).random(4096)
        self.codes = B.as_lattice_codes(w.N, float(self.shifts[0]))[: w.lanes].contiguous()
        self.iid = torch.from_numpy(synth.iid_codes(w.lanes, 4321 + rank)).cuda()
        self.tokens = torch.empty(w.lanes, dtype=torch.int32, device="cuda")
        self.codes_out = torch.empty(w.lanes, dtype=torch.float64, device="cuda")
        self.i = 0

    def l2_note(self) -> str:
        if len(self.ring) == 1:
            return "one input of %.0f MB (> L2) read end to end by every launch" % (self.ring_bytes / 1e6)
        return "inputs rotate through %d buffers (%.0f MB > 3x L2)" % (len(self.ring), self.ring_bytes / 1e6)

    def _next(self):
        buf = self.ring[self.i % len(self.ring)]
        self.i += 1
        return buf

    def step(self):
        """One pass of the hot path: the lattice codes of a fresh shift, formed in the step kernel
        (as_step_lattice: the same values as_lattice_codes would write), and the decode step."""
        B, w = self.B, self.w
        B.as_step_lattice(self._next(), w.N, float(self.shifts[self.i % 4096]), 0, w.temp, w.top_k, w.top_p,
                          tokens=self.tokens, codes_out=self.codes_out)

    def step_two_calls(self):
        """The same pass as two launches: as_lattice_codes, then as_step on the stored codes."""
        B, w = self.B, self.w
        B.as_lattice_codes(w.N, float(self.shifts[self.i % 4096]), out=self.codes)
        B.as_step(self._next(), self.codes, w.temp, w.top_k, w.top_p, tokens=self.tokens, codes_out=self.codes_out)

    def step_stored(self):
        """as_step on stored lattice codes (every step after the first in a decode loop)."""
        B, w = self.B, self.w
        B.as_step(self._next(), self.codes, w.temp, w.top_k, w.top_p, tokens=self.tokens, codes_out=self.codes_out)

    def step_iid(self):
        """The same kernel on iid uniform codes: ordinary ancestral sampling by inverse CDF."""
        B, w = self.B, self.w
        B.as_step(self._next(), self.iid, w.temp, w.top_k, w.top_p, tokens=self.tokens, codes_out=self.codes_out)

    def graph(self, fn, n: int):
        """n calls of fn captured into one CUDA graph (a ctypes call from Python costs more than
        a small kernel, so a Python launch loop would time the interpreter); the inputs still
        rotate through the ring inside the graph."""
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(n):
                    fn()
        torch.cuda.current_stream().wait_stream(side)
        return g

    def replay_ms(self, g) -> float:
        torch = self.torch
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    def per_launch_us(self, fn, replays: int = REPLAYS):
        """Median and minimum time of one launch of fn over `replays` replays of a graph that holds
        enough launches to last about 2 ms (at least 2, and a whole turn of the input ring)."""
        for _ in range(3):
            fn()
        self.torch.cuda.synchronize()
        probe = self.graph(fn, 2)
        self.replay_ms(probe)
        one = max(self.replay_ms(probe) / 2, 1e-3)
        n = int(min(400, max(2, len(self.ring), round(2.0 / one))))
        g = self.graph(fn, n)
        self.replay_ms(g)
        xs = [self.replay_ms(g) / n * 1e3 for _ in range(replays)]
        return median_min(xs) + (n,)


def roofline_block(w, med_us, min_us, launches, peak, bytes_per_launch, traffic_per_lane=None, kernel=None):
    gbs = bytes_per_launch / (med_us * 1e-6) / 1e9
    blk = {"bound": "hbm", "workload": workload_text(w), "bytes_per_launch": bytes_per_launch,
           "us_per_launch_median": med_us, "us_per_launch_min": min_us,
           "replays": REPLAYS, "launches_per_replay": launches,
           "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
           "frac_of_8TBs_nominal": gbs / NOMINAL_GBS, "frac_at_min": bytes_per_launch / (min_us * 1e-6) / 1e9 / peak,
           "logits_per_s": w.lanes * w.V / (med_us * 1e-6), "lane_steps_per_s": w.lanes / (med_us * 1e-6),
           "traffic": None if traffic_per_lane is None else traffic_per_lane * w.lanes}
    if kernel:
        blk["kernel"] = kernel
    return blk


def stream_kernel_name(w) -> str:
    resident = w.V * w.elem_bytes <= 6 * 16384
    return "step_stream_kernel (%s rows)" % ("ring-resident" if resident else "streamed")


def e2e_step(w, steps: int, warmup: int):
    """Same metric through the host-buffer entry point: every step copies the logits and codes
    from pinned host memory, runs the step and copies tokens and codes back."""
    import torch
    from paper_2210_15458_b200 import binding as B
    bias = synth.zipf_bias(w.V, w.seed_perm)
    tdt = torch.bfloat16 if w.dtype == synth.BF16 else torch.float32
    total = w.lanes * w.V * w.elem_bytes
    nslots = 1 if total > (1 << 30) else 4
    h_logits = []
    for i in range(nslots):
        h = torch.empty((w.lanes, w.V), dtype=tdt, pin_memory=True)
        h.copy_(device_rows(w.lanes, w.V, w.sigma, w.dtype, 900 + i, bias))
        h_logits.append(h)
    torch.cuda.empty_cache()
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


def oracle_rate(w, lanes: int, budget_s: float):
    """logits/s of the oracle as it stands on `lanes` rows of the workload (host recipe), all host cores."""
    from oracle import oracle
    cores = os.cpu_count() or 1
    arr = w.logits(lanes)
    codes = oracle.lattice_codes(w.N, w.shift())[:lanes]
    threads = min(cores, lanes)
    oracle.step(arr[:threads], w.dtype, codes[:threads], w.temp, w.top_k, w.top_p, threads=threads)
    t0 = time.perf_counter()
    reps = 0
    while True:
        oracle.step(arr, w.dtype, codes, w.temp, w.top_k, w.top_p, threads=threads)
        reps += 1
        dt = time.perf_counter() - t0
        if dt > budget_s or reps >= 20:
            break
    return reps * lanes * w.V / dt, threads, reps, dt


def cpu_baseline_step(w, budget_s: float = 12.0):
    """The oracle as it stands, on host cores, on a bounded sample of the same workload."""
    lanes = min(w.lanes, 64 if w.V > 100000 else 256)
    rate, threads, reps, dt = oracle_rate(w, lanes, budget_s)
    return {"value": rate, "unit": "logits/s", "cores": threads, "kind": "oracle",
            "sample": "%d x the first %d lanes of %s (V=%d), %.1f s" % (reps, lanes, w.name, w.V, dt)}


# ----------------------------------------------------------------------------- bigram workload (c4)
def bench_bigram(reps: int, warmup: int, S: int = 64, T: int = 128, eos_variant: bool = True):
    """tokens/s of the full decode loop over the 32128 x 32128 bf16 bigram table, lattice
    codes versus iid codes (ordinary ancestral sampling through the same kernel)."""
    import torch
    from paper_2210_15458_b200 import binding as B
    w = synth.c4(S=S, T=T)
    table = device_rows(w.V, w.V, w.sigma, w.dtype, w.seed_table, w.column_bias())
    starts = torch.from_numpy(w.starts()).cuda()
    out = {}
    seq = torch.empty((w.lanes, w.T), dtype=torch.int32, device="cuda")
    ln = torch.empty(w.lanes, dtype=torch.int32, device="cuda")
    prev = starts.repeat_interleave(w.N).contiguous()
    iid = torch.from_numpy(synth.iid_codes(w.lanes, 77)).cuda()
    peak, _ = measured_peaks()

    def timed(fn):
        for _ in range(max(1, warmup)):
            fn()
        xs = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            xs.append(a.elapsed_time(b))
        return median_min(xs)

    def dup_rates(s):
        s = s.cpu().numpy().reshape(w.S, w.N, w.T)
        res = {}
        for L in (1, 2, 4, 8, 16, 32, w.T):
            r = [1.0 - len({tuple(x[:L]) for x in grp}) / w.N for grp in s]
            res[str(L)] = float(np.mean(r))
        return res

    def decode_entry(fn, tbl_note=None):
        med, mn = timed(fn)
        tokens = int(ln.sum().item())
        gbs = tokens * w.V * w.elem_bytes / med / 1e6
        e = {"ms_per_decode_median": med, "ms_per_decode_min": mn, "repetitions": reps, "tokens": tokens,
             "tokens_per_s": tokens / med * 1e3, "mean_len": tokens / w.lanes,
             "row_gbs": gbs, "row_frac_of_peak": gbs / peak,
             "duplicate_prefix_rate": dup_rates(seq)}
        if tbl_note:
            e["table"] = tbl_note
        return e

    def run_lattice(tbl=table):
        B.as_decode_bigram(tbl, starts, w.N, w.shift(), w.T, w.eos, w.temp, w.top_k, w.top_p, seq=seq, length=ln)

    def run_iid(tbl=table):
        B.as_decode_bigram_codes(tbl, prev, iid, w.T, w.eos, w.temp, w.top_k, w.top_p, seq=seq, length=ln)

    out["lattice"] = decode_entry(run_lattice)
    out["iid"] = decode_entry(run_iid)
    # the same loop with a cut (Sec. 5.1 "Top-k sampling": k = 2 and 10; a nucleus): one launch of
    # the streaming step kernel per step, rows gathered from the table
    cf = torch.empty(w.lanes, dtype=torch.float64, device="cuda")
    for name, k, p in (("top_k_2", 2, 1.0), ("top_k_10", 10, 1.0), ("top_p_0.9", 0, 0.9)):
        med, mn = timed(lambda: B.as_decode_bigram(table, starts, w.N, w.shift(), w.T, w.eos, w.temp, k, p, seq=seq,
                                                   length=ln, codes_final=cf))
        tokens = int(ln.sum().item())
        out["lattice_" + name] = {"ms_per_decode_median": med, "ms_per_decode_min": mn, "tokens": tokens,
                                  "tokens_per_s": tokens / med * 1e3, "launches_per_decode": 2 * w.T + 2,
                                  "row_gbs": tokens * w.V * w.elem_bytes / med / 1e6}
    # the other direction on the sequences just decoded: sequence -> interval, same tokens
    run_iid()
    med, mn = timed(lambda: B.as_encode_bigram(table, prev, seq, ln, w.temp, w.top_k, w.top_p))
    tokens = int(ln.sum().item())
    out["encode"] = {"ms_per_encode_median": med, "ms_per_encode_min": mn, "tokens": tokens,
                     "tokens_per_s": tokens / med * 1e3, "row_gbs": tokens * w.V * w.elem_bytes / med / 1e6}
    # what is computed from the decoded groups: n-gram diversity (Sec. 5.1) and the sample-mean
    # estimator of an additive synthetic reward (Sec. 4.2 / 5.2), lattice codes against iid codes
    r = torch.from_numpy(synth.reward_table(w.V, 78)).cuda()
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
    stats["ms_ngram_diversity"] = timed(lambda: B.as_ngram_diversity(seq, ln, w.N))[0] if fits else None
    stats["ms_reward_mean"] = timed(lambda: B.as_reward_mean(seq, ln, w.N, r))[0]
    out["groups"] = stats
    # the same decode with extended-precision codes (the lattice steers every token, not only the
    # first ~50 bits' worth): time, whole-sequence duplicate rates, and the estimator's spread again
    st0 = B.as_xp_lattice_state(w.N, w.shift(), 0, w.N, w.S)
    state = st0.clone()

    def run_xp():
        state.copy_(st0)
        B.as_decode_bigram_xp(table, prev, state, w.N, w.T, w.eos, w.temp, w.top_k, w.top_p, seq=seq, length=ln)
    out["lattice_extended_precision"] = decode_entry(run_xp)

    def run_xp_topk():
        state.copy_(st0)
        B.as_decode_bigram_xp(table, prev, state, w.N, w.T, w.eos, w.temp, 10, 1.0, seq=seq, length=ln)
    med, mn = timed(run_xp_topk)
    tokens = int(ln.sum().item())
    out["lattice_extended_precision_top_k_10"] = {"ms_per_decode_median": med, "ms_per_decode_min": mn, "tokens": tokens,
                                                  "tokens_per_s": tokens / med * 1e3, "launches_per_decode": 2 * w.T + 2,
                                                  "duplicate_prefix_rate": dup_rates(seq)}
    means, divs = [], []
    for k in range(K):
        stk = B.as_xp_lattice_state(w.N, float(shifts[k]), 0, w.N, w.S)
        B.as_decode_bigram_xp(table, prev, stk, w.N, w.T, w.eos, w.temp, w.top_k, w.top_p, seq=seq, length=ln)
        means.append(B.as_reward_mean(seq, ln, w.N, r)[1])
        if fits:
            divs.append(B.as_ngram_diversity(seq, ln, w.N)[2])
    means = torch.stack(means)
    stats["lattice_extended_precision"] = {
        "estimator_sd_over_%d_runs_mean_over_groups" % K: float(means.std(dim=0).mean().item()),
        "ngram_diversity_mean": float(torch.stack(divs).mean().item()) if fits else None}
    if eos_variant:
        # SUPPLEMENTARY variant, not the configuration as specified: with a random permutation the
        # EOS column's bias makes P(EOS) ~ 1e-10 and no lane ever stops early; here that column's
        # bias is raised (on the device: fp32 add, rounded to bf16 again) so that lanes stop after
        # ~30 tokens on average and per-lane early stop, padding and ragged lengths are timed
        eb = -3.0
        col = table[:, w.eos].float() - float(w.column_bias()[w.eos]) + eb
        tbl2 = table.clone()
        tbl2[:, w.eos] = col.to(table.dtype)
        note = "EOS column bias raised from %.2f to %.2f" % (float(w.column_bias()[w.eos]), eb)
        out["eos_raised_lattice"] = decode_entry(lambda: run_lattice(tbl2), note)
        out["eos_raised_iid"] = decode_entry(lambda: run_iid(tbl2), note)
        del tbl2
    out["workload"] = "c4: bf16 bigram table 32128x32128, %d starts x 32 codes, T<=%d, temp 0.8, EOS 1" % (S, T)
    return out


# ----------------------------------------------------------------------------- arms
def side_measurements(B, peak, skip_key):
    """One roofline block per step configuration (the headline's is measured by the caller), the
    iid-code run of the step kernel beside the lattice run, the cluster kernel beside the streaming
    kernel, two shapes outside the configurations, and the bigram loop."""
    import torch
    blocks, extras = {}, {}
    for name, lanes in (("c2", None), ("c3", None), ("c5", 1024), ("c5", 4096), ("c5", 8192)):
        w = step_workload(name, lanes)
        key = step_key(w)
        if key == skip_key:
            continue
        sb = StepBench(w, 0)
        med, mn, n = sb.per_launch_us(sb.step_stored)
        tpl = captured_traffic("as_step_stream_%s.md" % w.name, w.name)
        blocks[key] = roofline_block(w, med, mn, n, peak, step_bytes(w), tpl, stream_kernel_name(w))
        imed, imn, _ = sb.per_launch_us(sb.step_iid)
        blocks[key]["iid_codes_us_per_launch_median"] = imed
        blocks[key]["iid_codes_us_per_launch_min"] = imn
        if key == "c2":
            fmed, fmn, _ = sb.per_launch_us(sb.step)
            tmed, tmn, _ = sb.per_launch_us(sb.step_two_calls)
            blocks[key]["fused_first_step_us_median"] = fmed          # as_step_lattice
            blocks[key]["two_calls_us_median"] = tmed                 # as_lattice_codes + as_step
        if key == "c2":
            # the typical cut in place of top-k (general routine: no fast path)
            def step_typical():
                B.as_step(sb._next(), sb.codes, w.temp, 0, 1.0, tokens=sb.tokens, codes_out=sb.codes_out, typical_p=0.9)
            ymed, ymn, _ = sb.per_launch_us(step_typical, replays=5)
            blocks[key]["typical_p_0.9_us_median"] = ymed
        if key == "c5_1024":
            # the row split over a thread-block cluster (4 and 8 CTAs per lane) beside the default
            for cs in (4, 8):
                try:
                    B.as_tune(B.TUNE_STEP_PATH, 2)
                    B.as_tune(B.TUNE_CLUSTER, cs)
                    cmed, cmn, _ = sb.per_launch_us(sb.step_stored)
                finally:
                    B.as_tune(B.TUNE_CLUSTER, 0)
                    B.as_tune(B.TUNE_STEP_PATH, 0)
                blocks[key]["cluster_kernel_cs%d_us_median" % cs] = cmed
                blocks[key]["cluster_kernel_cs%d_us_min" % cs] = cmn
        del sb
        torch.cuda.empty_cache()
    # shapes outside the configurations: many lanes of a 32000-token vocabulary, flat rows with a wide
    # nucleus, and a step without any cut (every token kept)
    for key, w in (("many_lanes_4096x32000_top_k_40",
                    synth.StepWorkload("x1", 4096, 32000, synth.BF16, 3.0, 0.7, 40, 1.0, 20, 21, 22)),
                   ("no_cut_2048x32128_temp_0.8",
                    synth.StepWorkload("x2", 2048, 32128, synth.BF16, 2.5, 0.8, 0, 1.0, 40, 41, 43))):
        sb = StepBench(w, 0)
        med, mn, n = sb.per_launch_us(sb.step_stored)
        extras[key] = roofline_block(w, med, mn, n, peak, step_bytes(w))
        del sb
        torch.cuda.empty_cache()
    w = synth.StepWorkload("x3", 1024, 128256, synth.BF16, 3.0, 0.8, 0, 0.9, 60, 61, 62)
    sb = StepBench(w, 0)
    sb.ring = [device_rows(w.lanes, w.V, w.sigma, w.dtype, 60, None)]      # no Zipf bias: flat rows
    med, mn, n = sb.per_launch_us(sb.step_stored, replays=5)
    extras["wide_nucleus_flat_1024x128256_top_p_0.9"] = roofline_block(w, med, mn, n, peak, step_bytes(w))
    del sb
    torch.cuda.empty_cache()
    extras["bigram_decode"] = bench_bigram(10, 2)
    return blocks, extras


def run_ours(args):
    import torch
    rank, local_rank, world = dist_env()
    check_world(args.gpus, world)
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2210_15458_b200 import binding as B
    B.lib()
    w = step_workload(args.workload, args.lanes)
    key = step_key(w)
    sb = StepBench(w, rank)
    for _ in range(args.warmup):
        sb.step()
    g = sb.graph(sb.step, args.steps)              # the timed region: exactly K steps
    sb.replay_ms(g)                                # untimed: the first replay uploads the graph
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier(world)
    ms = sb.replay_ms(g)
    barrier(world)
    if rank == 0:
        # keep the same load running for ~0.6 s so that nvidia-smi (100 ms period) sees its clocks
        t_end = time.perf_counter() + 0.6
        while time.perf_counter() < t_end:
            g.replay()
            torch.cuda.synchronize()
    ms = max_over_ranks(ms, world, torch.device("cuda", local_rank))
    clocks = sampler.stop() if rank == 0 else None
    del g
    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return
    peak, peak_kind = measured_peaks()
    # the dominant kernel: the step is a single launch of the step kernel, timed launch by launch
    med, mn, n = sb.per_launch_us(sb.step)
    tpl = captured_traffic("as_step_stream_%s.md" % w.name, w.name)
    head = roofline_block(w, med, mn, n, peak, step_bytes(w, stored_codes=False), tpl,
                          stream_kernel_name(w) + " via as_step_lattice")
    head["peak_kind"] = peak_kind
    smed, smn, _ = sb.per_launch_us(sb.step_stored)
    imed, imn, _ = sb.per_launch_us(sb.step_iid)
    head["stored_lattice_codes_us_per_launch_median"] = smed
    head["iid_codes_us_per_launch_median"] = imed
    head["iid_codes_us_per_launch_min"] = imn
    value = w.lanes * w.V * world * args.steps / (ms / 1e3)
    line = {
        "metric": "logits decoded/s", "value": value, "unit": "logits/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_text(w), "lanes_per_gpu": w.lanes, "V": w.V, "l2": sb.l2_note(),
                   "step": "one as_step_lattice call: lattice codes of a fresh shift formed in the streaming step kernel, then the "
                           "kernel for the lanes it defers to the general routine (none on this workload: it leaves at once)",
                   "timing": "the K steps captured in one CUDA graph, replayed once between CUDA events; per-launch "
                             "median / min from %d replays of a shorter graph" % REPLAYS,
                   "inputs": "drawn on the device in the configuration's distribution (seeded)",
                   "parallelism": "lanes sharded, no collective"},
        "lane_steps_per_s": w.lanes * world * args.steps / (ms / 1e3),
        "hbm_gbs": step_bytes(w, stored_codes=False) * world * args.steps / (ms / 1e3) / 1e9,
        "gpu_launches": 2 * args.steps,
        "clocks": clocks,
        "roofline": head,
    }
    del sb
    torch.cuda.empty_cache()
    if world == 1:
        e_steps = max(1, min(args.steps, 3 if w.lanes * w.V * w.elem_bytes > (1 << 30) else 50))
        e_ms, h2d, d2h = e2e_step(w, e_steps, 1 if e_steps <= 3 else 3)
        line["e2e"] = {"value": w.lanes * w.V * e_steps / (e_ms / 1e3), "unit": "logits/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e_ms / e_steps,
                       "steps": e_steps, "entry_point": "as_step_host (pinned host buffers)"}
        torch.cuda.empty_cache()
        line["cpu_baseline"] = cpu_baseline_step(w)
        line["rooflines"] = {key: head}
        if not args.no_extras:
            blocks, extras = side_measurements(B, peak, key)
            line["rooflines"].update(blocks)
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
    # each step is a bounded sample of the workload's lanes, sized from a short probe so that the
    # K steps take about a minute
    probe = min(w.lanes, 32)
    rate, _, _, _ = oracle_rate(w, probe, 2.0)
    lanes = int(max(1, min(w.lanes, 256, rate * 60.0 / (max(args.steps, 1) * w.V))))
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
        "config": {"workload": workload_text(w) + " (CPU oracle, %s)" % sample},
        "cpu_baseline": {"value": value, "unit": "logits/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "logits/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c2", "c3", "c5", "c4"],
                    help="c4 prints the bigram decode / encode loop's own line (a side measurement)")
    ap.add_argument("--lanes", type=int, default=None,
                    help="lanes for c3 / c5 / c4 (default: c5 8192, c3 1024, c4 2048; c4: a multiple of 32)")
    ap.add_argument("--T", type=int, default=128, help="c4 only: maximum steps per lane (512-1024: summarisation-sized outputs)")
    ap.add_argument("--no-extras", action="store_true", help="skip the other configurations' blocks")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.workload == "c4":
        if args.impl == "reference" or dist_env()[2] > 1:
            raise SystemExit("--workload c4 is a single-GPU side measurement of the CUDA path")
        print(json.dumps(bench_bigram(min(args.steps, 10), min(args.warmup, 3), S=(args.lanes or 2048) // 32,
                                      T=args.T)))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
