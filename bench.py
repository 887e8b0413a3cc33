#!/usr/bin/env python
"""Benchmark of the Batch-Max evicting-attention hot path (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3_max] [--impl ours|reference]

A step is one pass of the whole path over one batch of the named workload: cache creation, every
block-wise prefill call (attention, score reduction, top-k eviction with compaction) and every decode
step (attention, score update, eviction).  `value` counts the tokens the batch pushed through the path
(prompt + generated) per second with all inputs resident in HBM; `e2e` is the same path through the
host-fed entry points with pinned host buffers (copies inside the timed region).

The default workload, cfg3_max, is the configuration the metric is quoted on: the long-prompt shape at the
largest batch whose caches fit a 40 GiB arena (Sec. 1: the batch a memory budget admits), issued range by
range as a caller with such a batch must.  cfg4_max is the 32-layer stack in 120 GiB.  Any other name (cfg1,
cfg2, cfg3, cfg5 ...) runs that workload at its own batch with resident inputs inside one CUDA graph.
With N > 1 every rank runs an independent replica on its own GPU (the path has no exchange step); run
without a launcher, `--gpus N` starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "P&D evicting-attention tokens/s at max batch; % of TC (prefill) / HBM (decode) peak"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
GiB = 2 ** 30
MAX_BATCH = {"cfg3_max": ("cfg3", 40 * GiB), "cfg4_max": ("cfg4", 120 * GiB)}   # name -> (shape, cache budget)
PREFILL_MICRO, DECODE_MICRO = 256, 2048     # samples per call at the max-batch workloads


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg3_max")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the decode-only arm and the small-batch line")
    ap.add_argument("--no-graph", action="store_true", help="launch every call eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=20.0, help="target wall time of the oracle sample")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (roofline runs)")
    ap.add_argument("--prompt", type=int, default=None, help="override the workload's prompt length")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the workload's decode steps")
    ap.add_argument("--layers", type=int, default=None, help="run only the first N layers (cfg4_max)")
    ap.add_argument("--rule", default="average",
                    choices=["average", "sum_recent", "current_query", "window_pooled", "average_std"],
                    help="eviction rule: the paper's average attention, or one of the rules of Sec. 2 (H2O, TOVA, SnapKV "
                         "with window 32 / pool 7, RoCo with half of the kept pairs by standard deviation)")
    ap.add_argument("--compaction", default="stable", choices=["stable", "fill"],
                    help="stable: a cache's rows stay in position order (rows behind a pair that leaves move up); "
                         "fill: unordered rows, pairs that stay never move (same kept sets and outputs)")
    ap.add_argument("--ranges", type=int, default=4,
                    help="resident workloads: split the batch into this many sample ranges, each range's calls on a "
                         "stream of its own (all inside the step's graph)")
    ap.add_argument("--ragged", action="store_true",
                    help="left-padded samples: seeded padding counts in [0, s/2] (sample 0 unpadded); launches eagerly")
    ap.add_argument("--cpu-stub", action="store_true",
                    help="self-test of the multi-rank plumbing: no GPU, gloo, a fixed host-side step per rank")
    return ap.parse_args(argv)


# ------------------------------------------------------------------------------------------------
def workload_tokens(wl) -> int:
    return wl.b * (wl.s + wl.steps) * wl.L


def prefill_pairs(wl) -> int:
    """Visible (query, key) pairs of one sample's q-head over the whole prompt schedule."""
    n, pos, pairs = 0, 0, 0
    while pos < wl.s:
        I = min(wl.B, wl.s - pos)
        pairs += I * n + I * (I + 1) // 2
        n = min(n + I, wl.K)
        pos += I
    return pairs


def decode_bytes_per_cache(wl, calls) -> int:
    """Algorithmic bytes of all decode steps of one (sample, kv-head) cache: K and V rows read once per group,
    sum_weights and kv_ids read and written, the step's pair appended, q and out; compaction moves not counted."""
    e, n, total = wl.elem_bytes, min(wl.K, wl.s), 0
    for kind, pos0, I, ev in calls:
        if kind != "decode":
            continue
        n1 = n + 1
        total += n1 * (2 * wl.d * e + 16) + 2 * wl.d * e + 2 * wl.g * wl.d * e
        n = n1 if ev < 0 else min(n1, ev)
    return total


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d.get(k, FALLBACK_PEAKS[k])) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def dram_traffic(kernel: str, samples_per_launch: int):
    """DRAM bytes per launch of `kernel` from the committed ncu summary (dram__bytes_read.sum + dram__bytes_write.sum
    of one capture), scaled by the samples one launch processes (traffic grows in proportion to them).  Rows of the
    table: | kernel | samples in the captured launch | bytes | ...  Returns None when the summary has no such row."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.md")
    if not os.path.exists(path):
        return None
    for line in open(path):
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if len(cells) >= 3 and cells[0] == kernel:
            try:
                return float(cells[2]) * samples_per_launch / float(cells[1])
            except ValueError:
                continue
    return None


def max_over_ranks(x: float, device="cpu") -> float:
    """Largest value of x over all ranks of the default process group (x itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Replicas: every rank pushes the same number of tokens per step; the job's step time is the slowest rank's."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def spawn_ranks(n: int, argv) -> int:
    """`bench.py --gpus N` started without a launcher: run N ranks of this script, one per GPU, under torch's
    launcher on this node, and pass their exit code on.  Rank 0 prints the JSON line."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    return subprocess.call(cmd, env=env)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, pw, mx, reasons = [], [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                pw.append(float(r[2]))
                for nm, val in zip(names, r[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                continue
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm), "sm_mhz_min": sm[0] if sm else None, "power_w_max": max(pw) if pw else None}


# ------------------------------------------------------------------------------------------------
# The CPU oracle as it stands, timed on the host cores on a bounded sample of the workload's caches.
_ORACLE_JOB = {}


def _oracle_unit(idx):
    """One (sample, kv-head) cache through the whole schedule; returns the seconds spent inside the oracle."""
    from oracle import UnitCache
    job = _ORACLE_JOB
    wl, calls = job["wl"], job["calls"]
    qs, ks, vs = job["inputs"][idx]
    u = UnitCache(wl.d, wl.g)
    t0 = time.perf_counter()
    row = 0
    for kind, pos0, I, ev in calls:
        u.process_block(qs[row:row + I], ks[row:row + I], vs[row:row + I], pos0, ev)
        row += I
    return time.perf_counter() - t0


def _oracle_worker_init():
    try:                                     # one BLAS thread per worker: the cores are shared out by unit
        from threadpoolctl import threadpool_limits
        threadpool_limits(1)
    except Exception:
        pass


class OracleSample:
    """Inputs of `units` caches of layer 0 (whole schedule each), drawn once; run() times the oracle over them with
    one cache per task on `procs` worker processes."""

    def __init__(self, wl, units: int):
        import numpy as np
        from paper_2412_05693_b200.workloads import Inputs, schedule
        self.wl, self.calls = wl, schedule(wl)
        nb = min(wl.b, 64)                                  # the sample comes from the first samples of the batch
        inp = Inputs(wl.with_(b=nb), "cpu")
        self.units = [(i // wl.Hkv, i % wl.Hkv) for i in range(min(units, nb * wl.Hkv))]
        per_unit = {u: ([], [], []) for u in self.units}
        chunk = Inputs.CHUNK                                # the generator draws this many samples at a time
        for kind, pos0, I, ev in self.calls:
            for c0 in sorted({u[0] // chunk * chunk for u in self.units}):
                ns = min(chunk, nb - c0)
                q, k, v = inp.block(0, pos0, I, c0, ns)
                for (s2, kh) in self.units:
                    if c0 <= s2 < c0 + ns:
                        a = per_unit[(s2, kh)]
                        a[0].append(q[s2 - c0, :, kh * wl.g:(kh + 1) * wl.g].float().numpy())
                        a[1].append(k[s2 - c0, :, kh].float().numpy())
                        a[2].append(v[s2 - c0, :, kh].float().numpy())
        self.inputs = [tuple(np.concatenate(x) for x in per_unit[u]) for u in self.units]

    def run(self, procs: int):
        """Returns (wall seconds, CPU seconds inside the oracle summed over the caches)."""
        import multiprocessing as mp
        _ORACLE_JOB.update(wl=self.wl, calls=self.calls, inputs=self.inputs)
        idx = list(range(len(self.units)))
        t0 = time.perf_counter()
        if procs <= 1:
            _oracle_worker_init()
            cpu = [_oracle_unit(i) for i in idx]
        else:
            with mp.get_context("fork").Pool(procs, initializer=_oracle_worker_init) as pool:
                cpu = pool.map(_oracle_unit, idx, chunksize=1)
        return time.perf_counter() - t0, sum(cpu)

    def tokens(self) -> float:
        """Tokens the sampled caches stand for: a sample's tokens are shared by its Hkv caches (one layer)."""
        return len(self.units) * (self.wl.s + self.wl.steps) / self.wl.Hkv


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_baseline(wl, seconds: float):
    """cpu_baseline: a single-core figure from one cache, then as many caches as fit `seconds` over all cores."""
    cores = host_cores()
    one = OracleSample(wl, 1)
    wall1, _ = one.run(1)
    single = one.tokens() / wall1
    rounds = max(1, int(seconds / max(wall1 * 1.5, 1e-3)))          # workers slow each other down a little
    units = max(1, min(wl.b * wl.Hkv, cores * min(rounds, 4)))
    smp = OracleSample(wl, units)
    wall, cpu = smp.run(min(cores, units))
    value = smp.tokens() / wall
    return {"value": value, "unit": UNIT, "cores": min(cores, units), "kind": "oracle",
            "single_core_value": single, "wall_s": wall, "cpu_s": cpu,
            "sample": (f"{units} of {wl.b * wl.Hkv * wl.L} (layer, sample, kv-head) caches, whole schedule each "
                       f"(s={wl.s}, {wl.steps} decode steps), one cache per task on {min(cores, units)} worker "
                       f"processes; tokens/s extrapolated linearly over caches (independent, equal cost)")}


def run_reference(args, wl):
    """`--impl reference`: every step times the oracle over the same bounded sample of caches on all host cores."""
    cores = host_cores()
    one = OracleSample(wl, 1)
    wall1, _ = one.run(1)
    budget = max(args.cpu_seconds * 6.0 / max(1, args.steps + args.warmup), wall1)
    units = max(1, min(wl.b * wl.Hkv, cores * max(1, int(budget / (wall1 * 1.5)))))
    units = min(units, cores * 2)
    smp = OracleSample(wl, units)
    procs = min(cores, units)
    walls = []
    for it in range(args.warmup + args.steps):
        wall, _ = smp.run(procs)
        if it >= args.warmup:
            walls.append(wall)
    t = sum(walls) / len(walls)
    sample = (f"{units} of {wl.b * wl.Hkv * wl.L} (layer, sample, kv-head) caches per step, whole schedule each, one "
              f"cache per task on {procs} worker processes; tokens/s extrapolated linearly over caches")
    return smp.tokens() / t, t * 1e3, procs, sample, one.tokens() / wall1


def cfg_dict(wl, extra=None):
    d = {"workload": wl.name, "b": wl.b, "Hq": wl.Hq, "Hkv": wl.Hkv, "d": wl.d, "s": wl.s, "block": wl.B,
         "kv_max": wl.K, "decode_steps": wl.steps, "layers": wl.L, "p_dec": wl.p_dec}
    if extra:
        d.update(extra)
    return d


def forward_roofline(wl, attn_ms, attn_n, pk, pk_src, clocks, samples_per_launch):
    """Tensor-core roofline of the forward kernel: useful FLOPs (4*d per visible pair) over its launches' time."""
    flops = 4.0 * wl.d * prefill_pairs(wl) * wl.b * wl.Hq * wl.L
    achieved = flops / (attn_ms * 1e-3) / 1e12
    half = 1.0 if wl.dtype == "bf16" else 0.5
    burst, sust = pk["bf16_tflops"] * half, pk["bf16_tflops_sustained"] * half
    at_max = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz")
                  and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    peak = burst if at_max else sust
    return {"bound": "tensor", "kernel": "prefill-block attention forward (attn_fwd_split)", "achieved": achieved,
            "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
            "frac_of_burst_peak": achieved / burst, "frac_of_sustained_peak": achieved / sust,
            "peak_source": f"{pk_src} bf16 matmul, " + ("burst figure: the sampled SM clock stayed at its maximum"
                                                         if at_max else
                                                         "sustained figure: the sampled SM clock was below its maximum"),
            "traffic": dram_traffic("attn_fwd_split", samples_per_launch),
            "launches_per_step": attn_n, "avg_launch_ms": attn_ms / max(attn_n, 1),
            "algorithmic": "4*d FLOP per visible (query, key) pair; the score pass's recompute is not counted"}


# ------------------------------------------------------------------------------------------------
def run_max_batch(args, name, rank, world, local_rank, sampler):
    """cfg3_max / cfg4_max: the batch that fills the budget, calls issued range by range, eager launches (every
    call is milliseconds of GPU work), per-launch CUDA events of the library bracketing every kernel of the timed
    steps."""
    import torch
    import paper_2412_05693_b200 as bm
    from paper_2412_05693_b200.workloads import WORKLOADS, Inputs, schedule, config_for
    shape, budget = MAX_BATCH[name]
    wl = WORKLOADS[shape]
    over = {k: v for k, v in (("s", args.prompt), ("steps", args.decode_steps), ("L", args.layers)) if v is not None}
    wl = wl.with_(name=name + ("+" + ",".join(f"{k}={v}" for k, v in over.items()) if over else ""), **over)
    full_L = WORKLOADS[shape].L
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()

    def arm_config(batch, decode_only):
        growth = (wl.s + max(1, wl.p_dec) - wl.K) if decode_only else None
        c = config_for(wl.with_(L=full_L), device=local_rank, batch=batch, growth=growth,
                       max_call_samples=min(batch, DECODE_MICRO), rule=args.rule, compaction=args.compaction)
        return c

    b_pd = bm.max_batch(arm_config(1, False), budget) if args.batch is None else args.batch
    b_do = bm.max_batch(arm_config(1, True), budget)
    wl = wl.with_(b=b_pd)
    cfg = arm_config(b_pd, False)
    arena = torch.empty(bm.arena_bytes(cfg), dtype=torch.uint8, device=dev)
    workspace = torch.empty(max(bm.workspace_bytes(cfg), 256), dtype=torch.uint8, device=dev)

    # ---- inputs of ONE range of samples resident in HBM, reused by every range and layer (the prompts of the whole
    # batch do not fit: one block of cfg3 at b = 10072 is 63 GB of Q/K/V)
    calls = schedule(wl)
    inp = Inputs(wl.with_(b=max(PREFILL_MICRO, DECODE_MICRO)), dev)
    dev_in = []
    for kind, pos0, I, ev in calls:
        if kind == "prefill":
            dev_in.append(inp.block(0, pos0, I, 0, PREFILL_MICRO))
        else:
            q, k, v = inp.block(0, pos0, 1, 0, DECODE_MICRO)
            dev_in.append((q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous()))
    out_blk = torch.empty(PREFILL_MICRO * wl.B * wl.Hq * wl.d, dtype=wl.torch_dtype, device=dev)
    out_dec = torch.empty(DECODE_MICRO, wl.Hq, wl.d, dtype=wl.torch_dtype, device=dev)

    def one_step(config, batch, decode_only=False, moved=None):
        cache = bm.BatchMaxCache(config, arena=arena, workspace=workspace)
        if moved is not None:
            cache.count_moved_rows(True)
        for layer in range(wl.L):
            in_decode = False
            for ci, (kind, pos0, I, ev) in enumerate(calls):
                q, k, v = dev_in[ci]
                if kind == "prefill":
                    for s0 in range(0, batch, PREFILL_MICRO):
                        ns = min(PREFILL_MICRO, batch - s0)
                        o = out_blk[:ns * I * wl.Hq * wl.d].view(ns, I, wl.Hq, wl.d)
                        cache.prefill_block(q[:ns], k[:ns], v[:ns], pos0, out=o, evict_to=-1 if decode_only else ev,
                                            layer=layer, sample0=s0)
                else:
                    if not in_decode:
                        in_decode = True
                        if decode_only:               # ONE compression to kv_max after the prompt (Sec. 1)
                            for s0 in range(0, batch, DECODE_MICRO):
                                cache.evict(wl.K, layer=layer, sample0=s0, nsamples=min(DECODE_MICRO, batch - s0))
                        if moved is not None:
                            moved["prefill"] = moved.get("prefill", 0) + cache.moved_rows(reset=True)
                    for s0 in range(0, batch, DECODE_MICRO):
                        ns = min(DECODE_MICRO, batch - s0)
                        cache.decode_step(q[:ns], k[:ns], v[:ns], out=out_dec[:ns], evict_to=ev, layer=layer,
                                          sample0=s0)
            if moved is not None:
                moved["decode"] = moved.get("decode", 0) + cache.moved_rows(reset=True)
        return cache

    def timed(n_warm, n_steps, config, batch, decode_only=False, profile=False, moved=None):
        import torch.distributed as dist
        for w in range(n_warm):
            one_step(config, batch, decode_only, moved if w == 0 else None).close()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ms, prof = [], {}
        L = bm.lib()
        if profile:
            bm.binding.profile_pass(lambda: None)      # drop anything recorded earlier
            L.bm_profile_enable(1)
        try:
            for _ in range(n_steps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                one_step(config, batch, decode_only).close()
                e1.record(stream)
                e1.synchronize()
                ms.append(e0.elapsed_time(e1))
                if profile:
                    for k, (t, n) in bm.binding.profile_read().items():
                        a = prof.setdefault(k, [0.0, 0])
                        a[0] += t
                        a[1] += n
        finally:
            if profile:
                L.bm_profile_enable(0)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return max_over_ranks(sum(ms), dev) / n_steps, {k: (t / n_steps, n // n_steps) for k, (t, n) in prof.items()}

    launches0 = bm.kernel_launch_count()
    moved = {}
    ms_step, prof = timed(max(args.warmup, 1), args.steps, cfg, b_pd, profile=True, moved=moved)
    launches = (bm.kernel_launch_count() - launches0) * args.steps // (max(args.warmup, 1) + args.steps)   # timed steps
    clocks = sampler.stop() if sampler is not None else None
    tokens = workload_tokens(wl)
    value = whole_job_value(tokens, world, ms_step)
    pk, pk_src = peaks()

    kernel_ms = {k: v[0] for k, v in prof.items()}
    kernel_n = {k: v[1] for k, v in prof.items()}
    rooflines = {}
    if kernel_ms.get("attn_fwd", 0) > 0:
        rooflines["attn_fwd"] = forward_roofline(wl, kernel_ms["attn_fwd"], kernel_n["attn_fwd"], pk, pk_src, clocks,
                                                 PREFILL_MICRO)
        call_ms = kernel_ms["attn_fwd"] + kernel_ms.get("score", 0.0) + kernel_ms.get("evict", 0.0)
        flops = 4.0 * wl.d * prefill_pairs(wl) * wl.b * wl.Hq * wl.L
        whole = flops / (call_ms * 1e-3) / 1e12
        rooflines["prefill_call"] = {
            "bound": "tensor", "kernel": "whole bm_prefill_block: forward + score pass + eviction kernels",
            "achieved": whole, "peak": rooflines["attn_fwd"]["peak"], "unit": "TFLOP/s",
            "frac": whole / rooflines["attn_fwd"]["peak"],
            "frac_of_burst_peak": whole / pk["bf16_tflops"], "frac_of_sustained_peak": whole / pk["bf16_tflops_sustained"],
            "algorithmic": "the same useful FLOPs; recompute and eviction count as overhead"}
    if kernel_ms.get("decode", 0) > 0:
        dec_bytes = decode_bytes_per_cache(wl, calls) * wl.b * wl.Hkv * wl.L
        move_bytes = moved.get("decode", 0) * 2.0 * wl.d * wl.elem_bytes
        gbs = dec_bytes / (kernel_ms["decode"] * 1e-3) / 1e9
        gbs_mv = (dec_bytes + move_bytes) / (kernel_ms["decode"] * 1e-3) / 1e9
        rooflines["decode"] = {
            "bound": "hbm", "kernel": "decode step with score update and eviction (decode_mma_kernel)",
            "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
            "achieved_with_compaction_writes": gbs_mv, "frac_with_compaction_writes": gbs_mv / pk["hbm_gbs"],
            "rows_moved_per_cache_and_step": moved.get("decode", 0) / max(1, wl.b * wl.Hkv * wl.L * wl.steps),
            "traffic": dram_traffic("decode_mma_kernel", DECODE_MICRO),
            "peak_source": f"{pk_src} (HBM copy)", "launches_per_step": kernel_n["decode"],
            "avg_launch_ms": kernel_ms["decode"] / max(kernel_n["decode"], 1),
            "algorithmic": "(n+1)*(2*d*e+16) + 2*d*e + 2*g*d*e bytes per cache and step, compaction moves not counted"}
    by_time = [k for k in ("attn_fwd", "decode") if k in rooflines]
    dominant = max(by_time, key=lambda k: kernel_ms[k]) if by_time else None
    roofline = dict(rooflines[dominant]) if dominant else None
    if roofline is not None:
        roofline["share_of_kernel_time"] = kernel_ms[dominant] / sum(kernel_ms.values())

    # ---- variants: the decode-only compression arm at ITS largest batch in the same arena (Sec. 1), cfg2 at b = 16
    variants = {}
    if not args.no_variants and args.batch is None:
        cfg_do = arm_config(b_do, True)
        assert bm.arena_bytes(cfg_do) <= arena.numel()
        ms_do, _ = timed(1, min(3, args.steps), cfg_do, b_do, decode_only=True)
        tok_do = b_do * (wl.s + wl.steps) * wl.L
        variants["decode_only_compression"] = {
            "b": b_do, "ms_per_step": ms_do, "value": whole_job_value(tok_do, world, ms_do), "unit": UNIT,
            "generated_tokens_per_s": world * b_do * wl.steps * wl.L / (ms_do * 1e-3),
            "note": "whole prompt cached during prefilling (cap = s + 1), one compression to kv_max, then the same "
                    "decode steps; largest batch of that layout in the same arena"}
        variants["pd_generated_tokens_per_s"] = world * b_pd * wl.steps * wl.L / (ms_step * 1e-3)

    # ---- end to end: a stated sub-batch through the host-fed entry points, inputs and outputs in a bounded ring of
    # pinned host buffers (the whole batch's prompts would be a terabyte of pinned memory)
    e2e = None
    if not args.no_e2e:
        e2e_b, e2e_micro, ring_n = 128, 64, 4
        wl_e = wl.with_(b=e2e_b)
        cfg_e = config_for(wl_e.with_(L=full_L), device=local_rank, batch=e2e_b, max_call_samples=e2e_b, rule=args.rule,
                           compaction=args.compaction)
        ring_blk, ring_dec = [], []
        for r in range(ring_n):
            q, k, v = dev_in[r % len(dev_in)] if calls[r % len(calls)][0] == "prefill" else dev_in[0]
            hq, hk, hv = (t[:e2e_micro].cpu().pin_memory() for t in (q, k, v))
            ring_blk.append((hq, hk, hv, torch.empty_like(hq).pin_memory()))
        dq, dk, dv = dev_in[-1] if calls[-1][0] == "decode" else (None, None, None)
        if dq is not None:
            for r in range(ring_n):
                hq, hk, hv = (t[:e2e_b].cpu().pin_memory() for t in (dq, dk, dv))
                ring_dec.append((hq, hk, hv, torch.empty_like(hq).pin_memory()))
        h2d = d2h = 0

        def e2e_step(count=False):
            nonlocal h2d, d2h
            cache = bm.BatchMaxCache(cfg_e, arena=arena, workspace=workspace)
            turn = 0
            for layer in range(wl.L):
                for kind, pos0, I, ev in calls:
                    if kind == "prefill":
                        for s0 in range(0, e2e_b, e2e_micro):
                            hq, hk, hv, ho = ring_blk[turn % ring_n]
                            turn += 1
                            cache.prefill_block_host(hq[:, :I], hk[:, :I], hv[:, :I], pos0, ho[:, :I], evict_to=ev,
                                                     layer=layer, sample0=s0)
                            if count:
                                h2d += sum(t[:, :I].numel() * t.element_size() for t in (hq, hk, hv))
                                d2h += ho[:, :I].numel() * ho.element_size()
                    else:
                        hq, hk, hv, ho = ring_dec[turn % ring_n]
                        turn += 1
                        cache.decode_step_host(hq, hk, hv, ho, evict_to=ev, layer=layer)
                        if count:
                            h2d += sum(t.numel() * t.element_size() for t in (hq, hk, hv))
                            d2h += ho.numel() * ho.element_size()
            return cache

        assert all(I == wl.B for kind, _, I, _ in calls if kind == "prefill"), "host ring holds whole blocks"
        e2e_step(count=True).close()
        torch.cuda.synchronize()
        ms = []
        for _ in range(max(1, min(args.steps, 3))):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            e2e_step().close()
            e1.record(stream)
            e1.synchronize()
            ms.append(e0.elapsed_time(e1))
        ms_e2e = max_over_ranks(sum(ms), dev) / len(ms)
        e2e = {"value": whole_job_value(workload_tokens(wl_e), world, ms_e2e), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "batch": e2e_b,
               "note": f"sub-batch of {e2e_b} samples in calls of {e2e_micro}, whole schedule, through "
                       f"bm_prefill_block_host / bm_decode_step_host; inputs and outputs in a ring of {ring_n} pinned "
                       "host buffers per call kind (copies of every call inside the timed region)"}
        del ring_blk, ring_dec

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 1), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
            "config": cfg_dict(wl, {
                "budget_GiB": budget / GiB, "arena_GiB": arena.numel() / GiB, "cap": cfg.kv_max + cfg.growth,
                "b_decode_only_compression": b_do, "batch_ratio": b_pd / b_do,
                "batch_ratio_predicted": (wl.s + max(1, wl.p_dec)) / (wl.K + max(1, wl.p_dec)),
                "prefill_samples_per_call": PREFILL_MICRO, "decode_samples_per_call": DECODE_MICRO,
                "inputs": f"Q/K/V of one range of samples ({PREFILL_MICRO} for prefill, {DECODE_MICRO} for decode) "
                          "resident in HBM and reused by every range and layer; the whole batch's prompts do not fit",
                "l2": "no flush needed: a step streams the whole arena and tens of GB of inputs, far beyond L2",
                "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                "launch": "eager, one call per sample range", "rule": args.rule, "compaction": args.compaction,
                "prefill_path": "tcgen05" if bm.last_prefill_path() == 1 else "simt-fp32"}),
            "roofline": roofline, "rooflines": rooflines, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks, "kernel_ms_per_step": kernel_ms, "kernel_launches_per_step": kernel_n,
            "timing": "value: CUDA events around each timed step; kernel_ms_per_step and every roofline: CUDA events "
                      "around every kernel launch of the same timed steps",
            "prefill_useful_tflop_per_step": 4.0 * wl.d * prefill_pairs(wl) * wl.b * wl.Hq * wl.L / 1e12,
            "rows_moved_per_step": moved}
    if variants:
        line["variants"] = variants
    return line, wl


# ------------------------------------------------------------------------------------------------
def run_resident(args, wl, rank, world, local_rank, sampler, light=False):
    """A workload at its own (small) batch: inputs of the whole schedule resident, the step captured in one CUDA
    graph and replayed.  `light`: only the step time (used for the small-batch entry of the default line)."""
    import torch
    import torch.distributed as dist
    import paper_2412_05693_b200 as bm
    from paper_2412_05693_b200.workloads import Inputs, schedule
    from paper_2412_05693_b200.workloads import config_for as make_config
    dev = torch.device("cuda", local_rank)
    calls = schedule(wl)
    cfg = make_config(wl, device=local_rank, rule=args.rule, compaction=args.compaction)
    cfg_now = [cfg]      # the configuration one_step() builds its cache with
    stream = torch.cuda.current_stream()

    # ---- inputs resident in HBM (layer 0's stream is reused for every layer: layers are independent)
    inp = Inputs(wl, dev)
    dev_in = []
    for kind, pos0, I, ev in calls:
        q, k, v = inp.block(0, pos0, I)
        if kind == "decode":
            q, k, v = q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous()
        dev_in.append((q, k, v))
    out_blk = torch.empty(wl.b * wl.B * wl.Hq * wl.d, dtype=wl.torch_dtype, device=dev)
    out_dec = torch.empty(wl.b, wl.Hq, wl.d, dtype=wl.torch_dtype, device=dev)
    arena = torch.empty(bm.arena_bytes(cfg), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)
    workspace = torch.empty(max(bm.workspace_bytes(cfg), 256), dtype=torch.uint8, device=dev)

    def blk_out(ns, I):
        return out_blk[:ns * I * wl.Hq * wl.d].view(ns, I, wl.Hq, wl.d)

    pads = None
    no_graph = args.no_graph
    if args.ragged and not light:
        import random
        rng = random.Random(wl.seed)
        pads = [0] + [rng.randrange(0, wl.s // 2 + 1) for _ in range(wl.b - 1)]
        no_graph = True     # the padding counts are copied from pageable host memory at the start of a step

    n_ranges = args.ranges if (args.ranges > 1 and wl.b % args.ranges == 0 and pads is None) else 1
    side = [torch.cuda.Stream(device=dev) for _ in range(n_ranges)] if n_ranges > 1 else []
    # every range writes its own part of the block output buffer
    out_rng = [torch.empty((wl.b // n_ranges) * wl.B * wl.Hq * wl.d, dtype=wl.torch_dtype, device=dev)
               for _ in range(n_ranges)] if n_ranges > 1 else []

    def step_in_ranges(cache, with_decode):
        """The same calls, one sample range per stream; forked from and joined to the current stream."""
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        nb = wl.b // n_ranges
        for r, st in enumerate(side):
            st.wait_event(fork)
            sl = slice(r * nb, (r + 1) * nb)
            with torch.cuda.stream(st):
                for layer in range(wl.L):
                    for ci, (kind, pos0, I, ev) in enumerate(calls):
                        q, k, v = dev_in[ci]
                        if kind == "prefill":
                            o = out_rng[r][:nb * I * wl.Hq * wl.d].view(nb, I, wl.Hq, wl.d)
                            cache.prefill_block(q[sl], k[sl], v[sl], pos0, out=o, evict_to=ev, layer=layer,
                                                sample0=r * nb)
                        elif with_decode:
                            cache.decode_step(q[sl], k[sl], v[sl], out=out_dec[sl], evict_to=ev, layer=layer,
                                              sample0=r * nb)
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    def one_step(host_bufs=None, with_decode=True, moved=None, ranges=True):
        cache = bm.BatchMaxCache(cfg_now[0], arena=arena, workspace=workspace)
        if pads is not None:
            cache.set_left_pad(pads)
        if n_ranges > 1 and ranges and host_bufs is None and moved is None:
            step_in_ranges(cache, with_decode)
            return cache
        if moved is not None:                 # count the rows the compactions move, prefill and decode apart
            cache.count_moved_rows(True)
        for layer in range(wl.L):
            for ci, (kind, pos0, I, ev) in enumerate(calls):
                if kind == "decode" and not with_decode:
                    continue
                if moved is not None and kind == "decode" and (ci == 0 or calls[ci - 1][0] != "decode"):
                    moved["prefill"] = moved.get("prefill", 0) + cache.moved_rows(reset=True)
                if host_bufs is None:
                    q, k, v = dev_in[ci]
                    if kind == "prefill":
                        cache.prefill_block(q, k, v, pos0, out=blk_out(wl.b, I), evict_to=ev, layer=layer)
                    else:
                        cache.decode_step(q, k, v, out=out_dec, evict_to=ev, layer=layer)
                else:
                    q, k, v, o = host_bufs[ci]
                    if kind == "prefill":
                        cache.prefill_block_host(q, k, v, pos0, o, evict_to=ev, layer=layer)
                    else:
                        cache.decode_step_host(q, k, v, o, evict_to=ev, layer=layer)
            if moved is not None:
                moved["decode"] = moved.get("decode", 0) + cache.moved_rows(reset=True)
        return cache

    def timed(n_warm, n_steps, host_bufs=None, use_graph=False, with_decode=True):
        for _ in range(n_warm):
            one_step(host_bufs, with_decode).close()
        torch.cuda.synchronize()
        graph = None
        if use_graph:
            # every call of the step is stream-ordered and allocation-free, so the whole step (cache creation,
            # all prefill blocks, all decode steps) is captured once and replayed
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                one_step(host_bufs, with_decode).close()
            graph.replay()
            torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ms = []
        for _ in range(n_steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            if graph is not None:
                graph.replay()
            else:
                one_step(host_bufs, with_decode).close()
            e1.record(stream)
            e1.synchronize()
            ms.append(e0.elapsed_time(e1))
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return max_over_ranks(sum(ms), dev) / n_steps

    launches0 = bm.kernel_launch_count()
    one_step().close()
    launches_per_step = bm.kernel_launch_count() - launches0
    ms_step = timed(args.warmup, args.steps, use_graph=not no_graph)
    tokens = workload_tokens(wl)
    value = whole_job_value(tokens, world, ms_step)
    if light:
        return {"value": value, "unit": UNIT, "ms_per_step": ms_step, "config": cfg_dict(wl),
                "launch": "one CUDA graph per step, replayed" + (f"; {n_ranges} sample ranges on {n_ranges} streams"
                                                                  if n_ranges > 1 else "")}, wl
    # the same step without its decode calls: the difference is the decode steps' time inside the timed region
    ms_prefill_only = timed(1, args.steps, use_graph=not no_graph, with_decode=False) if wl.steps > 0 else ms_step
    # the same step on unordered caches (pairs that stay never move; same kept sets and outputs), as a variant line
    variants = {}
    if args.compaction == "stable" and args.rule == "average" and not args.ragged and not args.no_variants:
        cfg_now[0] = make_config(wl, device=local_rank, rule=args.rule, compaction="fill")
        ms_fill = timed(args.warmup, args.steps, use_graph=not no_graph)
        cfg_now[0] = cfg
        variants["compaction_fill"] = {
            "ms_per_step": ms_fill, "value": whole_job_value(workload_tokens(wl), world, ms_fill), "unit": "tokens/s",
            "note": "BM_COMPACT_FILL: a cache's rows are an unordered set, the pairs that arrive take the rows that "
                    "were freed; the headline value is measured with rows kept in position order"}
    launches = launches_per_step * args.steps
    clocks = sampler.stop() if sampler is not None else None

    # ---- rooflines.  Forward kernel: every launch of an extra eager pass of whole-batch calls is bracketed by CUDA
    # events inside the library.  Decode kernel: its launches last ~10 us, which per-launch events overstate, so its
    # time is taken inside the timed region as the step's graph minus a graph of the prefill calls alone.
    prof = bm.binding.profile_pass(lambda: one_step(ranges=False).close())
    pk, pk_src = peaks()
    extra = {"kernel_ms_per_step": {k: v[0] for k, v in prof.items()},
             "kernel_launches_per_step": {k: v[1] for k, v in prof.items()},
             "timing": "value: CUDA events around each replayed step; attn_fwd roofline and kernel_ms_per_step: CUDA "
                       "events around every launch of one extra eager pass; decode roofline: replayed step minus "
                       "replayed prefill-only step"}
    rooflines = {}
    attn_ms, attn_n = prof["attn_fwd"]
    if attn_ms > 0:
        rooflines["attn_fwd"] = forward_roofline(wl, attn_ms, attn_n, pk, pk_src, clocks, wl.b)
    dec_ms, dec_n = prof.get("decode", (0.0, 0))
    if dec_ms > 0:
        dec_bytes = decode_bytes_per_cache(wl, calls) * wl.b * wl.Hkv * wl.L
        in_region_ms = max(ms_step - ms_prefill_only, 1e-6) if not no_graph else dec_ms
        gbs = dec_bytes / (in_region_ms * 1e-3) / 1e9
        moved = {}
        one_step(moved=moved).close()             # one more eager pass with the device-side counters on
        move_bytes = moved.get("decode", 0) * 2.0 * wl.d * wl.elem_bytes
        rooflines["decode"] = {
            "bound": "hbm", "kernel": "decode step with score update and eviction (decode_mma_kernel)",
            "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
            "achieved_with_per_launch_events": dec_bytes / (dec_ms * 1e-3) / 1e9, "ms_in_timed_region": in_region_ms,
            "achieved_with_compaction_writes": (dec_bytes + move_bytes) / (in_region_ms * 1e-3) / 1e9,
            "rows_moved_per_cache_and_step": moved.get("decode", 0) / max(1, wl.b * wl.Hkv * dec_n),
            "traffic": dram_traffic("decode_mma_kernel", wl.b),
            "in_timed_region": (f"every decode step runs as {n_ranges} concurrent launches, one per sample range; "
                                "achieved = bytes of all of them / their time in the region") if n_ranges > 1 else
                               "one launch per decode step",
            "peak_source": f"{pk_src} (HBM copy)", "launches_per_step": dec_n,
            "avg_launch_ms": dec_ms / max(dec_n, 1),
            "algorithmic": "(n+1)*(2*d*e+16) + 2*d*e + 2*g*d*e bytes per cache and step, compaction moves not counted"}
    # the kernel with the largest share of the step is the one reported as `roofline`
    dominant = max(rooflines, key=lambda k: extra["kernel_ms_per_step"][k]) if rooflines else None
    roofline = dict(rooflines[dominant]) if dominant else None
    if roofline is not None:
        roofline["share_of_kernel_time"] = extra["kernel_ms_per_step"][dominant] / sum(extra["kernel_ms_per_step"].values())
    extra["rooflines"] = rooflines

    # ---- end to end through the host-fed entry points (pinned host inputs, outputs read back)
    e2e = None
    if not args.no_e2e:
        host_bufs, h2d, d2h = [], 0, 0
        for (q, k, v) in dev_in:
            hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
            ho = torch.empty_like(hq).pin_memory()
            host_bufs.append((hq, hk, hv, ho))
            h2d += sum(t.numel() * t.element_size() for t in (hq, hk, hv))
            d2h += ho.numel() * ho.element_size()
        ms_e2e = timed(1, max(1, min(args.steps, 3)), host_bufs)
        e2e = {"value": whole_job_value(tokens, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d * wl.L,
               "d2h_bytes_per_step": d2h * wl.L, "ms_per_step": ms_e2e}
        del host_bufs

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
            "config": cfg_dict(wl, {"parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                                    "l2": "flushed between timed steps (256 MiB write); per-step inputs exceed L2",
                                    "prefill_path": "tcgen05" if bm.last_prefill_path() == 1 else "simt-fp32",
                                    "launch": ("eager" if no_graph else "one CUDA graph per step, replayed") +
                                    (f"; {n_ranges} sample ranges on {n_ranges} streams" if n_ranges > 1 else ""),
                                    "rule": args.rule, "compaction": args.compaction,
                                    "left_pad": "none" if pads is None else
                                    f"seeded, {sum(pads)} of {wl.b * wl.s} prompt positions are padding"}),
            "roofline": roofline, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks, "prefill_useful_tflop_per_step": 4.0 * wl.d * prefill_pairs(wl) * wl.b * wl.Hq * wl.L / 1e12}
    line.update(extra)
    if variants:
        line["variants"] = variants
    return line, wl


# ------------------------------------------------------------------------------------------------
def run_cpu_stub(args, rank, world):
    """Multi-rank plumbing without a GPU: every rank "runs" a replica whose step takes a rank-dependent time on the
    host, and the line is assembled as for the real benchmark (max over ranks, whole-job value, n_gpus)."""
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        time.sleep(0.002 * (1 + rank))               # rank r's replica takes 2 (r + 1) ms per step
        if it >= args.warmup:
            ms.append((time.perf_counter() - t0) * 1e3)
    ms_step = max_over_ranks(sum(ms)) / len(ms)
    tokens = 1000
    if world > 1:
        dist.barrier()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": whole_job_value(tokens, world, ms_step), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
                          "higher_is_better": True, "scaling": "weak", "data": "none (cpu stub of the rank plumbing)",
                          "config": {"workload": "cpu-stub", "parallelism": f"replicas x{world}"},
                          "gpu_launches": 0}))
    if world > 1:
        dist.destroy_process_group()


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    args = parse_args(argv)
    launched = "RANK" in os.environ and "WORLD_SIZE" in os.environ
    if args.gpus > 1 and not launched and args.impl == "ours":
        sys.exit(spawn_ranks(args.gpus, argv))          # one process per GPU, started by this script itself
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.cpu_stub:
        return run_cpu_stub(args, rank, world)
    from paper_2412_05693_b200.workloads import WORKLOADS

    def named_workload():
        if args.workload in MAX_BATCH:
            shape, budget = MAX_BATCH[args.workload]
            return WORKLOADS[shape], args.workload
        return WORKLOADS[args.workload], args.workload
    base, name = named_workload()
    over = {k: v for k, v in (("b", args.batch), ("s", args.prompt), ("steps", args.decode_steps)) if v is not None}

    if args.impl == "reference":
        if rank != 0:
            return
        wl = base
        if name in MAX_BATCH:                            # the product arm's batch: the budget's largest (memory model
            per_sample = wl.L * wl.Hkv * (wl.K + max(1, wl.p_dec)) * (2 * wl.d * wl.elem_bytes + 8)   # of Sec. 1)
            wl = wl.with_(b=(MAX_BATCH[name][1] - 1024) // per_sample, name=name)
        if over:
            wl = wl.with_(**over)
        value, ms, procs, sample, single = run_reference(args, wl)
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": cfg_dict(wl),
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": procs, "kind": "oracle", "sample": sample,
                                 "single_core_value": single},
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    from paper_2412_05693_b200.build import build
    if local_rank == 0 or world == 1:
        build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    torch.cuda.set_device(local_rank)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler is not None:
        sampler.start()
    if name in MAX_BATCH:
        line, wl = run_max_batch(args, name, rank, world, local_rank, sampler)
        if not args.no_variants and args.batch is None:
            small, _ = run_resident(args, WORKLOADS["cfg2"], rank, world, local_rank, None, light=True)
            small["note"] = "the small-batch configuration (b = 16): its cache state sits in L2"
            line.setdefault("variants", {})["cfg2"] = small
    else:
        wl = base
        if over:   # roofline runs: the named shape at another batch / prompt length (reported in `config`)
            wl = wl.with_(name=wl.name + "+" + ",".join(f"{k}={v}" for k, v in over.items()), **over)
        line, wl = run_resident(args, wl, rank, world, local_rank, sampler)
    torch.cuda.synchronize()
    if rank == 0:
        line["cpu_baseline"] = None
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = oracle_baseline(wl, args.cpu_seconds)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
