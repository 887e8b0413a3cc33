#!/usr/bin/env python
"""Benchmark of the Batch-Max evicting-attention hot path (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl ours|reference]

A step is one pass of the whole path over one batch of the named workload: cache creation, every
block-wise prefill call (attention, score reduction, top-k eviction with compaction) and every decode
step (attention, score update, eviction).  `value` counts the tokens the batch pushed through the path
(prompt + generated) per second with all inputs resident in HBM; `e2e` is the same pass through the
host-fed entry points with pinned host buffers (copies inside the timed region).
With N > 1 every rank runs an independent replica on its own GPU (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "P&D evicting-attention tokens/s at max batch; % of TC (prefill) / HBM (decode) peak"
UNIT = "tokens/s"
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of the same command).
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"cfg2": {"attn_fwd": 92.6e6, "decode": 34.3e6}}   # profiles/attn_fwd_split_cfg2_traffic.md
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every call eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (roofline runs)")
    ap.add_argument("--prompt", type=int, default=None, help="override the workload's prompt length")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the workload's decode steps")
    ap.add_argument("--rule", default="average", choices=["average", "sum_recent", "current_query"],
                    help="eviction rule: the paper's average attention, or one of the two rules of Sec. 2")
    ap.add_argument("--compaction", default="stable", choices=["stable", "fill"],
                    help="stable: a cache's rows stay in position order (rows behind a pair that leaves move up); "
                         "fill: unordered rows, pairs that stay never move (same kept sets and outputs)")
    ap.add_argument("--ranges", type=int, default=4,
                    help="split the batch into this many sample ranges, each range's calls on a stream of its own (all "
                         "inside the step's graph): the caches of different samples are independent, so the tail of one "
                         "range's kernel overlaps the next kernel of another range")
    ap.add_argument("--ragged", action="store_true",
                    help="left-padded samples: seeded padding counts in [0, s/2] (sample 0 unpadded); launches eagerly")
    return ap.parse_args()


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


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


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
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                for nm, val in zip(names, r[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                continue
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
def run_reference(args, wl):
    """The CPU oracle as it stands, timed on the host cores on a bounded sample of the workload."""
    import numpy as np
    import torch
    from oracle import UnitCache
    from paper_2412_05693_b200.workloads import Inputs, schedule
    inp = Inputs(wl, "cpu")
    calls = schedule(wl)
    cores = torch.get_num_threads()

    def one_unit(smp, kh, max_calls=None):
        u = UnitCache(wl.d, wl.g)
        t = 0.0
        for kind, pos0, I, ev in calls[:max_calls]:
            q, k, v = inp.block(0, pos0, I, smp, 1)
            qq = q[0, :, kh * wl.g:(kh + 1) * wl.g].double().numpy()
            kk, vv = k[0, :, kh].double().numpy(), v[0, :, kh].double().numpy()
            t0 = time.perf_counter()
            u.process_block(qq, kk, vv, pos0, ev)
            t += time.perf_counter() - t0
        return t

    # size the sample: time one unit, then as many units as fit the budget per step
    t_unit = one_unit(0, 0)
    per_step_budget = max(args.cpu_seconds / max(1, args.steps + args.warmup), t_unit)
    units_per_step = max(1, min(wl.b * wl.Hkv, int(per_step_budget / t_unit)))
    unit_list = [(i % wl.b, (i // wl.b) % wl.Hkv) for i in range(units_per_step)]
    times = []
    for it in range(args.warmup + args.steps):
        t = sum(one_unit(s, h) for s, h in unit_list)
        if it >= args.warmup:
            times.append(t)
    t_mean = sum(times) / len(times)
    tokens_per_unit = (wl.s + wl.steps) / wl.Hkv          # a sample's tokens are shared by its Hkv caches
    value = units_per_step * tokens_per_unit / t_mean
    sample = (f"{units_per_step} of {wl.b * wl.Hkv} (sample, kv-head) caches of layer 0, whole schedule each; "
              f"tokens/s extrapolated linearly over caches (independent, equal cost)")
    return value, t_mean * 1e3, cores, sample


def cfg_dict(wl, extra=None):
    d = {"workload": wl.name, "b": wl.b, "Hq": wl.Hq, "Hkv": wl.Hkv, "d": wl.d, "s": wl.s, "block": wl.B,
         "kv_max": wl.K, "decode_steps": wl.steps, "layers": wl.L, "p_dec": wl.p_dec,
         "l2": "flushed between timed steps (256 MiB write); per-step inputs exceed L2"}
    if extra:
        d.update(extra)
    return d


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    from paper_2412_05693_b200.workloads import WORKLOADS
    wl = WORKLOADS[args.workload]
    over = {k: v for k, v in (("b", args.batch), ("s", args.prompt), ("steps", args.decode_steps)) if v is not None}
    if over:   # roofline runs: the named shape at another batch / prompt length (reported in `config`)
        wl = wl.with_(name=wl.name + "+" + ",".join(f"{k}={v}" for k, v in over.items()), **over)

    if args.impl == "reference":
        if rank != 0:
            return
        value, ms, cores, sample = run_reference(args, wl)
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": cfg_dict(wl),
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    from paper_2412_05693_b200.build import build
    if rank == 0 or world == 1:
        build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    import paper_2412_05693_b200 as bm
    from paper_2412_05693_b200.workloads import Inputs, schedule
    from paper_2412_05693_b200.workloads import config_for as make_config
    torch.cuda.set_device(local_rank)
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
    out_blk = torch.empty(wl.b, wl.B, wl.Hq, wl.d, dtype=wl.torch_dtype, device=dev)
    out_dec = torch.empty(wl.b, wl.Hq, wl.d, dtype=wl.torch_dtype, device=dev)
    arena = torch.empty(bm.arena_bytes(cfg), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)

    workspace = torch.empty(max(bm.workspace_bytes(cfg), 256), dtype=torch.uint8, device=dev)

    pads = None
    if args.ragged:
        import random
        rng = random.Random(wl.seed)
        pads = [0] + [rng.randrange(0, wl.s // 2 + 1) for _ in range(wl.b - 1)]
        args.no_graph = True     # the padding counts are copied from pageable host memory at the start of a step

    n_ranges = args.ranges if (args.ranges > 1 and wl.b % args.ranges == 0 and pads is None) else 1
    side = [torch.cuda.Stream(device=dev) for _ in range(n_ranges)] if n_ranges > 1 else []

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
                            cache.prefill_block(q[sl], k[sl], v[sl], pos0, out=out_blk[sl, :I], evict_to=ev, layer=layer,
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
                        cache.prefill_block(q, k, v, pos0, out=out_blk[:, :I], evict_to=ev, layer=layer)
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

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = bm.kernel_launch_count()
    one_step().close()
    launches_per_step = bm.kernel_launch_count() - launches0
    ms_step = timed(args.warmup, args.steps, use_graph=not args.no_graph)
    # the same step without its decode calls: the difference is the decode steps' time inside the timed region
    ms_prefill_only = timed(1, args.steps, use_graph=not args.no_graph, with_decode=False) if wl.steps > 0 else ms_step
    # the same step on unordered caches (pairs that stay never move; same kept sets and outputs), as a variant line
    variants = {}
    if args.compaction == "stable" and args.rule == "average" and not args.ragged:
        cfg_now[0] = make_config(wl, device=local_rank, rule=args.rule, compaction="fill")
        ms_fill = timed(args.warmup, args.steps, use_graph=not args.no_graph)
        cfg_now[0] = cfg
        variants["compaction_fill"] = {
            "ms_per_step": ms_fill, "value": whole_job_value(workload_tokens(wl), world, ms_fill), "unit": "tokens/s",
            "note": "BM_COMPACT_FILL: a cache's rows are an unordered set, the pairs that arrive take the rows that "
                    "were freed; the headline value is measured with rows kept in position order"}
    launches = launches_per_step * args.steps
    clocks = sampler.stop() if rank == 0 else None
    tokens = workload_tokens(wl)
    value = whole_job_value(tokens, world, ms_step)

    # ---- rooflines: every launch of an extra eager pass is bracketed by CUDA events inside the library
    prof = bm.binding.profile_pass(lambda: one_step(ranges=False).close())   # whole-batch calls, one after the other
    pk, pk_src = peaks()
    extra = {"kernel_ms_per_step": {k: v[0] for k, v in prof.items()},
             "kernel_launches_per_step": {k: v[1] for k, v in prof.items()}}
    rooflines = {}
    attn_ms, attn_n = prof["attn_fwd"]
    if attn_ms > 0:
        flops_per_step = 4.0 * wl.d * prefill_pairs(wl) * wl.b * wl.Hq * wl.L
        achieved = flops_per_step / (attn_ms * 1e-3) / 1e12
        peak = pk["bf16_tflops_sustained"] if wl.dtype == "bf16" else pk["bf16_tflops_sustained"] / 2
        rooflines["attn_fwd"] = {
            "bound": "tensor", "kernel": "prefill-block attention forward (attn_fwd_split)", "achieved": achieved,
            "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
            "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get(wl.name, {}).get("attn_fwd"),
            "peak_source": f"{pk_src} (sustained bf16 matmul)", "launches_per_step": attn_n,
            "avg_launch_ms": attn_ms / max(attn_n, 1),
            "algorithmic": "4*d FLOP per visible (query, key) pair"}
    dec_ms, dec_n = prof.get("decode", (0.0, 0))
    if dec_ms > 0:
        n1 = min(wl.K, wl.s) + 1
        e = wl.elem_bytes
        per_unit = n1 * 2 * wl.d * e + 16 * n1 + 2 * wl.d * e + 2 * wl.g * wl.d * e
        dec_bytes = per_unit * wl.b * wl.Hkv * dec_n
        gbs = dec_bytes / (dec_ms * 1e-3) / 1e9
        # duration per launch inside the timed region (graph replay): step time minus the prefill-only step time;
        # the per-launch event timing of the eager pass adds ~4 us of event overhead to a ~16 us kernel
        in_region_ms = max(ms_step - ms_prefill_only, 1e-6) * wl.L if not args.no_graph else dec_ms
        gbs_events = gbs
        gbs = dec_bytes / (in_region_ms * 1e-3) / 1e9
        moved = {}
        one_step(moved=moved).close()             # one more eager pass with the device-side counters on
        move_bytes = moved.get("decode", 0) * 2.0 * wl.d * e
        rooflines["decode"] = {
            "bound": "hbm", "kernel": "decode step with score update and eviction (decode_mma_kernel)",
            "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
            "achieved_with_per_launch_events": gbs_events, "ms_in_timed_region": in_region_ms,
            "achieved_with_compaction_writes": (dec_bytes + move_bytes) / (in_region_ms * 1e-3) / 1e9,
            "rows_moved_per_cache_and_step": moved.get("decode", 0) / max(1, wl.b * wl.Hkv * dec_n),
            "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get(wl.name, {}).get("decode"),
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

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        a2 = argparse.Namespace(**vars(args))
        a2.steps, a2.warmup = 1, 0
        v, ms, cores, sample = run_reference(a2, wl)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}

    if rank == 0:
        ppairs = prefill_pairs(wl) * wl.b * wl.Hq * wl.L
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
                "config": cfg_dict(wl, {"parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                                        "prefill_path": "tcgen05" if bm.last_prefill_path() == 1 else "simt-fp32",
                                        "launch": ("eager" if args.no_graph else "one CUDA graph per step, replayed") +
                                        (f"; {n_ranges} sample ranges on {n_ranges} streams" if n_ranges > 1 else ""),
                                        "rule": args.rule, "compaction": args.compaction,
                                        "left_pad": "none" if pads is None else
                                        f"seeded, {sum(pads)} of {wl.b * wl.s} prompt positions are padding"}),
                "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": int(launches),
                "clocks": clocks, "prefill_useful_tflop_per_step": 4.0 * wl.d * ppairs / 1e12}
        line.update(extra)
        if variants:
            line["variants"] = variants
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
