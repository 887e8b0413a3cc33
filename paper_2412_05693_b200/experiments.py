"""Whole-workload runs at the paper-scale batch sizes (one JSON line per run on stdout).

    python -m paper_2412_05693_b200.experiments --run cfg3_max      # P&D arm at the batch that fills 40 GiB
    python -m paper_2412_05693_b200.experiments --run cfg3_ratio    # P&D vs decode-only compression, same arena
    python -m paper_2412_05693_b200.experiments --run cfg4          # 32 layers, batch that fills 120 GiB
    python -m paper_2412_05693_b200.experiments --run cfg5          # the six (block, kv_max) combinations
    python -m paper_2412_05693_b200.experiments --run sec4          # Sec. 4's arms: BM (Algorithm 1) vs ED vs FKV

Batches this large cannot keep their prompts resident (one block of cfg3 at b = 10072 is 63 GB of Q/K/V), so
inputs are drawn on the fly per (layer, block, range of samples) from the seeded generator and every library
call is timed on its own with CUDA events; generation time is outside the timed regions.  Only the C-ABI
library runs inside them.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2412_05693_b200 import BatchMaxCache, Config, arena_bytes, max_batch  # noqa: E402
from paper_2412_05693_b200.workloads import CFG5_SWEEP, WORKLOADS, Inputs, Workload  # noqa: E402

GiB = 2 ** 30


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), "measured"
    return 6650.0, 1400.0, "fallback"


DECODE_MICRO = 2048   # samples per decode call (decode inputs are tiny, so ranges can be much wider than in prefill)


ARMS = {
    "pd": "Batch-Max in the build's cadence: evict to K after every block and (when full) decode step",
    "do": "decoding-only compression (Sec. 1): whole prompt cached, one compression to K, then as pd",
    "alg1": "Batch-Max exactly as Algorithm 1: limit kv_bar, p pairs removed before each block of p / when full",
    "ed": "extreme decoding-only eviction (Algorithm 3): whole prompt cached, then only the newest pair kept",
    "fkv": "full KV cache: nothing is ever removed",
}


def make_cfg(wl: Workload, batch: int, arm: str, micro: int, device: int = 0, kv_bar: int | None = None,
             p: int = 64, compaction: str = "stable") -> Config:
    """Cache geometry of an arm; cap = kv_max + growth is what the memory model charges per cache."""
    block = wl.B
    if arm == "pd":
        kv_max, growth = wl.K, max(1, wl.p_dec)
    elif arm == "do":
        kv_max, growth = wl.K, wl.s + max(1, wl.p_dec) - wl.K
    elif arm == "alg1":
        kv_max, growth, block = kv_bar - p, p, max(p, min(wl.B, kv_bar))      # cap = kv_bar
    elif arm == "ed":
        kv_max, growth = wl.s, max(1, kv_bar - 1)                              # prompt, then <= kv_bar pairs
    elif arm == "fkv":
        kv_max, growth = wl.s, max(1, wl.steps)
    else:
        raise ValueError(arm)
    return Config(batch=batch, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.d, kv_max=kv_max, block_max=block,
                  growth=growth, dtype=wl.dtype, n_layers=wl.L, device=device,
                  max_call_samples=max(micro, min(batch, DECODE_MICRO)),
                  compaction="stable" if arm == "ed" else compaction)    # Algorithm 3's cut ranks rows by their order


def arm_calls(wl: Workload, arm: str, kv_bar: int | None = None, p: int = 64):
    """Calls of one layer as (kind, pos0, I, arg): kind in prefill / decode (arg = evict_to, -1 for none),
    evict (arg = target), recent (arg = pairs kept)."""
    calls, n = [], 0
    if arm == "alg1":
        # first min(s, kv_bar) tokens without eviction (any split gives the same result), then p out, <= p in
        t1 = min(wl.s, kv_bar)
        blk = max(p, min(wl.B, kv_bar))
        for pos0 in range(0, t1, blk):
            calls.append(("prefill", pos0, min(blk, t1 - pos0), -1))
        n = t1
        while t1 < wl.s:
            calls.append(("evict", 0, 0, n - p))
            I = min(p, wl.s - t1)
            calls.append(("prefill", t1, I, -1))
            n, t1 = n - p + I, t1 + I
        for t in range(wl.steps):
            if n == kv_bar:
                calls.append(("evict", 0, 0, n - p))
                n -= p
            calls.append(("decode", wl.s + t, 1, -1))
            n += 1
        return calls
    for pos0 in range(0, wl.s, wl.B):
        calls.append(("prefill", pos0, min(wl.B, wl.s - pos0), wl.K if arm == "pd" else -1))
    n = min(wl.s, wl.K) if arm == "pd" else wl.s
    if arm == "do":
        calls.append(("evict", 0, 0, wl.K))
        n = min(n, wl.K)
    if arm == "ed":
        calls.append(("recent", 0, 0, 1))
        n = 1
    for t in range(wl.steps):
        if arm in ("pd", "do"):
            full = n + 1 >= wl.K + wl.p_dec
            calls.append(("decode", wl.s + t, 1, wl.K if full else -1))
            n = wl.K if full else n + 1
        else:
            calls.append(("decode", wl.s + t, 1, -1))
            n += 1
            if arm == "ed" and n == kv_bar:
                calls.append(("recent", 0, 0, 1))
                n = 1
    return calls


GRAPH_DECODE_INPUT_BYTES = 256 << 20


def _decode_phase_as_graph(cache, inp, calls, layer, n, out_dec):
    """Captures the calls of a decode phase (decode steps and the cuts between them) on the whole batch in one CUDA
    graph, replays it once between two events; returns (ms, cached pairs at the end, rows read by the decode steps)."""
    ins = []
    for kind, pos0, I, arg in calls:
        if kind == "decode":
            q, k, v = inp.block(layer, pos0, 1)
            ins.append((q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous()))
    rows = 0
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        it = iter(ins)
        for kind, pos0, I, arg in calls:
            if kind == "decode":
                q, k, v = next(it)
                cache.decode_step(q, k, v, out=out_dec[:q.shape[0]], evict_to=arg, layer=layer)
                rows += n + 1
                n = n + 1 if arg < 0 else min(n + 1, arg)
            else:
                assert kind in ("evict", "recent"), kind
                (cache.evict if kind == "evict" else cache.keep_most_recent)(arg, layer=layer)
                n = min(n, arg)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record()
        graph.replay()
        e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1), n, rows


class Timer:
    def __init__(self):
        self.pairs = []

    def __call__(self, fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        self.pairs.append((e0, e1))

    def total_ms(self):
        torch.cuda.synchronize()
        t = sum(a.elapsed_time(b) for a, b in self.pairs)
        self.pairs = []
        return t


def run_arm(wl: Workload, batch: int, arm: str, micro: int, arena=None, layers=None, device: int = 0,
            kv_bar: int | None = None, p: int = 64, compaction: str = "stable"):
    """One arm (see ARMS) over the whole schedule.  Returns a dict of timings and derived rates."""
    wl = wl.with_(b=batch)
    cfg = make_cfg(wl, batch, arm, micro, device, kv_bar, p, compaction)
    dev = torch.device("cuda", device)
    need = arena_bytes(cfg)
    if arena is None:
        arena = torch.empty(need, dtype=torch.uint8, device=dev)
    assert arena.numel() >= need, "arena smaller than the memory model asks for"
    cache = BatchMaxCache(cfg, arena=arena[:need])
    cache.count_moved_rows(True)
    inp = Inputs(wl, dev)
    t_pre, t_dec = Timer(), Timer()
    moved_pre = None
    ms_pre = ms_dec = 0.0
    layers = range(wl.L) if layers is None else layers
    out_flat = torch.empty(micro * cfg.block_max * wl.Hq * wl.d, dtype=wl.torch_dtype, device=dev)

    def out_blk(ns, I):     # a contiguous (ns, I, Hq, d) view: the library writes the output with q's layout
        return out_flat[:ns * I * wl.Hq * wl.d].view(ns, I, wl.Hq, wl.d)
    micro_dec = max(micro, min(batch, DECODE_MICRO))
    out_dec = torch.empty(micro_dec, wl.Hq, wl.d, dtype=wl.torch_dtype, device=dev)
    calls = arm_calls(wl, arm, kv_bar, p)
    pairs = dec_rows = 0
    # a small batch decodes in steps of a few tens of microseconds, which eager launches from Python cannot feed: its
    # decode phase (every call from the first decode step on) is captured once in a CUDA graph and replayed
    e_in = (wl.Hq + 2 * wl.Hkv) * wl.d * wl.elem_bytes
    graph_decode = batch <= micro_dec and wl.steps * batch * e_in <= GRAPH_DECODE_INPUT_BYTES
    for layer in layers:
        n, in_decode, pending = 0, False, 0
        for ci, (kind, pos0, I, arg) in enumerate(calls):
            if kind == "decode" and not in_decode:
                moved_pre = cache.moved_rows(reset=True)
                if graph_decode:
                    ms, n, rows = _decode_phase_as_graph(cache, inp, calls[ci:], layer, n, out_dec)
                    ms_dec += ms
                    dec_rows += rows
                    break
            in_decode = in_decode or kind == "decode"
            timer = t_dec if in_decode else t_pre
            if kind == "prefill":
                for s0 in range(0, batch, micro):
                    ns = min(micro, batch - s0)
                    q, k, v = inp.block(layer, pos0, I, s0, ns)
                    timer(lambda: cache.prefill_block(q, k, v, pos0, out=out_blk(ns, I), evict_to=arg, layer=layer,
                                                      sample0=s0))
                pairs += I * n + I * (I + 1) // 2
                n = n + I if arg < 0 else min(n + I, arg)
            elif kind == "decode":
                # one token per sample is small: the step's inputs are drawn for the whole batch first, then the calls
                # of all sample ranges run back to back inside one timed region
                q, k, v = inp.block(layer, pos0, 1)
                q, k, v = q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous()

                def step_calls():
                    for s0 in range(0, batch, micro_dec):
                        ns = min(micro_dec, batch - s0)
                        cache.decode_step(q[s0:s0 + ns], k[s0:s0 + ns], v[s0:s0 + ns], out=out_dec[:ns], evict_to=arg,
                                          layer=layer, sample0=s0)
                timer(step_calls)
                dec_rows += n + 1
                n = n + 1 if arg < 0 else min(n + 1, arg)
            else:
                rule = cache.evict if kind == "evict" else cache.keep_most_recent
                step = micro_dec if in_decode else micro
                for s0 in range(0, batch, step):
                    ns = min(step, batch - s0)
                    timer(lambda: rule(arg, layer=layer, sample0=s0, nsamples=ns))
                n = min(n, arg)
            pending += 1
            if pending >= 16:
                ms_pre += t_pre.total_ms()
                ms_dec += t_dec.total_ms()
                pending = 0
        ms_pre += t_pre.total_ms()
        ms_dec += t_dec.total_ms()
    assert cache.status() == 0
    moved_dec = cache.moved_rows(reset=True)
    if moved_pre is None:
        moved_pre, moved_dec = moved_dec, 0
    n_layers = len(list(layers))
    n_end, cur = cache.length(layer=list(layers)[-1], sample=batch - 1)
    assert n_end == n, "host mirror disagrees with the schedule's own count"
    cache.close()
    hbm, tf, src = peaks()
    e = wl.elem_bytes
    flops = 4.0 * wl.d * (pairs / n_layers) * batch * wl.Hq * n_layers
    dec_bytes = batch * wl.Hkv * n_layers * ((dec_rows / n_layers) * (2 * wl.d * e + 16)
                                             + wl.steps * (2 * wl.d * e + 2 * wl.g * wl.d * e))
    res = {
        "workload": wl.name, "arm": arm, "compaction": cfg.compaction, "batch": batch, "layers_run": n_layers, "micro_batch": micro,
        "decode_micro_batch": micro_dec, "cap": cfg.kv_max + cfg.growth,
        "arena_GiB": need / GiB, "final_n": n_end, "final_curr_id": cur,
        "prefill_ms": ms_pre, "decode_ms": ms_dec,
        "prefill_tok_s": batch * wl.s * n_layers / (ms_pre * 1e-3),
        "decode_tok_s": batch * wl.steps * n_layers / (ms_dec * 1e-3) if ms_dec > 0 else None,
        "generated_tok_s": batch * wl.steps * n_layers / ((ms_pre + ms_dec) * 1e-3),
        "prefill_useful_tflops": flops / (ms_pre * 1e-3) / 1e12,
        "prefill_frac_of_peak": flops / (ms_pre * 1e-3) / 1e12 / tf,
        "decode_gbs": dec_bytes / (ms_dec * 1e-3) / 1e9 if ms_dec > 0 else None,
        "decode_frac_of_peak": dec_bytes / (ms_dec * 1e-3) / 1e9 / hbm if ms_dec > 0 else None,
        "decode_rows_moved": moved_dec, "prefill_rows_moved": moved_pre,
        "decode_gbs_with_moves": (dec_bytes + moved_dec * 2.0 * wl.d * e) / (ms_dec * 1e-3) / 1e9 if ms_dec > 0 else None,
        "decode_frac_with_moves": (dec_bytes + moved_dec * 2.0 * wl.d * e) / (ms_dec * 1e-3) / 1e9 / hbm
        if ms_dec > 0 else None,
        "peaks": {"hbm_gbs": hbm, "bf16_tflops_sustained": tf, "source": src},
        "note": "prefill = every call before the first decode step (attention, score pass, evictions; the whole call, "
                "not the forward kernel alone); decode = every call from the first decode step on; decode bytes "
                "exclude compaction moves; every prefill call and every decode step (all its sample ranges) timed with its own "
                "CUDA events" + ("; the decode phase of this small batch is one CUDA graph, replayed once between two events"
                                 if graph_decode else ""),
    }
    if arm in ("alg1", "ed"):
        res["kv_bar"] = kv_bar
    if arm == "alg1":
        res["p"] = p
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--run", required=True, choices=["cfg3_max", "cfg3_ratio", "cfg4", "cfg5", "sec4"])
    ap.add_argument("--budget-gib", type=float, default=None)
    ap.add_argument("--micro", type=int, default=256)
    ap.add_argument("--layers", type=int, default=None, help="run only the first N layers (cfg4)")
    ap.add_argument("--decode-steps", type=int, default=None)
    ap.add_argument("--compaction", default="stable", choices=["stable", "fill"],
                    help="fill: unordered caches (pairs that stay never move); Algorithm 3's arm always runs ordered")
    args = ap.parse_args()
    assert torch.cuda.is_available(), "needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(0)
    if args.run in ("cfg3_max", "cfg3_ratio"):
        wl = WORKLOADS["cfg3"]
        if args.decode_steps is not None:
            wl = wl.with_(steps=args.decode_steps)
        budget = int((args.budget_gib or 40.0) * GiB)
        b_pd = max_batch(make_cfg(wl, 1, "pd", args.micro), budget)
        b_do = max_batch(make_cfg(wl, 1, "do", args.micro), budget)
        arena = torch.empty(budget, dtype=torch.uint8, device="cuda")
        res_pd = run_arm(wl, b_pd, "pd", args.micro, arena=arena, compaction=args.compaction)
        out = {"run": args.run, "budget_GiB": budget / GiB, "b_pd": b_pd, "b_do": b_do,
               "batch_ratio": b_pd / b_do, "predicted_ratio": (wl.s + 1) / (wl.K + 1), "pd": res_pd}
        if args.run == "cfg3_ratio":
            out["do"] = run_arm(wl, b_do, "do", min(args.micro, 64), arena=arena, compaction=args.compaction)
            out["generated_tok_s_ratio"] = out["pd"]["generated_tok_s"] / out["do"]["generated_tok_s"]
        print(json.dumps(out))
    elif args.run == "cfg4":
        wl = WORKLOADS["cfg4"]
        if args.decode_steps is not None:
            wl = wl.with_(steps=args.decode_steps)
        budget = int((args.budget_gib or 120.0) * GiB)
        b = max_batch(make_cfg(wl, 1, "pd", args.micro), budget)
        arena = torch.empty(budget, dtype=torch.uint8, device="cuda")
        layers = range(wl.L) if args.layers is None else range(args.layers)
        res = run_arm(wl, b, "pd", args.micro, arena=arena, layers=layers, compaction=args.compaction)
        print(json.dumps({"run": "cfg4", "budget_GiB": budget / GiB, "batch": b, "pd": res}))
    elif args.run == "sec4":
        # The procedure of Sec. 4 on one attention layer of the larger model's shape (40 heads of 128, prompt
        # 3584, 512 tokens generated = 511 decode forwards): every arm runs at the largest batch whose caches
        # fit the same budget.  Only cache memory is modelled, so the batch ratios are those of the caches alone.
        wl = Workload("sec4", b=1, Hq=40, Hkv=40, d=128, dtype="bf16", s=3584, B=512, K=1024,
                      steps=args.decode_steps if args.decode_steps is not None else 511, seed=5, heavy_count=36)
        budget = int((args.budget_gib or 4.0) * GiB)
        arena = torch.empty(budget, dtype=torch.uint8, device="cuda")
        arms = [("alg1", 1024), ("alg1", 2048), ("ed", 2), ("ed", 65), ("fkv", None)]
        for arm, kv_bar in arms:
            b = max_batch(make_cfg(wl, 1, arm, args.micro, kv_bar=kv_bar), budget)
            res = run_arm(wl, b, arm, min(args.micro, b), arena=arena, kv_bar=kv_bar, compaction=args.compaction)
            print(json.dumps({"run": "sec4", "budget_GiB": budget / GiB, "arm": arm, "kv_bar": kv_bar, "batch": b,
                              "result": res}), flush=True)
    else:
        for B, K in CFG5_SWEEP:
            wl = WORKLOADS["cfg5"].with_(B=B, K=K, name=f"cfg5_B{B}_K{K}")
            if args.decode_steps is not None:
                wl = wl.with_(steps=args.decode_steps)
            res = run_arm(wl, wl.b, "pd", wl.b, compaction=args.compaction)
            print(json.dumps({"run": "cfg5", "block": B, "kv_max": K, "pd": res}), flush=True)


if __name__ == "__main__":
    main()
