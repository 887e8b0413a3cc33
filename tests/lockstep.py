"""Lock-step parity driver: runs a workload's schedule through the C-ABI library on the GPU and through the
fp64 oracle on the same input bits, call by call, for a chosen set of (sample, kv-head) caches.

Free-running comparison is meaningless after the first near-tie (one flipped choice changes every later kept
set), so after each call the GPU's kept ids are checked against the oracle's *own* ranking:
  - every candidate whose ave_weights is above cut*(1+band) must be kept, none below cut*(1-band) may be,
    the kept count equals the target and ids ascend;
  - if the sets differ only inside the band, the oracle adopts the GPU's set (keeping its own fp64 sums)
    and the adoption is counted.
Outputs are compared on every call, sum_weights after every call, and cached K/V rows bit for bit.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import UnitCache
from paper_2412_05693_b200 import BatchMaxCache, Config
from paper_2412_05693_b200.workloads import Inputs, Workload, config_for, schedule

BAND = 1e-4   # relative band around the cut inside which kept sets may differ
OUT_TOL = {"bf16": 2e-2, "f32": 1e-4}


def make_config(wl: Workload, device: int = 0, growth: int | None = None, batch: int | None = None,
                max_call_samples: int = 0, rule: str = "average", compaction: str = "stable", **rule_params) -> Config:
    return config_for(wl, device, growth, batch, max_call_samples, rule, compaction, **rule_params)


def _np(t):
    return t.detach().to(torch.float64).cpu().numpy()


def check_kept(unit: UnitCache, gpu_ids: np.ndarray, target: int, stats: dict, where: str):
    """Band check of the GPU's kept set against the oracle's ranking; the oracle then evicts (adopting the
    GPU's set when it differs inside the band)."""
    if target == 0:                               # everything leaves: nothing to rank
        assert len(gpu_ids) == 0, f"{where}: {len(gpu_ids)} pairs kept, target 0"
        unit.evict(0)
        stats["evictions"] += 1
        return
    ave = unit.ranking_scores(target)             # ave_weights under the paper's rule
    cand = unit.kv_ids
    is_pad = cand < unit.left_pad                 # padding pairs of a left-padded sample rank after every real pair
    order = np.lexsort((cand, -ave, is_pad))
    n_real = int((~is_pad).sum())
    gpu = np.asarray(gpu_ids, dtype=np.int64)
    assert gpu.shape[0] == target, f"{where}: kept {gpu.shape[0]} != target {target}"
    assert np.all(np.diff(gpu) > 0), f"{where}: kept ids not ascending"
    in_cand = np.isin(gpu, cand)
    assert in_cand.all(), f"{where}: kept ids that were never candidates: {gpu[~in_cand][:8]}"
    kept_mask = np.isin(cand, gpu)
    if target <= n_real:                          # the cut falls among the real pairs; all padding leaves
        cut = ave[order[target - 1]]
        must_keep = ~is_pad & (ave > cut * (1 + BAND))
        must_drop = is_pad | (ave < cut * (1 - BAND))
    else:                                         # every real pair stays, with the lowest padding positions
        lowest = np.zeros_like(is_pad)
        lowest[order[n_real:target]] = True
        must_keep = ~is_pad | lowest
        must_drop = is_pad & ~lowest
    assert not np.any(must_keep & ~kept_mask), f"{where}: dropped a pair clearly above the cut"
    assert not np.any(must_drop & kept_mask), f"{where}: kept a pair clearly below the cut"
    own = cand[np.sort(order[:target])]
    if not np.array_equal(own, gpu):
        stats["adoptions"] += 1
    unit.evict(target, kept_ids=gpu)
    stats["evictions"] += 1


STD_BAND = 2e-3   # relative band around the deviation cut: sqrt(E[w^2] - E[w]^2) in fp32 loses digits to cancellation


def check_kept_average_std(unit: UnitCache, gpu_ids: np.ndarray, target: int, stats: dict, where: str):
    """The rule with pairs protected by the standard deviation of their weights (Sec. 2, RoCo): two cuts, so the
    band check has two stages.  A pair whose deviation is clearly above the deviation cut must be kept; a pair near
    that cut may have been chosen by either side; every other pair is judged by its average against the averages
    next to the average cut (one rank of slack, since a different choice at the first cut shifts the second by one)."""
    if target == 0:
        assert len(gpu_ids) == 0
        unit.evict(0)
        stats["evictions"] += 1
        return
    cand = unit.kv_ids
    gpu = np.asarray(gpu_ids, dtype=np.int64)
    assert gpu.shape[0] == target and np.all(np.diff(gpu) > 0) and np.isin(gpu, cand).all(), f"{where}: bad kept set"
    ave = unit.ave_weights()
    cnt = unit.g * (unit.last_pos + 1 - cand)
    std = np.sqrt(np.maximum(unit.sum_sq / cnt - ave * ave, 0.0))
    n_std = int(np.floor(unit.std_share * target + 1e-9))
    kept = np.isin(cand, gpu)
    near = np.zeros(len(cand), dtype=bool)
    sure = np.zeros(len(cand), dtype=bool)
    if n_std > 0:
        cut_s = np.sort(std)[::-1][n_std - 1]
        sure = std > cut_s * (1 + STD_BAND)
        near = (std >= cut_s * (1 - STD_BAND)) & ~sure
        assert not np.any(sure & ~kept), f"{where}: dropped a pair whose deviation is clearly above the cut"
    score = unit.ranking_scores(target)                       # the oracle's own choice: protected pairs at +inf
    order = np.lexsort((cand, -score))
    rest = order[n_std:]                                      # by average, best first
    k = target - n_std                                        # pairs chosen by average
    if 0 < k < len(rest):
        hi = ave[rest[max(k - 2, 0)]]                         # one rank better than the last pair chosen by average
        lo = ave[rest[min(k + 1, len(rest) - 1)]]             # one rank worse than the first pair not chosen
        judged = ~sure & ~near
        assert not np.any(judged & ~kept & (ave > hi * (1 + BAND))), f"{where}: dropped a pair clearly above the average cut"
        assert not np.any(judged & kept & (ave < lo * (1 - BAND))), f"{where}: kept a pair clearly below the average cut"
    own = cand[np.sort(order[:target])]
    if not np.array_equal(own, gpu):
        stats["adoptions"] += 1
    unit.evict(target, kept_ids=gpu)
    stats["evictions"] += 1


def run_lockstep(wl: Workload, units, device: int = 0, layer: int = 0, calls=None, check_rows_every: int = 8,
                 growth: int | None = None, sum_rtol: float | None = None, pads=None, rule: str = "average",
                 compaction: str = "stable", micro: int | None = None, micro_dec: int | None = None, arena=None,
                 cache=None, rule_params: dict | None = None):
    """Run `calls` (default: the workload's spec schedule) on the GPU for the whole batch and on the
    oracle for `units` = [(sample, kv_head), ...].  Returns a dict of statistics; raises on any mismatch.

    `micro` / `micro_dec`: issue every prefill / decode call range by range (`sample0, nsamples`) with that many
    samples per call, drawing each range's inputs on the fly -- the call pattern of batches whose prompts cannot
    be resident at once; only the sampled units' slices of q/k/v/out are kept for the oracle.  `arena`: a caller-
    owned byte tensor the cache is built in.  `cache`: an existing handle to run on (it is left open)."""
    dev = torch.device("cuda", device)
    inp = Inputs(wl, dev)
    own_cache = cache is None
    if own_cache:
        mc = 0 if micro is None else max(micro, micro_dec or micro)
        cfg = make_config(wl, device, growth, rule=rule, compaction=compaction, max_call_samples=min(mc, wl.b),
                          **(rule_params or {}))
        cache = BatchMaxCache(cfg, arena=arena)
    if pads is not None:                            # left-padded samples: pads[sample] padding positions
        cache.set_left_pad(pads)
    g = wl.g
    oracles = {u: UnitCache(wl.d, g, left_pad=0 if pads is None else pads[u[0]], rule=rule, **(rule_params or {}))
               for u in units}
    stats = {"adoptions": 0, "evictions": 0, "max_out_err": 0.0, "max_sum_rel": 0.0, "calls": 0, "tc_calls": 0,
             "onepass_calls": 0}
    tol = OUT_TOL[wl.dtype]
    sum_rtol = sum_rtol if sum_rtol is not None else (2e-3 if wl.dtype == "bf16" else 2e-4)
    calls = schedule(wl) if calls is None else calls
    from paper_2412_05693_b200 import last_prefill_path

    def issue(kind, pos0, I, evict_to):
        """One call of the schedule on the whole batch; returns {unit: (q, k, v, out)} as fp64 arrays."""
        step = wl.b if micro is None else (micro if kind == "prefill" else (micro_dec or micro))
        got = {}
        for s0 in range(0, wl.b, step):
            ns = min(step, wl.b - s0)
            if kind == "evict":
                cache.evict(evict_to, layer=layer, sample0=s0, nsamples=ns)
                continue
            if kind == "recent":                    # Algorithm 3's rule; `evict_to` pairs stay
                cache.keep_most_recent(evict_to, layer=layer, sample0=s0, nsamples=ns)
                continue
            q, k, v = inp.block(layer, pos0, I, s0, ns)
            if kind == "prefill":
                out = cache.prefill_block(q, k, v, pos0, evict_to=evict_to, layer=layer, sample0=s0)
                stats["tc_calls"] += 1 if last_prefill_path() > 0 else 0
                stats["onepass_calls"] += 1 if last_prefill_path() == 2 else 0
            else:
                out = cache.decode_step(q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous(),
                                        evict_to=evict_to, layer=layer, sample0=s0)[:, None]
            for (smp, kh) in oracles:
                if s0 <= smp < s0 + ns:
                    r = smp - s0
                    got[(smp, kh)] = (_np(q[r, :, kh * g:(kh + 1) * g]), _np(k[r, :, kh]), _np(v[r, :, kh]),
                                      _np(out[r, :, kh * g:(kh + 1) * g]))
        return got

    for ci, (kind, pos0, I, evict_to) in enumerate(calls):
        got = issue(kind, pos0, I, evict_to)
        torch.cuda.synchronize(dev)
        assert cache.status() == 0
        stats["calls"] += 1
        for (smp, kh), unit in oracles.items():
            where = f"call {ci} ({kind} pos0={pos0} I={I}) unit ({smp},{kh})"
            if kind == "recent":
                unit.keep_most_recent(evict_to)
            elif kind != "evict":
                uq, uk, uv, uo = got[(smp, kh)]
                ref = unit.process_block(uq, uk, uv, pos0, -1)
                err = float(np.abs(uo - ref).max())
                stats["max_out_err"] = max(stats["max_out_err"], err)
                assert err <= tol, f"{where}: output max-abs error {err:.3e} > {tol}"
            want_rows = (ci % check_rows_every == 0) or ci == len(calls) - 1
            ids, sw, kr, vr = cache.export(layer, smp, kh, rows=want_rows)
            ids = ids.numpy().astype(np.int64)
            if compaction == "fill":                # an unordered cache exports its rows in storage order
                order = np.argsort(ids, kind="stable")
                assert len(np.unique(ids)) == len(ids), f"{where}: a position is cached twice"
                ids, sw = ids[order], sw[torch.from_numpy(order)]
                if want_rows:
                    kr, vr = kr[torch.from_numpy(order)], vr[torch.from_numpy(order)]
            if kind != "recent" and evict_to >= 0 and len(unit) > evict_to:
                if rule == "average_std":
                    check_kept_average_std(unit, ids, evict_to, stats, where)
                else:
                    check_kept(unit, ids, evict_to, stats, where)
            assert np.array_equal(ids, unit.kv_ids), f"{where}: kv_ids differ from the oracle's"
            n_gpu, cur = cache.length(layer, smp)
            assert n_gpu == len(unit) and cur == unit.last_pos, f"{where}: host mirror n/curr_id wrong"
            sw = sw.numpy().astype(np.float64)
            rel = float(np.max(np.abs(sw - unit.sum_weights) / np.maximum(np.abs(unit.sum_weights), 1e-3))) \
                if len(unit) else 0.0              # (an eviction call on a still-empty cache is legal)
            stats["max_sum_rel"] = max(stats["max_sum_rel"], rel)
            assert rel <= sum_rtol, f"{where}: sum_weights relative error {rel:.3e} > {sum_rtol}"
            if rule == "average_std" and len(unit):
                sq = cache.export_sum_sq(layer, smp, kh).numpy().astype(np.float64)
                rel = float(np.max(np.abs(sq - unit.sum_sq) / np.maximum(np.abs(unit.sum_sq), 1e-4)))
                assert rel <= sum_rtol, f"{where}: sums of squared weights off by {rel:.3e} > {sum_rtol}"
            if want_rows:
                assert np.array_equal(_np(kr), unit.k), f"{where}: cached K rows are not the oracle's rows"
                assert np.array_equal(_np(vr), unit.v), f"{where}: cached V rows are not the oracle's rows"
    from paper_2412_05693_b200 import debug_build
    if debug_build():                               # the checked build: no guard behind a slab was written over
        assert cache.check_canaries() == 0, "a guard behind one of the arena's slabs was damaged"
    if own_cache:
        cache.close()
    return stats
