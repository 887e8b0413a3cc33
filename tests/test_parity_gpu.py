"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle in lock-step on the same
seeded inputs.  Kept sets bit-exact outside a 1e-4 relative band around the cut, outputs within 2e-2 (bf16) /
1e-4 (fp32) max-abs, cached rows bit-exact."""
import numpy as np
import pytest
import torch

import paper_2412_05693_b200 as bm
from paper_2412_05693_b200.workloads import CFG5_SWEEP, WORKLOADS, Inputs, Workload, schedule
from tests.lockstep import make_config, run_lockstep

pytestmark = pytest.mark.gpu


def all_units(wl, samples=None):
    samples = range(wl.b) if samples is None else samples
    return [(s, h) for s in samples for h in range(wl.Hkv)]


def tiny(name, **kw):
    base = dict(b=2, Hq=4, Hkv=2, d=64, dtype="f32", s=200, B=48, K=40, steps=6, seed=123, heavy_count=4)
    base.update(kw)
    return Workload(name, **base)


# ------------------------------------------------------------------ configs of the benchmark table
def test_cfg1_everything():
    wl = WORKLOADS["cfg1"]
    st = run_lockstep(wl, all_units(wl), check_rows_every=1)
    assert st["evictions"] >= (6 + 16) * 8
    assert st["max_out_err"] <= 1e-4


@pytest.mark.parametrize("compaction", ["stable", "fill"])
def test_cfg2_full_size_sampled_units(compaction):
    wl = WORKLOADS["cfg2"]
    st = run_lockstep(wl, [(0, 0), (7, 3), (15, 7)], check_rows_every=16, compaction=compaction)
    assert st["evictions"] > 0 and st["max_out_err"] <= 2e-2


@pytest.mark.parametrize("compaction", ["stable", "fill"])
def test_cfg3_full_size_sampled_units(compaction):
    wl = WORKLOADS["cfg3"].with_(steps=8)
    run_lockstep(wl, [(3, 1), (12, 6)], check_rows_every=8, compaction=compaction)


def test_cfg3_decode_only_compression_arm():
    # whole prompt cached (cap = s + 1), one compression to K after the prompt, then decode (Sec. 1)
    wl = WORKLOADS["cfg3"].with_(b=2, s=2048, steps=4)
    calls = [("prefill", p, wl.B, -1) for p in range(0, wl.s, wl.B)] + [("evict", 0, 0, wl.K)]
    calls += [("decode", wl.s + t, 1, wl.K) for t in range(wl.steps)]
    run_lockstep(wl, [(0, 0), (1, 5)], calls=calls, growth=wl.s + 1 - wl.K)


def test_cfg4_layers_are_independent():
    wl = WORKLOADS["cfg4"].with_(b=2, L=3, s=2048, steps=3)
    for layer in (0, 2):
        run_lockstep(wl, [(1, 2)], layer=layer, check_rows_every=4)


@pytest.mark.parametrize("B,K", CFG5_SWEEP)      # all six (block, kv_max) pairs of the configuration
def test_cfg5_large_candidate_sets(B, K):
    wl = WORKLOADS["cfg5"].with_(b=2, B=B, K=K, s=8192, steps=4)
    run_lockstep(wl, [(1, 17)], check_rows_every=4)
    run_lockstep(wl, [(0, 30)], check_rows_every=4, compaction="fill")


def test_cfg5_full_length_prompt():
    # the largest candidate set of the table (2048 cached + 2048 new) at the full prompt length
    wl = WORKLOADS["cfg5"].with_(b=2, B=2048, K=2048, steps=2)
    run_lockstep(wl, [(0, 5)], check_rows_every=4)


def test_cfg4_all_32_layers_share_one_handle():
    wl = WORKLOADS["cfg4"].with_(b=2, s=1024, steps=2)
    for layer in (0, 17, 31):
        run_lockstep(wl, [(0, 0), (1, 7)], layer=layer, check_rows_every=2)


def random_workloads(n, seed=2024):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        g = int(rng.choice([1, 2, 4, 8]))
        hkv = int(rng.integers(1, 4))
        d = int(rng.choice([64, 128]))
        dtype = str(rng.choice(["bf16", "f32"]))
        B = int(rng.integers(1, 200))
        K = int(rng.integers(1, 300))
        s = int(rng.integers(1, 700))
        out.append(Workload(f"rand{i}_{dtype}_g{g}_d{d}_B{B}_K{K}_s{s}", b=int(rng.integers(1, 4)), Hq=g * hkv, Hkv=hkv,
                            d=d, dtype=dtype, s=s, B=B, K=K, steps=int(rng.integers(0, 12)), seed=1000 + i,
                            heavy_count=int(rng.integers(1, 9)), p_dec=int(rng.choice([1, 1, 3, 16]))))
    return out


@pytest.mark.parametrize("wl", random_workloads(10), ids=lambda w: w.name)
def test_random_shapes(wl):
    units = [(int(s), int(h)) for s in range(wl.b) for h in range(wl.Hkv)][:4]
    st = run_lockstep(wl, units, check_rows_every=2)
    assert st["calls"] == len(schedule(wl))


def random_cadence(wl, rng):
    """The workload's schedule with evictions switched off at random, explicit bm_evict / bm_keep_most_recent calls
    (targets from 0 up) thrown in, and an eviction forced wherever the cache would overflow."""
    growth = wl.B + 5
    calls, n = [], 0
    for kind, pos0, I, ev in schedule(wl):
        if n + I > wl.K + growth - 1 or rng.random() < 0.3:
            tgt = int(rng.integers(0, wl.K + 1))
            calls.append(("recent" if rng.random() < 0.3 else "evict", 0, 0, tgt))
            n = min(n, tgt)
        use_ev = ev if rng.random() < 0.5 else -1
        if use_ev < 0 and n + I > wl.K + growth:
            use_ev = wl.K
        calls.append((kind, pos0, I, use_ev))
        n = n + I if use_ev < 0 else min(n + I, use_ev)
    return calls, growth


@pytest.mark.parametrize("seed", range(8))
def test_random_cadences_rules_and_padding(seed):
    # seeded samples of the randomised sweep this suite was hardened with: any cadence of the four calls, any rule,
    # left padding, evictions down to an empty cache
    rng = np.random.default_rng(4200 + seed)
    g, hkv, d = int(rng.choice([1, 2, 4, 8])), int(rng.integers(1, 4)), int(rng.choice([64, 128]))
    wl = Workload(f"cad{seed}", b=int(rng.integers(1, 4)), Hq=g * hkv, Hkv=hkv, d=d, dtype=str(rng.choice(["bf16", "f32"])),
                  s=int(rng.integers(50, 900)), B=int(rng.integers(1, 300)), K=int(rng.integers(1, 400)),
                  steps=int(rng.integers(0, 16)), seed=4200 + seed, heavy_count=3, p_dec=int(rng.choice([1, 3])))
    rule = str(rng.choice(["average", "sum_recent", "current_query"]))
    if seed % 2 == 0:
        calls, growth = random_cadence(wl, rng)
        run_lockstep(wl, all_units(wl)[:3], calls=calls, growth=growth, rule=rule, check_rows_every=3)
    else:
        pads = [int(rng.integers(0, wl.s + 1)) for _ in range(wl.b)]
        run_lockstep(wl, all_units(wl)[:3], pads=pads, rule=rule, check_rows_every=3)


@pytest.mark.parametrize("seed", range(6))
def test_random_cadences_of_the_pooled_window_and_deviation_rules(seed):
    # the two rules with parameters of their own (Sec. 2: SnapKV, RoCo) under any cadence of the four calls
    rng = np.random.default_rng(5200 + seed)
    g, hkv, d = int(rng.choice([1, 2, 4])), int(rng.integers(1, 4)), int(rng.choice([64, 128]))
    wl = Workload(f"cad2_{seed}", b=int(rng.integers(1, 4)), Hq=g * hkv, Hkv=hkv, d=d, dtype=str(rng.choice(["bf16", "f32"])),
                  s=int(rng.integers(50, 700)), B=int(rng.integers(1, 250)), K=int(rng.integers(1, 300)),
                  steps=int(rng.integers(0, 12)), seed=5200 + seed, heavy_count=3, p_dec=int(rng.choice([1, 3])))
    calls, growth = random_cadence(wl, rng)
    if seed % 2 == 0:
        params = dict(window=int(rng.integers(1, 80)), pool=int(rng.choice([1, 3, 5, 9])))
        run_lockstep(wl, all_units(wl)[:3], calls=calls, growth=growth, rule="window_pooled", rule_params=params,
                     check_rows_every=3)
    else:
        params = dict(std_share=float(rng.choice([0.1, 0.333, 0.5, 0.9])))
        run_lockstep(wl, all_units(wl)[:3], calls=calls, growth=growth, rule="average_std", rule_params=params,
                     check_rows_every=3)


# ------------------------------------------------------------------ shapes, tails and degenerate cases
@pytest.mark.parametrize("wl", [
    tiny("ragged_f32"),                                               # I = 48, tail of 8, g = 2
    tiny("gqa8_bf16", Hq=16, Hkv=2, dtype="bf16", d=128, B=50, K=70, s=333),
    tiny("mha_bf16_d64", Hq=3 * 1, Hkv=3, dtype="bf16", d=64, B=64, K=64, s=256),
    tiny("block_gt_cache", B=96, K=16, s=300),                        # B > K: no Algorithm-1 counterpart
    tiny("short_prompt", s=30, B=16, K=64, steps=40),                 # s < K: eviction starts in decode
    tiny("one_token_blocks", s=40, B=1, K=8, steps=3),
    tiny("keep_one", s=64, B=16, K=1, steps=5),
    tiny("f32_d128_g4", Hq=8, Hkv=2, d=128, B=40, K=100, s=260),
    tiny("decode_growth", p_dec=8, s=96, B=32, K=32, steps=30),       # evict every 8th step
], ids=lambda w: w.name)
def test_small_shapes(wl):
    st = run_lockstep(wl, all_units(wl), check_rows_every=1)
    assert st["calls"] == len(schedule(wl))


@pytest.mark.parametrize("d,g,B,K,s", [
    (128, 2, 64, 320, 900),      # Algorithm 1's p = 64 on a short cache: 3 cached + 1 new key tile, 128 query rows
    (128, 1, 64, 300, 700),      # half a tile of query rows, ragged cached tile
    (128, 4, 32, 384, 600),      # grouped heads: 32 inputs x 4 heads
    (64, 1, 128, 256, 640),      # d = 64, a whole tile of inputs, causal part spans the tile
    (64, 8, 16, 100, 333),       # g = 8, ragged everything
    (128, 4, 20, 50, 171),       # rows past the block's end (80 of 128) must add nothing to the column sums
])
def test_short_blocks_take_forward_and_column_sums_in_one_kernel(d, g, B, K, s):
    # one exponential per pair, logits resident in tensor memory (the single-pass variant for short caches)
    wl = tiny(f"onepass_d{d}_g{g}_B{B}_K{K}", dtype="bf16", d=d, Hq=2 * g, Hkv=2, B=B, K=K, s=s, steps=3, b=3)
    st = run_lockstep(wl, all_units(wl), check_rows_every=2)
    assert st["onepass_calls"] == len([c for c in schedule(wl) if c[0] == "prefill"])
    # the same rule with evictions made by explicit calls before each block (Algorithm 1's order), limit K + B
    calls = []
    n = 0
    for kind, pos0, I, ev in schedule(wl):
        if n + I > K + B:                     # (a decode step is a block of one input)
            calls.append(("evict", 0, 0, K))
            n = K
        calls.append((kind, pos0, I, -1 if kind == "prefill" else ev))
        n = n + I if kind == "prefill" else min(n + 1, K)
    st = run_lockstep(wl, all_units(wl)[:3], calls=calls, growth=B, check_rows_every=2)
    assert st["onepass_calls"] > 0


def test_algorithm1_cadence_on_gpu():
    # Algorithm 1 as printed: limit kv_bar, remove p before each block / when full during decoding
    kv_bar, p, s, gen = 96, 32, 288, 70
    wl = tiny("alg1", s=s, B=p, K=kv_bar - p, steps=gen, p_dec=p, dtype="bf16", d=128, Hq=8, Hkv=2)
    calls = [("prefill", t, p, -1) for t in range(0, kv_bar, p)]
    t1 = kv_bar
    while t1 < s:
        calls.append(("evict", 0, 0, kv_bar - p))
        calls.append(("prefill", t1, min(p, s - t1), -1))
        t1 += p
    n = kv_bar
    for t in range(gen):
        if n == kv_bar:
            calls.append(("evict", 0, 0, kv_bar - p))
            n -= p
        calls.append(("decode", s + t, 1, -1))
        n += 1
    run_lockstep(wl, all_units(wl), calls=calls, growth=p, check_rows_every=3)


@pytest.mark.parametrize("dtype,d,kv_bar", [("bf16", 128, 2), ("bf16", 128, 65), ("f32", 64, 5)])
def test_extreme_decoding_arm_on_gpu(dtype, d, kv_bar):
    # Algorithm 3: full cache during the prompt, then only the most recent pair survives each cut
    s, gen = 200, 70
    wl = tiny("ed", s=s, B=48, K=s, steps=gen, dtype=dtype, d=d, Hq=8, Hkv=2)
    calls = [("prefill", t, min(48, s - t), -1) for t in range(0, s, 48)] + [("recent", 0, 0, 1)]
    n = 1
    for t in range(gen):
        calls.append(("decode", s + t, 1, -1))
        n += 1
        if n == kv_bar:
            calls.append(("recent", 0, 0, 1))
            n = 1
    st = run_lockstep(wl, all_units(wl), calls=calls, growth=kv_bar, check_rows_every=5)
    assert st["calls"] == len(calls)


@pytest.mark.parametrize("g", [1, 4])
def test_decode_with_more_caches_than_two_ctas_per_sm(g):
    # 320 caches: the decode kernel takes its 128-thread shape (four CTAs per SM); fewer caches take the 256-thread one
    wl = tiny("many_units", b=40, Hq=8 * g, Hkv=8, s=160, B=64, K=72, steps=10, dtype="bf16", d=128)
    units = [(0, 0), (13, 5), (39, 7), (27, 2)]
    st = run_lockstep(wl, units, check_rows_every=2)
    assert st["evictions"] >= len(units) * 10


@pytest.mark.parametrize("K,g", [(511, 4), (512, 1), (600, 4), (639, 2), (640, 4)])
def test_decode_with_one_cache_per_sm(K, g):
    # few caches of at most 640 pairs: the decode kernel's instance that keeps K in registers and stages V by TMA
    # (rows behind the pair that leaves move up as TMA tiles, their first rows and a tail past the staged rows by
    # plain stores); 641 pairs fall back to the other instance
    wl = tiny("one_per_sm", b=3, Hq=2 * g, Hkv=2, s=K + 140, B=128, K=K, steps=14, dtype="bf16", d=128)
    st = run_lockstep(wl, all_units(wl), check_rows_every=1)
    assert st["evictions"] >= 6 * 14


# ------------------------------------------------------------------ unordered caches (BM_COMPACT_FILL)
@pytest.mark.parametrize("name,kw", [
    ("f32_simt", dict(dtype="f32", d=64, Hq=4, Hkv=4, s=300, B=48, K=80, steps=12)),
    ("bf16_one_per_sm", dict(dtype="bf16", d=128, Hq=8, Hkv=2, s=700, B=128, K=512, steps=14)),
    ("bf16_ragged_tail", dict(dtype="bf16", d=128, Hq=4, Hkv=4, s=333, B=100, K=77, steps=9)),
    ("bf16_block_larger_than_cache", dict(dtype="bf16", d=64, Hq=2, Hkv=2, s=400, B=160, K=48, steps=6)),
    ("bf16_decode_cuts_of_8", dict(dtype="bf16", d=128, Hq=8, Hkv=2, s=256, B=64, K=64, steps=20, p_dec=8)),
])
def test_unordered_cache_lockstep(name, kw):
    # same kept sets, sums and outputs as the ordered cache; rows compared after sorting the export by position
    wl = tiny("fill_" + name, **kw)
    st = run_lockstep(wl, all_units(wl), compaction="fill", check_rows_every=1)
    assert st["evictions"] > 0


def test_unordered_cache_many_units_decode():
    wl = tiny("fill_many", b=40, Hq=32, Hkv=8, s=160, B=64, K=72, steps=10, dtype="bf16", d=128)
    run_lockstep(wl, [(0, 0), (13, 5), (39, 7), (27, 2)], compaction="fill", check_rows_every=2)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_unordered_cache_breaks_ties_by_position(dtype, d):
    # A crafted state: rows in shuffled order, every sum_weights zero, one key (position 0) whose logit exceeds all
    # others by more than 1000, so that every other weight underflows to exactly 0 in fp32 and in fp64 alike.  All
    # those pairs tie at the cut; the lower positions must stay (select on kv_ids in the block eviction, arg-min on
    # kv_ids in the decode step), pairs that stay must not move, and every row must keep its own position.
    import torch
    from paper_2412_05693_b200 import BatchMaxCache
    from paper_2412_05693_b200.binding import Config
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    g, Hkv, K, n0 = 2, 2, 24, 32
    cfg = Config(batch=1, n_q_heads=g * Hkv, n_kv_heads=Hkv, head_dim=d, kv_max=K, block_max=32, growth=40,
                 dtype=dtype, compaction="fill")
    cache = BatchMaxCache(cfg)
    dev = torch.device("cuda", 0)
    gen = torch.Generator().manual_seed(5)
    rnd = lambda *shape: torch.randn(*shape, generator=gen).to(td).to(dev)
    cache.prefill_block(rnd(1, n0, g * Hkv, d), rnd(1, n0, Hkv, d), rnd(1, n0, Hkv, d), 0, evict_to=-1)
    perm = {}
    for h in range(Hkv):
        ids = torch.randperm(n0, generator=gen).to(torch.int32)
        perm[h] = ids.tolist()
        kr = torch.zeros(n0, d, dtype=td)
        kr[ids == 0] = 10.0
        vr = ids.to(td)[:, None].expand(n0, d).contiguous()      # a row's value is its position
        cache.import_(ids, torch.zeros(n0), kr, vr, sample=0, kv_head=h)

    def check(expect, before):
        for h in range(Hkv):
            ids, sw, kr, vr = cache.export(0, 0, h, rows=True)
            ids = ids.tolist()
            assert sorted(ids) == sorted(expect), f"head {h}: kept {sorted(ids)}, expected {sorted(expect)}"
            assert torch.equal(vr[:, 0].float(), torch.tensor(ids, dtype=torch.float32)), "a row lost its position"
            assert all(float(kr[r].float().abs().max()) == (10.0 if i in hot else 0.0) for r, i in enumerate(ids))
            for r, i in enumerate(before[h][:len(ids)]):
                if i in expect:
                    assert ids[r] == i, f"head {h}: pair {i} stayed but moved from row {r}"
            before[h] = ids

    hot = {0}
    q10 = lambda n: torch.full((1, n, g * Hkv, d), 10.0, dtype=td, device=dev)
    vpos = lambda p0, n: torch.arange(p0, p0 + n, dtype=torch.float32)[None, :, None, None].expand(1, n, Hkv, d).to(td).to(dev)
    # a block of 16: every pair but position 0 ties at zero -> positions 0..23 stay, the block's pairs all leave
    cache.prefill_block(q10(16), torch.zeros(1, 16, Hkv, d, dtype=td, device=dev), vpos(n0, 16).contiguous(), n0, evict_to=K)
    expect = list(range(K))
    check(expect, perm)
    # decode steps whose own key matches the query as well as position 0 does: the step's pair stays, and of the pairs
    # tied at zero the highest position leaves
    for t in range(6):
        pos = n0 + 16 + t
        cache.decode_step(q10(1)[:, 0].contiguous(), torch.full((1, Hkv, d), 10.0, dtype=td, device=dev),
                          vpos(pos, 1)[:, 0].contiguous(), evict_to=K)
        hot.add(pos)
        expect.remove(max(i for i in expect if i not in hot))
        expect.append(pos)
        check(expect, perm)
    assert cache.status() == 0
    cache.close()


@pytest.mark.parametrize("dtype,d,s,B,K,pads", [
    ("f32", 64, 200, 48, 40, [0, 37, 150]),
    ("bf16", 128, 600, 128, 160, [0, 301, 77]),     # cached padding scattered over the rows of several key tiles
    ("bf16", 128, 333, 100, 77, [5, 250, 0]),
    ("bf16", 64, 256, 64, 300, [0, 200, 64]),       # nothing leaves during the prompt: padding stays cached in decoding
])
def test_unordered_cache_left_padding(dtype, d, s, B, K, pads):
    # padding pairs are masked by their kv_ids wherever their rows are, and leave first
    wl = tiny("fill_pad", b=3, s=s, B=B, K=K, steps=8, dtype=dtype, d=d, Hq=8 if d == 128 else 4, Hkv=2)
    run_lockstep(wl, all_units(wl), pads=pads, compaction="fill", check_rows_every=2)
    run_lockstep(wl, all_units(wl), pads=pads, compaction="fill", rule="sum_recent", check_rows_every=4)


@pytest.mark.parametrize("rule", ["sum_recent", "current_query"])
@pytest.mark.parametrize("dtype,d,Hq,Hkv,p_dec", [("bf16", 128, 8, 2, 1), ("f32", 64, 4, 4, 1), ("bf16", 128, 8, 2, 8)])
def test_unordered_cache_alternative_rules(rule, dtype, d, Hq, Hkv, p_dec):
    # the window of recent pairs is a select on kv_ids here, in the block eviction and in the decode step alike
    wl = tiny("fill_rules", s=400, B=128, K=96, steps=12, dtype=dtype, d=d, Hq=Hq, Hkv=Hkv, p_dec=p_dec)
    run_lockstep(wl, all_units(wl), rule=rule, compaction="fill", check_rows_every=2)


@pytest.mark.parametrize("kv_bar", [2, 33])
def test_unordered_cache_extreme_decoding_arm(kv_bar):
    # Algorithm 3's cut keeps the highest positions, wherever their rows are
    s, gen = 200, 70
    wl = tiny("fill_ed", s=s, B=48, K=s, steps=gen, dtype="bf16", d=128, Hq=8, Hkv=2)
    calls = [("prefill", t, min(48, s - t), -1) for t in range(0, s, 48)] + [("recent", 0, 0, 1)]
    n = 1
    for t in range(gen):
        calls.append(("decode", s + t, 1, -1))
        n += 1
        if n == kv_bar:
            calls.append(("recent", 0, 0, 1))
            n = 1
    run_lockstep(wl, all_units(wl), calls=calls, growth=kv_bar, compaction="fill", check_rows_every=5)


@pytest.mark.parametrize("seed", range(6))
def test_unordered_cache_random_cadences(seed):
    rng = np.random.default_rng(9100 + seed)
    g, hkv, d = int(rng.choice([1, 2, 4, 8])), int(rng.integers(1, 4)), int(rng.choice([64, 128]))
    wl = Workload(f"fillcad{seed}", b=int(rng.integers(1, 4)), Hq=g * hkv, Hkv=hkv, d=d, dtype=str(rng.choice(["bf16", "f32"])),
                  s=int(rng.integers(50, 900)), B=int(rng.integers(1, 300)), K=int(rng.integers(1, 400)),
                  steps=int(rng.integers(0, 16)), seed=9100 + seed, heavy_count=3, p_dec=int(rng.choice([1, 3])))
    rule = str(rng.choice(["average", "sum_recent", "current_query"]))
    if seed % 2 == 0:
        calls, growth = random_cadence(wl, rng)     # prefill / decode / evict / recency cuts in any order
        run_lockstep(wl, all_units(wl)[:3], calls=calls, growth=growth, rule=rule, compaction="fill", check_rows_every=3)
    else:
        pads = [int(rng.integers(0, wl.s + 1)) for _ in range(wl.b)]
        run_lockstep(wl, all_units(wl)[:3], pads=pads, rule=rule, compaction="fill", check_rows_every=3)


# ------------------------------------------------------------------ the rules of Sec. 2 on the same kernels
@pytest.mark.parametrize("rule", ["sum_recent", "current_query"])
@pytest.mark.parametrize("dtype,d,Hq,Hkv", [("bf16", 128, 8, 2), ("f32", 64, 4, 4)])
def test_alternative_eviction_rules_lockstep(rule, dtype, d, Hq, Hkv):
    wl = tiny("rules", s=400, B=128, K=96, steps=12, dtype=dtype, d=d, Hq=Hq, Hkv=Hkv)
    st = run_lockstep(wl, all_units(wl), rule=rule, check_rows_every=2)
    assert st["evictions"] >= 2 * Hkv * (3 + 12)


@pytest.mark.parametrize("window,pool", [(1, 1), (8, 3), (16, 7), (64, 5)])
@pytest.mark.parametrize("dtype,d,Hq,Hkv,B,K", [("bf16", 128, 8, 2, 48, 40), ("f32", 64, 4, 4, 20, 33), ("bf16", 128, 4, 4, 160, 150)])
def test_window_pooled_rule_lockstep(window, pool, dtype, d, Hq, Hkv, B, K):
    # Sec. 2, SnapKV: sums over the last `window` queries of the pass, max-pooled over neighbours, recent window kept
    wl = tiny(f"snap_{dtype}_w{window}_p{pool}", dtype=dtype, d=d, Hq=Hq, Hkv=Hkv, s=3 * B + 7, B=B, K=K, steps=5)
    st = run_lockstep(wl, all_units(wl), rule="window_pooled", rule_params=dict(window=window, pool=pool),
                      check_rows_every=2)
    assert st["evictions"] > 0


def test_window_pooled_rule_one_compression_after_the_prompt():
    # the rule's own cadence (Sec. 2): nothing leaves during prefilling, one compression after the prompt
    wl = tiny("snap_once", dtype="bf16", d=128, Hq=8, Hkv=2, s=300, B=64, K=96, steps=4)
    calls = [("prefill", p, min(wl.B, wl.s - p), -1) for p in range(0, wl.s, wl.B)] + [("evict", 0, 0, wl.K)]
    calls += [("decode", wl.s + t, 1, -1) for t in range(wl.steps)]
    st = run_lockstep(wl, all_units(wl), calls=calls, growth=wl.s + wl.steps - wl.K, rule="window_pooled",
                      rule_params=dict(window=32, pool=7), check_rows_every=2)
    assert st["evictions"] == len(all_units(wl))


def test_window_pooled_rule_with_left_padding():
    wl = tiny("snap_pad", dtype="bf16", d=128, Hq=8, Hkv=2, s=200, B=40, K=48, steps=6)
    run_lockstep(wl, all_units(wl), pads=[0, 57], rule="window_pooled", rule_params=dict(window=8, pool=3),
                 check_rows_every=2)


@pytest.mark.parametrize("share", [0.0, 0.25, 0.5, 1.0])
@pytest.mark.parametrize("dtype,d,Hq,Hkv,B,K,p_dec", [("bf16", 128, 8, 2, 48, 40, 1), ("f32", 64, 4, 4, 20, 33, 1),
                                                       ("bf16", 128, 4, 4, 160, 150, 4)])
def test_average_std_rule_lockstep(share, dtype, d, Hq, Hkv, B, K, p_dec):
    # Sec. 2 / Sec. 3.2 last paragraph, RoCo: part of the kept pairs by the standard deviation of their weights
    wl = tiny(f"roco_{dtype}_{share}", dtype=dtype, d=d, Hq=Hq, Hkv=Hkv, s=3 * B + 7, B=B, K=K, steps=9, p_dec=p_dec)
    st = run_lockstep(wl, all_units(wl), rule="average_std", rule_params=dict(std_share=share), check_rows_every=2)
    assert st["evictions"] > 0


def test_rules_that_need_ordered_rows_refuse_unordered_caches_and_padding():
    wl = tiny("refuse", dtype="bf16", d=128)
    for rule in ("window_pooled", "average_std"):
        with pytest.raises(bm.BMError):
            bm.arena_bytes(make_config(wl, rule=rule, compaction="fill"))
    cache = bm.BatchMaxCache(make_config(wl, rule="average_std"))
    with pytest.raises(bm.BMError):
        cache.set_left_pad([0, 3])
    # the memory model charges the second accumulator: 4 more bytes per row
    a = bm.cache_bytes_per_sample(make_config(wl, rule="average_std"))
    b = bm.cache_bytes_per_sample(make_config(wl, rule="average"))
    assert a - b == 4 * wl.Hkv * (wl.K + 1)


def test_alternative_rule_with_left_padding():
    # first blocks entirely padding: the recent window holds padding, which still ranks last
    wl = tiny("rules_pad", b=3, s=320, B=64, K=40, steps=6, dtype="bf16", d=128, Hq=8, Hkv=2)
    run_lockstep(wl, all_units(wl), rule="sum_recent", pads=[0, 100, 300], check_rows_every=2)
    run_lockstep(wl, all_units(wl), rule="current_query", pads=[5, 64, 250], check_rows_every=2)


def test_alternative_rule_with_growth_falls_back_to_the_general_select():
    # decode evicts 8 pairs at a time: the fused arg-min does not apply, the select kernel ranks by the rule
    wl = tiny("rules_g", s=256, B=64, K=64, steps=20, p_dec=8, dtype="bf16", d=128, Hq=8, Hkv=2)
    run_lockstep(wl, all_units(wl), rule="sum_recent", check_rows_every=4)


# ------------------------------------------------------------------ left-padded samples (Sec. 3)
@pytest.mark.parametrize("dtype,d,s,B,K,pads", [
    ("f32", 64, 200, 48, 40, [0, 37, 150]),         # SIMT path; padding inside a block and over whole blocks
    ("bf16", 128, 640, 128, 160, [0, 70, 300]),     # tensor-core path; a whole 128-key tile of cached padding
    ("bf16", 128, 640, 256, 96, [5, 255, 256]),     # padding ending at / just before a block boundary
    ("bf16", 64, 300, 64, 64, [299, 1, 128]),       # one sample almost entirely padding
])
def test_left_padded_samples_lockstep(dtype, d, s, B, K, pads):
    wl = tiny("leftpad", b=3, s=s, B=B, K=K, steps=6, dtype=dtype, d=d, Hq=8, Hkv=2)
    st = run_lockstep(wl, all_units(wl), pads=pads, check_rows_every=2)
    assert st["evictions"] > 0
    if dtype == "bf16":
        assert st["tc_calls"] == -(-s // B)          # every prefill call took the tensor-core kernels


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_left_padding_still_cached_during_decoding(dtype, d):
    # prompt shorter than the limit: the padding is still cached when decoding starts, is masked there, and is
    # what the first evicting decode steps remove (highest padding position first)
    wl = tiny("leftpad_dec", b=3, s=50, B=32, K=60, steps=24, dtype=dtype, d=d, Hq=8, Hkv=2)
    st = run_lockstep(wl, all_units(wl), pads=[0, 7, 30], check_rows_every=3)
    assert st["evictions"] >= 3 * 2 * 10


def test_left_pad_setter_errors():
    wl = tiny("leftpad_err", dtype="bf16", d=128)
    cache = bm.BatchMaxCache(make_config(wl))
    with pytest.raises(bm.BMError) as e:
        cache.set_left_pad([0, -1])
    assert e.value.code == 1
    cache.set_left_pad([3, 0])
    cache.set_left_pad(None)
    q, k, v = Inputs(wl, "cuda").block(0, 0, 48)
    cache.prefill_block(q, k, v, 0, evict_to=wl.K)
    with pytest.raises(bm.BMError) as e:
        cache.set_left_pad([1, 1])                                       # only while every cache is empty
    assert e.value.code == 4
    cache.close()


def test_moved_row_counters_match_the_kept_sets():
    # rows a compaction moves = rows from the first one whose content changes to the end of the kept set
    wl = tiny("moved", b=2, s=192, B=64, K=40, steps=10, dtype="bf16", d=128, Hq=8, Hkv=2)
    cache = bm.BatchMaxCache(make_config(wl))
    cache.count_moved_rows(True)
    inp = Inputs(wl, "cuda")
    units = all_units(wl)
    before = {u: [] for u in units}
    expected = 0
    for kind, pos0, I, ev in schedule(wl):
        q, k, v = inp.block(0, pos0, I)
        if kind == "prefill":
            cache.prefill_block(q, k, v, pos0, evict_to=ev)
        else:
            cache.decode_step(q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous(), evict_to=ev)
        for u in units:
            ids = cache.export(0, u[0], u[1])[0].tolist()
            n_old = len(before[u])
            cand = before[u] + list(range(pos0, pos0 + I))
            evicted = len(ids) < len(cand)
            if kind == "prefill" or evicted:      # a decode step that only appends moves nothing
                first = next((r for r in range(len(ids)) if ids[r] != cand[r] or r >= n_old), len(ids))
                expected += len(ids) - first
            before[u] = ids
    assert cache.moved_rows() == expected
    assert cache.moved_rows(reset=True) == expected
    assert cache.moved_rows() == 0
    cache.close()


# ------------------------------------------------------------------ API behaviour on the device
def test_error_codes_and_state_tracking():
    wl = tiny("errors", dtype="bf16", d=128)
    cfg = make_config(wl)
    cache = bm.BatchMaxCache(cfg)
    inp = Inputs(wl, "cuda")
    q, k, v = inp.block(0, 0, 48)
    with pytest.raises(bm.BMError) as e:
        cache.prefill_block(q, k, v, 5)                                  # pos0 must follow curr_id
    assert e.value.code == 4
    q2 = torch.randn(2, 49, wl.Hq, wl.d, device="cuda").to(wl.torch_dtype)
    with pytest.raises(bm.BMError) as e:
        cache.prefill_block(q2, q2[:, :, :wl.Hkv].contiguous(), q2[:, :, :wl.Hkv].contiguous(), 0)
    assert e.value.code == 1                                             # I > block_max
    with pytest.raises(bm.BMError) as e:
        cache.evict(-3)
    assert e.value.code == 1
    cache.close()
    # capacity: appending without eviction beyond cap
    cache = bm.BatchMaxCache(cfg)
    cache.prefill_block(q, k, v, 0, evict_to=wl.K)
    q, k, v = inp.block(0, 48, 48)
    with pytest.raises(bm.BMError) as e:
        cache.prefill_block(q, k, v, 48, evict_to=-1)
    assert e.value.code == 3
    assert cache.length() == (wl.K, 47)                                  # failed call left the mirror alone
    # sample ranges with unequal n cannot share a call
    cache.prefill_block(q[:1], k[:1], v[:1], 48, evict_to=wl.K, sample0=0)
    with pytest.raises(bm.BMError) as e:
        cache.prefill_block(q, k, v, 48, evict_to=wl.K)
    assert e.value.code == 4
    cache.prefill_block(q[1:], k[1:], v[1:], 48, evict_to=wl.K, sample0=1)
    assert cache.length(sample=0) == cache.length(sample=1) == (wl.K, 95)
    assert cache.status() == 0
    cache.close()
    # more caches in one prefill call than the launch grid can index: refused before anything is enqueued
    big = bm.BatchMaxCache(bm.Config(batch=8200, n_q_heads=8, n_kv_heads=8, head_dim=64, kv_max=4, block_max=2, dtype="bf16"))
    qb = torch.zeros(8200, 1, 8, 64, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(bm.BMError) as e:
        big.prefill_block(qb, qb, qb, 0)
    assert e.value.code == 3
    big.prefill_block(qb[:4096], qb[:4096], qb[:4096], 0, sample0=0)
    big.prefill_block(qb[4096:], qb[4096:], qb[4096:], 0, sample0=4096)
    assert big.length(sample=8199) == (1, 0) and big.status() == 0
    big.close()


def test_bounded_wait_times_out_and_context_survives():
    # failure detection without a GPU fault: a wait that nothing satisfies gives up, the status word says so,
    # and the same handle keeps working afterwards
    wl = tiny("timeout", dtype="bf16", d=128, Hq=8, Hkv=2, s=96, B=48, K=40, steps=0)
    cache = bm.BatchMaxCache(make_config(wl))
    assert cache.status() == 0
    cache.selftest_wait_timeout()
    assert cache.status() == 6                     # BM_ERR_TIMEOUT
    cache.clear_status()
    assert cache.status() == 0
    cache.close()
    st = run_lockstep(wl, all_units(wl), check_rows_every=1)
    assert st["calls"] == 2


def run_free(wl, host=False, micro=None):
    """Whole schedule on the GPU only; returns final state and all outputs (for determinism / variants)."""
    cfg = make_config(wl)
    cache = bm.BatchMaxCache(cfg)
    inp = Inputs(wl, "cuda")
    outs, keep = [], []
    for kind, pos0, I, ev in schedule(wl):
        q, k, v = inp.block(0, pos0, I)
        if kind == "decode":
            q, k, v = q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous()
        if host and not (host == "mixed" and len(outs) % 2 == 1):
            qh, kh, vh = (t.cpu().pin_memory() for t in (q, k, v))
            oh = torch.empty_like(qh).pin_memory()
            if kind == "prefill":
                cache.prefill_block_host(qh, kh, vh, pos0, oh, evict_to=ev)
            else:
                cache.decode_step_host(qh, kh, vh, oh, evict_to=ev)
            if host is True:
                torch.cuda.synchronize()
                outs.append(oh.clone())
            else:               # calls stay in flight; only the caller's stream is synchronised at the end
                outs.append(oh)
                keep.append((qh, kh, vh))
        elif micro and kind == "prefill":
            o = torch.empty_like(q)
            for s0 in range(0, wl.b, micro):
                cache.prefill_block(q[s0:s0 + micro], k[s0:s0 + micro], v[s0:s0 + micro], pos0, out=o[s0:s0 + micro],
                                    evict_to=ev, sample0=s0)
            outs.append(o.cpu())
        elif micro:
            o = torch.empty_like(q)
            for s0 in range(0, wl.b, micro):
                cache.decode_step(q[s0:s0 + micro], k[s0:s0 + micro], v[s0:s0 + micro], out=o[s0:s0 + micro],
                                  evict_to=ev, sample0=s0)
            outs.append(o.cpu())
        else:
            o = cache.prefill_block(q, k, v, pos0, evict_to=ev) if kind == "prefill" else \
                cache.decode_step(q, k, v, evict_to=ev)
            outs.append(o if host else o.cpu())
    torch.cuda.current_stream().synchronize()
    outs = [o.cpu().clone() for o in outs]
    state = [cache.export(0, s, h, rows=True) for s in range(wl.b) for h in range(wl.Hkv)]
    cache.close()
    return outs, state


def assert_same_run(a, b):
    for x, y in zip(a[0], b[0]):
        assert torch.equal(x, y)
    for sa, sb in zip(a[1], b[1]):
        for x, y in zip(sa, sb):
            assert torch.equal(x, y)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_bitwise_reproducible_and_variants_agree(dtype, d):
    wl = tiny("repro", b=4, dtype=dtype, d=d, Hq=8, Hkv=2, s=256, B=64, K=64, steps=5)
    base = run_free(wl)
    assert_same_run(base, run_free(wl))                 # run-to-run determinism (no float atomics)
    assert_same_run(base, run_free(wl, host=True))      # host-fed entry points
    assert_same_run(base, run_free(wl, host="pipelined"))   # ... with every call left in flight
    assert_same_run(base, run_free(wl, host="mixed"))       # ... alternating with device-fed calls, no syncs
    assert_same_run(base, run_free(wl, micro=1))        # sample ranges: micro-batched calls


@pytest.mark.parametrize("which", ["tiny", "cfg2"])
def test_cuda_graph_replay_matches_eager_launches(which):
    # the benchmark replays one CUDA graph per step; a captured schedule must leave the same bits as eager launches
    # (which the lock-step tests hold against the oracle) -- also at the benchmark's own full size
    wl = tiny("graph", b=4, dtype="bf16", d=128, Hq=8, Hkv=2, s=256, B=64, K=64, steps=6) if which == "tiny" \
        else WORKLOADS["cfg2"]
    eager_outs, eager_state = run_free(wl)
    cfg = make_config(wl)
    inp = Inputs(wl, "cuda")
    calls = schedule(wl)
    ins, outs = [], []
    for kind, pos0, I, ev in calls:
        q, k, v = inp.block(0, pos0, I)
        if kind == "decode":
            q, k, v = q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous()
        ins.append((q, k, v))
        outs.append(torch.empty_like(q))
    arena = torch.empty(bm.arena_bytes(cfg), dtype=torch.uint8, device="cuda")
    workspace = torch.empty(max(bm.workspace_bytes(cfg), 256), dtype=torch.uint8, device="cuda")

    def step():
        cache = bm.BatchMaxCache(cfg, arena=arena, workspace=workspace)
        for (kind, pos0, I, ev), (q, k, v), o in zip(calls, ins, outs):
            if kind == "prefill":
                cache.prefill_block(q, k, v, pos0, out=o, evict_to=ev)
            else:
                cache.decode_step(q, k, v, out=o, evict_to=ev)
        return cache

    step().close()                       # first use of every kernel outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        captured = step()
    for _ in range(2):                   # a replay starts from the re-created (zeroed) cache
        graph.replay()
    torch.cuda.synchronize()
    for o, ref in zip(outs, eager_outs):
        assert torch.equal(o.cpu(), ref)
    state = [captured.export(0, s_, h, rows=True) for s_ in range(wl.b) for h in range(wl.Hkv)]
    for sa, sb in zip(state, eager_state):
        for x, y in zip(sa, sb):
            assert torch.equal(x, y)
    assert captured.status() == 0
    captured.close()


@pytest.mark.parametrize("compaction", ["stable", "fill"])
def test_sample_ranges_on_concurrent_streams_match_whole_batch_calls(compaction):
    # the launch configuration of the benchmark: the batch split into sample ranges, each range's calls on a stream of
    # its own, all in flight together; every cache must end up bit-identical to the whole-batch run
    import torch
    from paper_2412_05693_b200 import BatchMaxCache
    from paper_2412_05693_b200.workloads import Inputs, schedule
    from tests.lockstep import make_config
    wl = WORKLOADS["cfg2"].with_(b=8, s=1536, steps=12)
    dev = torch.device("cuda", 0)
    inp = Inputs(wl, dev)
    ins = [(kind, pos0, I, ev, inp.block(0, pos0, I)) for kind, pos0, I, ev in schedule(wl)]

    def run(R):
        cache = BatchMaxCache(make_config(wl, compaction=compaction))
        outs = [torch.zeros(wl.b, I, wl.Hq, wl.d, dtype=torch.bfloat16, device=dev) for _, _, I, _, _ in ins]
        streams = [torch.cuda.Stream() for _ in range(R)]
        nb = wl.b // R
        torch.cuda.synchronize()
        for r in range(R):
            with torch.cuda.stream(streams[r]):
                for (kind, pos0, I, ev, (q, k, v)), o in zip(ins, outs):
                    sl = slice(r * nb, (r + 1) * nb)
                    if kind == "prefill":
                        cache.prefill_block(q[sl], k[sl], v[sl], pos0, out=o[sl], evict_to=ev, sample0=r * nb)
                    else:
                        cache.decode_step(q[sl, 0].contiguous(), k[sl, 0].contiguous(), v[sl, 0].contiguous(),
                                          out=o[sl, 0], evict_to=ev, sample0=r * nb)
        torch.cuda.synchronize()
        assert cache.status() == 0
        state = [cache.export(0, s_, h, rows=True) for s_ in range(wl.b) for h in (0, wl.Hkv - 1)]
        cache.close()
        return outs, state

    ref_out, ref_state = run(1)
    for R in (2, 4):
        outs, state = run(R)
        assert all(torch.equal(a, b) for a, b in zip(outs, ref_out)), f"{R} ranges: outputs differ"
        for got, want in zip(state, ref_state):
            assert all(torch.equal(a, b) for a, b in zip(got, want)), f"{R} ranges: cache state differs"


@pytest.mark.parametrize("rule", ["average", "average_std"])
def test_export_import_roundtrip_resumes_identically(rule):
    wl = tiny("ckpt", dtype="bf16", d=128, Hq=8, Hkv=2, s=192, B=64, K=48, steps=0)
    cfg = make_config(wl, rule=rule)
    inp = Inputs(wl, "cuda")
    a = bm.BatchMaxCache(cfg)
    for kind, pos0, I, ev in schedule(wl)[:2]:
        a.prefill_block(*inp.block(0, pos0, I), pos0, evict_to=ev)
    b = bm.BatchMaxCache(cfg)
    for s in range(wl.b):
        n, cur = a.length(sample=s)
        b.set_len(n, cur, sample=s)
        for h in range(wl.Hkv):
            b.import_(*a.export(0, s, h, rows=True), sample=s, kv_head=h)
            if rule == "average_std":       # the rule's second accumulator travels on its own pair of calls
                b.import_sum_sq(a.export_sum_sq(0, s, h), sample=s, kv_head=h)
    kind, pos0, I, ev = schedule(wl)[2]
    q, k, v = inp.block(0, pos0, I)
    oa, ob = a.prefill_block(q, k, v, pos0, evict_to=ev), b.prefill_block(q, k, v, pos0, evict_to=ev)
    assert torch.equal(oa, ob)
    for s in range(wl.b):
        for h in range(wl.Hkv):
            for x, y in zip(a.export(0, s, h, rows=True), b.export(0, s, h, rows=True)):
                assert torch.equal(x, y)
            if rule == "average_std":
                assert torch.equal(a.export_sum_sq(0, s, h), b.export_sum_sq(0, s, h))


def test_batch_sized_by_the_allocator_fits_its_arena():
    # allocator: batch = max fitting a budget; both arms (P&D, decode-only compression) live in arenas of that size
    wl = WORKLOADS["cfg3"].with_(s=1024, B=256, K=128, steps=2)
    budget = 64 * 2 ** 20
    pd_cfg = make_config(wl, batch=1)
    do_cfg = make_config(wl, batch=1, growth=wl.s + 1 - wl.K)
    b_pd, b_do = bm.max_batch(pd_cfg, budget), bm.max_batch(do_cfg, budget)
    assert b_pd / b_do == pytest.approx((wl.s + 1) / (wl.K + 1), rel=0.08)
    for b, growth in ((b_pd, None), (b_do, wl.s + 1 - wl.K)):
        w = wl.with_(b=b)
        cfg = make_config(w, growth=growth, max_call_samples=16)
        assert bm.arena_bytes(cfg) <= budget
        arena = torch.empty(budget + 512, dtype=torch.uint8, device="cuda")
        arena[budget:] = 0xA5                                            # canary behind the arena
        cache = bm.BatchMaxCache(cfg, arena=arena[:budget])
        inp = Inputs(w, "cuda")
        for pos0 in range(0, w.s, w.B):
            for s0 in range(0, b, 16):
                ns = min(16, b - s0)
                q, k, v = inp.block(0, pos0, w.B, s0, ns)
                cache.prefill_block(q, k, v, pos0, evict_to=(w.K if growth is None else -1), sample0=s0)
        if growth is not None:
            for s0 in range(0, b, 16):
                cache.evict(w.K, sample0=s0, nsamples=min(16, b - s0))
        torch.cuda.synchronize()
        assert cache.status() == 0
        assert cache.length(sample=b - 1)[0] == w.K
        assert bool((arena[budget:] == 0xA5).all())
        ids, sw, _, _ = cache.export(0, b - 1, w.Hkv - 1)
        assert np.all(np.diff(ids.numpy()) > 0) and float(sw.min()) >= 0
        cache.close()
