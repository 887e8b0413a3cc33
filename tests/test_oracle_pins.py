"""Pins for the CPU oracle: each test fixes it to something other than itself -- values the paper
states (Sec. 3.2), closed forms, the full-attention limit, brute force on tiny inputs, an exact
rational re-simulation, a masked-dense replay and invariants."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import (UnitCache, dense_causal_attention, run_algorithm1, run_decode_only, run_extreme_decoding,
                    run_north_star)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sec3_2_closed_forms.txt")


def rand_qkv(seed, n, g, d):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n, g, d)), rng.standard_normal((n, d)), rng.standard_normal((n, d))


def read_golden():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            kv = dict(p.split("=") for p in parts[1:-1])
            rows.append((parts[0], {a: int(b) for a, b in kv.items()}, Fraction(parts[-1])))
    return rows


# ---------------------------------------------------------------- P2: values printed in Sec. 3.2
def test_paper_stated_values():
    rows = read_golden()
    assert len(rows) >= 8
    for name, args, expected in rows:
        if name == "first_pair_initial_sum_weights":
            q, k, v = rand_qkv(1, 1, args["g"], 8)
            u = UnitCache(8, args["g"])
            u.process_block(q, k, v, 0)
            assert u.sum_weights[0] == pytest.approx(float(expected), abs=1e-15)
        elif name == "row_mean":
            # Algorithm 1 with cache limit kv and p = 1: the query at position i sees min(i+1, kv) pairs
            i, kv = args["i"], args["kv"]
            q, k, v = rand_qkv(2, i + 1, 1, 4)
            u = UnitCache(4, 1)
            first = min(i + 1, kv)
            _, w = u.process_block(q[:first], k[:first], v[:first], 0, return_weights=True)
            last_row = w[-1, 0]
            for t in range(first, i + 1):
                u.evict(len(u) - 1)
                _, w = u.process_block(q[t:t + 1], k[t:t + 1], v[t:t + 1], t, return_weights=True)
                last_row = w[-1, 0]
            assert last_row.shape[0] == min(i + 1, kv)
            assert last_row.mean() == pytest.approx(float(expected), rel=1e-13)
        elif name == "rows_accumulated":
            # a pair's sum_weights is a sum of curr_id + 1 - kv_id rows: with uniform attention and no
            # eviction each of those rows contributes 1/(row position + 1)
            c, j = args["curr_id"], args["kv_id"]
            u = UnitCache(4, 1)
            u.process_block(np.zeros((c + 1, 1, 4)), *rand_qkv(3, c + 1, 1, 4)[1:], 0)
            assert (c + 1 - u.kv_ids[j]) == expected
            assert u.sum_weights[j] == pytest.approx(sum(1.0 / (i + 1) for i in range(j, c + 1)), rel=1e-13)
            assert u.ave_weights()[j] * float(expected) == pytest.approx(u.sum_weights[j], rel=1e-14)
        else:
            raise AssertionError(name)


# ---------------------------------------------------------------- P1: full-attention limit
@pytest.mark.parametrize("block", [1, 3, 7, 24])
def test_full_attention_limit_any_block_partition(block):
    s, steps, g, d = 20, 4, 2, 8
    q, k, v = rand_qkv(10, s + steps, g, d)
    out, trace, unit = run_north_star(q, k, v, s, block, kv_max=s + steps + 5, steps=steps)
    ref = dense_causal_attention(q, k, v)
    np.testing.assert_allclose(out, ref, atol=1e-12)
    assert np.array_equal(unit.kv_ids, np.arange(s + steps))


def test_dense_definition_matches_torch_sdpa():
    s, g, d = 33, 3, 16
    q, k, v = rand_qkv(11, s, g, d)
    ref = dense_causal_attention(q, k, v)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]                      # (1, g, s, d)
    tk = torch.from_numpy(k)[None, None].expand(1, g, s, d)
    tv = torch.from_numpy(v)[None, None].expand(1, g, s, d)
    lib = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    np.testing.assert_allclose(ref, lib[0].permute(1, 0, 2).numpy(), atol=1e-12)
    # and the block-wise oracle against the library routine directly
    out, _, _ = run_north_star(q, k, v, s, 5, kv_max=1000, steps=0)
    np.testing.assert_allclose(out, lib[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_custom_scale_is_used():
    s, g, d = 9, 1, 4
    q, k, v = rand_qkv(12, s, g, d)
    out, _, _ = run_north_star(q, k, v, s, 4, kv_max=100, steps=0, scale=0.37)
    np.testing.assert_allclose(out, dense_causal_attention(q, k, v, scale=0.37), atol=1e-12)


# ---------------------------------------------------------------- hand-worked example
def test_hand_worked_two_tokens():
    # d = 1, scale 1: token 0 attends to itself (weight 1); token 1 has logits (0, ln 3) -> (1/4, 3/4)
    u = UnitCache(1, 1, scale=1.0)
    q = np.array([[[1.0]], [[1.0]]])
    k = np.array([[0.0], [math.log(3.0)]])
    v = np.array([[10.0], [20.0]])
    out = u.process_block(q, k, v, 0)
    np.testing.assert_allclose(out[:, 0, 0], [10.0, 0.25 * 10 + 0.75 * 20], rtol=1e-14)
    np.testing.assert_allclose(u.sum_weights, [1.25, 0.75], rtol=1e-14)
    np.testing.assert_allclose(u.ave_weights(), [0.625, 0.75], rtol=1e-14)   # /(2-0), /(2-1)
    u.evict(1)
    assert list(u.kv_ids) == [1] and u.evicted_mass == pytest.approx(1.25)
    # next token: sees the surviving pair and itself
    out = u.process_block(np.array([[[0.0]]]), np.array([[5.0]]), np.array([[40.0]]), 2)
    np.testing.assert_allclose(out[0, 0, 0], 30.0, rtol=1e-14)
    np.testing.assert_allclose(u.sum_weights, [1.25, 0.5], rtol=1e-14)
    np.testing.assert_allclose(u.ave_weights(), [1.25 / 2, 0.5], rtol=1e-14)


def test_tie_keeps_lower_position():
    # two pairs whose weights underflow to exactly 0 tie at ave = 0: the lower id stays
    k = np.array([[0.0], [-4000.0], [-4000.0], [0.0]])
    u = UnitCache(1, 1, scale=1.0)
    u.process_block(np.ones((4, 1, 1)), k, np.zeros((4, 1)), 0)
    assert u.ave_weights()[1] == 0.0 and u.ave_weights()[2] == 0.0
    u.evict(3)
    assert list(u.kv_ids) == [0, 1, 3]


# ---------------------------------------------------------------- P3: mass conservation
@pytest.mark.parametrize("g", [1, 4])
def test_mass_conservation(g):
    s, steps, d = 70, 9, 8
    q, k, v = rand_qkv(20 + g, s + steps, g, d)
    unit = UnitCache(d, g)
    pos = 0
    for I in [16, 16, 16, 16, 6]:
        _, w = unit.process_block(q[pos:pos + I], k[pos:pos + I], v[pos:pos + I], pos, evict_to=24,
                                  return_weights=True)
        np.testing.assert_allclose(w.sum(axis=2), 1.0, atol=1e-12)          # softmax rows sum to 1
        pos += I
        assert unit.sum_weights.sum() + unit.evicted_mass == pytest.approx(g * pos, rel=1e-12)
        assert unit.rows_processed == g * pos
    for t in range(steps):
        unit.decode_step(q[s + t], k[s + t], v[s + t], evict_to=24)
        assert unit.sum_weights.sum() + unit.evicted_mass == pytest.approx(g * (s + t + 1), rel=1e-12)
        assert len(unit) == 24


# ---------------------------------------------------------------- P4: uniform attention closed forms
@pytest.mark.parametrize("g", [1, 3])
def test_uniform_attention_harmonic_closed_form(g):
    s, d = 40, 4
    _, k, v = rand_qkv(30, s, g, d)
    unit = UnitCache(d, g)
    for pos in range(0, s, 8):
        unit.process_block(np.zeros((8, g, d)), k[pos:pos + 8], v[pos:pos + 8], pos)
    H = [Fraction(0)]
    for i in range(1, s + 1):
        H.append(H[-1] + Fraction(1, i))
    expect_sum = np.array([float(g * (H[s] - H[j])) for j in range(s)])
    expect_ave = np.array([float((H[s] - H[j]) / (s - j)) for j in range(s)])
    np.testing.assert_allclose(unit.sum_weights, expect_sum, rtol=1e-13)
    np.testing.assert_allclose(unit.ave_weights(), expect_ave, rtol=1e-13)
    assert np.all(np.diff(unit.ave_weights()) < 0)     # strictly decreasing: newest pairs go first
    unit.evict(25)
    assert list(unit.kv_ids) == list(range(25))


def exact_uniform_simulation(s, block, kv_max, steps, g):
    """Integer/rational re-simulation of the schedule under uniform attention: never calls exp."""
    ids, sums = [], []
    last = -1
    trace = []

    def evict(target):
        nonlocal ids, sums
        if len(ids) <= target:
            return
        ave = [sums[j] / (g * (last + 1 - ids[j])) for j in range(len(ids))]
        order = sorted(range(len(ids)), key=lambda j: (-ave[j], ids[j]))
        keep = sorted(order[:target])
        ids = [ids[j] for j in keep]
        sums = [sums[j] for j in keep]

    pos = 0
    while pos < s + steps:
        I = min(block, s - pos) if pos < s else 1
        n_old = len(ids)
        ids += list(range(pos, pos + I))
        sums += [Fraction(0)] * I
        for i in range(I):
            m = n_old + i + 1
            for j in range(m):
                sums[j] += Fraction(g, m)
        last = pos + I - 1
        pos += I
        evict(kv_max)
        trace.append(list(ids))
    return trace, ids, sums


@pytest.mark.parametrize("s,block,kv_max,steps,g", [(37, 5, 7, 6, 1), (64, 16, 16, 5, 2), (30, 12, 4, 3, 1)])
def test_uniform_attention_exact_simulation(s, block, kv_max, steps, g):
    d = 4
    _, k, v = rand_qkv(31, s + steps, g, d)
    q = np.zeros((s + steps, g, d))
    _, trace, unit = run_north_star(q, k, v, s, block, kv_max, steps)
    ref_trace, ref_ids, ref_sums = exact_uniform_simulation(s, block, kv_max, steps, g)
    assert len(trace) == len(ref_trace)
    for a, b in zip(trace, ref_trace):
        assert list(a) == b
    np.testing.assert_allclose(unit.sum_weights, [float(x) for x in ref_sums], rtol=1e-12)


# ---------------------------------------------------------------- P5: brute force on tiny inputs
def brute_force_keep(ids, ave, target):
    """All size-`target` subsets: maximise the summed ave; ties -> lexicographically smallest ids."""
    best = None
    for comb in itertools.combinations(range(len(ids)), target):
        key = (-sum(Fraction(ave[j]) for j in comb), tuple(ids[j] for j in comb))
        if best is None or key < best[0]:
            best = (key, comb)
    return [ids[j] for j in best[1]]


def test_eviction_equals_brute_force_subset_choice():
    rng = np.random.default_rng(40)
    for trial in range(30):
        n = int(rng.integers(2, 11))
        target = int(rng.integers(1, n))
        d, g = 4, int(rng.integers(1, 3))
        q, k, v = rand_qkv(100 + trial, n, g, d)
        if trial % 3 == 0:            # force exact ties through duplicated sums
            q[:] = 0.0
            k[:] = k[0]
        u = UnitCache(d, g)
        u.process_block(q, k, v, 0)
        if trial % 3 == 0:
            u.sum_weights[:] = np.round(u.sum_weights * 2) / 2 + 0.5    # many exact ties in the sums
            u.sum_weights *= (u.last_pos + 1 - u.kv_ids)                # -> exact ties in ave as well
        ids, ave = list(u.kv_ids), list(u.ave_weights())
        expect = brute_force_keep(ids, ave, target)
        snap = u.evict(target)
        assert list(u.kv_ids) == expect
        assert snap["cut"] == min(ave[ids.index(j)] for j in expect)


def brute_force_run(q, k, v, s, block, kv_max, steps, scale):
    """Whole schedule re-stated with python lists and scalar loops only."""
    n, g, d = q.shape
    ids, sums, outs = [], [], []
    pos = 0
    while pos < s + steps:
        I = min(block, s - pos) if pos < s else 1
        n_old = len(ids)
        ids += list(range(pos, pos + I))
        sums += [0.0] * I
        for i in range(I):
            vis = ids[:n_old + i + 1]
            for h in range(g):
                lg = [scale * sum(q[pos + i, h, c] * k[j, c] for c in range(d)) for j in vis]
                mx = max(lg)
                ex = [math.exp(x - mx) for x in lg]
                z = sum(ex)
                outs.append([sum(ex[t] / z * v[j, c] for t, j in enumerate(vis)) for c in range(d)])
                for t in range(len(vis)):
                    sums[t] += ex[t] / z
        last = pos + I - 1
        pos += I
        if len(ids) > kv_max:
            ave = [sums[t] / (g * (last + 1 - ids[t])) for t in range(len(ids))]
            keep_ids = brute_force_keep(ids, ave, kv_max)
            sums = [sums[ids.index(j)] for j in keep_ids]
            ids = keep_ids
    return np.array(outs).reshape(s + steps, g, d), ids, sums


@pytest.mark.parametrize("s,block,kv_max,steps,g", [(12, 3, 4, 3, 1), (13, 3, 4, 2, 2), (16, 2, 3, 0, 1),
                                                     (10, 5, 2, 4, 1), (9, 1, 4, 2, 2)])
def test_full_brute_force_runs(s, block, kv_max, steps, g):
    d = 3
    q, k, v = rand_qkv(50 + s, s + steps, g, d)
    out, _, unit = run_north_star(q, k, v, s, block, kv_max, steps)
    ref_out, ref_ids, ref_sums = brute_force_run(q, k, v, s, block, kv_max, steps, 1.0 / math.sqrt(d))
    np.testing.assert_allclose(out, ref_out, atol=1e-12)
    assert list(unit.kv_ids) == ref_ids
    np.testing.assert_allclose(unit.sum_weights, ref_sums, rtol=1e-12)


# ---------------------------------------------------------------- P6: Algorithm 1 as printed
@pytest.mark.parametrize("s,K,B,max_gen", [(96, 16, 8, 20), (104, 16, 8, 13), (64, 32, 16, 40), (20, 32, 8, 30)])
def test_algorithm1_equals_north_star_form(s, K, B, max_gen):
    g, d = 2, 8
    steps = max_gen - 1
    q, k, v = rand_qkv(60 + s, s + steps, g, d)
    out_p, trace_p, unit_p, sizes = run_algorithm1(q, k, v, s, kv_bar=K + B, p=B, max_gen=max_gen)
    out_n, trace_n, unit_n = run_north_star(q, k, v, s, B, K, steps, p_dec=B)
    np.testing.assert_allclose(out_p, out_n, atol=1e-11)
    # occupancy bound of Sec. 4.1: |kv| >= kv_bar - p right after every removal, never above kv_bar
    assert all(n == K for n in sizes)
    assert all(len(t) <= K + B for t in trace_p)
    # state before each Algorithm-1 removal == state after the matching spec eviction
    if s % B == 0 and s > K + B:
        unit_p.evict(K)
        ids_n = trace_n[s // B - 1] if steps == 0 else None
        if ids_n is not None:
            assert list(unit_p.kv_ids) == list(ids_n)


def test_algorithm1_ragged_tail_leaves_cache_below_limit():
    # Algorithm 1 still removes p pairs before a short last block, so the cache ends below kv_bar and the
    # first decode steps remove nothing (the two schedules coincide only for equal-sized blocks)
    s, K, B, g, d = 100, 16, 8, 1, 4
    q, k, v = rand_qkv(63, s + 6, g, d)
    _, trace, _, sizes = run_algorithm1(q, k, v, s, kv_bar=K + B, p=B, max_gen=7)
    n_prefill_calls = 1 + math.ceil((s - (K + B)) / B)
    assert len(trace[n_prefill_calls - 1]) == K + (s - (K + B)) % B
    assert [len(t) for t in trace[n_prefill_calls:]] == [K + 4 + t for t in range(1, 5)] + [K + 1, K + 2]


def test_algorithm1_kept_sets_match_north_star_blockwise():
    s, K, B, g, d = 128, 32, 16, 1, 8
    q, k, v = rand_qkv(61, s, g, d)
    _, trace_p, _, _ = run_algorithm1(q, k, v, s, kv_bar=K + B, p=B, max_gen=1)
    _, trace_n, _ = run_north_star(q, k, v, s, B, K, 0)
    # Algorithm-1 call c (c >= 1) starts from spec state after block (K+B)/B - 1 + c - 1 and adds a block
    first = (K + B) // B
    for c in range(1, len(trace_p)):
        kept_before = trace_n[first - 1 + c - 1]
        block_ids = list(range((first + c - 1) * B, (first + c) * B))
        assert list(trace_p[c]) == list(kept_before) + block_ids


def test_literal_decode_curr_id_changes_only_the_denominator():
    s, g, d = 40, 1, 4
    q, k, v = rand_qkv(62, s + 30, g, d)
    a = run_algorithm1(q, k, v, s, 16, 4, 31)
    b = run_algorithm1(q, k, v, s, 16, 4, 31, literal_decode_curr_id=True)
    assert len(a[1]) == len(b[1])
    assert list(a[1][(s - 16) // 4]) == list(b[1][(s - 16) // 4])     # prefill part is identical


def test_literal_decode_curr_id_flips_a_hand_counted_eviction():
    # Algorithm 1 with limit 3 and p = 1 on a prompt of 3 tokens, head dimension 1, scale 1.  Query 0 sees pair 0
    # alone (weight 1); query 1 is zero, so it weighs pairs 0 and 1 by 1/2 each; query 2 is 1 and the keys are
    # ln 11, ln 2, ln 7, so its weights are 11/20, 2/20, 7/20.  Column sums: 41/20, 12/20, 7/20.
    #   rows accumulated (Sec. 3.2's justification):  denominators 3, 2, 1 -> 41/60, 18/60, 21/60: pair 1 leaves;
    #   the decode loop's printed curr_id = s + t - 1 = 3: denominators 4, 3, 2 -> 41/80, 16/80, 14/80: pair 2 leaves.
    q = np.array([0.3, 0.0, 1.0, 0.7]).reshape(4, 1, 1)
    k = np.array([math.log(11), math.log(2), math.log(7), 0.25]).reshape(4, 1)
    v = np.array([1.0, 2.0, 3.0, 4.0]).reshape(4, 1)
    u = UnitCache(1, 1, scale=1.0)
    u.process_block(q[:3], k[:3], v[:3], 0)
    np.testing.assert_allclose(u.sum_weights, [41 / 20, 12 / 20, 7 / 20], rtol=1e-14)
    np.testing.assert_allclose(u.ave_weights(), [41 / 60, 18 / 60, 21 / 60], rtol=1e-14)
    np.testing.assert_allclose(u.ave_weights(curr_id=3), [41 / 80, 16 / 80, 14 / 80], rtol=1e-14)
    exact = run_algorithm1(q, k, v, 3, 3, 1, 2, scale=1.0)
    literal = run_algorithm1(q, k, v, 3, 3, 1, 2, scale=1.0, literal_decode_curr_id=True)
    assert list(exact[1][-1]) == [0, 2, 3]
    assert list(literal[1][-1]) == [0, 1, 3]
    # the decode query (0.7) then sees different pairs: softmax over keys {ln 11, ln 7, 1/4} against {ln 11, ln 2, 1/4}
    def expected(keys, vals):
        w = np.array([math.exp(0.7 * x) for x in keys])
        return float((w / w.sum()) @ np.array(vals))
    assert exact[0][3, 0, 0] == pytest.approx(expected([math.log(11), math.log(7), 0.25], [1.0, 3.0, 4.0]), rel=1e-13)
    assert literal[0][3, 0, 0] == pytest.approx(expected([math.log(11), math.log(2), 0.25], [1.0, 2.0, 4.0]), rel=1e-13)


def test_decode_only_compression_replayed_from_the_original_arrays():
    # whole prompt with a full cache, ONE compression to kv_max by the average of the dense column sums, then
    # every decode query sees the survivors of the previous call plus itself: all recomputed from the original
    # q/k/v by masked attention written from the definition, never touching the cache structure
    s, B, K, steps, g, d = 37, 8, 9, 11, 2, 8
    q, k, v = rand_qkv(95, s + steps, g, d)
    out, trace, unit = run_decode_only(q, k, v, s, B, K, steps)
    scale = 1.0 / math.sqrt(d)

    def weights(i, js):
        w = np.zeros((g, s + steps))
        for h in range(g):
            logits = np.array([scale * float(q[i, h] @ k[j]) for j in js])
            e = np.exp(logits - logits.max())
            w[h, js] = e / e.sum()
        return w

    col = np.zeros(s + steps)
    for i in range(s):
        w = weights(i, list(range(i + 1)))
        col += w.sum(axis=0)
        np.testing.assert_allclose(out[i], w @ v, atol=1e-12)
    ave = col[:s] / (g * (s - np.arange(s)))
    kept = sorted(sorted(range(s), key=lambda j: (-ave[j], j))[:K])
    assert list(trace[0]) == kept
    for t in range(steps):
        i = s + t
        js = kept + [i]
        w = weights(i, js)
        col += w.sum(axis=0)
        np.testing.assert_allclose(out[i], w @ v, atol=1e-12)
        ave = {j: col[j] / (g * (i + 1 - j)) for j in js}
        kept = sorted(sorted(js, key=lambda j: (-ave[j], j))[:K])
        assert list(trace[t + 1]) == kept
    np.testing.assert_allclose(unit.sum_weights, col[kept], rtol=1e-12)


# ---------------------------------------------------------------- P7: masked-dense replay
def test_masked_dense_replay():
    s, B, K, steps, g, d = 60, 8, 12, 7, 2, 8
    q, k, v = rand_qkv(70, s + steps, g, d)
    out, trace, unit = run_north_star(q, k, v, s, B, K, steps)
    scale = 1.0 / math.sqrt(d)
    n_tot = s + steps
    col_sum = np.zeros(n_tot)
    kept_prev = np.zeros(0, dtype=np.int64)
    pos, call = 0, 0
    while pos < n_tot:
        I = min(B, s - pos) if pos < s else 1
        for i in range(I):
            p_i = pos + i
            vis = np.concatenate([kept_prev, np.arange(pos, p_i + 1)])
            for h in range(g):
                lg = scale * (k[vis] @ q[p_i, h])
                w = np.exp(lg - lg.max())
                w /= w.sum()
                np.testing.assert_allclose(out[p_i, h], w @ v[vis], atol=1e-12)
                col_sum[vis] += w
        kept_prev = np.asarray(trace[call])
        pos += I
        call += 1
    np.testing.assert_allclose(unit.sum_weights, col_sum[unit.kv_ids], rtol=1e-12)
    np.testing.assert_allclose(unit.k, k[unit.kv_ids])
    np.testing.assert_allclose(unit.v, v[unit.kv_ids])


# ---------------------------------------------------------------- P8 / P9
def test_decode_is_block_of_one():
    g, d = 2, 8
    q, k, v = rand_qkv(80, 30, g, d)
    a, b = UnitCache(d, g), UnitCache(d, g)
    a.process_block(q[:20], k[:20], v[:20], 0, 8)
    b.process_block(q[:20], k[:20], v[:20], 0, 8)
    for t in range(20, 30):
        oa = a.decode_step(q[t], k[t], v[t], 8)
        ob = b.process_block(q[t:t + 1], k[t:t + 1], v[t:t + 1], t, 8)[0]
        np.testing.assert_array_equal(oa, ob)
    np.testing.assert_array_equal(a.kv_ids, b.kv_ids)


def test_invariants_and_symmetries():
    s, B, K, steps, g, d = 90, 16, 20, 10, 2, 8
    q, k, v = rand_qkv(90, s + steps, g, d)
    out, trace, unit = run_north_star(q, k, v, s, B, K, steps)
    prev = np.zeros(0, dtype=np.int64)
    pos = 0
    for c, ids in enumerate(trace):
        I = min(B, s - pos) if pos < s else 1
        assert len(ids) <= K and np.all(np.diff(ids) > 0)
        assert set(ids) <= set(prev) | set(range(pos, pos + I))
        prev, pos = ids, pos + I
    ave = unit.ave_weights()
    assert np.all(ave >= 0) and np.all(ave <= 1)
    assert out.min() >= v.min() - 1e-12 and out.max() <= v.max() + 1e-12
    # MHA with the KV head duplicated g times: same outputs as GQA, head by head
    for h in range(g):
        out_h, _, _ = run_north_star(q[:, h:h + 1], k, v, s, B, 10 ** 6, steps)
        out_all, _, _ = run_north_star(q, k, v, s, B, 10 ** 6, steps)
        np.testing.assert_allclose(out_all[:, h], out_h[:, 0], atol=1e-12)
    # GQA aggregation: the group's sum_weights is the sum over its heads' sums (no eviction)
    u_all = run_north_star(q, k, v, s, B, 10 ** 6, 0)[2]
    u_sep = [run_north_star(q[:, h:h + 1], k, v, s, B, 10 ** 6, 0)[2] for h in range(g)]
    np.testing.assert_allclose(u_all.sum_weights, sum(u.sum_weights for u in u_sep), rtol=1e-12)
    np.testing.assert_allclose(u_all.ave_weights(), sum(u.ave_weights() for u in u_sep) / g, rtol=1e-12)


def test_short_prompt_never_evicts_in_prefill_and_decode_only_arm():
    s, B, K, steps, g, d = 12, 4, 16, 8, 1, 4
    q, k, v = rand_qkv(91, s + steps, g, d)
    _, trace, unit = run_north_star(q, k, v, s, B, K, steps)
    assert [len(t) for t in trace[:3]] == [4, 8, 12]
    assert len(unit) == 16
    # decode-only compression: whole prompt cached, one compression, then decode
    s = 40
    q, k, v = rand_qkv(92, s + steps, g, d)
    out_do, trace_do, unit_do = run_decode_only(q, k, v, s, 8, 10, steps)
    np.testing.assert_allclose(out_do[:s], dense_causal_attention(q[:s], k[:s], v[:s]), atol=1e-12)
    assert all(len(t) == 10 for t in trace_do)


def test_out_of_order_position_rejected():
    u = UnitCache(4, 1)
    q, k, v = rand_qkv(93, 4, 1, 4)
    u.process_block(q[:2], k[:2], v[:2], 0)
    with pytest.raises(ValueError):
        u.process_block(q[2:], k[2:], v[2:], 3)


def test_kept_override_for_lockstep():
    q, k, v = rand_qkv(94, 10, 1, 4)
    u = UnitCache(4, 1)
    u.process_block(q, k, v, 0)
    snap = u.evict(5, kept_ids=[0, 2, 4, 6, 8])
    assert list(u.kv_ids) == [0, 2, 4, 6, 8]
    assert len(snap["kept_ids"]) == 5 and snap["cand_ids"].shape[0] == 10


# ---------------------------------------------------------------- Algorithm 3 (extreme decoding-only eviction)
def windowed_attention(q, k, v, visible, scale):
    """Row i attends to the positions visible(i); written straight from the softmax definition."""
    out = np.zeros((q.shape[0], q.shape[1], v.shape[1]))
    for i in range(q.shape[0]):
        js = visible(i)
        for h in range(q.shape[1]):
            logits = np.array([scale * float(q[i, h] @ k[j]) for j in js])
            w = np.exp(logits - logits.max())
            w /= w.sum()
            out[i, h] = sum(wj * v[j] for wj, j in zip(w, js))
    return out


@pytest.mark.parametrize("kv_bar,block", [(2, None), (2, 5), (5, None), (65, 7)])
def test_extreme_decoding_is_prompt_dense_then_window_since_last_cut(kv_bar, block):
    # Algorithm 3: the prompt sees everything; afterwards the cache is the pair kept at the last cut plus
    # what was generated since, so with a limit of 2 every decode query sees its predecessor and itself.
    s, g, d, max_gen = 23, 2, 8, 80
    q, k, v = rand_qkv(31, s + max_gen, g, d)
    out, unit, sizes = run_extreme_decoding(q, k, v, s, kv_bar, max_gen, block=block)
    scale = 1.0 / math.sqrt(d)

    def visible(i):
        if i < s:
            return list(range(i + 1))
        t = i - s                               # decode forwards since the prompt
        anchor = s - 1 + (t // (kv_bar - 1)) * (kv_bar - 1)   # pair kept at the most recent cut
        return list(range(anchor, i + 1))

    n_rows = s + max_gen - 1
    np.testing.assert_allclose(out, windowed_attention(q[:n_rows], k, v, visible, scale), atol=1e-12)
    assert max(sizes) == kv_bar and min(sizes) == 2
    assert len(unit) == (1 if (max_gen - 1) % (kv_bar - 1) == 0 else 1 + (max_gen - 1) % (kv_bar - 1))
    # mass conservation also holds under this rule
    assert unit.sum_weights.sum() + unit.evicted_mass == pytest.approx(g * n_rows, rel=1e-12)


def test_keep_most_recent_keeps_ids_and_sums_of_the_tail():
    u = UnitCache(4, 1)
    q, k, v = rand_qkv(5, 9, 1, 4)
    u.process_block(q, k, v, 0)
    before = (u.kv_ids.copy(), u.sum_weights.copy(), u.k.copy(), u.v.copy())
    u.keep_most_recent(3)
    assert list(u.kv_ids) == [6, 7, 8]
    for a, b in zip(before, (u.kv_ids, u.sum_weights, u.k, u.v)):
        assert np.array_equal(a[6:], b)
    u.keep_most_recent(5)                       # nothing to remove
    assert len(u) == 3


# ---------------------------------------------------------------- left padding (Sec. 3)
@pytest.mark.parametrize("pad,block", [(1, 4), (7, 4), (8, 8), (13, 5), (19, 32)])
def test_left_padding_full_cache_equals_dense_attention_over_the_real_tokens(pad, block):
    # nothing is evicted: the real queries must see exactly the un-padded sequence, whatever sits in the padding
    s, g, d = 29, 2, 8
    q, k, v = rand_qkv(41, s, g, d)
    out, _, unit = run_north_star(q, k, v, s, block, kv_max=1000, steps=0, left_pad=pad)
    np.testing.assert_allclose(out[pad:], dense_causal_attention(q[pad:], k[pad:], v[pad:]), atol=1e-12)
    assert np.all(out[:pad] == 0.0)
    assert np.all(unit.sum_weights[:pad] == 0.0)
    _, _, ref = run_north_star(q[pad:], k[pad:], v[pad:], s - pad, block, kv_max=1000, steps=0)
    np.testing.assert_allclose(unit.sum_weights[pad:], ref.sum_weights, rtol=1e-12)
    assert unit.rows_processed == g * (s - pad)


@pytest.mark.parametrize("pad_blocks", [1, 2])
@pytest.mark.parametrize("g", [1, 3])
def test_left_padding_by_whole_blocks_is_the_unpadded_run_shifted(pad_blocks, g):
    # padding fills the first blocks exactly, so block boundaries and every eviction line up with the run on the
    # real tokens alone: same outputs, same survivors (ids shifted by the padding), same sums
    s, B, K, steps, d = 48, 8, 5, 6, 4
    pad = pad_blocks * B
    q, k, v = rand_qkv(43, s + steps, g, d)
    out, trace, unit = run_north_star(q, k, v, s, B, K, steps, left_pad=pad)
    out0, trace0, unit0 = run_north_star(q[pad:], k[pad:], v[pad:], s - pad, B, K, steps)
    np.testing.assert_allclose(out[pad:], out0, atol=1e-12)
    assert np.array_equal(unit.kv_ids - pad, unit0.kv_ids)
    np.testing.assert_allclose(unit.sum_weights, unit0.sum_weights, rtol=1e-12)
    for ids, ids0 in zip(trace[pad_blocks + 1:], trace0[1:]):     # once one real block went through, padding is gone
        assert np.array_equal(np.asarray(ids) - pad, ids0)


def test_left_padding_leaves_first_and_from_the_top():
    s, B, K, g, d, pad = 40, 8, 12, 2, 4, 11
    q, k, v = rand_qkv(47, s, g, d)
    unit = UnitCache(d, g, left_pad=pad)
    for pos in range(0, s, B):
        before = set(unit.kv_ids.tolist()) | set(range(pos, pos + B))
        unit.process_block(q[pos:pos + B], k[pos:pos + B], v[pos:pos + B], pos, K)
        kept = set(unit.kv_ids.tolist())
        gone = before - kept
        pads_kept = sorted(i for i in kept if i < pad)
        if any(i >= pad for i in gone):
            assert not pads_kept                           # a real pair left only once all padding was gone
        assert pads_kept == list(range(len(pads_kept)))    # the padding that stays is the lowest positions
        assert np.all(unit.sum_weights[unit.kv_ids < pad] == 0.0)
    assert unit.sum_weights.sum() + unit.evicted_mass == pytest.approx(g * (s - pad), rel=1e-12)


def test_left_padding_masked_dense_replay():
    # outputs recomputed from the trace of visible ids over the original arrays, padding positions removed
    s, B, K, steps, g, d, pad = 37, 6, 7, 5, 2, 4, 9
    q, k, v = rand_qkv(53, s + steps, g, d)
    out, trace, _ = run_north_star(q, k, v, s, B, K, steps, left_pad=pad)
    scale = 1.0 / math.sqrt(d)
    cached, pos, call = [], 0, 0
    bounds = [(p0, min(B, s - p0)) for p0 in range(0, s, B)] + [(s + t, 1) for t in range(steps)]
    for p0, I in bounds:
        for i in range(I):
            qi = p0 + i
            if qi < pad:
                assert np.all(out[qi] == 0.0)
                continue
            js = [j for j in list(cached) + list(range(p0, qi + 1)) if j >= pad]
            for h in range(g):
                lg = np.array([scale * float(q[qi, h] @ k[j]) for j in js])
                w = np.exp(lg - lg.max())
                w /= w.sum()
                np.testing.assert_allclose(out[qi, h], sum(wj * v[j] for wj, j in zip(w, js)), atol=1e-12)
        cached = list(trace[call])
        call += 1


# ---------------------------------------------------------------- the rules Sec. 2 ascribes to other methods
def replay_weights(q, k, visible_sets, queries, scale):
    """weights[(query position, head)] = {key id: softmax weight} recomputed from the original arrays."""
    out = {}
    for qi, vis in zip(queries, visible_sets):
        for h in range(q.shape[1]):
            lg = np.array([scale * float(q[qi, h] @ k[j]) for j in vis])
            w = np.exp(lg - lg.max())
            w /= w.sum()
            out[(qi, h)] = dict(zip(vis, w))
    return out


@pytest.mark.parametrize("rule", ["current_query", "sum_recent"])
def test_alternative_rules_against_a_replay_from_the_original_arrays(rule):
    # every eviction is re-derived from the trace of kept ids and the ORIGINAL q/k arrays: column sums over the
    # queries that saw a pair (sum_recent) or the last query's weights alone (current_query), never the cache's state
    s, B, K, steps, g, d = 40, 8, 7, 6, 2, 4
    q, k, v = rand_qkv(61, s + steps, g, d)
    out, trace, unit = run_north_star(q, k, v, s, B, K, steps, rule=rule)
    scale = 1.0 / math.sqrt(d)
    cached, sums = [], {}
    calls = [(p0, min(B, s - p0)) for p0 in range(0, s, B)] + [(s + t, 1) for t in range(steps)]
    for call, (p0, I) in enumerate(calls):
        cand = list(cached) + list(range(p0, p0 + I))
        if rule == "current_query":
            sums = {}
        for i in range(I):
            qi = p0 + i
            vis = list(cached) + list(range(p0, qi + 1))
            if rule == "current_query" and i != I - 1:
                continue
            for (_, h), w in replay_weights(q, k, [vis], [qi], scale).items():
                for j, wj in w.items():
                    sums[j] = sums.get(j, 0.0) + wj
        if len(cand) > K:
            window = cand[len(cand) - K // 2:] if (rule == "sum_recent" and K // 2 > 0) else []
            rest = [j for j in cand if j not in window]
            rest.sort(key=lambda j: (-sums.get(j, 0.0), j))
            kept = sorted(window + rest[:K - len(window)])
        else:
            kept = cand
        assert kept == list(trace[call]), f"call {call}"
        sums = {j: sums.get(j, 0.0) for j in kept}
        cached = kept


@pytest.mark.parametrize("w,pool", [(3, 1), (4, 3), (20, 5), (2, 7)])
def test_window_pooled_rule_against_a_replay_from_the_original_arrays(w, pool):
    # SnapKV as Sec. 2 describes it: scores = attention weights summed over the last w queries of the pass, pooled
    # over neighbouring positions, a window of recent pairs always kept.  Re-derived from the trace and the original
    # arrays, with the pooling written as a plain loop over the candidates' order.
    s, B, K, steps, g, d = 44, 9, 10, 5, 2, 4
    q, k, v = rand_qkv(73, s + steps, g, d)
    out, trace, unit = run_north_star(q, k, v, s, B, K, steps, rule="window_pooled", window=w, pool=pool)
    scale = 1.0 / math.sqrt(d)
    cached = []
    calls = [(p0, min(B, s - p0)) for p0 in range(0, s, B)] + [(s + t, 1) for t in range(steps)]
    for call, (p0, I) in enumerate(calls):
        cand = list(cached) + list(range(p0, p0 + I))
        sums = {j: 0.0 for j in cand}
        for i in range(I - min(w, I), I):
            qi = p0 + i
            vis = list(cached) + list(range(p0, qi + 1))
            for (_, h), wt in replay_weights(q, k, [vis], [qi], scale).items():
                for j, wj in wt.items():
                    sums[j] += wj
        if len(cand) > K:
            recent = cand[len(cand) - min(w, K):]
            body = cand[:len(cand) - len(recent)]
            pooled = {}
            for x, j in enumerate(body):
                lo, hi = max(0, x - pool // 2), min(len(body), x + pool // 2 + 1)
                pooled[j] = max(sums[body[y]] for y in range(lo, hi))
            rest = sorted(body, key=lambda j: (-pooled[j], j))
            kept = sorted(recent + rest[:K - len(recent)])
        else:
            kept = cand
        assert kept == list(trace[call]), f"call {call}"
        cached = kept


@pytest.mark.parametrize("share,g", [(0.0, 1), (0.5, 2), (0.3, 1), (1.0, 2)])
def test_average_std_rule_against_a_replay_from_the_original_arrays(share, g):
    # RoCo as Sec. 2 / Sec. 3.2 describe it: part of the kept pairs by the standard deviation of their attention
    # weights, the rest by their average.  The replay keeps, per pair, the plain list of every weight it received.
    s, B, K, steps, d = 40, 8, 9, 6, 4
    q, k, v = rand_qkv(79, s + steps, g, d)
    out, trace, unit = run_north_star(q, k, v, s, B, K, steps, rule="average_std", std_share=share)
    scale = 1.0 / math.sqrt(d)
    cached, got = [], {}
    calls = [(p0, min(B, s - p0)) for p0 in range(0, s, B)] + [(s + t, 1) for t in range(steps)]
    for call, (p0, I) in enumerate(calls):
        cand = list(cached) + list(range(p0, p0 + I))
        for i in range(I):
            qi = p0 + i
            vis = list(cached) + list(range(p0, qi + 1))
            for (_, h), wt in replay_weights(q, k, [vis], [qi], scale).items():
                for j, wj in wt.items():
                    got.setdefault(j, []).append(wj)
        if len(cand) > K:
            assert all(len(got[j]) == g * (p0 + I - j) for j in cand)      # one weight per later-or-equal query and head
            std = {j: float(np.std(got[j])) for j in cand}                 # population standard deviation
            ave = {j: float(np.mean(got[j])) for j in cand}
            n_std = int(math.floor(share * K + 1e-9))
            protected = sorted(cand, key=lambda j: (-std[j], j))[:n_std]
            rest = sorted([j for j in cand if j not in protected], key=lambda j: (-ave[j], j))
            kept = sorted(protected + rest[:K - n_std])
        else:
            kept = cand
        assert kept == list(trace[call]), f"call {call}"
        got = {j: got[j] for j in kept}
        cached = kept
    if share == 0.0:      # no pair chosen by deviation: the method's own rule
        _, trace_ave, _ = run_north_star(q, k, v, s, B, K, steps)
        assert all(list(a) == list(b) for a, b in zip(trace, trace_ave))


def test_window_pooled_with_window_one_and_no_pooling_is_the_current_query_rule_plus_its_newest_pair():
    # w = 1, pool = 1: scores are the last query's weights (as under current_query); the one difference is that
    # the newest pair is never a candidate for removal
    s, B, K, g, d = 30, 6, 5, 1, 4
    q, k, v = rand_qkv(83, s, g, d)
    u = UnitCache(d, g, rule="window_pooled", window=1, pool=1)
    u2 = UnitCache(d, g, rule="current_query")
    for p0 in range(0, s, B):
        u.process_block(q[p0:p0 + B], k[p0:p0 + B], v[p0:p0 + B], p0)
        u2.process_block(q[p0:p0 + B], k[p0:p0 + B], v[p0:p0 + B], p0)
        np.testing.assert_allclose(u.sum_weights, u2.sum_weights, rtol=1e-14)
        u.evict(K)
        assert u.kv_ids[-1] == p0 + B - 1
        u2.evict(K, kept_ids=u.kv_ids)


def test_sum_recent_keeps_its_window_and_current_query_forgets():
    g, d = 1, 4
    q, k, v = rand_qkv(67, 30, g, d)
    u = UnitCache(d, g, rule="sum_recent")
    u.process_block(q[:20], k[:20], v[:20], 0, evict_to=8)
    assert set(range(16, 20)) <= set(u.kv_ids.tolist())          # the 4 most recent of 8 always stay
    u2 = UnitCache(d, g, rule="current_query")
    _, w = u2.process_block(q[:20], k[:20], v[:20], 0, return_weights=True)
    np.testing.assert_allclose(u2.sum_weights, w[19, 0], rtol=1e-14)   # the last query's row and nothing else
    u2.decode_step(q[20], k[20], v[20])
    assert u2.sum_weights.sum() == pytest.approx(1.0)             # previous sums are gone


def test_padding_ranks_last_even_inside_the_recent_window():
    # a block that is all padding: the window of the most recent candidates holds padding only, which still
    # leaves from the top, so the lowest padding positions are what stays
    g, d = 1, 4
    q, k, v = rand_qkv(71, 40, g, d)
    u = UnitCache(d, g, left_pad=30, rule="sum_recent")
    u.process_block(q[:20], k[:20], v[:20], 0, evict_to=8)
    assert u.kv_ids.tolist() == list(range(8))
    u.process_block(q[20:40], k[20:40], v[20:40], 20, evict_to=8)     # 10 more padding positions, then 10 real ones
    assert u.kv_ids.tolist()[-4:] == [36, 37, 38, 39]                  # the window of recent real pairs
    assert all(i >= 30 for i in u.kv_ids.tolist())                     # every real pair outranks padding
