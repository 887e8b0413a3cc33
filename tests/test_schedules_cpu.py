"""Host logic of the timed arms: the call lists that experiments.py feeds to the library (no GPU, no library call)."""
import pytest

from paper_2412_05693_b200.experiments import arm_calls, make_cfg
from paper_2412_05693_b200.workloads import Workload, schedule

WL = Workload("t", b=3, Hq=8, Hkv=8, d=128, dtype="bf16", s=3584, B=512, K=1024, steps=511, seed=5, heavy_count=4)


def sizes(calls):
    """Cache size after every call, following the documented transition of each call kind."""
    n, out = 0, []
    for kind, pos0, I, arg in calls:
        if kind == "prefill":
            n = n + I if arg < 0 else min(n + I, arg)
        elif kind == "decode":
            n = n + 1 if arg < 0 else min(n + 1, arg)
        else:
            n = min(n, arg)
        out.append((kind, n))
    return out


@pytest.mark.parametrize("kv_bar,p", [(1024, 64), (2048, 64), (96, 32)])
def test_algorithm1_arm_keeps_the_cache_between_kv_bar_minus_p_and_kv_bar(kv_bar, p):
    calls = arm_calls(WL, "alg1", kv_bar=kv_bar, p=p)
    positions = [c[1] for c in calls if c[0] in ("prefill", "decode")]
    lengths = [c[2] for c in calls if c[0] in ("prefill", "decode")]
    assert positions[0] == 0 and all(a + l == b for a, l, b in zip(positions, lengths, positions[1:]))
    assert positions[-1] + lengths[-1] == WL.s + WL.steps               # every token processed exactly once
    seen_full = False
    for kind, n in sizes(calls):
        assert n <= kv_bar                                                # the limit of Algorithm 1
        seen_full = seen_full or n == kv_bar
        if seen_full:
            assert n >= kv_bar - p                                        # Sec. 4: |kv| >= limit - p from then on
    assert make_cfg(WL, 1, "alg1", 1, kv_bar=kv_bar, p=p).cap == kv_bar
    evicts = [c for c in calls if c[0] == "evict"]
    assert all(c[3] == kv_bar - p for c in evicts)                        # p pairs removed whenever the cache is full


@pytest.mark.parametrize("kv_bar", [2, 65])
def test_extreme_decoding_arm(kv_bar):
    calls = arm_calls(WL, "ed", kv_bar=kv_bar)
    sz = sizes(calls)
    assert max(n for _, n in sz) == WL.s                                  # the whole prompt is cached once
    after_prompt = [n for kind, n in sz[len([c for c in calls if c[0] == "prefill"]):]]
    assert max(after_prompt[1:]) == kv_bar and min(after_prompt) == 1     # then at most kv_bar, cut back to one pair
    assert make_cfg(WL, 1, "ed", 1, kv_bar=kv_bar).cap == WL.s + max(1, kv_bar - 1)


def test_full_cache_and_decode_only_arms():
    assert all(arg < 0 for kind, _, _, arg in arm_calls(WL, "fkv"))
    assert make_cfg(WL, 1, "fkv", 1).cap == WL.s + WL.steps
    do = arm_calls(WL, "do")
    assert [c[0] for c in do].count("evict") == 1 and make_cfg(WL, 1, "do", 1).cap == WL.s + 1
    pd = arm_calls(WL, "pd")
    assert pd == [(k, p0, I, ev) for k, p0, I, ev in schedule(WL)]        # the benchmark's own schedule
    assert make_cfg(WL, 1, "pd", 1).cap == WL.K + 1
