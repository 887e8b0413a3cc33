"""bm_prefill_block_static: the block forward pass for callers that cannot allocate device scratch (frozen
memory plan, allocator owned by a framework, threads barred from allocating CUDA calls).  It must give the
same outputs and the same cache state as bm_prefill_block, call after call, while sharing one built-in array.
Collected last on purpose: a failure here cannot hide the result of any other test."""
import pytest
import torch

import paper_2412_05693_b200 as bm
from paper_2412_05693_b200.workloads import Inputs, Workload
from tests.lockstep import make_config

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_static_scratch_entry_point_matches_workspace_entry_point(dtype, d):
    wl = Workload("static_scratch", b=3, Hq=8, Hkv=2, d=d, dtype=dtype, s=384, B=128, K=96, steps=0, seed=77,
                  heavy_count=4)
    cfg = make_config(wl)
    inp = Inputs(wl, "cuda")
    ref, sta = bm.BatchMaxCache(cfg), bm.BatchMaxCache(cfg)
    tol = 0.0   # same kernels, same inputs, only the scratch location differs: results are bit-identical
    for call, pos0 in enumerate(range(0, wl.s, wl.B)):        # three calls in a row through the C ABI
        q, k, v = inp.block(0, pos0, wl.B)
        o_ref = ref.prefill_block(q, k, v, pos0, evict_to=wl.K)
        o_sta = sta.prefill_block_static(q, k, v, pos0, evict_to=wl.K)
        torch.cuda.synchronize()
        assert float((o_ref.float() - o_sta.float()).abs().max()) <= tol, f"outputs differ on call {call}"
        for s in range(wl.b):
            for h in range(wl.Hkv):
                a, b_ = ref.export(0, s, h, rows=True), sta.export(0, s, h, rows=True)
                for x, y in zip(a, b_):
                    assert torch.equal(x, y), f"cache state differs on call {call}, unit ({s},{h})"
    assert ref.length() == sta.length() == (wl.K, wl.s - 1)
    assert sta.status() == 0


def test_static_scratch_rejects_oversized_calls():
    # nsamples * Hq * I = 40 * 32 * 1024 exceeds the built-in array: refused before anything is enqueued
    wl = Workload("too_big", b=40, Hq=32, Hkv=8, d=64, dtype="bf16", s=1024, B=1024, K=64, steps=0)
    cfg = make_config(wl)
    cache = bm.BatchMaxCache(cfg)
    q = torch.zeros(wl.b, wl.B, wl.Hq, wl.d, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(wl.b, wl.B, wl.Hkv, wl.d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bm.BMError) as e:
        cache.prefill_block_static(q, kv, kv, 0, evict_to=wl.K)
    assert e.value.code == 3
    assert cache.length() == (0, -1)
