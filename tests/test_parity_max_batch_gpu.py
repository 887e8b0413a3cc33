"""GPU parity at the batch sizes the metric is quoted on: the largest batch whose caches fill a fixed HBM budget
(Sec. 1: the batch a memory budget admits is the method's point), issued range by range (`sample0, nsamples`) as a
caller with a batch this large has to, with inputs drawn on the fly per range.  Sampled caches at the first, a middle
and the last sample (slab offsets beyond 2^32 bytes, last rows of the arena) run in lock-step against the fp64
oracle: kept sets, outputs, sum_weights, cached rows.  The prompts are shortened so that a case stays well under a
minute; shapes, block size, kv_max, batch, arena size and call pattern are the full configuration's."""
import pytest
import torch

import paper_2412_05693_b200 as bm
from paper_2412_05693_b200.workloads import WORKLOADS
from tests.lockstep import make_config, run_lockstep

pytestmark = pytest.mark.gpu
GiB = 2 ** 30
PREFILL_MICRO, DECODE_MICRO = 256, 2048     # samples per call, as the benchmark issues them


def _arena_for(wl, budget):
    cfg = make_config(wl, max_call_samples=min(wl.b, DECODE_MICRO))
    need = bm.arena_bytes(cfg)
    assert need <= budget
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < need + 24 * GiB:
        pytest.skip(f"needs {need / GiB:.0f} GiB of free device memory for the arena plus inputs")
    return torch.empty(need, dtype=torch.uint8, device="cuda")


@pytest.mark.parametrize("compaction", ["stable", "fill"])
def test_cfg3_at_the_batch_that_fills_40_gib(compaction):
    wl = WORKLOADS["cfg3"].with_(s=2048, steps=4)
    b = bm.max_batch(make_config(wl, batch=1), 40 * GiB)
    assert b == 10072                                   # (40 GiB - header) / (8 heads * 1025 rows * 520 B)
    wl = wl.with_(b=b)
    arena = _arena_for(wl, 40 * GiB)
    assert arena.numel() > 2 ** 32                      # offsets into the slabs do not fit 32 bits
    units = [(0, 0), (0, 7), (b // 2, 3), (b // 2 + 1, 4), (b - 1, 0), (b - 1, 7)]
    st = run_lockstep(wl, units, check_rows_every=2, compaction=compaction, micro=PREFILL_MICRO,
                      micro_dec=DECODE_MICRO, arena=arena)
    assert st["evictions"] == (2 + 4) * len(units) and st["tc_calls"] > 0
    del arena
    torch.cuda.empty_cache()


def test_cfg4_at_the_batch_that_fills_120_gib_with_32_layers_in_one_arena():
    wl = WORKLOADS["cfg4"].with_(s=1536, steps=4)
    b = bm.max_batch(make_config(wl, batch=1), 120 * GiB)
    assert b == 1886                                    # 32 layers * 8 heads * 513 rows * 520 B per sample
    wl = wl.with_(b=b)
    arena = _arena_for(wl, 120 * GiB)
    cfg = make_config(wl, max_call_samples=min(b, DECODE_MICRO))
    cache = bm.BatchMaxCache(cfg, arena=arena)
    units = [(0, 0), (b // 2, 5), (b - 1, 7)]
    for layer in (0, 13, 31):                           # first, a middle and the last layer's slabs
        st = run_lockstep(wl, units, layer=layer, check_rows_every=2, micro=PREFILL_MICRO, micro_dec=DECODE_MICRO,
                          cache=cache)
        assert st["evictions"] == (2 + 4) * len(units)
    # the layers in between were never touched: still empty
    assert cache.length(layer=1, sample=b - 1) == (0, -1)
    cache.close()
    del arena
    torch.cuda.empty_cache()
