"""Named workloads and their seeded synthetic inputs.

This module only describes shapes and draws random Q/K/V tensors; it contains none of the method's
arithmetic (no attention, no scores, no eviction).  The same bits feed the CUDA path and the test
oracle.  The inputs stand in for the paper's long-prompt / short-generation tasks (Sec. 4): i.i.d.
N(0, 1) queries, keys and values plus a few "heavy" key positions per (sample, kv-head) that every
query of the head group is biased towards, so that eviction has a signal to find.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    b: int          # batch
    Hq: int
    Hkv: int
    d: int
    dtype: str      # "f32" | "bf16"
    s: int          # prompt length
    B: int          # prefill block
    K: int          # kv_max: size a cache is cut back to
    steps: int      # decode steps
    L: int = 1      # independent layers
    seed: int = 0
    heavy: str = "uniform"        # "uniform" | "zipf"
    heavy_count: int = 8          # heavy draws per (sample, kv-head)
    recency: int = 0              # keys in the last `recency` positions of each block get +1.0*u
    p_dec: int = 1                # decode growth above K between evictions

    @property
    def g(self) -> int:
        return self.Hq // self.Hkv

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _pct(s):  # 1 % of the prompt positions
    return max(1, round(0.01 * s))


WORKLOADS = {
    # tiny single layer, fp32, 8 heavy positions per head
    "cfg1": Workload("cfg1", b=2, Hq=4, Hkv=4, d=64, dtype="f32", s=512, B=64, K=128, steps=16, seed=0,
                     heavy_count=8),
    # Llama-3-8B attention shape (GQA 4:1), 1 % heavy positions, 64-token recency bias
    "cfg2": Workload("cfg2", b=16, Hq=32, Hkv=8, d=128, dtype="bf16", s=4096, B=256, K=512, steps=128, seed=1,
                     heavy_count=_pct(4096), recency=64),
    # summarisation-style long prompt; batch swept up to what fits a 40 GiB arena
    "cfg3": Workload("cfg3", b=16, Hq=32, Hkv=8, d=128, dtype="bf16", s=8192, B=512, K=1024, steps=64, seed=2,
                     heavy_count=_pct(8192)),
    # 32 independent layers; batch = max fitting 120 GiB of caches
    "cfg4": Workload("cfg4", b=16, Hq=32, Hkv=8, d=128, dtype="bf16", s=4096, B=512, K=512, steps=64, L=32, seed=3,
                     heavy_count=_pct(4096)),
    # Llama-2-7B-shaped MHA, Zipf(1.1) heavy positions; (B, K) swept by the tests
    "cfg5": Workload("cfg5", b=32, Hq=32, Hkv=32, d=128, dtype="bf16", s=16384, B=1024, K=1024, steps=256, seed=4,
                     heavy="zipf", heavy_count=_pct(16384)),
}
CFG5_SWEEP = [(B, K) for B in (1024, 2048) for K in (256, 1024, 2048)]


def _gen(device, *parts) -> torch.Generator:
    seed = 0x9E3779B97F4A7C15
    for p in parts:
        seed = (seed * 6364136223846793005 + int(p) + 1442695040888963407) % (1 << 63)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


class Inputs:
    """Seeded Q/K/V stream of one workload on one device.

    ``block(layer, pos0, I)`` returns q (ns, I, Hq, d), k, v (ns, I, Hkv, d) in the workload dtype for the
    sample range; the values depend only on (seed, layer, pos0, I, sample index, device type), never on
    call order or on how the batch is cut into ranges.  A decode step is a block with I = 1.
    """

    CHUNK = 16   # samples per independently seeded chunk (lets huge batches be drawn piecewise)

    def __init__(self, wl: Workload, device="cpu"):
        self.wl = wl
        self.device = torch.device(device)
        self._layer_cache = {}

    def _layer_consts(self, layer: int):
        if layer in self._layer_cache:
            return self._layer_cache[layer]
        wl = self.wl
        g = _gen("cpu", wl.seed + layer, 7)
        u = torch.randn(wl.Hkv, wl.d, generator=g)
        u = u / u.norm(dim=-1, keepdim=True)
        total = wl.s + wl.steps
        if wl.heavy == "zipf":
            # rank r ~ Zipf(1.1) truncated to the prompt, heavy position r - 1 (duplicates collapse)
            ranks = torch.arange(1, wl.s + 1, dtype=torch.float64)
            prob = ranks.pow(-1.1)
            pos = torch.multinomial(prob / prob.sum(), wl.b * wl.Hkv * wl.heavy_count, replacement=True, generator=g)
            pos = pos.view(wl.b, wl.Hkv, wl.heavy_count)
        else:
            pos = torch.randint(0, wl.s, (wl.b, wl.Hkv, wl.heavy_count), generator=g)
        mask = torch.zeros(wl.b, wl.Hkv, total, dtype=torch.bool)
        mask.scatter_(2, pos, True)
        out = (u.to(self.device), mask.to(self.device))
        self._layer_cache = {layer: out}   # keep one layer resident
        return out

    def heavy_mask(self, layer: int = 0):
        return self._layer_consts(layer)[1]

    def block(self, layer: int, pos0: int, I: int, sample0: int = 0, nsamples: int | None = None):
        wl = self.wl
        ns = wl.b - sample0 if nsamples is None else nsamples
        u, mask = self._layer_consts(layer)
        dev = self.device
        qs, ks, vs = [], [], []
        c0, c1 = sample0 // self.CHUNK, (sample0 + ns - 1) // self.CHUNK
        for c in range(c0, c1 + 1):      # values are drawn per chunk of CHUNK samples
            gen = _gen(dev, wl.seed + layer, 11, pos0, I, c)
            qs.append(torch.randn(self.CHUNK, I, wl.Hq, wl.d, generator=gen, device=dev))
            ks.append(torch.randn(self.CHUNK, I, wl.Hkv, wl.d, generator=gen, device=dev))
            vs.append(torch.randn(self.CHUNK, I, wl.Hkv, wl.d, generator=gen, device=dev))
        lo = sample0 - c0 * self.CHUNK
        q = (qs[0] if len(qs) == 1 else torch.cat(qs))[lo:lo + ns]
        k = (ks[0] if len(ks) == 1 else torch.cat(ks))[lo:lo + ns]
        v = (vs[0] if len(vs) == 1 else torch.cat(vs))[lo:lo + ns]
        # every query of a group leans towards its kv-head's direction u; heavy keys carry +3u
        q = q + 0.5 * u.repeat_interleave(wl.g, dim=0)[None, None]
        hm = mask[sample0:sample0 + ns, :, pos0:pos0 + I].permute(0, 2, 1)            # (ns, I, Hkv)
        k = k + 3.0 * hm[..., None].to(k.dtype) * u[None, None]
        if wl.recency > 0:
            p = torch.arange(pos0, pos0 + I, device=dev)
            near_end = ((p % wl.B) >= wl.B - wl.recency) & (p < wl.s)
            k = k + near_end[None, :, None, None].to(k.dtype) * u[None, None]
        td = wl.torch_dtype
        return q.to(td).contiguous(), k.to(td).contiguous(), v.to(td).contiguous()


def schedule(wl: Workload):
    """The north-star schedule as a list of calls: ("prefill", pos0, I, evict_to) for every prompt block
    (ragged tail allowed, cache cut back to K after each) and ("decode", pos, 1, evict_to) for every
    generated token (cut back to K whenever the cache has grown to K + p_dec, else -1)."""
    calls = []
    n = 0
    pos = 0
    while pos < wl.s:
        I = min(wl.B, wl.s - pos)
        calls.append(("prefill", pos, I, wl.K))
        n = min(n + I, wl.K)
        pos += I
    for t in range(wl.steps):
        full = n + 1 >= wl.K + wl.p_dec
        calls.append(("decode", wl.s + t, 1, wl.K if full else -1))
        n = wl.K if full else n + 1
    return calls


def config_for(wl: Workload, device: int = 0, growth: int | None = None, batch: int | None = None,
               max_call_samples: int = 0, rule: str = "average", compaction: str = "stable", **rule_params):
    """The library configuration of a workload in the build's cadence (cap = kv_max + growth)."""
    from .binding import Config
    return Config(batch=wl.b if batch is None else batch, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.d,
                  kv_max=wl.K, block_max=wl.B, growth=max(1, wl.p_dec) if growth is None else growth,
                  dtype=wl.dtype, n_layers=wl.L, device=device, max_call_samples=max_call_samples, rule=rule,
                  compaction=compaction, **rule_params)   # window / pool / std_share of the rules that take them
