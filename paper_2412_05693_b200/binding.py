"""ctypes binding of libbatchmax.so: same names as include/batchmax.h, argument marshalling only.

Device buffers are torch tensors (torch owns device memory and streams); every step of the path runs
inside the library's kernels.  Importing this module without the built library raises on first use.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

_PKG = os.path.dirname(os.path.abspath(__file__))
# BATCHMAX_LIB selects another build of the same library, e.g. the checked one (libbatchmax_debug.so)
LIB_PATH = os.environ.get("BATCHMAX_LIB") or os.path.join(_PKG, "libbatchmax.so")

BM_F32, BM_BF16 = 0, 1
STATUS = {0: "BM_OK", 1: "BM_ERR_INVALID", 2: "BM_ERR_OOM", 3: "BM_ERR_CAPACITY", 4: "BM_ERR_STATE",
          5: "BM_ERR_CUDA", 6: "BM_ERR_TIMEOUT", 7: "BM_ERR_BOUNDS"}


class BMError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().bm_status_string(code).decode() if _lib is not None else ""
        if code == 5 and _lib is not None:
            msg += ": " + lib().bm_last_cuda_error().decode()
        super().__init__(f"{where}: {STATUS.get(code, code)} ({msg})")


class bm_config_t(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_layers", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("kv_max", C.c_int32),
                ("block_max", C.c_int32), ("growth", C.c_int32), ("dtype", C.c_int32),
                ("softmax_scale", C.c_float), ("device", C.c_int32), ("max_call_samples", C.c_int32),
                ("rule", C.c_int32), ("compaction", C.c_int32), ("window", C.c_int32), ("pool", C.c_int32),
                ("std_share_permille", C.c_int32)]


_lib = None
RULES = {"average": 0, "sum_recent": 1, "current_query": 2, "window_pooled": 3, "average_std": 4}

# name -> (restype, argtypes); every symbol include/batchmax.h declares
_vp, _i32, _sz = C.c_void_p, C.c_int32, C.c_size_t
_cfgp = C.POINTER(bm_config_t)
SIGNATURES = {
    "bm_cache_bytes_per_sample": (_i32, [_cfgp, C.POINTER(_sz)]),
    "bm_arena_bytes": (_i32, [_cfgp, C.POINTER(_sz)]),
    "bm_max_batch": (_i32, [_cfgp, _sz, C.POINTER(_i32)]),
    "bm_workspace_bytes": (_i32, [_cfgp, C.POINTER(_sz)]),
    "bm_cache_create": (_i32, [_cfgp, _vp, _sz, _vp, _sz, _vp, C.POINTER(_vp)]),
    "bm_cache_destroy": (_i32, [_vp]),
    "bm_prefill_block": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _i32, _vp, _i32, _vp]),
    "bm_prefill_block_static": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _i32, _vp, _i32, _vp]),
    "bm_decode_step": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _vp]),
    "bm_evict": (_i32, [_vp, _i32, _i32, _i32, _i32, _vp]),
    "bm_keep_most_recent": (_i32, [_vp, _i32, _i32, _i32, _i32, _vp]),
    "bm_cache_set_left_pad": (_i32, [_vp, _vp, _vp]),
    "bm_cache_count_moved_rows": (_i32, [_vp, _i32]),
    "bm_cache_moved_rows": (_i32, [_vp, C.POINTER(C.c_uint64), _i32, _vp]),
    "bm_staging_bytes": (_i32, [_cfgp, _i32, _i32, C.POINTER(_sz)]),
    "bm_prefill_block_host": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _i32, _vp, _i32, _vp, _sz, _vp]),
    "bm_decode_step_host": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _vp, _sz, _vp]),
    "bm_cache_len": (_i32, [_vp, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32)]),
    "bm_cache_export": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, C.POINTER(_i32), _vp]),
    "bm_cache_import": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _vp]),
    "bm_cache_set_len": (_i32, [_vp, _i32, _i32, _i32, _i32]),
    "bm_cache_export_sum_sq": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp]),
    "bm_cache_import_sum_sq": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp]),
    "bm_cache_status": (_i32, [_vp, C.POINTER(_i32), _vp]),
    "bm_cache_clear_status": (_i32, [_vp, _vp]),
    "bm_selftest_wait_timeout": (_i32, [_vp, _vp]),
    "bm_debug_build": (_i32, []),
    "bm_selftest_row_check": (_i32, [_vp, _vp]),
    "bm_cache_check_canaries": (_i32, [_vp, C.POINTER(_i32), _vp]),
    "bm_profile_enable": (_i32, [_i32]),
    "bm_profile_read": (_i32, [_i32, C.POINTER(C.c_float), C.POINTER(_i32)]),
    "bm_kernel_launch_count": (C.c_uint64, []),
    "bm_last_prefill_path": (_i32, []),
    "bm_status_string": (C.c_char_p, [_i32]),
    "bm_last_cuda_error": (C.c_char_p, []),
}


def lib():
    """Load libbatchmax.so (built by ``python -m paper_2412_05693_b200.build``); no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2412_05693_b200.build`; "
                               "there is no CPU fallback")
        h = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(h, name)
            fn.restype, fn.argtypes = res, args
        _lib = h
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise BMError(code, where)


@dataclass
class Config:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    kv_max: int
    block_max: int
    growth: int = 1
    dtype: str = "bf16"          # "bf16" | "f32"
    n_layers: int = 1
    softmax_scale: float = 0.0
    device: int = 0
    max_call_samples: int = 0
    rule: str = "average"        # "average" (the paper's) | "sum_recent" | "current_query" | "window_pooled" | "average_std"
    compaction: str = "stable"   # "stable": rows stay in position order | "fill": unordered, kept pairs never move
    window: int = 32             # window_pooled: queries observed = recent pairs kept
    pool: int = 7                # window_pooled: width of the max-pooling (odd)
    std_share: float = 0.5       # average_std: share of the kept pairs chosen by standard deviation

    def c(self) -> bm_config_t:
        return bm_config_t(self.batch, self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim, self.kv_max,
                           self.block_max, self.growth, BM_BF16 if self.dtype == "bf16" else BM_F32,
                           self.softmax_scale, self.device, self.max_call_samples,
                           RULES[self.rule], {"stable": 0, "fill": 1}[self.compaction], self.window, self.pool,
                           int(round(self.std_share * 1000)))

    @property
    def cap(self) -> int:
        return self.kv_max + self.growth


def _size_query(fn_name: str, cfg: Config) -> int:
    out = _sz(0)
    c = cfg.c()
    _check(getattr(lib(), fn_name)(C.byref(c), C.byref(out)), fn_name)
    return out.value


def cache_bytes_per_sample(cfg: Config) -> int:
    return _size_query("bm_cache_bytes_per_sample", cfg)


def arena_bytes(cfg: Config) -> int:
    return _size_query("bm_arena_bytes", cfg)


def workspace_bytes(cfg: Config) -> int:
    return _size_query("bm_workspace_bytes", cfg)


def max_batch(cfg: Config, hbm_budget_bytes: int) -> int:
    out = _i32(0)
    c = cfg.c()
    _check(lib().bm_max_batch(C.byref(c), hbm_budget_bytes, C.byref(out)), "bm_max_batch")
    return out.value


def staging_bytes(cfg: Config, nsamples: int, I: int) -> int:
    out = _sz(0)
    c = cfg.c()
    _check(lib().bm_staging_bytes(C.byref(c), nsamples, I, C.byref(out)), "bm_staging_bytes")
    return out.value


def debug_build() -> bool:
    """True when the loaded library is the checked build (row-index checks in the kernels, guards behind the slabs)."""
    return bool(lib().bm_debug_build())


def kernel_launch_count() -> int:
    return int(lib().bm_kernel_launch_count())


def last_prefill_path() -> int:
    return int(lib().bm_last_prefill_path())


KERNEL_CLASSES = {"attn_fwd": 0, "score": 1, "evict": 2, "decode": 3}


def profile_pass(fn):
    """Run fn() with per-launch event timing on; returns {kernel class: (total ms, launches)}."""
    L = lib()
    for c in KERNEL_CLASSES.values():      # drop anything recorded earlier
        L.bm_profile_read(c, C.byref(C.c_float()), C.byref(_i32()))
    L.bm_profile_enable(1)
    try:
        fn()
    finally:
        L.bm_profile_enable(0)
    out = {}
    for name, c in KERNEL_CLASSES.items():
        ms, n = C.c_float(0), _i32(0)
        _check(L.bm_profile_read(c, C.byref(ms), C.byref(n)), "bm_profile_read")
        out[name] = (float(ms.value), int(n.value))
    return out


def profile_read():
    """Durations recorded since the last read, {kernel class: (total ms, launches)}; waits for them and forgets them."""
    out = {}
    for name, c in KERNEL_CLASSES.items():
        ms, n = C.c_float(0), _i32(0)
        _check(lib().bm_profile_read(c, C.byref(ms), C.byref(n)), "bm_profile_read")
        out[name] = (float(ms.value), int(n.value))
    return out


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


class BatchMaxCache:
    """Handle of one bm_cache_t plus the torch tensors backing its arena and workspace."""

    def __init__(self, cfg: Config, arena=None, stream=None, workspace=None):
        import torch
        self.cfg = cfg
        self.torch = torch
        dev = torch.device("cuda", cfg.device)
        need = arena_bytes(cfg)
        self.arena = arena if arena is not None else torch.empty(need, dtype=torch.uint8, device=dev)
        self.workspace = workspace if workspace is not None else \
            torch.empty(max(workspace_bytes(cfg), 256), dtype=torch.uint8, device=dev)
        self.tdtype = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        self._staging = None
        h = _vp(None)
        c = cfg.c()
        with torch.cuda.device(dev):
            _check(lib().bm_cache_create(C.byref(c), _ptr(self.arena), self.arena.numel(), _ptr(self.workspace),
                                         self.workspace.numel(), _stream(stream), C.byref(h)), "bm_cache_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None) is not None and self.h:
            lib().bm_cache_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check_out(self, out, q):
        """The library writes `out` with q's layout: a strided view would scatter rows over other samples' slots."""
        assert out.is_contiguous() and out.dtype == self.tdtype and out.shape == q.shape, \
            "out must be a contiguous tensor of q's shape and dtype"

    # -- the four calls of the hot path -------------------------------------------------------------
    def prefill_block(self, q, k, v, pos0: int, out=None, evict_to: int = -1, layer: int = 0, sample0: int = 0,
                      stream=None):
        """q (ns, I, Hq, d), k/v (ns, I, Hkv, d) contiguous device tensors; returns out (ns, I, Hq, d)."""
        ns, I = q.shape[0], q.shape[1]
        assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and q.dtype == self.tdtype
        if out is None:
            out = self.torch.empty_like(q)
        self._check_out(out, q)
        _check(lib().bm_prefill_block(self.h, layer, sample0, ns, _ptr(q), _ptr(k), _ptr(v), I, pos0, _ptr(out),
                                      evict_to, _stream(stream)), "bm_prefill_block")
        return out

    def prefill_block_static(self, q, k, v, pos0: int, out=None, evict_to: int = -1, layer: int = 0,
                             sample0: int = 0, stream=None):
        """bm_prefill_block_static: same pass, scratch taken from the array built into the library (for callers
        that cannot allocate a workspace).  Size limits and sharing rules are in include/batchmax.h."""
        ns, I = q.shape[0], q.shape[1]
        assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and q.dtype == self.tdtype
        if out is None:
            out = self.torch.empty_like(q)
        self._check_out(out, q)
        _check(lib().bm_prefill_block_static(self.h, layer, sample0, ns, _ptr(q), _ptr(k), _ptr(v), I, pos0,
                                             _ptr(out), evict_to, _stream(stream)), "bm_prefill_block_static")
        return out

    def decode_step(self, q, k, v, out=None, evict_to: int = -1, layer: int = 0, sample0: int = 0, stream=None):
        """q (ns, Hq, d), k/v (ns, Hkv, d); returns out (ns, Hq, d)."""
        ns = q.shape[0]
        assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and q.dtype == self.tdtype
        if out is None:
            out = self.torch.empty_like(q)
        self._check_out(out, q)
        _check(lib().bm_decode_step(self.h, layer, sample0, ns, _ptr(q), _ptr(k), _ptr(v), _ptr(out), evict_to,
                                    _stream(stream)), "bm_decode_step")
        return out

    def evict(self, target: int, layer: int = 0, sample0: int = 0, nsamples: int | None = None, stream=None):
        ns = self.cfg.batch - sample0 if nsamples is None else nsamples
        _check(lib().bm_evict(self.h, layer, sample0, ns, target, _stream(stream)), "bm_evict")

    def keep_most_recent(self, keep: int = 1, layer: int = 0, sample0: int = 0, nsamples: int | None = None,
                         stream=None):
        """Algorithm 3's rule: all but the `keep` most recent pairs leave the cache."""
        ns = self.cfg.batch - sample0 if nsamples is None else nsamples
        _check(lib().bm_keep_most_recent(self.h, layer, sample0, ns, keep, _stream(stream)), "bm_keep_most_recent")

    def set_left_pad(self, pads, stream=None):
        """pads[s] = padding positions at the start of sample s (a sequence of cfg.batch ints, or None)."""
        if pads is None:
            _check(lib().bm_cache_set_left_pad(self.h, None, _stream(stream)), "bm_cache_set_left_pad")
            return
        pads = [int(x) for x in pads]
        assert len(pads) == self.cfg.batch
        arr = (C.c_int32 * len(pads))(*pads)
        _check(lib().bm_cache_set_left_pad(self.h, C.cast(arr, C.c_void_p), _stream(stream)),
               "bm_cache_set_left_pad")

    def count_moved_rows(self, on: bool = True):
        _check(lib().bm_cache_count_moved_rows(self.h, 1 if on else 0), "bm_cache_count_moved_rows")

    def moved_rows(self, reset: bool = False, stream=None) -> int:
        out = C.c_uint64(0)
        _check(lib().bm_cache_moved_rows(self.h, C.byref(out), 1 if reset else 0, _stream(stream)), "bm_cache_moved_rows")
        return int(out.value)

    # -- host-fed variants ---------------------------------------------------------------------------
    def _stage(self, ns, I):
        """Four staging buffers used in turn, so that consecutive host-fed calls overlap their copies and passes."""
        need = staging_bytes(self.cfg, ns, I)
        if self._staging is None or self._staging[0].numel() < need:
            dev = self.torch.device("cuda", self.cfg.device)
            self._staging = [self.torch.empty(need, dtype=self.torch.uint8, device=dev) for _ in range(4)]
            self._stage_turn = 0
        self._stage_turn = (self._stage_turn + 1) % 4
        return self._staging[self._stage_turn]

    def prefill_block_host(self, q, k, v, pos0: int, out, evict_to: int = -1, layer: int = 0, sample0: int = 0,
                           stream=None):
        """Same pass with q/k/v/out in (pinned) host memory; copies are inside the call."""
        ns, I = q.shape[0], q.shape[1]
        st = self._stage(ns, I)
        _check(lib().bm_prefill_block_host(self.h, layer, sample0, ns, _ptr(q), _ptr(k), _ptr(v), I, pos0, _ptr(out),
                                           evict_to, _ptr(st), st.numel(), _stream(stream)), "bm_prefill_block_host")
        return out

    def decode_step_host(self, q, k, v, out, evict_to: int = -1, layer: int = 0, sample0: int = 0, stream=None):
        ns = q.shape[0]
        st = self._stage(ns, 1)
        _check(lib().bm_decode_step_host(self.h, layer, sample0, ns, _ptr(q), _ptr(k), _ptr(v), _ptr(out), evict_to,
                                         _ptr(st), st.numel(), _stream(stream)), "bm_decode_step_host")
        return out

    # -- state ----------------------------------------------------------------------------------------
    def length(self, layer: int = 0, sample: int = 0):
        n, cur = _i32(0), _i32(0)
        _check(lib().bm_cache_len(self.h, layer, sample, C.byref(n), C.byref(cur)), "bm_cache_len")
        return n.value, cur.value

    def set_len(self, n: int, curr_id: int, layer: int = 0, sample: int = 0):
        _check(lib().bm_cache_set_len(self.h, layer, sample, n, curr_id), "bm_cache_set_len")

    def export(self, layer: int = 0, sample: int = 0, kv_head: int = 0, rows: bool = False, stream=None):
        """Returns (kv_ids int32[n], sum_weights float32[n], k_rows, v_rows) as CPU tensors."""
        torch = self.torch
        n0, _ = self.length(layer, sample)
        ids = torch.empty(max(n0, 1), dtype=torch.int32)
        sw = torch.empty(max(n0, 1), dtype=torch.float32)
        kr = torch.empty(max(n0, 1), self.cfg.head_dim, dtype=self.tdtype) if rows else None
        vr = torch.empty(max(n0, 1), self.cfg.head_dim, dtype=self.tdtype) if rows else None
        n = _i32(0)
        _check(lib().bm_cache_export(self.h, layer, sample, kv_head, _ptr(ids), _ptr(sw), _ptr(kr), _ptr(vr),
                                     C.byref(n), _stream(stream)), "bm_cache_export")
        cut = lambda t: None if t is None else t[: n.value]
        return cut(ids), cut(sw), cut(kr), cut(vr)

    def import_(self, ids, sw, kr, vr, layer: int = 0, sample: int = 0, kv_head: int = 0, stream=None):
        ids, sw, kr, vr = (t.contiguous() for t in (ids, sw, kr, vr))   # kept alive until the call has returned
        _check(lib().bm_cache_import(self.h, layer, sample, kv_head, _ptr(ids), _ptr(sw), _ptr(kr), _ptr(vr),
                                     ids.shape[0], _stream(stream)), "bm_cache_import")

    def export_sum_sq(self, layer: int = 0, sample: int = 0, kv_head: int = 0, stream=None):
        """Sums of squared attention weights of one cache (rule "average_std"), float32[n] on the CPU."""
        n0, _ = self.length(layer, sample)
        sq = self.torch.empty(max(n0, 1), dtype=self.torch.float32)
        _check(lib().bm_cache_export_sum_sq(self.h, layer, sample, kv_head, _ptr(sq), _stream(stream)),
               "bm_cache_export_sum_sq")
        return sq[:n0]

    def import_sum_sq(self, sq, layer: int = 0, sample: int = 0, kv_head: int = 0, stream=None):
        sq = sq.contiguous()
        _check(lib().bm_cache_import_sum_sq(self.h, layer, sample, kv_head, _ptr(sq), _stream(stream)),
               "bm_cache_import_sum_sq")

    def selftest_row_check(self, stream=None):
        """Enqueue the row-test self-test: in the checked build status() then reports 7 (BM_ERR_BOUNDS)."""
        _check(lib().bm_selftest_row_check(self.h, _stream(stream)), "bm_selftest_row_check")

    def check_canaries(self, stream=None) -> int:
        """Number of damaged guards behind the arena's slabs (always 0 in the ordinary build, which has none)."""
        bad = _i32(0)
        _check(lib().bm_cache_check_canaries(self.h, C.byref(bad), _stream(stream)), "bm_cache_check_canaries")
        return bad.value

    def clear_status(self, stream=None):
        _check(lib().bm_cache_clear_status(self.h, _stream(stream)), "bm_cache_clear_status")

    def selftest_wait_timeout(self, stream=None):
        """Enqueue the bounded-wait self-test: afterwards status() reports 6 (BM_ERR_TIMEOUT)."""
        _check(lib().bm_selftest_wait_timeout(self.h, _stream(stream)), "bm_selftest_wait_timeout")

    def status(self, stream=None) -> int:
        w = _i32(0)
        _check(lib().bm_cache_status(self.h, C.byref(w), _stream(stream)), "bm_cache_status")
        return w.value
