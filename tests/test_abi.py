"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its host logic
(memory model, allocator arithmetic, argument validation) behaves as the header states."""
import ctypes as C
import os
import re

import pytest

import paper_2412_05693_b200 as bm
from paper_2412_05693_b200 import binding
from paper_2412_05693_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GiB = 2 ** 30


@pytest.fixture(scope="module", autouse=True)
def built():
    build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "batchmax.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bm_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 18
    h = C.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(h, n), f"{n} declared in batchmax.h but not exported"
    assert set(names) == set(binding.SIGNATURES), "binding and header disagree on the entry points"


def test_checked_build_exports_the_same_symbols_and_charges_its_guards():
    # libbatchmax_debug.so: same entry points; its arena header holds a 256-byte guard behind every slab
    h = C.CDLL(build(debug=True))
    for n in declared_symbols():
        assert hasattr(h, n), f"{n} missing from the checked build"
    h.bm_debug_build.restype = C.c_int32
    assert h.bm_debug_build() == 1 and bm.lib().bm_debug_build() == 0
    cfg = llama_cfg().c()
    need = C.c_size_t(0)
    h.bm_arena_bytes.argtypes = [C.POINTER(binding.bm_config_t), C.POINTER(C.c_size_t)]
    assert h.bm_arena_bytes(C.byref(cfg), C.byref(need)) == 0
    assert need.value == 4096 + 16 * 8 * 1025 * 520
    # the memory model also charges the rule that keeps a second accumulator per row
    assert bm.cache_bytes_per_sample(llama_cfg(rule="average_std")) == 8 * 1025 * (2 * 128 * 2 + 12)


def llama_cfg(**kw):
    base = dict(batch=16, n_q_heads=32, n_kv_heads=8, head_dim=128, kv_max=1024, block_max=512, growth=1)
    base.update(kw)
    return bm.Config(**base)


def test_memory_model_formula():
    # bytes/sample = L * Hkv * cap * (2 d e + 8)
    assert bm.cache_bytes_per_sample(llama_cfg()) == 8 * 1025 * (2 * 128 * 2 + 8)
    assert bm.cache_bytes_per_sample(llama_cfg(dtype="f32", head_dim=64, n_layers=3)) == 3 * 8 * 1025 * (2 * 64 * 4 + 8)
    assert bm.arena_bytes(llama_cfg()) == 1024 + 16 * 8 * 1025 * 520


def test_max_batch_under_budget_and_pd_vs_decode_only_ratio():
    # 40 GiB arena, s = 8192, K = 1024: P&D caches hold K + G rows, decode-only compression holds s + G rows
    pd = bm.max_batch(llama_cfg(), 40 * GiB)
    do = bm.max_batch(llama_cfg(growth=8192 + 1 - 1024), 40 * GiB)
    assert (pd, do) == (10072, 1260)
    assert pd / do == pytest.approx((8192 + 1) / (1024 + 1), rel=2e-3)      # ratio the memory model predicts
    assert bm.max_batch(llama_cfg(growth=64), 40 * GiB) == 9489
    # 32 layers in 120 GiB (K = 512)
    assert bm.max_batch(llama_cfg(kv_max=512, n_layers=32), 120 * GiB) == 1886
    # the returned batch fits and one more sample does not
    cfg = llama_cfg()
    for budget in (3 * GiB + 12345, 40 * GiB):
        b = bm.max_batch(cfg, budget)
        assert bm.arena_bytes(llama_cfg(batch=b)) <= budget < bm.arena_bytes(llama_cfg(batch=b + 1))
    assert bm.max_batch(cfg, 100) == 0


def test_workspace_and_staging_sizes():
    cfg = llama_cfg(max_call_samples=4)
    # log-sum-exp of the query rows + column sums of the new pairs (per call) + one padding count per sample
    assert bm.workspace_bytes(cfg) == 4 * (4 * 32 * 512 + 4 * 8 * 512) + 256
    assert binding.staging_bytes(cfg, 2, 512) == 2 * (2 * 512 * 32 * 128 * 2) + 2 * (2 * 512 * 8 * 128 * 2)


@pytest.mark.parametrize("bad", [dict(n_kv_heads=5), dict(head_dim=96), dict(kv_max=0), dict(growth=0),
                                 dict(block_max=0), dict(n_q_heads=24, n_kv_heads=8), dict(n_layers=0),
                                 dict(softmax_scale=-1.0)])
def test_invalid_configs_are_rejected(bad):
    with pytest.raises(bm.BMError) as e:
        bm.cache_bytes_per_sample(llama_cfg(**bad))
    assert e.value.code == 1


def test_null_handles_and_arguments_return_invalid_without_touching_cuda():
    L = bm.lib()
    n = C.c_int32(0)
    assert L.bm_cache_len(None, 0, 0, C.byref(n), None) == 1
    assert L.bm_cache_destroy(None) == 1
    assert L.bm_evict(None, 0, 0, 1, 4, None) == 1
    assert L.bm_prefill_block(None, 0, 0, 1, None, None, None, 1, 0, None, -1, None) == 1
    assert L.bm_decode_step(None, 0, 0, 1, None, None, None, None, -1, None) == 1
    cfg = llama_cfg().c()
    h = C.c_void_p(None)
    assert L.bm_cache_create(C.byref(cfg), None, 1 << 30, None, 1 << 20, None, C.byref(h)) == 1
    # misaligned arena
    assert L.bm_cache_create(C.byref(cfg), C.c_void_p(0x1001), 1 << 40, C.c_void_p(0x1000), 1 << 30, None,
                             C.byref(h)) == 1
    # arena too small is reported before any CUDA call
    assert L.bm_cache_create(C.byref(cfg), C.c_void_p(0x1000), 4096, C.c_void_p(0x2000), 1 << 30, None,
                             C.byref(h)) == 2
    assert L.bm_status_string(3).decode().startswith("cache capacity")
    assert L.bm_kernel_launch_count() == 0


def test_binding_fails_loudly_without_the_library(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libbatchmax.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2412_05693_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "workloads.py", f
    assert "import oracle" not in open(os.path.join(pkg, "workloads.py")).read()


def test_benchmark_reaches_the_oracle_only_in_its_cpu_legs():
    # importing the benchmark (and everything its GPU arm imports at module level) must not load the oracle;
    # the oracle is imported inside the CPU-baseline / reference-arm function only
    import subprocess
    import sys
    code = ("import sys; sys.path.insert(0, %r); import bench, paper_2412_05693_b200, "
            "paper_2412_05693_b200.workloads, paper_2412_05693_b200.experiments; "
            "assert not any(m == 'oracle' or m.startswith('oracle.') for m in sys.modules), 'oracle imported'; "
            "assert not any(m.startswith('tests') for m in sys.modules), 'tests imported'") % ROOT
    subprocess.run([sys.executable, "-c", code], check=True, cwd=ROOT)
    src = open(os.path.join(ROOT, "bench.py")).read()
    assert src.count("from oracle import") == 1 and "tests.lockstep" not in src
