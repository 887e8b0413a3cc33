"""N > 1 is N independent replicas (the path has no exchange step): only the timing reduction is shared.
World-size-2 gloo run on CPU of the helpers bench.py uses for the max-over-ranks time and the whole-job value."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    local_ms = 10.0 + 5.0 * rank            # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, "cpu")
    value = bench.whole_job_value(1000, world, ms)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"ms": ms, "value": value, "world": world}))
    dist.destroy_process_group()
""") % ROOT


def test_two_rank_gloo_reduction(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(SCRIPT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    r = json.loads(line)
    assert r["world"] == 2 and r["ms"] == 15.0                 # slowest rank sets the step time
    assert r["value"] == 2 * 1000 / 15e-3                      # replicas: tokens of both ranks over that time


def test_single_process_helpers():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(100, 4, 2.0) == 4 * 100 / 2e-3
    from paper_2412_05693_b200.workloads import WORKLOADS
    wl = WORKLOADS["cfg2"]
    # useful prefill pairs: 16 blocks of 256 against min(512, 256 t) cached pairs plus the causal triangle
    want = sum(256 * min(512, 256 * t) + 256 * 257 // 2 for t in range(16))
    assert bench.prefill_pairs(wl) == want
    assert bench.workload_tokens(wl) == 16 * (4096 + 128)
