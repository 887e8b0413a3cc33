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


def test_gpus_flag_starts_the_ranks_itself():
    # `python bench.py --gpus 2` with no launcher around it: the script starts two ranks under torch's launcher,
    # rank 0 prints one line that counts both replicas and carries the slower rank's step time
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--cpu-stub", "--steps", "5",
                          "--warmup", "1"], capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    r = json.loads(lines[0])
    assert r["n_gpus"] == 2 and r["config"]["parallelism"] == "replicas x2"
    assert r["ms_per_step"] >= 4.0                              # rank 1's replica sleeps 4 ms per step, rank 0's 2 ms
    assert abs(r["value"] - 2 * 1000 / (r["ms_per_step"] * 1e-3)) < 1e-6 * r["value"]
    # the same stub on one rank: no launcher, n_gpus 1
    one = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--cpu-stub", "--steps", "3", "--warmup", "1"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert one.returncode == 0 and json.loads(one.stdout.splitlines()[-1])["n_gpus"] == 1


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
    # decode bytes of one cache: 128 steps over 513 rows of 2*128*2 + 16 bytes, the appended pair, q and out (g = 4)
    from paper_2412_05693_b200.workloads import schedule
    assert bench.decode_bytes_per_cache(wl, schedule(wl)) == 128 * (513 * (512 + 16) + 512 + 2 * 4 * 256)
