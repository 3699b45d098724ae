"""The N > 1 plumbing of bench.py on CPU: two `gloo` ranks.

The path shards by batch/head with no data-path collective, so the only multi-rank logic is the
barrier, the max-over-ranks time and the whole-job value; the reference arm runs on rank 0 alone."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    dist.barrier()
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(torch, dist, ms_local, torch.device("cpu"))
    value = bench.whole_job_value(world, 1000, ms / 4)
    print(json.dumps({"rank": rank, "ms": ms, "value": value}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = [json.loads(p.communicate(timeout=120)[0].strip().splitlines()[-1]) for p in procs]
    assert all(p.returncode == 0 for p in procs)
    for o in outs:
        assert o["ms"] == 15.0                                   # max over ranks, on every rank
        assert abs(o["value"] - 2 * 1000 / (15.0 / 4 * 1e-3)) < 1e-6  # all ranks' units / slowest time


def test_reference_arm_runs_on_rank_zero_only():
    env1 = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r1 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "0"], env=env1, capture_output=True, text=True, timeout=120)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    r0 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "0"], env=env0, capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["metric"] == "linear_attn_tokens_heads_per_s"
