"""Host-side logic of the multi-GPU benchmark path, run as two gloo ranks on the CPU: the
slowest rank's time decides, and the reported value is the whole job's (per-rank units x ranks).
The data path itself has no collective (chunks are independent; every rank owns its batch)."""
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
    per_rank_ms = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]          # rank 1 is slower on the first entry
    got = bench.max_over_ranks(per_rank_ms, torch.device("cpu"), world)
    rate = bench.aggregate_rate(1000, world, got[0] * 1e-3)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"max": got, "rate": rate, "world": world}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_maximum_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["world"] == 2
    assert res["max"] == [15.0, 3.0, 7.0]
    assert abs(res["rate"] - 2 * 1000 / 15e-3) < 1e-6


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "8b",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    res = json.loads(out.stdout.strip().splitlines()[-1])
    assert res["impl"] == "reference" and res["unit"] == "chunks/s" and res["value"] > 0
    assert res["cpu_baseline"]["kind"] == "oracle" and res["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` without a torchrun environment starts two ranks of itself (here on the
    reference arm, which needs no GPU: rank 0 measures and prints, rank 1 exits)."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    env["MASTER_PORT"] = "29547"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--workload", "8b", "--steps", "1", "--warmup", "0"], capture_output=True, text=True,
                         timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                              # one rank prints
    res = json.loads(lines[0])
    assert res["impl"] == "reference" and res["n_gpus"] == 2 and res["ranks_started"] == 2
