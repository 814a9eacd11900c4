"""The N > 1 path of bench.py (independent replicas, max-over-ranks timing) on CPU with gloo, world size 2."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slow replica: every rank must end up with ITS timings
    mine = [10.0 + 5.0 * rank, 20.0 - 3.0 * rank, 1.0]
    got = bench.max_over_ranks(mine, dist, "cpu")
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_rate_world2():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        for r in range(world):
            assert out[r] == [15.0, 20.0, 1.0]
    sys.path.insert(0, ROOT)
    import bench
    # two replicas of batch 4 doing 512 steps in 12.8 s -> 320 tokens/s for the whole job
    assert abs(bench.aggregate_rate(2, 4, 512, 12800.0) - 320.0) < 1e-9
    assert bench.max_over_ranks([3.0, 4.0], None, "cpu") == [3.0, 4.0]


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    import json
    import subprocess
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself (torch.distributed.run on
    127.0.0.1); here in the CPU self-test mode (gloo, made-up timings, the real max-over-ranks reduction)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "10", "--selftest-cpu"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms"] == 200.0           # the slower rank's time
    assert abs(line["value"] - 2 * 4 * 10 / 0.2) < 1e-9
