"""The N > 1 path of bench.py on CPU: the hot path has no exchange step, so ranks run independent
replicas and only the timing is reduced (MAX over ranks).  Two gloo ranks exercise that host logic;
the reference arm is checked for "rank 0 alone works and prints"."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r measured (10 + r) ms for the device-resident steps and (100 - r) ms end to end
    total_ms, e2e_ms = bench.reduce_over_ranks(dist, [10.0 + rank, 100.0 - rank], torch.device("cpu"))
    dist.barrier()
    Path(out_dir, f"rank{rank}.json").write_text(json.dumps({"total_ms": total_ms, "e2e_ms": e2e_ms}))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_rank_time(tmp_path):
    world, port = 2, 29500 + os.getpid() % 500
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in range(world)]
    assert got[0] == got[1] == {"total_ms": 11.0, "e2e_ms": 100.0}


def test_job_value_counts_every_replica():
    import bench

    one = bench.job_value(1, 2.0e12, 5, 10.0)    # 5 steps of 2 TFLOP in 10 ms
    assert abs(one - 1000.0) < 1e-9
    assert abs(bench.job_value(8, 2.0e12, 5, 10.0) - 8 * one) < 1e-9   # weak scaling: 8 replicas, same time
    assert bench.reduce_over_ranks(None, [3.0, 4.0], torch.device("cpu")) == [3.0, 4.0]


def _run_bench(extra_env, *args):
    env = dict(os.environ, **extra_env)
    return subprocess.run([sys.executable, str(ROOT / "bench.py"), *args], capture_output=True, text=True, env=env,
                          timeout=600)


def test_reference_arm_rank0_prints_and_other_ranks_stay_silent():
    args = ("--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0", "--gpus", "2")
    r1 = _run_bench({"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"}, *args)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = _run_bench({"RANK": "0", "WORLD_SIZE": "2", "LOCAL_RANK": "0"}, *args)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
