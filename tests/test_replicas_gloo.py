"""The multi-GPU form of the benchmark is "replicas only": every rank runs its own prefill and the
only cross-rank step is the MAX of the step times.  That host logic is exercised here with two gloo
ranks on CPU, and the reference arm's rank rule (rank 0 works, the others exit) is checked too."""
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")       # rank 1 is the slow replica
    out[rank] = (ms, bench.whole_job_value(3376, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_step_time_is_the_max_over_replicas_and_value_is_the_aggregate():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, 29731, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0
    assert abs(res[0][1] - 2 * 3376 / 15e-3) < 1e-6
    import bench
    assert bench.max_over_ranks(7.0, 1, "cpu") == 7.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
