"""Multi-rank logic of the benchmark (replicas only: no data-path collective), on CPU with gloo:
every rank contributes its own device times, the job's time is the maximum, the job's
throughput the sum of all ranks' bytes over that time."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 5.0 - rank, 1.0]
    got = bench.max_over_ranks(mine, torch.device("cpu"), world)
    dist.barrier()
    q.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_world_2():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [11.0, 5.0, 1.0]


def test_single_rank_and_throughput():
    import bench
    assert bench.max_over_ranks([3.0, 4.0], torch.device("cpu"), 1) == [3.0, 4.0]
    # 4 replicas, 2 GB each, slowest takes 1 ms -> 8 GB / ms = 8000 GB/s
    assert abs(bench.whole_job_gbs(2e9, 1.0, 4) - 8000.0) < 1e-9


def test_plain_gpus_2_starts_two_ranks_that_meet():
    """`python bench.py --gpus 2` with no rank variables in the environment starts its two ranks
    itself; with --rendezvous-check they form the process group on CPU, reduce stub timings with the
    same max-over-ranks code as the real run and rank 0 prints one line."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rendezvous-check"],
                       capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                              # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["requested_gpus"] == 2
    assert line["ms_max_over_ranks"] == 11.0            # the slower rank's time
    assert abs(line["value"] - 2 * 1e9 / (11.0 * 1e6)) < 1e-9


def test_spawn_command_is_one_rank_per_gpu_on_localhost():
    import bench
    cmd = bench.spawn_command(4, ["--gpus", "4", "--steps", "2"])
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"]
