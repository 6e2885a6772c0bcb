"""The multi-process plumbing of the benchmark on CPU: two gloo ranks."""
import json
import os
import subprocess
import sys

import pytest

torch = pytest.importorskip("torch")

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist

    from paper_2505_07239_b200 import ranks
    from paper_2505_07239_b200 import workloads as wl

    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert ranks.rank_world_local() == (rank, world, rank)
    # every rank draws its own problem: different seeds give different activations and masks
    seed = ranks.rank_seed(1000, rank)
    cfg = wl.CONFIGS["tiny"]
    _, X0, _ = wl.activation_shares(cfg, seed)
    # the slowest rank decides the time
    mx = ranks.max_over_ranks([10.0 + rank, 5.0 - rank])
    dist.barrier()
    out.put((rank, seed, int(X0[0, 0]), mx))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_without_a_collective_and_reduce_times():
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, x0, m0), (r1, s1, x1, m1) = got
    assert (r0, r1) == (0, 1) and s0 != s1 and x0 != x1          # independent problems per rank
    assert m0 == m1 == [11.0, 5.0]                                 # max over ranks, the same on every rank


def test_whole_job_throughput_counts_every_rank():
    from paper_2505_07239_b200 import ranks

    assert ranks.whole_job_throughput(1e9, 1, 10, 100.0) == pytest.approx(1e11)
    assert ranks.whole_job_throughput(1e9, 8, 10, 100.0) == pytest.approx(8e11)
    assert ranks.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]          # no process group: identity


def test_reference_arm_only_rank_zero_prints():
    """`bench.py --impl reference` under a 2-process launch: rank 1 leaves with status 0 and prints nothing."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
