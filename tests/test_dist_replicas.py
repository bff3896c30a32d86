"""The N > 1 path of the benchmark is 'independent replicas + max time / summed rows': checked with two gloo ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_06412_b200 import dist_util


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert dist_util.env_rank_world() == (rank, world, rank)
        ms = [10.0, 25.0][rank]                      # rank 1 is the slow replica
        rows = [300, 500][rank]                      # ragged work per replica
        tput, worst = dist_util.job_throughput(rows, ms)
        seeds = [dist_util.replica_seed(7, r) for r in range(world)]
        out.put((rank, tput, worst, dist_util.max_over_ranks(float(rank)), dist_util.sum_over_ranks(1.0), seeds))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_max_time_and_summed_rows():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    ps = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in ps:
        p.start()
    res = sorted(out.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, tput, worst, mx, sm, seeds in res:
        assert worst == 25.0                         # the job is as slow as its slowest rank
        assert abs(tput - 800 / 0.025) < 1e-6        # all rows of all replicas / that time
        assert mx == 1.0 and sm == 2.0
        assert len(set(seeds)) == 2                  # replicas do not run identical streams


def test_single_process_passthrough():
    assert dist_util.max_over_ranks(3.5) == 3.5 and dist_util.sum_over_ranks(2.0) == 2.0
    assert dist_util.job_throughput(100, 50.0) == (2000.0, 50.0)


def test_bench_starts_its_own_ranks_when_asked_for_more_than_one_gpu():
    """`python bench.py --gpus 2` without a launcher starts two ranks itself (torch.distributed.run, rendezvous on
    127.0.0.1).  Run here on the CPU-only reference arm: rank 0 alone does the work and prints the one JSON line, which
    names two ranks; the other rank leaves with exit code 0."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload",
                        "tiny", "--steps", "1", "--warmup", "0"], capture_output=True, text=True, cwd=root, timeout=600,
                       env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0


def test_bench_with_more_ranks_than_gpus_fails_loudly():
    """The library arm with two ranks on a box that shows fewer than two GPUs ends with a non-zero exit code and says
    why (here: no CUDA device at all, or a single one)."""
    import subprocess
    import sys
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        return
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--workload", "tiny", "--steps", "1",
                        "--warmup", "0", "--no-cpu-baseline", "--sampler-steps", "0", "--ratios", ""], capture_output=True,
                       text=True, cwd=root, timeout=600, env=env)
    assert r.returncode != 0
    assert "CUDA device" in r.stderr or "GPU" in r.stderr
