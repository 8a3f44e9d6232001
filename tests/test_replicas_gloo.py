"""The N > 1 path is replicas only: what crosses ranks is the timing reduction.  Exercised here with two CPU processes
over gloo (no GPU): both ranks must get the slowest rank's time, the whole-job rate counts every rank's units, only
rank 0 reports, and the CPU reference arm does nothing on other ranks."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2604_06832_b200 import replicas as R
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms = R.max_over_ranks_ms(10.0 + 5.0 * rank, dist)
    rate = R.whole_job_rate(256, world, ms)
    out.put((rank, ms, rate, R.prints_result(rank)))
    dist.barrier()
    dist.destroy_process_group()


def test_timing_is_reduced_to_the_slowest_rank_and_rate_counts_all_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert all(abs(r[2] - 2 * 256 / 0.015) < 1e-6 for r in res)
    assert [r[3] for r in res] == [True, False]


def test_single_process_needs_no_process_group():
    from paper_2604_06832_b200 import replicas as R
    assert R.max_over_ranks_ms(3.5) == 3.5 and R.whole_job_rate(10, 1, 1000.0) == 10.0


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
