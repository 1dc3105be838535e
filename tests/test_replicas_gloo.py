"""Two CPU processes over gloo: the replica bookkeeping bench.py uses for --gpus N > 1
(barrier, max over ranks of the timings, whole-job rate)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2302_07863_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    replicas.barrier(dist, world)
    ms = replicas.max_over_ranks(dist, world, 10.0 + 5.0 * rank)
    rate = replicas.whole_job_rate(64, world, ms)
    out.put((rank, ms, rate))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_sum_of_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    ps = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    got = sorted(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]
    assert all(abs(g[2] - 2 * 64 / 0.015) < 1e-6 for g in got)


def test_single_rank_is_a_no_op():
    assert replicas.max_over_ranks(None, 1, 3.5) == 3.5
    assert replicas.whole_job_rate(64, 1, 32.0) == 2000.0
