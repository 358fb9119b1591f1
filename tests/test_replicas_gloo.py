"""The multi-rank bookkeeping of the benchmark on CPU: two gloo ranks, no GPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_25431_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 10.0 if rank == 0 else 25.0                   # rank 1 is the slow replica
        payload = 1e9 * (rank + 1)
        dist.barrier()
        value, worst = replicas.job_throughput(payload, ms)
        out.put((rank, replicas.world(), value, worst, replicas.slowest(ms), replicas.total(payload)))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_sum_over_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, value, worst, slow, tot in res:
        assert world == 2 and worst == 25.0 and slow == 25.0 and tot == 3e9
        assert abs(value - 3e9 / 25e-3 / 1e9) < 1e-9       # both ranks agree on the job's number


def test_single_process_is_identity():
    assert replicas.world() == 1
    assert replicas.job_throughput(2e9, 10.0) == (2e9 / 10e-3 / 1e9, 10.0)
