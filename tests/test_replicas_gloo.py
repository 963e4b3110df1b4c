"""The N > 1 path of bench.py (replicas, max-over-ranks timing, whole-job aggregate) on two gloo ranks on the CPU."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2508_02124_b200 import replicas
    dist.barrier()
    slowest = replicas.max_over_ranks(10.0 + 5.0 * rank)           # rank 1 is slower
    rate = replicas.whole_job_rate(7.0, slowest)
    out.put((rank, slowest, rate))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_step_and_the_aggregate_rate():
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
    for rank, slowest, rate in res:
        assert slowest == 15.0
        assert abs(rate - 2 * 7.0 / 15e-3) < 1e-6
