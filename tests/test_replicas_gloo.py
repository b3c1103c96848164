"""The N > 1 bookkeeping of the benchmark (max time over ranks, summed throughput) on two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2509_25996_b200 import replicas
    local_ms = 10.0 * (rank + 1)                       # rank 1 is the slow one: 20 ms
    value, ms = replicas.whole_job_throughput(1000, 4, local_ms)
    out.put((rank, replicas.world_size(), value, ms, replicas.max_over_ranks(float(-rank))))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_clock_and_the_summed_throughput():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, value, ms, mx in got:
        assert world == 2
        assert ms == 20.0                              # the slowest rank's time, on every rank
        assert value == 2 * 1000 * 4 / 20e-3           # both replicas' units over that time
        assert mx == 0.0


def test_single_process_needs_no_group():
    from paper_2509_25996_b200 import replicas
    assert replicas.world_size() == 1
    assert replicas.whole_job_throughput(500, 2, 5.0) == (500 * 2 / 5e-3, 5.0)
