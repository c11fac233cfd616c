"""The N > 1 path of the benchmark on CPU: two gloo ranks (independent replicas) agree on the
slowest rank's time, and the whole-job figure divides it by the number of replicas."""
import os
import socket
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
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                      # rank 1 is the slow replica: 15 ms for its steps
    slowest = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    dist.barrier()
    out.put((rank, slowest, bench.whole_job_us_per_step(slowest / 5, world)))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in got:
        assert slowest == 15.0                    # max over ranks, seen by every rank
        assert abs(value - 15.0 / 5 * 1e3 / 2) < 1e-9   # 5 steps each, 2 replicas
