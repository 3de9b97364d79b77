"""The N > 1 path of the benchmark is N independent replicas; what crosses processes is the timing protocol only.
Two gloo ranks on CPU: the barrier completes, the maximum is taken over ranks, the whole-job rate uses it."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2601_08273_b200 import replicas
    cpu = torch.device("cpu")
    replicas.barrier(cpu)
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    q.put((rank, replicas.world(), replicas.max_over_ranks(ms, cpu), replicas.whole_job_rate(3.0e9, ms, cpu)))
    replicas.barrier(cpu)
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, mx, rate in got:
        assert world == 2
        assert mx == 15.0                                        # max over ranks, on every rank
        assert abs(rate - 2 * 3.0e9 / 15.0e-3) < 1e-3 * rate     # both ranks' units over the slowest rank's time


def test_single_process_is_the_identity():
    from paper_2601_08273_b200 import replicas
    assert replicas.world() == 1
    assert replicas.max_over_ranks(7.5, torch.device("cpu")) == 7.5
