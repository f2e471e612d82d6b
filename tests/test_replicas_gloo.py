"""The N > 1 bookkeeping of the benchmark (replicas: no data-path collective), on two gloo ranks on CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    import torch.distributed as dist
    from paper_2512_02551_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    replicas.barrier(dist)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = replicas.slowest_rank_ms(local_ms, dist, "cpu")
    value = replicas.job_throughput(1.0e12, world, ms)
    out.put((rank, ms, value))
    replicas.barrier(dist)
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1]
    for _, ms, value in got:
        assert ms == 15.0                                   # the max over ranks, on every rank
        assert abs(value - 2 * 1.0e12 / 15.0e-3) < 1e-3 * value


def test_single_process_is_identity():
    from paper_2512_02551_b200 import replicas
    assert replicas.slowest_rank_ms(3.5) == 3.5
    assert replicas.job_throughput(2.0, 1, 1000.0) == 2.0
    replicas.barrier(None)
