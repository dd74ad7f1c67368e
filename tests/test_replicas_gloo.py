"""The N > 1 benchmark mode is N independent replicas; its host logic (slowest-rank time, total
units) is exercised here with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2210_13149_b200 import replicas
    assert replicas.env_rank() == (rank, rank, world)
    assert replicas.init("gloo")
    replicas.barrier()
    # rank 1 is the slower replica; both process 1000 units per step
    value, ms = replicas.throughput(10.0 + 5.0 * rank, 1000, torch.device("cpu"))
    out.put((rank, value, ms))
    replicas.barrier()
    replicas.finish()


def test_two_replicas_report_sum_of_units_over_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for rank, value, ms in got:
        assert ms == 15.0
        assert abs(value - 2000 / 15e-3) < 1e-6


def test_single_process_is_its_own_aggregate():
    from paper_2210_13149_b200 import replicas
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.env_rank() == (0, 0, 1)
    assert not replicas.init("gloo")
    assert replicas.throughput(4.0, 100, torch.device("cpu")) == (100 / 4e-3, 4.0)
