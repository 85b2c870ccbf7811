"""The N > 1 path of the benchmark (independent replicas, barrier + max-over-ranks timing) on
two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_11886_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.world() == (rank, world)
        replicas.barrier()
        mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        worst = replicas.max_over_ranks(mine)
        replicas.barrier()
        out.put((rank, worst, replicas.aggregate_us_per_step(worst, steps=100, n_replicas=world)))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
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
    assert [g[1] for g in got] == [15.0, 15.0]
    assert abs(got[0][2] - 15.0 * 1e3 / 100 / 2) < 1e-9


def test_single_process_is_identity():
    assert replicas.world() == (0, 1)
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.aggregate_us_per_step(2.0, 100, 1) == 20.0
