"""The N>1 path of the benchmark (independent replicas, max-over-ranks timing) on CPU:
two gloo ranks on 127.0.0.1."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2209_15203_b200 import replicas, sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        local_ms = 2.0 if rank == 0 else 5.0          # rank 1 is the slow replica
        value, ms = replicas.whole_job_throughput(local_ms, units_per_step=1000, steps=10)
        # the uplink exchange of the sharded step: every rank fills its own rows of the message buffer
        N, K = 6, 5
        row0, rows = sharding.row_range(N, rank, world)
        msgs = torch.full((N, K), -1, dtype=torch.int64)
        msgs[row0:row0 + rows] = torch.arange(rows * K).view(rows, K) + 1000 * rank
        sharding.all_gather_messages(msgs, row0, rows)
        expect = torch.cat([torch.arange(rows * K).view(rows, K) + 1000 * r for r in range(world)])
        assert torch.equal(msgs, expect), "rank %d does not hold all messages in worker order" % rank
        out.put((rank, replicas.world_size(), value, ms, replicas.max_over_ranks(float(rank))))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ws, value, ms, mx in results:
        assert ws == 2 and ms == 5.0 and mx == 1.0
        assert value == 2 * 1000 * 10 / 5e-3           # both replicas' units over the slowest time


def test_row_ranges():
    assert [sharding.row_range(8, r, 4) for r in range(4)] == [(0, 2), (2, 2), (4, 2), (6, 2)]
    import pytest
    with pytest.raises(ValueError):
        sharding.row_range(7, 0, 2)


def test_single_process_is_the_identity():
    assert replicas.world_size() == 1
    assert replicas.max_over_ranks(3.5) == 3.5
    value, ms = replicas.whole_job_throughput(4.0, 100, 2)
    assert ms == 4.0 and value == 100 * 2 / 4e-3
