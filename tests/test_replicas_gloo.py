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


class _FakeContext:
    """Stands in for binding.Context on CPU: the same three calls sharded_step makes, with a toy
    'message' (the first K values of a row, tagged with the worker's number) instead of a Top_K."""

    def __init__(self, N, d, K):
        self.N, self.d, self.K_up = N, d, K
        self.msgs = torch.full((N, K), -1, dtype=torch.int64)
        self.calls = []

    def tk_step_uplink(self, grads_local, row0, alpha, mode):
        rows = grads_local.numel() // self.d
        self.calls.append(("uplink", row0, rows))
        g = grads_local.view(rows, self.d)
        for r in range(rows):
            self.msgs[row0 + r] = (g[r, :self.K_up] * 1000).to(torch.int64) + 10 ** 9 * (row0 + r)

    def tk_messages(self):
        return self.msgs

    def tk_step_server(self, w, alpha, mode):
        self.calls.append(("server",))
        assert (self.msgs >= 0).all(), "a worker's message is missing on this rank"
        # fixed worker order, as the real server step
        for q in range(self.N):
            w[:self.K_up] -= alpha * (self.msgs[q] - 10 ** 9 * q).to(torch.float64) * (q + 1)


def _sharded_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        N, d, K = 6, 40, 5
        g = torch.Generator().manual_seed(99)
        G = torch.randint(0, 1000, (N, d), generator=g).to(torch.float64) / 1000     # the same on every rank
        row0, rows = sharding.row_range(N, rank, world)
        ctx = _FakeContext(N, d, K)
        w = torch.zeros(d, dtype=torch.float64)
        for step in range(2):
            sharding.sharded_step(ctx, w, (G[row0:row0 + rows] + step).contiguous(), 0.5, 1)
        out.put((rank, ctx.calls, ctx.msgs.clone(), w.clone()))
    finally:
        dist.destroy_process_group()


def test_sharded_step_bookkeeping_on_two_ranks():
    # sharding.sharded_step itself under world size 2: each rank steps its own rows, the gather
    # puts all N messages in worker order on both ranks, and the replicas of w stay identical
    world, port = 2, _free_port()
    mpc = mp.get_context("spawn")
    out = mpc.Queue()
    procs = [mpc.Process(target=_sharded_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted((out.get(timeout=120) for _ in range(world)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # one process holding every row is the reference
    N, d, K = 6, 40, 5
    g = torch.Generator().manual_seed(99)
    G = torch.randint(0, 1000, (N, d), generator=g).to(torch.float64) / 1000
    ref = _FakeContext(N, d, K)
    w_ref = torch.zeros(d, dtype=torch.float64)
    for step in range(2):
        sharding.sharded_step(ref, w_ref, (G + step).contiguous(), 0.5, 1)
    for rank, calls, msgs, w in results:
        assert calls == [("uplink", 3 * rank, 3), ("server",)] * 2
        assert torch.equal(msgs, ref.msgs), "rank %d: messages not in worker order" % rank
        assert torch.equal(w, w_ref)
    assert torch.equal(results[0][3], results[1][3])


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
