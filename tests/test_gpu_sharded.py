"""The row-sharded step (tk_step_uplink / exchange / tk_step_server) on one GPU: two contexts
play two ranks, each selects its own half of the workers, the halves of the message buffer
are copied across (what the all-gather does), and both servers must reproduce the oracle's
step and each other bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_15203_b200 import binding, sharding, workloads as W
from util import assert_message_equal, assert_values_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("mode", [0, 1, 1 | binding.TK_MODE_EF])
def test_two_emulated_ranks(mode):
    wl = W.workload(2, d=700_001, N=6)
    p = W.make_p(wl)
    world = 2
    ef = bool(mode & binding.TK_MODE_EF)
    ctxs = [binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, p) for _ in range(world)]
    if ef:
        for c in ctxs:
            c.tk_ef_attach()
    ws = [W.make_w(wl, DEV) for _ in range(world)]
    w_ref = ws[0].cpu().numpy()
    eps = np.zeros((wl.N, wl.d), np.float32)
    delta = np.zeros(wl.d, np.float32)
    for s in range(3):
        G = W.make_grads(wl, s, DEV)
        ranges = [sharding.row_range(wl.N, r, world) for r in range(world)]
        for r, (row0, rows) in enumerate(ranges):
            ctxs[r].tk_step_uplink(G[row0:row0 + rows].contiguous(), row0, wl.alpha, mode)
        msgs = [c.tk_messages() for c in ctxs]
        for r, (row0, rows) in enumerate(ranges):          # the all-gather, by hand
            for other in range(world):
                if other != r:
                    msgs[other][row0:row0 + rows].copy_(msgs[r][row0:row0 + rows])
        for r in range(world):
            ctxs[r].tk_step_server(ws[r], wl.alpha, mode)
        if ef:
            ref = oracle.ref_step_ef(w_ref, eps, delta, G.cpu().numpy(), wl.K_up, wl.K_up, p.numpy(), wl.alpha, mode & 1)
            eps, delta = ref.eps, (ref.delta if mode & 1 else delta)
        else:
            ref = oracle.ref_step(w_ref, G.cpu().numpy(), wl.K_up, wl.K_up, p.numpy(), wl.alpha, mode)
        w_ref = ref.w
        for r in range(world):
            assert ctxs[r].tk_status().device_status == 0
            assert_values_close(ws[r].cpu().numpy(), ref.w, "rank %d w step %d" % (r, s))
            uidx, uval = ctxs[r].tk_last_uplink()
            assert_message_equal(uidx, uval, ref.up_idx, ref.up_val, "rank %d gathered messages" % r)
            midx, mval = ctxs[r].tk_last_downlink()
            assert np.array_equal(midx.cpu().numpy(), ref.msg_idx)
        assert torch.equal(ws[0].view(torch.int32), ws[1].view(torch.int32)), "replicas of w diverged"
        if ef:
            # each rank keeps the memories of its own workers only; the server memory is replicated
            for r, (row0, rows) in enumerate(ranges):
                e, dl = ctxs[r].tk_ef_state()
                assert_values_close(e[row0:row0 + rows].cpu().numpy(), ref.eps[row0:row0 + rows], "rank %d eps" % r)
                if mode & 1:
                    assert_values_close(dl.cpu().numpy(), ref.delta, "rank %d delta" % r)


def test_single_process_sharded_step_is_tk_step():
    wl = W.workload(5, d=900_000, N=4)
    p = W.make_p(wl)
    G = W.make_grads(wl, 0, DEV)
    a, b = binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, p), binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, p)
    wa, wb = W.make_w(wl, DEV), W.make_w(wl, DEV)
    a.tk_step(wa, G, wl.alpha, 1)
    sharding.sharded_step(b, wb, G, wl.alpha, 1)
    assert torch.equal(wa.view(torch.int32), wb.view(torch.int32))
