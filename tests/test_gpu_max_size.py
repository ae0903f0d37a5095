"""The longest vector the library accepts, d = 2^31 - 1 (indices up to 2^31 - 2, rows that
start beyond 2^32 bytes and, d being odd, off the 16-byte grid).

The CPU oracle cannot chew through 2^31 values per row in test time, so it is given the
problem restricted to the coordinates that can matter: every coordinate where some row
holds a value of magnitude >= a threshold low enough that each row has more than K of them.
Restricting to a superset of every row's K largest, with the coordinates kept in ascending
order, changes neither the selected sets nor the tie-breaks, so the oracle's answer on the
restricted problem, mapped back, is the answer on the full one.  The restriction itself is
done with plain torch comparisons, not with the library under test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_15203_b200 import binding
from util import assert_message_equal, assert_values_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
D_MAX = 2 ** 31 - 1
CHUNK = 1 << 28
THRESHOLD = 4.5          # about 14,600 of 2^31 standard normals exceed it in magnitude
TIE = 50.0               # planted magnitude, above every random value


def _need_memory(gib):
    free, _ = torch.cuda.mem_get_info(0)
    if free < gib * 2 ** 30:
        pytest.skip("needs %d GiB of free device memory" % gib)


def _fill_rows(rows, seed):
    """[rows][D_MAX] standard normals plus a group of equal magnitudes that includes both
    ends of the row; returns the tensor."""
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    x = torch.empty((rows, D_MAX), device=DEV, dtype=torch.float32)
    for r in range(rows):
        for a in range(0, D_MAX, CHUNK):
            x[r, a:min(D_MAX, a + CHUNK)].normal_(generator=g)
        pos = torch.unique(torch.randint(0, D_MAX, (600,), generator=g, device=DEV))
        sgn = torch.where(torch.rand(pos.numel(), generator=g, device=DEV) < 0.5, -1.0, 1.0)
        x[r, pos] = TIE * sgn
        x[r, 0] = TIE
        x[r, D_MAX - 1] = -TIE
        x[r, D_MAX - 2] = TIE
    return x


def _coords_that_matter(x):
    """Ascending coordinates where any row of x reaches THRESHOLD in magnitude."""
    parts = []
    for a in range(0, D_MAX, CHUNK):
        blk = x[:, a:min(D_MAX, a + CHUNK)]
        hit = (blk.abs() >= THRESHOLD).any(dim=0)
        parts.append(torch.nonzero(hit).flatten() + a)
        del blk, hit
    return torch.cat(parts)


@pytest.mark.parametrize("K", [500, 3000])
def test_topk_at_the_largest_length(K):
    # K = 500 cuts through the ~603 equal magnitudes (lowest indices win, the last two coordinates
    # lose); K = 3000 takes all of them, the last coordinate included, and goes on into the tail
    _need_memory(40)
    rows = 2
    x = _fill_rows(rows, 9001)
    S = _coords_that_matter(x)
    sub = x[:, S].cpu().numpy()
    assert ((np.abs(sub) >= THRESHOLD).sum(axis=1) > K).all()
    ridx, rval = oracle.ref_topk_rows(sub, K)
    S_host = S.cpu().numpy()
    idx, val = binding.tk_topk(x, K)
    torch.cuda.synchronize()
    assert_message_equal(idx, val, S_host[ridx].astype(np.int32), rval, "tk_topk d=2^31-1 K=%d" % K)
    last = int(D_MAX - 1)
    for r in range(rows):
        assert (last in idx[r].cpu().numpy()) == (K == 3000)


@pytest.mark.parametrize("mode", [0, 1])
def test_step_at_the_largest_length(mode):
    _need_memory(70)
    N, K_up, K_down, alpha = 2, 2000, 1500, 0.1
    G = _fill_rows(N, 9002)
    G[1, D_MAX - 1] = TIE            # the two workers cancel at the last coordinate, add up at the first
    S = _coords_that_matter(G)
    S_host = S.cpu().numpy()
    p = torch.tensor([0.5, 0.5], dtype=torch.float32)
    w = torch.empty(D_MAX, device=DEV, dtype=torch.float32)
    g = torch.Generator(device=DEV)
    g.manual_seed(9003)
    for a in range(0, D_MAX, CHUNK):
        w[a:min(D_MAX, a + CHUNK)].normal_(generator=g)
    w_before = w.clone()
    ref = oracle.ref_step(w[S].cpu().numpy(), G[:, S].cpu().numpy(), K_up, K_down, p.numpy(), alpha, mode)

    ctx = binding.Context(D_MAX, N, K_up, K_down, p)
    ctx.tk_step(w, G, alpha, mode)
    st = ctx.tk_status()
    assert st.device_status == 0
    uidx, uval = ctx.tk_last_uplink()
    assert_message_equal(uidx, uval, S_host[ref.up_idx].astype(np.int32), ref.up_val, "uplink at d=2^31-1")
    U = np.nonzero(ref.touched)[0]
    aidx, aval = ctx.tk_last_aggregate()
    assert np.array_equal(aidx.cpu().numpy(), S_host[U].astype(np.int32))
    assert_values_close(aval.cpu().numpy(), ref.A[U], "aggregate at d=2^31-1")
    midx, mval = ctx.tk_last_downlink()
    assert np.array_equal(midx.cpu().numpy(), S_host[ref.msg_idx].astype(np.int32))
    assert_values_close(mval.cpu().numpy(), ref.msg_val, "downlink at d=2^31-1")
    # the update: the oracle's values on the restricted coordinates, no change anywhere else
    assert_values_close(w[S].cpu().numpy(), ref.w, "w at d=2^31-1")
    changed = []
    for a in range(0, D_MAX, CHUNK):
        b = min(D_MAX, a + CHUNK)
        diff = w[a:b].view(torch.int32) != w_before[a:b].view(torch.int32)
        changed.append((torch.nonzero(diff).flatten() + a).cpu().numpy())
    changed = np.concatenate(changed)
    assert np.isin(changed, S_host[ref.msg_idx]).all() and 0 < changed.size <= ref.msg_idx.size
    # a second step on the same context: the dense server buffer was left clean up to its last word
    ctx.tk_step(w, G, alpha, mode)
    aidx2, _ = ctx.tk_last_aggregate()
    assert np.array_equal(aidx2.cpu().numpy(), S_host[U].astype(np.int32))
    ctx.close()
