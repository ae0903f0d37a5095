"""The synthetic workloads: sizes, K values and structure (CPU, small d)."""
import numpy as np
import torch

from paper_2209_15203_b200 import workloads as W


def test_k_values_of_the_five_configurations():
    assert (W.workload(1).K_up, W.workload(1).K_down) == (1000, (1000,))
    assert W.workload(2).K_up == 11_700
    assert W.workload(3).K_up == 25_600
    assert (W.workload(4).K_up, W.workload(4).K_down) == (1_170, (1_170, 11_700, 117_000))
    assert W.workload(5).K_up == 12_400
    # Section 4's K = d - floor((1 - 0.001) d) on the paper's own model sizes
    assert [W.k_from_ratio(d, 1, 1000) for d in (29_034, 50_890, 242_762, 1_199_882, 20_040_522)] == \
        [30, 51, 243, 1_200, 20_041]


def test_paper_shapes():
    assert [(W.workload(c).N, W.workload(c).d, W.workload(c).K_up) for c in (6, 7, 8, 9, 10)] == \
        [(100, 242_762, 243), (20, 20_040_522, 20_041), (50, 1_199_882, 1_200), (20, 29_034, 30), (100, 50_890, 51)]


def test_block_layout_covers_d():
    for cid, d in ((2, 117_001), (3, 25_603), (5, 1_240_000)):
        wl = W.workload(cid, d=d)
        sizes = W.block_sizes(wl)
        assert int(sizes.sum()) == d and int(sizes.min()) >= 1 and sizes.numel() == wl.blocks
        s = W.scale_vector(wl, "cpu")
        assert s.shape == (d,) and float(s.min()) >= wl.sigma_lo * 0.999 and float(s.max()) <= wl.sigma_hi * 1.001


def test_grads_are_seeded_and_fresh_per_step():
    wl = W.workload(3, d=20_000, N=3)
    a = W.make_grads(wl, 0, "cpu")
    b = W.make_grads(wl, 0, "cpu")
    c = W.make_grads(wl, 1, "cpu")
    assert a.shape == (3, 20_000) and a.dtype == torch.float32
    assert torch.equal(a, b) and not torch.equal(a, c)
    assert W.checksum(a) == W.checksum(b)
    p = W.make_p(wl)
    assert p.shape == (3,) and abs(float(p.sum()) - 1) < 1e-6 and float(p.min()) > 0


def test_adversarial_rows_have_zeros_and_straddling_ties():
    wl = W.workload(4, d=200_000, N=4)
    G = W.make_grads(wl, 0, "cpu").numpy()
    K = wl.K_up
    for q in range(4):
        mag = np.abs(G[q])
        assert 0.03 < np.mean(mag == 0) < 0.07
        kth = np.sort(mag)[::-1][K - 1]
        assert np.sum(mag == kth) > 10          # the K-th magnitude sits inside a group of equal values
    # paired workers carry the planted magnitudes with opposite signs
    both = (np.abs(G[0]) == np.abs(G[1])) & (G[0] != 0)
    assert both.sum() >= 1500 and np.all(G[0][both] == -G[1][both])


def test_agreeing_workers_share_their_large_coordinates():
    wl = W.workload(2, d=200_000, N=6)
    A = W.make_grads(wl, 0, "cpu", agree=0.01)
    B = W.make_grads(wl, 0, "cpu", agree=0.01)
    assert torch.equal(A, B)
    assert not torch.equal(A, W.make_grads(wl, 0, "cpu"))          # the default rows are independent draws
    top = [set(torch.topk(A[q].abs(), wl.K_up).indices.tolist()) for q in range(wl.N)]
    common = set.intersection(*top)
    assert len(common) > 0.7 * wl.K_up
    ratio = A[1] / A[0]
    assert 0.005 < float(ratio[torch.isfinite(ratio)].std()) < 0.03
