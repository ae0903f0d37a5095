"""Pins for the CPU oracle: checks against things that are NOT the oracle —
brute-force rank counting, closed forms, the contraction bound of
Eq. "topk_bound", torch.topk on tie-free data, exact-arithmetic identities and
a hand-computed first iteration of Algorithm 2."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def key(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def brute_topk(x, K):
    """j is selected iff fewer than K components beat it, where i beats j when
    |x_i| > |x_j|, or |x_i| == |x_j| and i < j (Section 1's definition of top_K
    plus the lower-index tie rule)."""
    k = key(x).astype(np.int64)
    d = k.size
    i = np.arange(d)
    beats = (k[None, :] > k[:, None]) | ((k[None, :] == k[:, None]) & (i[None, :] < i[:, None]))
    sel = np.nonzero(beats.sum(axis=1) < K)[0].astype(np.int32)
    return sel, np.asarray(x, dtype=np.float32)[sel]


def tie_heavy(rng, d):
    mags = np.array([0.0, 1e-3, 0.5, 0.5, 2.0, 7.25, 1e-41], dtype=np.float32)  # includes a denormal
    x = mags[rng.integers(0, mags.size, d)] * rng.choice(np.array([-1.0, 1.0], dtype=np.float32), d)
    return x.astype(np.float32)


@pytest.mark.parametrize("d,K", [(1, 1), (7, 3), (64, 1), (257, 100), (1000, 999), (2000, 37)])
def test_p1_bruteforce_rank_definition(d, K):
    rng = np.random.default_rng(100 + d + K)
    for x in (rng.standard_normal(d).astype(np.float32), tie_heavy(rng, d)):
        idx, val = oracle.ref_topk(x, K)
        bidx, bval = brute_topk(x, K)
        assert np.array_equal(idx, bidx)
        assert np.array_equal(val.view(np.uint32), bval.view(np.uint32))


def test_p2_invariants_large():
    rng = np.random.default_rng(7)
    d, K = 300_001, 2_345
    x = (rng.standard_t(3, d) * 1e-3).astype(np.float32)
    x[rng.integers(0, d, 5000)] = np.float32(0.004)      # a tie group near the threshold
    idx, val = oracle.ref_topk(x, K)
    assert idx.shape == (K,) and np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < d
    assert np.array_equal(val.view(np.uint32), x[idx].view(np.uint32))
    k = key(x)
    mask = np.zeros(d, bool)
    mask[idx] = True
    thr = k[mask].min()
    assert thr >= k[~mask].max()
    # among the entries equal to the threshold, the selected ones are the lowest indices
    eq = np.nonzero(k == thr)[0]
    n_sel = int(mask[eq].sum())
    assert np.array_equal(eq[:n_sel], eq[mask[eq]])


def test_p3_k_equals_d_is_identity():
    rng = np.random.default_rng(3)
    x = tie_heavy(rng, 513)
    idx, val = oracle.ref_topk(x, x.size)
    assert np.array_equal(idx, np.arange(x.size, dtype=np.int32))
    assert np.array_equal(val.view(np.uint32), x.view(np.uint32))


@pytest.mark.parametrize("K", [1, 10, 500, 4095])
def test_p4_contraction_bound(K):
    # || Top_K(x) - x ||^2 <= (d - K)/d ||x||^2   (Eq. "topk_bound"), in float64
    rng = np.random.default_rng(K)
    d = 4096
    x = (rng.standard_t(3, d)).astype(np.float32)
    idx, _ = oracle.ref_topk(x, K)
    x64 = x.astype(np.float64)
    resid = x64.copy()
    resid[idx] = 0.0
    assert (resid ** 2).sum() <= (d - K) / d * (x64 ** 2).sum() * (1 + 1e-12)


def test_p5_closed_forms():
    d, K = 1001, 17
    j = np.arange(d)
    x = (((-1.0) ** j) * (j + 1)).astype(np.float32)          # magnitudes increase with the index
    idx, val = oracle.ref_topk(x, K)
    assert np.array_equal(idx, np.arange(d - K, d, dtype=np.int32))
    assert np.array_equal(val, x[d - K:])
    idx, val = oracle.ref_topk(np.full(d, -2.5, np.float32), K)  # constant: first K indices
    assert np.array_equal(idx, np.arange(K, dtype=np.int32)) and np.all(val == -2.5)
    z = np.zeros(d, np.float32)
    z[::2] = -0.0                                              # -0 ties with +0; sign bit survives
    idx, val = oracle.ref_topk(z, K)
    assert np.array_equal(idx, np.arange(K, dtype=np.int32))
    assert np.array_equal(val.view(np.uint32), z[:K].view(np.uint32))


def test_p6_matches_torch_topk_on_tie_free_data():
    g = torch.Generator().manual_seed(11)
    x = torch.randn(200_000, generator=g)
    K = 777
    head = torch.topk(x.abs(), K + 1).values            # no ties at or above the K-th magnitude
    assert torch.unique(head).numel() == K + 1
    idx, _ = oracle.ref_topk(x.numpy(), K)
    t = torch.topk(x.abs(), K).indices.sort().values.numpy().astype(np.int32)
    assert np.array_equal(idx, t)


def test_rows_threads_agree():
    rng = np.random.default_rng(5)
    x = tie_heavy(rng, 6 * 999).reshape(6, 999)
    a = oracle.ref_topk_rows(x, 50, nthreads=1)
    b = oracle.ref_topk_rows(x, 50, nthreads=4)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    for r in range(6):
        i, v = oracle.ref_topk(x[r], 50)
        assert np.array_equal(a[0][r], i)


def test_p7_aggregate_support():
    rng = np.random.default_rng(9)
    N, d, K = 5, 4000, 40
    G = rng.standard_normal((N, d)).astype(np.float32)
    p = rng.dirichlet(np.ones(N)).astype(np.float32)
    r = oracle.ref_step(np.zeros(d, np.float32), G, K, K, p, 1.0, 0)
    U = np.nonzero(r.touched)[0]
    assert np.count_nonzero(r.A) <= U.size <= N * K
    assert np.all(r.A[r.touched == 0] == 0)
    assert np.array_equal(np.unique(r.up_idx), U)
    # independent re-summation, index by index, in float32 with two roundings
    for j in U[:200]:
        acc = np.float32(0)
        for q in range(N):
            hit = np.nonzero(r.up_idx[q] == j)[0]
            if hit.size:
                acc = np.float32(acc + np.float32(p[q] * r.up_val[q, hit[0]]))
        assert acc == r.A[j]


def test_p8_single_worker_downlink_is_identity():
    rng = np.random.default_rng(12)
    d, K = 5000, 64
    G = rng.standard_normal((1, d)).astype(np.float32)
    w = rng.standard_normal(d).astype(np.float32)
    one = np.ones(1, np.float32)
    uni = oracle.ref_step(w, G, K, K + 10, one, 0.25, 0)
    bi = oracle.ref_step(w, G, K, K, one, 0.25, 1)
    assert np.array_equal(uni.w, bi.w)
    assert np.array_equal(bi.msg_idx, bi.up_idx[0])
    assert np.array_equal(bi.A[bi.up_idx[0]].view(np.uint32), bi.up_val[0].view(np.uint32))
    # K_down > K_up pads with zero-valued entries at the lowest free indices: w is unchanged by them
    bi2 = oracle.ref_step(w, G, K, K + 10, one, 0.25, 1)
    assert np.array_equal(bi2.w, uni.w) and bi2.msg_idx.size == K + 10
    assert np.count_nonzero(bi2.msg_val) == K


def test_p9_identical_workers_power_of_two():
    rng = np.random.default_rng(13)
    d, K, N = 3000, 30, 8
    # values with 12 significant bits, so that every partial sum k*v/8 (k <= 8) is exact in fp32
    g = (rng.standard_normal(d).astype(np.float32).view(np.uint32) & np.uint32(0xFFFFF000)).view(np.float32)
    w = rng.standard_normal(d).astype(np.float32)
    single = oracle.ref_step(w, g[None, :], K, K, np.ones(1, np.float32), 0.1, 1)
    multi = oracle.ref_step(w, np.repeat(g[None, :], N, 0), K, K, np.full(N, 1.0 / N, np.float32), 0.1, 1)
    assert np.array_equal(single.w, multi.w)
    assert np.array_equal(single.msg_idx, multi.msg_idx)
    assert np.array_equal(single.A, multi.A)


def test_p10_positive_homogeneity():
    rng = np.random.default_rng(14)
    x = tie_heavy(rng, 5000) + (rng.standard_normal(5000) * 0.1).astype(np.float32)
    i1, _ = oracle.ref_topk(x, 123)
    for c in (0.5, 4.0, 2.0 ** -20):
        i2, v2 = oracle.ref_topk((x * np.float32(c)).astype(np.float32), 123)
        assert np.array_equal(i1, i2)


def test_p11_fixed_worker_order_and_two_roundings():
    d = 16
    G = np.full((3, d), 0.01, np.float32)
    G[0, 5], G[1, 5], G[2, 5] = 1e8, -1e8, 1.0
    one = np.ones(3, np.float32)
    r = oracle.ref_step(np.zeros(d, np.float32), G, 1, 1, one, 1.0, 0)
    assert r.A[5] == np.float32(1.0)            # (1e8 - 1e8) + 1; the reverse order would give 0
    rev = oracle.ref_step(np.zeros(d, np.float32), G[::-1].copy(), 1, 1, one, 1.0, 0)
    assert rev.A[5] == np.float32(0.0)
    # p*v is rounded before it is added: with a fused multiply-add the sum below is 2^-24, not 0
    a = np.float32(1 + 2.0 ** -12)
    G2 = np.full((2, d), 0.01, np.float32)
    G2[0, 3] = -np.float32(1 + 2.0 ** -11)
    G2[1, 3] = a
    r2 = oracle.ref_step(np.zeros(d, np.float32), G2, 1, 1, np.array([1.0, a], np.float32), 1.0, 0)
    assert r2.A[3] == np.float32(0.0) and r2.touched[3] == 1
    # same for alpha * s in the update
    w = np.zeros(d, np.float32)
    w[3] = np.float32(1 + 2.0 ** -11)
    G3 = np.full((1, d), 0.01, np.float32)
    G3[0, 3] = a
    r3 = oracle.ref_step(w, G3, 1, 1, np.ones(1, np.float32), float(a), 1)
    assert r3.w[3] == np.float32(0.0)


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = [float(t) for t in v]
    return out


def test_p12_hand_computed_first_iteration():
    g = _read_golden("alg2_first_iteration.txt")
    d, N = int(g["d"][0]), int(g["N"][0])
    K_up, K_down, alpha = int(g["K_up"][0]), int(g["K_down"][0]), g["alpha"][0]
    G = np.array([g["g1"], g["g2"], g["g3"]], np.float32)
    assert G.shape == (N, d)
    p = np.array(g["p"], np.float32)
    w0 = np.array(g["w0"], np.float32)
    bi = oracle.ref_step(w0, G, K_up, K_down, p, alpha, 1)
    for q in range(N):
        assert bi.up_idx[q].tolist() == [int(v) for v in g["up_idx%d" % (q + 1)]]
    assert bi.A.tolist() == g["A"]
    assert bi.msg_idx.tolist() == [int(v) for v in g["bi_msg_idx"]]
    assert bi.msg_val.tolist() == g["bi_msg_val"]
    assert bi.w.tolist() == g["w_bi"]
    uni = oracle.ref_step(w0, G, K_up, K_down, p, alpha, 0)
    assert uni.msg_idx.tolist() == [int(v) for v in g["uni_msg_idx"]]
    assert uni.w.tolist() == g["w_uni"]


def test_rejects_bad_arguments():
    with pytest.raises(ValueError):
        oracle.ref_topk(np.zeros(4, np.float32), 5)
    with pytest.raises(ValueError):
        oracle.ref_topk(np.zeros(4, np.float32), 0)


def test_lost_energy_closed_forms_and_bound():
    # constant vector: Top_K keeps K of d equal squares, so the bound of Eq. "topk_bound" is attained
    d, K = 1000, 37
    x = np.full(d, -1.5, np.float32)
    idx, _ = oracle.ref_topk(x, K)
    assert abs(oracle.ref_lost_energy(x, idx) - (d - K) / d) < 1e-15
    # at most K non-zeros: nothing is lost; zero vector: defined as 0
    y = np.zeros(d, np.float32)
    y[[3, 500, 999]] = [2.0, -7.0, 0.5]
    idx, _ = oracle.ref_topk(y, 3)
    assert oracle.ref_lost_energy(y, idx) == 0.0
    assert oracle.ref_lost_energy(np.zeros(d, np.float32), idx) == 0.0
    # one dominant component: what is lost is the rest, by hand
    z = np.array([3.0, 4.0, 12.0], np.float32)
    idx, _ = oracle.ref_topk(z, 1)
    assert abs(oracle.ref_lost_energy(z, idx) - 25.0 / 169.0) < 1e-15
    # random data: below the bound, and scale-free
    rng = np.random.default_rng(21)
    r = rng.standard_t(3, 5000).astype(np.float32)
    idx, _ = oracle.ref_topk(r, 50)
    v = oracle.ref_lost_energy(r, idx)
    assert 0 < v <= (5000 - 50) / 5000
    assert abs(oracle.ref_lost_energy((r * np.float32(0.25)).astype(np.float32), idx) - v) < 1e-12


def test_gap_constants_hand_example_and_special_cases():
    g = _read_golden("alg2_first_iteration.txt")
    G = np.array([g["g1"], g["g2"], g["g3"]], np.float32)
    p = np.array(g["p"], np.float32)
    den = g["rho_sq_den"][0]
    assert abs(oracle.ref_rho(G, None, None, 2, 2, p, 0.5, 0) - (g["rho_hat_sq_num"][0] / den) ** 0.5) < 1e-12
    assert abs(oracle.ref_rho(G, None, None, 2, 2, p, 0.5, 1) - (g["rho_sq_num"][0] / den) ** 0.5) < 1e-12
    # one worker: the aggregate of its message IS Top_K of the sum, both constants vanish
    rng = np.random.default_rng(31)
    x = rng.standard_normal((1, 4000)).astype(np.float32)
    one = np.ones(1, np.float32)
    assert oracle.ref_rho(x, None, None, 40, 40, one, 1.0, 0) == 0.0
    assert oracle.ref_rho(x, None, None, 40, 40, one, 1.0, 1) == 0.0
    # no compression at all: nothing differs
    y = rng.standard_normal((3, 50)).astype(np.float32)
    w3 = np.array([0.5, 0.25, 0.25], np.float32)
    assert oracle.ref_rho(y, None, None, 50, 50, w3, 1.0, 0) == 0.0
    # with memories at zero and alpha a power of two the ratio equals the memory-free one
    z = rng.standard_normal((4, 3000)).astype(np.float32)
    w4 = np.full(4, 0.25, np.float32)
    free = oracle.ref_rho(z, None, None, 30, 30, w4, 1.0, 1)
    mem = oracle.ref_rho(z, np.zeros_like(z), np.zeros(3000, np.float32), 30, 30, w4, 0.25, 1)
    assert free > 0 and abs(free - mem) < 1e-12
    # the toy example's message: workers that disagree make the unidirectional gap large
    c = np.array([1.0, 5.0, 10.0], np.float32)
    wv = np.full(100, 5.4, np.float32)
    wv[::7] += 0.3
    Gq = (wv[None, :] - c[:, None]).astype(np.float32)
    assert oracle.ref_rho(Gq, None, None, 1, 1, np.full(3, 1 / 3, np.float32), 0.01, 0) > 1.0
