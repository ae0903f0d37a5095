"""Pins for the oracle of the iteration with error memories (Algorithm 1 / 2 as printed):
a hand-worked two-step example, the exact recursion of the error-corrected sequence
(first lemma of Section 3.2), reductions to the memory-free oracle and to plain SGD, and the
paper's toy example."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, *v = line.split()
                out[k] = [float(t) for t in v]
    return out


def test_hand_worked_two_iterations():
    g = _read("alg12_two_iterations_with_memories.txt")
    d, N, K = int(g["d"][0]), int(g["N"][0]), int(g["K"][0])
    p = np.array(g["p"], np.float32)
    for mode, tag in ((1, "bi"), (0, "uni")):
        w = np.zeros(d, np.float32)
        eps = np.zeros((N, d), np.float32)
        delta = np.zeros(d, np.float32)
        for t in (1, 2):
            G = np.array([g["g1_t%d" % t], g["g2_t%d" % t]], np.float32)
            r = oracle.ref_step_ef(w, eps, delta, G, K, K, p, g["alpha"][0], mode)
            w, eps = r.w, r.eps
            assert eps[0].tolist() == g["eps1_t%d" % t] and eps[1].tolist() == g["eps2_t%d" % t]
            assert w.tolist() == g["%s_w_t%d" % (tag, t)]
            if mode == 1:
                delta = r.delta
                assert delta.tolist() == g["bi_delta_t%d" % t]
                assert r.msg_idx.tolist() == [int(v) for v in g["bi_msg_idx_t%d" % t]]


def _quadratic_grads(w, centres):
    return (w[None, :] - centres[:, None]).astype(np.float32)


@pytest.mark.parametrize("mode", [0, 1])
def test_error_corrected_sequence_follows_plain_sgd_exactly(mode):
    # w~_t = w_t - sum_q p_q eps_t^q - delta_t  obeys  w~_t = w~_{t-1} - alpha sum_q p_q g^q(w_{t-1}).
    # With small dyadic numbers every fp32 operation is exact, so the identity holds bit for bit.
    rng = np.random.default_rng(3)
    d, N, K = 16, 4, 2
    p = np.full(N, 0.25, np.float32)
    centres = np.array([1, 5, 10, -4], np.float32)
    w = rng.integers(-8, 9, d).astype(np.float32)
    eps = np.zeros((N, d), np.float32)
    delta = np.zeros(d, np.float32)
    wt = w.astype(np.float64)
    for _ in range(3):
        G = _quadratic_grads(w, centres)
        wt = wt - 0.5 * (p[:, None].astype(np.float64) * G).sum(0)
        r = oracle.ref_step_ef(w, eps, delta, G, K, K, p, 0.5, mode)
        w, eps = r.w, r.eps
        if mode == 1:
            delta = r.delta
        corrected = w.astype(np.float64) - (p[:, None].astype(np.float64) * eps).sum(0) - delta
        assert np.array_equal(corrected, wt)


@pytest.mark.parametrize("mode", [0, 1])
def test_error_corrected_sequence_to_rounding(mode):
    rng = np.random.default_rng(4)
    d, N, K = 500, 5, 7
    p = rng.dirichlet(np.ones(N)).astype(np.float32)
    w = rng.standard_normal(d).astype(np.float32)
    eps = np.zeros((N, d), np.float32)
    delta = np.zeros(d, np.float32)
    wt = w.astype(np.float64)
    for t in range(25):
        G = (rng.standard_normal((N, d)) + w[None, :]).astype(np.float32)
        wt = wt - 0.05 * (p[:, None].astype(np.float64) * G).sum(0)
        r = oracle.ref_step_ef(w, eps, delta, G, K, 2 * K, p, 0.05, mode)
        w, eps = r.w, r.eps
        if mode == 1:
            delta = r.delta
    corrected = w.astype(np.float64) - (p[:, None].astype(np.float64) * eps).sum(0) - delta
    assert np.max(np.abs(corrected - wt)) < 1e-4 * max(1.0, np.max(np.abs(wt)))


@pytest.mark.parametrize("mode", [0, 1])
def test_first_step_from_zero_memories_is_the_memory_free_step(mode):
    rng = np.random.default_rng(5)
    d, N, K = 3000, 3, 25
    G = rng.standard_normal((N, d)).astype(np.float32)
    w = rng.standard_normal(d).astype(np.float32)
    p = rng.dirichlet(np.ones(N)).astype(np.float32)
    a = oracle.ref_step(w, G, K, K, p, 1.0, mode)           # alpha = 1: a^q = g^q exactly
    b = oracle.ref_step_ef(w, np.zeros((N, d), np.float32), np.zeros(d, np.float32), G, K, K, p, 1.0, mode)
    assert np.array_equal(a.w, b.w) and np.array_equal(a.up_idx, b.up_idx)
    assert np.array_equal(a.msg_idx, b.msg_idx) and np.array_equal(a.msg_val, b.msg_val)
    # the memories hold exactly what was not sent
    sent = np.zeros((N, d), np.float32)
    for q in range(N):
        sent[q, b.up_idx[q]] = b.up_val[q]
    assert np.array_equal(b.eps + sent, G) and np.all(b.eps[sent != 0] == 0)
    if mode == 1:
        down = np.zeros(d, np.float32)
        down[b.msg_idx] = b.msg_val
        assert np.array_equal(b.delta + down, a.A)


def test_no_compression_is_plain_sgd():
    rng = np.random.default_rng(6)
    d, N = 64, 3
    G = rng.standard_normal((N, d)).astype(np.float32)
    w = rng.standard_normal(d).astype(np.float32)
    p = np.array([0.5, 0.25, 0.25], np.float32)
    for mode in (0, 1):
        r = oracle.ref_step_ef(w, np.zeros((N, d), np.float32), np.zeros(d, np.float32), G, d, d, p, 0.125, mode)
        acc = np.zeros(d, np.float32)
        for q in range(N):                                   # Eq. 2, summed in worker order in fp32
            acc = (acc + p[q] * (np.float32(0.125) * G[q])).astype(np.float32)
        assert np.array_equal(r.w, (w - acc).astype(np.float32))
        assert not r.eps.any() and (mode == 0 or not r.delta.any())


def test_toy_example_of_the_paper():
    g = _read("toy_example.txt")
    F_star = g["F_star_num"][0] / g["F_star_den"][0]
    w_star = g["w_star_num"][0] / g["w_star_den"][0]
    centres = np.array([1.0, 5.0, 10.0], np.float32)
    F = lambda w: sum(0.5 * np.sum((w.astype(np.float64) - c) ** 2) for c in (1.0, 5.0, 10.0)) / 3
    assert abs(F(np.full(100, w_star)) - F_star) < 1e-9      # the printed optimum is the optimum
    np.random.seed(10)
    w0 = np.random.normal(20, 1, 100).astype(np.float32)
    p = np.full(3, 1 / 3, np.float32)
    w, eps = w0.copy(), np.zeros((3, 100), np.float32)
    for t in range(1, 211):
        G = _quadratic_grads(w, centres)
        a = eps + np.float32(0.01) * G
        r = oracle.ref_step_ef(w, eps, None, G, 1, 1, p, 0.01, 0)
        w, eps = r.w, r.eps
    sent = np.zeros(100, np.float32)
    for q in range(3):
        sent[r.up_idx[q]] += r.up_val[q]
    full = a.sum(0)
    norm_uplink = np.linalg.norm(full - sent)
    both = np.zeros(100, np.float32)
    j = int(np.argmax(np.abs(sent)))
    both[j] = sent[j]
    norm_both = np.linalg.norm(full - both)
    # generator and exact iteration count are not stated: agreement to a few per cent is the pin
    assert abs(norm_uplink - g["norm_uplink"][0]) < 0.03 * g["norm_uplink"][0]
    assert abs(norm_both - g["norm_both"][0]) < 0.03 * g["norm_both"][0]
    # both variants hover at a distance from F*, as the paper describes, far below the start
    assert F_star < F(w) < F_star + 0.2 * (F(w0) - F_star)


def test_gap_constants_from_nonzero_memories_hand_worked():
    # one iteration that STARTS from non-zero eps and delta (Section 3's two gap assumptions with
    # a^q = eps^q + alpha g^q); all values by hand in the golden file
    g = _read("gap_constants_with_memories.txt")
    p = np.array(g["p"], np.float32)
    K_up, K_down, alpha = int(g["K_up"][0]), int(g["K_down"][0]), g["alpha"][0]
    G = np.array([g["g1"], g["g2"]], np.float32)
    eps = np.array([g["eps1"], g["eps2"]], np.float32)
    delta = np.array(g["delta"], np.float32)
    den = g["rho_sq_den"][0]
    uni = oracle.ref_rho(G, eps, None, K_up, K_down, p, alpha, 0)
    bi = oracle.ref_rho(G, eps, delta, K_up, K_down, p, alpha, 1)
    assert abs(uni - (g["rho_hat_sq_num"][0] / den) ** 0.5) < 1e-12
    assert abs(bi - (g["rho_sq_num"][0] / den) ** 0.5) < 1e-12
    # the unidirectional iteration has no server memory: passing one changes nothing
    assert oracle.ref_rho(G, eps, delta, K_up, K_down, p, alpha, 0) == uni
    # the step size sits inside a^q and in the denominator: halving it and doubling the gradients
    # leaves every a^q, hence both ratios, unchanged
    assert oracle.ref_rho(2 * G, eps, None, K_up, K_down, p, alpha / 2, 0) == uni
    assert oracle.ref_rho(2 * G, eps, delta, K_up, K_down, p, alpha / 2, 1) == bi
    # ... and the memories matter: without them the values are different ones
    assert abs(oracle.ref_rho(G, np.zeros_like(eps), np.zeros_like(delta), K_up, K_down, p, alpha, 1) - bi) > 0.1

    # second iteration of the two-iteration example (memories eps_1, delta_1 of its first iteration)
    h = _read("alg12_two_iterations_with_memories.txt")
    p2 = np.array(h["p"], np.float32)
    G2 = np.array([h["g1_t2"], h["g2_t2"]], np.float32)
    eps1 = np.array([h["eps1_t1"], h["eps2_t1"]], np.float32)
    delta1 = np.array(h["bi_delta_t1"], np.float32)
    K = int(h["K"][0])
    den2 = h["rho_sq_den_t2"][0]
    assert abs(oracle.ref_rho(G2, eps1, None, K, K, p2, h["alpha"][0], 0) - (h["rho_hat_sq_num_t2"][0] / den2) ** 0.5) < 1e-12
    assert abs(oracle.ref_rho(G2, eps1, delta1, K, K, p2, h["alpha"][0], 1) - (h["rho_sq_num_t2"][0] / den2) ** 0.5) < 1e-12


def test_compensated_value_takes_two_roundings():
    # a = fl(eps + fl(alpha * g)) (first worker line of Algorithm 1/2), not a fused multiply-add.
    # alpha = g = 1 + 2^-12: alpha*g = 1 + 2^-11 + 2^-24, which rounds (tie to even) to 1 + 2^-11;
    # with eps = -(1 + 2^-11) the two-roundings value is exactly 0, the fused one 2^-24.
    one_p = np.float32(1.0 + 2.0 ** -12)
    tiny = np.float32(2.0 ** -30)
    G = np.array([[one_p, tiny, 0.0]], np.float32)
    eps = np.array([[-(1.0 + 2.0 ** -11), 0.0, 0.0]], np.float32)
    p = np.ones(1, np.float32)
    # exact products, as a check of the construction itself (float64 holds them exactly)
    assert float(one_p) * float(one_p) == 1.0 + 2.0 ** -11 + 2.0 ** -24
    assert np.float32(float(one_p) * float(one_p)) == np.float32(1.0 + 2.0 ** -11)
    a1 = np.float32(float(one_p) * float(tiny))              # alpha * 2^-30, far below 2^-24
    assert 0 < a1 < 2.0 ** -24
    for mode in (0, 1):
        r = oracle.ref_step_ef(np.zeros(3, np.float32), eps, np.zeros(3, np.float32), G, 1, 1, p, float(one_p), mode)
        # coordinate 0 compensates to exactly 0, so the tiny coordinate 1 is the one sent ...
        assert r.up_idx.tolist() == [[1]] and r.up_val[0, 0] == a1
        # ... and what stays in the memory at coordinate 0 is exactly zero (fused: 2^-24 would be sent)
        assert r.eps.tolist() == [[0.0, 0.0, 0.0]]
        assert r.w.tolist() == [0.0, -float(a1), 0.0]
    # the gap constants use the same a: Top_1(a) = {1}, Top_2(D_a) = {1, 0 (a zero)} -> difference 0;
    # a fused a_0 = 2^-24 would be sent instead of coordinate 1 and leave a non-zero difference
    assert oracle.ref_rho(G, eps, None, 1, 2, p, float(one_p), 0) == 0.0
    assert oracle.ref_rho(G, eps, np.zeros(3, np.float32), 1, 2, p, float(one_p), 1) == 0.0
