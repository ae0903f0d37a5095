"""tk_step with the error memories (TK_MODE_EF: Algorithm 1 / 2 as printed) against the CPU
oracle: w, epsilon, delta and both messages, every step, state carried from step to step."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_15203_b200 import binding, workloads as W
from util import assert_message_equal, assert_values_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
EF = binding.TK_MODE_EF


def run_ef(wl, steps, mode, K_down=None, force_general=False, misalign=0, alpha=None, keep=None):
    K_down = K_down or wl.K_down[0]
    alpha = wl.alpha if alpha is None else alpha
    p = W.make_p(wl)
    ctx = binding.Context(wl.d, wl.N, wl.K_up, K_down, p)
    ctx.tk_set_force_general(force_general)
    ctx.tk_ef_attach()
    eps_dev, delta_dev = ctx.tk_ef_state()
    assert not eps_dev.any() and not delta_dev.any()
    w_dev = W.make_w(wl, DEV)
    w = w_dev.cpu().numpy()
    eps = np.zeros((wl.N, wl.d), np.float32)
    delta = np.zeros(wl.d, np.float32)
    scale = W.scale_vector(wl, DEV)
    buf = torch.empty(wl.N * wl.d + 8, device=DEV, dtype=torch.float32)
    G = buf[misalign:misalign + wl.N * wl.d].view(wl.N, wl.d)
    for s in range(steps):
        W.make_grads(wl, s, DEV, out=G, scale=scale)
        if keep is not None:   # sparse gradients: all but a fraction `keep` of the components are exactly zero
            gen = torch.Generator(device=DEV)
            gen.manual_seed(77 + s)
            G.mul_((torch.rand(G.shape, generator=gen, device=DEV) < keep).to(torch.float32))
        ctx.tk_step(w_dev, G, alpha, mode | EF)
        ref = oracle.ref_step_ef(w, eps, delta, G.cpu().numpy(), wl.K_up, K_down, p.numpy(), alpha, mode)
        what = "config%d ef mode=%d step=%d" % (wl.cid, mode, s)
        st = ctx.tk_status()
        assert st.device_status == 0
        uidx, uval = ctx.tk_last_uplink()
        assert_message_equal(uidx, uval, ref.up_idx, ref.up_val, what + " uplink")
        midx, mval = ctx.tk_last_downlink()
        assert np.array_equal(midx.cpu().numpy(), ref.msg_idx), what + " downlink indices"
        assert_values_close(mval.cpu().numpy(), ref.msg_val, what + " downlink values")
        assert_values_close(w_dev.cpu().numpy(), ref.w, what + " w")
        assert_values_close(eps_dev.cpu().numpy(), ref.eps, what + " epsilon")
        if mode == 1:
            assert_values_close(delta_dev.cpu().numpy(), ref.delta, what + " delta")
            delta = ref.delta
        w, eps = ref.w, ref.eps
    ctx.close()


def test_hand_worked_two_iterations():
    p = torch.tensor([0.5, 0.5])
    G1 = torch.tensor([[4, 1, 0, -2], [1, -3, 2, 0]], dtype=torch.float32, device=DEV)
    G2 = torch.tensor([[0, 1, 0, -1], [2, 0, 1, 0]], dtype=torch.float32, device=DEV)
    for mode, w2 in ((1, [-3.5, 0, 0, 0]), (0, [-3.5, 1.5, 0, 1.5])):
        ctx = binding.Context(4, 2, 1, 1, p)
        ctx.tk_ef_attach()
        w = torch.zeros(4, device=DEV)
        ctx.tk_step(w, G1, 1.0, mode | EF)
        ctx.tk_step(w, G2, 1.0, mode | EF)
        eps, delta = ctx.tk_ef_state()
        assert ctx.tk_status().device_status == 0
        assert w.cpu().tolist() == w2
        assert eps.cpu().tolist() == [[0, 2, 0, 0], [0, 0, 3, 0]]
        if mode == 1:
            assert delta.cpu().tolist() == [0, -1.5, 0, -1.5]


@pytest.mark.parametrize("mode", [0, 1])
def test_long_rows_fused_path(mode):
    run_ef(W.workload(2, d=1_170_004, N=4), 4, mode)


@pytest.mark.parametrize("mode", [0, 1])
def test_short_rows_multi_pass_path(mode):
    run_ef(W.workload(1, d=50_001), 4, mode)


def test_ragged_rows_and_unaligned_gradients():
    run_ef(W.workload(5, d=1_000_003, N=3), 3, 1)                  # d % 4 != 0
    run_ef(W.workload(2, d=600_000, N=3), 3, 1, misalign=1)        # gradients not aligned like the memories


@pytest.mark.parametrize("mode", [0, 1])
def test_sparse_gradients_fewer_nonzeros_than_k(mode):
    # the compensated vectors and the server memory are nearly all zeros: the K-th largest is a zero
    run_ef(W.workload(2, d=1_170_004, N=4), 4, mode, keep=2e-4)


def test_forced_multi_pass_path():
    run_ef(W.workload(2, d=400_000, N=3), 3, 1, force_general=True)


def test_ties_zeros_and_large_kdown():
    wl = W.workload(4, d=600_000, N=6)
    run_ef(wl, 3, 1, K_down=wl.K_down[1])
    run_ef(wl, 2, 1, K_down=wl.K_down[2])


def test_student_dirichlet_many_steps():
    run_ef(W.workload(3, d=700_000, N=5), 6, 1)


@pytest.mark.parametrize("mode", [0, 1])
def test_toy_example_trajectory(mode):
    # the paper's toy example (appendix): three quadratics in R^100, K = 1, alpha = 0.01; 300
    # iterations with the gradients taken at the current w, GPU and oracle side by side
    d, N = 100, 3
    centres = np.array([1.0, 5.0, 10.0], np.float32)
    p = torch.full((N,), 1.0 / 3.0)
    np.random.seed(10)
    w_ref = np.random.normal(20, 1, d).astype(np.float32)
    ctx = binding.Context(d, N, 1, 1, p)
    ctx.tk_ef_attach()
    ctx.tk_set_diagnostics(2)
    w_dev = torch.from_numpy(w_ref.copy()).to(DEV)
    c_dev = torch.from_numpy(centres).to(DEV)
    eps = np.zeros((N, d), np.float32)
    delta = np.zeros(d, np.float32)
    rhos = []
    for t in range(300):
        G = (w_dev[None, :] - c_dev[:, None]).contiguous()
        Gh = (w_ref[None, :] - centres[:, None]).astype(np.float32)
        assert np.array_equal(G.cpu().numpy(), Gh)
        ctx.tk_step(w_dev, G, 0.01, mode | EF)
        ref = oracle.ref_step_ef(w_ref, eps, delta, Gh, 1, 1, p.numpy(), 0.01, mode)
        w_ref, eps = ref.w, ref.eps
        if mode == 1:
            delta = ref.delta
        if t % 50 == 49:
            assert np.array_equal(w_dev.cpu().numpy().view(np.uint32), w_ref.view(np.uint32)), "w diverged at t=%d" % t
            rhos.append(ctx.tk_diagnostics()[0].rho)
    e_dev, d_dev = ctx.tk_ef_state()
    assert np.array_equal(e_dev.cpu().numpy().view(np.uint32), eps.view(np.uint32))
    if mode == 1:
        assert np.array_equal(d_dev.cpu().numpy().view(np.uint32), delta.view(np.uint32))
    assert ctx.tk_status().device_status == 0 and all(r >= 0 for r in rhos)
    F = sum(0.5 * np.sum((w_ref.astype(np.float64) - c) ** 2) for c in (1.0, 5.0, 10.0)) / 3
    assert 6100 / 9 < F < 6100 / 9 + 40          # hovers near F* = 6100/9, as the paper describes


def test_needs_attached_memories():
    wl = W.workload(1, d=2000)
    ctx = binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, W.make_p(wl))
    w = torch.zeros(wl.d, device=DEV)
    G = torch.zeros((wl.N, wl.d), device=DEV)
    with pytest.raises(binding.TkError):
        ctx.tk_step(w, G, 0.1, binding.TK_MODE_BIDIR | EF)
    ctx.tk_ef_attach()
    ctx.tk_step(w, G, 0.1, binding.TK_MODE_BIDIR | EF)
    ctx.tk_set_kdown(2 * wl.K_up)                                   # larger than what was attached for
    with pytest.raises(binding.TkError):
        ctx.tk_step(w, G, 0.1, binding.TK_MODE_BIDIR | EF)
    ctx.tk_ef_attach()
    ctx.tk_step(w, G, 0.1, binding.TK_MODE_BIDIR | EF)
    assert ctx.tk_status().device_status == 0


def test_memory_free_steps_still_work_after_attach():
    wl = W.workload(2, d=300_000, N=3)
    ctx = binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, W.make_p(wl))
    ctx.tk_ef_attach()
    G = W.make_grads(wl, 0, DEV)
    w = W.make_w(wl, DEV)
    ref = oracle.ref_step(w.cpu().numpy(), G.cpu().numpy(), wl.K_up, wl.K_up, W.make_p(wl).numpy(), 0.1, 1)
    ctx.tk_step(w, G, 0.1, binding.TK_MODE_BIDIR)
    assert_values_close(w.cpu().numpy(), ref.w, "memory-free step")
    eps, delta = ctx.tk_ef_state()
    assert not eps.any() and not delta.any()


@pytest.mark.parametrize("cid,steps", [(2, 2), (5, 1)])
def test_full_size_configs_with_memories(cid, steps):
    import psutil
    wl = W.workload(cid)
    if psutil.virtual_memory().available < wl.N * wl.d * 4 * 6 + 16 * wl.d * 8:
        pytest.skip("not enough host memory for the oracle at this size")
    run_ef(wl, steps, 1)


def test_random_small_problems_with_memories():
    # many small shapes (every row alignment, tiny and large K, K_down above and below the union),
    # five steps each with the memories carried along
    rng = np.random.default_rng(915203)
    for case in range(16):
        N = int(rng.integers(1, 7))
        d = int(rng.integers(8, 30_000))
        K_up = int(rng.integers(1, max(2, d // 20)))
        K_down = int(rng.integers(1, min(d, 3 * N * K_up) + 1))
        mode = int(rng.integers(0, 2))
        p = torch.from_numpy(rng.dirichlet(np.ones(N)).astype(np.float32))
        ctx = binding.Context(d, N, K_up, K_down, p)
        ctx.tk_ef_attach()
        w_dev = torch.from_numpy(rng.standard_normal(d).astype(np.float32)).to(DEV)
        w = w_dev.cpu().numpy()
        eps = np.zeros((N, d), np.float32)
        delta = np.zeros(d, np.float32)
        for s in range(5):
            Gh = (rng.standard_t(3, (N, d)) * 1e-2).astype(np.float32)
            if case % 3 == 0:
                Gh = np.round(Gh * 64) / 64                      # coarse values: many ties
            G = torch.from_numpy(Gh.astype(np.float32)).to(DEV)
            ctx.tk_step(w_dev, G, 0.25, mode | EF)
            ref = oracle.ref_step_ef(w, eps, delta, Gh, K_up, K_down, p.numpy(), 0.25, mode)
            what = "case %d (N=%d d=%d K=%d/%d mode=%d) step %d" % (case, N, d, K_up, K_down, mode, s)
            midx, _ = ctx.tk_last_downlink()
            assert np.array_equal(midx.cpu().numpy(), ref.msg_idx), what
            assert_values_close(w_dev.cpu().numpy(), ref.w, what + " w")
            e_dev, d_dev = ctx.tk_ef_state()
            assert_values_close(e_dev.cpu().numpy(), ref.eps, what + " epsilon")
            if mode == 1:
                assert_values_close(d_dev.cpu().numpy(), ref.delta, what + " delta")
                delta = ref.delta
            w, eps = ref.w, ref.eps
        assert ctx.tk_status().device_status == 0
        ctx.close()
