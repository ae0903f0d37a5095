"""tk_step against the CPU oracle: every stage, every step, on the five workloads."""
import numpy as np
import psutil
import pytest
import torch

import oracle
from paper_2209_15203_b200 import binding, workloads as W
from util import assert_message_equal, assert_values_close, bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def check_step(ctx, wl, w_dev, w_ref, G, alpha, mode, K_down, what):
    """One step on both sides; returns the oracle's new w."""
    ctx.tk_step(w_dev, G, alpha, mode)
    ref = oracle.ref_step(w_ref, G.cpu().numpy(), wl.K_up, K_down, ctx_p(ctx), alpha, mode)
    st = ctx.tk_status()
    assert st.device_status == 0
    # stage 1: the uplink messages
    uidx, uval = ctx.tk_last_uplink()
    assert_message_equal(uidx, uval, ref.up_idx, ref.up_val, what + " uplink")
    # stage 2: the aggregate over the union
    U = np.nonzero(ref.touched)[0].astype(np.int32)
    aidx, aval = ctx.tk_last_aggregate()
    assert st.union_size == U.size <= wl.N * wl.K_up
    assert np.array_equal(aidx.cpu().numpy(), U), what + " union"
    assert_values_close(aval.cpu().numpy(), ref.A[U], what + " aggregate")
    # stage 3: the downlink message
    midx, mval = ctx.tk_last_downlink()
    assert np.array_equal(midx.cpu().numpy(), ref.msg_idx), what + " downlink indices"
    assert_values_close(mval.cpu().numpy(), ref.msg_val, what + " downlink values")
    # stage 4: the update
    assert_values_close(w_dev.cpu().numpy(), ref.w, what + " w")
    # housekeeping: the dense server buffer is back to zero (checked through the next step's union)
    return ref.w


_P = {}


def ctx_p(ctx):
    return _P[id(ctx)]


def make_ctx(wl, K_down):
    p = W.make_p(wl)
    ctx = binding.Context(wl.d, wl.N, wl.K_up, K_down, p)
    _P[id(ctx)] = p.numpy()
    return ctx


def run_workload(wl, steps, modes=None, force_general=False):
    scale = W.scale_vector(wl, DEV)
    G = torch.empty((wl.N, wl.d), device=DEV, dtype=torch.float32)
    for mode in (modes or wl.modes):
        for K_down in wl.K_down:
            ctx = make_ctx(wl, K_down)
            ctx.tk_set_force_general(force_general)
            w_dev = W.make_w(wl, DEV)
            w_ref = w_dev.cpu().numpy()
            for s in range(steps):
                W.make_grads(wl, s, DEV, out=G, scale=scale)
                what = "config%d mode=%d K_down=%d step=%d" % (wl.cid, mode, K_down, s)
                w_ref = check_step(ctx, wl, w_dev, w_ref, G, wl.alpha, mode, K_down, what)
            ctx.close()


def test_hand_computed_iteration():
    G = np.array([[1, -8, 0.5, 3, 0, -2, 4, 0.25], [-6, 2, 2, 1, 0, 5, -0.5, 3], [4, 4, -4, 1, 2, 0, 6, -1]],
                 np.float32)
    p = torch.tensor([0.5, 0.25, 0.25])
    for mode, expect in ((1, [1, 3, 1, 1, 1, 1, -0.75, 1]), (0, [1.25, 3, 1, 1, 1, 0.375, -0.75, 1])):
        ctx = binding.Context(8, 3, 2, 2, p)
        w = torch.ones(8, device=DEV)
        ctx.tk_step(w, torch.from_numpy(G).to(DEV), 0.5, mode)
        assert ctx.tk_status().device_status == 0
        assert w.cpu().tolist() == expect


def test_config1_full_size_all_steps_both_modes():
    wl = W.workload(1)
    run_workload(wl, wl.steps)


@pytest.mark.parametrize("cid,d", [(2, 1_170_003), (3, 1_280_001), (4, 1_170_000), (5, 3_100_002)])
def test_scaled_configs_every_step(cid, d):
    wl = W.workload(cid, d=d)
    run_workload(wl, 3)


@pytest.mark.parametrize("cid", [6, 8, 9, 10])
def test_paper_shaped_workloads(cid):
    # N = 20..100 workers, d not a multiple of 4 (rows start at every alignment), tiny K
    wl = W.workload(cid)
    assert wl.d % 4 != 0
    run_workload(wl, 2)


def test_paper_vgg19_shape_one_step():
    wl = W.workload(7)
    run_workload(wl, 1, modes=(1,))


def test_scaled_configs_forced_general_path():
    run_workload(W.workload(2, d=600_001, N=4), 2, force_general=True)
    run_workload(W.workload(4, d=500_000, N=6), 2, force_general=True)


def test_forced_list_overflow_redoes_every_row_exactly():
    # host-side fault injection: with the candidate lists capped just above K every row of an ordinary
    # input overflows its list in the streaming pass, fails verification and is redone by the exact
    # multi-pass path; the results are the oracle's all the same
    for wl in (W.workload(2, d=600_001, N=4), W.workload(3, d=700_002, N=5)):
        ctx = make_ctx(wl, wl.K_down[0])
        w_dev = W.make_w(wl, DEV)
        w_ref = w_dev.cpu().numpy()
        for s, cap in enumerate((wl.K_up + 5, 1, 0, wl.K_up)):     # 1 is raised to K; 0 restores the full lists
            ctx.tk_set_cand_cap(cap)
            G = W.make_grads(wl, s, DEV)
            w_ref = check_step(ctx, wl, w_dev, w_ref, G, wl.alpha, 1, wl.K_down[0], "capped lists cap=%d" % cap)
            st = ctx.tk_status()
            assert st.rows_general == (0 if cap == 0 else wl.N), (cap, st.rows_general)
        # the standalone selection with the same context obeys the cap too
        ctx.tk_set_cand_cap(wl.K_up + 1)
        G = W.make_grads(wl, 9, DEV)
        idx, val = ctx.tk_topk(G, wl.K_up)
        ref_idx, ref_val = oracle.ref_topk_rows(G.cpu().numpy(), wl.K_up)
        assert_message_equal(idx, val, ref_idx, ref_val, "tk_topk with capped lists")
        assert ctx.tk_status().rows_general == wl.N
        ctx.close()


def test_kept_bounds_survive_changes_of_scale():
    # A row starts from the threshold of the step before, minus a margin (tk_set_bound_reuse, on by
    # default).  Steps of the same distribution then take the single streaming pass without sampling; a
    # step whose vectors are a thousand times smaller (the warm-started bound admits nothing) must be
    # redone by the exact multi-pass path, and after such a jump the rows sample afresh (their
    # thresholds have just shown that they move).  Results are the oracle's throughout; with reuse off
    # no step needs the multi-pass path.
    wl = W.workload(2, d=700_003, N=5)
    scales = (1.0, 1.0, 1e-3, 1.0, 1.0, 1e3, 1.0, 0.97, 1.04)
    for reuse in (True, False):
        ctx = make_ctx(wl, wl.K_down[0])
        ctx.tk_set_bound_reuse(reuse)
        w_dev = W.make_w(wl, DEV)
        w_ref = w_dev.cpu().numpy()
        general = []
        for s, c in enumerate(scales):
            G = W.make_grads(wl, s, DEV) * c
            w_ref = check_step(ctx, wl, w_dev, w_ref, G, wl.alpha, 1, wl.K_down[0], "scale %g reuse=%s" % (c, reuse))
            general.append(ctx.tk_status().rows_general)
        if reuse:
            # (after a failed attempt the rows sample for two steps before a bound is kept again)
            assert general == [0, 0, wl.N, 0, 0, 0, 0, 0, 0] or general == [0, 0, wl.N, 0, 0, wl.N, 0, 0, 0], general
        else:
            assert general == [0] * len(scales), general
        if reuse:
            # thresholds that jump every step: the back-off (2, 4, 8 ... steps of sampling after each failed
            # attempt) keeps the failed attempts few
            failed = 0
            for s in range(14):
                G = W.make_grads(wl, 20 + s, DEV) * (1e-3 if s % 2 else 1.0)
                w_ref = check_step(ctx, wl, w_dev, w_ref, G, wl.alpha, 1, wl.K_down[0], "alternating scale step %d" % s)
                failed += 1 if ctx.tk_status().rows_general else 0
            assert failed <= 3, failed
        ctx.close()


def test_kdown_larger_than_union_pads_with_zero_entries():
    wl = W.workload(4, d=400_000, N=4)          # K_up = 40, union <= 160; K_down = 4000 > |U|
    assert wl.K_down[-1] > wl.N * wl.K_up
    run_workload(wl, 2)


def test_set_kdown_between_steps():
    wl = W.workload(2, d=300_000, N=3)
    ctx = make_ctx(wl, wl.K_up)
    w_dev = W.make_w(wl, DEV)
    w_ref = w_dev.cpu().numpy()
    for s, kd in enumerate((wl.K_up, 7, 3 * wl.K_up, 1)):
        ctx.tk_set_kdown(kd)
        G = W.make_grads(wl, s, DEV)
        w_ref = check_step(ctx, wl, w_dev, w_ref, G, 0.05, 1, kd, "set_kdown %d" % kd)


def test_warm_started_steps_on_a_random_walk():
    # What the library carries from step to step only steers speed: the rows' kept bounds and the
    # centre of the downlink selection's first-level buckets.  Thirty steps whose scale drifts by up to
    # +-15 % a step (sometimes jumping), with K_down and the mode changing under way, on a long-row
    # workload whose union takes several CTAs: every step must equal the oracle's, with graph replay
    # as the benchmark runs it.
    rng = np.random.default_rng(2209)
    for cid, d, N in ((2, 900_001, 12), (3, 600_002, 9)):
        wl = W.workload(cid, d=d, N=N)
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            p = W.make_p(wl)
            ctx = binding.Context(wl.d, wl.N, wl.K_up, wl.K_down[0], p, stream=stream)
            _P[id(ctx)] = p.numpy()
            ctx.tk_set_graph(True)
            w_dev = W.make_w(wl, DEV)
            w_ref = w_dev.cpu().numpy()
            scale = 1.0
            redone = 0
            for s in range(30):
                scale *= float(np.exp(rng.uniform(-0.15, 0.15)))
                if s in (11, 23):
                    scale *= 0.05 if s == 11 else 30.0
                kd = int(rng.choice([wl.K_up, wl.K_up // 7 + 1, 5 * wl.K_up, wl.K_up]))
                mode = int(rng.random() < 0.8)
                ctx.tk_set_kdown(kd)
                G = W.make_grads(wl, s, DEV) * scale
                torch.cuda.synchronize()
                w_ref = check_step(ctx, wl, w_dev, w_ref, G, wl.alpha, mode, kd, "walk config%d step %d scale %.3g" % (cid, s, scale))
                redone += 1 if ctx.tk_status().rows_general else 0
            assert redone <= 6, redone       # the two jumps, and what a 15 % drift occasionally costs
            ctx.close()


def test_cancelling_workers_and_zero_weights():
    d, K = 50_000, 64
    rng = np.random.default_rng(5)
    g = rng.standard_normal(d).astype(np.float32)
    G = np.stack([g, -g, g * 0.5, rng.standard_normal(d).astype(np.float32)])
    for p in ([0.25, 0.25, 0.25, 0.25], [0.5, 0.5, 0.0, 0.0], [0.0, 0.0, 0.0, 1.0]):
        pt = torch.tensor(p)
        for mode in (0, 1):
            ctx = binding.Context(d, 4, K, K, pt)
            _P[id(ctx)] = pt.numpy()
            wl = W.workload(1, d=d)
            wl = wl.__class__(**{**wl.__dict__, "N": 4, "K_up": K, "K_down": (K,)})
            w_dev = torch.zeros(d, device=DEV)
            check_step(ctx, wl, w_dev, np.zeros(d, np.float32), torch.from_numpy(G).to(DEV), 1.0, mode, K,
                       "cancel p=%s mode=%d" % (p, mode))


@pytest.mark.parametrize("N,d,K_up,K_down", [(5000, 2003, 3, 40), (65535, 4001, 2, 300)])
def test_many_workers(N, d, K_up, K_down):
    # more workers than one selection launch takes (4096), and the largest N the ABI accepts
    rng = np.random.default_rng(N)
    G = torch.from_numpy(rng.standard_normal((N, d)).astype(np.float32)).to(DEV)
    p = torch.from_numpy((rng.random(N) / N).astype(np.float32))
    wl = W.workload(1, d=d, N=N)
    wl = wl.__class__(**{**wl.__dict__, "K_up": K_up, "K_down": (K_down,)})
    for mode in (0, 1):
        ctx = binding.Context(d, N, K_up, K_down, p)
        _P[id(ctx)] = p.numpy()
        w_dev = torch.from_numpy(rng.standard_normal(d).astype(np.float32)).to(DEV)
        w_ref = w_dev.cpu().numpy()
        for s in range(2):
            w_ref = check_step(ctx, wl, w_dev, w_ref, G, 0.05, mode, K_down, "N=%d mode=%d step=%d" % (N, mode, s))
        ctx.close()


@pytest.mark.parametrize("N,d,K_up", [(128, 400_003, 2500), (200, 300_002, 1600)])
def test_more_entries_than_one_wave_of_server_threads(N, d, K_up):
    # N*K_up above 148 * 2048 threads: the server sum runs in several waves of CTAs, with the slot table
    # (N = 128) and with chains (N = 200); each coordinate is sent by 1.6 workers on average
    rng = np.random.default_rng(N + K_up)
    p = torch.from_numpy((rng.random(N) / N).astype(np.float32))
    wl = W.workload(1, d=d, N=N)
    K_down = 3 * K_up
    wl = wl.__class__(**{**wl.__dict__, "K_up": K_up, "K_down": (K_down,)})
    ctx = binding.Context(d, N, K_up, K_down, p)
    _P[id(ctx)] = p.numpy()
    w_dev = torch.from_numpy(rng.standard_normal(d).astype(np.float32)).to(DEV)
    w_ref = w_dev.cpu().numpy()
    for s, mode in enumerate((1, 0, 1)):
        G = torch.from_numpy(rng.standard_normal((N, d), dtype=np.float32)).to(DEV)
        w_ref = check_step(ctx, wl, w_dev, w_ref, G, 0.05, mode, K_down, "N=%d K_up=%d mode=%d step=%d" % (N, K_up, mode, s))
    ctx.close()


@pytest.mark.parametrize("N,noise", [(20, 0.01), (100, 0.01), (150, 0.0)])
def test_workers_that_agree(N, noise):
    # correlated gradients: almost every selected coordinate is sent by all N workers, so the sums
    # have N terms (more than one window of workers, and with N = 150 more than the server step
    # remembers from its first walk of a chain)
    d, K = 60_002, 300
    rng = np.random.default_rng(1000 + N)
    base = rng.standard_normal(d)
    G = torch.from_numpy((base[None, :] * (1.0 + noise * rng.standard_normal((N, d)))).astype(np.float32)).to(DEV)
    p = torch.from_numpy((rng.random(N) + 0.5).astype(np.float32) / N)
    wl = W.workload(1, d=d, N=N)
    wl = wl.__class__(**{**wl.__dict__, "K_up": K, "K_down": (K,)})
    for mode in (0, 1):
        ctx = binding.Context(d, N, K, K, p)
        _P[id(ctx)] = p.numpy()
        w_dev = torch.from_numpy(rng.standard_normal(d).astype(np.float32)).to(DEV)
        w_ref = check_step(ctx, wl, w_dev, w_dev.cpu().numpy(), G, 0.05, mode, K, "agreeing workers N=%d mode=%d" % (N, mode))
        assert ctx.tk_status().union_size < 2 * K
        check_step(ctx, wl, w_dev, w_ref, G, 0.05, mode, K, "agreeing workers N=%d mode=%d step 2" % (N, mode))
        ctx.close()


@pytest.mark.parametrize("mode", [0, 1])
def test_sparse_gradients_fewer_nonzeros_than_k(mode):
    # rows of nearly all zeros (some of them -0): the messages are padded with the first zeros by index
    wl = W.workload(2, d=1_170_004, N=5)
    ctx = make_ctx(wl, wl.K_down[0])
    gen = torch.Generator(device=DEV)
    gen.manual_seed(4242)
    w_dev = W.make_w(wl, DEV)
    w_ref = w_dev.cpu().numpy()
    for s in range(2):
        G = W.make_grads(wl, s, DEV)
        G.mul_((torch.rand(G.shape, generator=gen, device=DEV) < 3e-4).to(torch.float32))
        w_ref = check_step(ctx, wl, w_dev, w_ref, G, wl.alpha, mode, wl.K_down[0], "sparse rows mode=%d step=%d" % (mode, s))
        assert ctx.tk_status().rows_general == 0
    ctx.close()


def test_random_problems_sweep():
    # many shapes at every alignment: short rows (multi-pass path) and rows long enough for the sampled
    # path; N from 1 to 140 (slot table up to 128 workers, chains above); coarse values make the workers
    # share coordinates and tie; K_down below and above the union size
    rng = np.random.default_rng(220915)
    for case in range(24):
        long_rows = case % 4 == 3
        N = int(rng.integers(1, 9)) if long_rows else int(rng.choice([1, 2, 3, 5, 17, 64, 129, 140]))
        d = int(rng.integers(140_000, 400_000)) if long_rows else int(rng.integers(4, 9_000))
        K_up = int(rng.integers(1, max(2, d // (200 if long_rows else 12))))
        K_down = int(rng.integers(1, min(d, 2 * N * K_up) + 1))
        p = torch.from_numpy(rng.dirichlet(np.ones(N)).astype(np.float32))
        wl = W.workload(1, d=d, N=N)
        wl = wl.__class__(**{**wl.__dict__, "K_up": K_up, "K_down": (K_down,)})
        for mode in (0, 1):
            ctx = binding.Context(d, N, K_up, K_down, p)
            _P[id(ctx)] = p.numpy()
            w_dev = torch.from_numpy(rng.standard_normal(d).astype(np.float32)).to(DEV)
            w_ref = w_dev.cpu().numpy()
            for s in range(2):
                Gh = rng.standard_t(3, (N, d)) * 1e-2
                if case % 3 == 0:
                    Gh = np.round(Gh * 32) / 32
                if case % 5 == 0 and N > 1:
                    Gh[1:] = Gh[0] * (1 + 0.05 * rng.standard_normal((N - 1, d)))
                G = torch.from_numpy(Gh.astype(np.float32)).to(DEV)
                w_ref = check_step(ctx, wl, w_dev, w_ref, G, 0.3, mode, K_down,
                                   "sweep case %d N=%d d=%d K=%d/%d mode=%d step=%d" % (case, N, d, K_up, K_down, mode, s))
            ctx.close()


def test_step_host_matches_device_step():
    wl = W.workload(2, d=500_000, N=4)
    G = W.make_grads(wl, 0, DEV)
    w0 = W.make_w(wl, DEV)
    ctx = make_ctx(wl, wl.K_up)
    w_dev = w0.clone()
    ctx.tk_step(w_dev, G, 0.1, 1)
    w_host = w0.cpu().pin_memory()
    ctx.tk_step_host(w_host, G.cpu().pin_memory(), 0.1, 1)
    assert torch.equal(w_host, w_dev.cpu())


def test_same_input_twice_gives_identical_bytes():
    wl = W.workload(3, d=900_000, N=8)
    G = W.make_grads(wl, 0, DEV)
    outs = []
    for _ in range(2):
        ctx = make_ctx(wl, wl.K_up)
        w = W.make_w(wl, DEV)
        ctx.tk_step(w, G, 0.1, 1)
        i, v = ctx.tk_last_downlink()
        outs.append((w.clone(), i.clone(), v.clone()))
    assert torch.equal(outs[0][0].view(torch.int32), outs[1][0].view(torch.int32))
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2].view(torch.int32), outs[1][2].view(torch.int32))


def test_diagnostics_match_the_oracle():
    # Section 4.2's non-zero fraction and the appendix's 1 - gamma, memory-free and with memories
    for wl, ef in ((W.workload(4, d=600_000, N=6), False), (W.workload(2, d=500_000, N=4), True),
                   (W.workload(1, d=30_000), False)):
        p = W.make_p(wl)
        K_down = wl.K_down[0]
        ctx = make_ctx(wl, K_down)
        ctx.tk_set_diagnostics(1)
        if ef:
            ctx.tk_ef_attach()
        w = W.make_w(wl, DEV)
        w_ref = w.cpu().numpy()
        eps = np.zeros((wl.N, wl.d), np.float32)
        delta = np.zeros(wl.d, np.float32)
        for s in range(2):
            G = W.make_grads(wl, s, DEV)
            Gh = G.cpu().numpy()
            ctx.tk_step(w, G, wl.alpha, 1 | (binding.TK_MODE_EF if ef else 0))
            diag, per = ctx.tk_diagnostics()
            if ef:
                a = (eps + np.float32(wl.alpha) * Gh).astype(np.float32)
                ref = oracle.ref_step_ef(w_ref, eps, delta, Gh, wl.K_up, K_down, p.numpy(), wl.alpha, 1)
                S, _ = oracle.ref_aggregate(ref.up_idx, ref.up_val, p.numpy(), wl.d)
                g = (S + delta).astype(np.float32)
                eps, delta = ref.eps, ref.delta
            else:
                a = Gh
                ref = oracle.ref_step(w_ref, Gh, wl.K_up, K_down, p.numpy(), wl.alpha, 1)
                S = g = ref.A
            w_ref = ref.w
            want = [oracle.ref_lost_energy(a[q], ref.up_idx[q]) for q in range(wl.N)]
            assert np.allclose(per, want, rtol=0, atol=2e-5)
            assert abs(diag.one_minus_gamma_up_max - max(want)) < 2e-5
            assert diag.one_minus_gamma_up_max <= (wl.d - wl.K_up) / wl.d + 2e-5     # Eq. "topk_bound"
            assert abs(diag.one_minus_gamma_down - oracle.ref_lost_energy(g, ref.msg_idx)) < 2e-5
            assert diag.nonzero_fraction == np.count_nonzero(S) / wl.d
            assert diag.nonzero_fraction <= diag.union_fraction <= wl.N * wl.K_up / wl.d
            assert diag.compression_factor == K_down / (wl.K_up * wl.N)
        ctx.close()


def test_graph_replay_matches_direct_launches():
    wl = W.workload(2, d=500_000, N=4)
    p = W.make_p(wl)
    bufs = [W.make_grads(wl, s, DEV) for s in range(3)]
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for ef in (False, True):
        mode = 1 | (binding.TK_MODE_EF if ef else 0)
        direct = binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, p)
        with torch.cuda.stream(side):
            graphed = binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, p, stream=side)
            graphed.tk_set_graph(True)
        if ef:
            direct.tk_ef_attach()
            graphed.tk_ef_attach()
        wa, wb = W.make_w(wl, DEV), W.make_w(wl, DEV)
        torch.cuda.synchronize()
        for s in range(9):                       # every buffer is captured once and replayed twice
            kd = wl.K_up if s < 6 else 7         # a new K_down is a new graph
            direct.tk_set_kdown(kd)
            graphed.tk_set_kdown(kd)
            direct.tk_step(wa, bufs[s % 3], wl.alpha, mode)
            with torch.cuda.stream(side):
                graphed.tk_step(wb, bufs[s % 3], wl.alpha, mode)
        torch.cuda.synchronize()
        assert graphed.tk_status().device_status == 0
        assert torch.equal(wa.view(torch.int32), wb.view(torch.int32))
        assert graphed.tk_launch_count() == direct.tk_launch_count()
        ia, va = direct.tk_last_downlink()
        ib, vb = graphed.tk_last_downlink()
        assert torch.equal(ia, ib) and torch.equal(va.view(torch.int32), vb.view(torch.int32))


@pytest.mark.parametrize("ef", [False, True])
@pytest.mark.parametrize("mode", [0, 1])
def test_gap_constant_matches_the_oracle(mode, ef):
    # rho_hat (unidirectional) / rho (bidirectional) of every step, memories carried along
    for wl in (W.workload(2, d=400_000, N=4), W.workload(1, d=20_000)):
        p = W.make_p(wl)
        K_down = wl.K_down[0]
        ctx = make_ctx(wl, K_down)
        if ef:
            ctx.tk_ef_attach()
        ctx.tk_set_diagnostics(2)
        w = W.make_w(wl, DEV)
        w_ref = w.cpu().numpy()
        eps = np.zeros((wl.N, wl.d), np.float32)
        delta = np.zeros(wl.d, np.float32)
        for s in range(3):
            G = W.make_grads(wl, s, DEV)
            Gh = G.cpu().numpy()
            ctx.tk_step(w, G, wl.alpha, mode | (binding.TK_MODE_EF if ef else 0))
            diag, _ = ctx.tk_diagnostics()
            if ef:
                want = oracle.ref_rho(Gh, eps, delta if mode == 1 else None, wl.K_up, K_down, p.numpy(), wl.alpha, mode)
                ref = oracle.ref_step_ef(w_ref, eps, delta, Gh, wl.K_up, K_down, p.numpy(), wl.alpha, mode)
                eps = ref.eps
                if mode == 1:
                    delta = ref.delta
            else:
                want = oracle.ref_rho(Gh, None, None, wl.K_up, K_down, p.numpy(), wl.alpha, mode)
                ref = oracle.ref_step(w_ref, Gh, wl.K_up, K_down, p.numpy(), wl.alpha, mode)
            w_ref = ref.w
            assert want > 0
            assert abs(diag.rho - want) <= 1e-5 * want, (mode, ef, s, diag.rho, want)
            assert_values_close(w.cpu().numpy(), ref.w, "w with diagnostics on")
        assert ctx.tk_status().device_status == 0
        ctx.close()


def test_bad_arguments_are_rejected():
    wl = W.workload(1, d=1000)
    ctx = make_ctx(wl, 10)
    w = torch.zeros(1000, device=DEV)
    G = torch.zeros((4, 1000), device=DEV)
    with pytest.raises(binding.TkError):
        ctx.tk_step(w, G, float("nan"), 1)
    with pytest.raises(binding.TkError):
        ctx.tk_step(w, G, 0.1, 2)
    with pytest.raises(binding.TkError):
        ctx.tk_set_kdown(1001)
    with pytest.raises(binding.TkError):
        binding.Context(1000, 4, 10, 10, torch.tensor([0.5, -0.1, 0.3, 0.3]))


# ---- full sizes, in the launch configuration the benchmark times ----

def _host_can_hold(wl):
    need = wl.N * wl.d * 4 * 2 + min(wl.N, oracle.ref.default_threads()) * wl.d * 16 + wl.d * 40
    return psutil.virtual_memory().available > need * 1.2


@pytest.mark.parametrize("cid,steps,mode,kdowns", [(2, 2, 1, None), (3, 1, 1, None), (3, 1, 0, None), (4, 1, 1, (0, 2)),
                                                   (4, 1, 1, (1,)), (5, 1, 1, None)])
def test_full_size_configs(cid, steps, mode, kdowns):
    # every leg the five configurations name, a slice of its steps each (the opt-in acceptance run
    # of test_gpu_acceptance.py does all steps): config 3 in both modes, config 4 at its three K_down
    wl = W.workload(cid)
    if not _host_can_hold(wl):
        pytest.skip("not enough host memory for the oracle at this size")
    if kdowns is not None:
        wl = wl.__class__(**{**wl.__dict__, "K_down": tuple(wl.K_down[i] for i in kdowns)})
    run_workload(wl, steps, modes=(mode,))
