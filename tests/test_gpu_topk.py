"""tk_topk (stage 1 alone) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_15203_b200 import binding, workloads as W
from util import assert_message_equal

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_both(x_host: np.ndarray, K: int, ctx=None, x_dev=None):
    x_host = np.ascontiguousarray(x_host, dtype=np.float32)
    if x_dev is None:
        x_dev = torch.from_numpy(x_host).to(DEV)
    idx, val = binding.tk_topk(x_dev, K, ctx=ctx)
    torch.cuda.synchronize()
    if x_host.ndim == 1:
        ridx, rval = oracle.ref_topk(x_host, K)
    else:
        ridx, rval = oracle.ref_topk_rows(x_host, K)
    assert_message_equal(idx, val, ridx, rval, "tk_topk d=%s K=%d" % (x_host.shape, K))


@pytest.mark.parametrize("d,K", [(1, 1), (2, 1), (3, 3), (5, 2), (7, 7), (8, 1), (33, 5), (1000, 10),
                                 (4097, 4097), (8192, 1), (8193, 100), (100_003, 1_000)])
def test_small_random(d, K):
    rng = np.random.default_rng(d * 31 + K)
    run_both(rng.standard_normal(d).astype(np.float32), K)
    run_both((rng.standard_t(3, (3, d)) * 1e-3).astype(np.float32), K)


def test_special_values():
    d = 5000
    rng = np.random.default_rng(0)
    run_both(np.zeros(d, np.float32), 17)                       # all zero: first K indices
    z = np.zeros(d, np.float32); z[::3] = -0.0
    run_both(z, 100)                                            # -0 ties with +0, sign bit is copied
    run_both(np.full(d, -3.5, np.float32), 999)                 # all equal
    x = rng.standard_normal(d).astype(np.float32)
    x[10], x[20], x[30] = np.inf, -np.inf, np.float32(3e38)
    run_both(x, 5)
    den = (rng.integers(1, 2 ** 22, d).astype(np.uint32)).view(np.float32)   # denormals only
    run_both(den, 50)
    mix = x.copy(); mix[::2] = den[::2]
    run_both(mix, d - 1)
    j = np.arange(d)
    run_both((((-1.0) ** j) * (j + 1)).astype(np.float32), 33)  # closed form: the last K indices


def test_nan_and_inf_are_ordered_by_bit_pattern():
    # inputs are meant to be finite; if they are not, NaN (largest keys) and Inf are still selected
    # exactly as the integer-key order says, on the sampled path and on the multi-pass path
    rng = np.random.default_rng(8)
    for d, K in ((300_000, 200), (20_000, 50)):
        x = rng.standard_normal((2, d)).astype(np.float32)
        x[0, [5, 77_77, d - 1]] = np.nan
        x[0, 123] = -np.inf
        x[1, 4_000] = np.float32(np.nan)
        x[1, 4_001] = np.inf
        run_both(x, K)


def test_k_equals_d_and_k_one():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 30_001)).astype(np.float32)
    run_both(x, 30_001)
    run_both(x, 1)


def test_ties_straddling_the_threshold():
    rng = np.random.default_rng(2)
    d = 200_000
    x = (rng.standard_normal((4, d)) * 1e-3).astype(np.float32)
    x[:, rng.integers(0, d, 30_000)] = np.float32(0.0021)       # a huge group of equal magnitudes
    x[1, rng.integers(0, d, 5_000)] = np.float32(-0.0021)
    for K in (10, 2_000, 31_000):
        run_both(x, K)


@pytest.mark.parametrize("off", [1, 2, 3])
def test_unaligned_rows(off):
    rng = np.random.default_rng(3 + off)
    d, rows = 40_001 + off, 3                                    # d % 4 != 0: rows start at every alignment
    buf = rng.standard_normal(rows * d + 8).astype(np.float32)
    dev = torch.from_numpy(buf).to(DEV)
    x_dev = dev[off:off + rows * d].view(rows, d)
    assert x_dev.data_ptr() % 16 != 0
    run_both(buf[off:off + rows * d].reshape(rows, d), 123, x_dev=x_dev)


def test_predicted_path_large_rows():
    # rows long enough for the sampled threshold; d is ragged against every tile size
    wl = W.workload(5, d=2_000_003, N=5)
    G = W.make_grads(wl, 0, DEV)
    run_both(G.cpu().numpy(), wl.K_up, x_dev=G)
    wl = W.workload(3, d=1_500_001, N=3)
    G = W.make_grads(wl, 0, DEV)
    run_both(G.cpu().numpy(), wl.K_up, x_dev=G)


@pytest.mark.parametrize("K", [15_000, 40_000, 300_000])
def test_large_k_on_long_rows(K):
    # 1 % (sampled path), 2.7 % and 20 % (beyond d/64: multi-pass path with large candidate lists)
    wl = W.workload(3, d=1_500_000, N=3)
    G = W.make_grads(wl, 2, DEV)
    run_both(G.cpu().numpy(), K, x_dev=G)


def test_rows_whose_prediction_must_fail():
    d, K = 1_200_000, 1_000
    rng = np.random.default_rng(4)
    x = (rng.standard_normal((4, d)) * 1e-3).astype(np.float32)
    x[0, :] = 0.5                                                # all equal: every candidate list overflows
    x[1, :] = 0.0
    x[1, 7] = 1.0                                                # one non-zero, the rest tie at zero
    x[2, :600_000] = np.float32(0.25)                            # half the row ties above the rest
    x[3, :] *= 1e-3                                              # an ordinary row next to the failing ones
    run_both(x, K)


def test_rows_the_sample_misjudges_stay_on_the_single_pass_path():
    # (a) fewer non-zeros than K: the K-th largest is a zero, zeros rank by index;
    # (b) the K largest packed into one short block of huge values, which the sample under-counts;
    # (c) a few more non-zeros than K.  All exact, and none needs the multi-pass path.
    d, K, rows = 4_000_003, 2_000, 4
    rng = np.random.default_rng(515)
    x = np.zeros((rows, d), dtype=np.float32)
    x[0, rng.choice(d, 700, replace=False)] = rng.standard_normal(700).astype(np.float32)
    x[0, rng.choice(d, 5000, replace=False)] *= np.float32(-1.0)        # some of the zeros become -0
    x[1] = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    x[1, 1_234_567:1_234_567 + 20_000] *= np.float32(1000.0)
    x[2, rng.choice(d, 2_300, replace=False)] = rng.standard_normal(2_300).astype(np.float32)
    x[3] = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    ctx = binding.Context(d, rows, K, K, torch.full((rows,), 1.0 / rows))
    run_both(x, K, ctx=ctx)
    st = ctx.tk_status()
    assert st.rows_general == 0, "every row should verify with its sampled bound"
    assert st.cand_max < 40_000
    ctx.close()


def test_predicted_and_general_paths_agree_bitwise():
    wl = W.workload(2, d=1_170_000, N=6)
    G = W.make_grads(wl, 1, DEV)
    ctx = binding.Context(wl.d, wl.N, wl.K_up, wl.K_up, W.make_p(wl))
    a = binding.tk_topk(G, wl.K_up, ctx=ctx)
    st = ctx.tk_status()
    assert st.rows_general == 0, "the sampled threshold should verify on this input"
    ctx.tk_set_force_general(True)
    b = binding.tk_topk(G, wl.K_up, ctx=ctx)
    st = ctx.tk_status()
    assert st.rows_general == wl.N
    assert torch.equal(a[0], b[0]) and torch.equal(a[1].view(torch.int32), b[1].view(torch.int32))
    run_both(G.cpu().numpy(), wl.K_up, x_dev=G, ctx=ctx)


def test_repeatable_bits():
    wl = W.workload(4, d=1_170_000, N=4)
    G = W.make_grads(wl, 0, DEV)
    a = binding.tk_topk(G, wl.K_up)
    b = binding.tk_topk(G, wl.K_up)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1].view(torch.int32), b[1].view(torch.int32))
    run_both(G.cpu().numpy(), wl.K_up, x_dev=G)


def test_random_shapes_sweep():
    # many small problems of random shape, half of them tie-heavy: rows, d, K at every alignment
    rng = np.random.default_rng(2209)
    mags = np.array([0.0, 1e-3, 0.5, 0.5, 2.0, 7.25, 1e-41], dtype=np.float32)
    for case in range(60):
        rows = int(rng.integers(1, 6))
        d = int(rng.integers(1, 40_000))
        K = int(rng.integers(1, d + 1)) if case % 3 else int(rng.integers(1, min(d, 50) + 1))
        if case % 2:
            x = mags[rng.integers(0, mags.size, (rows, d))] * rng.choice(np.array([-1.0, 1.0], np.float32), (rows, d))
        else:
            x = rng.standard_normal((rows, d)) * np.exp(rng.standard_normal((rows, d)) * 2)
        run_both(x.astype(np.float32), K)


def test_more_rows_than_one_launch_takes():
    # rows are processed in batches of 4096: short rows (multi-pass path) across two batch boundaries
    rng = np.random.default_rng(77)
    run_both(rng.standard_normal((9000, 301)).astype(np.float32), 7)
    # ... and rows just long enough for the sampled path (its many-rows variant); the oracle checks
    # a sample of the rows, among them the ones on either side of the batch boundary
    rows, d, K = 4200, 131_102, 100
    g = torch.Generator(device=DEV)
    g.manual_seed(78)
    x = torch.randn((rows, d), generator=g, device=DEV, dtype=torch.float32)
    idx, val = binding.tk_topk(x, K)
    torch.cuda.synchronize()
    pick = np.unique(np.concatenate([[0, 1, 4094, 4095, 4096, 4097, rows - 1], rng.integers(0, rows, 40)]))
    ridx, rval = oracle.ref_topk_rows(x[torch.from_numpy(pick).to(DEV)].cpu().numpy(), K)
    assert_message_equal(idx[pick], val[pick], ridx, rval, "tk_topk 4200 rows (sampled rows)")
    # all rows: the selected magnitudes are the K largest of the row (torch.topk on |x|, values only)
    top = torch.topk(x.abs(), K, dim=1).values.sort(dim=1).values
    assert torch.equal(val.abs().sort(dim=1).values, top)


def test_argument_errors():
    x = torch.zeros(100, device=DEV)
    with pytest.raises(binding.TkError):
        binding.tk_topk(x, 101)
    with pytest.raises(binding.TkError):
        binding.tk_topk(x, 0)
