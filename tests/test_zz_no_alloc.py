"""tk_topk_noalloc: the allocation-free variant of tk_topk.

Some users of the library run where cudaMalloc is off limits (a plugin inside
another program's memory budget, a loop that must never hit the allocator's
locks or cudaFree's device-wide synchronisation).  For them the library keeps
its scratch in a fixed array inside its own image.  This file checks, through
the C ABI, that the variant returns exactly what the CPU oracle and tk_topk
return, on calls in a row that find each other's leftovers in the shared
array and between them cover every path the selection can take; that the
device's free memory does not move across such calls; and that a problem larger
than the array is refused instead of overrunning it.
It is named so that pytest collects it after every other test file.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_15203_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check(x, K, against_tk_topk=True):
    rows = x.shape[0]
    idx = torch.full((rows, K), -1, dtype=torch.int32, device=DEV)
    val = torch.full((rows, K), float("nan"), dtype=torch.float32, device=DEV)
    binding.tk_topk_noalloc(x, K, idx, val)
    torch.cuda.synchronize()
    ref_idx, ref_val = oracle.ref_topk_rows(x.cpu().numpy(), K)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    assert np.array_equal(val.cpu().numpy().view(np.uint32), ref_val.view(np.uint32))
    if against_tk_topk:
        ridx, rval = binding.tk_topk(x, K)
        torch.cuda.synchronize()
        assert torch.equal(idx, ridx)
        assert torch.equal(val.view(torch.int32), rval.view(torch.int32))
    assert binding.tk_topk_noalloc_status() == 0


def _cases():
    wl = W.workload(4, d=1_170_000, N=6)
    g = torch.Generator(device=DEV).manual_seed(7)
    # long rows: sampled bound + one streaming pass; planted ties and zeros
    long_rows = W.make_grads(wl, 0, DEV), wl.K_up
    # few short rows: selected straight from the rows by one cluster per row
    short = torch.randn((3, 50_001), generator=g, device=DEV)
    short[1, ::7] = 0.5
    # rows just below the sampled path's minimum length and too long for the direct selection: the
    # exact multi-pass path (row reset, full-row histograms in the array's histogram region)
    mid = torch.randn((3, 120_001), generator=g, device=DEV)
    mid[2, 5::3] = -0.25
    # a long row on the sampled path whose candidates overflow the list kept in the array
    # (4K + 8192 entries): 20,000 copies of one large magnitude straddle the K-th value, the row
    # fails verification and is redone by the multi-pass path, ties resolved by index
    crowded = torch.randn((1, 1_000_003), generator=g, device=DEV) * 1e-3
    crowded[0, 1000:400_000:20][:20_000] = 3.0
    crowded[0, 7::50_000] = -5.0
    return [long_rows, (short, 1_000), (mid, 1_000), (crowded, 1_000), (W.make_grads(wl, 1, DEV), wl.K_up)]


def test_calls_in_a_row_match_the_oracle_and_tk_topk():
    # each call reuses the array the previous one filled, with another shape and another path
    for x, K in _cases():
        _check(x, K)


def test_no_device_memory_is_allocated():
    cases = _cases()
    outs = [(torch.empty((x.shape[0], K), dtype=torch.int32, device=DEV),
             torch.empty((x.shape[0], K), dtype=torch.float32, device=DEV)) for x, K in cases]
    binding.tk_topk_noalloc(cases[0][0], cases[0][1], *outs[0])      # first call on the device: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for (x, K), (idx, val) in zip(cases, outs):                      # every path, outputs already there
        binding.tk_topk_noalloc(x, K, idx, val)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0, "the device's free memory moved across a call"
    assert binding.tk_topk_noalloc_status() == 0
    ref_idx, _ = oracle.ref_topk_rows(cases[3][0].cpu().numpy(), cases[3][1])
    assert np.array_equal(outs[3][0].cpu().numpy(), ref_idx)


def test_oversized_problem_is_refused():
    x = torch.zeros((2, 1_000_000), device=DEV)
    K = 200_000
    idx = torch.empty((2, K), dtype=torch.int32, device=DEV)
    val = torch.empty((2, K), dtype=torch.float32, device=DEV)
    with pytest.raises(binding.TkError) as e:
        binding.tk_topk_noalloc(x, K, idx, val)
    assert e.value.code == -6 and "scratch" in str(e.value)
