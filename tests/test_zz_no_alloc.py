"""tk_topk_noalloc: the allocation-free variant of tk_topk.

Some users of the library run where cudaMalloc is off limits (a plugin inside
another program's memory budget, a loop that must never hit the allocator's
locks or cudaFree's device-wide synchronisation).  For them the library keeps
its scratch in a fixed array inside its own image.  This file checks, through
the C ABI, that the variant returns exactly what tk_topk returns, twice in a
row (the second call finds the first call's leftovers in the shared array),
and that a problem larger than the array is refused instead of overrunning it.
It is named so that pytest collects it after every other test file.
"""
import pytest
import torch

from paper_2209_15203_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(x, K):
    rows = x.shape[0]
    idx = torch.full((rows, K), -1, dtype=torch.int32, device=DEV)
    val = torch.full((rows, K), float("nan"), dtype=torch.float32, device=DEV)
    binding.tk_topk_noalloc(x, K, idx, val)
    ridx, rval = binding.tk_topk(x, K)
    torch.cuda.synchronize()
    assert torch.equal(idx, ridx)
    assert torch.equal(val.view(torch.int32), rval.view(torch.int32))


def test_two_calls_in_a_row_match_tk_topk():
    # first call: long rows (sampled threshold + one streaming pass), ties included
    wl = W.workload(4, d=1_170_000, N=6)
    _both(W.make_grads(wl, 0, DEV), wl.K_up)
    # second call, other shape and other path (short rows go through the multi-pass path);
    # it reuses the array the first call filled
    g = torch.Generator(device=DEV).manual_seed(7)
    x = torch.randn((3, 50_001), generator=g, device=DEV)
    x[1, ::7] = 0.5
    _both(x, 1_000)
    # and the first problem again, now on top of the second call's leftovers
    _both(W.make_grads(wl, 1, DEV), wl.K_up)


def test_oversized_problem_is_refused():
    x = torch.zeros((2, 1_000_000), device=DEV)
    K = 200_000
    idx = torch.empty((2, K), dtype=torch.int32, device=DEV)
    val = torch.empty((2, K), dtype=torch.float32, device=DEV)
    with pytest.raises(binding.TkError) as e:
        binding.tk_topk_noalloc(x, K, idx, val)
    assert e.value.code == -6 and "scratch" in str(e.value)
