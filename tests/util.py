"""Helpers shared by the GPU parity tests."""
import warnings

import numpy as np
import torch

REL_TOL = 1e-6   # relative tolerance on fp32 values (bit-equality is expected and warned about if lost)


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def assert_values_close(got, ref, what):
    got = np.asarray(got, dtype=np.float32)
    ref = np.asarray(ref, dtype=np.float32)
    assert got.shape == ref.shape, what
    if np.array_equal(bits(got), bits(ref)):
        return
    # -0 == +0 numerically; anything else must be within the relative tolerance
    g64, r64 = got.astype(np.float64), ref.astype(np.float64)
    bad = np.abs(g64 - r64) > REL_TOL * np.abs(r64)
    assert not bad.any(), "%s: %d values differ beyond %g relative" % (what, int(bad.sum()), REL_TOL)
    n = int((bits(got) != bits(ref)).sum())
    if np.any((got != ref)):
        warnings.warn("%s: %d values are within tolerance but not bit-equal" % (what, n))


def assert_message_equal(idx, val, ref_idx, ref_val, what):
    idx = idx.cpu().numpy() if isinstance(idx, torch.Tensor) else np.asarray(idx)
    val = val.cpu().numpy() if isinstance(val, torch.Tensor) else np.asarray(val)
    assert idx.dtype == np.int32
    assert idx.shape == ref_idx.shape, "%s: %s vs %s entries" % (what, idx.shape, ref_idx.shape)
    assert np.array_equal(idx, ref_idx), "%s: indices differ at %d positions" % (what, int((idx != ref_idx).sum()))
    assert np.array_equal(bits(val), bits(ref_val)), "%s: values are not bit-copies" % what
