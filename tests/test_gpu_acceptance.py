"""Acceptance run: every configured step, mode and K_down of the five benchmark workloads at
full size, tk_step against the CPU oracle, with a record of what was compared.

The oracle needs 4-21 s per full-size step, so the whole run takes about half an hour; it is
therefore opt-in:

    TK_ACCEPTANCE=1 [TK_ACCEPTANCE_OUT=file.json] [TK_ACCEPTANCE_CONFIGS=2,3] \
        python -m pytest tests/test_gpu_acceptance.py -m gpu -x -q -s

The same with the error memories of Algorithm 1 / 2 kept (TK_MODE_EF; a few steps per workload, the
memories of all N workers and of the server compared after each):

    TK_ACCEPTANCE_EF=1 [TK_ACCEPTANCE_EF_OUT=file.json] [TK_ACCEPTANCE_EF_CONFIGS=2,5] [TK_ACCEPTANCE_EF_STEPS=3] \
        python -m pytest tests/test_gpu_acceptance.py -m gpu -x -q -s

Without TK_ACCEPTANCE the ordinary parity suite (test_gpu_step.py) covers a slice of every
workload at full size and all legs at a tenth of the size.  Each step is launched the way the
benchmark launches it (context on its own stream, CUDA-graph replay on, plain tk_step).
"""
import json
import os
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2209_15203_b200 import binding, workloads as W
from util import REL_TOL, bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

RUN = os.environ.get("TK_ACCEPTANCE") == "1"
CONFIGS = [int(c) for c in os.environ.get("TK_ACCEPTANCE_CONFIGS", "1,2,3,4,5").split(",")]
RECORD = []


def _compare(got, ref, what, stats):
    """Values within the tolerance (asserted); counts how many are bit-equal."""
    got = np.ascontiguousarray(got, dtype=np.float32)
    ref = np.ascontiguousarray(ref, dtype=np.float32)
    assert got.shape == ref.shape, what
    same = bits(got) == bits(ref)
    n_diff = int((~same).sum())
    if n_diff:
        g64, r64 = got.astype(np.float64), ref.astype(np.float64)
        bad = np.abs(g64 - r64) > REL_TOL * np.abs(r64)
        assert not bad.any(), "%s: %d values beyond %g relative" % (what, int(bad.sum()), REL_TOL)
        # what remains may only be the sign of a zero
        n_diff = int(np.count_nonzero(got[~same] != ref[~same]))
    stats["values_compared"] += got.size
    stats["values_not_bit_equal"] += n_diff


@pytest.mark.skipif(not RUN, reason="opt-in: set TK_ACCEPTANCE=1 (about half an hour of oracle time)")
@pytest.mark.parametrize("cid", CONFIGS)
def test_every_step_of_the_configuration(cid):
    wl = W.workload(cid)
    p = W.make_p(wl)
    scale = W.scale_vector(wl, DEV)
    stream = torch.cuda.Stream()
    G = torch.empty((wl.N, wl.d), device=DEV, dtype=torch.float32)
    for mode in wl.modes:
        for K_down in wl.K_down:
            with torch.cuda.stream(stream):
                ctx = binding.Context(wl.d, wl.N, wl.K_up, K_down, p, stream=stream)
                ctx.tk_set_graph(True)
            w_dev = W.make_w(wl, DEV)
            w_ref = w_dev.cpu().numpy()
            torch.cuda.synchronize()
            leg = {"config": cid, "N": wl.N, "d": wl.d, "K_up": wl.K_up, "K_down": K_down,
                   "mode": "bidirectional" if mode == 1 else "unidirectional", "steps": 0,
                   "index_mismatches": 0, "values_compared": 0, "values_not_bit_equal": 0,
                   "input_checksums": [], "union_sizes": [], "rows_general": [], "oracle_s": 0.0}
            for s in range(wl.steps):
                W.make_grads(wl, s, DEV, out=G, scale=scale)
                leg["input_checksums"].append("%016x" % W.checksum(G))
                torch.cuda.synchronize()
                with torch.cuda.stream(stream):
                    ctx.tk_step(w_dev, G, wl.alpha, mode)
                t0 = time.perf_counter()
                ref = oracle.ref_step(w_ref, G.cpu().numpy(), wl.K_up, K_down, p.numpy(), wl.alpha, mode)
                leg["oracle_s"] += time.perf_counter() - t0
                with torch.cuda.stream(stream):
                    st = ctx.tk_status()
                    assert st.device_status == 0
                    what = "config%d mode=%d K_down=%d step=%d" % (cid, mode, K_down, s)
                    uidx, uval = ctx.tk_last_uplink()
                    aidx, aval = ctx.tk_last_aggregate()
                    midx, mval = ctx.tk_last_downlink()
                torch.cuda.synchronize()
                U = np.nonzero(ref.touched)[0].astype(np.int32)
                for got, want, name in ((uidx, ref.up_idx, "uplink"), (aidx, U, "union"), (midx, ref.msg_idx, "downlink")):
                    g = got.cpu().numpy()
                    assert g.shape == want.shape, what + " " + name
                    bad = int((g != want).sum())
                    leg["index_mismatches"] += bad
                    assert bad == 0, "%s: %d %s indices differ" % (what, bad, name)
                assert np.array_equal(bits(uval.cpu().numpy()), bits(ref.up_val)), what + " uplink values are not bit copies"
                leg["values_compared"] += ref.up_val.size
                _compare(aval.cpu().numpy(), ref.A[U], what + " aggregate", leg)
                _compare(mval.cpu().numpy(), ref.msg_val, what + " downlink values", leg)
                _compare(w_dev.cpu().numpy(), ref.w, what + " w", leg)
                assert st.union_size == U.size <= wl.N * wl.K_up
                leg["union_sizes"].append(int(U.size))
                leg["rows_general"].append(int(st.rows_general))
                leg["steps"] += 1
                w_ref = ref.w
            ctx.close()
            leg["oracle_s"] = round(leg["oracle_s"], 1)
            RECORD.append(leg)
            print("ACCEPT", json.dumps({k: v for k, v in leg.items() if k != "input_checksums"}), flush=True)
            out = os.environ.get("TK_ACCEPTANCE_OUT")
            if out:
                with open(out, "w") as f:
                    json.dump({"torch": torch.__version__, "gpu": torch.cuda.get_device_name(0),
                               "tolerance": REL_TOL, "legs": RECORD}, f, indent=1)


RUN_EF = os.environ.get("TK_ACCEPTANCE_EF") == "1"
EF_CONFIGS = [int(c) for c in os.environ.get("TK_ACCEPTANCE_EF_CONFIGS", "2,3,4,5").split(",")]
EF_STEPS = int(os.environ.get("TK_ACCEPTANCE_EF_STEPS", "3"))
RECORD_EF = []


@pytest.mark.skipif(not RUN_EF, reason="opt-in: set TK_ACCEPTANCE_EF=1 (several minutes of oracle time)")
@pytest.mark.parametrize("cid", EF_CONFIGS)
def test_steps_with_error_memories(cid):
    """Algorithm 1 / 2 as printed (memories epsilon and delta carried from step to step) at full size:
    both messages, w, every worker's epsilon and delta against the oracle after every step."""
    wl = W.workload(cid)
    p = W.make_p(wl)
    scale = W.scale_vector(wl, DEV)
    stream = torch.cuda.Stream()
    G = torch.empty((wl.N, wl.d), device=DEV, dtype=torch.float32)
    K_down = wl.K_down[0]
    for mode in wl.modes:
        with torch.cuda.stream(stream):
            ctx = binding.Context(wl.d, wl.N, wl.K_up, K_down, p, stream=stream)
            ctx.tk_set_graph(True)
            ctx.tk_ef_attach()
            eps_dev, delta_dev = ctx.tk_ef_state()
        w_dev = W.make_w(wl, DEV)
        w = w_dev.cpu().numpy()
        eps = np.zeros((wl.N, wl.d), np.float32)
        delta = np.zeros(wl.d, np.float32)
        torch.cuda.synchronize()
        leg = {"config": cid, "N": wl.N, "d": wl.d, "K_up": wl.K_up, "K_down": K_down,
               "mode": "bidirectional" if mode == 1 else "unidirectional", "steps": 0,
               "index_mismatches": 0, "values_compared": 0, "values_not_bit_equal": 0,
               "input_checksums": [], "rows_general": [], "oracle_s": 0.0}
        for s in range(EF_STEPS):
            W.make_grads(wl, s, DEV, out=G, scale=scale)
            leg["input_checksums"].append("%016x" % W.checksum(G))
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                ctx.tk_step(w_dev, G, wl.alpha, mode | binding.TK_MODE_EF)
            t0 = time.perf_counter()
            ref = oracle.ref_step_ef(w, eps, delta, G.cpu().numpy(), wl.K_up, K_down, p.numpy(), wl.alpha, mode)
            leg["oracle_s"] += time.perf_counter() - t0
            what = "config%d with memories mode=%d step=%d" % (cid, mode, s)
            with torch.cuda.stream(stream):
                st = ctx.tk_status()
                assert st.device_status == 0
                uidx, uval = ctx.tk_last_uplink()
                midx, mval = ctx.tk_last_downlink()
            torch.cuda.synchronize()
            for got, want, name in ((uidx, ref.up_idx, "uplink"), (midx, ref.msg_idx, "downlink")):
                g = got.cpu().numpy()
                assert g.shape == want.shape, what + " " + name
                bad = int((g != want).sum())
                leg["index_mismatches"] += bad
                assert bad == 0, "%s: %d %s indices differ" % (what, bad, name)
            _compare(uval.cpu().numpy(), ref.up_val, what + " uplink values", leg)
            _compare(mval.cpu().numpy(), ref.msg_val, what + " downlink values", leg)
            _compare(w_dev.cpu().numpy(), ref.w, what + " w", leg)
            _compare(eps_dev.cpu().numpy(), ref.eps, what + " epsilon", leg)
            if mode == 1:
                _compare(delta_dev.cpu().numpy(), ref.delta, what + " delta", leg)
                delta = ref.delta
            w, eps = ref.w, ref.eps
            leg["rows_general"].append(int(st.rows_general))
            leg["steps"] += 1
        ctx.close()
        del eps_dev, delta_dev
        leg["oracle_s"] = round(leg["oracle_s"], 1)
        RECORD_EF.append(leg)
        print("ACCEPT-EF", json.dumps({k: v for k, v in leg.items() if k != "input_checksums"}), flush=True)
        out = os.environ.get("TK_ACCEPTANCE_EF_OUT")
        if out:
            with open(out, "w") as f:
                json.dump({"torch": torch.__version__, "gpu": torch.cuda.get_device_name(0),
                           "tolerance": REL_TOL, "steps_per_leg": EF_STEPS, "legs": RECORD_EF}, f, indent=1)
