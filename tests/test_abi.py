"""The C-ABI library loads and exports every entry point include/topk.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2209_15203_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "topk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tk_[a-z_]+)\s*\(", text)))


def test_header_and_binding_agree():
    assert declared_symbols() == sorted(binding.EXPORTS)


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    assert os.path.exists(binding.library_path())
    for name in declared_symbols():
        assert getattr(lib, name) is not None


def test_host_side_argument_checks_need_no_gpu():
    lib = binding.load()
    assert lib.tk_workspace_bytes(0, 1, 1, 1) == 0
    assert lib.tk_workspace_bytes(100, 1, 101, 1) == 0
    assert lib.tk_workspace_bytes(100, 0, 1, 1) == 0
    assert lib.tk_workspace_bytes(2 ** 31, 1, 1, 1) == 0
    assert lib.tk_workspace_bytes(124_000_000, 8, 12_400, 12_400) > 124_000_000 * 4
    assert lib.tk_init(None, 10, 1, 1, 1, None, None, 0, None) == -1
    h = ctypes.c_void_p()
    assert lib.tk_init(ctypes.byref(h), 10, 1, 1, 1, None, None, 0, None) == -1
    assert lib.tk_step(None, None, None, 0.1, 1) == -1
    assert lib.tk_topk(None, None, 1, 10, 1, None, None) == -1
    assert binding.strerror(0) == "ok" and "invalid" in binding.strerror(-1)
    assert lib.tk_launch_count(None) == 0


def test_transfer_model_matches_the_hand_worked_example():
    # Section 4.2's two formulas on the d = 8, N = 3 example (values by hand in the golden file)
    g = {}
    with open(os.path.join(ROOT, "tests", "golden", "alg2_first_iteration.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *v = line.split()
                g[k] = [float(t) for t in v]
    N, K_up, K_down = int(g["N"][0]), int(g["K_up"][0]), int(g["K_down"][0])
    union = len(g["uni_msg_idx"])
    c = binding.tk_comm_model(N, K_up, K_down, union, *g["comm_costs"])
    assert [c.uplink_words, c.downlink_words_uni_max, c.downlink_words_uni, c.downlink_words_bi] == g["comm_words"]
    assert [c.time_uni, c.time_uni_union, c.time_bi] == g["comm_times"]
    assert c.compression_factor == K_down / (K_up * N)
    # no union known: the bound only
    c = binding.tk_comm_model(N, K_up, K_down, -1, *g["comm_costs"])
    assert c.downlink_words_uni == -1 and c.time_uni_union == -1.0 and c.time_uni == g["comm_times"][0]
    # the bidirectional iteration is cheaper exactly when K_down < N K_up (and beta2 > 0)
    assert binding.tk_comm_model(4, 10, 40, -1, 0, 1, 0, 1).time_bi == binding.tk_comm_model(4, 10, 40, -1, 0, 1, 0, 1).time_uni
    assert binding.tk_comm_model(4, 10, 39, -1, 0, 1, 0, 1).time_bi < binding.tk_comm_model(4, 10, 39, -1, 0, 1, 0, 1).time_uni
    import pytest
    for bad in ((0, 1, 1, -1, 0, 0, 0, 0), (2, 3, 1, 7, 0, 0, 0, 0), (2, 3, 1, -1, -1.0, 0, 0, 0),
                (2, 3, 1, -1, 0, float("nan"), 0, 0)):
        with pytest.raises(binding.TkError):
            binding.tk_comm_model(*bad)
