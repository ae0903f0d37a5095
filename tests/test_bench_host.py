"""Host-side pieces of bench.py that need no GPU: the captured DRAM traffic it reports must be the
figures of the committed ncu summary, and the reference arm (the CPU oracle) must print the
contract's JSON line for the stated configuration."""
import json
import os
import re
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2209_15203_b200 import workloads as W  # noqa: E402


def _table_mean_mb(text, counter):
    row = next(l for l in text.splitlines() if l.startswith("| " + counter))
    vals = [float(v) for v in re.findall(r"([0-9.]+) MB", row)]
    assert len(vals) == 2
    return sum(vals) / 2 * 1e6


def test_reported_traffic_is_the_profile_summary_figure(tmp_path):
    text = open(bench.PROFILE_SUMMARY).read()
    cap = bench.captured_traffic()
    assert cap is not None and cap["rows"] == 2
    # the machine-readable lines agree with the counters' table of the same file
    assert abs(cap["read"] - _table_mean_mb(text, "dram__bytes_read.sum")) <= 1e-4 * cap["read"]
    assert abs(cap["write"] - _table_mean_mb(text, "dram__bytes_write.sum")) <= 2e-3 * cap["write"]
    wl = W.workload(5)
    got = bench.traffic_for(wl, 0, False)
    if cap["sha256"] == bench.kernel_source_digest():
        assert got == (cap["read"] + cap["write"]) / 2 * wl.N
        assert 1.0 <= got / (4 * wl.N * wl.d) < 1.01          # one pass over the gradients
    else:
        assert got is None                                     # kernel changed since the capture
    # any other workload, a changed d, or the path with memories has no captured figure
    assert bench.traffic_for(W.workload(2), 0, False) is None
    assert bench.traffic_for(wl, 31_000_000, False) is None
    assert bench.traffic_for(wl, 0, True) is None
    # a summary taken on other sources is not used
    other = tmp_path / "other.md"
    other.write_text(re.sub(r"kernel_source_sha256: \S+", "kernel_source_sha256: " + "0" * 64, text))
    assert bench.captured_traffic(str(other))["sha256"] == "0" * 64
    assert bench.captured_traffic(str(tmp_path / "missing.md")) is None


def test_reference_arm_prints_the_contract_line_for_the_stated_config():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "3", "--warmup", "1"], capture_output=True, text=True, check=True, cwd=ROOT)
    line = json.loads(out.stdout.strip().splitlines()[-1])
    wl = W.workload(1)
    assert line["impl"] == "reference" and line["unit"] == "elements/s" and line["higher_is_better"] is True
    assert line["config"]["d"] == wl.d and line["config"]["N"] == wl.N and line["config"]["K_up"] == wl.K_up
    assert line["steps"] == 3 and line["steps_timed"] == 3 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["ms_per_step_min"] <= line["ms_per_step_median"]
