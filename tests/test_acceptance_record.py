"""The committed record of the full-size acceptance run (profiles/acceptance_five_configs.md, written
from the output of tests/test_gpu_acceptance.py) must cover every leg the five benchmark workloads
name — every mode, every K_down, every step — and report no mismatch.  No GPU needed: this reads
the record and the workload definitions only."""
import os
import re

from paper_2209_15203_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_record_covers_every_configured_leg_without_a_mismatch():
    text = open(os.path.join(ROOT, "profiles", "acceptance_five_configs.md")).read()
    rows = {}
    for line in text.splitlines():
        m = re.match(r"^\| (\d+) \| (unidirectional|bidirectional) \| (\d+) \| (\d+) \| (\d+) \| (\d+) \| (\d+) \|", line)
        if m:
            cid, mode, kdown, steps, idx_bad, compared, not_equal = m.groups()
            rows[(int(cid), mode, int(kdown))] = (int(steps), int(idx_bad), int(compared), int(not_equal))
    want = 0
    for cid in (1, 2, 3, 4, 5):
        wl = W.workload(cid)
        for mode in wl.modes:
            for kdown in wl.K_down:
                key = (cid, "bidirectional" if mode == 1 else "unidirectional", kdown)
                assert key in rows, "no record of %r" % (key,)
                steps, idx_bad, compared, not_equal = rows[key]
                assert steps == wl.steps, (key, steps, wl.steps)
                assert idx_bad == 0 and not_equal == 0 and compared > 0, (key, rows[key])
                want += 1
    assert len(rows) == want


def test_record_with_error_memories_covers_the_four_large_workloads_without_a_mismatch():
    """profiles/acceptance_error_memories.md: Algorithm 1 / 2 with the memories kept, configs 2-5 at full
    size, every mode a config names; at least two consecutive steps (state carried), nothing differing."""
    text = open(os.path.join(ROOT, "profiles", "acceptance_error_memories.md")).read()
    rows = {}
    for line in text.splitlines():
        m = re.match(r"^\| (\d+) \| (unidirectional|bidirectional) \| (\d+) \| (\d+) \| (\d+) \| (\d+) \| (\d+) \|", line)
        if m:
            cid, mode, kdown, steps, idx_bad, compared, not_equal = m.groups()
            rows[(int(cid), mode)] = (int(kdown), int(steps), int(idx_bad), int(compared), int(not_equal))
    for cid in (2, 3, 4, 5):
        wl = W.workload(cid)
        for mode in wl.modes:
            key = (cid, "bidirectional" if mode == 1 else "unidirectional")
            assert key in rows, "no record of %r" % (key,)
            kdown, steps, idx_bad, compared, not_equal = rows[key]
            assert kdown == wl.K_down[0] and steps >= 2, (key, rows[key])
            # the memories of all workers are among the values compared
            assert compared >= steps * wl.N * wl.d, (key, rows[key])
            assert idx_bad == 0 and not_equal == 0, (key, rows[key])
