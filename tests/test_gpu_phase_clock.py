"""The phase clock (tk_debug_phase_clock): the ordinary library records nothing and says so; the tool
around the instrumented build prints, for every kernel of a step, stamps in the order the kernels run."""
import os
import re
import subprocess
import sys

import pytest
import torch

from paper_2209_15203_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_ordinary_build_has_no_clock():
    wl = W.workload(1)
    ctx = binding.Context(wl.d, wl.N, wl.K_up, wl.K_down[0], W.make_p(wl))
    with pytest.raises(binding.TkError):
        ctx.tk_debug_phase_clock()
    ctx.close()


def test_tool_prints_the_kernels_of_a_step_in_order():
    # config 2 (16 rows of 11.7M values): the sampled single-pass path, six kernels per step
    env = dict(os.environ)
    env.pop("TOPK_LIBRARY", None)
    run = subprocess.run([sys.executable, "-m", "paper_2209_15203_b200.phase_clock", "2"], cwd=ROOT, env=env,
                         capture_output=True, text=True, timeout=900)
    assert run.returncode == 0, run.stderr[-2000:]
    first, last = {}, {}
    for line in run.stdout.splitlines():
        m = re.match(r"\s+(.*?)\s+first((?:\s+-?[\d.]+)+)\s+last((?:\s+-?[\d.]+)+)\s*$", line)
        if m:
            f = sorted(float(t) for t in m.group(2).split())
            l = sorted(float(t) for t in m.group(3).split())
            first[m.group(1)] = f[len(f) // 2]
            last[m.group(1)] = l[len(l) // 2]
    names = binding.Context.PHASE_STAMPS
    assert [n for n in names if n in first] == list(names), run.stdout[-2000:]
    f = [first[n] for n in names]
    l = [last[n] for n in names]
    assert f[0] == 0.0
    assert all(x >= 0.0 for x in f + l), (f, l)           # every stamp was passed
    assert all(a <= b for a, b in zip(f, l))
    assert all(f[i] <= f[i + 1] for i in range(len(f) - 1)), f   # in the order the kernels run
    # a kernel's first CTA starts after the last CTA of the kernel before it has ended (same stream)
    ends = {"sampling ends": "streaming pass starts", "streaming pass ends": "verification starts",
            "verification ends": "uplink select starts", "uplink select ends": "server sum starts",
            "server sum ends": "downlink select starts"}
    for e, s in ends.items():
        assert last[e] <= first[s] + 0.5, (e, last[e], s, first[s])
    # the streaming pass is most of the step, and the step of this workload takes well under a millisecond
    assert l[-1] < 1000.0
    assert last["streaming pass ends"] - first["streaming pass starts"] > 0.5 * l[-1]
