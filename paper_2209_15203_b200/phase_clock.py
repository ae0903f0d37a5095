"""Where the time of one step goes: device timestamps at the start and end of every kernel
of tk_step and at the milestones of the two selections, from a build of the library with the
phase clock compiled in (tk_debug_phase_clock).

    python -m paper_2209_15203_b200.phase_clock [--no-bound-reuse] [--no-graph] [configs ...]

For each workload (default 5 2 3) it steps a few times to warm up, then prints, for six single
steps, the earliest and the latest time any CTA passed each stamp (microseconds since the
step's first stamp), and for four pairs of back-to-back steps where the first one ended and
the second one began.  Steps run the way bench.py runs them (CUDA graph replay on a stream of
their own).  The clock build is slower by a microsecond or two per step (two atomics per CTA
and stamp); the ordinary library records nothing.
"""
from __future__ import annotations

import argparse
import sys


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("configs", nargs="*", type=int, default=[5, 2, 3])
    ap.add_argument("--no-bound-reuse", action="store_true")
    ap.add_argument("--no-graph", action="store_true")
    args = ap.parse_args()

    from . import build as _build
    _build.LIB = _build.build_phase_clock()   # the binding opens whatever build.LIB names
    import torch
    from . import binding, workloads as W

    dev = "cuda:0"
    for cid in args.configs:
        wl = W.workload(cid)
        stream = torch.cuda.Stream()
        torch.cuda.set_stream(stream)
        ctx = binding.Context(wl.d, wl.N, wl.K_up, wl.K_down[0], W.make_p(wl), stream=stream)
        if args.no_bound_reuse:
            ctx.tk_set_bound_reuse(False)
        if not args.no_graph:
            ctx.tk_set_graph(True)
        G = [W.make_grads(wl, s, dev) for s in range(2)]
        w = W.make_w(wl, dev)
        for s in range(4):
            ctx.tk_step(w, G[s % 2], wl.alpha, binding.TK_MODE_BIDIR)
        torch.cuda.synchronize()
        rows = []
        for r in range(6):
            ctx.tk_debug_phase_clock()                      # arm
            ctx.tk_step(w, G[r % 2], wl.alpha, binding.TK_MODE_BIDIR)
            rows.append(ctx.tk_debug_phase_clock())
        names = binding.Context.PHASE_STAMPS
        print("config %d: N=%d d=%d K_up=%d K_down=%d, bound reuse %s, %s" %
              (cid, wl.N, wl.d, wl.K_up, wl.K_down[0], "off" if args.no_bound_reuse else "on",
               "plain launches" if args.no_graph else "graph replay"))
        for i, n in enumerate(names):
            print("  %-28s first %s   last %s" % (n, " ".join("%7.1f" % r[0][i] for r in rows),
                                                   " ".join("%7.1f" % r[1][i] for r in rows)))
        pairs = []
        last = len(names) - 1
        for r in range(4):
            ctx.tk_debug_phase_clock()
            ctx.tk_step(w, G[0], wl.alpha, binding.TK_MODE_BIDIR)
            ctx.tk_step(w, G[1], wl.alpha, binding.TK_MODE_BIDIR)
            f, l = ctx.tk_debug_phase_clock()
            pairs.append("first step's earliest end %.1f, second step starts %.1f, ends %.1f" % (f[last], l[0], l[last]))
        print("  two steps back to back: " + " | ".join(pairs))
        ctx.close()
        del G, w
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
    sys.exit(0)
