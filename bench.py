#!/usr/bin/env python
"""Benchmark of one bidirectional top_K step (uplink select, ordered aggregation,
downlink select, update) through the C ABI, on the largest workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

Prints one JSON line.  `value` is gradient elements per second (N*d per step,
summed over GPUs) with the gradients already in HBM; `e2e` is the same metric
through tk_step_host with pinned host buffers (copies inside the timed region);
`roofline` is the streaming selection kernel against the measured HBM copy
bandwidth; `cpu_baseline` is the CPU oracle on the host cores.  With more than
one GPU every rank runs an independent replica of the workload (the path has
no exchange between GPUs).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2209_15203_b200 import workloads as W  # noqa: E402

METRIC = "gradient elements/sec per bidirectional top_K step"
UNIT = "elements/s"
NOMINAL_HBM_BPS = 8e12
FALLBACK_HBM_GBS = 6650.0
PROFILE_SUMMARY = os.path.join(ROOT, "profiles", "filter_kernel_config5_rows2.md")
KERNEL_SOURCES = ["paper_2209_15203_b200/csrc/common.cuh", "paper_2209_15203_b200/csrc/select.cuh"]


def kernel_source_digest():
    """sha256 over the sources of the streaming kernel (what decides whether captured counters still apply)."""
    import hashlib
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def captured_traffic(path=PROFILE_SUMMARY):
    """The `key: value` lines of the ncu summary of the streaming kernel: DRAM bytes read + written per
    launch, the rows that launch covered and the digest of the kernel sources it was taken on."""
    import re
    out = {}
    try:
        with open(path) as f:
            for line in f:
                m = re.match(r"^\s*(dram_bytes_read_per_launch|dram_bytes_write_per_launch|rows_per_launch|"
                             r"kernel_source_sha256)\s*:\s*(\S+)\s*$", line)
                if m:
                    out[m.group(1)] = m.group(2)
    except OSError:
        return None
    if len(out) != 4:
        return None
    return {"read": float(out["dram_bytes_read_per_launch"]), "write": float(out["dram_bytes_write_per_launch"]),
            "rows": int(out["rows_per_launch"]), "sha256": out["kernel_source_sha256"]}


def traffic_for(wl, overridden_d, ef):
    """DRAM traffic of one launch of the streaming kernel on the benchmark workload, scaled by rows from
    the captured case (traffic is proportional to the rows); None for any other workload, and None once
    the kernel sources differ from the ones the counters were taken on."""
    if wl.cid != 5 or overridden_d or ef:
        return None
    cap = captured_traffic()
    if cap is None or cap["sha256"] != kernel_source_digest():
        return None
    return (cap["read"] + cap["write"]) / cap["rows"] * wl.N


def measured_hbm_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Polls NVML for SM clock and throttle reasons while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
               0x10: "sync_boost", 0x100: "display_clock_setting"}

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self.stop_flag = False
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag:
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                break
            time.sleep(0.002)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def sum_checksum(t):
    """workloads.checksum row by row (bounded temporary memory), wrapped to 64 bits."""
    total = 0
    for q in range(t.shape[0]):
        total = (total + W.checksum(t[q])) & 0xFFFFFFFFFFFFFFFF
    return total


def b_min_bytes(wl, k_apply):
    return 4 * wl.N * wl.d + 24 * wl.N * wl.K_up + 16 * k_apply


REFERENCE_BUDGET_S = 300.0   # wall-clock the reference arm may spend inside the oracle


def run_reference(args, rank, world):
    """The CPU oracle, as it stands, on the host cores (rank 0 only): full steps of the stated
    configuration (same N, d, K as the GPU arm).  A full step of the largest workload costs the oracle
    about 20 s, so what is bounded is the NUMBER of steps run and timed, never the problem: one warm-up
    step, then as many of the requested steps as fit REFERENCE_BUDGET_S (at least one)."""
    if rank != 0:
        return
    import oracle
    wl = W.workload(args.config)
    threads = min(wl.N, oracle.ref.default_threads())
    p = W.make_p(wl).numpy()
    w = W.make_w(wl, "cpu").numpy()
    K_down = wl.K_down[0]
    # one gradient tensor for all steps (generating 4 GB on the host costs as much as a step; the
    # oracle's time does not depend on the values, and w still changes from step to step)
    G = W.make_grads(wl, 0, "cpu", agree=args.agree).numpy()
    times = []
    spent = 0.0
    n_warm = 1 if args.warmup > 0 else 0
    s = 0
    while True:
        t0 = time.perf_counter()
        res = oracle.ref_step(w, G, wl.K_up, K_down, p, wl.alpha, 1, nthreads=threads, want_dense=False)
        dt = time.perf_counter() - t0
        w = res.w
        spent += dt
        if s >= n_warm:
            times.append(dt)
        s += 1
        if len(times) >= args.steps or (times and spent + dt > REFERENCE_BUDGET_S):
            break
    t = sum(times)
    value = wl.N * wl.d * len(times) / t
    ts = sorted(times)
    sample = ("%d full steps of config %d timed (of %d asked; N=%d rows of d=%d, K=%d) after %d warm-up, "
              "%.0f s in the oracle" % (len(times), wl.cid, args.steps, wl.N, wl.d, wl.K_up, n_warm, spent))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "steps_timed": len(times), "warmup_run": n_warm,
        "ms_per_step": 1e3 * t / len(times), "ms_per_step_median": 1e3 * ts[len(ts) // 2], "ms_per_step_min": 1e3 * ts[0],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": W.describe(wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=0, help="override the number of workers N (smaller case for profiling)")
    ap.add_argument("--d", type=int, default=0, help="override the vector length d (smaller case for profiling)")
    ap.add_argument("--ef", action="store_true", help="keep the error memories (Algorithm 2 as printed): "
                    "12 bytes per gradient value instead of 4")
    ap.add_argument("--sharded", action="store_true", help="with --gpus N > 1: shard the N workers over the ranks "
                    "(one all-gather of the messages per step) instead of running independent replicas")
    ap.add_argument("--force-general", action="store_true", help="time the exact multi-pass path instead of the "
                    "sampled single-pass one")
    ap.add_argument("--no-graph", action="store_true", help="issue every step as plain stream launches instead of "
                    "replaying captured CUDA graphs (tk_set_graph)")
    ap.add_argument("--profile-every", type=int, default=0, help="timestamp the streaming kernel of every n-th timed "
                    "step (such a step is issued as plain launches, which costs it some tens of microseconds); "
                    "default: about eight samples over the run, at most every 10th step")
    ap.add_argument("--agree", type=float, default=None, metavar="C",
                    help="workers see noisy copies of one shared vector, row_q = base * (1 + C z_q), instead of "
                         "independent rows: their selections then mostly coincide (union near K)")
    ap.add_argument("--no-bound-reuse", action="store_true", help="sample every row's bound in every step instead of "
                    "keeping the bounds that served the step before (tk_set_bound_reuse)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.profile_every <= 0:
        args.profile_every = max(1, min(10, args.steps // 8))

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch.distributed as dist
    from paper_2209_15203_b200 import binding, replicas, sharding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    warmup = max(args.warmup, 3)
    wl = W.workload(args.config, d=args.d or None, N=args.rows or None)
    K_down = wl.K_down[0]
    p = W.make_p(wl)
    # graphs need a capturable (non-default) stream; everything below runs on it
    args.graph = not args.no_graph
    run_stream = torch.cuda.Stream(dev) if args.graph else torch.cuda.current_stream(dev)
    torch.cuda.set_stream(run_stream)
    ctx = binding.Context(wl.d, wl.N, wl.K_up, K_down, p, stream=run_stream)
    scale = W.scale_vector(wl, dev)
    nbuf = max(1, min(args.steps, 8))
    bufs = [W.make_grads(wl, s, dev, scale=scale, agree=args.agree) for s in range(nbuf)]
    del scale
    w = W.make_w(wl, dev)
    mode = binding.TK_MODE_BIDIR | (binding.TK_MODE_EF if args.ef else 0)
    if args.ef:
        ctx.tk_ef_attach()
    if args.force_general:
        ctx.tk_set_force_general(True)
    if args.no_bound_reuse:
        ctx.tk_set_bound_reuse(False)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    if args.sharded:
        # strong scaling: this rank keeps (and steps) its own workers' rows only
        row0, nrows = sharding.row_range(wl.N, rank, world)
        bufs = [b[row0:row0 + nrows].clone() for b in bufs]
        torch.cuda.empty_cache()

        def step(g):
            sharding.sharded_step(ctx, w, g, wl.alpha, mode)
    else:
        def step(g):
            ctx.tk_step(w, g, wl.alpha, mode)

    if args.graph:
        ctx.tk_set_graph(True)
        for s in range(nbuf):                 # capture every buffer's step before anything is timed
            step(bufs[s % nbuf])
    for s in range(warmup):
        step(bufs[s % nbuf])
    st = ctx.tk_status()
    ctx.tk_set_profile(max(1, args.profile_every))

    sampler = ClockSampler(physical_gpu_index(local))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.tk_launch_count()
    barrier()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]   # one behind every step
    sampler.start()
    ev0.record()
    for s in range(args.steps):
        step(bufs[s % nbuf])
        marks[s].record()
    ev1.record()
    barrier()
    sampler.stop_flag = True
    ms = ev0.elapsed_time(ev1)
    per_step = sorted(a.elapsed_time(b) for a, b in zip([ev0] + marks[:-1], marks))
    launches = ctx.tk_launch_count() - launches0
    st = ctx.tk_status()
    sampler.join(timeout=2.0)
    ctx.tk_set_profile(0)

    elems = wl.N * wl.d
    value, ms_max = replicas.whole_job_throughput(ms, elems, args.steps, dev)
    if args.sharded:
        value /= world          # one job of N*d values per step, not one per rank
    ms_per_step = ms_max / args.steps

    # roofline of the dominant kernel (the streaming selection pass)
    peak, peak_kind = measured_hbm_gbs()
    roof = None
    if st.select_samples > 0 and st.select_ms_sum > 0:
        k_ms = st.select_ms_sum / st.select_samples
        bytes_per_elem = 12.0 if args.ef else 4.0   # with memories: read g, read and write epsilon
        elems_rank = (elems // world) if args.sharded else elems     # what one launch on this rank reads
        achieved = bytes_per_elem * elems_rank / (k_ms * 1e-3) / 1e9
        step_bytes = b_min_bytes(wl, K_down) + (8 * elems + 4 * wl.d if args.ef else 0)
        step_gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
        roof = {"bound": "hbm", "kernel": "filter_kernel" if st.rows_general == 0 else "general_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": peak_kind,
                "peak_note": "a read+write copy; a read-only stream can exceed it slightly",
                "traffic": traffic_for(wl, args.d, args.ef),
                "algorithmic_bytes": int(bytes_per_elem) * elems_rank, "kernel_ms": k_ms, "launches_timed": st.select_samples,
                # the whole step (all kernels, minimum bytes of the method) against the same peak and the nominal one
                "whole_step": {"algorithmic_bytes": step_bytes, "achieved": step_gbs, "frac": step_gbs / peak,
                               "frac_of_nominal_8TBps": step_gbs * 1e9 / NOMINAL_HBM_BPS}}

    # end to end through tk_step_host: pinned host buffers, copies inside the timed region
    e2e = None
    if not args.no_e2e and not args.sharded:
        g_host = torch.empty((wl.N, wl.d), dtype=torch.float32, pin_memory=True)
        g_host.copy_(bufs[0])
        w_host = torch.empty(wl.d, dtype=torch.float32, pin_memory=True)
        w_host.copy_(w)
        n_e2e = max(1, min(args.steps, 5))
        ctx.tk_step_host(w_host, g_host, wl.alpha, mode)          # warm-up: allocates the staging buffers
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            ctx.tk_step_host(w_host, g_host, wl.alpha, mode)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        e2e_value, e2e_ms = replicas.whole_job_throughput(dt * 1e3, elems, n_e2e, dev)
        e2e = {"value": e2e_value, "unit": UNIT,
               "h2d_bytes_per_step": 4 * (elems + wl.d), "d2h_bytes_per_step": 4 * wl.d, "steps": n_e2e,
               "ms_per_step": e2e_ms / n_e2e}
        del g_host, w_host

    # the CPU oracle on this host's cores: one full step of the same workload (rank 0, single GPU only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.sharded:
        import oracle
        threads = min(wl.N, oracle.ref.default_threads())
        G = bufs[0].cpu().numpy()
        w_cpu = w.cpu().numpy()
        t0 = time.perf_counter()
        if args.ef:
            import numpy as np
            oracle.ref_step_ef(w_cpu, np.zeros_like(G), np.zeros_like(w_cpu), G, wl.K_up, K_down, p.numpy(), wl.alpha, 1,
                               nthreads=threads)
        else:
            oracle.ref_step(w_cpu, G, wl.K_up, K_down, p.numpy(), wl.alpha, 1, nthreads=threads, want_dense=False)
        dt = time.perf_counter() - t0
        # ... and Top_K of one row on one thread (the unit of work the rows are spread over)
        t0 = time.perf_counter()
        oracle.ref_topk(G[0], wl.K_up)
        dt_row = time.perf_counter() - t0
        cpu = {"value": elems / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": "1 full step of config %d (N=%d rows of d=%d), %.1f s" % (wl.cid, wl.N, wl.d, dt),
               "one_row_topk_single_thread_s": dt_row, "one_row_topk_single_thread_elements_per_s": wl.d / dt_row}

    if rank == 0:
        cfg = W.describe(wl)
        cfg.update({"mode": "bidirectional with error memories" if args.ef else "bidirectional", "cold_inputs": "each step reads a %d MB gradient tensor (>> L2), "
                    "%d distinct tensors cycled" % (4 * elems // 10 ** 6, nbuf),
                    "launch": ("CUDA graph replay; every %d-th step plain launches with timestamps around the "
                               "streaming kernel" % max(1, args.profile_every)) if args.graph else "stream launches",
                    "parallelism": ("workers sharded over %d ranks, one all-gather per step" if args.sharded
                                    else "replicas x%d") % world,
                    "bounds": "sampled in every step" if args.no_bound_reuse else
                              "warm-started from the step before (last threshold minus a margin of 1.5-3 % or four times its "
                              "recent movement; verified exactly every step), sampled otherwise; --no-bound-reuse samples "
                              "every step"})
        if args.agree is not None:
            cfg["rows"] = "shared vector x (1 + %g z_q)" % args.agree
        cfg["input_checksum_step0"] = "%016x" % sum_checksum(bufs[0])
        # Section 4.2's transfer model for this workload.  beta = one 32-bit word at the 770 GB/s a peer copy
        # reaches on this pool's NVLink (from the pool's measurements, not this run); latencies are not
        # measurable on one GPU and are left at 0, so the times are the bandwidth terms alone.
        beta = 4.0 / 770e9
        cm = binding.tk_comm_model(wl.N, wl.K_up, K_down, int(st.union_size), 0.0, beta, 0.0, beta)
        comm = {"uplink_words_per_worker": cm.uplink_words, "downlink_words_uni_bound": cm.downlink_words_uni_max,
                "downlink_words_uni_last_step": cm.downlink_words_uni, "downlink_words_bi": cm.downlink_words_bi,
                "compression_factor": cm.compression_factor,
                "alpha_s": 0.0, "beta_s_per_word": beta, "time_uni_s": cm.time_uni, "time_uni_union_s": cm.time_uni_union,
                "time_bi_s": cm.time_bi, "note": "beta assumed from the pool's peer-copy rate, latencies not measured"}
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step,
            "ms_per_step_median": per_step[len(per_step) // 2], "ms_per_step_min": per_step[0],
            "higher_is_better": True,
            "scaling": "strong" if args.sharded else "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg,
            "hbm_frac_of_8TBps": (b_min_bytes(wl, K_down) + (8 * elems + 4 * wl.d if args.ef else 0))
            / (ms_per_step * 1e-3) / NOMINAL_HBM_BPS,
            "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": sampler.summary(), "comm_model": comm,
            "stats": {"rows_general": st.rows_general, "union_size": st.union_size,
                      "cand_min": st.cand_min, "cand_max": st.cand_max, "device_status": st.device_status},
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
