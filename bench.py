#!/usr/bin/env python
"""Benchmark of the nested Forward-AD activation pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step = one pass of the whole hot path over one batch of the workload: for
every activation kind the workload names, forward (x -> y, f') and backward
(g, f' -> grad_in), each one kernel launched through the C-ABI binding.  The
default workload is the BERT-base feed-forward activation (bf16 [32,128,3072],
GELU erf and tanh forms).  Prints ONE JSON line.

Timing: CUDA events on the launching stream; W >= 3 warm-up steps; buffer sets
are rotated so that the bytes touched between two uses of a buffer exceed 4x the
L2 capacity, and backward consumes the f' that a forward wrote half a rotation
earlier (as in training, where backward comes long after forward), so no tensor
is served from L2.  With N > 1 every rank runs the same workload on its own GPU
(the path has no exchange step: weak scaling, no collective in the data path);
the barrier and the max-over-ranks of the device time use torch.distributed.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fwd+bwd elements/s"
UNIT = "elements/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0          # an earlier copy-bandwidth measurement on this machine's B200s

# DRAM bytes per element (read + write) of the dominant kernel measured by ncu
# (dram__bytes_read.sum + dram__bytes_write.sum over one launch, divided by the
# elements of that launch); the capture is summarised under profiles/.
NCU_TRAFFIC_BYTES_PER_ELEMENT = {
    # (134.26 MB read + 211.51 MB written) / 2^26 elements, captured at n = 2^26 where the tensors
    # exceed L2; at the bench's 12.6M elements most writes are still in L2 when the kernel ends
    "gelu_erf_bf16_forward": 5.152,
}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                return float(json.load(f)["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


from paper_2209_10778_b200.clocks import ClockSampler  # noqa: E402


# --------------------------------------------------------------------------- reference arm (the oracle on host cores)

def _oracle_sample_rate(kinds, dtype, x_std, g_std, budget_s: float, threads: int, n_max: int = 1 << 26):
    """elements/s of the fp64 oracle (forward + rounding + backward) on a bounded sample."""
    import numpy as np
    import oracle
    from paper_2209_10778_b200 import workloads as W
    oracle.set_threads(threads)
    n_probe = 1 << 18
    x = W.raw_numpy(W.normal(n_probe, dtype, 0, x_std))
    g = W.raw_numpy(W.normal(n_probe, dtype, 1, g_std))
    t = time.perf_counter()
    for k in kinds:
        oracle.forward_backward(k, dtype, x, g)
    probe = time.perf_counter() - t
    rate = n_probe * len(kinds) / max(probe, 1e-9)
    n = int(min(max(rate * budget_s / len(kinds), n_probe), n_max))
    x = W.raw_numpy(W.normal(n, dtype, 0, x_std))
    g = W.raw_numpy(W.normal(n, dtype, 1, g_std))
    passes = 0
    t = time.perf_counter()
    while True:                                   # whole passes over the sample until the budget is spent
        for k in kinds:
            oracle.forward_backward(k, dtype, x, g)
        passes += 1
        dt = time.perf_counter() - t
        if dt >= budget_s or passes >= 64:
            break
    return n * len(kinds) * passes / dt, n * passes, dt


def run_reference(args, w):
    """--impl reference: the oracle, as it stands, timed on the host cores.  Each step is
    one fwd+round+bwd pass over a bounded sample, sized so that warm-up plus K steps take
    about two minutes in all."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2209_10778_b200 import workloads as W
    threads = oracle.max_threads()
    oracle.set_threads(threads)
    probe_rate, _, _ = _oracle_sample_rate(w.kinds, w.dtype, w.x_std, w.g_std, 1.0, threads)
    total = max(1, args.steps + args.warmup)
    n_s = int(min(max(probe_rate * 120.0 / total / len(w.kinds), 4096), w.numel(0)))
    x = W.raw_numpy(W.normal(n_s, w.dtype, w.x_seed, w.x_std))
    g = W.raw_numpy(W.normal(n_s, w.dtype, w.g_seed, w.g_std))
    times = []
    for i in range(total):
        t = time.perf_counter()
        for k in w.kinds:
            oracle.forward_backward(k, w.dtype, x, g)
        if i >= args.warmup:
            times.append(time.perf_counter() - t)
    dt = sum(times)
    value = n_s * len(w.kinds) * len(times) / dt if dt > 0 else 0.0
    n_total = w.numel(0) * len(w.kinds)
    sample = f"first {n_s} of {w.numel(0)} elements per kind, {len(w.kinds)} kinds, fwd+round+bwd in fp64, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": (n_total / value * 1e3) if value else None, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "kinds": list(w.kinds), "shape": list(w.shapes[0]),
                   "note": "ms_per_step is the sample rate extrapolated to the full workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm

def run_ours(args, w):
    import torch
    from paper_2209_10778_b200 import ranks
    from paper_2209_10778_b200 import binding as nfad
    from paper_2209_10778_b200 import workloads as W

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the path has no CPU implementation")
    nfad.load()                                    # fails loudly if libnfad.so is missing

    wd = ranks.world_from_env()
    world, rank, local_rank = wd.size, wd.rank, wd.local_rank
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    ranks.init(wd, "nccl", dev)

    n = w.numel(0)
    es = 4 if w.dtype == "f32" else 2
    kinds = list(w.kinds)
    per_set = 5 * n * es
    n_sets = max(12, -(-4 * L2_BYTES // per_set) + 1)
    n_sets += n_sets % 2
    half = n_sets // 2

    sets = []
    for i in range(n_sets):
        x = W.normal(n, w.dtype, w.x_seed + 100 * i, w.x_std, dev)
        g = W.normal(n, w.dtype, w.g_seed + 100 * i, w.g_std, dev)
        sets.append({"x": x, "g": g, "y": torch.empty_like(x), "d": torch.empty_like(x), "gin": torch.empty_like(x)})
    for s in sets:                                  # every f' buffer holds a real derivative before timing
        nfad.nfad_act_forward(kinds[0], s["x"], s["y"], s["d"])
    torch.cuda.synchronize()

    ev = {"fwd": [], "bwd": []}

    def step(i: int, timed: bool):
        for j, kind in enumerate(kinds):
            a = sets[(len(kinds) * i + j) % n_sets]
            b = sets[(len(kinds) * i + j + half) % n_sets]
            nfad.nfad_act_forward(kind, a["x"], a["y"], a["d"])
            nfad.nfad_act_backward(kind, b["g"], b["d"], b["gin"])

    # One period of the buffer rotation (after it every launch sees the buffers of period
    # steps ago) is captured in a CUDA graph: the step is four ~15 us kernels, and replaying
    # the graph keeps the host's launch cost out of the device time.  The last `period` steps of
    # the timed region are launched from the host with events (step_group), which gives the
    # per-kernel durations live, inside the timed region.
    import math
    period = n_sets // math.gcd(n_sets, len(kinds))
    graph = None
    if not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(period):
                step(i, False)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(period):
                step(i, False)

    def group_launches(j: int, kind: str, first: int, count: int, backward: bool):
        for i in range(first, first + count):
            if backward:
                b = sets[(len(kinds) * i + j + half) % n_sets]
                nfad.nfad_act_backward(kind, b["g"], b["d"], b["gin"])
            else:
                a = sets[(len(kinds) * i + j) % n_sets]
                nfad.nfad_act_forward(kind, a["x"], a["y"], a["d"])

    # The same period of steps with its launches reordered kernel by kernel (all forwards of the first
    # kind, all its backwards, then the next kind), each run captured in a graph of its own: the
    # launches of a step are independent of one another, so this is the same work on the same buffers,
    # and one event pair around a replay brackets `period` back-to-back launches of ONE kernel with
    # neither the host's launch rate nor per-launch event latency in the figure.
    group_graphs = None
    if graph is not None:
        group_graphs = []
        for j, kind in enumerate(kinds):
            pair = []
            for backward in (False, True):
                gg = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gg):
                    group_launches(j, kind, 0, period, backward)
                pair.append(gg)
            group_graphs.append(pair)

    def step_group(first: int, count: int):
        """`count` whole steps, kernel-major (see above); `first` is a multiple of the period when graphs are used."""
        for j, kind in enumerate(kinds):
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record()
            if group_graphs is not None and count == period:
                group_graphs[j][0].replay()
            else:
                group_launches(j, kind, first, count, False)
            e1.record()
            if group_graphs is not None and count == period:
                group_graphs[j][1].replay()
            else:
                group_launches(j, kind, first, count, True)
            e2.record()
            if j == 0:
                ev["fwd"].append((e0, e1, count))
                ev["bwd"].append((e1, e2, count))

    def run_steps(first: int, count: int, with_events: bool):
        """`count` steps starting at step index `first` (a multiple of the period when a graph is used)."""
        i = first
        tail = min(count, period) if with_events else 0
        if graph is not None:
            while count - tail >= period:
                graph.replay()
                i += period
                count -= period
        while count > tail:
            step(i, False)
            i += 1
            count -= 1
        if tail:
            step_group(i, tail)

    def barrier():
        ranks.barrier(wd, cuda=True)

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
    warm = max(3, args.warmup)
    run_steps(0, warm + (-warm) % period, False)
    barrier()
    t_wall0 = time.time()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    run_steps(0, args.steps, True)
    end.record()
    barrier()
    t_wall1 = time.time()
    ms = start.elapsed_time(end)
    window = "timed region"
    if sampler and (t_wall1 - t_wall0) < 1.5:
        # the timed region is shorter than nvidia-smi's sampling period: keep the same loop
        # running, untimed, so that the clock record is taken under the same load
        window = "untimed continuation of the same loop (timed region < 1.5 s)"
        t_wall0 = time.time()
        while time.time() - t_wall0 < 1.5:
            run_steps(0, 50 * period, False)
            torch.cuda.synchronize()
        t_wall1 = time.time()
    if sampler:
        sampler.stop()
    ms = ranks.max_over_ranks(wd, ms, dev)

    timing_source = ("one event pair around the last %d steps' launches of this kernel, %s back to back "
                     "at the end of the timed region" % (min(args.steps, period),
                                                         "replayed from a graph" if graph is not None and args.steps >= period else "issued"))
    src = ev
    fwd_ms = statistics.mean(a.elapsed_time(b) / c for a, b, c in src["fwd"]) if src["fwd"] else None
    bwd_ms = statistics.mean(a.elapsed_time(b) / c for a, b, c in src["bwd"]) if src["bwd"] else None

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    hx = [torch.empty(n, dtype=sets[0]["x"].dtype).pin_memory() for _ in kinds]
    hg = [torch.empty(n, dtype=sets[0]["x"].dtype).pin_memory() for _ in kinds]
    hy = [torch.empty(n, dtype=sets[0]["x"].dtype).pin_memory() for _ in kinds]
    hgin = [torch.empty(n, dtype=sets[0]["x"].dtype).pin_memory() for _ in kinds]
    for j in range(len(kinds)):
        hx[j].copy_(sets[j]["x"])
        hg[j].copy_(sets[j]["g"])

    e2e_ws = torch.empty(nfad.nfad_host_step_workspace_bytes(sets[0]["x"].dtype, n), dtype=torch.uint8, device=dev)

    def e2e_step(i: int):
        # the C-ABI call with HOST buffers: chunked host-to-device copies, both kernels, device-to-host copies,
        # pipelined inside the library; y and grad_in come back, f' stays on the device
        for j, kind in enumerate(kinds):
            nfad.nfad_host_step(kind, hx[j], hg[j], hy[j], None, hgin[j], e2e_ws, inputs_ready=True)

    e2e_steps = max(3, min(args.steps, 20))
    for i in range(3):
        e2e_step(i)
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    s1.record()
    barrier()
    e2e_ms = s0.elapsed_time(s1)
    e2e_ms = ranks.max_over_ranks(wd, e2e_ms, dev)

    if rank != 0:
        ranks.finish(wd)
        return

    elems_per_step = n * len(kinds)
    value = ranks.whole_job_rate(wd, elems_per_step, args.steps, ms)
    e2e_value = ranks.whole_job_rate(wd, elems_per_step, e2e_steps, e2e_ms)
    peak, peak_kind = _peaks()
    algo_bytes = 3 * es * n                       # forward: read x, write y and f'
    achieved = algo_bytes / (fwd_ms / 1e3) / 1e9 if fwd_ms else None
    key = f"{kinds[0]}_{w.dtype}_forward"
    tpe = NCU_TRAFFIC_BYTES_PER_ELEMENT.get(key)
    roofline = {
        "bound": "hbm", "kernel": f"nfad_act_forward[{kinds[0]},{w.dtype}]", "achieved": achieved, "peak": peak,
        "unit": "GB/s", "frac": (achieved / peak) if achieved else None, "peak_source": f"{peak_kind} copy bandwidth",
        "frac_of_nominal_8000": (achieved / 8000.0) if achieved else None,
        "algorithmic_bytes_per_launch": algo_bytes, "avg_launch_ms": fwd_ms, "timing": timing_source,
        "step": {"algorithmic_bytes": 2 * len(kinds) * algo_bytes,
                 "achieved": 2 * len(kinds) * algo_bytes / (ms / args.steps / 1e3) / 1e9,
                 "frac": 2 * len(kinds) * algo_bytes / (ms / args.steps / 1e3) / 1e9 / peak,
                 "note": "all four launches of a step (same bytes each) over ms_per_step, launch gaps included"},
        "traffic": (tpe * n) if tpe else None,
        "backward": {"achieved": (3 * es * n / (bwd_ms / 1e3) / 1e9) if bwd_ms else None, "avg_launch_ms": bwd_ms},
    }

    threads = 1
    cpu_baseline = None
    try:
        import oracle
        threads = oracle.max_threads()
        rate, n_used, dt = _oracle_sample_rate(kinds, w.dtype, w.x_std, w.g_std, 10.0, threads, 4 * n)
        rate1, n1, dt1 = _oracle_sample_rate(kinds, w.dtype, w.x_std, w.g_std, 3.0, 1, 4 * n)
        cpu_baseline = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": f"{n_used} elements per kind drawn like the workload's {n}, {len(kinds)} kinds, "
                                  f"fwd+round+bwd in fp64, {dt:.1f} s",
                        "single_thread": {"value": rate1, "unit": UNIT, "sample": f"{n1} elements per kind, {dt1:.1f} s"}}
    except Exception as exc:  # the oracle is test infrastructure; its absence must not hide the GPU number
        cpu_baseline = {"value": None, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": f"unavailable: {exc}"}

    large = None
    if not args.no_large:
        # the same kernels on one [64,512,3072] tensor (100.7M elements, larger than L2): where the
        # >= 85 %-of-peak target is stated
        from paper_2209_10778_b200 import sweep
        del sets
        torch.cuda.empty_cache()
        large = {}
        for kind in kinds:
            for op in ("forward", "backward"):
                r = sweep.time_case(kind, w.dtype, op, 64 * 512 * 3072, reps=20, dev=dev)
                large[f"{kind}_{op}"] = {"GBps": r["GBps"], "frac_of_peak": r["frac_of_peak"], "ms": r["ms"]}

    saved = {lay: nfad.nfad_saved_bytes_per_element(kinds[0], w.dtype, lay) for lay in nfad.LAYOUTS}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "kinds": kinds, "shape": list(w.shapes[0]), "elements": n,
                   "l2": f"{n_sets} rotating buffer sets ({n_sets * per_set >> 20} MiB), backward reads the f' written "
                         f"{half} sets earlier: no tensor is re-used from L2",
                   "saved_bytes_per_element": saved},
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 2 * n * es * len(kinds),
                "d2h_bytes_per_step": 2 * n * es * len(kinds), "steps": e2e_steps,
                "api": "nfad_host_step: pinned host x, grad_out in; y, grad_in out; copies and kernels pipelined by the library"},
        "gpu_launches": 2 * len(kinds) * args.steps,
        "launch": ("CUDA graph of one buffer-rotation period (%d steps); the last %d steps replayed from kernel-major graphs (one per kernel) between events" % (period, period))
                  if graph is not None else "every kernel launched from the host",
        "large_tensor_100663296": large,
        "clocks": sampler.summary(t_wall0, t_wall1, window) if sampler else None,
    }
    print(json.dumps(line), flush=True)
    ranks.finish(wd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="bert_base_ffn")
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host instead of replaying a CUDA graph")
    ap.add_argument("--no-large", action="store_true", help="skip the per-kernel numbers at 100.7M elements")
    args = ap.parse_args()
    from paper_2209_10778_b200 import workloads as W
    w = W.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
