"""Per-kernel timing sweep of the activation pass (one JSON line per case).

    python -m paper_2209_10778_b200.sweep --n 100663296 --dtypes bf16 --kinds gelu_erf --ops forward,backward
    python -m paper_2209_10778_b200.sweep --config sizes      # every kind x dtype at n = 2^16 ... 2^30
    python -m paper_2209_10778_b200.sweep --config resnet50   # Mish / Swish on the five ResNet-50 stage shapes
    python -m paper_2209_10778_b200.sweep --config stack      # 12 stacked GELU layers under three layouts
    python -m paper_2209_10778_b200.sweep --config probe      # plain 1:1 / 1:2 / 2:1 traffic through the same engine
    python -m paper_2209_10778_b200.sweep --config opbyop     # nested vs operator-by-operator back-propagation, measured
    python -m paper_2209_10778_b200.sweep --config bias       # bias-add and bias gradient fused into the pass vs separate launches

Each case launches one kernel `reps` times back to back between two CUDA events
on the launching stream, after 3 warm-up launches; buffers are rotated so that
at least 4x the L2 capacity is touched between two uses of the same buffer
(tensors larger than L2 need no rotation).  GB/s is algorithmic bytes (the
tensors the call must read and write, once) over the mean launch time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

import torch

from . import binding as nfad
from . import workloads as W

L2_BYTES = 126 * 1024 * 1024

# tensors read / written per element by each call
OPS = {
    "forward": (1, 2), "infer": (1, 1), "backward": (2, 1),
    "conv_backward": (2, 1), "recompute_backward": (2 + 1 + 1, 1 + 1),   # phase 1: x -> h; phase 2: g, x, h -> gin
    "forward_strict": (1, 2),                                              # fp32 storage only
    "bias_forward": (1, 2), "bias_backward": (2, 1),                       # + cols elements of bias / cols floats: negligible
}


def _peak():
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def _make_sets(n, dtype, n_tensors, dev, std=1.0, dist="normal"):
    """dist: how x is drawn -- "normal" (N(0, std^2)), "uniform20" (U(-20, 20)), "mix" (the stress mix with
    magnitudes up to 80), or "tiny" (x ~ N(0,1), and grad_out ~ N(0, (1e-38)^2) -- 1e-6 for fp16 --
    so that most backward products land in the storage type's subnormal range)."""
    es = 4 if dtype == "f32" else 2
    per_set = n_tensors * n * es
    n_sets = 1 if n * es > L2_BYTES else max(2, -(-4 * L2_BYTES // per_set))
    n_sets = min(n_sets, 256)
    sets = []
    for i in range(n_sets):
        x = W.normal(n, dtype, 10 + i, std, dev) if dist in ("normal", "tiny") else W.draw(dist, n, dtype, 10 + i, dev)
        g = W.normal(n, dtype, 500 + i, (1e-6 if dtype == "f16" else 1e-38) if dist == "tiny" else 1.0, dev)
        s = {"x": x, "g": g, "y": torch.empty_like(x), "d": torch.empty_like(x), "gin": torch.empty_like(x)}
        sets.append(s)
    return sets


def time_case(kind: str, dtype: str, op: str, n: int, reps: int = 20, dev="cuda", std=1.0, cols: int = 3072, repeats: int = 10,
              dist: str = "normal"):
    """cols: row length for the bias-fused calls (n must be a multiple of it)."""
    es = 4 if dtype == "f32" else 2
    sets = _make_sets(n, dtype, 5, dev, std, dist)
    if op.startswith("bias_"):
        rows = n // cols
        bias = W.normal(cols, dtype, 3, 0.5, dev)
        gb = torch.empty(cols, dtype=torch.float32, device=dev)
        nb = nfad.nfad_bias_act_backward_scratch_bytes(dtype, rows, cols)
        bias_scratch = torch.empty(max(nb, 4), dtype=torch.uint8, device=dev) if nb else None
    for s in sets:
        nfad.nfad_act_forward(kind, s["x"], s["y"], s["d"])
    scratch = None
    if op == "recompute_backward":
        scratch = [torch.empty(nfad.nfad_cmp_recompute_scratch_bytes(kind, dtype, n), dtype=torch.uint8, device=dev)
                   for _ in sets]

    def launch(i):
        s = sets[i % len(sets)]
        if op == "forward":
            nfad.nfad_act_forward(kind, s["x"], s["y"], s["d"])
        elif op == "forward_strict":
            nfad.nfad_act_forward_strict(kind, s["x"], s["y"], s["d"])
        elif op == "infer":
            nfad.nfad_act_forward_infer(kind, s["x"], s["y"])
        elif op == "backward":
            nfad.nfad_act_backward(kind, s["g"], s["d"], s["gin"])
        elif op == "conv_backward":
            nfad.nfad_cmp_conv_backward(kind, s["g"], s["x"], s["gin"])
        elif op == "recompute_backward":
            nfad.nfad_cmp_recompute_backward(kind, s["g"], s["x"], scratch[i % len(sets)], s["gin"])
        elif op == "bias_forward":
            nfad.nfad_bias_act_forward(kind, s["x"], bias, s["y"], s["d"])
        elif op == "bias_backward":
            nfad.nfad_bias_act_backward(kind, s["g"], s["d"], s["gin"], gb, bias_scratch)
        else:
            raise ValueError(op)

    def burst(first: int, count: int) -> float:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(count):
            launch(first + i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / count

    for i in range(3):
        launch(i)
    torch.cuda.synchronize()
    # `repeats` bursts of `reps` back-to-back launches, the burst sized to last >= 20 ms; the median burst is reported
    est = burst(3, max(3, min(reps, 8)))
    per_burst = max(reps, min(4096, int(20.0 / max(est, 1e-4)) + 1)) if repeats > 1 else reps
    samples = [burst(3 + r * per_burst, per_burst) for r in range(repeats)]
    ms = statistics.median(samples)
    r, w = OPS[op]
    algo = (r + w) * es * n
    peak, src = _peak()
    gbs = algo / (ms / 1e3) / 1e9
    return {"kind": kind, "dtype": dtype, "op": op, "n": n, "ms": ms, "elements_per_s": n / (ms / 1e3),
            "algorithmic_bytes": algo, "GBps": gbs, "frac_of_peak": gbs / peak, "peak_GBps": peak, "peak_source": src,
            "frac_of_nominal_8000": gbs / 8000.0, "buffer_sets": len(sets), "launches_per_burst": per_burst, "bursts": repeats,
            "ms_min": min(samples), "ms_max": max(samples), "x_std": std, "dist": dist,
            "inputs": {"generator": "torch.Generator(device).manual_seed", "x_seed": "10 + set index", "g_seed": "500 + set index",
                       "torch": torch.__version__}}


def run_probe(n_words: int, reps: int = 20, dev="cuda"):
    """Bandwidth of plain 1:1, 1:2 and 2:1 read/write mixes through the streaming engine, and of
    cudaMemcpy-like torch copy_, on tensors of n_words fp32 words each."""
    out = []
    a = torch.randn(n_words, device=dev)
    b = torch.randn(n_words, device=dev)
    o0 = torch.empty_like(a)
    o1 = torch.empty_like(a)
    peak, src = _peak()
    sink = torch.zeros(4, device=dev)
    cases = [("probe 1R:0W (read only)", 1, lambda: nfad.nfad_probe_stream(1, 0, a, None, sink, None)),
             ("probe 0R:1W (write only)", 1, lambda: nfad.nfad_probe_stream(0, 1, None, None, o0, None)),
             ("probe 1R:1W", 2, lambda: nfad.nfad_probe_stream(1, 1, a, None, o0, None)),
             ("probe 1R:2W (forward's mix)", 3, lambda: nfad.nfad_probe_stream(1, 2, a, None, o0, o1)),
             ("probe 2R:1W (backward's mix)", 3, lambda: nfad.nfad_probe_stream(2, 1, a, b, o0, None)),
             ("torch copy_ 1R:1W", 2, lambda: o0.copy_(a))]
    for name, tensors, fn in cases:
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        gbs = tensors * 4 * n_words / (ms / 1e3) / 1e9
        out.append({"config": "probe", "case": name, "bytes_per_tensor": 4 * n_words, "ms": ms, "GBps": gbs,
                    "frac_of_peak": gbs / peak, "peak_GBps": peak, "peak_source": src})
    return out


def run_opbyop(n: int, dtype: str, kinds, reps: int = 5, dev="cuda"):
    """Forward + backward of each activation under four executions of the SAME function: the
    dedicated nested kernels, the run-time FAD sequence (one generic kernel), and operator-by-
    operator back-propagation (one kernel per primitive, every rule keeping what it needs) --
    the layout the paper's memory comparison is made against.  Reports kept bytes and time."""
    from . import sequence
    out = []
    x = W.normal(n, dtype, 0, 1.0, dev)
    g = W.normal(n, dtype, 1, 1.0, dev)
    es = x.element_size()

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    for kind in kinds:
        prog = sequence.PROGRAMS[kind]()
        y, d, gin = torch.empty_like(x), torch.empty_like(x), torch.empty_like(x)

        def nested():
            nfad.nfad_act_forward(kind, x, y, d)
            nfad.nfad_act_backward(kind, g, d, gin)

        def fused_seq():
            nfad.nfad_seq_forward(prog.ops, x, [y], [d])
            nfad.nfad_seq_backward([g], [d], gin)

        def compiled_seq():
            nfad.nfad_seq_set_executor("compiled")
            fused_seq()

        def interpreted_seq():
            nfad.nfad_seq_set_executor("interpreter")
            fused_seq()

        ex = sequence.OpByOp(prog)
        kept = {}

        def op_by_op():
            ex.forward(x)
            kept["bytes"] = ex.saved_bytes()
            ex.backward([g])

        rows = [("nested (dedicated kernels)", nested, n * es),
                ("nested (run-time sequence, compiled)", compiled_seq, n * es),
                ("nested (run-time sequence, interpreted)", interpreted_seq, n * es),
                ("operator by operator", op_by_op, None)]
        for name, fn, saved in rows:
            ms = timed(fn)
            out.append({"config": "opbyop", "kind": kind, "dtype": dtype, "n": n, "execution": name, "ms_fwd_bwd": ms,
                        "kept_bytes": saved if saved is not None else kept["bytes"],
                        "kept_tensors": (saved if saved is not None else kept["bytes"]) / (n * es),
                        "launches": 2 if saved is not None else None})
            torch.cuda.empty_cache()
    nfad.nfad_seq_set_executor("auto")
    return out


def run_stack(layers: int, n: int, dtype: str, kind: str, dev="cuda", reps: int = 3):
    """L stacked activations: forward through all layers, then backward in reverse, under the three
    layouts; reports the bytes kept alive between the passes and the total device time."""
    es = 2 if dtype != "f32" else 4
    out = []
    x0 = W.normal(n, dtype, 0, 1.0, dev)
    gL = W.normal(n, dtype, 1, 1.0, dev)
    for layout in ("nested", "conventional", "recompute"):
        torch.cuda.empty_cache()
        torch.cuda.reset_peak_memory_stats()
        base = torch.cuda.memory_allocated()
        # nested: the layer input may be dropped at once (two ping-pong activations) and f'(x_i) is kept;
        # the other two keep every layer's input x_i alive instead (x_0 is the caller's tensor)
        saved = [torch.empty_like(x0) for _ in range(layers if layout == "nested" else layers - 1)]
        act = [torch.empty_like(x0), torch.empty_like(x0)]
        grad = [torch.empty_like(x0), torch.empty_like(x0)]
        scratch = torch.empty(nfad.nfad_cmp_recompute_scratch_bytes(kind, dtype, n), dtype=torch.uint8, device=dev) \
            if layout == "recompute" else None
        inputs = [x0] + saved if layout != "nested" else None        # x_i for i = 0 .. layers-1

        def one_pass():
            if layout == "nested":
                cur = x0
                for i in range(layers):
                    nxt = act[i % 2]
                    nfad.nfad_act_forward(kind, cur, nxt, saved[i])
                    cur = nxt
            else:
                for i in range(layers):
                    nxt = inputs[i + 1] if i + 1 < layers else act[0]
                    nfad.nfad_act_forward_infer(kind, inputs[i], nxt)
            g = gL
            for i in reversed(range(layers)):
                gn = grad[i % 2]
                if layout == "nested":
                    nfad.nfad_act_backward(kind, g, saved[i], gn)
                elif layout == "conventional":
                    nfad.nfad_cmp_conv_backward(kind, g, inputs[i], gn)
                else:
                    nfad.nfad_cmp_recompute_backward(kind, g, inputs[i], scratch, gn)
                g = gn

        one_pass()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            one_pass()
        e1.record()
        torch.cuda.synchronize()
        out.append({"config": "stack", "layout": layout, "kind": kind, "dtype": dtype, "layers": layers, "n": n,
                    "ms_fwd_bwd": e0.elapsed_time(e1) / reps,
                    "saved_bytes": layers * n * nfad.nfad_saved_bytes_per_element(kind, dtype, layout),
                    "saved_bytes_op_by_op_analytic": layers * n * nfad.nfad_saved_bytes_per_element(kind, dtype, "op_by_op"),
                    "transient_scratch_bytes": scratch.numel() if scratch is not None else 0,
                    "max_memory_allocated_delta": torch.cuda.max_memory_allocated() - base,
                    "note": "saved_bytes counts one kept tensor per layer (f'(x_i), or x_i itself)"})
        del saved, act, grad, scratch, inputs
    return out


def run_bias(rows: int, cols: int, dtype: str, kinds, reps: int = 20, dev="cuda"):
    """The pass with its producer's bias, fused (nfad_bias_act_*) against the same work as separate launches:
    forward = a torch add that writes the pre-activation + nfad_act_forward; backward = nfad_act_backward + a torch
    column sum (fp32 accumulate) over the stored grad_in.  Times are per forward / per backward."""
    n = rows * cols
    es = 4 if dtype == "f32" else 2
    peak, src = _peak()
    sets = _make_sets(n, dtype, 6, dev)
    bias = W.normal(cols, dtype, 3, 0.5, dev)
    gb = torch.empty(cols, dtype=torch.float32, device=dev)
    nb = nfad.nfad_bias_act_backward_scratch_bytes(dtype, rows, cols)
    scratch = torch.empty(max(nb, 4), dtype=torch.uint8, device=dev) if nb else None
    for s in sets:
        s["z"] = torch.empty_like(s["x"])

    def timed(fn):
        # `reps` launches replayed from one CUDA graph: at 12.6M elements a launch is ~15 us and the
        # host (Python binding, torch dispatch) would otherwise be what is timed
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(3):
                fn(sets[i % len(sets)])
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(reps):
                fn(sets[(3 + i) % len(sets)])
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    out = []
    for kind in kinds:
        for s in sets:
            nfad.nfad_bias_act_forward(kind, s["x"], bias, s["y"], s["d"])

        def fwd_fused(s):
            nfad.nfad_bias_act_forward(kind, s["x"], bias, s["y"], s["d"])

        def fwd_split(s):
            torch.add(s["x"].view(rows, cols), bias, out=s["z"].view(rows, cols))
            nfad.nfad_act_forward(kind, s["z"], s["y"], s["d"])

        def bwd_fused(s):
            nfad.nfad_bias_act_backward(kind, s["g"], s["d"], s["gin"], gb, scratch)

        def bwd_split(s):
            nfad.nfad_act_backward(kind, s["g"], s["d"], s["gin"])
            torch.sum(s["gin"].view(rows, cols), dim=0, dtype=torch.float32, out=gb)

        # The same separate launches with the extra pass costed at what a streaming kernel of this library needs for its
        # traffic alone: a copy of the tensor (read x, write the pre-activation) in place of the framework's broadcast
        # add, a read of the tensor in place of the column sum.  Only the bytes of the extra pass are reproduced (the
        # values are not): this is the floor for any separate implementation, not a usable one.
        words = lambda t: t.view(torch.uint8).view(torch.float32)      # the probe moves fp32 words: same bytes
        sink = torch.zeros(4, device=dev)

        def fwd_split_floor(s):
            nfad.nfad_probe_stream(1, 1, words(s["x"]), None, words(s["z"]), None)
            nfad.nfad_act_forward(kind, s["z"], s["y"], s["d"])

        def bwd_split_floor(s):
            nfad.nfad_act_backward(kind, s["g"], s["d"], s["gin"])
            nfad.nfad_probe_stream(1, 0, words(s["gin"]), None, sink, None)

        for s in sets:                                   # the copied pre-activation must hold real values for the forward
            s["z"].copy_(s["x"])
        for name, fn, tensors in (("forward fused", fwd_fused, 3), ("forward separate (framework add)", fwd_split, 5),
                                  ("forward separate (traffic floor)", fwd_split_floor, 5),
                                  ("backward fused", bwd_fused, 3), ("backward separate (framework sum)", bwd_split, 4),
                                  ("backward separate (traffic floor)", bwd_split_floor, 4)):
            ms = timed(fn)
            fused_bytes = 3 * es * n
            out.append({"config": "bias", "kind": kind, "dtype": dtype, "rows": rows, "cols": cols, "case": name, "ms": ms,
                        "tensor_passes": tensors, "GBps_of_fused_bytes": fused_bytes / (ms / 1e3) / 1e9,
                        "frac_of_peak": fused_bytes / (ms / 1e3) / 1e9 / peak, "peak_GBps": peak, "peak_source": src})
    return out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default=None, choices=[None, "sizes", "resnet50", "stack", "bert", "probe", "opbyop", "bias"])
    ap.add_argument("--cols", type=int, default=3072)
    ap.add_argument("--n", type=int, default=100663296)
    ap.add_argument("--kinds", default="gelu_erf,gelu_tanh,swish,mish")
    ap.add_argument("--dtypes", default="bf16")
    ap.add_argument("--dists", default="normal", help="input distributions: normal, uniform20, mix, tiny (backward: products in fp32's subnormal range)")
    ap.add_argument("--ops", default="forward,backward")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--max-log2", type=int, default=30)
    ap.add_argument("--min-log2", type=int, default=16)
    ap.add_argument("--repeats", type=int, default=10, help="bursts per case (1 under a profiler: the burst is then `reps` launches)")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("needs a CUDA device")
    nfad.load()
    from .clocks import ClockSampler
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    t_start = time.time()
    try:
        _run_config(args)
    finally:
        sampler.stop()
        print(json.dumps({"config": "clocks", **sampler.summary(t_start, time.time(), "the whole sweep")}), flush=True)


def _run_config(args):
    kinds, dtypes, ops = args.kinds.split(","), args.dtypes.split(","), args.ops.split(",")
    dists = args.dists.split(",")
    if args.config == "sizes":
        for n in W.SWEEP_SIZES:
            if n > (1 << args.max_log2) or n < (1 << args.min_log2):
                continue
            for dtype in dtypes:
                for dist in dists:
                    for kind in kinds:
                        for op in ops:
                            reps = max(3, min(args.reps, (1 << 28) // n + 3))
                            print(json.dumps(time_case(kind, dtype, op, n, reps, dist=dist)), flush=True)
                            torch.cuda.empty_cache()
    elif args.config == "resnet50":
        w = W.WORKLOADS["resnet50_stages"]
        for si, shape in enumerate(w.shapes):
            for kind in w.kinds:
                for op in ops:
                    r = time_case(kind, w.dtype, op, w.numel(si), args.reps)
                    r["shape"] = list(shape)
                    print(json.dumps(r), flush=True)
    elif args.config == "bert":
        w = W.WORKLOADS["bert_base_ffn"]
        for kind in w.kinds:
            for op in ops:
                r = time_case(kind, w.dtype, op, w.numel(0), args.reps, std=w.x_std)
                r["shape"] = list(w.shapes[0])
                print(json.dumps(r), flush=True)
    elif args.config == "probe":
        for r in run_probe(args.n // 2, args.reps):          # n bf16-sized elements -> n/2 words
            print(json.dumps(r), flush=True)
    elif args.config == "opbyop":
        for dtype in dtypes:
            for r in run_opbyop(args.n, dtype, kinds):
                print(json.dumps(r), flush=True)
    elif args.config == "bias":
        for dtype in dtypes:
            for r in run_bias(args.n // args.cols, args.cols, dtype, kinds, args.reps):
                print(json.dumps(r), flush=True)
            torch.cuda.empty_cache()
    elif args.config == "stack":
        w = W.WORKLOADS["gelu_stack_12"]
        for r in run_stack(w.layers, w.numel(0), w.dtype, w.kinds[0]):
            print(json.dumps(r), flush=True)
    else:
        for dtype in dtypes:
            for dist in dists:
                for kind in kinds:
                    for op in ops:
                        print(json.dumps(time_case(kind, dtype, op, args.n, args.reps, cols=args.cols, repeats=args.repeats,
                                                   dist=dist)), flush=True)
                        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
