#!/usr/bin/env python
"""Throughput of MoFQ per-layer format selection on B200.

A step is one whole-model selection (Algorithm 1 over every linear layer of the workload):
quantise every weight tensor (and, for the layer-output criterion, the calibration activations)
onto each candidate grid, reduce the errors, pick per layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference] [--shard]

Prints ONE JSON line (rank 0).  The headline workload is the largest one that stays resident in
HBM: the LLaMA-33B-shaped weight-only 4-bit model scored under per-channel AND group-128 scales
from one read (64.2 GB of fp16 weights, four candidates per element).  `value` counts fp16 bytes of
tensor quantised+scored per second over all ranks; `e2e` is the same metric through the
host-buffer entry point (pinned host tensors, host->device copies inside the timed region);
`roofline` relates the scoring kernel to the measured HBM copy bandwidth; `cpu_baseline` is the
CPU oracle on a bounded sample.  At one GPU the line also carries `workloads`: one record per
workload of the list in paper_2305_12356_b200/inputs.py (time per whole-model pass, GB/s, roofline
of its dominant kernel, share of layers that chose an FP format, smallest decision margin).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "GB/s of fp16 tensor quantized+scored (both formats)"
UNIT = "GB/s"
HEADLINE = "llama33b_w4_channel_and_group128"
WORKLOAD_ORDER = ["single_4096_w4_channel", "llama7b_w4_group128", "llama13b_w8a8_layer",
                  "llama33b_w4_channel_and_group128", "llama65b_w8a8_layer"]
# DRAM bytes per element of the scoring kernels, from the ncu captures summarised in profiles/ (read + write bytes
# over the elements of the captured case; traffic is proportional to the elements processed).  None: not captured
# for the kernel as it stands.
DRAM_BYTES_PER_ELEMENT = {"kq_score_mt": (809.61e6 + 3.57e6) / 404750336,          # 14 layers of the 7B-shaped model
                          "kq_score_rows_mt": (2140.22e6 + 4.90e6) / 1070071808}  # 14 layers of the 33B-shaped model
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126e6


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--blocks", type=int, default=None, help="decoder blocks to build (default: the workload's)")
    ap.add_argument("--shard", action="store_true",
                    help="N > 1: split ONE model's layer list over the ranks instead of one model per rank")
    ap.add_argument("--only", action="store_true", help="time the headline workload only (no `workloads` map)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-gb", type=float, default=6.5, help="fp16 GB of the workload's first layers that the host-buffer pass copies")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return json.load(open(path)), "measured"
        except Exception:
            pass
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def static_config(workload, blocks=None):
    """The facts that name a workload; identical in both arms of the bench."""
    from paper_2305_12356_b200 import inputs
    wl = inputs.WORKLOADS[workload]
    shapes = inputs.workload_layers(workload, blocks)
    n_elems = sum(o * i for _, o, i in shapes)
    return {"workload": workload, "layers": len(shapes), "elements": n_elems, "fp16_GB": 2 * n_elems / 1e9,
            "candidates": list(wl["candidates"]), "granularity": list(wl["w_gran"]), "group": wl["group"],
            "criterion": wl["metric"], "tokens": wl["tokens"],
            "l2": "inputs larger than L2" if 2 * n_elems > 2 * L2_BYTES else "L2 flushed between timed steps"}


# --------------------------------------------------------------------------------------------------
def host_cpu():
    """Logical CPUs of the host and its CPU model string (for the oracle's baseline record)."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "cpu_model": model}


def cpu_oracle_sample(workload, budget_s=12.0, max_chunks=64):
    """Time the CPU oracle (as it stands) on chunks of the workload's first layers."""
    from oracle import api as orc
    from paper_2305_12356_b200 import inputs
    wl = inputs.WORKLOADS[workload]
    layers = inputs.workload_layers(workload)
    cands = [getattr(orc, c) for c in wl["candidates"]]
    grans = [{"channel": orc.PER_CHANNEL, "group": orc.PER_GROUP, "tensor": orc.PER_TENSOR}[g] for g in wl["w_gran"]]
    orc.lib()
    done_bytes, t_total, chunks = 0, 0.0, 0
    if wl["metric"] == "layer_output":
        # the double-precision triple loop is far too slow for a whole layer: score 256 output rows against 64 of the
        # calibration tokens and scale the throughput by 64 / tokens (the oracle's cost is linear in the token count)
        t_s, rows = 64, 256
        while t_total < budget_s and chunks < max_chunks:
            li = chunks % len(layers)
            name, out_f, in_f = layers[li]
            w = inputs.weight_cpu(wl["w_kind"], min(rows, out_f), in_f, wl["seed"], li, **wl["w_args"])
            x = inputs.activation_cpu(t_s, in_f, wl["seed"], li, **wl["a_args"])
            t0 = time.perf_counter()
            errs = [orc.layer_output_error(x, w, f, False)[0] for f in cands]
            orc.select(errs)
            t_total += time.perf_counter() - t0
            done_bytes += w.numel() * 2
            chunks += 1
        scale = t_s / wl["tokens"]
        return {"value": done_bytes / t_total / 1e9 * scale, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "host": host_cpu(),
                "sample": f"{chunks} slices of {rows} output rows x {t_s} tokens from the first layers, {t_total:.1f} s of CPU "
                          f"work, layer-output criterion; value extrapolated to {wl['tokens']} tokens (x{scale:.4f})"}, done_bytes * scale, t_total
    while t_total < budget_s and chunks < max_chunks:
        name, out_f, in_f = layers[chunks % len(layers)]
        rows = min(out_f, 1024)
        w = inputs.weight_cpu(wl["w_kind"], rows, in_f, wl["seed"], chunks % len(layers), **wl["w_args"])
        t0 = time.perf_counter()
        for g in grans:
            errs = [orc.tensor_mse(w, f, g, wl["group"]) for f in cands]
            orc.select(errs)
        t_total += time.perf_counter() - t0
        done_bytes += w.numel() * 2
        chunks += 1
    return {"value": done_bytes / t_total / 1e9, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "host": host_cpu(),
            "sample": f"{chunks} chunks of <=1024 rows from the first layers ({done_bytes / 1e6:.0f} MB fp16), "
                      f"{t_total:.1f} s of CPU work, tensor-MSE criterion, {len(grans)} scale granularit{'ies' if len(grans) > 1 else 'y'}"}, done_bytes, t_total


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times, nbytes = [], 0
    per_step_budget = max(2.0, min(15.0, 120.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        cb, b, t = cpu_oracle_sample(args.workload, budget_s=per_step_budget)
        if i >= args.warmup:
            times.append(t)
            nbytes += b
    value = nbytes / sum(times) / 1e9
    cb["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times), "higher_is_better": True,
        "scaling": "strong" if args.shard else "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": static_config(args.workload, args.blocks),
        "note": "CPU oracle on a bounded sample of the workload per step",
        "cpu_baseline": cb,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# --------------------------------------------------------------------------------------------------
class Workload:
    """One workload built on a device: synthetic tensors, the marshalled layer list, a `step()`."""

    def __init__(self, name, dev, rank=0, blocks=None, layer_subset=None):
        import torch
        import paper_2305_12356_b200 as mofq
        from paper_2305_12356_b200 import binding as B
        from paper_2305_12356_b200 import inputs
        self.name, self.dev = name, dev
        wl = self.wl = inputs.WORKLOADS[name]
        self.layer_metric = wl["metric"] == "layer_output"
        all_shapes = inputs.workload_layers(name, blocks)
        self.index = list(range(len(all_shapes))) if layer_subset is None else list(layer_subset)
        shapes = self.shapes = [all_shapes[i] for i in self.index]
        seed = self.seed = wl["seed"] + 1000 * rank       # weak scaling: every rank scores a model of its own
        self.n_elems = sum(o * i for _, o, i in shapes)
        self.fp16_bytes = 2 * self.n_elems
        T = self.T = wl["tokens"]
        grans = self.grans = wl["w_gran"]
        self.cfg = mofq.make_config(wl["bits"], wl["candidates"], metric=wl["metric"], is_w_only=not self.layer_metric,
                                    w_gran=grans[0], w_group=wl["group"], w_gran2=grans[1] if len(grans) > 1 else None)
        self.n_rec = len(shapes) * len(grans)
        self.results = torch.empty(max(1, self.n_rec) * B.RESULT_BYTES, dtype=torch.uint8, device=dev)
        x_bytes = sum(2 * T * i for _, o, i in shapes) if self.layer_metric else 0
        self.streaming = self.fp16_bytes + x_bytes > 100e9          # synthesise each layer on the device inside the step
        self.layers, self.synth_ms, self.overlap_ms = [], 0.0, None
        if not shapes:
            self.step = lambda: None
            return
        if not self.streaming:
            for li, (_, out_f, in_f) in zip(self.index, shapes):
                w = torch.empty((out_f, in_f), dtype=torch.float16, device=dev)
                inputs.device_weight(w, wl["w_kind"], seed, li, **wl["w_args"])
                if self.layer_metric:
                    x = torch.empty((T, in_f), dtype=torch.bfloat16, device=dev)
                    inputs.device_activation(x, seed, li, **wl["a_args"])
                    self.layers.append((w, x))
                else:
                    self.layers.append(w)
            self.prepared = mofq.prepare_layers(self.layers)      # marshal the layer list once; a step is one C-ABI call
            self.ws = torch.empty(mofq.workspace_bytes(self.prepared, self.cfg), dtype=torch.uint8, device=dev)

            def step():
                mofq.select_formats(self.prepared, self.cfg, workspace=self.ws, results=self.results, parse=False)

            self.step = step
        else:
            # Two weight/activation buffers: layer i+1 is synthesised on a second stream while layer i is scored, so the
            # ~130 GB of weights are never resident at once and the generator hides behind the selection.
            max_w = max(o * i for _, o, i in shapes)
            max_x = max(T * i for _, o, i in shapes)
            self.bufs = [(torch.empty(max_w, dtype=torch.float16, device=dev), torch.empty(max_x, dtype=torch.bfloat16, device=dev))
                         for _ in range(2)]
            views = [[(wb[:o * i].view(o, i), xb[:T * i].view(T, i)) for _, o, i in shapes] for wb, xb in self.bufs]
            distinct = {tuple(v[0].shape): v for v in views[0]}
            self.ws = torch.empty(max(mofq.workspace_bytes([v], self.cfg) for v in distinct.values()), dtype=torch.uint8, device=dev)
            preps = [[mofq.prepare_layers([v]) for v in vs] for vs in views]
            res_views = [self.results[k * B.RESULT_BYTES:(k + 1) * B.RESULT_BYTES] for k in range(len(shapes))]
            side = torch.cuda.Stream(device=dev)
            filled = [torch.cuda.Event() for _ in range(2)]
            scored = [torch.cuda.Event() for _ in range(2)]

            def synth(k, b):
                w, x = views[b][k]
                inputs.device_weight(w, wl["w_kind"], seed, self.index[k], **wl["w_args"])
                inputs.device_activation(x, seed, self.index[k], **wl["a_args"])

            def step_serial():
                for k in range(len(shapes)):                 # one layer resident at a time, generator and selection back to back
                    synth(k, 0)
                    mofq.select_formats(preps[0][k], self.cfg, workspace=self.ws, results=res_views[k], parse=False)

            def step():
                main = torch.cuda.current_stream(dev)
                side.wait_stream(main)
                for k in range(len(shapes)):
                    b = k & 1
                    with torch.cuda.stream(side):
                        if k >= 2:
                            side.wait_event(scored[b])       # the buffer's previous layer has been scored
                        synth(k, b)
                        filled[b].record(side)
                    main.wait_event(filled[b])
                    mofq.select_formats(preps[b][k], self.cfg, workspace=self.ws, results=res_views[k], parse=False)
                    scored[b].record(main)
                main.wait_stream(side)

            def synth_only():
                for k in range(len(shapes)):
                    synth(k, 0)

            self.step, self.step_serial, self.synth_only = step, step_serial, synth_only

    def free(self):
        import torch
        for attr in ("layers", "prepared", "ws", "bufs", "results"):
            if hasattr(self, attr):
                delattr(self, attr)
        self.step = None
        torch.cuda.empty_cache()


def time_loop(fn, steps, warmup, barrier, flush=None):
    """ms per call of fn over `steps` calls after `warmup` calls, CUDA events on the current stream.  With `flush`
    (a callable that evicts L2) every call is timed on its own and the flush runs between the timed calls."""
    import torch
    for _ in range(warmup):
        fn()
    barrier()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return e0.elapsed_time(e1) / steps
    total = 0.0
    for _ in range(steps):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        total += e0.elapsed_time(e1)
    barrier()
    return total / steps


def kernel_facts(w):
    """Dominant kernel of a workload, its launches per step and all kernel launches per step (counted from the
    launch lists in profiles/)."""
    n = len(w.shapes)
    F = w.cfg.n_candidates
    if w.layer_metric:
        gemm = 2 if w.wl["bits"] == 8 else 1 + F          # 8-bit W+A: the candidates' products share one launch
        # per layer besides the products: activation abs-max, weight codes, activation codes (+ fp16 copy), finalize
        return "gemm_err_kernel", n * gemm, n * (gemm + 4) + (2 * n if w.streaming else 0)
    if w.grans == ("group",):
        return "kq_score_mt", 1, 2 + (n + 511) // 512      # table uploads (512 layers each) + persistent kernel + finalize
    if n == 1:
        return "kq_score_rows_mt", 1, 2                    # header clear + scoring launch (its last block applies Algorithm 1's comparison)
    return "kq_score_rows_mt", 1, 2 + (n + 255) // 256     # table uploads (256 layers each) + persistent kernel + finalize


def measure(w, args, barrier, peaks, which, steps, warmup, flusher):
    """Time one workload and return its record."""
    import torch
    from paper_2305_12356_b200 import binding as B
    flush = flusher if (w.fp16_bytes < 2 * L2_BYTES and not w.layer_metric) else None
    ms = time_loop(w.step, steps, warmup, barrier, flush)
    rec = {"ms_per_step": ms, "steps": steps, "warmup": warmup, "layers": len(w.shapes), "fp16_GB": w.fp16_bytes / 1e9,
           "value": w.fp16_bytes / (ms * 1e-3) / 1e9, "unit": UNIT, "criterion": w.wl["metric"],
           "l2": "L2 flushed between timed steps (each step timed on its own)" if flush else "inputs larger than L2"}
    if flush is not None:
        rec["ms_per_step_l2_resident"] = time_loop(w.step, steps, warmup, barrier, None)
        # the same call captured once into a CUDA graph and replayed (what a caller bound by launch latency would do)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            w.step()
        rec["ms_per_step_graph_replay"] = time_loop(graph.replay, steps, warmup, barrier, flush)
        rec["ms_per_step_graph_replay_l2_resident"] = time_loop(graph.replay, steps, warmup, barrier, None)
        del graph
    kernel, dom, launches = kernel_facts(w)
    rec["gpu_launches_per_step"] = launches
    recs = B._parse_results(bytes(w.results.cpu().numpy()), w.n_rec, w.cfg.n_candidates)
    assert all(r["status"] == 0 and 0 <= r["chosen"] < w.cfg.n_candidates for r in recs), "selection records are not clean"
    rec["fp_share"] = sum(1 for r in recs if w.wl["candidates"][r["chosen"]].startswith("FP")) / len(recs)
    rec["min_rel_margin"] = min(r["rel_margin"] for r in recs)
    w.records = recs
    if w.layer_metric:
        F, T = w.cfg.n_candidates, w.T
        flops = sum(2.0 * T * o * i * (1 + F) for _, o, i in w.shapes)
        sel_ms = ms
        if w.streaming:
            w.synth_ms = time_loop(w.synth_only, 1, 1, barrier)
            serial_ms = time_loop(w.step_serial, max(1, steps // 2), 1, barrier)
            sel_ms = serial_ms - w.synth_ms
            rec["model_select_time_ms"] = {"with_synthesis_overlapped": ms, "with_synthesis_serial": serial_ms,
                                           "synthesis_alone": w.synth_ms, "without_synthesis": sel_ms}
        else:
            rec["model_select_time_ms"] = ms
        tf = flops / (sel_ms * 1e-3) / 1e12
        p16 = float(peaks.get("bf16_tflops_sustained", 1400.0))
        # One fp16 reference GEMM plus F candidate GEMMs per layer.  In the 8-bit weight-and-activation setting the
        # candidates run on the 8-bit tensor kinds, whose peak is taken as twice the measured 16-bit one (nominal
        # ratio); the peak of the mix is total flop / (time of each part at its own peak).
        rate = 2.0 if w.wl["bits"] == 8 else 1.0
        tpeak = p16 * (1 + F) / (1.0 + F / rate)
        rec["roofline"] = {"bound": "tensor", "kernel": kernel, "achieved": tf, "peak": tpeak,
                           "peak_source": f"of {which}: sustained 16-bit dense {p16:.0f} TFLOP/s for the fp16 reference GEMM, "
                                          f"x{rate:.0f} for the {F} candidate GEMMs, combined by time",
                           "unit": "TFLOP/s", "frac": tf / tpeak, "flops_per_step": flops, "launches_per_step": dom,
                           "avg_launch_us": 1e3 * sel_ms / dom,
                           "note": "whole selection step (synthesis excluded) over the GEMM flops; operand preparation included",
                           "traffic": None}
    else:
        peak = float(peaks["hbm_gbs"])
        ach = w.fp16_bytes / (ms * 1e-3) / 1e9
        per_elem = DRAM_BYTES_PER_ELEMENT.get(kernel)
        rec["model_select_time_ms"] = ms
        rec["roofline"] = {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "peak_source": f"of {which}",
                           "unit": "GB/s", "frac": ach / peak, "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                           "launches_per_step": dom, "avg_launch_us": 1e3 * ms / dom,
                           "algorithmic_bytes_per_launch": w.fp16_bytes / dom,
                           "traffic": per_elem * w.n_elems / dom if per_elem else None}
    return rec


def emit_winners_ms(w, barrier):
    """Algorithm 1's last step, for context (not part of the metric): every layer quantised to its winner, which the
    kernels read on the device from the records the last selection step left."""
    import torch
    import paper_2305_12356_b200 as mofq
    from paper_2305_12356_b200 import binding as B
    bufs = B.EmitBuffers(w.prepared, w.cfg)
    ms = time_loop(lambda: mofq.emit_selected(w.prepared, w.cfg, w.results, buffers=bufs), 2, 1, barrier)
    assert int(bufs.ws[:4].view(torch.int32).item()) == 0
    del bufs
    return ms


def e2e_pass(w, args, dev, barrier, world):
    """The same metric through mofq_select_formats_host: pinned host tensors, host->device copies and the read-back of
    the records inside the timed region.  Bounded to the workload's first layers (args.e2e_gb of fp16) so that the
    pinned staging stays small; the throughput is PCIe-bound and does not depend on how many layers are copied."""
    import ctypes as C
    import torch
    import paper_2305_12356_b200 as mofq
    from paper_2305_12356_b200 import binding as B
    from paper_2305_12356_b200 import inputs
    from paper_2305_12356_b200.sharded import max_over_ranks
    wl = w.wl
    picked, nbytes, xbytes = [], 0, 0
    for k, (_, o, i) in enumerate(w.shapes):
        if picked and nbytes + 2 * o * i > args.e2e_gb * 1e9:
            break
        picked.append(k)
        nbytes += 2 * o * i
        xbytes += 2 * w.T * i if w.layer_metric else 0
    host_layers = []
    for k in picked:
        _, o, i = w.shapes[k]
        if w.streaming:
            wd = torch.empty((o, i), dtype=torch.float16, device=dev)
            inputs.device_weight(wd, wl["w_kind"], w.seed, w.index[k], **wl["w_args"])
            xd = torch.empty((w.T, i), dtype=torch.bfloat16, device=dev)
            inputs.device_activation(xd, w.seed, w.index[k], **wl["a_args"])
            src = (wd, xd)
        else:
            src = w.layers[k]
        if w.layer_metric:
            hw = torch.empty(src[0].shape, dtype=src[0].dtype, pin_memory=True)
            hx = torch.empty(src[1].shape, dtype=src[1].dtype, pin_memory=True)
            hw.copy_(src[0])
            hx.copy_(src[1])
            host_layers.append((hw, hx))
        else:
            h = torch.empty(src.shape, dtype=src.dtype, pin_memory=True)
            h.copy_(src)
            host_layers.append(h)
    torch.cuda.synchronize()
    arr = B._layer_array(host_layers, require_cuda=False)
    hws = torch.empty(mofq.lib().mofq_host_workspace_bytes(arr, len(host_layers), C.byref(w.cfg)), dtype=torch.uint8, device=dev)
    mofq.select_formats_host(host_layers[:1], w.cfg, dev, workspace=hws)        # warm-up
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        hrecs = mofq.select_formats_host(host_layers, w.cfg, dev, workspace=hws)
    e1.record()
    barrier()
    e_ms = max_over_ranks(e0.elapsed_time(e1), dev) / args.e2e_steps
    n_sets = len(w.grans)
    want = [r["chosen"] for k in picked for r in w.records[k * n_sets:(k + 1) * n_sets]]
    assert [r["chosen"] for r in hrecs] == want, "host-buffer pass disagrees with the device-resident pass"
    return {"value": world * nbytes / (e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": nbytes + xbytes,
            "d2h_bytes_per_step": len(hrecs) * B.RESULT_BYTES, "steps": args.e2e_steps, "ms_per_step": e_ms,
            "sample": f"first {len(picked)} of {len(w.shapes)} layers ({nbytes / 1e9:.2f} GB of fp16 weights) from pinned host memory"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    import paper_2305_12356_b200 as mofq
    from paper_2305_12356_b200 import inputs
    from paper_2305_12356_b200.sharded import layer_costs, max_over_ranks, partition_layers, select_formats_sharded

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    mofq.lib()
    peaks, which = measured_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    flush_buf = torch.empty(int(2.2 * L2_BYTES) // 4, dtype=torch.float32, device=dev)

    def flusher():
        flush_buf.add_(1.0)                          # reads and writes 2.2x the L2 capacity

    # ---- headline workload ------------------------------------------------------------------------------
    subset = None
    sharded = args.shard and world > 1
    if sharded:
        # ONE model, its layer list split over the ranks by cost (bytes of W for the tensor criterion, flops for the
        # layer-output criterion); no tensor data moves between GPUs, the records are gathered on the host
        wl0 = inputs.WORKLOADS[args.workload]
        costs = layer_costs(inputs.workload_layers(args.workload, args.blocks), wl0["metric"], wl0["tokens"])
        subset = partition_layers(costs, world)[rank]
    w = Workload(args.workload, dev, 0 if sharded else rank, args.blocks, subset)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    flush = flusher if (w.fp16_bytes < 2 * L2_BYTES and not w.layer_metric) else None
    ms_local = time_loop(w.step, args.steps, max(3, args.warmup), barrier, flush)
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = max_over_ranks(ms_local, dev)
    total_bytes = w.fp16_bytes
    if world > 1:
        t = torch.tensor([float(w.fp16_bytes)], dtype=torch.float64, device=dev)
        dist.all_reduce(t)
        total_bytes = float(t.item())
    value = total_bytes / (ms_per_step * 1e-3) / 1e9
    head = measure(w, args, barrier, peaks, which, max(1, min(args.steps, 5)), 1, flusher)   # records + roofline bookkeeping
    head["ms_per_step"], head["value"], head["steps"], head["warmup"] = ms_per_step, value, args.steps, max(3, args.warmup)
    if not w.layer_metric:
        ach = w.fp16_bytes / (ms_local * 1e-3) / 1e9
        head["roofline"].update(achieved=ach, frac=ach / head["roofline"]["peak"], frac_of_nominal_8TBs=ach / NOMINAL_HBM_GBS,
                                avg_launch_us=1e3 * ms_local / head["roofline"]["launches_per_step"])
        head["model_select_time_ms"] = ms_per_step
    if sharded:
        n_sets = len(w.grans)
        merged = select_formats_sharded(costs, lambda idx: [w.records[k * n_sets:(k + 1) * n_sets] for k in range(len(idx))])
        assert all(m is not None for m in merged)
        head["sharding"] = {"layers_per_rank": [len(p) for p in partition_layers(costs, world)], "records_gathered": len(merged)}

    # the same step timed alone (idle gaps between launches, so the board is not at its power cap): context for the
    # roofline fraction, which is quoted against a copy bandwidth measured as a burst; never the bench value
    if rank == 0 and not w.layer_metric and not w.streaming:
        samples = []
        for _ in range(5):
            torch.cuda.synchronize()
            time.sleep(0.05)
            b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            b0.record()
            w.step()
            b1.record()
            torch.cuda.synchronize()
            samples.append(b0.elapsed_time(b1))
        burst_ms = sorted(samples)[len(samples) // 2]
        head["roofline"]["isolated_step"] = {"ms": burst_ms, "achieved": w.fp16_bytes / (burst_ms * 1e-3) / 1e9,
                                             "frac": w.fp16_bytes / (burst_ms * 1e-3) / 1e9 / head["roofline"]["peak"],
                                             "note": "median of 5 steps launched alone after 50 ms idle (no power-cap throttling); context only"}

    if rank == 0 and w.grans == ("group",) and not w.layer_metric and not w.streaming and w.fp16_bytes < 40e9:
        head["emit_winners_ms"] = emit_winners_ms(w, torch.cuda.synchronize)   # rank 0 alone: no collective in its barrier
    e2e = None
    if not args.no_e2e:
        e2e = e2e_pass(w, args, dev, barrier, world)
    w.free()

    # ---- the other workloads (one GPU only: they would hold the other ranks idle) -----------------------------
    workloads = {}
    if rank == 0:
        workloads[args.workload] = dict(head, config_index=WORKLOAD_ORDER.index(args.workload) + 1 if args.workload in WORKLOAD_ORDER else None)
    if world == 1 and not args.only and args.blocks is None:
        for name in WORKLOAD_ORDER:
            if name == args.workload:
                continue
            ow = Workload(name, dev, 0)
            steps = max(1, min(args.steps, 3 if ow.streaming else 10 if ow.layer_metric else 50))
            rec = measure(ow, args, barrier, peaks, which, steps, 3, flusher)
            rec["config_index"] = WORKLOAD_ORDER.index(name) + 1
            if ow.grans == ("group",) and not ow.layer_metric:
                rec["emit_winners_ms"] = emit_winners_ms(ow, barrier)
            if ow.layer_metric and not args.no_e2e:
                rec["e2e"] = e2e_pass(ow, args, dev, barrier, world)
            if ow.layer_metric and not args.no_cpu_baseline:
                rec["cpu_baseline"] = cpu_oracle_sample(name, budget_s=8.0)[0]
            ow.free()
            workloads[name] = rec

    if rank == 0:
        _, _, launches = kernel_facts(w)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if sharded else "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": static_config(args.workload, args.blocks),
            "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * launches, "roofline": head["roofline"],
            "model_select_time_ms": head.get("model_select_time_ms"), "fp_share": head["fp_share"],
            "min_rel_margin": head["min_rel_margin"], "workloads": workloads,
        }
        if sharded:
            out["sharding"] = head["sharding"]
        if not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_oracle_sample(args.workload)[0]
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
