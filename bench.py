#!/usr/bin/env python
"""Throughput of MoFQ per-layer format selection on B200.

A step is one whole-model selection (Algorithm 1 over every linear layer of the workload):
quantise every weight tensor onto each candidate grid, reduce the errors, pick per layer.
Default workload: LLaMA-7B-shaped, weight-only 4-bit, group-128 scales, INT4 vs FP4-E2M1 by
tensor MSE, synthetic fp16 weights resident in HBM (12.95 GB, larger than L2).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` counts fp16 bytes of tensor quantised+scored per second
over all ranks; `e2e` is the same metric through the host-buffer entry point (pinned host
tensors, host->device copies inside the timed region); `roofline` relates the scoring kernel to
the measured HBM copy bandwidth; `cpu_baseline` is the CPU oracle on a bounded sample.
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
# DRAM bytes per element of kq_score_mt from the ncu capture summarised in profiles/ (read 809.63 MB + write 4.65 MB
# for 404,750,336 elements on a 14-layer case; traffic is proportional to the elements processed)
KQ_MT_DRAM_BYTES_PER_ELEMENT = (809.63e6 + 4.65e6) / 404750336
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b_w4_group128")
    ap.add_argument("--blocks", type=int, default=None, help="decoder blocks to build (default: the workload's)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=2)
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


# --------------------------------------------------------------------------------------------------
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
        return {"value": done_bytes / t_total / 1e9 * scale, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
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
    return {"value": done_bytes / t_total / 1e9, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{chunks} chunks of <=1024 rows from the first layers ({done_bytes / 1e6:.0f} MB fp16), "
                      f"{t_total:.1f} s of CPU work, tensor-MSE criterion"}, done_bytes, t_total


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2305_12356_b200 import inputs
    wl = inputs.WORKLOADS[args.workload]
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
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "candidates": list(wl["candidates"]), "granularity": list(wl["w_gran"]),
                   "group": wl["group"], "criterion": wl["metric"], "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": cb,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# --------------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    import paper_2305_12356_b200 as mofq
    from paper_2305_12356_b200 import binding as B
    from paper_2305_12356_b200 import inputs
    from paper_2305_12356_b200.sharded import max_over_ranks

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

    wl = inputs.WORKLOADS[args.workload]
    layer_metric = wl["metric"] == "layer_output"
    shapes = inputs.workload_layers(args.workload, args.blocks)
    # weak scaling: every rank scores a whole model of its own (seed offset by rank); no data-path collective
    seed = wl["seed"] + 1000 * rank
    n_elems = sum(o * i for _, o, i in shapes)
    fp16_bytes = 2 * n_elems
    T = wl["tokens"]
    grans = wl["w_gran"]
    cfg = mofq.make_config(wl["bits"], wl["candidates"], metric=wl["metric"], is_w_only=not layer_metric,
                           w_gran=grans[0], w_group=wl["group"], w_gran2=grans[1] if len(grans) > 1 else None)
    n_rec = len(shapes) * len(grans)
    results = torch.empty(n_rec * B.RESULT_BYTES, dtype=torch.uint8, device=dev)
    x_bytes = sum(2 * T * i for _, o, i in shapes) if layer_metric else 0
    streaming = fp16_bytes + x_bytes > 100e9          # synthesise each layer on the device inside the step
    layers = []
    if not streaming:
        for li, (_, out_f, in_f) in enumerate(shapes):
            w = torch.empty((out_f, in_f), dtype=torch.float16, device=dev)
            inputs.device_weight(w, wl["w_kind"], seed, li, **wl["w_args"])
            if layer_metric:
                x = torch.empty((T, in_f), dtype=torch.bfloat16, device=dev)
                inputs.device_activation(x, seed, li, **wl["a_args"])
                layers.append((w, x))
            else:
                layers.append(w)
        prepared = mofq.prepare_layers(layers)          # marshal the layer list once; a step is one C-ABI call
        ws = torch.empty(mofq.workspace_bytes(prepared, cfg), dtype=torch.uint8, device=dev)

        def step():
            mofq.select_formats(prepared, cfg, workspace=ws, results=results, parse=False)

        synth_ms = 0.0
    else:
        max_w = max(o * i for _, o, i in shapes)
        max_x = max(T * i for _, o, i in shapes)
        wbuf = torch.empty(max_w, dtype=torch.float16, device=dev)
        xbuf = torch.empty(max_x, dtype=torch.bfloat16, device=dev)
        views = [(wbuf[:o * i].view(o, i), xbuf[:T * i].view(T, i)) for _, o, i in shapes]
        distinct = {tuple(v[0].shape): v for v in views}
        ws = torch.empty(max(mofq.workspace_bytes([v], cfg) for v in distinct.values()), dtype=torch.uint8, device=dev)
        preps = [mofq.prepare_layers([v]) for v in views]
        res_views = [results[li * B.RESULT_BYTES:(li + 1) * B.RESULT_BYTES] for li in range(len(shapes))]

        def synth(li):
            w, x = views[li]
            inputs.device_weight(w, wl["w_kind"], seed, li, **wl["w_args"])
            inputs.device_activation(x, seed, li, **wl["a_args"])

        def step():
            for li in range(len(shapes)):                # one layer resident at a time (stream-ordered reuse of the buffers)
                synth(li)
                mofq.select_formats(preps[li], cfg, workspace=ws, results=res_views[li], parse=False)

        torch.cuda.synchronize()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for li in range(len(shapes)):
            synth(li)
        s0.record()
        for li in range(len(shapes)):
            synth(li)
        s1.record()
        torch.cuda.synchronize()
        synth_ms = s0.elapsed_time(s1)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(ev0.elapsed_time(ev1), dev)
    ms_per_step = ms / args.steps
    value = world * fp16_bytes / (ms_per_step * 1e-3) / 1e9

    # the same step timed alone (idle gaps between launches, so the board is not at its power cap): context for the
    # roofline fraction, which is quoted against a copy bandwidth measured as a burst; never the bench value
    burst_ms = None
    if rank == 0 and not layer_metric and not streaming:
        import time
        samples = []
        for _ in range(5):
            torch.cuda.synchronize()
            time.sleep(0.05)
            b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            b0.record()
            step()
            b1.record()
            torch.cuda.synchronize()
            samples.append(b0.elapsed_time(b1))
        burst_ms = sorted(samples)[len(samples) // 2]

    # Algorithm 1's last step, for context (not part of the metric): every layer quantised to its winner, read on
    # the device from the records the last step left
    emit_ms = None
    if rank == 0 and not layer_metric and not streaming and len(grans) == 1 and fp16_bytes < 40e9:
        bufs = B.EmitBuffers(prepared, cfg)
        mofq.emit_selected(prepared, cfg, results, buffers=bufs)
        torch.cuda.synchronize()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record()
        mofq.emit_selected(prepared, cfg, results, buffers=bufs)
        q1.record()
        torch.cuda.synchronize()
        emit_ms = q0.elapsed_time(q1)
        assert int(bufs.ws[:4].view(torch.int32).item()) == 0
        del bufs

    # decisions (for the record) and a sanity check that the step produced them
    recs = B._parse_results(bytes(results.cpu().numpy()), n_rec, cfg.n_candidates)
    assert all(r["status"] == 0 and 0 <= r["chosen"] < cfg.n_candidates for r in recs)
    fp_share = sum(1 for r in recs if wl["candidates"][r["chosen"]].startswith("FP")) / len(recs)
    min_margin = min(r["rel_margin"] for r in recs)

    # end to end through the host-buffer entry point (N ranks each copy their own model)
    e2e = None
    if not args.no_e2e and not streaming and not layer_metric:
        host_layers = [torch.empty(w.shape, dtype=w.dtype, pin_memory=True) for w in layers]
        for h, w in zip(host_layers, layers):
            h.copy_(w)
        torch.cuda.synchronize()
        arr = B._layer_array(host_layers, require_cuda=False)
        import ctypes as C
        hws = torch.empty(mofq.lib().mofq_host_workspace_bytes(arr, len(host_layers), C.byref(cfg)), dtype=torch.uint8, device=dev)
        mofq.select_formats_host(host_layers[:2], cfg, dev, workspace=hws)        # warm-up
        barrier()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            hrecs = mofq.select_formats_host(host_layers, cfg, dev, workspace=hws)
        e1.record()
        barrier()
        e_ms = max_over_ranks(e0.elapsed_time(e1), dev)
        assert [r["chosen"] for r in hrecs] == [r["chosen"] for r in recs]
        e2e = {"value": world * fp16_bytes / (e_ms / args.e2e_steps * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": fp16_bytes, "d2h_bytes_per_step": n_rec * B.RESULT_BYTES,
               "steps": args.e2e_steps, "ms_per_step": e_ms / args.e2e_steps}
        del host_layers, hws

    if rank == 0:
        peaks, which = measured_peaks()
        peak = float(peaks["hbm_gbs"])
        # algorithmic bytes: 2 B per element read once (+ 4 B per 128 elements of scale state never leaves the SM)
        F = cfg.n_candidates
        flops = sum(2.0 * T * o * i * (1 + F) for _, o, i in shapes) if layer_metric else 0.0
        # kernels per step, counted from the launch lists in profiles/: layer-output path = GEMM launches + abs-max,
        # operand conversion, two code-emission kernels and the finalize per layer; multi-tensor path = table uploads
        # (64 layers each) + the persistent kernel + the finalize; otherwise one scoring kernel per layer
        gemm_launches = 2 if (layer_metric and wl["bits"] == 8) else 1 + F   # 8-bit W+A: the candidates share one launch
        launches_per_step = len(shapes) * (gemm_launches + 5) if layer_metric else (2 + (len(shapes) + 63) // 64 if grans == ("group",) else len(shapes))
        mt = grans == ("group",)
        dom_launches = 1 if mt else len(shapes)      # launches of the dominant kernel per step
        roofline = {"bound": "hbm", "kernel": "kq_score_mt" if mt else "kq_score_rows_stream", "achieved": fp16_bytes / (ms_per_step * 1e-3) / 1e9,
                    "peak": peak, "peak_source": f"of {which}", "unit": "GB/s",
                    "frac": fp16_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
                    "frac_of_nominal_8TBs": fp16_bytes / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                    "launches_per_step": dom_launches, "avg_launch_us": 1e3 * ms_per_step / dom_launches,
                    "algorithmic_bytes_per_launch": fp16_bytes / dom_launches,
                    "traffic": KQ_MT_DRAM_BYTES_PER_ELEMENT * n_elems if mt else None}
        if burst_ms:
            roofline["isolated_step"] = {"ms": burst_ms, "achieved": fp16_bytes / (burst_ms * 1e-3) / 1e9,
                                         "frac": fp16_bytes / (burst_ms * 1e-3) / 1e9 / peak,
                                         "note": "median of 5 steps launched alone after 50 ms idle (no power-cap throttling); context only"}
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "layers": len(shapes), "elements": n_elems, "fp16_GB": fp16_bytes / 1e9,
                       "candidates": list(wl["candidates"]), "granularity": list(grans), "group": wl["group"],
                       "criterion": wl["metric"], "tokens": T, "streaming_synthesis": streaming, "synthesis_ms_per_step": synth_ms,
                       "l2": "inputs larger than L2" if fp16_bytes > 2.5e8 else "inputs fit in L2",
                       "model_select_time_ms": ms_per_step, "emit_winners_ms": emit_ms, "fp_share": fp_share, "min_rel_margin": min_margin},
            "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * launches_per_step, "roofline": roofline,
        }
        if layer_metric:
            gemm_ms = ms_per_step - synth_ms
            tf = flops / (gemm_ms * 1e-3) / 1e12
            p16 = float(peaks.get("bf16_tflops_sustained", 1400.0))
            # One fp16 reference GEMM plus F candidate GEMMs per layer.  In the 8-bit weight-and-activation setting the
            # candidates run on the 8-bit tensor kinds, whose peak is taken as twice the measured 16-bit one (nominal
            # ratio); the peak of the mix is total flop / (time of each part at its own peak).
            native8 = layer_metric and wl["bits"] == 8      # layer-output workloads here quantise weights and activations
            rate = 2.0 if native8 else 1.0
            tpeak = p16 * (1 + F) / (1.0 + F / rate)
            out["roofline"] = {"bound": "tensor", "kernel": "gemm_err_kernel", "achieved": tf, "peak": tpeak,
                               "peak_source": f"of {which}: sustained 16-bit dense {p16:.0f} TFLOP/s for the fp16 reference GEMM, "
                                              f"x{rate:.0f} for the {F} candidate GEMMs, combined by time",
                               "unit": "TFLOP/s", "frac": tf / tpeak, "flops_per_step": flops,
                               "note": "whole step minus synthesis time; includes the operand-preparation kernels", "traffic": None}
        if not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_oracle_sample(args.workload)[0]
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
