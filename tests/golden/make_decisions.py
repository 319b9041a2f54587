#!/usr/bin/env python
"""Writes tests/golden/decisions_<workload>.json: the CPU oracle's errors and per-layer format choices on a stated
sample of each workload's layers.  Calls only ``oracle/`` (and the seeded input generators, which hold none of the
method's arithmetic); nothing here touches the CUDA library.  The GPU test tests/test_gpu_decisions.py rebuilds the
same tensors with the same CPU generators and compares.

Sample:
  * tensor-criterion workloads: every distinct layer shape (attention projection, MLP up, MLP down) in the first,
    a middle and the last decoder block, at full size; the single-layer workload whole;
  * layer-output workloads: the same three layer kinds of the first block with all calibration tokens and the full
    input width, the weight cut to its first 256 output channels (per-channel scales make that a layer in its own
    right; the oracle's double-precision triple loop could not finish a full layer in reasonable time).

    python tests/golden/make_decisions.py [workload ...]
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import api as orc                      # noqa: E402
from paper_2305_12356_b200 import inputs           # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))
LAYER_KINDS = (0, 4, 6)          # q, gate, down inside a decoder block of seven linear layers
TRUNCATED_ROWS = 256
GRAN = {"channel": orc.PER_CHANNEL, "group": orc.PER_GROUP, "tensor": orc.PER_TENSOR}


def sample_layers(name):
    """Global layer indices of the sample."""
    wl = inputs.WORKLOADS[name]
    if wl["model"] is None:
        return [0]
    blocks = wl["model"][2]
    picks = (0,) if wl["metric"] == "layer_output" else (0, blocks // 2, blocks - 1)
    return [b * 7 + k for b in picks for k in LAYER_KINDS]


def build_layer(name, li):
    """The sample's CPU tensors for global layer index li: (W, X or None)."""
    wl = inputs.WORKLOADS[name]
    _, out_f, in_f = inputs.workload_layers(name)[li]
    if wl["metric"] == "layer_output":
        w = inputs.weight_cpu(wl["w_kind"], min(TRUNCATED_ROWS, out_f), in_f, wl["seed"], li, **wl["w_args"])
        x = inputs.activation_cpu(wl["tokens"], in_f, wl["seed"], li, **wl["a_args"])
        return w, x
    return inputs.weight_cpu(wl["w_kind"], out_f, in_f, wl["seed"], li, **wl["w_args"]), None


def score(name, li):
    wl = inputs.WORKLOADS[name]
    w, x = build_layer(name, li)
    cands = [getattr(orc, c) for c in wl["candidates"]]
    rec = {"layer": li, "rows": int(w.shape[0]), "cols": int(w.shape[1]), "sets": []}
    if wl["metric"] == "layer_output":
        out = [orc.layer_output_error(x, w, f, False) for f in cands]
        errs = [o[0] for o in out]
        rec["tokens"] = int(x.shape[0])
        rec["sets"].append({"gran": "channel", "errors": errs, "nsr": [o[1] for o in out], "chosen": int(orc.select(errs))})
    else:
        for g in wl["w_gran"]:
            errs = [orc.tensor_mse(w, f, GRAN[g], wl["group"]) for f in cands]
            rec["sets"].append({"gran": g, "errors": errs, "chosen": int(orc.select(errs))})
    for s in rec["sets"]:
        e = sorted(s["errors"])
        s["rel_margin"] = (e[1] - e[0]) / e[0] if len(e) > 1 and e[0] > 0 else None
    return rec


def main():
    names = sys.argv[1:] or list(inputs.WORKLOADS)
    orc.lib()
    for name in names:
        wl = inputs.WORKLOADS[name]
        doc = {"workload": name, "candidates": list(wl["candidates"]), "criterion": wl["metric"], "group": wl["group"],
               "generator": "paper_2305_12356_b200.inputs.weight_cpu / activation_cpu (numpy Philox)",
               "truncated_rows": TRUNCATED_ROWS if wl["metric"] == "layer_output" else None,
               "layers": [score(name, li) for li in sample_layers(name)]}
        path = os.path.join(HERE, f"decisions_{name}.json")
        with open(path, "w") as f:
            json.dump(doc, f, indent=1)
            f.write("\n")
        print(path, [(r["layer"], [s["chosen"] for s in r["sets"]]) for r in doc["layers"]], flush=True)


if __name__ == "__main__":
    main()
