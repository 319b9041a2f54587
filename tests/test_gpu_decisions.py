"""GPU parity with the oracle's stored decisions on every workload (-m gpu).

tests/golden/decisions_<workload>.json (written by tests/golden/make_decisions.py, which calls only the CPU
oracle) holds, for a stated sample of each workload's layers at full size, every candidate's error and the chosen
format.  Here the same tensors are rebuilt with the same seeded CPU generators, copied to the device and scored
through the C ABI in the configuration the bench times: errors within the stated tolerance, choices exact.
"""
import importlib.util
import json
import os

import pytest
import torch

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import inputs

from gpu_util import rel_err

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
MSE_RTOL = 1e-5
LAYER_RTOL = 1e-2

_spec = importlib.util.spec_from_file_location("make_decisions", os.path.join(HERE, "golden", "make_decisions.py"))
make_decisions = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(make_decisions)


def _golden(name):
    with open(os.path.join(HERE, "golden", f"decisions_{name}.json")) as f:
        return json.load(f)


@pytest.mark.parametrize("name", list(inputs.WORKLOADS))
def test_stored_oracle_decisions(name):
    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    wl = inputs.WORKLOADS[name]
    doc = _golden(name)
    assert doc["candidates"] == list(wl["candidates"]) and doc["criterion"] == wl["metric"]
    assert [r["layer"] for r in doc["layers"]] == make_decisions.sample_layers(name)
    layer_metric = wl["metric"] == "layer_output"
    grans = wl["w_gran"]
    cfg = mofq.make_config(wl["bits"], wl["candidates"], metric=wl["metric"], is_w_only=not layer_metric,
                           w_gran=grans[0], w_group=wl["group"], w_gran2=grans[1] if len(grans) > 1 else None)
    layers = []
    for r in doc["layers"]:
        w, x = make_decisions.build_layer(name, r["layer"])
        assert tuple(w.shape) == (r["rows"], r["cols"])
        layers.append((w.to(dev), x.to(dev)) if layer_metric else w.to(dev))
    recs = mofq.select_formats(layers, cfg)                      # one call over the sampled layers, as the bench makes it
    assert len(recs) == len(doc["layers"]) * len(grans)
    tol = LAYER_RTOL if layer_metric else MSE_RTOL
    for k, r in enumerate(doc["layers"]):
        for s, want in enumerate(r["sets"]):
            got = recs[k * len(grans) + s]
            assert want["gran"] == grans[s]
            assert got["status"] == 0
            assert rel_err(got["errors"], want["errors"]).max() < tol, (name, r["layer"], want["gran"], got, want)
            if layer_metric:
                assert rel_err(got["nsr"], want["nsr"]).max() < tol
            assert got["chosen"] == want["chosen"], (name, r["layer"], want["gran"], got, want)
            assert want["rel_margin"] is None or want["rel_margin"] > 1e-4      # the stored decisions are far from ties
    del layers
    torch.cuda.empty_cache()
