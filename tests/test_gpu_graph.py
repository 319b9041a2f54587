"""The device entry points only enqueue work on the caller's stream (kernels, memsets; no allocation, no
synchronisation), so a call can be captured into a CUDA graph and replayed (-m gpu).

Each case captures one call, replays the graph on fresh inputs written into the same buffers, and compares the
replay's records bit for bit with a plain call on those inputs.
"""
import pytest
import torch

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import binding as B
from paper_2305_12356_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available()
    mofq.lib()
    return torch.device("cuda:0")


def _weights(dev, shapes, seed):
    out = []
    for i, (o, k) in enumerate(shapes):
        w = torch.empty((o, k), dtype=torch.float16, device=dev)
        inputs.device_weight(w, "student_t", seed, i)
        out.append(w)
    return out


CASES = {
    # one tensor, per-channel scales: header-clear kernel + chained scoring launch
    "single_rows": dict(shapes=[(512, 1024)], cfg=dict(bit_width=4, candidates=["INT4", "FP4_E2M1"], w_gran="channel")),
    # layer list, per-channel and group-128 scales: table uploads + persistent launch + finalize
    "rows_list": dict(shapes=[(256, 1024), (384, 512), (128, 2048)],
                      cfg=dict(bit_width=4, candidates=["INT4", "FP4_E2M1"], w_gran="channel", w_group=128, w_gran2="group")),
    # layer list, group-128 scales: the group kernel
    "group_list": dict(shapes=[(256, 1024), (384, 512)], cfg=dict(bit_width=4, candidates=["FP4_E2M1", "INT4"], w_gran="group", w_group=128)),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_tensor_metric_call_replays_from_a_graph(dev, case):
    spec = CASES[case]
    cfg = mofq.make_config(**spec["cfg"])
    layers = _weights(dev, spec["shapes"], 71)
    prep = mofq.prepare_layers(layers)
    n_rec = len(layers) * (2 if spec["cfg"].get("w_gran2") else 1)
    ws = torch.empty(mofq.workspace_bytes(prep, cfg), dtype=torch.uint8, device=dev)
    res = torch.zeros(n_rec * B.RESULT_BYTES, dtype=torch.uint8, device=dev)
    mofq.select_formats(prep, cfg, workspace=ws, results=res, parse=False)       # warm-up outside the capture (function attributes)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        mofq.select_formats(prep, cfg, workspace=ws, results=res, parse=False)
    for seed in (72, 73):
        for w, fresh in zip(layers, _weights(dev, spec["shapes"], seed)):
            w.copy_(fresh)
        res.zero_()
        graph.replay()
        torch.cuda.synchronize()
        replayed = bytes(res.cpu().numpy())
        plain = mofq.select_formats(prep, cfg, parse=False)
        torch.cuda.synchronize()
        assert replayed == bytes(plain.cpu().numpy())
        recs = B._parse_results(replayed, n_rec, cfg.n_candidates)
        assert all(r["status"] == 0 and r["errors"][0] > 0 for r in recs)


def test_layer_metric_call_replays_from_a_graph(dev):
    T, n_in, n_out = 256, 512, 384
    w = _weights(dev, [(n_out, n_in)], 74)[0]
    x = torch.empty((T, n_in), dtype=torch.bfloat16, device=dev)
    inputs.device_activation(x, 74, 0)
    cfg = mofq.make_config(8, ["INT8", "FP8_E4M3", "FP8_E5M2"], metric="layer_output", is_w_only=False, w_gran="channel", a_gran="tensor")
    prep = mofq.prepare_layers([(w, x)])
    ws = torch.empty(mofq.workspace_bytes(prep, cfg), dtype=torch.uint8, device=dev)
    res = torch.zeros(B.RESULT_BYTES, dtype=torch.uint8, device=dev)
    mofq.select_formats(prep, cfg, workspace=ws, results=res, parse=False)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        mofq.select_formats(prep, cfg, workspace=ws, results=res, parse=False)
    inputs.device_activation(x, 75, 0)
    w.copy_(_weights(dev, [(n_out, n_in)], 75)[0])
    res.zero_()
    graph.replay()
    torch.cuda.synchronize()
    replayed = bytes(res.cpu().numpy())
    plain = mofq.select_formats(prep, cfg, parse=False)
    torch.cuda.synchronize()
    assert replayed == bytes(plain.cpu().numpy())
    assert B._parse_results(replayed, 1, 3)[0]["status"] == 0
