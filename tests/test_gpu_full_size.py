"""GPU parity at the workloads' full layer sizes, in the launch configuration that bench.py times (-m gpu).

The oracle cannot score a whole model in seconds, so: the whole model is scored on the GPU in one call and
sampled layers are compared with the oracle; properties that hold at any size cover the rest (status clean,
reruns bit-identical, one-hot activations reduce the layer-output error to a column-sampled tensor error).
"""
import numpy as np
import pytest
import torch

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import inputs

from gpu_util import host, rel_err

pytestmark = pytest.mark.gpu

MSE_RTOL = 1e-5
LAYER_RTOL = 1e-2


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available()
    mofq.lib()
    return torch.device("cuda:0")


def _build(dev, name, blocks=None):
    wl = inputs.WORKLOADS[name]
    layers = []
    for li, (_, o, i) in enumerate(inputs.workload_layers(name, blocks)):
        w = torch.empty((o, i), dtype=torch.float16, device=dev)
        layers.append(inputs.device_weight(w, wl["w_kind"], wl["seed"], li, **wl["w_args"]))
    return wl, layers


def test_llama7b_group128_whole_model_sampled_layers(orc, dev):
    wl, layers = _build(dev, "llama7b_w4_group128")                       # all 224 layers, 12.95 GB, one persistent launch
    cfg = mofq.make_config(4, wl["candidates"], w_gran="group", w_group=128)
    prepared = mofq.prepare_layers(layers)
    recs = mofq.select_formats(prepared, cfg)
    again = mofq.select_formats(prepared, cfg)
    assert recs == again and len(recs) == 224
    assert all(r["status"] == 0 and r["chosen"] in (0, 1) and r["rel_margin"] > 1e-4 for r in recs)
    cands = [getattr(orc, c) for c in wl["candidates"]]
    for li in (0, 4, 6, 117, 223):                                         # q, gate, down, mid-model, last
        want = [orc.tensor_mse(host(layers[li]), f, orc.PER_GROUP, 128) for f in cands]
        assert rel_err(recs[li]["errors"], want).max() < MSE_RTOL, (li, recs[li], want)
        assert recs[li]["chosen"] == orc.select(want)
    del layers, prepared
    torch.cuda.empty_cache()


def test_llama33b_channel_and_group_full_size_layers(orc, dev):
    wl, layers = _build(dev, "llama33b_w4_channel_and_group128", blocks=1)   # the 7 layer shapes at full size
    cfg = mofq.make_config(4, wl["candidates"], w_gran="channel", w_group=128, w_gran2="group")
    recs = mofq.select_formats(layers, cfg)
    assert len(recs) == 14 and all(r["status"] == 0 for r in recs)
    cands = [getattr(orc, c) for c in wl["candidates"]]
    for li in (0, 4):                                                      # 6656 x 6656 and 17920 x 6656
        wh = host(layers[li])
        for s, (g, grp) in enumerate(((orc.PER_CHANNEL, 0), (orc.PER_GROUP, 128))):
            want = [orc.tensor_mse(wh, f, g, grp) for f in cands]
            r = recs[2 * li + s]
            assert rel_err(r["errors"], want).max() < MSE_RTOL, (li, s, r, want)
            assert r["chosen"] == orc.select(want)
    del layers
    torch.cuda.empty_cache()


def test_mixed_winners_at_full_layer_shapes(orc, dev):
    """Decisions that can go either way, at the workloads' layer shapes: flat-distributed layers (the INT grid wins)
    between heavy-tailed ones (the FP grid wins), scored in one call under per-channel and group-128 scales."""
    g = torch.Generator().manual_seed(91)
    layers = []
    for li, (o, i, kind) in enumerate([(4096, 4096, "flat"), (11008, 4096, "student_t"), (4096, 11008, "flat"), (6656, 6656, "laplace")]):
        if kind == "flat":
            w = ((torch.rand((o, i), generator=g) - 0.5) * 0.1).to(torch.float16).to(dev)
        else:
            w = inputs.device_weight(torch.empty((o, i), dtype=torch.float16, device=dev), kind, 92, li)
        layers.append(w)
    names = ["INT4", "FP4_E2M1"]
    cands = [orc.INT4, orc.FP4_E2M1]
    cfg = mofq.make_config(4, names, w_gran="channel", w_group=128, w_gran2="group")
    recs = mofq.select_formats(layers, cfg)
    only_group = mofq.select_formats(layers, mofq.make_config(4, names, w_gran="group", w_group=128))   # the multi-tensor kernel
    winners = set()
    for li, w in enumerate(layers):
        wh = host(w)
        for s, (gr, grp) in enumerate(((orc.PER_CHANNEL, 0), (orc.PER_GROUP, 128))):
            want = [orc.tensor_mse(wh, f, gr, grp) for f in cands]
            r = recs[2 * li + s]
            assert r["status"] == 0
            assert rel_err(r["errors"], want).max() < MSE_RTOL, (li, s, r, want)
            assert r["chosen"] == orc.select(want), (li, s, r, want)
            winners.add(r["chosen"])
            if s == 1:
                assert rel_err(only_group[li]["errors"], want).max() < MSE_RTOL
                assert only_group[li]["chosen"] == r["chosen"]
    assert winners == {0, 1}, "the fixture is meant to produce both winners"
    del layers
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name,layer_index", [("llama65b_w8a8_layer", 6), ("llama13b_w8a8_layer", 4)])
def test_layer_output_full_size_one_hot_activations(orc, dev, name, layer_index):
    """X = T one-hot rows: Y[t,:] is column c_t of W, and (the value 1 being exact in every format) the quantised
    output is the same column of dq(W); so the layer-output error equals the tensor error of W restricted to the
    chosen columns, which the oracle's per-channel quantiser gives directly at full size."""
    wl = inputs.WORKLOADS[name]
    _, n_out, n_in = inputs.workload_layers(name)[layer_index]
    T = wl["tokens"]
    w = torch.empty((n_out, n_in), dtype=torch.float16, device=dev)
    inputs.device_weight(w, wl["w_kind"], wl["seed"], layer_index, **wl["w_args"])
    g = torch.Generator().manual_seed(7)
    cols = torch.randperm(n_in, generator=g)[:T]
    x = torch.zeros((T, n_in), dtype=torch.bfloat16, device=dev)
    x[torch.arange(T), cols.to(dev)] = 1.0
    cfg = mofq.make_config(8, wl["candidates"], metric="layer_output", is_w_only=False)
    rec = mofq.select_formats([(w, x)], cfg)[0]
    assert rec["status"] == 0
    wh = host(w)
    wsel = wh[:, cols].to(torch.float64).numpy()
    want_mse, want_nsr = [], []
    for c in wl["candidates"]:
        q = orc.quantize(wh, getattr(orc, c), orc.PER_CHANNEL)
        dq = orc.decode_table(getattr(orc, c))[q["codes"][:, cols.numpy()]] * q["scales"].astype(np.float64)[:, None]
        noise = float(((wsel - dq) ** 2).sum())
        want_mse.append(noise / (T * n_out))
        want_nsr.append(noise / float((wsel ** 2).sum()))
    assert rel_err(rec["errors"], want_mse).max() < LAYER_RTOL, (rec, want_mse)
    assert rel_err(rec["nsr"], want_nsr).max() < LAYER_RTOL
    assert rec["chosen"] == orc.select(want_mse)
    del w, x
    torch.cuda.empty_cache()


def test_large_single_tensor_group_scales_takes_the_streaming_route(orc, dev):
    """A dense tensor of >= 32 Mi elements with group scales is scored by the multi-tensor kernel as a one-layer list."""
    w = torch.empty((11008, 4096), dtype=torch.float16, device=dev)       # 45 M elements, a LLaMA-7B gate projection
    inputs.device_weight(w, "student_t", 5, 1)
    names = ["FP4_E2M1", "INT4"]
    got, st = mofq.tensor_error(w, names, "group", group=128)
    want = [orc.tensor_mse(host(w), getattr(orc, n), orc.PER_GROUP, 128) for n in names]
    assert int(st.item()) == 0
    assert rel_err(got.cpu().numpy(), want).max() < MSE_RTOL
    again, _ = mofq.tensor_error(w, names, "group", group=128)
    assert torch.equal(got, again)                                         # fixed summation order
    w[7000, 123] = float("inf")
    _, st = mofq.tensor_error(w, names, "group", group=128)
    assert int(st.item()) & mofq.binding.STATUS_NONFINITE_INPUT


def test_tensor_beyond_2_to_31_elements_splits_consistently(dev):
    """Index arithmetic past 2^31 elements: a 65536 x 65536 tensor (8.6 GB) scored whole equals its halves combined."""
    w = torch.empty((65536, 65536), dtype=torch.float16, device=dev)
    for q in range(4):                                                     # four seeded quarters (the generator is per call)
        inputs.device_weight(w[q * 16384:(q + 1) * 16384], "student_t", 9, q)
    names = ["INT4", "FP4_E2M1"]
    for gran, group in (("group", 128), ("channel", 0)):
        whole, st = mofq.tensor_error(w, names, gran, group=group)
        top, _ = mofq.tensor_error(w[:32768], names, gran, group=group)
        bot, _ = mofq.tensor_error(w[32768:], names, gran, group=group)
        assert int(st.item()) == 0
        both = (top.double() + bot.double()) / 2
        assert rel_err(whole.cpu().numpy(), both.cpu().numpy()).max() < MSE_RTOL, (gran, whole, both)
    got = mofq.quantize_tensor(w, "FP4_E2M1", "group", 128, want_scales=True)
    part = mofq.quantize_tensor(w[65000:], "FP4_E2M1", "group", 128)       # the tail rows, quantised on their own
    n_tail = (65536 - 65000) * 65536
    assert torch.equal(got["codes"][-n_tail // 2:], part["codes"])
    assert torch.equal(got["scales"][-n_tail // 128:], part["scales"])
    del w, got, part
    torch.cuda.empty_cache()
