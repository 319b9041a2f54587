"""GPU parity: layer-output error (tcgen05 GEMM path) against the CPU oracle (-m gpu).

Bar: MSE and noise/signal ratio within 1e-2 relative (fp32 tensor-core accumulation of exact
operands against the oracle's double sums); per-layer decisions exact.
"""
import numpy as np
import pytest
import torch

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import binding as B
from paper_2305_12356_b200 import inputs

from gpu_util import host, rel_err

pytestmark = pytest.mark.gpu

LAYER_RTOL = 1e-2


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available()
    mofq.lib()
    return torch.device("cuda:0")


def _layer(dev, T, n_in, n_out, seed, layer=0, xdtype=torch.bfloat16, wdtype=torch.float16, a_args=None):
    w = torch.empty((n_out, n_in), dtype=torch.float16, device=dev)
    inputs.device_weight(w, "student_t", seed, layer)
    x = torch.empty((T, n_in), dtype=torch.bfloat16, device=dev)
    inputs.device_activation(x, seed, layer, **(a_args or {}))
    return w.to(wdtype), x.to(xdtype)


def _oracle(orc, w, x, names, w_only):
    out = [orc.layer_output_error(host(x), host(w), getattr(orc, n), w_only) for n in names]
    return [o[0] for o in out], [o[1] for o in out]


@pytest.mark.parametrize("T,n_in,n_out", [(128, 256, 128), (256, 512, 384), (200, 264, 328), (130, 1152, 330), (512, 2048, 256)])
@pytest.mark.parametrize("names,w_only,bits", [(["INT8", "FP8_E4M3", "FP8_E5M2"], False, 8), (["INT8", "FP8_E4M3"], True, 8),
                                               (["INT4", "FP4_E2M1"], True, 4)])
def test_layer_output_error_matches_oracle(orc, dev, T, n_in, n_out, names, w_only, bits):
    w, x = _layer(dev, T, n_in, n_out, seed=51, layer=T % 7)
    cfg = mofq.make_config(bits, names, metric="layer_output", is_w_only=w_only, w_gran="channel", a_gran="tensor")
    mse, nsr, st = mofq.layer_output_error(x, w, cfg)
    torch.cuda.synchronize()
    want_mse, want_nsr = _oracle(orc, w, x, names, w_only)
    assert int(st.item()) == 0
    assert rel_err(mse.cpu().numpy(), want_mse).max() < LAYER_RTOL, (mse, want_mse)
    assert rel_err(nsr.cpu().numpy(), want_nsr).max() < LAYER_RTOL, (nsr, want_nsr)


@pytest.mark.parametrize("names", [["FP8_E5M2", "INT8"], ["FP8_E4M3", "FP8_E5M2", "INT8"], ["FP8_E5M2", "FP8_E4M3"], ["FP8_E4M3"],
                                   ["INT8", "FP8_E4M3", "INT8"], ["FP8_E5M2", "FP8_E5M2"]])
def test_candidate_order_and_repeats_in_the_8bit_setting(orc, dev, names):
    """The code-emission kernels take the formats in a fixed class order and exist for distinct classes only: any
    caller's order, and a list that repeats a format, must still give each candidate its own error."""
    T, n_in, n_out = 256, 512, 384
    w, x = _layer(dev, T, n_in, n_out, seed=57, layer=3)
    cfg = mofq.make_config(8, names, metric="layer_output", is_w_only=False, w_gran="channel", a_gran="tensor")
    mse, nsr, st = mofq.layer_output_error(x, w, cfg)
    torch.cuda.synchronize()
    want_mse, want_nsr = _oracle(orc, w, x, names, False)
    assert int(st.item()) == 0
    assert rel_err(mse.cpu().numpy(), want_mse).max() < LAYER_RTOL, (mse, want_mse)
    assert rel_err(nsr.cpu().numpy(), want_nsr).max() < LAYER_RTOL, (nsr, want_nsr)
    res = mofq.select_formats([(w, x)], cfg)
    assert res[0]["chosen"] == int(np.argmin(want_mse)) and res[0]["status"] == 0      # (first minimum: strict '<')


@pytest.mark.parametrize("T,n_in,n_out", [(512, 1024, 8192), (256, 22016, 512)])
def test_dense_outlier_activations_paired_tiles_and_full_depth(orc, dev, T, n_in, n_out):
    """Dense calibration activations with outlier channels (the 65B-shaped workload's recipe) at sizes whose cost
    model picks the two-CTA 256 x 256 tile (512 x 8192 outputs) and at the workload's deepest contraction
    (22016 input features): every output is a long accumulation of real products, unlike the one-hot cases."""
    a_args = dict(n_ch=8, ch_gain=80.0, row_frac=0.0, row_gain=1.0)
    w, x = _layer(dev, T, n_in, n_out, seed=56, layer=3, a_args=a_args)
    names = ["INT8", "FP8_E4M3"]
    cfg = mofq.make_config(8, names, metric="layer_output", is_w_only=False, w_gran="channel", a_gran="tensor")
    rec = mofq.select_formats([(w, x)], cfg)[0]
    want_mse, want_nsr = _oracle(orc, w, x, names, False)
    assert rec["status"] == 0
    assert rel_err(rec["errors"], want_mse).max() < LAYER_RTOL, (rec, want_mse)
    assert rel_err(rec["nsr"], want_nsr).max() < LAYER_RTOL, (rec, want_nsr)
    assert rec["chosen"] == orc.select(want_mse)
    assert rec["chosen"] == 1                       # activation outliers: the floating-point grid wins (Section 3.2)


def test_wide_tile_variant(orc, dev):
    # 2 x 74 tiles of 128 x 256 fill 148 SMs in one wave, so the 256-wide tile is chosen; the right edge is ragged
    T, n_in, n_out = 256, 128, 18936
    w, x = _layer(dev, T, n_in, n_out, seed=55)
    for names, w_only, bits in ((["INT8", "FP8_E4M3"], False, 8), (["INT4", "FP4_E2M1"], True, 4)):
        cfg = mofq.make_config(bits, names, metric="layer_output", is_w_only=w_only)
        mse, nsr, st = mofq.layer_output_error(x, w, cfg)
        want_mse, want_nsr = _oracle(orc, w, x, names, w_only)
        assert int(st.item()) == 0
        assert rel_err(mse.cpu().numpy(), want_mse).max() < LAYER_RTOL
        assert rel_err(nsr.cpu().numpy(), want_nsr).max() < LAYER_RTOL


@pytest.mark.parametrize("xdtype,wdtype", [(torch.float16, torch.float16), (torch.bfloat16, torch.bfloat16)])
def test_layer_output_error_dtype_combinations(orc, dev, xdtype, wdtype):
    w, x = _layer(dev, 256, 512, 256, seed=52, xdtype=xdtype, wdtype=wdtype, a_args=dict(ch_gain=8.0))
    names = ["INT8", "FP8_E4M3"]
    cfg = mofq.make_config(8, names, metric="layer_output", is_w_only=False)
    mse, nsr, _ = mofq.layer_output_error(x, w, cfg)
    want_mse, want_nsr = _oracle(orc, w, x, names, False)
    assert rel_err(mse.cpu().numpy(), want_mse).max() < LAYER_RTOL
    assert rel_err(nsr.cpu().numpy(), want_nsr).max() < LAYER_RTOL


def test_identity_activations_reduce_to_tensor_error(orc, dev):
    # X = I, weights only: the layer-output error times T*out is the tensor SSE of W
    n_in, n_out = 256, 128
    w = torch.empty((n_out, n_in), dtype=torch.float16, device=dev)
    inputs.device_weight(w, "gauss_outlier", 0, 0)
    x = torch.eye(n_in, dtype=torch.bfloat16, device=dev)
    cfg = mofq.make_config(4, ["INT4", "FP4_E2M1"], metric="layer_output", is_w_only=True)
    mse, _, _ = mofq.layer_output_error(x, w, cfg)
    want = [orc.quantize(host(w), f, orc.PER_CHANNEL)["sse"] / (n_in * n_out) for f in (orc.INT4, orc.FP4_E2M1)]
    assert rel_err(mse.cpu().numpy(), want).max() < 1e-4


def test_select_formats_layer_metric(orc, dev):
    shapes = [(256, 512, 256), (128, 384, 640), (384, 256, 128)]
    layers = [_layer(dev, T, i, o, seed=53, layer=l) for l, (T, i, o) in enumerate(shapes)]
    names = ["INT8", "FP8_E4M3", "FP8_E5M2"]
    cfg = mofq.make_config(8, names, metric="layer_output", is_w_only=False)
    recs = mofq.select_formats(layers, cfg)
    again = mofq.select_formats(layers, cfg)
    assert recs == again
    for (w, x), r in zip(layers, recs):
        want_mse, want_nsr = _oracle(orc, w, x, names, False)
        assert r["status"] == 0
        assert rel_err(r["errors"], want_mse).max() < LAYER_RTOL
        assert rel_err(r["nsr"], want_nsr).max() < LAYER_RTOL
        assert r["chosen"] == orc.select(want_mse)
    zero = (torch.zeros(128, 256, dtype=torch.float16, device=dev), layers[0][1][:, :256].contiguous())
    r = mofq.select_formats([zero], cfg)[0]
    assert r["chosen"] == 0 and r["errors"] == [0.0, 0.0, 0.0]


def test_layer_metric_rejects_unsupported_granularities(dev):
    w, x = _layer(dev, 128, 256, 128, seed=54)
    cfg = mofq.make_config(8, ["INT8"], metric="layer_output", is_w_only=False, w_gran="group", w_group=128)
    with pytest.raises(B.MofqError):
        mofq.layer_output_error(x, w, cfg)
