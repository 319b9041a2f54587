"""Pins for the oracle's layer-output error (CPU only): Y = X W^T with quantised inputs.

The tensor quantiser is pinned in test_oracle_quantize.py; here the contraction, its orientation,
the W-only / WA switch and the two normalisations (MSE, noise/signal ratio) are fixed against
library matmuls, exact integer arithmetic and special cases that collapse to the tensor error.
"""
import numpy as np
import pytest
import torch

from paper_2305_12356_b200 import inputs


def _f64(x):
    return x.to(torch.float64).numpy()


def _dq(orc, x, fmt, gran, group=0):
    q = orc.quantize(x, fmt, gran, group)
    rows, cols = q["codes"].shape
    s = q["scales"].astype(np.float64)
    if gran == orc.PER_CHANNEL:
        s = s[:, None]
    elif gran == orc.PER_GROUP:
        s = np.repeat(s.reshape(rows, cols // group), group, axis=1)
    return orc.decode_table(fmt)[q["codes"]] * s, q


@pytest.mark.parametrize("name", ["INT8", "FP8_E4M3", "FP8_E5M2", "INT4", "FP4_E2M1"])
@pytest.mark.parametrize("w_only", [True, False])
def test_against_library_matmul(orc, name, w_only):
    fmt = getattr(orc, name)
    T, n_in, out = 24, 256, 40                                   # three different extents: a transposed operand cannot pass
    W = inputs.weight_cpu("student_t", out, n_in, seed=2, layer=1)
    X = inputs.activation_cpu(T, n_in, seed=2, layer=1)
    Wq, _ = _dq(orc, W, fmt, orc.PER_CHANNEL)
    Xq = _dq(orc, X, fmt, orc.PER_TENSOR)[0] if not w_only else _f64(X)
    Y = _f64(X) @ _f64(W).T
    Yq = Xq @ Wq.T
    mse, nsr = orc.layer_output_error(X, W, fmt, w_only)
    assert mse == pytest.approx(np.mean((Y - Yq) ** 2), rel=1e-10)
    assert nsr == pytest.approx(np.sum((Y - Yq) ** 2) / np.sum(Y ** 2), rel=1e-10)
    assert Y.shape == (T, out)


def test_group_scales_for_weights(orc):
    T, n_in, out = 8, 256, 12
    W = inputs.weight_cpu("laplace", out, n_in, seed=3, layer=0)
    X = inputs.activation_cpu(T, n_in, seed=3, layer=0)
    Wq, _ = _dq(orc, W, orc.INT4, orc.PER_GROUP, 128)
    Y, Yq = _f64(X) @ _f64(W).T, _f64(X) @ Wq.T
    mse, _ = orc.layer_output_error(X, W, orc.INT4, True, w_gran=orc.PER_GROUP, w_group=128)
    assert mse == pytest.approx(np.mean((Y - Yq) ** 2), rel=1e-10)


@pytest.mark.parametrize("name", ["INT4", "FP4_E2M1", "INT8", "FP8_E4M3"])
def test_identity_activations_reduce_to_tensor_error(orc, name):
    # X = I (T = in), weights only: Y - Yq = (W - Wq)^T, so mse * T * out = tensor SSE of W.
    fmt = getattr(orc, name)
    n_in, out = 128, 20
    W = inputs.weight_cpu("gauss_outlier", out, n_in, seed=0, layer=0)
    X = torch.eye(n_in, dtype=torch.bfloat16)
    mse, nsr = orc.layer_output_error(X, W, fmt, True)
    sse = orc.quantize(W, fmt, orc.PER_CHANNEL)["sse"]
    assert mse * n_in * out == pytest.approx(sse, rel=1e-12)
    assert nsr == pytest.approx(sse / np.sum(_f64(W) ** 2), rel=1e-12)


@pytest.mark.parametrize("name", ["INT8", "FP8_E4M3"])
def test_activations_on_grid_reduce_to_weight_only(orc, name):
    fmt = getattr(orc, name)
    T, n_in, out = 16, 128, 24
    tab = orc.decode_table(fmt)
    vals = tab[~np.isnan(tab)]
    vals = vals[np.abs(vals) <= orc.format_max(fmt)]
    if name == "FP8_E4M3":
        vals = vals[np.abs(vals) >= 2.0 ** -6]                   # keep them exactly representable in bf16 after scaling
    g = np.random.default_rng(5)
    X = torch.from_numpy(g.choice(vals, (T, n_in)) * 2.0 ** -4).to(torch.bfloat16)
    X[0, 0] = orc.format_max(fmt) * 2.0 ** -4
    assert orc.tensor_mse(X, fmt, orc.PER_TENSOR) == 0.0
    W = inputs.weight_cpu("student_t", out, n_in, seed=2, layer=5)
    wa = orc.layer_output_error(X, W, fmt, False)
    wo = orc.layer_output_error(X, W, fmt, True)
    assert wa[0] == pytest.approx(wo[0], rel=1e-12) and wa[1] == pytest.approx(wo[1], rel=1e-12)


def test_int8_product_is_exact_integer(orc):
    # For INT8 the quantised output is s_x * s_w[o] * (Cx Cw^T) with an exact integer matrix product.
    T, n_in, out = 20, 384, 28
    W = inputs.weight_cpu("student_t", out, n_in, seed=2, layer=9)
    X = inputs.activation_cpu(T, n_in, seed=2, layer=9)
    qw, qx = orc.quantize(W, orc.INT8, orc.PER_CHANNEL), orc.quantize(X, orc.INT8, orc.PER_TENSOR)
    cw = qw["codes"].view(np.int8).astype(np.int64)
    cx = qx["codes"].view(np.int8).astype(np.int64)
    P = cx @ cw.T                                                # int64, exact
    Yq = P.astype(np.float64) * float(qx["scales"][0]) * qw["scales"].astype(np.float64)[None, :]
    Y = _f64(X) @ _f64(W).T
    mse, nsr = orc.layer_output_error(X, W, orc.INT8, False)
    assert mse == pytest.approx(np.mean((Y - Yq) ** 2), rel=1e-9)


def test_zero_weights_and_selection_over_layers(orc):
    T, n_in, out = 8, 128, 8
    X = inputs.activation_cpu(T, n_in, seed=4, layer=0)
    Wz = torch.zeros(out, n_in, dtype=torch.float16)
    assert orc.layer_output_error(X, Wz, orc.INT8, False) == (0.0, 0.0)
    W = inputs.weight_cpu("student_t", out, n_in, seed=4, layer=0)
    res = orc.mofq_select([(Wz, X), (W, X)], [orc.INT8, orc.FP8_E4M3], metric="layer_output", is_w_only=False)
    assert res[0]["chosen"] == 0                                 # tie at zero error -> first candidate
    e = res[1]["errors"]
    assert res[1]["chosen"] == (0 if e[0] <= e[1] else 1)


def test_outlier_activations_favour_fp8_at_the_layer_output(orc):
    # Section 3.2, layer analysis (W8A8): with activation outliers FP8 gives the lower output error in most layers.
    T, n_in, out = 64, 512, 64
    wins = 0
    for layer in range(4):
        W = inputs.weight_cpu("student_t", out, n_in, seed=2, layer=layer)
        X = inputs.activation_cpu(T, n_in, seed=2, layer=layer)
        e_int = orc.layer_output_error(X, W, orc.INT8, False)[0]
        e_fp = orc.layer_output_error(X, W, orc.FP8_E4M3, False)[0]
        wins += e_fp < e_int
    assert wins >= 3
