"""Seeded synthetic inputs: LLaMA-shaped weight and calibration-activation tensors.

This module holds no quantisation arithmetic.  It serves both the CUDA library's tests/bench and
the CPU oracle's tests.  The synthetic tensors stand in for the LLaMA weights and calibration
activations that the paper analysed; shapes are the public LLaMA linear-layer shapes.

Two back ends with the same recipes:
  * ``*_cpu`` functions: numpy Philox streams -> CPU torch tensors (used where no GPU exists);
  * ``device_*`` functions: a counter-based Philox4x32-10 CUDA generator (``libmofq_synth.so``)
    that fills a caller-provided device tensor, so that a 130 GB model can be produced layer by
    layer.  The two back ends follow the same distributions but not the same bits; a parity test
    always copies the device tensor to the host and feeds the same bits to both sides.

Recipes (kind):
  "gauss_outlier"  N(0, std^2); each element independently replaced with prob. p by N(0, (10 std)^2)
  "student_t"      Student-t(nu=4) scaled to standard deviation `std`, times a per-layer factor
                   2^(2u-1), u ~ U[0,1) drawn from (seed, layer)
  "laplace"        Laplace(0, b); each element independently multiplied by 10 with prob. p
  "activation"     N(0,1); n_ch channels (fixed per (seed, in_features)) times ch_gain; a fraction
                   row_frac of token rows times row_gain
"""
import ctypes as C
import math
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
SYNTH_LIB = os.path.join(_HERE, "libmofq_synth.so")

KIND_GAUSS_OUTLIER, KIND_STUDENT_T, KIND_LAPLACE, KIND_ACTIVATION = range(4)


# ------------------------------------------------------------------------------------------------
# model shapes
# ------------------------------------------------------------------------------------------------
def llama_layers(hidden, mlp, blocks):
    """[(name, out_features, in_features)] for every linear layer of a LLaMA-style decoder stack."""
    per_block = [("q", hidden, hidden), ("k", hidden, hidden), ("v", hidden, hidden), ("o", hidden, hidden),
                 ("gate", mlp, hidden), ("up", mlp, hidden), ("down", hidden, mlp)]
    return [(f"b{b}.{n}", o, i) for b in range(blocks) for (n, o, i) in per_block]


# The five workloads.  `model`: (hidden, mlp, blocks); None for the single-layer case.
WORKLOADS = {
    "single_4096_w4_channel": dict(
        model=None, layers=[("w", 4096, 4096)], seed=0, w_kind="gauss_outlier",
        w_args=dict(std=0.02, p=1e-3), bits=4, candidates=("INT4", "FP4_E2M1"),
        w_gran=("channel",), group=0, metric="tensor", tokens=0),
    "llama7b_w4_group128": dict(
        model=(4096, 11008, 32), seed=1, w_kind="student_t", w_args=dict(std=0.02),
        bits=4, candidates=("INT4", "FP4_E2M1"), w_gran=("group",), group=128, metric="tensor", tokens=0),
    "llama13b_w8a8_layer": dict(
        model=(5120, 13824, 40), seed=2, w_kind="student_t", w_args=dict(std=0.02),
        bits=8, candidates=("INT8", "FP8_E4M3", "FP8_E5M2"), w_gran=("channel",), group=0,
        metric="layer_output", tokens=2048, a_args=dict(n_ch=6, ch_gain=50.0, row_frac=0.01, row_gain=10.0)),
    "llama33b_w4_channel_and_group128": dict(
        model=(6656, 17920, 60), seed=3, w_kind="laplace", w_args=dict(b=0.014, p=5e-4),
        bits=4, candidates=("INT4", "FP4_E2M1"), w_gran=("channel", "group"), group=128, metric="tensor", tokens=0),
    "llama65b_w8a8_layer": dict(
        model=(8192, 22016, 80), seed=4, w_kind="student_t", w_args=dict(std=0.02),
        bits=8, candidates=("INT8", "FP8_E4M3"), w_gran=("channel",), group=0,
        metric="layer_output", tokens=512, a_args=dict(n_ch=8, ch_gain=80.0, row_frac=0.0, row_gain=1.0)),
}


def workload_layers(name, blocks=None):
    w = WORKLOADS[name]
    if w["model"] is None:
        return list(w["layers"])
    hidden, mlp, nb = w["model"]
    return llama_layers(hidden, mlp, nb if blocks is None else blocks)


# ------------------------------------------------------------------------------------------------
# CPU back end (numpy Philox)
# ------------------------------------------------------------------------------------------------
def _rng(seed, layer, tensor_id):
    return np.random.Generator(np.random.Philox(key=[(seed << 20) ^ layer, tensor_id]))


def layer_scale_factor(seed, layer):
    """Per-layer std jitter in [0.5, 2): 2^(2u-1)."""
    u = _rng(seed, layer, 7).random()
    return float(2.0 ** (2.0 * u - 1.0))


def weight_cpu(kind, rows, cols, seed, layer=0, **args):
    """fp16 CPU torch tensor [rows, cols]."""
    g = _rng(seed, layer, 0)
    if kind == "gauss_outlier":
        std, p = args.get("std", 0.02), args.get("p", 1e-3)
        w = g.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)
        mask = g.random((rows, cols), dtype=np.float32) < p
        out = g.standard_normal((rows, cols), dtype=np.float32) * np.float32(10.0 * std)
        w = np.where(mask, out, w)
    elif kind == "student_t":
        std = args.get("std", 0.02)
        f = layer_scale_factor(seed, layer)
        w = g.standard_t(4.0, (rows, cols)).astype(np.float32) * np.float32(std / math.sqrt(2.0) * f)
    elif kind == "laplace":
        b, p = args.get("b", 0.014), args.get("p", 5e-4)
        w = g.laplace(0.0, b, (rows, cols)).astype(np.float32)
        mask = g.random((rows, cols), dtype=np.float32) < p
        w = np.where(mask, w * np.float32(10.0), w)
    else:
        raise ValueError(kind)
    return torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).to(torch.float16)


def outlier_channels(seed, n_in, n_ch):
    """The fixed outlier channel indices for a given input width."""
    g = np.random.Generator(np.random.Philox(key=[seed, 0xC0FFEE ^ n_in]))
    return np.sort(g.choice(n_in, size=min(n_ch, n_in), replace=False))


def activation_cpu(tokens, n_in, seed, layer=0, n_ch=6, ch_gain=50.0, row_frac=0.01, row_gain=10.0):
    """bf16 CPU torch tensor [tokens, n_in]."""
    g = _rng(seed, layer, 1)
    x = g.standard_normal((tokens, n_in), dtype=np.float32)
    x[:, outlier_channels(seed, n_in, n_ch)] *= np.float32(ch_gain)
    if row_frac > 0:
        rows = g.random(tokens) < row_frac
        x[rows, :] *= np.float32(row_gain)
    return torch.from_numpy(x).to(torch.bfloat16)


# ------------------------------------------------------------------------------------------------
# device back end (CUDA Philox generator, its own shared library)
# ------------------------------------------------------------------------------------------------
_synth = None


def _synth_lib():
    global _synth
    if _synth is None:
        if not os.path.exists(SYNTH_LIB):
            raise RuntimeError(f"{SYNTH_LIB} is missing: run `python -c 'import __graft_entry__ as g; g.build()'`")
        L = C.CDLL(SYNTH_LIB)
        L.mofq_synth_fill.restype = C.c_int
        L.mofq_synth_fill.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int,
                                      C.c_uint64, C.c_uint32, C.c_uint32, C.c_float, C.c_float, C.c_float,
                                      C.c_float, C.POINTER(C.c_int32), C.c_int, C.c_void_p]
        _synth = L
    return _synth


def _fill(t, kind, seed, layer, tensor_id, p0, p1, p2, p3, channels=None):
    assert t.is_cuda and t.dim() == 2 and t.stride(1) == 1
    dt = {torch.float16: 0, torch.bfloat16: 1}[t.dtype]
    ch = (C.c_int32 * max(1, len(channels or [])))(*(channels or [0]))
    rc = _synth_lib().mofq_synth_fill(t.data_ptr(), dt, t.shape[0], t.shape[1], t.stride(0), kind,
                                      seed, layer, tensor_id, p0, p1, p2, p3, ch, len(channels or []),
                                      torch.cuda.current_stream(t.device).cuda_stream)
    if rc != 0:
        raise RuntimeError(f"mofq_synth_fill failed with status {rc}")
    return t


def device_weight(out, kind, seed, layer=0, **args):
    """Fill the fp16 CUDA tensor `out` [rows, cols] in place and return it."""
    if kind == "gauss_outlier":
        return _fill(out, KIND_GAUSS_OUTLIER, seed, layer, 0, args.get("std", 0.02), args.get("p", 1e-3), 10.0, 0.0)
    if kind == "student_t":
        f = layer_scale_factor(seed, layer)
        return _fill(out, KIND_STUDENT_T, seed, layer, 0, args.get("std", 0.02) / math.sqrt(2.0) * f, 0.0, 0.0, 0.0)
    if kind == "laplace":
        return _fill(out, KIND_LAPLACE, seed, layer, 0, args.get("b", 0.014), args.get("p", 5e-4), 10.0, 0.0)
    raise ValueError(kind)


def device_activation(out, seed, layer=0, n_ch=6, ch_gain=50.0, row_frac=0.01, row_gain=10.0):
    """Fill the bf16 CUDA tensor `out` [tokens, n_in] in place and return it."""
    ch = [int(c) for c in outlier_channels(seed, out.shape[1], n_ch)]
    return _fill(out, KIND_ACTIVATION, seed, layer, 1, ch_gain, row_frac, row_gain, 0.0, ch)
