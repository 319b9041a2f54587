"""GPU parity: quantise / score kernels against the CPU oracle, element by element (-m gpu).

Bars: codes, scales, dequantised values and per-layer decisions bit-exact; MSE within 1e-5
relative (the kernels accumulate squared errors in binary32 chains of at most 128 terms and sum
those in double; the oracle sums in double).
"""
import numpy as np
import pytest
import torch

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import binding as B
from paper_2305_12356_b200 import inputs

from gpu_util import host, orc_gran, rel_err, unpack_codes

pytestmark = pytest.mark.gpu

MSE_RTOL = 1e-5
FMT4 = ["INT4", "FP4_E2M1", "FP4_E2M1_IEEE"]
FMT8 = ["INT8", "FP8_E4M3", "FP8_E5M2"]


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    mofq.lib()
    return torch.device("cuda:0")


def _weights(dev, rows, cols, kind="student_t", seed=1, layer=0, dtype=torch.float16, **kw):
    w = torch.empty((rows, cols), dtype=torch.float16, device=dev)
    inputs.device_weight(w, kind, seed, layer, **kw)
    if dtype == torch.bfloat16:
        w = (w.float() * 3.0).to(torch.bfloat16)
    return w


def _check_quantize(orc, x, name, gran, group=0, scales_in=None):
    fmt_o = getattr(orc, name)
    bits = orc.format_bits(fmt_o)
    got = mofq.quantize_tensor(x, name, gran, group, scales_in=scales_in, want_dequant=True)
    torch.cuda.synchronize()
    xh = host(x)
    want = orc.quantize(xh, fmt_o, orc_gran(orc, gran), group,
                        scales_in=None if scales_in is None else scales_in.cpu().numpy(), want_dequant=True)
    n = x.numel()
    np.testing.assert_array_equal(unpack_codes(got["codes"], bits, n), want["codes"].reshape(-1))
    np.testing.assert_array_equal(got["scales"].cpu().numpy().view(np.uint32), want["scales"].view(np.uint32))
    deq = got["dequant"].cpu().view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(deq, want["dequant"])
    assert int(got["status"].item()) == 0
    return got, want


# ---- quantize: every format x granularity x dtype, several tiles and a ragged tail ------------------------
@pytest.mark.parametrize("name", FMT4 + FMT8)
@pytest.mark.parametrize("gran,group", [("channel", 0), ("group", 128), ("group", 32), ("tensor", 0)])
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_quantize_matches_oracle(orc, dev, name, gran, group, dtype):
    x = _weights(dev, 301, 1152, seed=11, layer=3, dtype=dtype)      # 301 rows: ragged against every tile shape
    _check_quantize(orc, x, name, gran, group)


@pytest.mark.parametrize("name", ["INT4", "FP4_E2M1", "INT8", "FP8_E4M3", "FP8_E5M2"])
def test_quantize_every_finite_fp16_pattern(orc, dev, name):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    bits = bits[(bits & 0x7C00) != 0x7C00]                            # drop Inf/NaN
    pad = (-bits.size) % 1024
    bits = np.concatenate([bits, np.zeros(pad, np.uint16)])
    x = torch.from_numpy(bits.view(np.int16).copy()).view(torch.float16).reshape(-1, 1024).to(dev)
    for gran, group in (("channel", 0), ("group", 128), ("group", 8), ("tensor", 0)):
        _check_quantize(orc, x, name, gran, group)


@pytest.mark.parametrize("name", ["INT8", "FP8_E4M3", "FP8_E5M2"])
def test_quantize_every_finite_bf16_pattern_in_range(orc, dev, name):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    e = (bits >> 7) & 0xFF
    bits = bits[(e >= 100) & (e <= 140) | (e == 0) & ((bits & 0x7F) == 0)]   # 2^-27 .. 2^13 and +-0
    pad = (-bits.size) % 512
    bits = np.concatenate([bits, np.zeros(pad, np.uint16)])
    x = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).reshape(-1, 512).to(dev)
    for gran, group in (("channel", 0), ("group", 64), ("tensor", 0)):
        _check_quantize(orc, x, name, gran, group)


@pytest.mark.parametrize("name", FMT4 + FMT8)
def test_quantize_with_supplied_scales_saturates(orc, dev, name):
    x = _weights(dev, 40, 512, seed=12, layer=1)
    for gran, group in (("tensor", 0), ("channel", 0), ("group", 128)):
        ns = B.n_scales(gran, 40, 512, group)
        g = torch.Generator().manual_seed(3)
        scales = (torch.rand(ns, generator=g) * 0.004 + 0.0005).to(dev)      # small scales: many values clip
        _check_quantize(orc, x, name, gran, group, scales_in=scales)


def test_quantize_zero_rows_and_tiny_shapes(orc, dev):
    x = _weights(dev, 9, 256, seed=13)
    x[2].zero_()
    x[5, :128].zero_()
    x[7, 3] = -0.0
    for name in ("INT4", "FP4_E2M1", "INT8", "FP8_E4M3"):
        for gran, group in (("channel", 0), ("group", 128), ("tensor", 0)):
            _check_quantize(orc, x, name, gran, group)
    one = _weights(dev, 1, 8, seed=14)
    for gran, group in (("channel", 0), ("group", 8), ("tensor", 0)):
        _check_quantize(orc, one, "FP4_E2M1", gran, group)
    z = torch.zeros(4, 128, dtype=torch.float16, device=dev)
    got, _ = _check_quantize(orc, z, "INT4", "tensor")
    assert float(got["scales"][0]) == 1.0


def test_quantize_strided_input(orc, dev):
    full = _weights(dev, 64, 1024, seed=15)
    view = full[:, 256:768]                                                   # ld = 1024, cols = 512
    got = mofq.quantize_tensor(view, "FP4_E2M1", "group", 128)
    want = orc.quantize(host(view).contiguous(), orc.FP4_E2M1, orc.PER_GROUP, 128)
    np.testing.assert_array_equal(unpack_codes(got["codes"], 4, view.numel()), want["codes"].reshape(-1))
    np.testing.assert_array_equal(got["scales"].cpu().numpy(), want["scales"])


def test_nonfinite_input_sets_status(dev):
    x = _weights(dev, 16, 256, seed=16)
    x[3, 7] = float("inf")
    for gran, group in (("channel", 0), ("group", 128), ("tensor", 0)):
        got = mofq.quantize_tensor(x, "INT4", gran, group)
        assert int(got["status"].item()) & B.STATUS_NONFINITE_INPUT
        _, st = mofq.tensor_error(x, ["INT4", "FP4_E2M1"], gran, group=group)
        assert int(st.item()) & B.STATUS_NONFINITE_INPUT
    tiny = torch.full((8, 128), 1e-38, dtype=torch.bfloat16, device=dev)     # Q / absmax overflows binary32
    got = mofq.quantize_tensor(tiny, "FP8_E5M2", "channel")
    assert int(got["status"].item()) & B.STATUS_SCALE_OVERFLOW


# ---- tensor error ------------------------------------------------------------------------------------------------
def _oracle_mse(orc, xh, names, gran, group):
    return [orc.tensor_mse(xh, getattr(orc, n), orc_gran(orc, gran), group) for n in names]


@pytest.mark.parametrize("names", [["INT4", "FP4_E2M1"], ["FP4_E2M1", "INT4", "FP4_E2M1_IEEE"], ["INT8", "FP8_E4M3", "FP8_E5M2"],
                                   ["FP8_E5M2"], ["INT8"], ["FP8_E4M3", "FP8_E5M2"]])
@pytest.mark.parametrize("gran,group", [("channel", 0), ("group", 128), ("tensor", 0)])
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_tensor_error_matches_oracle(orc, dev, names, gran, group, dtype):
    x = _weights(dev, 333, 1408, seed=21, layer=2, dtype=dtype)               # 1408 = 11 * 128
    got, st = mofq.tensor_error(x, names, gran, group=group)
    want = _oracle_mse(orc, host(x), names, gran, group)
    assert rel_err(got.cpu().numpy(), want).max() < MSE_RTOL
    assert int(st.item()) == 0


@pytest.mark.parametrize("absmax", [1.6e20, 1e-16])
@pytest.mark.parametrize("gran,group,gran2", [("channel", 128, "group"), ("channel", 0, None), ("tensor", 0, None)])
def test_tensor_error_bf16_extreme_magnitudes(orc, dev, absmax, gran, group, gran2):
    """bfloat16 tensors whose largest scales, squared, leave the binary32 range (abs-max 1.6e20: scale^2 up to 7e38) or sit
    a few decades above its subnormals (abs-max 1e-16: ~3e-34): the FP candidates' sums are kept in units of the scale
    and scaled back in double, so the errors (which still fit binary32) and the decisions must agree with the oracle
    as for ordinary magnitudes.  (Covers the kernels behind whole-model selection and per-tensor activation scales;
    the block-wise selection kernel sums unscaled squares in binary32 and is documented to need |x| < 1e18.)"""
    w = _weights(dev, 64, 1152, seed=23, layer=4).float()
    x = (w * (absmax / float(w.abs().max()))).to(torch.bfloat16)
    names = ["INT4", "FP4_E2M1"]
    got, st = mofq.tensor_error(x, names, gran, gran2=gran2, group=group)
    want = _oracle_mse(orc, host(x), names, gran, group if gran == "group" else 0)
    if gran2:
        want = want + _oracle_mse(orc, host(x), names, gran2, group)
    assert int(st.item()) == 0
    got = got.cpu().numpy().reshape(-1)
    assert np.all(np.isfinite(got)) and np.all(got > 0)
    assert rel_err(got, want).max() < MSE_RTOL, (got, want)
    cfg = mofq.make_config(4, names, w_gran=gran, w_group=group, w_gran2=gran2)
    recs = mofq.select_formats([x, x], cfg)
    n_sets = 2 if gran2 else 1
    for k, r in enumerate(recs):
        w = want[(k % n_sets) * 2:(k % n_sets) * 2 + 2]
        assert r["status"] == 0 and r["chosen"] == orc.select(w)


@pytest.mark.parametrize("kind,kw", [("gauss_outlier", {}), ("laplace", {}), ("student_t", {})])
def test_tensor_error_two_granularities_from_one_read(orc, dev, kind, kw):
    x = _weights(dev, 150, 6656, kind=kind, seed=22, layer=4)                 # LLaMA-33B hidden width: 52 groups per row
    names = ["INT4", "FP4_E2M1"]
    for g1, g2 in (("channel", "group"), ("group", "channel")):
        got, _ = mofq.tensor_error(x, names, g1, gran2=g2, group=128)
        want = np.array([_oracle_mse(orc, host(x), names, g1, 128), _oracle_mse(orc, host(x), names, g2, 128)])
        assert rel_err(got.cpu().numpy(), want).max() < MSE_RTOL


def test_tensor_error_strided_group_scales(orc, dev):
    full = _weights(dev, 48, 2048, seed=23)
    view = full[:, 512:1536]
    got, _ = mofq.tensor_error(view, ["INT4", "FP4_E2M1"], "group", group=128)
    want = _oracle_mse(orc, host(view).contiguous(), ["INT4", "FP4_E2M1"], "group", 128)
    assert rel_err(got.cpu().numpy(), want).max() < MSE_RTOL


def test_tensor_error_is_deterministic(dev):
    x = _weights(dev, 512, 4096, seed=24)
    for gran, group in (("channel", 0), ("group", 128), ("tensor", 0)):
        a, _ = mofq.tensor_error(x, ["INT4", "FP4_E2M1"], gran, group=group)
        b, _ = mofq.tensor_error(x, ["INT4", "FP4_E2M1"], gran, group=group)
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_zero_tensor_and_grid_tensor(orc, dev):
    z = torch.zeros(64, 512, dtype=torch.float16, device=dev)
    got, _ = mofq.tensor_error(z, ["INT4", "FP4_E2M1"], "channel")
    assert got.tolist() == [0.0, 0.0]
    tab = orc.decode_table(orc.FP4_E2M1)
    g = np.random.default_rng(1)
    x = torch.from_numpy(g.choice(tab, (64, 512)) / 64.0).to(torch.float16)
    x[:, 0] = 6.0 / 64
    got, _ = mofq.tensor_error(x.to(dev), ["INT4", "FP4_E2M1"], "channel")
    assert got[1].item() == 0.0 and got[0].item() > 0.0


# ---- the single-layer workload at full size (4096 x 4096, per-channel, INT4 vs FP4) ---------------------------------
def test_single_layer_workload_full_size(orc, dev):
    wl = inputs.WORKLOADS["single_4096_w4_channel"]
    w = torch.empty((4096, 4096), dtype=torch.float16, device=dev)
    inputs.device_weight(w, wl["w_kind"], wl["seed"], 0, **wl["w_args"])
    wh = host(w)
    cfg = mofq.make_config(4, wl["candidates"], w_gran="channel")
    rec = mofq.select_formats([w], cfg)[0]
    want = [orc.tensor_mse(wh, getattr(orc, n), orc.PER_CHANNEL) for n in wl["candidates"]]
    assert rel_err(rec["errors"], want).max() < MSE_RTOL
    assert rec["chosen"] == orc.select(want) and rec["status"] == 0
    for name in wl["candidates"]:
        got = mofq.quantize_tensor(w, name, "channel")
        ref = orc.quantize(wh, getattr(orc, name), orc.PER_CHANNEL)
        np.testing.assert_array_equal(unpack_codes(got["codes"], 4, w.numel()), ref["codes"].reshape(-1))
        np.testing.assert_array_equal(got["scales"].cpu().numpy().view(np.uint32), ref["scales"].view(np.uint32))


# ---- selection over a layer list (Algorithm 1) ------------------------------------------------------------------------
def _small_model(dev, kind, seed, shapes, **kw):
    return [_weights(dev, o, i, kind=kind, seed=seed, layer=l, **kw) for l, (o, i) in enumerate(shapes)]


@pytest.mark.parametrize("gran,group,gran2", [("group", 128, None), ("channel", 0, None), ("channel", 128, "group"), ("tensor", 0, None)])
def test_select_formats_matches_oracle(orc, dev, gran, group, gran2):
    shapes = [(256, 512), (256, 512), (688, 512), (512, 1408), (128, 128), (40, 256)]
    layers = _small_model(dev, "student_t", 31, shapes)
    layers[4].zero_()                                                         # tie at zero error -> first candidate
    cands = ["INT4", "FP4_E2M1"]
    cfg = mofq.make_config(4, cands, w_gran=gran, w_group=group, w_gran2=gran2)
    recs = mofq.select_formats(layers, cfg)
    n_sets = 2 if gran2 else 1
    assert len(recs) == len(layers) * n_sets
    for li, w in enumerate(layers):
        for s, g in enumerate([gran, gran2][:n_sets]):
            want = [orc.tensor_mse(host(w), getattr(orc, n), orc_gran(orc, g), 128 if g == "group" else 0) for n in cands]
            r = recs[li * n_sets + s]
            assert r["status"] == 0
            if max(want) > 0:
                assert rel_err(r["errors"], want).max() < MSE_RTOL
            assert r["chosen"] == orc.select(want), (li, g, want, r)
    assert recs[4 * n_sets]["chosen"] == 0 and recs[4 * n_sets]["errors"] == [0.0, 0.0]
    swapped = mofq.make_config(4, cands[::-1], w_gran=gran, w_group=group, w_gran2=gran2)
    recs2 = mofq.select_formats(layers, swapped)
    assert recs2[4 * n_sets]["chosen"] == 0                                   # still the first in the caller's order
    for a, b in zip(recs, recs2):
        if a["errors"][0] != a["errors"][1]:
            assert a["chosen"] == 1 - b["chosen"]


def test_select_formats_host_buffers(orc, dev):
    shapes = [(256, 512), (128, 1024), (64, 256)]
    layers = [host(w).pin_memory() for w in _small_model(dev, "laplace", 32, shapes)]
    cfg = mofq.make_config(4, ["INT4", "FP4_E2M1"], w_gran="group", w_group=128)
    recs = mofq.select_formats_host(layers, cfg, dev)
    for w, r in zip(layers, recs):
        want = [orc.tensor_mse(w, f, orc.PER_GROUP, 128) for f in (orc.INT4, orc.FP4_E2M1)]
        assert rel_err(r["errors"], want).max() < MSE_RTOL and r["chosen"] == orc.select(want)


def test_margins_are_reported(dev):
    layers = _small_model(dev, "student_t", 33, [(256, 512)])
    cfg = mofq.make_config(4, ["INT4", "FP4_E2M1"], w_gran="channel")
    r = mofq.select_formats(layers, cfg)[0]
    e = sorted(r["errors"])
    assert r["rel_margin"] == pytest.approx((e[1] - e[0]) / e[0], rel=1e-4)


# ---- the persistent multi-tensor scoring path (dense tensors, per-group scales) ------------------------------------------
@pytest.mark.parametrize("bits,cands", [(4, ["INT4", "FP4_E2M1"]), (4, ["FP4_E2M1_IEEE", "INT4", "FP4_E2M1"]), (4, ["FP4_E2M1"]),
                                        (8, ["INT8", "FP8_E4M3", "FP8_E5M2"]), (8, ["FP8_E5M2", "FP8_E4M3"]), (8, ["INT8"])])
@pytest.mark.parametrize("group", [128, 32, 256])
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_multi_tensor_path_matches_oracle(orc, dev, bits, cands, group, dtype):
    # many small layers (several per block), a big one spanning many blocks, ragged last tiles, a zero layer
    shapes = [(8, 256), (56, 768), (3000, 2048), (1, 256), (130, 1280), (16, 512), (1000, 4352)]
    layers = [_weights(dev, o, i, kind=["student_t", "laplace", "gauss_outlier"][l % 3], seed=41, layer=l, dtype=dtype)
              for l, (o, i) in enumerate(shapes)]
    layers[5].zero_()
    cfg = mofq.make_config(bits, cands, w_gran="group", w_group=group)
    recs = mofq.select_formats(layers, cfg)
    again = mofq.select_formats(layers, cfg)
    assert recs == again                                                      # fixed summation order: bit-identical reruns
    for li, (w, r) in enumerate(zip(layers, recs)):
        want = [orc.tensor_mse(host(w), getattr(orc, n), orc.PER_GROUP, group) for n in cands]
        assert r["status"] == 0
        if max(want) > 0:
            assert rel_err(r["errors"], want).max() < MSE_RTOL, (li, r, want)
        assert r["chosen"] == orc.select(want), (li, r, want)
    assert recs[5]["chosen"] == 0 and recs[5]["errors"] == [0.0] * len(cands)


def test_multi_tensor_path_status_per_layer(dev):
    layers = [_weights(dev, 64, 512, seed=42, layer=l) for l in range(4)]
    layers[2][7, 300] = float("nan")
    cfg = mofq.make_config(4, ["INT4", "FP4_E2M1"], w_gran="group", w_group=128)
    recs = mofq.select_formats(layers, cfg)
    assert [bool(r["status"] & B.STATUS_NONFINITE_INPUT) for r in recs] == [False, False, True, False]


# ---- the hardware converts used by the scoring kernels round like the definition ------------------------------------------
@pytest.mark.parametrize("name", ["FP4_E2M1", "FP8_E4M3", "FP8_E5M2"])
def test_hardware_fp_rounding_matches_oracle(orc, dev, name):
    fmt = getattr(orc, name)
    half = 2 ** (orc.format_bits(fmt) - 1)
    pos = orc.decode_table(fmt)[:half]
    pos = pos[~np.isnan(pos)]
    mids = (pos[:-1] + pos[1:]) / 2
    pts = [pos, mids]
    for d in (-2, -1, 1, 2):                                                   # neighbours of every tie in binary32
        pts.append((mids.astype(np.float32).view(np.uint32).astype(np.int64) + d).astype(np.uint32).view(np.float32).astype(np.float64))
    g = np.random.default_rng(9)
    pts.append(g.uniform(0, pos[-1] * 1.5, 20000))
    pts.append(np.exp(g.uniform(np.log(pos[1] / 64), np.log(pos[-1] * 2), 20000)))
    t = np.concatenate(pts).astype(np.float32)
    t = np.concatenate([t, -t, np.array([0.0, -0.0, 1e30, -1e30], np.float32)])
    from paper_2305_12356_b200.binding import diag_fp_round
    got = diag_fp_round(name, torch.from_numpy(t).to(dev)).cpu().numpy()
    tab = orc.decode_table(fmt)
    want = np.array([tab[orc.encode_fp_arith(fmt, v)] for v in t])
    np.testing.assert_array_equal(got.astype(np.float64), want)
    np.testing.assert_array_equal(np.signbit(got), np.signbit(t))               # the sign survives rounding to zero


# ---- calibration scales applied to unseen batches (Section 3.2, dynamic tensor analysis) --------------------------------------
def test_calibration_scales_and_saturation_match_oracle(orc, dev):
    n_in, T = 1024, 256
    batches = []
    for b in range(5):
        x = torch.empty((T, n_in), dtype=torch.bfloat16, device=dev)
        inputs.device_activation(x, 61, b, n_ch=6, ch_gain=50.0 if b < 4 else 120.0)   # the unseen batch has larger outliers
        batches.append(x)
    cal = torch.zeros(1, dtype=torch.float32, device=dev)
    for x in batches[:4]:
        mofq.absmax_update(x, cal)
    want_cal = max(float(host(x).abs().max()) for x in batches[:4])
    assert float(cal.item()) == want_cal                                         # the largest value over the calibration batches
    names = ["INT8", "FP8_E4M3", "FP8_E5M2"]
    scales = torch.tensor([np.float32(want_cal) / np.float32(orc.format_max(getattr(orc, n))) for n in names], dtype=torch.float32, device=dev)
    for x in (batches[1], batches[4]):                                           # a calibration batch and the unseen, clipping batch
        got, st = mofq.tensor_error_scaled(x, names, scales)
        want = [orc.quantize(host(x), getattr(orc, n), orc.PER_TENSOR, scales_in=[float(s)])["sse"] / x.numel()
                for n, s in zip(names, scales.cpu())]
        assert int(st.item()) == 0
        assert rel_err(got.cpu().numpy(), want).max() < MSE_RTOL, (got, want)
    # the paper's observation: with calibration scales FP8 has the lower error on activations with outliers
    assert got[1].item() < got[0].item()
    # candidate order is the caller's
    got2, _ = mofq.tensor_error_scaled(batches[4], names[::-1], scales.flip(0))
    assert torch.equal(got2.flip(0), got)


@pytest.mark.parametrize("names", [["INT4", "FP4_E2M1"], ["FP4_E2M1_IEEE", "INT4", "FP4_E2M1"], ["FP8_E4M3"], ["INT8"]])
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_supplied_scales_small_and_ragged(orc, dev, names, dtype):
    x = torch.empty((37, 1000), dtype=dtype, device=dev)                        # ragged: 37000 elements
    inputs.device_weight(x, "gauss_outlier", 62, 0)
    amax = float(host(x).abs().max())
    for shrink in (1.0, 0.37, 2.5):                                              # exact, clipping, and wasteful scales
        sc = torch.tensor([np.float32(amax * shrink) / np.float32(orc.format_max(getattr(orc, n))) for n in names],
                          dtype=torch.float32, device=dev)
        got, st = mofq.tensor_error_scaled(x, names, sc)
        want = [orc.quantize(host(x), getattr(orc, n), orc.PER_TENSOR, scales_in=[float(s)])["sse"] / x.numel()
                for n, s in zip(names, sc.cpu())]
        assert int(st.item()) == 0
        assert rel_err(got.cpu().numpy(), want).max() < MSE_RTOL, (names, shrink, got, want)


# ---- streamed-row scoring kernel: tile shapes, ragged last tile, strided rows, widest row ------------------------------------
@pytest.mark.parametrize("rows,cols,ld", [(13, 128, 128), (37, 4096, 4096), (29, 6656, 6656 + 256), (5, 22016, 22016), (1, 24576, 24576),
                                          (1100, 256, 256)])
def test_streamed_rows_shapes(orc, dev, rows, cols, ld):
    full = _weights(dev, rows, ld, seed=41, layer=rows % 7)
    x = full[:, :cols]
    names = ["INT4", "FP4_E2M1"]
    got, st = mofq.tensor_error(x, names, "channel")
    want = _oracle_mse(orc, host(x).contiguous(), names, "channel", 0)
    assert int(st.item()) == 0
    assert rel_err(got.cpu().numpy(), want).max() < MSE_RTOL
    got2, _ = mofq.tensor_error(x, names, "group", gran2="channel", group=128)
    want2 = _oracle_mse(orc, host(x).contiguous(), names, "group", 128) + want
    assert rel_err(got2.cpu().numpy().reshape(-1), want2).max() < MSE_RTOL


@pytest.mark.parametrize("rows,cols,group", [(37, 1000, 8), (9, 1096, 8), (3, 40000, 64), (70, 1160, 0)])
def test_row_fallback_kernel_for_rows_the_streamed_kernel_does_not_take(orc, dev, rows, cols, group):
    """Row lengths that are not a multiple of 128 elements, rows longer than the largest tile, and group sizes other
    than 128 beside per-channel scales go through the one-row-per-CTA kernel."""
    x = _weights(dev, rows, cols, seed=47, layer=rows % 5)
    names = ["INT4", "FP4_E2M1"]
    got, st = mofq.tensor_error(x, names, "channel", gran2="group" if group else None, group=group)
    want = _oracle_mse(orc, host(x), names, "channel", 0)
    if group:
        want = want + _oracle_mse(orc, host(x), names, "group", group)
    assert int(st.item()) == 0
    assert rel_err(got.cpu().numpy().reshape(-1), want).max() < MSE_RTOL, (got, want)
    cfg = mofq.make_config(4, names, w_gran="channel", w_group=group, w_gran2="group" if group else None)
    recs = mofq.select_formats([x, x], cfg)                                # a list that the persistent kernel refuses
    assert [r["chosen"] for r in recs[:len(recs) // 2]] == [orc.select(want[k:k + 2]) for k in range(0, len(want), 2)]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_streamed_rows_random_layer_lists(orc, dev, seed):
    """One persistent launch over lists of layers of unrelated shapes (single rows, rows of one segment, rows close
    to the longest tile, more layers than CTAs' worth of work, a change of the ring's division at every layer): each
    layer's errors and choice must be what the oracle gives for that layer alone, under every candidate set."""
    rng = np.random.default_rng(100 + seed)
    col_choices = [128, 256, 384, 1024, 2176, 4096, 6656, 11008, 17920, 24576, 35840]
    shapes = [(int(rng.integers(1, 40 if c > 8000 else 200)), int(c)) for c in rng.choice(col_choices, size=23)]
    shapes += [(1, 128), (1, 35840), (513, 128)]
    dtype = (torch.float16, torch.bfloat16)[seed % 2]
    xs = [_weights(dev, r, c, kind=("student_t", "laplace", "gauss_outlier")[i % 3], seed=60 + seed, layer=i, dtype=dtype)
          for i, (r, c) in enumerate(shapes)]
    cases = [(4, ["INT4", "FP4_E2M1"], "channel", "group"), (4, ["FP4_E2M1", "INT4"], "group", "channel"),
             (8, ["INT8", "FP8_E4M3", "FP8_E5M2"], "channel", None), (4, ["FP4_E2M1_IEEE", "INT4", "FP4_E2M1"], "channel", "group")]
    for bits, names, g1, g2 in (cases[seed % 4], cases[(seed + 2) % 4]):
        cfg = mofq.make_config(bits, names, w_gran=g1, w_group=128, w_gran2=g2)
        recs = mofq.select_formats(xs, cfg)
        again = mofq.select_formats(xs, cfg)
        assert recs == again                                              # fixed summation order
        n_sets = 2 if g2 else 1
        for i, x in enumerate(xs):
            for s, g in enumerate((g1, g2)[:n_sets]):
                want = _oracle_mse(orc, host(x), names, g, 128 if g == "group" else 0)
                r = recs[i * n_sets + s]
                assert r["status"] == 0
                assert rel_err(r["errors"], want).max() < MSE_RTOL, (shapes[i], g, r, want)
                if min(abs(a - b) for k, a in enumerate(want) for b in want[k + 1:]) > 1e-4 * max(want):
                    assert r["chosen"] == orc.select(want), (shapes[i], g, r, want)


@pytest.mark.parametrize("g1,g2,n_layers", [("channel", "group", 601), ("group", None, 1100)])
def test_layer_lists_longer_than_one_table_upload(orc, dev, g1, g2, n_layers):
    """The work table reaches the device as kernel parameters, a few hundred entries per launch: lists that need
    three launches (the last one partly filled) must give every layer what that layer gives alone."""
    names = ["INT4", "FP4_E2M1"]
    base = [_weights(dev, r, c, seed=66, layer=i) for i, (r, c) in enumerate([(3, 256), (1, 128), (5, 384), (2, 1024), (7, 128)])]
    xs = [base[i % len(base)] for i in range(n_layers)]
    cfg = mofq.make_config(4, names, w_gran=g1, w_group=128, w_gran2=g2)
    recs = mofq.select_formats(xs, cfg)
    n_sets = 2 if g2 else 1
    assert len(recs) == n_layers * n_sets
    for s, g in enumerate((g1, g2)[:n_sets]):
        for k, x in enumerate(base):
            want = _oracle_mse(orc, host(x), names, g, 128 if g == "group" else 0)
            for i in range(k, n_layers, len(base)):
                r = recs[i * n_sets + s]
                assert r["status"] == 0 and rel_err(r["errors"], want).max() < MSE_RTOL, (i, g, r, want)
            assert all(recs[i * n_sets + s] == recs[k * n_sets + s] for i in range(k, n_layers, len(base)))


def test_streamed_rows_layers_of_one_call_overlap_safely(orc, dev):
    """Within one selection call the streamed-row kernel lets the next layer's launch start before the current one has
    drained; the header and the partial sums they share are only touched after the earlier launch has completed.
    Many short layers in one call, and calls back to back without host synchronisation, must give for every layer
    exactly what that layer gives when scored alone."""
    names = ["INT4", "FP4_E2M1"]
    shapes = [(300, 6656), (17, 4096), (640, 1024), (96, 17920), (1, 128), (410, 6656)] * 4
    xs = [_weights(dev, r, c, seed=43, layer=i % 6) for i, (r, c) in enumerate(shapes)]
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device=dev)
    alone = []
    for x in xs[:6]:
        got, st = mofq.tensor_error(x, names, "channel", gran2="group", group=128, workspace=ws)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        alone.append(got.cpu().numpy().copy())
    want0 = np.concatenate([_oracle_mse(orc, host(xs[0]), names, "channel", 0), _oracle_mse(orc, host(xs[0]), names, "group", 128)])
    assert rel_err(alone[0].reshape(-1), want0).max() < MSE_RTOL
    cfg = mofq.make_config(4, names, w_gran="channel", w_group=128, w_gran2="group")
    prepared = mofq.prepare_layers(xs)
    wsel = torch.zeros(mofq.workspace_bytes(prepared, cfg), dtype=torch.uint8, device=dev)
    raw = [torch.empty(2 * len(xs) * B.RESULT_BYTES, dtype=torch.uint8, device=dev) for _ in range(3)]
    for out in raw:                                         # three calls in a row, nothing synchronises in between
        mofq.select_formats(prepared, cfg, workspace=wsel, results=out, parse=False)
    torch.cuda.synchronize()
    for out in raw:
        recs = B._parse_results(bytes(out.cpu().numpy()), 2 * len(xs), len(names))
        for li in range(len(xs)):
            for s_ in range(2):
                r = recs[2 * li + s_]
                assert r["status"] == 0
                np.testing.assert_array_equal(np.asarray(r["errors"], np.float32).view(np.uint32), alone[li % 6][s_].view(np.uint32))


@pytest.mark.parametrize("name", FMT4 + FMT8)
def test_fast_scale_pair_is_correctly_rounded_for_every_binary16_magnitude(orc, dev, name):
    from paper_2305_12356_b200.binding import diag_scale_pair
    bits = np.arange(0x7C00, dtype=np.uint16)                                    # 0, every subnormal and normal magnitude
    a = bits.view(np.float16).astype(np.float32)
    s, inv = diag_scale_pair(name, torch.from_numpy(a).to(dev))
    Q = np.float32(orc.format_max(getattr(orc, name)))
    with np.errstate(divide="ignore"):
        want_s = np.where(a == 0, np.float32(1), a / Q).astype(np.float32)       # numpy float32 division is correctly rounded
        want_i = np.where(a == 0, np.float32(1), Q / a).astype(np.float32)
    np.testing.assert_array_equal(s.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    np.testing.assert_array_equal(inv.cpu().numpy().view(np.uint32), want_i.view(np.uint32))
    for k in (0, 1, 2, 1000, 0x3C00, 0x7BFF):                                    # and the oracle's own routine on a few
        so, io = orc.scale_from_absmax(getattr(orc, name), a[k])
        assert so == want_s[k] and io == want_i[k]


# ---- codes + scales only: the register-resident emission kernel (group and per-tensor scales) ---------------------------------
def _check_codes_only(orc, x, name, gran, group=0):
    fmt_o = getattr(orc, name)
    bits = orc.format_bits(fmt_o)
    got = mofq.quantize_tensor(x, name, gran, group)
    want = orc.quantize(host(x).contiguous(), fmt_o, orc_gran(orc, gran), group)
    np.testing.assert_array_equal(unpack_codes(got["codes"], bits, x.numel()), want["codes"].reshape(-1))
    np.testing.assert_array_equal(got["scales"].cpu().numpy().view(np.uint32), want["scales"].view(np.uint32))
    assert int(got["status"].item()) == 0


@pytest.mark.parametrize("name", FMT4 + FMT8)
@pytest.mark.parametrize("gran,group", [("group", 128), ("group", 256), ("group", 32), ("group", 16), ("group", 8), ("tensor", 0)])
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_codes_only_emission_matches_oracle(orc, dev, name, gran, group, dtype):
    x = _weights(dev, 301, 1280, seed=51, layer=2, dtype=dtype)                  # 301 rows: ragged against the warp teams
    x[5, 100:228] = 0                                                             # an all-zero group
    x[9, 3] = -0.0
    _check_codes_only(orc, x, name, gran, group)


def test_codes_only_emission_strided_and_every_fp16_pattern(orc, dev):
    full = _weights(dev, 40, 1024 + 64, seed=52)
    view = full[:, 32:1056]
    for name in ("INT4", "FP4_E2M1", "INT8", "FP8_E5M2"):
        _check_codes_only(orc, view, name, "group", 128)
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    bits = bits[(bits & 0x7C00) != 0x7C00]
    bits = np.concatenate([bits, np.zeros((-bits.size) % 1024, np.uint16)])
    x = torch.from_numpy(bits.view(np.int16).copy()).view(torch.float16).reshape(-1, 1024).to(dev)
    for name in FMT4 + FMT8:
        for gran, group in (("group", 128), ("group", 8), ("tensor", 0)):
            _check_codes_only(orc, x, name, gran, group)


def test_bounded_wait_expires_and_leaves_the_context_usable(orc, dev):
    """A wait that can never be satisfied ends after its limit with a status bit; the GPU stays usable."""
    import time
    from paper_2305_12356_b200.binding import diag_wait_expiry
    t0 = time.time()
    st = diag_wait_expiry(dev)
    torch.cuda.synchronize()
    dt = time.time() - t0
    assert int(st.item()) == B.STATUS_TIMEOUT
    assert 0.5 < dt < 10.0, dt                                                    # about two seconds, never a hang
    x = _weights(dev, 16, 256, seed=61)                                           # and ordinary work still runs
    got, s2 = mofq.tensor_error(x, ["INT4", "FP4_E2M1"], "channel")
    want = _oracle_mse(orc, host(x), ["INT4", "FP4_E2M1"], "channel", 0)
    assert int(s2.item()) == 0 and rel_err(got.cpu().numpy(), want).max() < MSE_RTOL
