"""Pins for the oracle's tensor quantiser, tensor MSE and selection rule (CPU only).

Each test fixes the oracle to something outside it: exact rational arithmetic on tiny tensors,
closed forms for uniform data, algebraic invariants of round-to-nearest on a symmetric grid, and
special inputs whose answer is known in advance.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2305_12356_b200 import inputs

FP_NAMES = ["FP4_E2M1", "FP4_E2M1_IEEE", "FP8_E4M3", "FP8_E5M2"]
ALL_NAMES = ["INT4", "INT8"] + FP_NAMES


def _rand16(shape, seed, scale=0.02, dtype=torch.float16):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(dtype)


def _values(x):
    return x.to(torch.float64).numpy()


def _decoded(orc, fmt, codes):
    tab = orc.decode_table(fmt)
    return tab[codes]


# ---- scales -------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ALL_NAMES)
def test_scale_is_absmax_over_q(orc, name):
    fmt = getattr(orc, name)
    Q = np.float32(orc.format_max(fmt))
    x = _rand16((6, 256), 1)
    x[2, 17] = 0.75          # planted maxima
    x[4, 200] = -1.5
    x[5, :] = 0              # all-zero row
    q = orc.quantize(x, fmt, orc.PER_CHANNEL)
    am = _values(x.abs()).max(axis=1).astype(np.float32)
    want = np.where(am > 0, am / Q, np.float32(1.0)).astype(np.float32)
    np.testing.assert_array_equal(q["scales"], want)
    assert q["scales"][2] == np.float32(0.75) / Q and q["scales"][4] == np.float32(1.5) / Q
    assert q["scales"][5] == 1.0 and not q["codes"][5].any()
    # per-group: 128 consecutive input-dim elements; per-tensor: one scale
    qg = orc.quantize(x, fmt, orc.PER_GROUP, 128)
    amg = _values(x.abs()).reshape(6, 2, 128).max(axis=2).astype(np.float32).reshape(-1)
    np.testing.assert_array_equal(qg["scales"], np.where(amg > 0, amg / Q, np.float32(1.0)).astype(np.float32))
    qt = orc.quantize(x, fmt, orc.PER_TENSOR)
    assert qt["scales"].shape == (1,) and qt["scales"][0] == np.float32(1.5) / Q


def _round_to_binary32(q):
    """Correctly rounded (nearest, ties to even) binary32 of a positive exact rational in the normal range."""
    e = 0
    while q >= 2:
        q /= 2
        e += 1
    while q < 1:
        q *= 2
        e -= 1
    assert -126 <= e <= 127
    m = q * (1 << 23)                       # 2^23 <= m < 2^24
    n, rem = divmod(m.numerator, m.denominator)
    twice = 2 * rem
    if twice > m.denominator or (twice == m.denominator and (n & 1)):
        n += 1
    return np.float32(float(Fraction(n, 1 << 23) * Fraction(2) ** e))   # n <= 2^24: exact in binary64 and binary32


@pytest.mark.parametrize("name", ALL_NAMES)
def test_scale_pair_is_two_correctly_rounded_quotients(orc, name):
    """scale = RN32(absmax / Q) and inv = RN32(Q / absmax), each rounded once from the exact quotient (exact rational
    arithmetic here); in particular inv is NOT the reciprocal of the rounded scale."""
    fmt = getattr(orc, name)
    Q = Fraction(orc.format_max(fmt))
    rng = np.random.default_rng(11)
    bits = np.unique(np.concatenate([rng.integers(0x0001, 0x7C00, size=400), [0x0001, 0x03FF, 0x0400, 0x3C00, 0x7BFF]])).astype(np.uint16)
    differs = 0
    for b in bits:
        a = np.array([b], dtype=np.uint16).view(np.float16)[0]
        fa = Fraction(float(a))
        scale, inv = orc.scale_from_absmax(fmt, float(a))
        want_s, want_i = _round_to_binary32(fa / Q), _round_to_binary32(Q / fa)
        assert np.float32(scale) == want_s and np.float32(inv) == want_i, (hex(int(b)), scale, inv, want_s, want_i)
        differs += int(want_i != np.float32(1.0) / want_s)
    assert differs > 0      # the sample tells the two definitions apart
    assert orc.scale_from_absmax(fmt, 0.0) == (1.0, 1.0)


@pytest.mark.parametrize("name", ALL_NAMES)
def test_absmax_element_gets_top_code_and_no_reserved_codes(orc, name):
    fmt = getattr(orc, name)
    x = _rand16((16, 384), 2)
    q = orc.quantize(x, fmt, orc.PER_CHANNEL)
    dec = _decoded(orc, fmt, q["codes"])
    assert not np.isnan(dec).any()                                   # reserved codes never emitted
    assert np.abs(dec).max() <= orc.format_max(fmt)                   # INT: -qmax-1 unreachable with abs-max scales
    v = _values(x)
    idx = np.abs(v).argmax(axis=1)
    top = dec[np.arange(16), idx]
    np.testing.assert_array_equal(np.abs(top), orc.format_max(fmt))
    np.testing.assert_array_equal(np.sign(top), np.sign(v[np.arange(16), idx]))


# ---- invariants of round-to-nearest on a symmetric grid --------------------------------------------
@pytest.mark.parametrize("name", ALL_NAMES)
def test_odd_symmetry_including_negative_zero(orc, name):
    fmt = getattr(orc, name)
    k = orc.format_bits(fmt)
    x = _rand16((8, 256), 3)
    x[0, :4] = torch.tensor([0.0, -0.0, 1e-7, -1e-7], dtype=torch.float16)
    a, b = orc.quantize(x, fmt, orc.PER_CHANNEL), orc.quantize(-x, fmt, orc.PER_CHANNEL)
    np.testing.assert_array_equal(a["scales"], b["scales"])
    da, db = _decoded(orc, fmt, a["codes"]), _decoded(orc, fmt, b["codes"])
    np.testing.assert_array_equal(da, -db)
    assert a["sse"] == pytest.approx(b["sse"], rel=1e-12)       # OpenMP sum order may differ
    if name.startswith("FP"):                                         # sign bit follows the input's sign bit
        sign = (x.view(torch.int16).numpy().view(np.uint16) >> 15).astype(np.uint8)
        np.testing.assert_array_equal(a["codes"] >> (k - 1), sign)
        np.testing.assert_array_equal(a["codes"] ^ (1 << (k - 1)), b["codes"])


@pytest.mark.parametrize("name", ALL_NAMES)
def test_monotone_and_within_half_a_gap(orc, name):
    fmt = getattr(orc, name)
    x = torch.sort(_rand16((1, 4096), 4).flatten()).values.reshape(1, -1)
    q = orc.quantize(x, fmt, orc.PER_CHANNEL)
    s = float(q["scales"][0])
    d = _decoded(orc, fmt, q["codes"][0]) * s
    assert np.all(np.diff(d) >= 0)
    grid = np.unique(orc.decode_table(fmt)[~np.isnan(orc.decode_table(fmt))]) * s
    v = _values(x)[0]
    # distance to the chosen point is the distance to the nearest grid point (up to the fp32 rounding of x*inv)
    nearest = np.abs(v[:, None] - grid[None, :]).min(axis=1)
    assert np.all(np.abs(v - d) <= nearest * (1 + 1e-5) + 1e-12)


@pytest.mark.parametrize("name", ALL_NAMES)
def test_idempotent(orc, name):
    fmt = getattr(orc, name)
    x = _rand16((8, 256), 5, scale=0.3)
    q = orc.quantize(x, fmt, orc.PER_CHANNEL, want_dequant=False)
    # feed back code values times a power-of-two scale: every element is on the grid -> same codes, zero error
    tab = orc.decode_table(fmt)
    on_grid = torch.from_numpy(tab[q["codes"]] * 2.0 ** -6).to(torch.float16)   # every grid value is exact in fp16
    assert np.array_equal(_values(on_grid), tab[q["codes"]] * 2.0 ** -6)
    q2 = orc.quantize(on_grid, fmt, orc.PER_CHANNEL)
    np.testing.assert_array_equal(tab[q2["codes"]], tab[q["codes"]])
    assert q2["sse"] == 0.0
    np.testing.assert_array_equal(q2["scales"], np.float32(2.0 ** -6))


@pytest.mark.parametrize("name", ALL_NAMES)
@pytest.mark.parametrize("p", [-3, 4])
def test_power_of_two_scaling(orc, name, p):
    fmt = getattr(orc, name)
    x = _rand16((8, 256), 6, scale=0.05)
    x = torch.where(x.abs() < 2.0 ** -8, torch.full_like(x, 2.0 ** -8), x)    # keep x * 2^p out of the fp16 subnormals
    y = (x.float() * 2.0 ** p).to(torch.float16)
    assert torch.equal(y.float(), x.float() * 2.0 ** p)               # no subnormal/overflow losses at this scale
    a, b = orc.quantize(x, fmt, orc.PER_GROUP, 128), orc.quantize(y, fmt, orc.PER_GROUP, 128)
    np.testing.assert_array_equal(a["codes"], b["codes"])
    np.testing.assert_array_equal(a["scales"] * np.float32(2.0 ** p), b["scales"])
    assert b["sse"] == pytest.approx(a["sse"] * 4.0 ** p, rel=1e-12)


# ---- tensor MSE ---------------------------------------------------------------------------------------
def _fraction_of_bits(x):
    return [[Fraction(float(v)) for v in row] for row in _values(x)]


@pytest.mark.parametrize("name", ALL_NAMES)
@pytest.mark.parametrize("gran", ["PER_TENSOR", "PER_CHANNEL", "PER_GROUP"])
def test_mse_brute_force_exact_rationals(orc, name, gran):
    """Nearest grid point by exhaustive search in exact rational arithmetic on a tiny tensor."""
    fmt, g = getattr(orc, name), getattr(orc, gran)
    group = 4 if gran == "PER_GROUP" else 0
    x = _rand16((3, 8), 7, scale=0.4)
    X = _fraction_of_bits(x)
    tab = orc.decode_table(fmt)
    grid = sorted({Fraction(float(v)) for v in tab if not np.isnan(v)})
    Q = Fraction(orc.format_max(fmt))
    total = Fraction(0)
    for r in range(3):
        for c in range(8):
            if gran == "PER_TENSOR":
                block = [v for row in X for v in row]
            elif gran == "PER_CHANNEL":
                block = X[r]
            else:
                block = X[r][(c // 4) * 4:(c // 4) * 4 + 4]
            am = max(abs(v) for v in block)
            s = Fraction(float(np.float32(float(am)) / np.float32(float(Q))))    # the stored fp32 scale
            best = min(abs(X[r][c] - gv * s) for gv in grid)
            total += best * best
    want = float(total / 24)
    got = orc.tensor_mse(x, fmt, g, group)
    # Rounding x*inv in fp32 can pick the other neighbour only within 2^-23 of a midpoint, where both are equally far.
    assert got == pytest.approx(want, rel=1e-6)


@pytest.mark.parametrize("name,coef", [
    ("INT4", 1.0 / (12 * 49)),                                           # (a/7)^2 / 12
    ("INT8", 1.0 / (12 * 127 ** 2)),
    ("FP4_E2M1", (4 * 0.5 ** 3 + 2 * 1.0 + 8.0) / 12 / 6 / 36),          # sum(gap^3)/12 / range, gaps .5,.5,.5,.5,1,1,2 on [0,6]
])
def test_uniform_data_closed_form_and_decision(orc, name, coef):
    """x ~ U[-a, a], per-tensor scale: MSE = a^2 * sum_j w_j^3 / (12 * range) over the scaled grid gaps."""
    fmt = getattr(orc, name)
    a = 0.5
    g = np.random.default_rng(11)
    x = torch.from_numpy(g.uniform(-a, a, (256, 2048)).astype(np.float32)).to(torch.float16)
    x[0, 0] = a
    got = orc.tensor_mse(x, fmt, orc.PER_TENSOR)
    # fp16 input granularity (2^-12 at |x|~0.5) matters only for INT8, whose step is a/127 ~ 2^-8
    tol = 0.02 if name != "INT8" else 0.05
    assert got == pytest.approx(coef * a * a, rel=tol)


def test_uniform_data_prefers_int4(orc):
    g = np.random.default_rng(12)
    x = torch.from_numpy(g.uniform(-1, 1, (64, 1024)).astype(np.float32)).to(torch.float16)
    errs = [orc.tensor_mse(x, f, orc.PER_CHANNEL) for f in (orc.INT4, orc.FP4_E2M1)]
    assert orc.select(errs) == 0 and errs[0] < errs[1]
    # 1.701e-3 vs 4.051e-3 (times a^2) for a per-tensor scale: ratio ~ 2.38
    assert errs[1] / errs[0] == pytest.approx(4.051 / 1.701, rel=0.05)


@pytest.mark.parametrize("name", ALL_NAMES)
def test_grid_valued_tensor_has_zero_error_and_wins(orc, name):
    fmt = getattr(orc, name)
    tab = orc.decode_table(fmt)
    vals = tab[~np.isnan(tab)]
    vals = vals[np.abs(vals) <= orc.format_max(fmt)]                 # INT's -qmax-1 lies outside the abs-max range
    g = np.random.default_rng(13)
    x = torch.from_numpy(g.choice(vals, (4, 256)) * 2.0 ** -7).to(torch.float16)
    x[:, 0] = float(orc.format_max(fmt) * 2.0 ** -7)                 # make the abs-max the top of the grid
    assert orc.tensor_mse(x, fmt, orc.PER_CHANNEL) == 0.0
    bits = orc.format_bits(fmt)
    cands = [f for f in (orc.INT4, orc.FP4_E2M1, orc.FP4_E2M1_IEEE) if bits == 4] or [orc.INT8, orc.FP8_E4M3, orc.FP8_E5M2]
    errs = [orc.tensor_mse(x, f, orc.PER_CHANNEL) for f in cands]
    assert cands[orc.select(errs)] == fmt or errs[orc.select(errs)] == 0.0


def test_mse_is_mean_over_whole_tensor_for_every_granularity(orc):
    x = _rand16((4, 256), 14)
    for gran, group in ((orc.PER_TENSOR, 0), (orc.PER_CHANNEL, 0), (orc.PER_GROUP, 128)):
        q = orc.quantize(x, orc.FP4_E2M1, gran, group)
        s = q["scales"]
        if gran == orc.PER_CHANNEL:
            s = s[:, None]
        elif gran == orc.PER_GROUP:
            s = np.repeat(s.reshape(4, 2), 128, axis=1)
        d = orc.decode_table(orc.FP4_E2M1)[q["codes"]] * s.astype(np.float64)
        want = np.mean((_values(x) - d) ** 2)
        assert orc.tensor_mse(x, orc.FP4_E2M1, gran, group) == pytest.approx(want, rel=1e-12)
        assert q["sse"] == pytest.approx(want * x.numel(), rel=1e-12)


def test_finer_granularity_never_hurts_int(orc):
    x = inputs.weight_cpu("student_t", 32, 512, seed=1, layer=3)
    e_t = orc.tensor_mse(x, orc.INT4, orc.PER_TENSOR)
    e_c = orc.tensor_mse(x, orc.INT4, orc.PER_CHANNEL)
    e_g = orc.tensor_mse(x, orc.INT4, orc.PER_GROUP, 128)
    assert e_g < e_c < e_t


# ---- dequantised output, packing, supplied scales ------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_dequant_output(orc, dtype):
    x = _rand16((4, 256), 15, dtype=dtype)
    q = orc.quantize(x, orc.FP8_E4M3, orc.PER_CHANNEL, want_dequant=True)
    v = orc.decode_table(orc.FP8_E4M3)[q["codes"]].astype(np.float32) * q["scales"][:, None]   # one fp32 multiply
    want = torch.from_numpy(v).to(dtype)                                                         # library RNE cast
    got = torch.from_numpy(q["dequant"].view(np.int16)).view(dtype)
    assert torch.equal(got, want)


def test_pack4_low_nibble_first(orc):
    codes = np.array([1, 2, 3, 4, 15, 0, 9], np.uint8)
    np.testing.assert_array_equal(orc.pack4(codes), np.array([0x21, 0x43, 0x0F, 0x09], np.uint8))


@pytest.mark.parametrize("name", ALL_NAMES)
def test_supplied_scale_saturates(orc, name):
    fmt = getattr(orc, name)
    k = orc.format_bits(fmt)
    x = torch.tensor([[0.5, -0.5, 4.0, -4.0, 0.01, -100.0, 100.0, 0.0]], dtype=torch.float16)
    s = np.float32(1.0 / orc.format_max(fmt))                        # grid covers [-1, 1]
    q = orc.quantize(x, fmt, orc.PER_TENSOR, scales_in=[s])
    dec = orc.decode_table(fmt)[q["codes"][0]]
    assert not np.isnan(dec).any()
    lo = -orc.format_max(fmt) - (0 if name.startswith("FP") else 1)
    np.testing.assert_array_equal(dec[[2, 3, 5, 6]], [orc.format_max(fmt), lo, lo, orc.format_max(fmt)])
    assert q["codes"].max() < 2 ** k


# ---- selection (Algorithm 1) ------------------------------------------------------------------------------
def test_selection_strict_less_first_wins_ties(orc):
    assert orc.select([1.0, 1.0]) == 0
    assert orc.select([2.0, 1.0, 1.0]) == 1
    assert orc.select([0.0, 0.0, 0.0]) == 0
    assert orc.select([3.0, 2.0, 1.0]) == 2
    zero = torch.zeros(4, 256, dtype=torch.float16)
    r = orc.mofq_select([zero], [orc.INT4, orc.FP4_E2M1], gran=orc.PER_CHANNEL)[0]
    assert r["chosen"] == 0 and r["errors"] == [0.0, 0.0]
    r = orc.mofq_select([zero], [orc.FP4_E2M1, orc.INT4], gran=orc.PER_CHANNEL)[0]
    assert r["chosen"] == 0                                          # swapping the order swaps the tie result


def test_selection_planted_layers(orc):
    g = np.random.default_rng(21)
    uni = torch.from_numpy(g.uniform(-1, 1, (32, 512)).astype(np.float32)).to(torch.float16)
    fp_vals = orc.decode_table(orc.FP4_E2M1)
    onfp = torch.from_numpy(g.choice(fp_vals, (32, 512)) / 64.0).to(torch.float16)
    onfp[:, 0] = 6.0 / 64
    res = orc.mofq_select([uni, onfp], [orc.INT4, orc.FP4_E2M1], gran=orc.PER_CHANNEL)
    assert [r["chosen"] for r in res] == [0, 1]


# ---- qualitative findings of the paper on synthetic data (sanity) ---------------------------------------------
def test_paper_findings_on_synthetic_tensors(orc):
    # Static weights at 8 bits: INT8 has lower error than FP8 (Section 3.2, static tensor analysis).
    w = _rand16((64, 1024), 31)
    assert orc.tensor_mse(w, orc.INT8, orc.PER_CHANNEL) < orc.tensor_mse(w, orc.FP8_E4M3, orc.PER_CHANNEL)
    # Activations with outlier channels, per-tensor scale: FP8 has lower error than INT8 (dynamic tensor analysis).
    x = inputs.activation_cpu(256, 1024, seed=2, layer=0)
    assert orc.tensor_mse(x, orc.FP8_E4M3, orc.PER_TENSOR) < orc.tensor_mse(x, orc.INT8, orc.PER_TENSOR)
    # Section 4.2: the FP4 grid without NaN/Inf has clearly lower error than the IEEE-aligned one.
    w4 = inputs.weight_cpu("student_t", 64, 1024, seed=1, layer=0)
    ours = orc.tensor_mse(w4, orc.FP4_E2M1, orc.PER_CHANNEL)
    ieee = orc.tensor_mse(w4, orc.FP4_E2M1_IEEE, orc.PER_CHANNEL)
    assert ours < ieee
