"""Pins for the oracle's number formats and grid rounding (CPU only).

Sources of truth used here, none of which is the oracle itself: Table 3 of the paper, the paper's
statement that a k-bit format has 2^k codes and that INT codes are 1 apart, numpy's float16
and torch's float8 decoders/casts (library routines for formats the paper leaves to hardware
convention), and hand-made tie grids.
"""
import math
import os

import numpy as np
import pytest
import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_rows(name):
    rows = []
    for line in open(os.path.join(GOLD, name)):
        line = line.split("#")[0].split()
        if line:
            rows.append(line)
    return rows


def _same(a, b):
    if math.isnan(b):
        return math.isnan(a)
    return a == b and math.copysign(1, a) == math.copysign(1, b)


# ---- Table 3 -----------------------------------------------------------------------------------
def test_fp4_table3_both_variants(orc):
    for code, ieee, ours in _read_rows("fp4_e2m1_table3.txt"):
        code = int(code)
        want_ours = float(ours)
        got = orc.decode(orc.FP4_E2M1, code)
        assert _same(got, want_ours), (code, got, want_ours)
        got_ieee = orc.decode(orc.FP4_E2M1_IEEE, code)
        if ieee in ("Inf", "NaN"):           # reserved in the IEEE-aligned variant
            assert math.isnan(got_ieee)
        else:
            assert _same(got_ieee, float(ieee))
    assert orc.format_max(orc.FP4_E2M1) == 6 and orc.format_max(orc.FP4_E2M1_IEEE) == 3


def test_reallocated_codes_give_4_and_6(orc):
    # Section 4.2: re-using the four Inf/NaN codes adds exactly +-4 and +-6.
    ours = {v for v in orc.decode_table(orc.FP4_E2M1)}
    ieee = {v for v in orc.decode_table(orc.FP4_E2M1_IEEE) if not math.isnan(v)}
    assert ours - ieee == {4.0, 6.0, -4.0, -6.0}


# ---- code counts, monotonicity, library decodes --------------------------------------------------
@pytest.mark.parametrize("name,finite,distinct,vmax,vmin", [
    ("FP4_E2M1", 16, 15, 6.0, 0.5),
    ("FP4_E2M1_IEEE", 12, 11, 3.0, 0.5),
    ("FP8_E4M3", 254, 253, 448.0, 2.0 ** -9),
    ("FP8_E5M2", 248, 247, 57344.0, 2.0 ** -16),
    ("INT4", 16, 16, 7.0, 1.0),
    ("INT8", 256, 256, 127.0, 1.0),
])
def test_enumeration_counts(orc, name, finite, distinct, vmax, vmin):
    fmt = getattr(orc, name)
    tab = orc.decode_table(fmt)
    assert tab.size == 2 ** orc.format_bits(fmt)          # "2^8 = 256 values" for an 8-bit format
    fin = tab[~np.isnan(tab)]
    assert fin.size == finite
    assert np.unique(fin).size == distinct                # +0 and -0 coincide for FP formats
    assert fin.max() == vmax == orc.format_max(fmt)
    assert np.abs(fin[fin != 0]).min() == vmin


@pytest.mark.parametrize("name", ["INT4", "INT8"])
def test_int_codes_are_consecutive_integers(orc, name):
    fmt = getattr(orc, name)
    k = orc.format_bits(fmt)
    vals = np.sort(orc.decode_table(fmt))
    assert np.all(np.diff(vals) == 1)                     # "difference of 1 between two consecutive numbers"
    assert vals[0] == -(2 ** (k - 1)) and vals[-1] == 2 ** (k - 1) - 1
    # two's complement layout
    for c in range(2 ** k):
        assert orc.decode(fmt, c) == (c if c < 2 ** (k - 1) else c - 2 ** k)


@pytest.mark.parametrize("name", ["FP4_E2M1", "FP4_E2M1_IEEE", "FP8_E4M3", "FP8_E5M2"])
def test_fp_magnitudes_increase_with_code(orc, name):
    fmt = getattr(orc, name)
    half = 2 ** (orc.format_bits(fmt) - 1)
    tab = orc.decode_table(fmt)
    pos = tab[:half]
    pos = pos[~np.isnan(pos)]
    assert np.all(np.diff(pos) > 0)
    neg = tab[half:]
    for c in range(pos.size):
        assert _same(neg[c], -pos[c])


def test_e5m2_decode_matches_numpy_float16(orc):
    # E5M2 is binary16 with the low 8 mantissa bits dropped: code c has the value of half bits c<<8.
    codes = np.arange(256, dtype=np.uint16)
    lib = (codes << 8).view(np.float16).astype(np.float64)
    for c in range(256):
        got = orc.decode(orc.FP8_E5M2, c)
        if not np.isfinite(lib[c]):
            assert math.isnan(got)
        else:
            assert _same(got, float(lib[c]))


def test_fp8_decode_matches_torch_float8(orc):
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    for name, tdt in (("FP8_E4M3", torch.float8_e4m3fn), ("FP8_E5M2", torch.float8_e5m2)):
        lib = codes.view(tdt).to(torch.float64).numpy()
        for c in range(256):
            got = orc.decode(getattr(orc, name), c)
            if not np.isfinite(lib[c]):
                assert math.isnan(got), (name, c)
            else:
                assert _same(got, float(lib[c])), (name, c, got, lib[c])


# ---- rounding ----------------------------------------------------------------------------------------
def test_e2m1_midpoints_round_to_even_code(orc):
    for mid, mag, code in _read_rows("e2m1_midpoints.txt"):
        mid, mag, code = float(mid), float(mag), int(code)
        for enc in (orc.encode_fp_arith, orc.encode_fp_table):
            assert enc(orc.FP4_E2M1, mid) == code
            assert orc.decode(orc.FP4_E2M1, enc(orc.FP4_E2M1, mid)) == mag
            assert enc(orc.FP4_E2M1, -mid) == code | 8
        # one binary32 ulp on either side goes to the nearer neighbour
        lo, hi = np.nextafter(np.float32(mid), np.float32(0)), np.nextafter(np.float32(mid), np.float32(10))
        tab = orc.decode_table(orc.FP4_E2M1)[:8]
        below = tab[tab < mid].max()
        above = tab[tab > mid].min()
        assert orc.decode(orc.FP4_E2M1, orc.encode_fp_arith(orc.FP4_E2M1, lo)) == below
        assert orc.decode(orc.FP4_E2M1, orc.encode_fp_arith(orc.FP4_E2M1, hi)) == above


@pytest.mark.parametrize("name", ["FP4_E2M1", "FP4_E2M1_IEEE", "FP8_E4M3", "FP8_E5M2"])
def test_all_midpoints_and_grid_points(orc, name):
    fmt = getattr(orc, name)
    half = 2 ** (orc.format_bits(fmt) - 1)
    pos = orc.decode_table(fmt)[:half]
    pos = pos[~np.isnan(pos)]
    for c, v in enumerate(pos):                           # decode(encode(v)) == v for every grid value
        for enc in (orc.encode_fp_arith, orc.encode_fp_table):
            assert enc(fmt, v) == c
            assert enc(fmt, -v, True) == c | half
    for c in range(pos.size - 1):                         # every midpoint -> even code
        mid = (pos[c] + pos[c + 1]) / 2
        assert float(np.float32(mid)) == mid
        want = c if c % 2 == 0 else c + 1
        assert orc.encode_fp_arith(fmt, mid) == want
        assert orc.encode_fp_table(fmt, mid) == want
    # saturation (only reachable with caller-supplied scales); reserved codes never appear
    for big in (pos[-1] * 1.01, pos[-1] * 4, 3.0e38, float("inf")):
        assert orc.encode_fp_arith(fmt, big) == pos.size - 1
        assert orc.encode_fp_arith(fmt, -big) == (pos.size - 1) | half


@pytest.mark.parametrize("name", ["FP8_E4M3", "FP8_E5M2"])
def test_fp8_rounding_matches_torch_cast(orc, name):
    # torch's float32 -> float8 cast is round-to-nearest-even; compare inside the finite range.
    fmt = getattr(orc, name)
    tdt = {"FP8_E4M3": torch.float8_e4m3fn, "FP8_E5M2": torch.float8_e5m2}[name]
    g = torch.Generator().manual_seed(5)
    vmax = orc.format_max(fmt)
    x = torch.cat([torch.randn(20000, generator=g) * s for s in (1e-3, 0.05, 1.0, 30.0, vmax / 3)])
    x = x[x.abs() <= vmax].float()
    lib_codes = x.to(tdt).view(torch.uint8).numpy()
    xn = x.numpy()
    for i in range(0, xn.size, 7):
        assert orc.encode_fp_arith(fmt, xn[i]) == int(lib_codes[i]), (xn[i],)


@pytest.mark.parametrize("name", ["INT4", "INT8"])
def test_int_rounding_ties_to_even_and_clamp(orc, name):
    fmt = getattr(orc, name)
    k = orc.format_bits(fmt)
    qmax = 2 ** (k - 1) - 1
    mask = 2 ** k - 1
    for n in range(-qmax - 1, qmax):
        mid = n + 0.5
        want = n if n % 2 == 0 else n + 1
        assert orc.encode_int(fmt, mid) == want & mask
        assert orc.encode_int(fmt, np.nextafter(np.float32(mid), np.float32(-1e9))) == n & mask
        assert orc.encode_int(fmt, np.nextafter(np.float32(mid), np.float32(1e9))) == (n + 1) & mask
    assert orc.encode_int(fmt, 1e9) == qmax
    assert orc.encode_int(fmt, -1e9) == (-qmax - 1) & mask
    assert orc.encode_int(fmt, -0.0) == 0


@pytest.mark.parametrize("name", ["FP4_E2M1", "FP4_E2M1_IEEE", "FP8_E4M3", "FP8_E5M2"])
def test_arith_and_table_rounding_agree(orc, name):
    # Two independent statements of "nearest grid point, ties to even" must agree on every
    # binary32 pattern near each rounding boundary and on a strided sweep of [0, 2*fmt_max].
    fmt = getattr(orc, name)
    hi = np.float32(2 * orc.format_max(fmt)).view(np.uint32)
    bad, first = orc.crosscheck_fp(fmt, 0, int(hi), 1021)
    assert bad == 0, hex(first)
    half = 2 ** (orc.format_bits(fmt) - 1)
    pos = orc.decode_table(fmt)[:half]
    pos = pos[~np.isnan(pos)]
    for c in range(pos.size - 1):
        mid = np.float32((pos[c] + pos[c + 1]) / 2).view(np.uint32)
        bad, first = orc.crosscheck_fp(fmt, int(mid) - 64, int(mid) + 64, 1)
        assert bad == 0, hex(first)


def test_arith_and_table_rounding_agree_exhaustive_e2m1(orc):
    # every positive binary32 pattern up to 2*fmt_max for the 4-bit format
    hi = np.float32(12.0).view(np.uint32)
    bad, first = orc.crosscheck_fp(orc.FP4_E2M1, 0, int(hi), 1)
    assert bad == 0, hex(first)


# ---- storage types ---------------------------------------------------------------------------------
def test_half_and_bf16_loaders_match_libraries(orc):
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    ref16 = bits.view(np.float16).astype(np.float64)
    got16 = orc.bits_to_float(bits[::13], orc.F16)
    np.testing.assert_array_equal(np.nan_to_num(got16, nan=-7.0), np.nan_to_num(ref16[::13], nan=-7.0))
    refbf = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    gotbf = orc.bits_to_float(bits[::13], orc.BF16)
    np.testing.assert_array_equal(np.nan_to_num(gotbf, nan=-7.0), np.nan_to_num(refbf[::13], nan=-7.0))


def test_half_and_bf16_store_match_libraries(orc):
    import ctypes as C
    g = np.random.default_rng(3)
    vals = np.concatenate([g.standard_normal(3000) * s for s in (1e-7, 1e-4, 1.0, 300.0, 6e4)]).astype(np.float32)
    L = orc.lib()
    got16 = np.array([L.orc_store(C.c_float(float(v)), orc.F16) for v in vals], dtype=np.uint16)
    with np.errstate(over="ignore"):
        np.testing.assert_array_equal(got16, vals.astype(np.float16).view(np.uint16))
    gotbf = np.array([L.orc_store(C.c_float(float(v)), orc.BF16) for v in vals], dtype=np.uint16)
    refbf = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(gotbf, refbf)
