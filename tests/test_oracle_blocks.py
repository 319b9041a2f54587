"""Pins for the oracle's block-wise (finer than a layer) format selection (CPU only).

The block errors are fixed from outside the new code: a block scored alone as a tensor of its own must give
the same error, the blocks must add up to the tensor error, a hand-worked two-row tensor has a known answer
in exact rational arithmetic, and mixing formats per block can never be worse than the best single format.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

NAMES4 = ["INT4", "FP4_E2M1"]
NAMES8 = ["INT8", "FP8_E4M3", "FP8_E5M2"]


def _rand16(shape, seed, scale=0.02, dtype=torch.float16):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(shape, generator=g) * scale
    x[torch.rand(shape, generator=g) < 0.01] *= 8.0          # a few outliers so that the formats disagree per block
    return x.to(dtype)


@pytest.mark.parametrize("name", NAMES4 + NAMES8 + ["FP4_E2M1_IEEE"])
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_block_equals_the_slice_scored_as_its_own_tensor(orc, name, dtype):
    fmt = getattr(orc, name)
    x = _rand16((7, 384), 5, dtype=dtype)
    rows = orc.block_sse(x, fmt, orc.PER_CHANNEL)
    groups = orc.block_sse(x, fmt, orc.PER_GROUP, 128)
    assert rows.shape == (7,) and groups.shape == (21,)
    for r in range(7):
        alone = orc.quantize(x[r:r + 1].contiguous(), fmt, orc.PER_TENSOR)["sse"]
        assert rows[r] == pytest.approx(alone, rel=1e-12)
        for g in range(3):
            alone = orc.quantize(x[r:r + 1, 128 * g:128 * (g + 1)].contiguous(), fmt, orc.PER_TENSOR)["sse"]
            assert groups[3 * r + g] == pytest.approx(alone, rel=1e-12)          # row-major, groups left to right


@pytest.mark.parametrize("name", NAMES4 + NAMES8)
@pytest.mark.parametrize("gran,group", [("PER_CHANNEL", 0), ("PER_GROUP", 64), ("PER_TENSOR", 0)])
def test_blocks_add_up_to_the_tensor_error(orc, name, gran, group):
    fmt, g = getattr(orc, name), getattr(orc, gran)
    x = _rand16((9, 320), 6)
    assert orc.block_sse(x, fmt, g, group).sum() == pytest.approx(orc.quantize(x, fmt, g, group)["sse"], rel=1e-12)


def test_hand_worked_two_rows(orc):
    # row 0 lies on the INT4 grid (abs-max 7 -> scale 1), row 1 on the FP4 grid (abs-max 6 -> scale 1)
    x = torch.tensor([[7.0, 3.0, -7.0, 1.0, 5.0, -2.0, 0.0, 4.0],
                      [6.0, 0.5, 0.5, -6.0, 1.5, -4.0, 2.0, 1.0]], dtype=torch.float16)
    got = orc.select_blocks(x, [orc.INT4, orc.FP4_E2M1], orc.PER_CHANNEL)
    assert got["choice"].tolist() == [0, 1]
    assert got["block_sse"][0, 0] == 0.0 and got["block_sse"][1, 1] == 0.0
    assert got["mixed_mse"] == 0.0
    # the losing entries, in exact rationals: FP4 on row 0 has scale RN32(7/6), INT4 on row 1 has scale RN32(6/7)
    grid_fp = [Fraction(v) for v in (0, 0.5, 1, 1.5, 2, 3, 4, 6)]
    grid_fp = sorted(set(grid_fp + [-v for v in grid_fp]))
    grid_int = [Fraction(v) for v in range(-8, 8)]
    for row, grid, q, col in ((0, grid_fp, 6, 1), (1, grid_int, 7, 0)):
        amax = np.float32(max(abs(float(v)) for v in x[row]))
        s = Fraction(float(np.float32(amax / np.float32(q))))
        sse = Fraction(0)
        for v in x[row].tolist():
            # nearest grid point of the exact v / s: none of these values sits within an fp32 rounding of a tie
            best = min(grid, key=lambda gpt: abs(Fraction(v) - gpt * s))
            sse += (Fraction(v) - best * s) ** 2
        assert got["block_sse"][row, col] == pytest.approx(float(sse), rel=1e-12)


@pytest.mark.parametrize("names", [NAMES4, NAMES8, ["FP4_E2M1", "INT4", "FP4_E2M1_IEEE"]])
@pytest.mark.parametrize("gran,group", [("PER_CHANNEL", 0), ("PER_GROUP", 128)])
def test_mixture_is_never_worse_than_the_best_single_format(orc, names, gran, group):
    fmts, g = [getattr(orc, n) for n in names], getattr(orc, gran)
    x = _rand16((24, 512), 7)
    flat = (torch.rand((12, 512), generator=torch.Generator().manual_seed(8)) - 0.5) * 0.1
    x[::2] = flat.to(torch.float16)                                                 # flat rows favour the integer grid
    got = orc.select_blocks(x, fmts, g, group)
    single = [orc.tensor_mse(x, f, g, group) for f in fmts]
    assert got["mixed_mse"] <= min(single) * (1 + 1e-12)
    sse = got["block_sse"]
    np.testing.assert_array_equal(got["choice"], np.argmin(sse, axis=1))          # argmin returns the first minimum too
    assert got["mixed_mse"] == pytest.approx(sse.min(axis=1).sum() / x.numel(), rel=1e-12)
    assert len(set(got["choice"].tolist())) > 1                                     # the fixture does mix formats


def test_ties_keep_the_first_candidate(orc):
    z = torch.zeros((3, 128), dtype=torch.float16)                                  # every format is exact on zeros
    assert orc.select_blocks(z, [orc.FP4_E2M1, orc.INT4], orc.PER_CHANNEL)["choice"].tolist() == [0, 0, 0]
    assert orc.select_blocks(z, [orc.INT4, orc.FP4_E2M1], orc.PER_GROUP, 64)["choice"].tolist() == [0] * 6
