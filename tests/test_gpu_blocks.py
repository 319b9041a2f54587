"""GPU parity: block-wise (per-channel / per-group) format selection against the CPU oracle (-m gpu).

Bars: every block's errors within 1e-5 relative; the whole-tensor and mixture MSEs within 1e-5; the format map
bit-exact wherever the oracle's two best errors differ by more than the error tolerance (where they are closer
either winner is correct, and the test then checks that the kernel's pick is one of the near-minimal ones).
"""
import numpy as np
import pytest
import torch

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import inputs

from gpu_util import host, orc_gran, rel_err

pytestmark = pytest.mark.gpu

RTOL = 1e-5


@pytest.fixture(scope="module")
def dev():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    mofq.lib()
    return torch.device("cuda:0")


def _tensor(dev, rows, cols, dtype, seed):
    """Rows alternate between heavy-tailed and flat value distributions so that both kinds of grid win somewhere."""
    w = torch.empty((rows, cols), dtype=torch.float16, device=dev)
    inputs.device_weight(w, "student_t", seed, 0)
    g = torch.Generator().manual_seed(seed)
    flat = ((torch.rand((rows, cols), generator=g) - 0.5) * 0.08).to(torch.float16).to(dev)
    w[1::2] = flat[1::2]
    return w if dtype == torch.float16 else (w.float() * 3.0).to(torch.bfloat16)


def _check(orc, x, names, gran, group):
    got = mofq.select_blocks(x, names, gran, group, want_block_sse=True)
    torch.cuda.synchronize()
    want = orc.select_blocks(host(x), [getattr(orc, n) for n in names], orc_gran(orc, gran), group)
    assert int(got["status"].item()) == 0
    sse = got["block_sse"].cpu().numpy().astype(np.float64)
    ref = want["block_sse"]
    nz = ref > 0
    assert rel_err(sse[nz], ref[nz]).max() < RTOL
    assert np.all(sse[~nz] == 0.0)
    # whole-tensor MSE per candidate, then the mixture
    n_el = x.numel()
    mse = got["mse"].cpu().numpy()
    assert rel_err(mse[:-1], ref.sum(axis=0) / n_el).max() < RTOL
    assert rel_err(mse[-1:], [want["mixed_mse"]]).max() < RTOL
    # the format map
    choice = got["choice"].cpu().numpy()
    srt = np.sort(ref, axis=1)
    clear = (srt[:, 1] - srt[:, 0] > 4 * RTOL * srt[:, 1]) if ref.shape[1] > 1 else np.ones(len(ref), bool)
    np.testing.assert_array_equal(choice[clear], want["choice"][clear])
    picked = ref[np.arange(len(ref)), choice]
    assert np.all(picked <= srt[:, 0] * (1 + 4 * RTOL) + 1e-300)               # near-ties: a near-minimal candidate
    return want, choice


@pytest.mark.parametrize("names", [["INT4", "FP4_E2M1"], ["FP4_E2M1_IEEE", "INT4", "FP4_E2M1"], ["INT8", "FP8_E4M3", "FP8_E5M2"], ["FP8_E5M2"]])
@pytest.mark.parametrize("gran,group", [("channel", 0), ("group", 128), ("group", 32), ("group", 256)])
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_block_selection_matches_oracle(orc, dev, names, gran, group, dtype):
    x = _tensor(dev, 203, 1536, dtype, 31)                                      # 203 rows: ragged against the warp teams
    want, choice = _check(orc, x, names, gran, group)
    if len(names) > 1 and gran == "channel":
        assert len(set(choice.tolist())) > 1                                     # the map does mix formats


@pytest.mark.parametrize("names,dtype", [(["INT4", "FP4_E2M1"], torch.float16), (["FP4_E2M1", "INT4"], torch.bfloat16),
                                         (["FP8_E4M3", "INT8"], torch.float16)])
def test_large_dense_tensor_takes_the_streamed_route(orc, dev, names, dtype):
    """8 Mi elements and more with group-128 blocks and the 4-bit pair go through the persistent TMA-fed kernel in its
    block-wise form (the 8-bit pair stays with the register-resident kernel): several tiles per CTA, a ragged last tile
    (4099 rows), winners that mix, a zero group and a planted Inf's status."""
    x = _tensor(dev, 4099, 2048, dtype, 36)
    x[7, 128:256] = 0
    want, choice = _check(orc, x, names, "group", 128)
    assert len(set(choice.tolist())) > 1
    assert choice[7 * 16 + 1] == 0                                                # the zero group: a tie, first candidate
    again = mofq.select_blocks(x, names, "group", 128, want_block_sse=True)
    np.testing.assert_array_equal(again["choice"].cpu().numpy(), choice)         # same launch geometry, same sums
    x[4098, 2047] = float("inf")
    got = mofq.select_blocks(x, names, "group", 128)
    assert int(got["status"].item()) & mofq.binding.STATUS_NONFINITE_INPUT


def test_block_selection_odd_row_length_and_strided_view(orc, dev):
    full = _tensor(dev, 37, 1000 + 24, torch.float16, 32)
    view = full[:, 16:1016]                                                      # 1000 columns: 125 chunks per row, ld = 1024
    got = mofq.select_blocks(view, ["INT4", "FP4_E2M1"], "channel", want_block_sse=True)
    want = orc.select_blocks(host(view).contiguous(), [orc.INT4, orc.FP4_E2M1], orc.PER_CHANNEL)
    assert rel_err(got["block_sse"].cpu().numpy(), want["block_sse"]).max() < RTOL
    assert rel_err(got["mse"].cpu().numpy()[-1:], [want["mixed_mse"]]).max() < RTOL
    short = _tensor(dev, 9, 192, torch.float16, 33)                              # 24 chunks per row: fewer than a warp
    _check(orc, short, ["INT4", "FP4_E2M1"], "channel", 0)
    _check(orc, short, ["INT8", "FP8_E4M3"], "group", 8)                         # one chunk per block


def test_block_selection_degenerate_inputs(orc, dev):
    z = torch.zeros((5, 256), dtype=torch.float16, device=dev)
    got = mofq.select_blocks(z, ["FP4_E2M1", "INT4"], "group", 128, want_block_sse=True)
    assert got["choice"].cpu().tolist() == [0] * 10                              # ties keep the first candidate
    assert float(got["mse"].abs().max()) == 0.0
    x = _tensor(dev, 4, 256, torch.float16, 34)
    x[1, 5] = float("nan")
    got = mofq.select_blocks(x, ["INT4", "FP4_E2M1"], "channel")
    assert int(got["status"].item()) & mofq.binding.STATUS_NONFINITE_INPUT
    with pytest.raises(mofq.MofqError):
        mofq.select_blocks(x, ["INT4", "FP4_E2M1"], "tensor")                    # one block per tensor is select_formats


def test_mixture_beats_layerwise_choice_on_mixed_rows(orc, dev):
    x = _tensor(dev, 128, 2048, torch.float16, 35)
    got = mofq.select_blocks(x, ["INT4", "FP4_E2M1"], "channel")
    mse = got["mse"].cpu().numpy()
    assert mse[2] < min(mse[0], mse[1])                                          # finer selection lowers the error
