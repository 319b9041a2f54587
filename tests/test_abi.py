"""CPU-only checks of the C-ABI library: it loads, exports every symbol that include/mofq.h
declares, its static format facts agree with the paper's Table 3 / the oracle, and host-side
argument validation returns the documented error codes (no kernel is launched)."""
import ctypes as C
import os
import re

import pytest

import paper_2305_12356_b200 as mofq
from paper_2305_12356_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mofq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mofq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = mofq.lib()
    names = _declared_functions()
    assert {"mofq_quantize_tensor", "mofq_tensor_error", "mofq_layer_output_error", "mofq_select_formats"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_struct_layouts_match_header():
    assert C.sizeof(B.MofqTensor) == 40
    assert C.sizeof(B.MofqLayer) == 80
    assert C.sizeof(B.MofqConfig) == 4 * (2 + 4 + 7)
    assert C.sizeof(B.MofqResult) == 4 * (2 + 4 + 4 + 2)


def test_format_facts(orc):
    L = mofq.lib()
    for name, fid in B.FORMATS.items():
        assert L.mofq_format_bits(fid) == orc.format_bits(getattr(orc, name))
        assert L.mofq_format_max(fid) == orc.format_max(getattr(orc, name))
    assert L.mofq_format_bits(99) == -1 and L.mofq_format_max(-3) == 0.0
    assert L.mofq_format_max(B.FP4_E2M1) == 6.0          # Table 3, "w/o NaN&Inf": largest value 6
    assert L.mofq_format_max(B.FP4_E2M1_IEEE) == 3.0      # Table 3, "w/ NaN&Inf": largest value 3


def _desc(ptr=0x10000, dtype=B.F16, rows=16, cols=256, ld=256):
    return B.MofqTensor(ptr, dtype, 0, rows, cols, ld)


def _tensor_error(desc, formats, gran, gran2=B.GRAN_NONE, group=0, ws=0x20000, ws_bytes=1 << 20, out=0x30000):
    fm = (C.c_int32 * len(formats))(*formats)
    return mofq.lib().mofq_tensor_error(C.byref(desc), fm, len(formats), gran, gran2, group, out, ws, ws_bytes, None)


def test_argument_validation_returns_error_codes():
    L = mofq.lib()
    ok = [B.INT4, B.FP4_E2M1]
    assert _tensor_error(_desc(ptr=0), ok, B.PER_CHANNEL) == -1                    # NULL data
    assert _tensor_error(_desc(rows=0), ok, B.PER_CHANNEL) == -1
    assert _tensor_error(_desc(dtype=7), ok, B.PER_CHANNEL) == -1
    assert _tensor_error(_desc(ld=128), ok, B.PER_CHANNEL) == -1                   # ld < cols
    assert _tensor_error(_desc(ptr=0x10008), ok, B.PER_CHANNEL) == -3              # misaligned data
    assert _tensor_error(_desc(cols=252, ld=252), ok, B.PER_CHANNEL) == -3         # cols % 8
    assert _tensor_error(_desc(), [B.INT4, B.FP8_E4M3], B.PER_CHANNEL) == -2       # mixed bit-widths
    assert _tensor_error(_desc(), [B.INT4, 42], B.PER_CHANNEL) == -1               # bad format
    assert _tensor_error(_desc(), ok, B.PER_GROUP, group=96) == -2                 # group not a power of two
    assert _tensor_error(_desc(cols=320, ld=320), ok, B.PER_GROUP, group=128) == -2  # cols % group
    assert _tensor_error(_desc(), ok, 5) == -1                                     # bad granularity
    assert _tensor_error(_desc(), ok, B.PER_CHANNEL, ws_bytes=1024) == -4          # workspace too small
    assert _tensor_error(_desc(), ok, B.PER_CHANNEL, ws=0x20010) == -3             # workspace alignment
    assert _tensor_error(_desc(), ok, B.PER_CHANNEL, out=0) == -1
    assert _tensor_error(_desc(), ok, B.PER_CHANNEL, gran2=B.PER_CHANNEL) == -1    # same granularity twice
    d = _desc()
    assert L.mofq_quantize_tensor(C.byref(d), 17, B.PER_CHANNEL, 0, None, None, None, None, 0x20000, 1 << 20, None) == -1
    assert L.mofq_quantize_tensor(C.byref(d), B.INT4, B.PER_CHANNEL, 0, None, None, None, None, None, 1 << 20, None) == -1
    cfg = mofq.make_config(4, ["INT4", "FP4_E2M1"])
    layers = (B.MofqLayer * 1)()
    layers[0].W = _desc()
    assert L.mofq_select_formats(layers, 0, C.byref(cfg), 0x40000, 0x20000, 1 << 20, None) == -1
    assert L.mofq_select_formats(layers, 1, C.byref(cfg), None, 0x20000, 1 << 20, None) == -1
    cfg.bit_width = 5
    assert L.mofq_select_formats(layers, 1, C.byref(cfg), 0x40000, 0x20000, 1 << 20, None) == -1
    cfg = mofq.make_config(8, ["INT4"])
    assert L.mofq_select_formats(layers, 1, C.byref(cfg), 0x40000, 0x20000, 1 << 20, None) == -2
    assert L.mofq_status_string(-4) == b"workspace too small"


def test_workspace_size_queries():
    L = mofq.lib()
    d = _desc()
    n = L.mofq_tensor_workspace_bytes(C.byref(d))
    assert n >= 256 and n % 256 == 0
    cfg = mofq.make_config(4, ["INT4", "FP4_E2M1"], w_gran="group", w_group=128)
    layers = (B.MofqLayer * 2)()
    layers[0].W = _desc(rows=64, cols=512, ld=512)
    layers[1].W = _desc(rows=32, cols=1024, ld=1024)
    dev = L.mofq_workspace_bytes(layers, 2, C.byref(cfg))
    host = L.mofq_host_workspace_bytes(layers, 2, C.byref(cfg))
    assert host >= dev + 64 * 512 * 2 + 2 * B.RESULT_BYTES


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libmofq.so"))
    with pytest.raises(B.MofqError):
        B.lib()


def test_added_entry_points_validate_their_arguments():
    L = mofq.lib()
    d = _desc()
    fm = (C.c_int32 * 2)(B.INT4, B.FP4_E2M1)
    vp = C.c_void_p
    # block-wise selection: channel or group only, at most three candidates, outputs required
    assert L.mofq_select_blocks(C.byref(d), fm, 2, B.PER_TENSOR, 0, vp(0x50000), None, vp(0x30000), vp(0x20000), 1 << 20, None) == -2
    assert L.mofq_select_blocks(C.byref(d), fm, 2, B.PER_CHANNEL, 0, None, None, vp(0x30000), vp(0x20000), 1 << 20, None) == -1
    assert L.mofq_select_blocks(C.byref(d), fm, 2, B.PER_GROUP, 96, vp(0x50000), None, vp(0x30000), vp(0x20000), 1 << 20, None) == -2
    four = (C.c_int32 * 4)(B.INT4, B.FP4_E2M1, B.FP4_E2M1_IEEE, B.INT4)
    assert L.mofq_select_blocks(C.byref(d), four, 4, B.PER_CHANNEL, 0, vp(0x50000), None, vp(0x30000), vp(0x20000), 1 << 20, None) == -1
    assert L.mofq_select_blocks(C.byref(d), fm, 2, B.PER_CHANNEL, 0, vp(0x50000), None, vp(0x30000), vp(0x20000), 64, None) == -4
    # calibration scales
    assert L.mofq_absmax_update(C.byref(d), None, None) == -1
    assert L.mofq_absmax_update(C.byref(_desc(ptr=0)), vp(0x30000), None) == -1
    assert L.mofq_tensor_error_scaled(C.byref(d), fm, 2, None, vp(0x30000), vp(0x20000), 1 << 20, None) == -1
    assert L.mofq_tensor_error_scaled(C.byref(d), fm, 0, vp(0x60000), vp(0x30000), vp(0x20000), 1 << 20, None) == -1
    mixed = (C.c_int32 * 2)(B.INT4, B.FP8_E4M3)
    assert L.mofq_tensor_error_scaled(C.byref(d), mixed, 2, vp(0x60000), vp(0x30000), vp(0x20000), 1 << 20, None) == -2
    # emission of the selected formats
    cfg = mofq.make_config(4, ["INT4", "FP4_E2M1"], w_gran="group", w_group=128)
    layers = (B.MofqLayer * 1)()
    layers[0].W = _desc()
    out = (B.MofqPacked * 1)()
    assert L.mofq_emit_selected(layers, 1, C.byref(cfg), vp(0x40000), out, None, vp(0x20000), 256, None) == -1   # NULL destinations
    out[0].codes, out[0].scales = 0x70000, 0x80000
    assert L.mofq_emit_selected(layers, 1, C.byref(cfg), None, out, None, vp(0x20000), 256, None) == -1
    assert L.mofq_emit_selected(layers, 1, C.byref(cfg), vp(0x40000), out, None, vp(0x20000), 16, None) == -4
    bad = mofq.make_config(4, ["INT4", "FP4_E2M1"], w_gran="group", w_group=96)
    assert L.mofq_emit_selected(layers, 1, C.byref(bad), vp(0x40000), out, None, vp(0x20000), 256, None) == -2
    # diagnostics
    assert L.mofq_diag_scale_pair(B.INT4, None, vp(0x30000), vp(0x30100), 4, None) == -1
    assert L.mofq_diag_scale_pair(77, vp(0x20000), vp(0x30000), vp(0x30100), 4, None) == -1
