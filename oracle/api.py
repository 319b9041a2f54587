"""numpy-facing wrapper over the C oracle (test infrastructure; see mofq_oracle.c).

Tensors are passed as 2-D arrays of raw 16-bit patterns plus a dtype tag, so that both sides of a
parity test consume exactly the same bits.  ``as_bits`` converts numpy float16 arrays and CPU
torch tensors (float16 / bfloat16) without touching the values.
"""
import ctypes as C

import numpy as np

from .build import build

INT4, INT8, FP4_E2M1, FP4_E2M1_IEEE, FP8_E4M3, FP8_E5M2 = range(6)
PER_TENSOR, PER_CHANNEL, PER_GROUP = range(3)
F16, BF16 = 0, 1

FORMAT_NAMES = {INT4: "INT4", INT8: "INT8", FP4_E2M1: "FP4_E2M1", FP4_E2M1_IEEE: "FP4_E2M1_IEEE",
                FP8_E4M3: "FP8_E4M3", FP8_E5M2: "FP8_E5M2"}

_lib = None


def lib():
    global _lib
    if _lib is None:
        import os
        L = C.CDLL(os.environ.get("MOFQ_ORACLE_LIB") or build())   # the override serves the mutation test only
        u16p, u8p, f32p, f64p = (C.POINTER(t) for t in (C.c_uint16, C.c_uint8, C.c_float, C.c_double))
        i64 = C.c_int64
        L.orc_format_bits.restype = C.c_int
        L.orc_format_bits.argtypes = [C.c_int]
        L.orc_format_max.restype = C.c_double
        L.orc_format_max.argtypes = [C.c_int]
        L.orc_decode.restype = C.c_double
        L.orc_decode.argtypes = [C.c_int, C.c_int]
        for name in ("orc_encode_fp_arith", "orc_encode_fp_table"):
            getattr(L, name).restype = C.c_int
            getattr(L, name).argtypes = [C.c_int, C.c_float, C.c_int]
        L.orc_encode_int.restype = C.c_int
        L.orc_encode_int.argtypes = [C.c_int, C.c_float]
        L.orc_scale_from_absmax.restype = None
        L.orc_scale_from_absmax.argtypes = [C.c_int, C.c_float, f32p, f32p]
        L.orc_load.restype = C.c_float
        L.orc_load.argtypes = [u16p, C.c_int]
        L.orc_store.restype = C.c_uint16
        L.orc_store.argtypes = [C.c_float, C.c_int]
        L.orc_absmax.restype = None
        L.orc_absmax.argtypes = [u16p, C.c_int, i64, i64, i64, C.c_int, C.c_int, f32p]
        L.orc_quantize.restype = C.c_int
        L.orc_quantize.argtypes = [u16p, C.c_int, i64, i64, i64, C.c_int, C.c_int, C.c_int, f32p,
                                   u8p, f32p, u16p, f64p]
        L.orc_pack4.restype = None
        L.orc_pack4.argtypes = [u8p, i64, u8p]
        L.orc_tensor_mse.restype = C.c_int
        L.orc_tensor_mse.argtypes = [u16p, C.c_int, i64, i64, i64, C.c_int, C.c_int, C.c_int, f64p]
        L.orc_layer_output_error.restype = C.c_int
        L.orc_layer_output_error.argtypes = [u16p, C.c_int, i64, i64, u16p, C.c_int, i64, i64, i64,
                                             C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, f64p, f64p]
        L.orc_select.restype = C.c_int
        L.orc_select.argtypes = [f64p, C.c_int]
        L.orc_block_sse.restype = C.c_int
        L.orc_block_sse.argtypes = [u16p, C.c_int, i64, i64, i64, C.c_int, C.c_int, C.c_int, f64p]
        L.orc_select_blocks.restype = C.c_int
        L.orc_select_blocks.argtypes = [u16p, C.c_int, i64, i64, i64, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int,
                                        u8p, f64p, f64p]
        L.orc_num_threads.restype = C.c_int
        L.orc_num_threads.argtypes = []
        L.orc_crosscheck_fp.restype = C.c_int64
        L.orc_crosscheck_fp.argtypes = [C.c_int, C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(C.c_uint32)]
        _lib = L
    return _lib


def _ptr(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def as_bits(x):
    """Return (uint16 2-D C-contiguous array of raw bit patterns, dtype tag)."""
    if isinstance(x, tuple):
        bits, dt = x
        return np.ascontiguousarray(bits, dtype=np.uint16), dt
    if isinstance(x, np.ndarray):
        if x.dtype != np.float16:
            raise TypeError("numpy input must be float16 (pass (uint16 bits, BF16) for bfloat16)")
        return np.ascontiguousarray(x).view(np.uint16), F16
    import torch  # CPU tensors only
    if x.dtype == torch.float16:
        dt = F16
    elif x.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise TypeError(f"unsupported dtype {x.dtype}")
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16), dt


def bits_to_float(bits, dt):
    """Exact float64 values of raw 16-bit patterns (through the oracle's own loader)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, np.float64)
    L, flat, of = lib(), bits.reshape(-1), out.reshape(-1)
    for i in range(flat.size):
        of[i] = L.orc_load(_ptr(flat[i:i + 1], C.c_uint16), dt)
    return out


def num_threads():
    return lib().orc_num_threads()


def format_bits(fmt):
    return lib().orc_format_bits(fmt)


def format_max(fmt):
    return lib().orc_format_max(fmt)


def decode(fmt, code):
    return lib().orc_decode(fmt, int(code))


def decode_table(fmt):
    """All 2^k code values in code order (NaN for reserved codes)."""
    return np.array([decode(fmt, c) for c in range(1 << format_bits(fmt))])


def encode_fp_arith(fmt, t, negative=None):
    t = np.float32(t)
    neg = bool(np.signbit(t)) if negative is None else bool(negative)
    return lib().orc_encode_fp_arith(fmt, float(t), int(neg))


def encode_fp_table(fmt, t, negative=None):
    t = np.float32(t)
    neg = bool(np.signbit(t)) if negative is None else bool(negative)
    return lib().orc_encode_fp_table(fmt, float(t), int(neg))


def encode_int(fmt, t):
    return lib().orc_encode_int(fmt, float(np.float32(t)))


def scale_from_absmax(fmt, absmax):
    s, i = C.c_float(), C.c_float()
    lib().orc_scale_from_absmax(fmt, float(np.float32(absmax)), C.byref(s), C.byref(i))
    return np.float32(s.value), np.float32(i.value)


def n_scales(gran, rows, cols, group):
    return 1 if gran == PER_TENSOR else rows if gran == PER_CHANNEL else rows * (cols // group)


def absmax(x, gran, group=0):
    bits, dt = as_bits(x)
    rows, cols = bits.shape
    out = np.empty(n_scales(gran, rows, cols, group), np.float32)
    lib().orc_absmax(_ptr(bits, C.c_uint16), dt, rows, cols, cols, gran, group, _ptr(out, C.c_float))
    return out


def quantize(x, fmt, gran, group=0, scales_in=None, want_dequant=False):
    """Returns dict(codes uint8 [rows, cols] unpacked, scales float32, sse float, dequant uint16 bits or None)."""
    bits, dt = as_bits(x)
    rows, cols = bits.shape
    ns = n_scales(gran, rows, cols, group)
    codes = np.empty((rows, cols), np.uint8)
    scales = np.empty(ns, np.float32)
    deq = np.empty((rows, cols), np.uint16) if want_dequant else None
    sse = C.c_double()
    sin = None
    if scales_in is not None:
        sin = np.ascontiguousarray(scales_in, dtype=np.float32)
        assert sin.size == ns
    rc = lib().orc_quantize(_ptr(bits, C.c_uint16), dt, rows, cols, cols, fmt, gran, group,
                            _ptr(sin, C.c_float) if sin is not None else None,
                            _ptr(codes, C.c_uint8), _ptr(scales, C.c_float),
                            _ptr(deq, C.c_uint16) if deq is not None else None, C.byref(sse))
    if rc:
        raise ValueError("oracle: bad argument")
    return dict(codes=codes, scales=scales, sse=sse.value, dequant=deq)


def pack4(codes):
    flat = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    out = np.empty((flat.size + 1) // 2, np.uint8)
    lib().orc_pack4(_ptr(flat, C.c_uint8), flat.size, _ptr(out, C.c_uint8))
    return out


def tensor_mse(x, fmt, gran, group=0):
    bits, dt = as_bits(x)
    rows, cols = bits.shape
    mse = C.c_double()
    rc = lib().orc_tensor_mse(_ptr(bits, C.c_uint16), dt, rows, cols, cols, fmt, gran, group, C.byref(mse))
    if rc:
        raise ValueError("oracle: bad argument")
    return mse.value


def layer_output_error(X, W, fmt, is_w_only, w_gran=PER_CHANNEL, w_group=0, a_gran=PER_TENSOR, a_group=0):
    """Returns (mse, nsr) of Y = X W^T when W (and X unless is_w_only) are quantised to fmt."""
    xb, xdt = as_bits(X)
    wb, wdt = as_bits(W)
    T, n_in = xb.shape
    out, n_in2 = wb.shape
    assert n_in == n_in2
    mse, nsr = C.c_double(), C.c_double()
    rc = lib().orc_layer_output_error(_ptr(xb, C.c_uint16), xdt, T, n_in, _ptr(wb, C.c_uint16), wdt, out, n_in, n_in,
                                      fmt, int(bool(is_w_only)), w_gran, w_group, a_gran, a_group,
                                      C.byref(mse), C.byref(nsr))
    if rc:
        raise ValueError("oracle: bad argument")
    return mse.value, nsr.value


def select(errors):
    e = np.ascontiguousarray(errors, dtype=np.float64)
    return lib().orc_select(_ptr(e, C.c_double), e.size)


def block_sse(x, fmt, gran, group=0):
    """Sum of squared errors of every scale block (row or group), each quantised with its own abs-max scale."""
    bits, dt = as_bits(x)
    rows, cols = bits.shape
    out = np.empty(n_scales(gran, rows, cols, group), np.float64)
    if lib().orc_block_sse(_ptr(bits, C.c_uint16), dt, rows, cols, cols, fmt, gran, group, _ptr(out, C.c_double)):
        raise ValueError("oracle: bad argument")
    return out


def select_blocks(x, fmts, gran, group=0):
    """Block-wise format selection.  Returns dict(choice uint8 [blocks], block_sse float64 [blocks, n], mixed_mse)."""
    bits, dt = as_bits(x)
    rows, cols = bits.shape
    nb = n_scales(gran, rows, cols, group)
    fm = (C.c_int * len(fmts))(*fmts)
    choice = np.empty(nb, np.uint8)
    sse = np.empty((nb, len(fmts)), np.float64)
    mixed = C.c_double()
    if lib().orc_select_blocks(_ptr(bits, C.c_uint16), dt, rows, cols, cols, fm, len(fmts), gran, group,
                               _ptr(choice, C.c_uint8), _ptr(sse, C.c_double), C.byref(mixed)):
        raise ValueError("oracle: bad argument")
    return dict(choice=choice, block_sse=sse, mixed_mse=mixed.value)


def crosscheck_fp(fmt, lo_bits, hi_bits, stride=1):
    first = C.c_uint32()
    bad = lib().orc_crosscheck_fp(fmt, lo_bits, hi_bits, stride, C.byref(first))
    return bad, first.value


def mofq_select(layers, candidates, metric="tensor", gran=PER_CHANNEL, group=0, is_w_only=True,
                a_gran=PER_TENSOR, a_group=0):
    """Algorithm 1 over a list of layers.  layers: list of W (tensor metric) or (W, X) pairs.

    Returns a list of dict(chosen=index into candidates, errors=[...], nsr=[...] or None).
    """
    results = []
    for layer in layers:
        errs, nsrs = [], []
        for fmt in candidates:
            if metric == "tensor":
                W = layer[0] if isinstance(layer, (tuple, list)) and not _is_bits_pair(layer) else layer
                errs.append(tensor_mse(W, fmt, gran, group))
            else:
                W, X = layer
                m, n = layer_output_error(X, W, fmt, is_w_only, gran, group, a_gran, a_group)
                errs.append(m)
                nsrs.append(n)
        results.append(dict(chosen=select(errs), errors=errs, nsr=nsrs or None))
    return results


def _is_bits_pair(obj):
    return (isinstance(obj, tuple) and len(obj) == 2 and isinstance(obj[0], np.ndarray)
            and obj[0].dtype == np.uint16 and isinstance(obj[1], int))
