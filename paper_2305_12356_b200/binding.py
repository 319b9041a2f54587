"""Thin ctypes binding over libmofq.so (include/mofq.h).  Argument marshalling only.

Every function takes torch CUDA tensors (device memory and streams are torch's), passes raw
pointers and sizes through the C ABI and returns torch tensors.  There is no CPU fallback: if the
shared library is missing the first call raises.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmofq.so")

MAX_CAND = 4
INT4, INT8, FP4_E2M1, FP4_E2M1_IEEE, FP8_E4M3, FP8_E5M2 = range(6)
PER_TENSOR, PER_CHANNEL, PER_GROUP = range(3)
GRAN_NONE = -1
F16, BF16 = 0, 1
TENSOR_MSE, LAYER_OUTPUT_MSE = 0, 1
STATUS_NONFINITE_INPUT, STATUS_SCALE_OVERFLOW, STATUS_TIMEOUT = 1, 2, 4

FORMATS = {"INT4": INT4, "INT8": INT8, "FP4_E2M1": FP4_E2M1, "FP4_E2M1_IEEE": FP4_E2M1_IEEE,
           "FP8_E4M3": FP8_E4M3, "FP8_E5M2": FP8_E5M2}
GRANS = {"tensor": PER_TENSOR, "channel": PER_CHANNEL, "group": PER_GROUP}


class MofqTensor(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("reserved", C.c_int32),
                ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64)]


class MofqLayer(C.Structure):
    _fields_ = [("W", MofqTensor), ("X", MofqTensor)]


class MofqConfig(C.Structure):
    _fields_ = [("bit_width", C.c_int32), ("n_candidates", C.c_int32), ("candidates", C.c_int32 * MAX_CAND),
                ("is_w_only", C.c_int32), ("w_gran", C.c_int32), ("w_group", C.c_int32), ("w_gran2", C.c_int32),
                ("a_gran", C.c_int32), ("a_group", C.c_int32), ("metric", C.c_int32)]


class MofqResult(C.Structure):
    _fields_ = [("chosen", C.c_int32), ("status", C.c_int32), ("error", C.c_float * MAX_CAND),
                ("nsr", C.c_float * MAX_CAND), ("rel_margin", C.c_float), ("reserved", C.c_int32)]


RESULT_BYTES = C.sizeof(MofqResult)

_lib = None


class MofqError(RuntimeError):
    pass


def lib():
    """Load libmofq.so; fail loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise MofqError(f"{LIB_PATH} not found: build it with `python -m paper_2305_12356_b200.build` "
                            "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, sz = C.c_void_p, C.c_size_t
        L.mofq_quantize_tensor.restype = C.c_int
        L.mofq_quantize_tensor.argtypes = [C.POINTER(MofqTensor), C.c_int, C.c_int, C.c_int, vp, vp, vp, vp, vp, sz, vp]
        L.mofq_tensor_error.restype = C.c_int
        L.mofq_tensor_error.argtypes = [C.POINTER(MofqTensor), C.POINTER(C.c_int32), C.c_int, C.c_int, C.c_int, C.c_int,
                                        vp, vp, sz, vp]
        L.mofq_tensor_error_noalloc.restype = C.c_int
        L.mofq_tensor_error_noalloc.argtypes = [C.POINTER(MofqTensor), C.POINTER(C.c_int32), C.c_int, C.c_int, C.c_int, C.c_int,
                                                vp, vp, vp]
        L.mofq_noalloc_scratch_bytes.restype = sz
        L.mofq_noalloc_scratch_bytes.argtypes = []
        L.mofq_emit_selected.restype = C.c_int
        L.mofq_emit_selected.argtypes = [vp, C.c_int, C.POINTER(MofqConfig), vp, vp, vp, vp, sz, vp]
        L.mofq_select_blocks.restype = C.c_int
        L.mofq_select_blocks.argtypes = [C.POINTER(MofqTensor), C.POINTER(C.c_int32), C.c_int, C.c_int, C.c_int, vp, vp, vp, vp, sz, vp]
        L.mofq_absmax_update.restype = C.c_int
        L.mofq_absmax_update.argtypes = [C.POINTER(MofqTensor), vp, vp]
        L.mofq_tensor_error_scaled.restype = C.c_int
        L.mofq_tensor_error_scaled.argtypes = [C.POINTER(MofqTensor), C.POINTER(C.c_int32), C.c_int, vp, vp, vp, sz, vp]
        L.mofq_diag_wait_expiry.restype = C.c_int
        L.mofq_diag_wait_expiry.argtypes = [vp, vp]
        L.mofq_diag_scale_pair.restype = C.c_int
        L.mofq_diag_scale_pair.argtypes = [C.c_int, vp, vp, vp, C.c_int64, vp]
        L.mofq_diag_fp_round.restype = C.c_int
        L.mofq_diag_fp_round.argtypes = [C.c_int, vp, vp, C.c_int64, vp]
        L.mofq_layer_output_error.restype = C.c_int
        L.mofq_layer_output_error.argtypes = [C.POINTER(MofqLayer), C.POINTER(MofqConfig), vp, vp, vp, sz, vp]
        for name in ("mofq_select_formats", "mofq_select_formats_host"):
            f = getattr(L, name)
            f.restype = C.c_int
            f.argtypes = [C.POINTER(MofqLayer), C.c_int, C.POINTER(MofqConfig), vp, vp, sz, vp]
        L.mofq_tensor_workspace_bytes.restype = sz
        L.mofq_tensor_workspace_bytes.argtypes = [C.POINTER(MofqTensor)]
        for name in ("mofq_workspace_bytes", "mofq_host_workspace_bytes"):
            f = getattr(L, name)
            f.restype = sz
            f.argtypes = [C.POINTER(MofqLayer), C.c_int, C.POINTER(MofqConfig)]
        L.mofq_format_bits.restype = C.c_int
        L.mofq_format_bits.argtypes = [C.c_int]
        L.mofq_format_max.restype = C.c_float
        L.mofq_format_max.argtypes = [C.c_int]
        L.mofq_status_string.restype = C.c_char_p
        L.mofq_status_string.argtypes = [C.c_int]
        _lib = L
    return _lib


def _check(rc):
    if rc != 0:
        raise MofqError(f"mofq error {rc}: {lib().mofq_status_string(rc).decode()}")


def _fmt(f):
    return FORMATS[f] if isinstance(f, str) else int(f)


def _gran(g):
    if g is None:
        return GRAN_NONE
    return GRANS[g] if isinstance(g, str) else int(g)


def _dtype_tag(t):
    if t.dtype == torch.float16:
        return F16
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def tensor_desc(t, require_cuda=True):
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 2-D tensor with unit inner stride")
    if require_cuda and not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    return MofqTensor(t.data_ptr(), _dtype_tag(t), 0, t.shape[0], t.shape[1], t.stride(0))


def make_config(bit_width, candidates, metric="tensor", is_w_only=True, w_gran="channel", w_group=0, w_gran2=None,
                a_gran="tensor", a_group=0):
    cfg = MofqConfig()
    cfg.bit_width = bit_width
    cfg.n_candidates = len(candidates)
    for i, c in enumerate(candidates):
        cfg.candidates[i] = _fmt(c)
    cfg.is_w_only = int(bool(is_w_only))
    cfg.w_gran, cfg.w_group, cfg.w_gran2 = _gran(w_gran), int(w_group), _gran(w_gran2)
    cfg.a_gran, cfg.a_group = _gran(a_gran), int(a_group)
    cfg.metric = {"tensor": TENSOR_MSE, "layer_output": LAYER_OUTPUT_MSE}[metric] if isinstance(metric, str) else metric
    return cfg


def _stream(device):
    return torch.cuda.current_stream(device).cuda_stream


def _workspace(nbytes, device):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


class PreparedLayers:
    """A marshalled layer list (ctypes array) that can be reused across calls; keeps the tensors alive."""

    def __init__(self, layers, require_cuda=True):
        self.layers = list(layers)
        self.array = _layer_array(self.layers, require_cuda)
        first = self.layers[0] if torch.is_tensor(self.layers[0]) else self.layers[0][0]
        self.device = first.device

    def __len__(self):
        return len(self.layers)


def prepare_layers(layers, require_cuda=True):
    return layers if isinstance(layers, PreparedLayers) else PreparedLayers(layers, require_cuda)


def _layer_array(layers, require_cuda=True):
    if isinstance(layers, PreparedLayers):
        return layers.array
    arr = (MofqLayer * len(layers))()
    for i, layer in enumerate(layers):
        W, X = (layer, None) if torch.is_tensor(layer) else layer
        arr[i].W = tensor_desc(W, require_cuda)
        if X is not None:
            arr[i].X = tensor_desc(X, require_cuda)
    return arr


def n_scales(gran, rows, cols, group):
    gran = _gran(gran)
    return 1 if gran == PER_TENSOR else rows if gran == PER_CHANNEL else rows * (cols // group)


def quantize_tensor(x, fmt, gran, group=0, scales_in=None, want_codes=True, want_scales=True, want_dequant=False,
                    workspace=None):
    """mofq_quantize_tensor.  Returns dict(codes uint8, scales float32, dequant like x, status int tensor)."""
    L = lib()
    fmt, g = _fmt(fmt), _gran(gran)
    rows, cols = x.shape
    d = tensor_desc(x)
    bits = L.mofq_format_bits(fmt)
    codes = torch.empty(rows * cols * max(bits, 4) // 8, dtype=torch.uint8, device=x.device) if want_codes else None
    scales = torch.empty(n_scales(g, rows, cols, group) if g != PER_GROUP or group > 0 else 0,
                         dtype=torch.float32, device=x.device) if want_scales else None
    deq = torch.empty((rows, cols), dtype=x.dtype, device=x.device) if want_dequant else None
    ws = workspace if workspace is not None else _workspace(L.mofq_tensor_workspace_bytes(C.byref(d)), x.device)
    sin = scales_in.contiguous().float() if scales_in is not None else None
    _check(L.mofq_quantize_tensor(C.byref(d), fmt, g, group, sin.data_ptr() if sin is not None else None,
                                  codes.data_ptr() if codes is not None else None,
                                  scales.data_ptr() if scales is not None else None,
                                  deq.data_ptr() if deq is not None else None,
                                  ws.data_ptr(), ws.numel(), _stream(x.device)))
    return dict(codes=codes, scales=scales, dequant=deq, status=ws[:4].view(torch.int32), workspace=ws)


def tensor_error(x, formats, gran, gran2=None, group=0, workspace=None):
    """mofq_tensor_error.  Returns (mse float32 tensor [n] or [2, n], status int32 tensor view)."""
    L = lib()
    d = tensor_desc(x)
    n = len(formats)
    fm = (C.c_int32 * n)(*[_fmt(f) for f in formats])
    g2 = _gran(gran2)
    out = torch.empty((2, n) if g2 != GRAN_NONE else (n,), dtype=torch.float32, device=x.device)
    ws = workspace if workspace is not None else _workspace(L.mofq_tensor_workspace_bytes(C.byref(d)), x.device)
    _check(L.mofq_tensor_error(C.byref(d), fm, n, _gran(gran), g2, group, out.data_ptr(), ws.data_ptr(), ws.numel(),
                               _stream(x.device)))
    return out, ws[:4].view(torch.int32)


def tensor_error_noalloc(x, formats, gran, gran2=None, group=0, mse_out=None, status_out=None):
    """mofq_tensor_error_noalloc: same result as tensor_error, no workspace argument.

    For callers that cannot allocate device memory: pass preallocated `mse_out` (float32, n or
    2n elements) and optionally `status_out` (int32, 1 element) and nothing is allocated here or
    in the library.  Without them this wrapper allocates the two small outputs for convenience.
    """
    L = lib()
    d = tensor_desc(x)
    n = len(formats)
    fm = (C.c_int32 * n)(*[_fmt(f) for f in formats])
    g2 = _gran(gran2)
    if mse_out is None:
        mse_out = torch.empty((2, n) if g2 != GRAN_NONE else (n,), dtype=torch.float32, device=x.device)
    if status_out is None:
        status_out = torch.zeros(1, dtype=torch.int32, device=x.device)
    _check(L.mofq_tensor_error_noalloc(C.byref(d), fm, n, _gran(gran), g2, group, mse_out.data_ptr(),
                                       status_out.data_ptr(), _stream(x.device)))
    return mse_out, status_out


def select_blocks(x, formats, gran, group=0, want_block_sse=False, workspace=None):
    """mofq_select_blocks.  Returns dict(choice uint8 [blocks], block_sse float32 [blocks, n] or None,
    mse float32 [n + 1] (candidates, then the mixture), status int32 tensor); nothing synchronises."""
    L = lib()
    d = tensor_desc(x)
    n = len(formats)
    fm = (C.c_int32 * n)(*[_fmt(f) for f in formats])
    rows, cols = x.shape
    nb = n_scales(gran, rows, cols, group)
    choice = torch.empty(nb, dtype=torch.uint8, device=x.device)
    sse = torch.empty((nb, n), dtype=torch.float32, device=x.device) if want_block_sse else None
    mse = torch.empty(n + 1, dtype=torch.float32, device=x.device)
    ws = workspace if workspace is not None else _workspace(L.mofq_tensor_workspace_bytes(C.byref(d)), x.device)
    _check(L.mofq_select_blocks(C.byref(d), fm, n, _gran(gran), group, choice.data_ptr(), sse.data_ptr() if sse is not None else None,
                                mse.data_ptr(), ws.data_ptr(), ws.numel(), _stream(x.device)))
    return dict(choice=choice, block_sse=sse, mse=mse, status=ws[:4].view(torch.int32))


def absmax_update(x, absmax):
    """mofq_absmax_update: absmax (1-element float32 CUDA tensor) <- max(absmax, max|x|)."""
    d = tensor_desc(x)
    _check(lib().mofq_absmax_update(C.byref(d), absmax.data_ptr(), _stream(x.device)))
    return absmax


def tensor_error_scaled(x, formats, scales, workspace=None):
    """mofq_tensor_error_scaled: MSE of each candidate under the given per-tensor scales (float32 CUDA tensor [n])."""
    L = lib()
    d = tensor_desc(x)
    n = len(formats)
    fm = (C.c_int32 * n)(*[_fmt(f) for f in formats])
    sc = scales.contiguous().float()
    assert sc.numel() == n and sc.is_cuda
    out = torch.empty(n, dtype=torch.float32, device=x.device)
    ws = workspace if workspace is not None else _workspace(L.mofq_tensor_workspace_bytes(C.byref(d)), x.device)
    _check(L.mofq_tensor_error_scaled(C.byref(d), fm, n, sc.data_ptr(), out.data_ptr(), ws.data_ptr(), ws.numel(), _stream(x.device)))
    return out, ws[:4].view(torch.int32)


def diag_wait_expiry(device):
    """mofq_diag_wait_expiry: returns a 1-element int32 CUDA tensor that holds MOFQ_STATUS_TIMEOUT once the kernel ends."""
    out = torch.zeros(1, dtype=torch.int32, device=device)
    _check(lib().mofq_diag_wait_expiry(out.data_ptr(), _stream(device)))
    return out


def diag_scale_pair(fmt, absmax):
    """mofq_diag_scale_pair: (scale, inv) of the multi-tensor kernel for a float32 CUDA tensor of abs-max values."""
    a = absmax.contiguous().float()
    s, inv = torch.empty_like(a), torch.empty_like(a)
    _check(lib().mofq_diag_scale_pair(_fmt(fmt), a.data_ptr(), s.data_ptr(), inv.data_ptr(), a.numel(), _stream(a.device)))
    return s, inv


def diag_fp_round(fmt, t):
    """mofq_diag_fp_round: the scoring kernels' FP grid rounding applied to a float32 CUDA tensor."""
    t = t.contiguous().float()
    out = torch.empty_like(t)
    _check(lib().mofq_diag_fp_round(_fmt(fmt), t.data_ptr(), out.data_ptr(), t.numel(), _stream(t.device)))
    return out


def layer_output_error(X, W, cfg, workspace=None):
    """mofq_layer_output_error.  Returns (mse [n], nsr [n], status view)."""
    L = lib()
    layer = MofqLayer(tensor_desc(W), tensor_desc(X))
    n = cfg.n_candidates
    mse = torch.empty(n, dtype=torch.float32, device=W.device)
    nsr = torch.empty(n, dtype=torch.float32, device=W.device)
    ws = workspace if workspace is not None else _workspace(L.mofq_workspace_bytes(C.byref(layer), 1, C.byref(cfg)), W.device)
    _check(L.mofq_layer_output_error(C.byref(layer), C.byref(cfg), mse.data_ptr(), nsr.data_ptr(), ws.data_ptr(),
                                     ws.numel(), _stream(W.device)))
    return mse, nsr, ws[:4].view(torch.int32)


def workspace_bytes(layers, cfg):
    arr = prepare_layers(layers).array
    return lib().mofq_workspace_bytes(arr, len(layers), C.byref(cfg))


def _parse_results(buf, n_records, n_cand):
    raw = (MofqResult * n_records).from_buffer_copy(buf)
    return [dict(chosen=r.chosen, status=r.status, errors=[r.error[i] for i in range(n_cand)],
                 nsr=[r.nsr[i] for i in range(n_cand)], rel_margin=r.rel_margin) for r in raw]


def select_formats(layers, cfg, workspace=None, results=None, parse=True):
    """mofq_select_formats over a list of W tensors or (W, X) pairs on the device.

    With parse=True the records are copied to the host (synchronises) and returned as a list of
    dicts; with parse=False the raw device byte tensor is returned and nothing synchronises.
    """
    L = lib()
    prep = prepare_layers(layers)
    arr, dev = prep.array, prep.device
    n_sets = 2 if cfg.w_gran2 != GRAN_NONE else 1
    n_rec = len(layers) * n_sets
    res = results if results is not None else torch.empty(n_rec * RESULT_BYTES, dtype=torch.uint8, device=dev)
    ws = workspace if workspace is not None else _workspace(L.mofq_workspace_bytes(arr, len(layers), C.byref(cfg)), dev)
    _check(L.mofq_select_formats(arr, len(layers), C.byref(cfg), res.data_ptr(), ws.data_ptr(), ws.numel(), _stream(dev)))
    if not parse:
        return res
    return _parse_results(bytes(res.cpu().numpy()), n_rec, cfg.n_candidates)


class MofqPacked(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p)]


class EmitBuffers:
    """Preallocated destinations of emit_selected for a layer list (codes, scales, format tags, status word)."""

    def __init__(self, layers, cfg):
        prep = prepare_layers(layers)
        dev = prep.device
        n = len(prep)
        self.array = (MofqPacked * n)()
        self.packed = []
        for i, layer in enumerate(prep.layers):
            W = layer if torch.is_tensor(layer) else layer[0]
            rows, cols = W.shape
            codes = torch.empty(rows * cols * cfg.bit_width // 8, dtype=torch.uint8, device=dev)
            scales = torch.empty(n_scales(cfg.w_gran, rows, cols, cfg.w_group), dtype=torch.float32, device=dev)
            self.array[i].codes, self.array[i].scales = codes.data_ptr(), scales.data_ptr()
            self.packed.append(dict(codes=codes, scales=scales))
        self.formats = torch.empty(n, dtype=torch.int32, device=dev)
        self.ws = _workspace(256, dev)


def emit_selected(layers, cfg, results, buffers=None):
    """mofq_emit_selected: quantise every layer's W to the format its selection record names (read on the device).

    `results` is the raw device byte tensor of select_formats(..., parse=False).  Returns (packed, formats, status):
    packed = list of dict(codes uint8 tensor, scales float32 tensor) per layer, formats = int32 device tensor of
    mofq_format tags, status = 1-element int32 device tensor.  Nothing synchronises.  Pass an EmitBuffers to reuse
    the destinations across calls.
    """
    L = lib()
    prep = prepare_layers(layers)
    b = buffers if buffers is not None else EmitBuffers(prep, cfg)
    _check(L.mofq_emit_selected(prep.array, len(prep), C.byref(cfg), results.data_ptr(), C.cast(b.array, C.c_void_p),
                                b.formats.data_ptr(), b.ws.data_ptr(), b.ws.numel(), _stream(prep.device)))
    return b.packed, b.formats, b.ws[:4].view(torch.int32)


def select_formats_host(layers, cfg, device, workspace=None):
    """mofq_select_formats_host: `layers` are CPU tensors (pinned recommended); returns parsed records."""
    L = lib()
    arr = _layer_array(layers, require_cuda=False)
    n_sets = 2 if cfg.w_gran2 != GRAN_NONE else 1
    n_rec = len(layers) * n_sets
    out = (MofqResult * n_rec)()
    ws = workspace if workspace is not None else _workspace(L.mofq_host_workspace_bytes(arr, len(layers), C.byref(cfg)), device)
    _check(L.mofq_select_formats_host(arr, len(layers), C.byref(cfg), C.cast(out, C.c_void_p), ws.data_ptr(), ws.numel(),
                                      _stream(device)))
    return _parse_results(bytes(out), n_rec, cfg.n_candidates)
