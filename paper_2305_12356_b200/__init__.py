"""B200-native MoFQ (Mixture of Formats Quantization) format selection: Python binding of libmofq.so."""
from .binding import (  # noqa: F401
    BF16, F16, FORMATS, FP4_E2M1, FP4_E2M1_IEEE, FP8_E4M3, FP8_E5M2, GRAN_NONE, GRANS, INT4, INT8, LAYER_OUTPUT_MSE,
    PER_CHANNEL, PER_GROUP, PER_TENSOR, TENSOR_MSE, MofqError, prepare_layers, layer_output_error, lib, make_config, quantize_tensor,
    select_formats, select_formats_host, tensor_error, tensor_error_noalloc, workspace_bytes, absmax_update, emit_selected, select_blocks,
    tensor_error_scaled)
