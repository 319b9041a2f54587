/*
 * mofq.h - C ABI of the B200 (sm_100a) MoFQ format-selection library.
 *
 * MoFQ = Mixture of Formats Quantization ("Integer or Floating Point? New Outlooks for Low-Bit
 * Quantization on Large Language Models").  For every linear layer the library quantises the
 * weight tensor (and, in the weight+activation setting, the calibration activations) onto the
 * INT-k and FP-k grids of one bit-width with abs-max scales, reduces each candidate's error and
 * keeps the candidate with the strictly smallest error (Algorithm 1).
 *
 * General conventions
 *   - Every data pointer is a DEVICE pointer unless its comment says "host".  Structs that
 *     describe tensors/layers/configs are read on the host.
 *   - Tensors are row-major with leading dimension `ld` (elements).  Weights are [out, in]
 *     (a Linear layer's weight, A_out = W * A_in, Section 3.2); activations are [tokens, in].
 *   - `data` must be 16-byte aligned, `cols` a multiple of 8 and `ld` a multiple of 8.
 *   - The caller owns every buffer, the workspace included; the library allocates nothing and
 *     keeps no state between calls.  The one exception is mofq_tensor_error_noalloc, which works
 *     in a fixed scratch array inside the library (see there).  All work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL = default stream) and the call returns without
 *     synchronising, unless stated.
 *   - The device entry points enqueue kernels and memsets only, so a call whose arguments stay valid
 *     can be captured into a CUDA graph and replayed; make one plain call of the same kind first
 *     (it sets the kernels' function attributes, which is not a stream operation).  The *_host
 *     variants copy from host memory and synchronise: they are not for capture.
 *   - Return value: 0 on success, a negative MOFQ_ERR_* for a synchronous argument error.  After
 *     a negative return the call's outputs are not produced.  Pointer, size, alignment, enum,
 *     candidate and workspace errors are found before anything is enqueued; a combination that
 *     only a kernel's launcher can refuse (MOFQ_ERR_UNSUPPORTED for a per-tensor scale together
 *     with a second granularity, rows too long for shared memory, more than 2^31 chunks) may be
 *     found after the clear of the workspace header has been enqueued, and in
 *     mofq_select_formats / mofq_emit_selected after the layers before the refused one.
 *     Conditions found on the device (non-finite input, a reciprocal scale that overflows
 *     binary32) are reported as MOFQ_STATUS_* bits in a device status word.
 *   - Input values must be finite.  Every fp16 tensor and any bf16 tensor of magnitude below 1e18 is
 *     in range for every call.  Beyond that (bf16 only) the whole-model selection kernels and the
 *     per-tensor-scale scoring still work, because they sum squared errors in units of the scale;
 *     mofq_select_blocks, group scales on a single small or strided tensor and
 *     mofq_tensor_error_scaled sum unscaled squares in binary32 and report +Inf there.  A reported
 *     error must itself fit binary32.
 *   - Candidates: at most MOFQ_MAX_CAND entries per call, of which at most one INT format and two
 *     distinct FP formats (three distinct formats); a list may repeat a format.
 *   - What the arithmetic contract below binds: the code-writing calls (mofq_quantize_tensor,
 *     mofq_emit_selected) follow it operation by operation, so codes, scales and dequantised
 *     values are determined bit for bit.  The scoring calls report errors that agree with the
 *     contract's to within 1e-5 relative: they may fuse the multiply into the INT rounding and
 *     form the FP candidates' differences in units of the scale, which can move a value only where
 *     x * inv lies within one binary32 ulp of a rounding tie (where both neighbours have the same
 *     error).
 *
 * Arithmetic contract (what "quantise" means here; the paper states round-to-nearest linear
 * quantisation with abs-max scales and leaves the rest open):
 *   absmax a of the scale block is exact; scale = RN32(a / Q), inv = RN32(Q / a) with
 *   Q = 2^(k-1)-1 (INT) or the largest finite magnitude of the FP grid; an all-zero block has
 *   scale = inv = 1.  t = RN32(x * inv).  INT code = RNE(t) as k-bit two's complement.  FP code =
 *   nearest grid magnitude to |t| (ties to the even code), sign bit copied from x.  With
 *   caller-supplied scales inv = RN32(1 / scale) and out-of-range values saturate.  The error of
 *   a candidate is mean (x - value(code) * scale)^2 over the whole tensor.
 */
#ifndef MOFQ_H
#define MOFQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOFQ_MAX_CAND 4 /* most candidate formats per call */

/* Number formats (Section 2; Section 4.2 and Table 3 for the two FP4 variants). */
typedef enum {
    MOFQ_INT4 = 0,          /* two's complement, codes -8..7, abs-max maps to 7                     */
    MOFQ_INT8 = 1,          /* two's complement, codes -128..127, abs-max maps to 127               */
    MOFQ_FP4_E2M1 = 2,      /* Table 3 "w/o NaN&Inf": 0 .5 1 1.5 2 3 4 6 and negatives, max 6       */
    MOFQ_FP4_E2M1_IEEE = 3, /* Table 3 "w/ NaN&Inf": exponent field 3 reserved, max 3               */
    MOFQ_FP8_E4M3 = 4,      /* bias 7, only S.1111.111 reserved, max 448 (hardware-compatible)      */
    MOFQ_FP8_E5M2 = 5       /* bias 15, exponent field 31 reserved, max 57344                       */
} mofq_format;

/* Scale granularity (Section 3.2: per-channel weights, per-tensor activations; per-group =
 * `group` consecutive elements along the input dimension: a power of two in [8, 256] that divides cols). */
typedef enum { MOFQ_PER_TENSOR = 0, MOFQ_PER_CHANNEL = 1, MOFQ_PER_GROUP = 2 } mofq_gran;
#define MOFQ_GRAN_NONE (-1)

typedef enum { MOFQ_F16 = 0, MOFQ_BF16 = 1 } mofq_dtype;

/* Error metric of Algorithm 1 (Section 4.1: tensor error or layer output error). */
typedef enum { MOFQ_TENSOR_MSE = 0, MOFQ_LAYER_OUTPUT_MSE = 1 } mofq_metric;

/* Synchronous error codes. */
#define MOFQ_OK 0
#define MOFQ_ERR_INVALID_ARG (-1)         /* NULL pointer, non-positive size, bad enum, too many candidates  */
#define MOFQ_ERR_UNSUPPORTED (-2)         /* candidate bit-width != bit_width, cols % group != 0, ...         */
#define MOFQ_ERR_MISALIGNED (-3)          /* data not 16-byte aligned, or cols / ld not a multiple of 8       */
#define MOFQ_ERR_WORKSPACE_TOO_SMALL (-4) /* workspace_bytes below the matching *_workspace_bytes() value     */
#define MOFQ_ERR_CUDA (-5)                /* a CUDA runtime call or kernel launch failed                      */
#define MOFQ_ERR_SCRATCH_LIMIT (-6)       /* mofq_tensor_error_noalloc: tensor beyond the built-in scratch    */

/* Asynchronous status bits (device status word / mofq_result.status). */
#define MOFQ_STATUS_NONFINITE_INPUT 1 /* an Inf or NaN was found in the input           */
#define MOFQ_STATUS_SCALE_OVERFLOW 2  /* Q / absmax is not finite in binary32           */
#define MOFQ_STATUS_TIMEOUT 4         /* a bounded device-side wait expired             */

typedef struct {
    const void *data; /* device, row-major                           */
    int32_t dtype;    /* mofq_dtype                                  */
    int32_t reserved;
    int64_t rows, cols, ld;
} mofq_tensor;

/* One linear layer: W [out, in]; X [tokens, in] calibration activations (data == NULL when the
 * metric does not need them). */
typedef struct {
    mofq_tensor W;
    mofq_tensor X;
} mofq_layer;

/* The arguments of Algorithm 1: MoFQ(model, is_w_only, format_candidates, bit_width, error_metric)
 * plus the scale granularities. */
typedef struct {
    int32_t bit_width;                 /* 4 or 8; every candidate must have this width                 */
    int32_t n_candidates;              /* 1..MOFQ_MAX_CAND                                              */
    int32_t candidates[MOFQ_MAX_CAND]; /* mofq_format, in the caller's order: ties go to the first      */
    int32_t is_w_only;                 /* 1: quantise W only; 0: W and X (same format for both)         */
    int32_t w_gran;                    /* mofq_gran for W                                               */
    int32_t w_group;                   /* group size when a W granularity is MOFQ_PER_GROUP             */
    int32_t w_gran2;                   /* MOFQ_GRAN_NONE, or a second W granularity scored from the     */
                                       /* same read (tensor metric only); results then hold 2 records   */
                                       /* per layer: [layer][0] for w_gran, [layer][1] for w_gran2      */
    int32_t a_gran;                    /* mofq_gran for X (MOFQ_PER_TENSOR in the paper)                */
    int32_t a_group;
    int32_t metric;                    /* mofq_metric                                                   */
} mofq_config;

/* One selection record (device memory). */
typedef struct {
    int32_t chosen;             /* index into mofq_config.candidates                                    */
    int32_t status;             /* MOFQ_STATUS_* bits                                                   */
    float error[MOFQ_MAX_CAND]; /* MSE per candidate, caller's order                                    */
    float nsr[MOFQ_MAX_CAND];   /* layer metric only: sum (Y-Yq)^2 / sum Y^2 (noise/signal power)       */
    float rel_margin;           /* (second smallest - smallest) / smallest; +Inf if smallest is 0       */
    int32_t reserved;
} mofq_result;

/*
 * mofq_quantize_tensor - round-to-nearest linear quantisation of one tensor to one format
 * (the plain RTN quantiser of Section 1, Algorithm 1 `quantize_layer`; granularities Section 3.2).
 *   x           tensor to quantise
 *   scales_in   NULL: abs-max scales are derived.  Else device array of n_scales floats
 *               (calibration scales, Section 3.2 dynamic tensor analysis); values saturate.
 *   codes_out   nullable.  8-bit formats: rows*cols bytes.  4-bit: rows*cols/2 bytes, element 2j in
 *               the low nibble of byte j.  Dense (leading dimension = cols).  INT codes are two's
 *               complement; FP codes are sign|exponent|mantissa with Table 3's numbering.
 *   scales_out  nullable.  n_scales floats: [1], [rows] or [rows, cols/group] row-major.
 *   dequant_out nullable.  rows*cols elements of x's dtype: RN32(value*scale) rounded to nearest even.
 *   workspace   at least mofq_tensor_workspace_bytes(x) bytes, 256-byte aligned.  On completion
 *               the first int32 of the workspace holds the MOFQ_STATUS_* bits of this call.
 */
int mofq_quantize_tensor(const mofq_tensor *x, int format, int gran, int group, const float *scales_in,
                         void *codes_out, float *scales_out, void *dequant_out,
                         void *workspace, size_t workspace_bytes, void *stream);

/*
 * mofq_tensor_error - tensor MSE (quantised against original tensor) of n candidate formats of one
 * bit-width from ONE read of x (Section 3.2, static tensor analysis; Algorithm 1 `compute_error`
 * with the tensor metric).
 *   formats     host array of n mofq_format values of equal bit-width
 *   gran2       MOFQ_GRAN_NONE or a second granularity scored from the same read
 *   mse_out     device, n floats (2n when gran2 is given: [gran][candidate])
 *   workspace   at least mofq_tensor_workspace_bytes(x); first int32 = status bits on completion
 */
int mofq_tensor_error(const mofq_tensor *x, const int32_t *formats, int n, int gran, int gran2, int group,
                      float *mse_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * mofq_select_blocks - format selection finer than a layer: one winner per scale block, i.e. per output channel
 * (gran = MOFQ_PER_CHANNEL) or per group of `group` elements (MOFQ_PER_GROUP).  Section 7 names channel-wise and
 * block-wise mixing of formats as the step after layer-wise selection; the rule applied to every block is
 * Algorithm 1's (strictly smaller error, caller's candidate order), the error being the block's sum of squared
 * errors under its own abs-max scale.
 *   formats        n candidates of one bit-width, n <= 3
 *   choice_out     device, one byte per block (row-major, groups left to right): index into formats - the format map
 *   block_sse_out  device, blocks*n floats (nullable): every block's error per candidate, caller's order
 *   mse_out        device, n + 1 floats: whole-tensor MSE of each candidate, then of the per-block mixture
 *   workspace      as for mofq_tensor_error
 */
int mofq_select_blocks(const mofq_tensor *x, const int32_t *formats, int n, int gran, int group, uint8_t *choice_out,
                       float *block_sse_out, float *mse_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * mofq_absmax_update - running abs-max over calibration batches: *absmax_inout = max(*absmax_inout, max |x|)
 * (Section 3.2, dynamic tensor analysis: the calibration process keeps the largest value seen over several batches to
 * determine the scaling factor).  absmax_inout: device float, initialise it to 0 before the first batch.
 */
int mofq_absmax_update(const mofq_tensor *x, float *absmax_inout, void *stream);

/*
 * mofq_tensor_error_scaled - tensor MSE of n candidates under CALLER-SUPPLIED per-tensor scales, e.g. calibration scales
 * applied to an unseen activation batch (Section 3.2, dynamic tensor analysis).  scales_in: device, n floats, one scale
 * per candidate in the caller's order (typically calibration abs-max / format maximum); inv = RN32(1/scale); values
 * beyond the grid saturate.  Every candidate has its own scale, so a format may appear only once in `formats`
 * (MOFQ_ERR_UNSUPPORTED otherwise).  mse_out: device, n floats.  workspace as for mofq_tensor_error.
 */
int mofq_tensor_error_scaled(const mofq_tensor *x, const int32_t *formats, int n, const float *scales_in, float *mse_out,
                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * mofq_layer_output_error - error of the layer output Y = X W^T when its inputs are quantised
 * (Section 3.2 layer analysis; Algorithm 1 `compute_error` with the layer output metric).
 * is_w_only: Yq = X dq(W)^T; otherwise Yq = dq(X) dq(W)^T with the same format for both tensors.
 * Scales: the paper's (Section 3.2) and the only ones this metric takes: cfg->w_gran = MOFQ_PER_CHANNEL and, unless
 * is_w_only, cfg->a_gran = MOFQ_PER_TENSOR, so that the scales factor out of the contraction; anything else is
 * MOFQ_ERR_UNSUPPORTED, as are fp16 activations with bf16 weights (no exact common 16-bit operand type).
 *   mse_out, nsr_out   device, cfg->n_candidates floats each, caller's order
 *   workspace          at least mofq_workspace_bytes(L, 1, cfg); first int32 = status bits
 */
int mofq_layer_output_error(const mofq_layer *L, const mofq_config *cfg, float *mse_out, float *nsr_out,
                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * mofq_select_formats - Algorithm 1 over a model's layer list: score every candidate on every
 * layer and keep the strict minimum in the caller's candidate order.
 *   layers       host array of n_layers descriptors (device tensors)
 *   results_out  device array of n_layers records (2*n_layers when cfg->w_gran2 is given)
 *   workspace    at least mofq_workspace_bytes(layers, n_layers, cfg)
 * The layers' kernels of one call may overlap on the device (a layer's launch can start while the previous
 * layer's drains); seen from the stream the call is one unit: it starts after everything enqueued before
 * it and everything enqueued after it sees all its records.  The output buffers of the layers
 * (results_out here, codes / scales in mofq_emit_selected) must therefore not alias each other.
 */
int mofq_select_formats(const mofq_layer *layers, int n_layers, const mofq_config *cfg,
                        mofq_result *results_out, void *workspace, size_t workspace_bytes, void *stream);

/* Where one layer's quantised weights go (device memory, caller-owned). */
typedef struct mofq_packed {
    void *codes;     /* rows*cols*bit_width/8 bytes, packed as by mofq_quantize_tensor */
    float *scales;   /* one per row (per-channel), per group, or one (per-tensor)      */
} mofq_packed;

/*
 * mofq_emit_selected - the last step of Algorithm 1: every layer keeps the quantisation of the format that
 * won its selection.  The winner is read ON THE DEVICE from the layer's selection record, so this call can be
 * enqueued right behind mofq_select_formats on the same stream with no host round trip in between.
 *   results      device records written by mofq_select_formats with the same cfg (first granularity's record
 *                of each layer when cfg->w_gran2 is given)
 *   out          HOST array of n_layers destinations (device pointers inside); scales follow cfg->w_gran / w_group
 *   formats_out  device, n_layers int32 (nullable): the mofq_format each layer was quantised to - the
 *                per-layer format tag of the mixed-format model
 *   workspace    device, at least 256 bytes; its first int32 holds the OR of the layers' status bits afterwards
 */
int mofq_emit_selected(const mofq_layer *layers, int n_layers, const mofq_config *cfg, const mofq_result *results,
                       const mofq_packed *out, int32_t *formats_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * mofq_select_formats_host - the same selection for a model whose tensors live in HOST memory
 * (pinned memory recommended).  Layer data pointers are host pointers and the tensors are dense
 * (ld == cols); the call copies each layer into a staging area of the device workspace, scores it
 * there, copies the records back and SYNCHRONISES before returning.
 *   results_host host array of n_layers (or 2*n_layers) records
 *   workspace    device, at least mofq_host_workspace_bytes(layers, n_layers, cfg)
 */
int mofq_select_formats_host(const mofq_layer *layers_host_data, int n_layers, const mofq_config *cfg,
                             mofq_result *results_host, void *workspace, size_t workspace_bytes, void *stream);

/*
 * mofq_tensor_error_noalloc - mofq_tensor_error without a caller-provided workspace.
 * (The paper has no counterpart for this call; it exists for deployment reasons only.)
 *
 * Who needs it: code that may not call cudaMalloc at the moment it wants a tensor scored - a
 * host application that gave all device memory to its own pool at start-up, a plug-in that must
 * not enlarge the process, a latency-critical loop where an allocation would serialise the
 * device.  Such callers pass inputs and outputs only; the scratch that the scoring kernels need
 * (block counters, status word, per-block partial sums) is a fixed array of
 * MOFQ_NOALLOC_SCRATCH_BYTES bytes built into the library.  Every GPU context that loads the
 * library carries that array until the process ends.  The call itself performs no cudaMalloc,
 * cudaFree or other allocating call.
 *
 *   x, formats, n, gran, gran2, group, mse_out   exactly as for mofq_tensor_error
 *   status_out   nullable device int32: receives the MOFQ_STATUS_* bits of this call
 *
 * Limits and rules:
 *   - Tensors of more than MOFQ_NOALLOC_MAX_ELEMENTS elements, or whose scoring pass would need
 *     more scratch than the built-in array holds, are refused with MOFQ_ERR_SCRATCH_LIMIT and
 *     nothing is enqueued.  Use mofq_tensor_error with your own workspace for those.
 *   - The first call on each device looks up the device address of the array (a one-time
 *     set-up, done with that device current) and keeps it for the life of the process.  Make
 *     that first call outside any stream capture.  A device that is reset (cudaDeviceReset) after
 *     that first call must not use this entry point again: the kept address would be stale.
 *   - All calls on a device share the one array, and it still holds the previous call's data when
 *     the next call starts; each call clears the words that must start at zero.  Two calls that
 *     can run on the GPU at the same time (different streams, or different host threads without
 *     ordering) race on it: order them on one stream, or with events.
 */
#define MOFQ_NOALLOC_SCRATCH_BYTES 131328
#define MOFQ_NOALLOC_MAX_ELEMENTS 2147483648LL /* 2^31 elements = 4 GiB of fp16/bf16 */
int mofq_tensor_error_noalloc(const mofq_tensor *x, const int32_t *formats, int n, int gran, int gran2, int group,
                              float *mse_out, int32_t *status_out, void *stream);
size_t mofq_noalloc_scratch_bytes(void);

/*
 * mofq_diag_fp_round - diagnostic: rounds n binary32 values onto the unscaled FP grid (Section 2, Table 3) exactly as
 * the scoring kernels do (hardware convert, round-to-nearest-even, saturating at the grid maximum) and writes the
 * grid values.  format: MOFQ_FP4_E2M1, MOFQ_FP8_E4M3 or MOFQ_FP8_E5M2.  t, out: device, n floats.
 */
int mofq_diag_fp_round(int format, const float *t, float *out, int64_t n, void *stream);

/*
 * mofq_diag_wait_expiry - diagnostic: runs the bounded wait that every pipelined kernel of the library uses on a
 * barrier that nothing will ever complete.  The wait gives up after about two seconds, the kernel returns and
 * *status_out (device int32) holds MOFQ_STATUS_TIMEOUT: a broken pipeline ends as a status bit, not as a hung GPU.
 * (The paper has no counterpart; this exists so that a test can show it.)
 */
int mofq_diag_wait_expiry(int32_t *status_out, void *stream);

/*
 * mofq_diag_scale_pair - diagnostic: scale = RN32(a / Q) and inv = RN32(Q / a) (Section 3.2: abs-max scaling; a = 0
 * gives 1, 1) as the multi-tensor scoring kernel computes them for binary16 tensors, i.e. without the general
 * division routine.  Valid for abs-max values a binary16 tensor can have (0 or 2^-24 ... 65504); a test compares
 * every such value with two correctly rounded divisions.  absmax, scale_out, inv_out: device, n floats.
 */
int mofq_diag_scale_pair(int format, const float *absmax, float *scale_out, float *inv_out, int64_t n, void *stream);

/* Workspace sizes in bytes (host-side arithmetic only). */
size_t mofq_tensor_workspace_bytes(const mofq_tensor *x);
size_t mofq_workspace_bytes(const mofq_layer *layers, int n_layers, const mofq_config *cfg);
size_t mofq_host_workspace_bytes(const mofq_layer *layers, int n_layers, const mofq_config *cfg);

/* Static facts about a format: bit-width (4/8) and largest finite magnitude; -1 / 0 for a bad enum. */
int mofq_format_bits(int format);
float mofq_format_max(int format);

/* Human-readable name of a MOFQ_ERR_* code. */
const char *mofq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MOFQ_H */
