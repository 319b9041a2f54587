/*
 * MoFQ oracle: a plain, slow, CPU-only restatement of the per-layer format selection of
 * "Integer or Floating Point? New Outlooks for Low-Bit Quantization on Large Language Models"
 * (Mixture of Formats Quantization).
 *
 * THIS IS TEST INFRASTRUCTURE. It exists to check the CUDA library and to be timed as a CPU
 * baseline. It shares no code, table, header or helper with the CUDA path, and the CUDA path
 * never calls it.
 *
 * Everything here is the definition written out: enumerate the grid, scale by abs-max, round to
 * the nearest grid point (ties to even), decode, square the difference, take the mean, pick the
 * smaller error with a strict '<' in the caller's candidate order.  Error sums are in double.
 * The three fp32 operations that decide an integer code (scale, reciprocal, scaled value) are
 * single IEEE binary32 operations, because the quantised code must be decided in one stated
 * precision; this file must be compiled with -ffp-contract=off and without -ffast-math.
 *
 * Pins (tests/test_oracle_*.py): Table 3 of the paper for the FP4 code->value map, enumeration
 * counts and library decodes for FP8, hand-made tie grids, the scale pair against correctly
 * rounded exact-rational quotients, closed-form uniform-noise MSE,
 * exact-rational brute force on tiny tensors, identity-activation and exact-integer special
 * cases for the layer output error; block-wise selection against row/group slices scored as
 * tensors of their own and a hand-worked two-row case.  No function in this file is "parity unpinned".
 *
 * OpenMP is used only over rows / output rows (independent work items).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- enumerations (values are part of the oracle's own interface) -------------------------- */
enum { ORC_INT4 = 0, ORC_INT8 = 1, ORC_FP4_E2M1 = 2, ORC_FP4_E2M1_IEEE = 3, ORC_FP8_E4M3 = 4, ORC_FP8_E5M2 = 5 };
enum { ORC_PER_TENSOR = 0, ORC_PER_CHANNEL = 1, ORC_PER_GROUP = 2 };
enum { ORC_F16 = 0, ORC_BF16 = 1 };

/* ---- storage types -> value ------------------------------------------------------------------ */

/* IEEE binary16 bit pattern -> exact float. */
static float half_bits_to_float(uint16_t h)
{
    int s = (h >> 15) & 1, e = (h >> 10) & 0x1F, m = h & 0x3FF;
    double v;
    if (e == 0)        v = ldexp((double)m, -24);                 /* subnormal: m * 2^-24 */
    else if (e == 31)  v = m ? NAN : INFINITY;
    else               v = ldexp(1.0 + (double)m / 1024.0, e - 15);
    return (float)(s ? -v : v);
}

/* bfloat16 bit pattern -> exact float (upper 16 bits of a binary32). */
static float bf16_bits_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

float orc_load(const uint16_t *p, int dtype)
{
    return dtype == ORC_F16 ? half_bits_to_float(*p) : bf16_bits_to_float(*p);
}

static int sign_bit16(uint16_t v) { return (v >> 15) & 1; }

/* float -> nearest binary16 / bfloat16 bit pattern, ties to even (used only for dequant output). */
static uint16_t float_to_half_bits(float f)
{
    if (isnan(f)) return 0x7E00;
    int s = signbit(f) ? 1 : 0;
    double a = fabs((double)f);
    if (a == 0.0) return (uint16_t)(s << 15);
    int e;
    (void)frexp(a, &e);           /* a = fr * 2^e, fr in [0.5,1) -> floor(log2 a) = e-1 */
    int E = e - 1;
    if (E < -14) E = -14;         /* subnormal quantum */
    double q = nearbyint(ldexp(a, 10 - E));       /* units of 2^(E-10), RNE */
    double v = ldexp(q, E - 10);
    if (v >= 65520.0 || isinf(a)) return (uint16_t)((s << 15) | 0x7C00);
    /* re-derive fields from the rounded value */
    if (v < ldexp(1.0, -14)) return (uint16_t)((s << 15) | (int)ldexp(v, 24));
    (void)frexp(v, &e);
    E = e - 1;
    int mant = (int)(ldexp(v, 10 - E)) - 1024;
    return (uint16_t)((s << 15) | ((E + 15) << 10) | mant);
}

static uint16_t float_to_bf16_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if (isnan(f)) return 0x7FC0;
    uint32_t lsb = (u >> 16) & 1;
    u += 0x7FFFu + lsb;           /* round to nearest, ties to even, on the dropped 16 bits */
    return (uint16_t)(u >> 16);
}

uint16_t orc_store(float f, int dtype)
{
    return dtype == ORC_F16 ? float_to_half_bits(f) : float_to_bf16_bits(f);
}

/* ---- Section 2 "Integer vs. Floating Point Formats", Section 4.2 / Table 3: the grids --------- */

typedef struct { int is_fp, bits, E, M, bias, top_reserved; double fmt_max; } fmt_t;

static int fmt_lookup(int fmt, fmt_t *f)
{
    memset(f, 0, sizeof *f);
    switch (fmt) {
    case ORC_INT4: f->bits = 4; f->fmt_max = 7; return 0;
    case ORC_INT8: f->bits = 8; f->fmt_max = 127; return 0;
    case ORC_FP4_E2M1:      f->is_fp = 1; f->bits = 4; f->E = 2; f->M = 1; f->bias = 1;  f->top_reserved = 0; f->fmt_max = 6; return 0;
    case ORC_FP4_E2M1_IEEE: f->is_fp = 1; f->bits = 4; f->E = 2; f->M = 1; f->bias = 1;  f->top_reserved = 1; f->fmt_max = 3; return 0;
    case ORC_FP8_E4M3:      f->is_fp = 1; f->bits = 8; f->E = 4; f->M = 3; f->bias = 7;  f->top_reserved = 2; f->fmt_max = 448; return 0;
    case ORC_FP8_E5M2:      f->is_fp = 1; f->bits = 8; f->E = 5; f->M = 2; f->bias = 15; f->top_reserved = 1; f->fmt_max = 57344; return 0;
    }
    return -1;
}

int orc_format_bits(int fmt) { fmt_t f; return fmt_lookup(fmt, &f) ? -1 : f.bits; }
double orc_format_max(int fmt) { fmt_t f; return fmt_lookup(fmt, &f) ? NAN : f.fmt_max; }

/*
 * Code -> value.  INT-k: two's complement integer (consecutive codes differ by 1).
 * FP-k: sign | exponent | mantissa with bias 2^(E-1)-1 and gradual underflow; this is the only
 * reading that gives Table 3's 0, 0.5, 1, 1.5, 2, 3, 4, 6 for E2M1.  Reserved codes return NaN:
 *   top_reserved = 1: the whole all-ones exponent (IEEE Inf/NaN: E2M1_IEEE, E5M2)
 *   top_reserved = 2: only all-ones exponent with all-ones mantissa (hardware E4M3)
 */
double orc_decode(int fmt, int code)
{
    fmt_t f;
    if (fmt_lookup(fmt, &f)) return NAN;
    code &= (1 << f.bits) - 1;
    if (!f.is_fp) {
        int half = 1 << (f.bits - 1);
        return (double)(code >= half ? code - 2 * half : code);
    }
    int s = (code >> (f.bits - 1)) & 1;
    int e = (code >> f.M) & ((1 << f.E) - 1);
    int m = code & ((1 << f.M) - 1);
    int emax_field = (1 << f.E) - 1;
    if (f.top_reserved == 1 && e == emax_field) return NAN;
    if (f.top_reserved == 2 && e == emax_field && m == (1 << f.M) - 1) return NAN;
    double v = (e == 0) ? ldexp((double)m / (double)(1 << f.M), 1 - f.bias)
                        : ldexp(1.0 + (double)m / (double)(1 << f.M), e - f.bias);
    return s ? -v : v;
}

/* number of finite non-negative magnitudes, i.e. magnitude codes 0 .. n-1 are usable */
static int n_magnitudes(const fmt_t *f, int fmt)
{
    int n = 0, half = 1 << (f->bits - 1);
    for (int c = 0; c < half; ++c)
        if (!isnan(orc_decode(fmt, c))) n = c + 1;
    return n;
}

/*
 * Inverse of orc_decode for a non-negative value that lies on the grid: below the smallest normal
 * 2^(1-bias) the code is the count of subnormal steps 2^(1-bias-M); otherwise the exponent field
 * is floor(log2 v) + bias and the mantissa field is the fraction above 1 in units of 2^-M.
 */
static int fp_magnitude_to_code(const fmt_t *f, double v)
{
    if (v < ldexp(1.0, 1 - f->bias)) return (int)ldexp(v, f->bias - 1 + f->M);
    int ex;
    (void)frexp(v, &ex);
    int e = ex - 1;
    int m = (int)ldexp(v, f->M - e) - (1 << f->M);
    return ((e + f->bias) << f->M) | m;
}

/*
 * FP grid rounding, arithmetic form: with e = max(floor(log2|t|), 1-bias) the grid spacing at t is
 * u = 2^(e-M); the nearest grid point is RNE(|t|/u)*u (the division is exact: u is a power of
 * two), saturated at fmt_max.  The code is the position of that magnitude in the format's
 * magnitude order, with the sign bit on top.
 */
int orc_encode_fp_arith(int fmt, float t, int negative)
{
    fmt_t f;
    if (fmt_lookup(fmt, &f) || !f.is_fp) return -1;
    double a = fabs((double)t), v;
    if (a == 0.0) v = 0.0;
    else if (isinf(a)) v = f.fmt_max;
    else {
        int ex;
        (void)frexp(a, &ex);
        int e = ex - 1;
        if (e < 1 - f.bias) e = 1 - f.bias;
        double m = nearbyint(ldexp(a, f.M - e));     /* RNE: default rounding mode */
        v = ldexp(m, e - f.M);
        if (v > f.fmt_max) v = f.fmt_max;
    }
    int code = fp_magnitude_to_code(&f, v);
    return code | (negative ? 1 << (f.bits - 1) : 0);
}

/*
 * FP grid rounding, table form (independent of the arithmetic form): scan the sorted magnitudes,
 * keep the nearest; on an exact midpoint keep the neighbour whose code is even.
 */
int orc_encode_fp_table(int fmt, float t, int negative)
{
    fmt_t f;
    if (fmt_lookup(fmt, &f) || !f.is_fp) return -1;
    double a = fabs((double)t);
    int n = n_magnitudes(&f, fmt), best = 0;
    double bestd = INFINITY;
    for (int c = 0; c < n; ++c) {
        double d = fabs(orc_decode(fmt, c) - a);
        if (d < bestd || (d == bestd && (c & 1) == 0)) { bestd = d; best = c; }
    }
    return best | (negative ? 1 << (f.bits - 1) : 0);
}

/* INT grid rounding: nearest integer, ties to even, then clamp to the two's complement range. */
int orc_encode_int(int fmt, float t)
{
    fmt_t f;
    if (fmt_lookup(fmt, &f) || f.is_fp) return -1;
    double q = nearbyint((double)t);
    double lo = -f.fmt_max - 1.0, hi = f.fmt_max;
    if (q < lo) q = lo;
    if (q > hi) q = hi;
    return (int)q & ((1 << f.bits) - 1);
}

/* ---- abs-max scales (Section 3.2: per-channel weights, per-tensor activations; group = 128) --- */

/*
 * scale = RN32(absmax / Q), inv = RN32(Q / absmax), Q = fmt_max (FP) or 2^(k-1)-1 (INT);
 * an all-zero block gets scale = inv = 1.
 */
void orc_scale_from_absmax(int fmt, float absmax, float *scale, float *inv)
{
    fmt_t f;
    fmt_lookup(fmt, &f);
    float Q = (float)f.fmt_max;
    if (absmax == 0.0f) { *scale = 1.0f; *inv = 1.0f; return; }
    *scale = absmax / Q;
    *inv = Q / absmax;
}

static int64_t n_scales(int gran, int64_t rows, int64_t cols, int group)
{
    if (gran == ORC_PER_TENSOR) return 1;
    if (gran == ORC_PER_CHANNEL) return rows;
    return rows * (cols / group);
}

static int64_t scale_index(int gran, int64_t r, int64_t c, int64_t cols, int group)
{
    if (gran == ORC_PER_TENSOR) return 0;
    if (gran == ORC_PER_CHANNEL) return r;
    return r * (cols / group) + c / group;
}

/* abs-max of every scale block, as exact floats.  absmax_out has n_scales entries. */
void orc_absmax(const uint16_t *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                int gran, int group, float *absmax_out)
{
    int64_t ns = n_scales(gran, rows, cols, group);
    for (int64_t i = 0; i < ns; ++i) absmax_out[i] = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float a = fabsf(orc_load(x + r * ld + c, dtype));
            int64_t si = scale_index(gran, r, c, cols, group);
            if (a > absmax_out[si] || isnan(a)) absmax_out[si] = a;
        }
}

/* ---- round-to-nearest linear quantisation of one tensor (Section 1: "naive linear quantization
 *      with round-to-nearest") ----------------------------------------------------------------- */

/*
 * codes_out   : one byte per element (unpacked, low k bits), row-major with leading dimension cols
 * scales_out  : n_scales floats (written even when scales_in is given)
 * dequant_out : optional, same dtype as x, leading dimension cols: RN(value*scale) in binary32, then RNE to dtype
 * sse_out     : optional, sum over all elements of (x - value*scale)^2 in double
 * scales_in   : optional caller-supplied scales (e.g. from calibration); then inv = RN32(1/scale) and
 *               out-of-range values saturate at the ends of the grid.
 * returns 0, or -1 on a bad argument.
 */
int orc_quantize(const uint16_t *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                 int fmt, int gran, int group, const float *scales_in,
                 uint8_t *codes_out, float *scales_out, uint16_t *dequant_out, double *sse_out)
{
    fmt_t f;
    if (fmt_lookup(fmt, &f)) return -1;
    if (gran == ORC_PER_GROUP && (group <= 0 || cols % group)) return -1;
    int64_t ns = n_scales(gran, rows, cols, group);
    float *scale = (float *)malloc(sizeof(float) * (size_t)ns);
    float *inv = (float *)malloc(sizeof(float) * (size_t)ns);
    if (scales_in) {
        for (int64_t i = 0; i < ns; ++i) { scale[i] = scales_in[i]; inv[i] = 1.0f / scales_in[i]; }
    } else {
        float *am = (float *)malloc(sizeof(float) * (size_t)ns);
        orc_absmax(x, dtype, rows, cols, ld, gran, group, am);
        for (int64_t i = 0; i < ns; ++i) orc_scale_from_absmax(fmt, am[i], &scale[i], &inv[i]);
        free(am);
    }
    if (scales_out) memcpy(scales_out, scale, sizeof(float) * (size_t)ns);

    double sse = 0.0;
#pragma omp parallel for reduction(+ : sse) schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double row_sse = 0.0;
        for (int64_t c = 0; c < cols; ++c) {
            uint16_t raw = x[r * ld + c];
            float xv = orc_load(&raw, dtype);
            int64_t si = scale_index(gran, r, c, cols, group);
            float t = xv * inv[si];                          /* one binary32 multiply */
            int code = f.is_fp ? orc_encode_fp_arith(fmt, t, sign_bit16(raw)) : orc_encode_int(fmt, t);
            double value = orc_decode(fmt, code);
            double d = value * (double)scale[si];            /* exact in double */
            double e = (double)xv - d;
            row_sse += e * e;
            if (codes_out) codes_out[r * cols + c] = (uint8_t)code;
            if (dequant_out) dequant_out[r * cols + c] = orc_store((float)value * scale[si], dtype);
        }
        sse += row_sse;
    }
    if (sse_out) *sse_out = sse;
    free(scale);
    free(inv);
    return 0;
}

/* 4-bit packing used at the library boundary: element 2j in the low nibble of byte j. */
void orc_pack4(const uint8_t *codes, int64_t n, uint8_t *packed)
{
    for (int64_t j = 0; j < (n + 1) / 2; ++j) {
        uint8_t lo = codes[2 * j] & 0xF;
        uint8_t hi = (2 * j + 1 < n) ? (codes[2 * j + 1] & 0xF) : 0;
        packed[j] = (uint8_t)(lo | (hi << 4));
    }
}

/* ---- tensor error (Section 3.2 "Static (Weight) Tensor Analysis": MSE between quantised and
 *      original tensors), mean over the whole tensor whatever the scale granularity ------------- */
int orc_tensor_mse(const uint16_t *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                   int fmt, int gran, int group, double *mse_out)
{
    double sse;
    int rc = orc_quantize(x, dtype, rows, cols, ld, fmt, gran, group, NULL, NULL, NULL, NULL, &sse);
    if (rc) return rc;
    *mse_out = (rows > 0 && cols > 0) ? sse / (double)(rows * cols) : 0.0;
    return 0;
}

/* ---- layer output error (Section 3.2 "Layer (Operator) Analysis") -----------------------------
 * Linear layer A_out = W * A_in, stored as Y[t,o] = sum_i X[t,i] W[o,i].
 *   is_w_only != 0 : Yq = X . dq(W)^T            (W4A16-style)
 *   is_w_only == 0 : Yq = dq(X) . dq(W)^T        (W8A8-style), the same format for both tensors
 * W uses w_gran/w_group scales, X uses a_gran/a_group scales.
 * mse = mean (Y - Yq)^2 ; nsr = sum (Y - Yq)^2 / sum Y^2  (noise / signal power).
 * X: [T, in] dtype_x, W: [out, in] dtype_w; all sums in double.
 */
int orc_layer_output_error(const uint16_t *X, int dtype_x, int64_t T, int64_t ldx,
                           const uint16_t *W, int dtype_w, int64_t out, int64_t ldw, int64_t in,
                           int fmt, int is_w_only, int w_gran, int w_group, int a_gran, int a_group,
                           double *mse_out, double *nsr_out)
{
    fmt_t f;
    if (fmt_lookup(fmt, &f)) return -1;
    double *Xd = (double *)malloc(sizeof(double) * (size_t)(T * in));
    double *Xq = (double *)malloc(sizeof(double) * (size_t)(T * in));
    double *Wd = (double *)malloc(sizeof(double) * (size_t)(out * in));
    double *Wq = (double *)malloc(sizeof(double) * (size_t)(out * in));
    uint8_t *cw = (uint8_t *)malloc((size_t)(out * in));
    float *sw = (float *)malloc(sizeof(float) * (size_t)n_scales(w_gran, out, in, w_group));
    int rc = orc_quantize(W, dtype_w, out, in, ldw, fmt, w_gran, w_group, NULL, cw, sw, NULL, NULL);
    for (int64_t o = 0; o < out && !rc; ++o)
        for (int64_t i = 0; i < in; ++i) {
            Wd[o * in + i] = (double)orc_load(W + o * ldw + i, dtype_w);
            Wq[o * in + i] = orc_decode(fmt, cw[o * in + i]) * (double)sw[scale_index(w_gran, o, i, in, w_group)];
        }
    for (int64_t t = 0; t < T && !rc; ++t)
        for (int64_t i = 0; i < in; ++i)
            Xd[t * in + i] = (double)orc_load(X + t * ldx + i, dtype_x);
    if (!rc && !is_w_only) {
        uint8_t *cx = (uint8_t *)malloc((size_t)(T * in));
        float *sx = (float *)malloc(sizeof(float) * (size_t)n_scales(a_gran, T, in, a_group));
        rc = orc_quantize(X, dtype_x, T, in, ldx, fmt, a_gran, a_group, NULL, cx, sx, NULL, NULL);
        for (int64_t t = 0; t < T && !rc; ++t)
            for (int64_t i = 0; i < in; ++i)
                Xq[t * in + i] = orc_decode(fmt, cx[t * in + i]) * (double)sx[scale_index(a_gran, t, i, in, a_group)];
        free(cx);
        free(sx);
    } else if (!rc) {
        memcpy(Xq, Xd, sizeof(double) * (size_t)(T * in));
    }
    double noise = 0.0, signal = 0.0;
    if (!rc) {
#pragma omp parallel for reduction(+ : noise, signal) schedule(static)
        for (int64_t t = 0; t < T; ++t)
            for (int64_t o = 0; o < out; ++o) {
                double y = 0.0, yq = 0.0;
                for (int64_t i = 0; i < in; ++i) {
                    y += Xd[t * in + i] * Wd[o * in + i];
                    yq += Xq[t * in + i] * Wq[o * in + i];
                }
                noise += (y - yq) * (y - yq);
                signal += y * y;
            }
        *mse_out = (T > 0 && out > 0) ? noise / (double)(T * out) : 0.0;
        *nsr_out = signal > 0.0 ? noise / signal : 0.0;
    }
    free(Xd); free(Xq); free(Wd); free(Wq); free(cw); free(sw);
    return rc;
}

/* ---- Algorithm 1: keep the candidate with the strictly smallest error, in the caller's order -- */
int orc_select(const double *errors, int n)
{
    double min_error = INFINITY;
    int best = -1;
    for (int i = 0; i < n; ++i)
        if (errors[i] < min_error) { min_error = errors[i]; best = i; }
    return best;
}

/* ---- finer-than-layer selection (Section 7 names channel-wise / block-wise mixing of formats as the next step;
 *      Section 3.2 already scores per channel) ------------------------------------------------------------------
 * A "block" is one scale block: a row (per-channel scales) or a run of `group` elements of a row (group
 * scales).  Each block is quantised with its own abs-max scale; sse_out[b] is the block's sum of squared errors
 * in double.  Blocks are numbered like the scales: row-major, groups left to right.
 */
int orc_block_sse(const uint16_t *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                  int fmt, int gran, int group, double *sse_out)
{
    fmt_t f;
    if (fmt_lookup(fmt, &f)) return -1;
    if (gran == ORC_PER_GROUP && (group <= 0 || cols % group)) return -1;
    int64_t width = gran == ORC_PER_GROUP ? group : cols;     /* elements per block within a row */
    int64_t per_row = gran == ORC_PER_TENSOR ? 0 : cols / width;
    if (gran == ORC_PER_TENSOR) {                               /* degenerate: the whole tensor is the one block */
        return orc_quantize(x, dtype, rows, cols, ld, fmt, gran, group, NULL, NULL, NULL, NULL, sse_out);
    }
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < per_row; ++b) {
            const uint16_t *blk = x + r * ld + b * width;
            float amax = 0.0f;
            for (int64_t c = 0; c < width; ++c) {
                float a = fabsf(orc_load(blk + c, dtype));
                if (a > amax || isnan(a)) amax = a;
            }
            float scale, inv;
            orc_scale_from_absmax(fmt, amax, &scale, &inv);
            double sse = 0.0;
            for (int64_t c = 0; c < width; ++c) {
                float xv = orc_load(blk + c, dtype);
                float t = xv * inv;
                int code = f.is_fp ? orc_encode_fp_arith(fmt, t, sign_bit16(blk[c])) : orc_encode_int(fmt, t);
                double e = (double)xv - orc_decode(fmt, code) * (double)scale;
                sse += e * e;
            }
            sse_out[r * per_row + b] = sse;
        }
    return 0;
}

/* Per block, Algorithm 1's rule applied to the block errors: the first candidate (caller's order) with the strictly
 * smallest SSE.  choice_out[b] = index into fmts; mixed_mse_out = sum of the chosen SSEs / element count. */
int orc_select_blocks(const uint16_t *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                      const int *fmts, int n_fmts, int gran, int group, uint8_t *choice_out, double *block_sse_out,
                      double *mixed_mse_out)
{
    int64_t nb = n_scales(gran, rows, cols, group);
    double *sse = (double *)malloc(sizeof(double) * (size_t)(nb * n_fmts));
    int rc = 0;
    for (int k = 0; k < n_fmts && !rc; ++k)
        rc = orc_block_sse(x, dtype, rows, cols, ld, fmts[k], gran, group, sse + (int64_t)k * nb);
    double total = 0.0;
    for (int64_t b = 0; b < nb && !rc; ++b) {
        double e[8];
        for (int k = 0; k < n_fmts; ++k) e[k] = sse[(int64_t)k * nb + b];
        int best = orc_select(e, n_fmts);
        choice_out[b] = (uint8_t)best;
        total += e[best];
        if (block_sse_out)
            for (int k = 0; k < n_fmts; ++k) block_sse_out[b * n_fmts + k] = e[k];
    }
    if (!rc) *mixed_mse_out = (rows > 0 && cols > 0) ? total / (double)(rows * cols) : 0.0;
    free(sse);
    return rc;
}

/* ---- cross-check helper: arithmetic vs table FP rounding over a range of binary32 patterns ----
 * Compares the two encoders on every positive float whose bit pattern lies in [lo_bits, hi_bits]
 * (step `stride`) and returns the number of disagreements (first one stored in *first_bad).
 */
int64_t orc_crosscheck_fp(int fmt, uint32_t lo_bits, uint32_t hi_bits, uint32_t stride, uint32_t *first_bad)
{
    int64_t bad = 0;
    uint32_t fb = 0;
#pragma omp parallel for reduction(+ : bad) schedule(static)
    for (int64_t b = lo_bits; b <= (int64_t)hi_bits; b += stride) {
        uint32_t u = (uint32_t)b;
        float t;
        memcpy(&t, &u, 4);
        if (orc_encode_fp_arith(fmt, t, 0) != orc_encode_fp_table(fmt, t, 0)) {
            ++bad;
#pragma omp critical
            if (!fb) fb = u;
        }
    }
    if (first_bad) *first_bad = fb;
    return bad;
}

/* threads the OpenMP loops above will use (for reporting beside timings) */
int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
