// C ABI entry points: argument validation, workspace layout, the per-layer loop of Algorithm 1.
#include <algorithm>
#include <cmath>
#include <cstring>

#include "mofq_internal.h"

namespace mofq {

bool describe_format(int format, FmtDesc *d)
{
    FmtDesc f{};
    int E = 0;
    switch (format) {
    case MOFQ_INT4: f.bits = 4; f.Q = 7.0f; break;
    case MOFQ_INT8: f.bits = 8; f.Q = 127.0f; break;
    case MOFQ_FP4_E2M1: f.is_fp = 1; f.bits = 4; E = 2; f.M = 1; f.Q = 6.0f; break;
    case MOFQ_FP4_E2M1_IEEE: f.is_fp = 1; f.bits = 4; E = 2; f.M = 1; f.Q = 3.0f; break;
    case MOFQ_FP8_E4M3: f.is_fp = 1; f.bits = 8; E = 4; f.M = 3; f.Q = 448.0f; break;
    case MOFQ_FP8_E5M2: f.is_fp = 1; f.bits = 8; E = 5; f.M = 2; f.Q = 57344.0f; break;
    default: return false;
    }
    if (f.is_fp) {
        f.bias = (1 << (E - 1)) - 1;
        f.eminb = (uint32_t)(127 + 1 - f.bias) << 23;
        f.kadd = (uint32_t)(23 - f.M) << 23;
        f.min_normal = std::ldexp(1.0f, 1 - f.bias);
    }
    *d = f;
    return true;
}

// Map the caller's candidate list onto canonical kernel slots [INT][FP0][FP1].
int build_candset(const int32_t *formats, int n, int bit_width, CandSet *cs, int *perm, int *nc, int *fp_formats)
{
    if (!formats || n < 1 || n > MOFQ_MAX_CAND) return MOFQ_ERR_INVALID_ARG;
    CandSet c{};
    int fp_fmt[2] = {-1, -1};
    for (int i = 0; i < n; ++i) {
        FmtDesc d;
        if (!describe_format(formats[i], &d)) return MOFQ_ERR_INVALID_ARG;
        if (d.bits != bit_width) return MOFQ_ERR_UNSUPPORTED;
        if (!d.is_fp) {
            c.n_int = 1;
            c.int_q = d.Q;
        } else {
            int slot = -1;
            for (int k = 0; k < c.n_fp; ++k)
                if (fp_fmt[k] == formats[i]) slot = k;
            if (slot < 0) {
                if (c.n_fp == 2) return MOFQ_ERR_UNSUPPORTED;
                slot = c.n_fp++;
                fp_fmt[slot] = formats[i];
                c.fp_q[slot] = d.Q;
                c.fp_eminb[slot] = d.eminb;
                c.fp_kadd[slot] = d.kadd;
            }
        }
    }
    for (int i = 0; i < n; ++i) {
        FmtDesc d;
        describe_format(formats[i], &d);
        if (!d.is_fp) perm[i] = 0;
        else perm[i] = c.n_int + (fp_fmt[0] == formats[i] ? 0 : 1);
    }
    for (int i = n; i < MOFQ_MAX_CAND; ++i) perm[i] = 0;
    if (fp_formats) {
        fp_formats[0] = fp_fmt[0];
        fp_formats[1] = fp_fmt[1];
    }
    *cs = c;
    *nc = c.n_int + c.n_fp;
    return MOFQ_OK;
}

namespace {

int check_tensor(const mofq_tensor *x)
{
    if (!x || !x->data) return MOFQ_ERR_INVALID_ARG;
    if (x->dtype != MOFQ_F16 && x->dtype != MOFQ_BF16) return MOFQ_ERR_INVALID_ARG;
    if (x->rows <= 0 || x->cols <= 0 || x->ld < x->cols) return MOFQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x->data) & 15) || (x->cols & 7) || (x->ld & 7)) return MOFQ_ERR_MISALIGNED;
    return MOFQ_OK;
}

int check_gran(int gran, int group, int64_t cols)
{
    if (gran != MOFQ_PER_TENSOR && gran != MOFQ_PER_CHANNEL && gran != MOFQ_PER_GROUP) return MOFQ_ERR_INVALID_ARG;
    if (gran == MOFQ_PER_GROUP) {
        if (group < 8 || group > 256 || (group & (group - 1))) return MOFQ_ERR_UNSUPPORTED;  // power of two, 8..256
        if (cols % group) return MOFQ_ERR_UNSUPPORTED;
    }
    return MOFQ_OK;
}

int check_ws(const void *ws, size_t have, size_t need)
{
    if (!ws) return MOFQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return MOFQ_ERR_MISALIGNED;
    if (have < need) return MOFQ_ERR_WORKSPACE_TOO_SMALL;
    return MOFQ_OK;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

int check_config(const mofq_config *cfg)
{
    if (!cfg) return MOFQ_ERR_INVALID_ARG;
    if (cfg->bit_width != 4 && cfg->bit_width != 8) return MOFQ_ERR_INVALID_ARG;
    if (cfg->n_candidates < 1 || cfg->n_candidates > MOFQ_MAX_CAND) return MOFQ_ERR_INVALID_ARG;
    if (cfg->metric != MOFQ_TENSOR_MSE && cfg->metric != MOFQ_LAYER_OUTPUT_MSE) return MOFQ_ERR_INVALID_ARG;
    if (cfg->w_gran2 != MOFQ_GRAN_NONE && cfg->metric != MOFQ_TENSOR_MSE) return MOFQ_ERR_UNSUPPORTED;
    return MOFQ_OK;
}

// tensor metric for one layer: enqueue the scoring of W and the record(s) for it
// clear_header: the call has not cleared the workspace header yet
int score_layer_tensor(const mofq_tensor &W, const mofq_config *cfg, const CandSet &cs, const int *perm, int nc,
                       const int *fp_formats, mofq_result *res, float *mse_out, void *ws, cudaStream_t st, bool clear_header = false)
{
    if (int rc = check_tensor(&W)) return rc;
    if (int rc = check_gran(cfg->w_gran, cfg->w_group, W.cols)) return rc;
    if (cfg->w_gran2 != MOFQ_GRAN_NONE) {
        if (int rc = check_gran(cfg->w_gran2, cfg->w_group, W.cols)) return rc;
        if (cfg->w_gran2 == cfg->w_gran) return MOFQ_ERR_INVALID_ARG;
    }
    // a large dense tensor with group scales goes through the multi-tensor kernel as a list of one layer (its three
    // small helper launches cost more than they save below a few tens of MB)
    mofq_layer one{};
    one.W = W;
    if (cfg->metric == MOFQ_TENSOR_MSE && W.rows * W.cols >= (32LL << 20) && mt_applicable(&one, 1, cfg) &&
        sizeof(WsHeader) + mt_ws_bytes(1) <= score_ws_bytes()) {
        if (clear_header && cudaMemsetAsync(ws, 0, sizeof(WsHeader), st) != cudaSuccess) return MOFQ_ERR_CUDA;
        return mt_run(&one, 1, cfg, cs, perm, nc, fp_formats, res, static_cast<char *>(ws) + sizeof(WsHeader), st, mse_out,
                      res ? nullptr : &static_cast<WsHeader *>(ws)->status);   // a record carries its own status
    }
    ScoreJob job{};
    job.x = W;
    job.cs = cs;
    job.gran = cfg->w_gran;
    job.gran2 = cfg->w_gran2;
    job.group = cfg->w_group;
    job.fp_formats[0] = fp_formats[0];
    job.fp_formats[1] = fp_formats[1];
    job.hdr = static_cast<WsHeader *>(ws);
    job.partials = reinterpret_cast<double *>(static_cast<char *>(ws) + sizeof(WsHeader));
    job.fin.mse_out = mse_out;
    job.fin.res = res;
    job.fin.status_out = nullptr;
    job.fin.n_cand = cfg->n_candidates;
    job.fin.n_sets = cfg->w_gran2 != MOFQ_GRAN_NONE ? 2 : 1;
    job.fin.nc = nc;
    std::memcpy(job.fin.perm, perm, sizeof(job.fin.perm));
    job.fin.inv_n = 1.0 / ((double)W.rows * (double)W.cols);
    job.clear_header = clear_header;
    return launch_score(job, st);
}

}  // namespace
}  // namespace mofq

using namespace mofq;

extern "C" {

int mofq_format_bits(int format)
{
    FmtDesc d;
    return describe_format(format, &d) ? d.bits : -1;
}

float mofq_format_max(int format)
{
    FmtDesc d;
    return describe_format(format, &d) ? d.Q : 0.0f;
}

const char *mofq_status_string(int status)
{
    switch (status) {
    case MOFQ_OK: return "ok";
    case MOFQ_ERR_INVALID_ARG: return "invalid argument";
    case MOFQ_ERR_UNSUPPORTED: return "unsupported combination of arguments";
    case MOFQ_ERR_MISALIGNED: return "pointer or leading dimension not aligned";
    case MOFQ_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MOFQ_ERR_CUDA: return "CUDA runtime error";
    case MOFQ_ERR_SCRATCH_LIMIT: return "tensor too large for the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
    }
}

size_t mofq_tensor_workspace_bytes(const mofq_tensor *) { return align256(score_ws_bytes()); }

size_t mofq_workspace_bytes(const mofq_layer *layers, int n_layers, const mofq_config *cfg)
{
    size_t need = align256(score_ws_bytes());
    if (cfg && cfg->metric == MOFQ_LAYER_OUTPUT_MSE && layers) need += layer_metric_ws_bytes(layers, n_layers, cfg);
    if (cfg && layers && n_layers > 0 && mt_applicable(layers, n_layers, cfg)) need += mt_ws_bytes(n_layers);
    else if (cfg && layers && n_layers > 0 && rows_mt_applicable(layers, n_layers, cfg)) need += rows_mt_ws_bytes(n_layers);
    return need;
}

size_t mofq_host_workspace_bytes(const mofq_layer *layers, int n_layers, const mofq_config *cfg)
{
    if (!layers || !cfg || n_layers <= 0) return 0;
    size_t stage = 0;
    for (int i = 0; i < n_layers; ++i) {
        size_t b = align256((size_t)layers[i].W.rows * layers[i].W.cols * 2);
        if (layers[i].X.data) b += align256((size_t)layers[i].X.rows * layers[i].X.cols * 2);
        stage = std::max(stage, b);
    }
    const int n_sets = cfg->w_gran2 != MOFQ_GRAN_NONE ? 2 : 1;
    return mofq_workspace_bytes(layers, n_layers, cfg) + stage + align256(sizeof(mofq_result) * (size_t)n_layers * n_sets);
}

int mofq_quantize_tensor(const mofq_tensor *x, int format, int gran, int group, const float *scales_in,
                         void *codes_out, float *scales_out, void *dequant_out, void *workspace,
                         size_t workspace_bytes, void *stream)
{
    if (int rc = check_tensor(x)) return rc;
    FmtDesc f;
    if (!describe_format(format, &f)) return MOFQ_ERR_INVALID_ARG;
    if (int rc = check_gran(gran, group, x->cols)) return rc;
    if (int rc = check_ws(workspace, workspace_bytes, mofq_tensor_workspace_bytes(x))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st) != cudaSuccess) return MOFQ_ERR_CUDA;
    return launch_emit(*x, f, gran, group, scales_in, codes_out, scales_out, dequant_out, nullptr, MOFQ_F16,
                       static_cast<WsHeader *>(workspace), st, format);
}

int mofq_tensor_error(const mofq_tensor *x, const int32_t *formats, int n, int gran, int gran2, int group,
                      float *mse_out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (int rc = check_tensor(x)) return rc;
    if (!mse_out || !formats || n < 1 || n > MOFQ_MAX_CAND) return MOFQ_ERR_INVALID_ARG;
    FmtDesc d0;
    if (!describe_format(formats[0], &d0)) return MOFQ_ERR_INVALID_ARG;
    mofq_config cfg{};
    cfg.bit_width = d0.bits;
    cfg.n_candidates = n;
    for (int i = 0; i < n; ++i) cfg.candidates[i] = formats[i];
    cfg.is_w_only = 1;
    cfg.w_gran = gran;
    cfg.w_gran2 = gran2;
    cfg.w_group = group;
    cfg.metric = MOFQ_TENSOR_MSE;
    CandSet cs;
    int perm[MOFQ_MAX_CAND], nc, fp_formats[2];
    if (int rc = build_candset(formats, n, d0.bits, &cs, perm, &nc, fp_formats)) return rc;
    if (int rc = check_gran(gran, group, x->cols)) return rc;
    if (gran2 != MOFQ_GRAN_NONE) {
        if (int rc = check_gran(gran2, group, x->cols)) return rc;
        if (gran2 == gran) return MOFQ_ERR_INVALID_ARG;
    }
    if (int rc = check_ws(workspace, workspace_bytes, mofq_tensor_workspace_bytes(x))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return score_layer_tensor(*x, &cfg, cs, perm, nc, fp_formats, nullptr, mse_out, workspace, st, true);
}

int mofq_select_blocks(const mofq_tensor *x, const int32_t *formats, int n, int gran, int group, uint8_t *choice_out,
                       float *block_sse_out, float *mse_out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (int rc = check_tensor(x)) return rc;
    if (!choice_out || !mse_out || !formats || n < 1 || n > MOFQ_MAX_CAND - 1) return MOFQ_ERR_INVALID_ARG;
    if (gran != MOFQ_PER_CHANNEL && gran != MOFQ_PER_GROUP) return MOFQ_ERR_UNSUPPORTED;
    if (int rc = check_gran(gran, group, x->cols)) return rc;
    FmtDesc d0;
    if (!describe_format(formats[0], &d0)) return MOFQ_ERR_INVALID_ARG;
    CandSet cs;
    int perm[MOFQ_MAX_CAND], nc, fp_formats[2];
    if (int rc = build_candset(formats, n, d0.bits, &cs, perm, &nc, fp_formats)) return rc;
    if (int rc = check_ws(workspace, workspace_bytes, mofq_tensor_workspace_bytes(x))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st) != cudaSuccess) return MOFQ_ERR_CUDA;
    // a large dense tensor with group-128 blocks: the TMA-fed persistent kernel, as a list of one layer, in its
    // block-wise form (smaller tensors, other block widths and strided ones: the register-resident kernel below)
    if (gran == MOFQ_PER_GROUP && mt_blocks_applicable(*x, group, cs, fp_formats) && sizeof(WsHeader) + mt_ws_bytes(1) <= score_ws_bytes()) {
        mofq_config cfg{};
        cfg.bit_width = d0.bits;
        cfg.n_candidates = n;
        for (int i = 0; i < n; ++i) cfg.candidates[i] = formats[i];
        cfg.is_w_only = 1;
        cfg.w_gran = MOFQ_PER_GROUP;
        cfg.w_gran2 = MOFQ_GRAN_NONE;
        cfg.w_group = group;
        cfg.metric = MOFQ_TENSOR_MSE;
        mofq_layer one{};
        one.W = *x;
        BlockSel bs{};
        bs.choice = choice_out;
        bs.block_sse = block_sse_out;
        bs.n_cand = n;
        std::memcpy(bs.perm, perm, sizeof(bs.perm));
        return mt_run(&one, 1, &cfg, cs, perm, nc, fp_formats, nullptr, static_cast<char *>(workspace) + sizeof(WsHeader), st, mse_out,
                      &static_cast<WsHeader *>(workspace)->status, &bs);
    }
    ScoreJob job{};
    job.x = *x;
    job.cs = cs;
    job.gran = gran;
    job.gran2 = MOFQ_GRAN_NONE;
    job.group = group;
    job.fp_formats[0] = fp_formats[0];
    job.fp_formats[1] = fp_formats[1];
    job.hdr = static_cast<WsHeader *>(workspace);
    job.partials = reinterpret_cast<double *>(static_cast<char *>(workspace) + sizeof(WsHeader));
    job.fin.mse_out = mse_out;
    job.fin.n_cand = n;
    job.fin.n_sets = 1;
    job.fin.nc = nc;
    std::memcpy(job.fin.perm, perm, sizeof(job.fin.perm));
    job.fin.inv_n = 1.0 / ((double)x->rows * (double)x->cols);
    return launch_select_blocks(job, choice_out, block_sse_out, st);
}

int mofq_absmax_update(const mofq_tensor *x, float *absmax_inout, void *stream)
{
    if (int rc = check_tensor(x)) return rc;
    if (!absmax_inout) return MOFQ_ERR_INVALID_ARG;
    return launch_absmax_update(*x, absmax_inout, static_cast<cudaStream_t>(stream));
}

int mofq_tensor_error_scaled(const mofq_tensor *x, const int32_t *formats, int n, const float *scales_in, float *mse_out,
                             void *workspace, size_t workspace_bytes, void *stream)
{
    if (int rc = check_tensor(x)) return rc;
    if (!mse_out || !scales_in || !formats || n < 1 || n > MOFQ_MAX_CAND) return MOFQ_ERR_INVALID_ARG;
    FmtDesc d0;
    if (!describe_format(formats[0], &d0)) return MOFQ_ERR_INVALID_ARG;
    CandSet cs;
    int perm[MOFQ_MAX_CAND], nc, fp_formats[2];
    if (int rc = build_candset(formats, n, d0.bits, &cs, perm, &nc, fp_formats)) return rc;
    // every candidate carries a scale of its own, so a format may appear only once (a repeat would share a kernel slot,
    // and with it one scale)
    for (int i = 0; i < n; ++i)
        for (int k = 0; k < i; ++k)
            if (formats[i] == formats[k]) return MOFQ_ERR_UNSUPPORTED;
    if (x->cols / 8 > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
    if (int rc = check_ws(workspace, workspace_bytes, mofq_tensor_workspace_bytes(x))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st) != cudaSuccess) return MOFQ_ERR_CUDA;
    ScoreJob job{};
    job.x = *x;
    job.cs = cs;
    job.gran = MOFQ_PER_TENSOR;
    job.gran2 = MOFQ_GRAN_NONE;
    job.hdr = static_cast<WsHeader *>(workspace);
    job.partials = reinterpret_cast<double *>(static_cast<char *>(workspace) + sizeof(WsHeader));
    job.fin.mse_out = mse_out;
    job.fin.n_cand = n;
    job.fin.n_sets = 1;
    job.fin.nc = nc;
    std::memcpy(job.fin.perm, perm, sizeof(job.fin.perm));
    job.fin.inv_n = 1.0 / ((double)x->rows * (double)x->cols);
    return launch_score_supplied(job, scales_in, st);
}

int mofq_layer_output_error(const mofq_layer *L, const mofq_config *cfg, float *mse_out, float *nsr_out,
                            void *workspace, size_t workspace_bytes, void *stream)
{
    if (!L || !mse_out || !nsr_out) return MOFQ_ERR_INVALID_ARG;
    if (int rc = check_config(cfg)) return rc;
    if (int rc = check_tensor(&L->W)) return rc;
    if (int rc = check_tensor(&L->X)) return rc;
    mofq_config c = *cfg;
    c.metric = MOFQ_LAYER_OUTPUT_MSE;
    c.w_gran2 = MOFQ_GRAN_NONE;
    if (int rc = layer_metric_check(*L, &c)) return rc;
    if (int rc = check_ws(workspace, workspace_bytes, mofq_workspace_bytes(L, 1, &c))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st) != cudaSuccess) return MOFQ_ERR_CUDA;
    return layer_metric_run(*L, &c, nullptr, mse_out, nsr_out, workspace, workspace_bytes, st);
}

int mofq_select_formats(const mofq_layer *layers, int n_layers, const mofq_config *cfg, mofq_result *results_out,
                        void *workspace, size_t workspace_bytes, void *stream)
{
    if (!layers || n_layers <= 0 || !results_out) return MOFQ_ERR_INVALID_ARG;
    if (int rc = check_config(cfg)) return rc;
    CandSet cs;
    int perm[MOFQ_MAX_CAND], nc, fp_formats[2];
    if (int rc = build_candset(cfg->candidates, cfg->n_candidates, cfg->bit_width, &cs, perm, &nc, fp_formats)) return rc;
    if (int rc = check_ws(workspace, workspace_bytes, mofq_workspace_bytes(layers, n_layers, cfg))) return rc;
    // validate everything before anything is enqueued
    for (int i = 0; i < n_layers; ++i) {
        if (int rc = check_tensor(&layers[i].W)) return rc;
        if (int rc = check_gran(cfg->w_gran, cfg->w_group, layers[i].W.cols)) return rc;
        if (cfg->w_gran2 != MOFQ_GRAN_NONE) {
            if (int rc = check_gran(cfg->w_gran2, cfg->w_group, layers[i].W.cols)) return rc;
            if (cfg->w_gran2 == cfg->w_gran) return MOFQ_ERR_INVALID_ARG;
        }
        if (cfg->metric == MOFQ_LAYER_OUTPUT_MSE) {
            if (int rc = check_tensor(&layers[i].X)) return rc;
            if (layers[i].X.cols != layers[i].W.cols) return MOFQ_ERR_INVALID_ARG;
            if (int rc = layer_metric_check(layers[i], cfg)) return rc;
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mt_applicable(layers, n_layers, cfg))  // one persistent launch over the whole layer list
        return mt_run(layers, n_layers, cfg, cs, perm, nc, fp_formats, results_out,
                      static_cast<char *>(workspace) + align256(score_ws_bytes()), st);
    if (rows_mt_applicable(layers, n_layers, cfg))  // per-channel scales: one persistent launch over whole-row tiles
        return rows_mt_run(layers, n_layers, cfg, cs, perm, nc, fp_formats, results_out,
                           static_cast<char *>(workspace) + align256(score_ws_bytes()), st);
    if (cfg->metric != MOFQ_TENSOR_MSE && cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st) != cudaSuccess) return MOFQ_ERR_CUDA;
    const int n_sets = cfg->w_gran2 != MOFQ_GRAN_NONE ? 2 : 1;
    for (int i = 0; i < n_layers; ++i) {  // Algorithm 1: for layer in model.layers_to_quant
        int rc;
        if (cfg->metric == MOFQ_TENSOR_MSE)   // (the first layer's launch clears the workspace header)
            rc = score_layer_tensor(layers[i].W, cfg, cs, perm, nc, fp_formats, results_out + (size_t)i * n_sets, nullptr, workspace, st, i == 0);
        else
            rc = layer_metric_run(layers[i], cfg, results_out + i, nullptr, nullptr, workspace, workspace_bytes, st, i > 0);
        if (rc) return rc;
    }
    return MOFQ_OK;
}

int mofq_emit_selected(const mofq_layer *layers, int n_layers, const mofq_config *cfg, const mofq_result *results,
                       const mofq_packed *out, int32_t *formats_out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!layers || n_layers <= 0 || !results || !out) return MOFQ_ERR_INVALID_ARG;
    if (int rc = check_config(cfg)) return rc;
    if (int rc = check_ws(workspace, workspace_bytes, sizeof(WsHeader))) return rc;
    EmitSel sel{};
    for (int c = 0; c < cfg->n_candidates; ++c) {
        if (!describe_format(cfg->candidates[c], &sel.cand[c]) || sel.cand[c].bits != cfg->bit_width) return MOFQ_ERR_INVALID_ARG;
        sel.format[c] = cfg->candidates[c];
    }
    for (int i = 0; i < n_layers; ++i) {
        if (int rc = check_tensor(&layers[i].W)) return rc;
        if (int rc = check_gran(cfg->w_gran, cfg->w_group, layers[i].W.cols)) return rc;
        if (!out[i].codes || !out[i].scales) return MOFQ_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st) != cudaSuccess) return MOFQ_ERR_CUDA;
    const int n_sets = cfg->w_gran2 != MOFQ_GRAN_NONE ? 2 : 1;
    for (int i = 0; i < n_layers; ++i) {  // Algorithm 1, last step: the layer keeps the quantisation of its best format
        sel.res = results + (size_t)i * n_sets;
        sel.tag_out = formats_out ? formats_out + i : nullptr;
        if (int rc = launch_emit(layers[i].W, sel.cand[0], cfg->w_gran, cfg->w_group, nullptr, out[i].codes, out[i].scales, nullptr,
                                 nullptr, MOFQ_F16, static_cast<WsHeader *>(workspace), st, -1, &sel, i > 0))
            return rc;
    }
    return MOFQ_OK;
}

int mofq_select_formats_host(const mofq_layer *layers, int n_layers, const mofq_config *cfg, mofq_result *results_host,
                             void *workspace, size_t workspace_bytes, void *stream)
{
    if (!layers || n_layers <= 0 || !results_host) return MOFQ_ERR_INVALID_ARG;
    if (int rc = check_config(cfg)) return rc;
    const size_t need = mofq_host_workspace_bytes(layers, n_layers, cfg);
    if (int rc = check_ws(workspace, workspace_bytes, need)) return rc;
    for (int i = 0; i < n_layers; ++i) {
        if (!layers[i].W.data || layers[i].W.rows <= 0 || layers[i].W.cols <= 0 || layers[i].W.ld != layers[i].W.cols)
            return MOFQ_ERR_INVALID_ARG;  // host tensors must be dense
        if (cfg->metric == MOFQ_LAYER_OUTPUT_MSE && (!layers[i].X.data || layers[i].X.ld != layers[i].X.cols))
            return MOFQ_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_sets = cfg->w_gran2 != MOFQ_GRAN_NONE ? 2 : 1;
    const size_t inner = mofq_workspace_bytes(layers, n_layers, cfg);
    const size_t res_bytes = align256(sizeof(mofq_result) * (size_t)n_layers * n_sets);
    char *base = static_cast<char *>(workspace);
    mofq_result *res_dev = reinterpret_cast<mofq_result *>(base + inner);
    char *stage = base + inner + res_bytes;
    for (int i = 0; i < n_layers; ++i) {
        mofq_layer one = layers[i];
        const size_t wb = (size_t)one.W.rows * one.W.cols * 2;
        if (cudaMemcpyAsync(stage, one.W.data, wb, cudaMemcpyHostToDevice, st) != cudaSuccess) return MOFQ_ERR_CUDA;
        one.W.data = stage;
        if (cfg->metric == MOFQ_LAYER_OUTPUT_MSE) {
            char *xs = stage + align256(wb);
            if (cudaMemcpyAsync(xs, one.X.data, (size_t)one.X.rows * one.X.cols * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
                return MOFQ_ERR_CUDA;
            one.X.data = xs;
        }
        // one layer at a time: the staging buffer is reused in stream order
        if (int rc = mofq_select_formats(&one, 1, cfg, res_dev + (size_t)i * n_sets, workspace, inner, st)) return rc;
    }
    if (cudaMemcpyAsync(results_host, res_dev, sizeof(mofq_result) * (size_t)n_layers * n_sets, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return MOFQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MOFQ_ERR_CUDA;
    return MOFQ_OK;
}

}  // extern "C"
