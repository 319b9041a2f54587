// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <utility>

#include "mofq.h"

namespace mofq {

// ---- chained launches ------------------------------------------------------------------------------------
// The kernels of one library call that follow one another on the stream are launched with programmatic stream
// serialisation: the next kernel's blocks may be scheduled and run their prologue while the previous kernel drains.
// Every such kernel calls chain_enter() before its first global-memory access: it returns once the previous kernel
// has completed and its writes are visible, so the order of the data is the plain stream order; what is saved is the
// launch gap between short kernels.  Without the launch attribute both instructions do nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_enter()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
}
// The other form: a kernel entered with chain_enter_early() lets the launch chained behind it start at once; that
// launch may read its inputs freely and calls chain_leave() before the first access to anything the earlier kernel
// writes (used for the header clear in front of a single tensor's scoring launch).
__device__ __forceinline__ void chain_enter_early() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void chain_leave() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool chained,
                                  Args &&...args)
{
    cudaLaunchConfig_t lc{};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = chained ? 1 : 0;
    return cudaLaunchKernelEx(&lc, kernel, std::forward<Args>(args)...);
}

// ---- format description used by the kernels ------------------------------------------------------
// FP grid with E exponent bits, M mantissa bits, bias 2^(E-1)-1 (Section 2; Table 3 for E2M1):
//   Q      largest finite magnitude (abs-max maps here)
//   eminb  binary32 exponent field of the smallest normal 2^(1-bias), shifted into place
//   kadd   (23 - M) << 23: added to an exponent field it yields the power of two whose ulp is the
//          grid spacing of that binade
struct FmtDesc {
    int is_fp, bits, M, bias;
    float Q;
    uint32_t eminb, kadd;
    float min_normal;
};

// Candidate set in canonical slot order: [INT (if any)] [FP 0] [FP 1].
struct CandSet {
    int n_int, n_fp;
    float int_q;
    float fp_q[2];
    uint32_t fp_eminb[2], fp_kadd[2];
};

// abs-max targets of a candidate set's canonical slots and their rounded reciprocals (for the division-free scales)
struct RowQ {
    float q[3];   // abs-max target per canonical slot
    float rq[3];  // RN32(1 / q)
};
inline RowQ candset_rowq(const CandSet &cs)
{
    RowQ rq{};
    if (cs.n_int) rq.q[0] = cs.int_q;
    for (int f = 0; f < cs.n_fp; ++f) rq.q[cs.n_int + f] = cs.fp_q[f];
    for (int j = 0; j < 3; ++j) rq.rq[j] = rq.q[j] > 0.0f ? 1.0f / rq.q[j] : 0.0f;
    return rq;
}

constexpr int kMaxAcc = 8;        // accumulators per block: up to 2 granularities x 3 canonical slots (padded)
constexpr int kMaxSlots = 2048;   // most thread blocks a scoring kernel is launched with

// Header of the scoring workspace (device).  Zero before the first launch; every kernel that uses
// it leaves counter and absmax_bits zero again, and the last block moves `status` into the output.
struct WsHeader {
    int32_t status;        // MOFQ_STATUS_* bits of the running call
    uint32_t counter;      // blocks finished (last-block-done reduction)
    uint32_t absmax_bits;  // per-tensor abs-max as a 16-bit magnitude pattern
    uint32_t pad[61];
};
static_assert(sizeof(WsHeader) == 256, "header is one 256-byte line");

// What the last block writes once all partial sums are in.
struct Finalize {
    float *mse_out;        // nullable: [set][candidate] floats, caller's order
    mofq_result *res;      // nullable: one record per set
    int32_t *status_out;   // nullable: receives the status bits (else they stay in the header)
    int n_cand, n_sets, nc;
    int perm[MOFQ_MAX_CAND];   // caller's candidate index -> canonical slot
    double inv_n;          // 1 / element count
};

// Outputs of block-wise selection (one winner per scale block).
struct BlockSel {
    uint8_t *choice;     // [blocks] index into the caller's candidate list
    float *block_sse;    // nullable: [blocks][n_cand], caller's order
    int n_cand;
    int perm[MOFQ_MAX_CAND];   // caller's candidate index -> canonical slot
};

struct ScoreJob {
    mofq_tensor x;
    CandSet cs;
    int gran, gran2, group;    // gran2 = MOFQ_GRAN_NONE or second granularity
    int fp_formats[2];         // mofq_format held by each canonical FP slot (-1 if unused)
    Finalize fin;
    WsHeader *hdr;
    double *partials;          // kMaxSlots * kMaxAcc doubles
    bool clear_header;         // the call has not cleared *hdr yet: launch_score does it (for a single tensor on the
                               // streamed-rows route with a kernel that the scoring launch overlaps, else with a memset)
};

inline size_t score_ws_bytes() { return sizeof(WsHeader) + sizeof(double) * kMaxSlots * kMaxAcc; }

bool describe_format(int format, FmtDesc *d);
// fp_formats (nullable, 2 entries): the mofq_format held by each canonical FP slot
int build_candset(const int32_t *formats, int n, int bit_width, CandSet *cs, int *perm, int *nc, int *fp_formats = nullptr);

// One layer of the multi-tensor scoring kernel's work table (device memory).
struct MtLayer {
    const uint16_t *x;      // dense tensor
    long long n_groups;     // scale blocks in the tensor
    long long tile_begin;   // index of the layer's first tile in the concatenated tile list
    double inv_n;           // 1 / element count
    int first_cta;          // first block that owns a tile of this layer
    int n_slots;            // partial-sum slots of this layer (blocks spanning it x consumer warps)
    int slot_off;           // first slot
    int pad;
};

// multi-tensor path (mofq_kq_mt.cu)
bool mt_applicable(const mofq_layer *layers, int n_layers, const mofq_config *cfg);
size_t mt_ws_bytes(int n_layers);
// bs (one dense tensor with group-128 scales only): also pick a winner per group; mse_out then has one more entry, the
// error of the mixture.  mt_blocks_applicable says whether that form exists for the candidate set.
bool mt_blocks_applicable(const mofq_tensor &W, int group, const CandSet &cs, const int *fp_formats);
int mt_run(const mofq_layer *layers, int n_layers, const mofq_config *cfg, const CandSet &cs, const int *perm, int nc,
           const int *fp_formats, mofq_result *results /* nullable */, void *ws, cudaStream_t st,
           float *mse_out = nullptr /* [layer][candidate] */, int32_t *status_out = nullptr /* OR of the layers' status bits */,
           const BlockSel *bs = nullptr);
int sm_count();

// streamed-rows path (mofq_kq_rows.cu): per-channel scales, alone or with group-128 scales from the same read
bool rows_single_applicable(const ScoreJob &job);
int rows_single_run(const ScoreJob &job, cudaStream_t st);
bool rows_mt_applicable(const mofq_layer *layers, int n_layers, const mofq_config *cfg);
size_t rows_mt_ws_bytes(int n_layers);
int rows_mt_run(const mofq_layer *layers, int n_layers, const mofq_config *cfg, const CandSet &cs, const int *perm, int nc,
                const int *fp_formats, mofq_result *results, void *ws, cudaStream_t st);

// Format of an emit launch picked ON THE DEVICE from a selection record (Algorithm 1's last step without a host
// round trip): the kernel quantises with cand[res->chosen] and stores that candidate's mofq_format in *tag_out.
struct EmitSel {
    const mofq_result *res;   // nullptr: the launch uses the format passed by value
    int32_t *tag_out;         // nullable
    FmtDesc cand[MOFQ_MAX_CAND];
    int32_t format[MOFQ_MAX_CAND];
};

// kernels' host launchers (mofq_kq.cu)
int launch_score(const ScoreJob &job, cudaStream_t st);
int launch_absmax(const mofq_tensor &x, WsHeader *hdr, cudaStream_t st, bool chained = false /* follows a kernel of the same call */);
int launch_absmax_update(const mofq_tensor &x, float *absmax_inout, cudaStream_t st);
int launch_score_supplied(const ScoreJob &job, const float *scales, cudaStream_t st);
// one winner per scale block; job.fin.mse_out receives n_cand + 1 floats (candidates, then the mixture)
int launch_select_blocks(const ScoreJob &job, uint8_t *choice, float *block_sse, cudaStream_t st);
int launch_emit(const mofq_tensor &x, const FmtDesc &f, int gran, int group, const float *scales_in,
                void *codes_out, float *scales_out, void *dequant_out, void *values_out, int values_dtype,
                WsHeader *hdr, cudaStream_t st, int format_id = -1 /* mofq_format of f: enables the fused code kernel */,
                const EmitSel *sel = nullptr /* format chosen on the device; f then only fixes the code width */,
                bool overlap_prev = false /* the previous launch on st is the previous layer's emission of the same call */);
// x16_out / alpha_out (bf16 tensors only, nullable): also write the tensor as binary16, scaled by the power of two that
// puts its abs-max in [2^13, 2^14) (exact unless a value is more than 2^27 times smaller than the abs-max), and 1 / that power
int launch_emit_codes_uniform(const mofq_tensor &x, int n, const int *formats, void *const *codes, float *const *scales,
                              WsHeader *hdr, cudaStream_t st, uint16_t *x16_out = nullptr, float *alpha_out = nullptr,
                              bool chained = false);
int launch_emit_codes_rows(const mofq_tensor &x, int n, const int *formats, void *const *codes, float *const *scales,
                           WsHeader *hdr, cudaStream_t st, bool chained = false);

// layer-output metric (mofq_layer.cu): extra workspace beyond the scoring workspace, and one layer's run.
// Exactly one of `res` (selection record) or `mse_out`/`nsr_out` (raw errors, caller's order) is given.
size_t layer_metric_ws_bytes(const mofq_layer *layers, int n_layers, const mofq_config *cfg);
// the argument combinations layer_metric_run refuses (host-side checks only; nothing is enqueued)
int layer_metric_check(const mofq_layer &L, const mofq_config *cfg);
// after_own: the previous launch on st is the last kernel of the previous layer of the same call
int layer_metric_run(const mofq_layer &L, const mofq_config *cfg, mofq_result *res, float *mse_out, float *nsr_out,
                     void *workspace, size_t workspace_bytes, cudaStream_t st, bool after_own = false);

}  // namespace mofq
