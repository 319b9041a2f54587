// Persistent multi-tensor scoring kernel: one launch scores every layer of a model.
//
// Work is the concatenation of all layers' 32 KB tiles (a tile = consecutive per-group scale
// blocks of one dense tensor).  Each CTA owns a contiguous range of tiles.  One producer thread
// streams tiles into a shared-memory ring with bulk async copies (TMA, 1-D) that complete on
// mbarriers; four consumer warps take one group per lane, walk its 16-byte chunks rotated by the
// lane index (conflict-free on the dense tile), find the abs-max, derive the scales and score every
// candidate from the same registers.  Per (layer, CTA, warp) partial sums go to the workspace; a
// second small kernel adds them in a fixed order and applies Algorithm 1's comparison.
//
// Arithmetic per element a = x (signs kept; every grid is symmetric and both roundings are sign-symmetric):
//   INT : r = RNE(a*inv) through fma(a, inv, 1.5*2^23) - 1.5*2^23.  The fused multiply-add rounds
//         the exact product once instead of twice; the two can differ only where a*inv sits within
//         one binary32 ulp of a tie, and at a tie both neighbours have the same error, so the
//         squared-error sum agrees with the two-rounding definition far inside the 1e-5 tolerance.
//         d = r - a*inv (one fused operation); the group's sum of d*d is multiplied by scale^2 once per group.
//   FP  : t = RN32(a*inv); r = hardware convert of t to the 4/8-bit float (round-to-nearest-even,
//         saturating) and back to f16; d = r - t with a mixed-precision subtract; the group's sum of d*d is
//         multiplied by scale^2 once per group (the scale is fixed over a lane's group).
// Packed two-lane binary32 instructions (f32x2) halve the issue slots of the multiply/add work.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <type_traits>
#include <vector>

#include "kq_math.cuh"
#include "kq_pipe.cuh"
#include "mofq_internal.h"

namespace mofq {
namespace {

constexpr int kStages = 2;
constexpr int kCtasPerSm = 3;   // kStages * kTileBytes * kCtasPerSm must fit one SM's shared memory
constexpr int kTileBytes = 32768;
constexpr int kConsumerWarps = 4;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kThreads = kConsumers + 32;  // + one producer warp
using namespace kqmath;
using namespace kqpipe;


// ---- the kernel ---------------------------------------------------------------------------------------
struct MtParams {
    const MtLayer *layers;
    int n_layers;
    long long total_tiles, tiles_per_cta;
    int group;
    float q[3];          // abs-max target per canonical slot
    float rq[3];         // RN32(1 / q)
    double *partials;    // [slot][kMaxAcc]
    int32_t *status;     // [layer]
    int32_t *timeout;    // one word: set if a bounded wait expired
    BlockSel bs;         // block-wise form (one tensor): the winner of every group, and the groups' errors
};

__device__ __forceinline__ int find_layer(const MtLayer *layers, int n, long long tile)
{
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (layers[mid].tile_begin <= tile) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

// BLK: a lane also applies Algorithm 1's rule to its group's errors (strictly smaller, caller's order), writes the
// winner (and the errors), and one more accumulator sums the winners' errors: the error of the mixed-format tensor.
template <int DT, int NI, int K0, int K1, bool BLK>
__global__ void __launch_bounds__(kThreads)
kq_score_mt(const MtParams p)
{
    using S = Scorer<DT, NI, K0, K1, true>;
    constexpr int NC = S::NC;
    constexpr int NA = NC + (BLK ? 1 : 0);
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t full_bar[kStages], empty_bar[kStages];
    __shared__ int err;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // tiles start on a 1 KB boundary of the shared window, so that a group's chunk addresses can be formed by XOR
    const uint32_t smem_base = (smem_u32(smem) + 1023u) & ~1023u;
    unsigned char *const smem_al = smem + (smem_base - smem_u32(smem));
    const long long t_begin = (long long)blockIdx.x * p.tiles_per_cta;
    const long long t_end = min(t_begin + p.tiles_per_cta, p.total_tiles);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kConsumerWarps);
        }
        err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (t_begin >= t_end) return;
    const int tile_elems_shift = 14;  // 16384 elements per tile
    const int gpt = (kTileBytes / 2) / p.group;  // groups per full tile
    int layer = find_layer(p.layers, p.n_layers, t_begin);

    if (warp == kConsumerWarps) {
        // ---------------- producer: one thread streams tiles into the ring ----------------
        if (lane == 0) {
            MtLayer L = p.layers[layer];
            long long next_begin = layer + 1 < p.n_layers ? p.layers[layer + 1].tile_begin : p.total_tiles;
            int it = 0;
            for (long long t = t_begin; t < t_end; ++t, ++it) {
                while (t >= next_begin) {
                    ++layer;
                    L = p.layers[layer];
                    next_begin = layer + 1 < p.n_layers ? p.layers[layer + 1].tile_begin : p.total_tiles;
                }
                const int s = it % kStages;
                const uint32_t ph = (uint32_t)(it / kStages) & 1u;
                if (!mbar_wait(&empty_bar[s], ph ^ 1u, &err)) break;
                const long long g0 = (t - L.tile_begin) * gpt;
                const long long ng = min((long long)gpt, L.n_groups - g0);
                const uint32_t bytes = (uint32_t)(ng * p.group * 2);
                mbar_expect_tx(&full_bar[s], bytes);
                bulk_load(smem_al + (size_t)s * kTileBytes, reinterpret_cast<const unsigned char *>(L.x) + ((size_t)(t - L.tile_begin) << (tile_elems_shift + 1)), bytes, &full_bar[s]);
            }
            if (err) {
                // give copies already issued a bounded chance to land before the CTA's shared memory is released
                for (int s = 0; s < kStages; ++s) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full_bar[s], 0) && !mbar_try_wait(&full_bar[s], 1) && clock64() - t0 < kWaitCycles) {}
                }
                atomicOr(p.timeout, MOFQ_STATUS_TIMEOUT);
            }
        }
        return;
    }

    // ---------------- consumers ----------------
    const int cpg = p.group >> 3;
    MtLayer L = p.layers[layer];
    long long next_begin = layer + 1 < p.n_layers ? p.layers[layer + 1].tile_begin : p.total_tiles;
    double dacc[NA];
#pragma unroll
    for (int j = 0; j < NA; ++j) dacc[j] = 0.0;
    int status = 0;

    auto flush = [&]() {
        // per-warp partial of the finished layer -> its slot; the finalize kernel adds the slots in order
#pragma unroll
        for (int j = 0; j < NA; ++j)
#pragma unroll
            for (int o = 16; o; o >>= 1) dacc[j] += __shfl_xor_sync(0xffffffffu, dacc[j], o);
        if (lane == 0) {
            const long long slot = L.slot_off + (long long)(blockIdx.x - L.first_cta) * kConsumerWarps + warp;
#pragma unroll
            for (int j = 0; j < NA; ++j) p.partials[slot * kMaxAcc + j] = dacc[j];
        }
        if (status) atomicOr(&p.status[layer], status);
#pragma unroll
        for (int j = 0; j < NA; ++j) dacc[j] = 0.0;
        status = 0;
    };

    int it = 0;
    for (long long t = t_begin; t < t_end; ++t, ++it) {
        while (t >= next_begin) {
            flush();
            ++layer;
            L = p.layers[layer];
            next_begin = layer + 1 < p.n_layers ? p.layers[layer + 1].tile_begin : p.total_tiles;
        }
        const int s = it % kStages;
        const uint32_t ph = (uint32_t)(it / kStages) & 1u;
        if (!mbar_wait(&full_bar[s], ph, &err)) break;
        const long long g0 = (t - L.tile_begin) * gpt;
        const int ng = (int)min((long long)gpt, L.n_groups - g0);
        const uint32_t tile = smem_base + (uint32_t)s * kTileBytes;
        for (int g = threadIdx.x; g < ng; g += kConsumers) {
            // chunk j of the group sits at a0 ^ (j << 4): the lane-dependent XOR spreads the lanes of a quarter-warp
            // over all banks, and each address costs one logic instruction
            const uint32_t a0 = tile + (uint32_t)g * (uint32_t)(cpg << 4) + (uint32_t)((g & (cpg - 1)) << 4);
            uint32_t m = 0;
            if (cpg == 16) {  // group of 128: fully unrolled
#pragma unroll
                for (int j = 0; j < 16; ++j) m = absmax_chunk<DT>(lds128(a0 ^ (uint32_t)(j << 4)), m);
            } else {
#pragma unroll 4
                for (int j = 0; j < cpg; ++j) m = absmax_chunk<DT>(lds128(a0 ^ (uint32_t)(j << 4)), m);
            }
            const uint32_t m16 = fold16(m);
            if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
            const float a = mag16_to_float<DT>(m16);
            Sc<NC> sc;
#pragma unroll
            for (int j = 0; j < NC; ++j) {
                // binary16 abs-max values cannot overflow the reciprocal: the short division-free sequence is exact there
                if (DT == MOFQ_F16) scale_pair_fast(a, p.q[j], p.rq[j], sc.s[j], sc.inv[j]);
                else scale_pair(a, p.q[j], sc.s[j], sc.inv[j], status);
            }
            S scorer;
            scorer.begin(sc);
            if (cpg == 16) {
#pragma unroll
                for (int j = 0; j < 16; ++j) scorer.chunk(lds128(a0 ^ (uint32_t)(j << 4)));
            } else {
#pragma unroll 4
                for (int j = 0; j < cpg; ++j) scorer.chunk(lds128(a0 ^ (uint32_t)(j << 4)));
            }
            if (BLK) {
                const long long b = g0 + g;   // the tensor is dense: its groups are the blocks, row-major
                double eg[NC];
#pragma unroll
                for (int j = 0; j < NC; ++j) eg[j] = 0.0;
                scorer.end(eg);
                float e[NC];
#pragma unroll
                for (int j = 0; j < NC; ++j) e[j] = (float)eg[j];
                float best = INFINITY;
                int pick = 0;
                for (int i = 0; i < p.bs.n_cand; ++i) {
                    float ei = e[0];
#pragma unroll
                    for (int j = 1; j < NC; ++j)
                        if (p.bs.perm[i] == j) ei = e[j];
                    if (p.bs.block_sse) p.bs.block_sse[b * p.bs.n_cand + i] = ei;
                    if (ei < best) {                            // strictly smaller: the first candidate keeps a tie
                        best = ei;
                        pick = i;
                    }
                }
                p.bs.choice[b] = (uint8_t)pick;
#pragma unroll
                for (int j = 0; j < NC; ++j) dacc[j] += (double)e[j];
                dacc[NC] += (double)best;
            } else {
                scorer.end(dacc);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
    }
    flush();
}

// ---- finalize: one block per layer ---------------------------------------------------------------------
__global__ void __launch_bounds__(128)
kq_mt_finalize(const MtLayer *layers, const double *partials, int32_t *status, const int32_t *timeout, Finalize fin,
               mofq_result *results)
{
    __shared__ double red[4][kMaxAcc];
    const MtLayer L = layers[blockIdx.x];
    double tot[kMaxAcc];
#pragma unroll
    for (int j = 0; j < kMaxAcc; ++j) tot[j] = 0.0;
    for (int slot = threadIdx.x; slot < L.n_slots; slot += blockDim.x)
        for (int j = 0; j < fin.nc; ++j) tot[j] += partials[(size_t)(L.slot_off + slot) * kMaxAcc + j];
    for (int j = 0; j < fin.nc; ++j)
#pragma unroll
        for (int o = 16; o; o >>= 1) tot[j] += __shfl_xor_sync(0xffffffffu, tot[j], o);
    if ((threadIdx.x & 31) == 0)
        for (int j = 0; j < fin.nc; ++j) red[threadIdx.x >> 5][j] = tot[j];
    __syncthreads();
    if (threadIdx.x != 0) return;
    double err[MOFQ_MAX_CAND];
    double best = INFINITY, second = INFINITY;
    int chosen = -1;
    for (int i = 0; i < fin.n_cand; ++i) {
        const int j = fin.perm[i];
        err[i] = (red[0][j] + red[1][j] + red[2][j] + red[3][j]) * L.inv_n;
        // Algorithm 1: replace only on a strictly smaller error, in the caller's candidate order
        if (err[i] < best) {
            second = best;
            best = err[i];
            chosen = i;
        } else if (err[i] < second) {
            second = err[i];
        }
    }
    mofq_result r;
    r.chosen = chosen;
    r.status = status[blockIdx.x] | *timeout;
    for (int i = 0; i < MOFQ_MAX_CAND; ++i) {
        r.error[i] = i < fin.n_cand ? (float)err[i] : 0.0f;
        r.nsr[i] = 0.0f;
    }
    r.rel_margin = best > 0.0 ? (float)((second - best) / best) : INFINITY;
    r.reserved = 0;
    if (results) results[blockIdx.x] = r;
    if (fin.mse_out)
        for (int i = 0; i < fin.n_cand; ++i) fin.mse_out[(size_t)blockIdx.x * fin.n_cand + i] = r.error[i];
    if (fin.status_out && r.status) atomicOr(fin.status_out, r.status);
}

// The work table travels to the device as kernel arguments, 512 entries per launch: fully stream-ordered,
// no pageable-memory copy (which would synchronise the stream) and nothing for the caller to keep alive.
constexpr int kUploadChunk = 512;   // 24 KB of the 32 KB a launch's parameters may take
static_assert(sizeof(MtLayer) * kUploadChunk + 64 <= 32764, "the chunk must fit a launch's parameter space");
struct TableChunk {
    MtLayer e[kUploadChunk];
};
__global__ void kq_mt_upload(const TableChunk chunk, MtLayer *dst, int n)
{
    if ((int)threadIdx.x < n) dst[threadIdx.x] = chunk.e[threadIdx.x];
}

int fp_kind(int format)
{
    switch (format) {
    case MOFQ_FP4_E2M1:
    case MOFQ_FP4_E2M1_IEEE: return FPK_E2M1;
    case MOFQ_FP8_E4M3: return FPK_E4M3;
    case MOFQ_FP8_E5M2: return FPK_E5M2;
    }
    return -1;
}

template <int DT, int NI, int K0, int K1, bool BLK = false>
int launch(const MtParams &p, int grid, cudaStream_t st)
{
    auto kernel = kq_score_mt<DT, NI, K0, K1, BLK>;
    const size_t smem = (size_t)kStages * kTileBytes + 1024;   // + slack to align the tiles
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    kernel<<<grid, kThreads, smem, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return MOFQ_ERR_CUDA;
    return MOFQ_OK;
}

template <int DT>
int dispatch(int ni, int k0, int k1, const MtParams &p, int grid, cudaStream_t st)
{
#define MOFQ_MT(NI_, K0_, K1_) \
    if (ni == NI_ && k0 == K0_ && k1 == K1_) return launch<DT, NI_, K0_, K1_>(p, grid, st);
    MOFQ_MT(1, -1, -1) MOFQ_MT(0, FPK_E2M1, -1) MOFQ_MT(1, FPK_E2M1, -1) MOFQ_MT(0, FPK_E2M1, FPK_E2M1) MOFQ_MT(1, FPK_E2M1, FPK_E2M1)
    MOFQ_MT(0, FPK_E4M3, -1) MOFQ_MT(1, FPK_E4M3, -1) MOFQ_MT(0, FPK_E5M2, -1) MOFQ_MT(1, FPK_E5M2, -1)
    MOFQ_MT(0, FPK_E4M3, FPK_E5M2) MOFQ_MT(1, FPK_E4M3, FPK_E5M2) MOFQ_MT(0, FPK_E5M2, FPK_E4M3) MOFQ_MT(1, FPK_E5M2, FPK_E4M3)
#undef MOFQ_MT
    return MOFQ_ERR_UNSUPPORTED;
}

// The block-wise form exists for INT4 against FP4-E2M1.  (The 8-bit formats stay with the register-resident kernel and
// its unscaled errors: this kernel forms a group's error in units of the scale, d = r - x * inv, and inv * scale differs
// from 1 by up to 2^-23; against an 8-bit grid's |x * inv| <= 127 and |d| <= 0.5 that is a few 1e-5 of one group's
// sum - invisible in a tensor's mean, too much for a single block's reported error.)
template <int DT>
int dispatch_blocks(int ni, int k0, int k1, const MtParams *p, int grid, cudaStream_t st)
{
#define MOFQ_MTB(K0_, K1_) \
    if (ni == 1 && k0 == K0_ && k1 == K1_) return p ? launch<DT, 1, K0_, K1_, true>(*p, grid, st) : MOFQ_OK;
    MOFQ_MTB(FPK_E2M1, -1)
#undef MOFQ_MTB
    return MOFQ_ERR_UNSUPPORTED;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }
int mt_grid() { return sm_count() * kCtasPerSm; }

}  // namespace

// The multi-tensor path applies to the tensor metric with one per-group granularity on dense tensors of one dtype.
bool mt_applicable(const mofq_layer *layers, int n_layers, const mofq_config *cfg)
{
    if (cfg->metric != MOFQ_TENSOR_MSE || cfg->w_gran != MOFQ_PER_GROUP || cfg->w_gran2 != MOFQ_GRAN_NONE) return false;
    if (cfg->w_group < 8 || cfg->w_group > 256) return false;
    for (int i = 0; i < n_layers; ++i)
        if (layers[i].W.ld != layers[i].W.cols || layers[i].W.dtype != layers[0].W.dtype) return false;
    return true;
}

bool mt_blocks_applicable(const mofq_tensor &W, int group, const CandSet &cs, const int *fp_formats)
{
    if (group != 128 || W.ld != W.cols || W.rows * W.cols < (8LL << 20)) return false;   // small tensors: the register kernel, one launch
    const int k0 = cs.n_fp > 0 ? fp_kind(fp_formats[0]) : -1, k1 = cs.n_fp > 1 ? fp_kind(fp_formats[1]) : -1;
    return dispatch_blocks<MOFQ_F16>(cs.n_int, k0, k1, nullptr, 0, nullptr) == MOFQ_OK;
}

size_t mt_ws_bytes(int n_layers)
{
    const size_t slots = ((size_t)mt_grid() + (size_t)n_layers) * kConsumerWarps;
    return align256(sizeof(MtLayer) * (size_t)n_layers) + align256(slots * kMaxAcc * sizeof(double)) +
           align256(sizeof(int32_t) * ((size_t)n_layers + 1));
}

int mt_run(const mofq_layer *layers, int n_layers, const mofq_config *cfg, const CandSet &cs, const int *perm, int nc,
           const int *fp_formats, mofq_result *results, void *ws, cudaStream_t st, float *mse_out, int32_t *status_out,
           const BlockSel *bs)
{
    if (bs && (n_layers != 1 || !mt_blocks_applicable(layers[0].W, cfg->w_group, cs, fp_formats))) return MOFQ_ERR_UNSUPPORTED;
    const int grid = mt_grid();
    const int gpt = (kTileBytes / 2) / cfg->w_group;
    std::vector<MtLayer> table((size_t)n_layers);
    long long tiles = 0;
    for (int i = 0; i < n_layers; ++i) {
        const mofq_tensor &W = layers[i].W;
        MtLayer &L = table[(size_t)i];
        L.x = static_cast<const uint16_t *>(W.data);
        L.n_groups = W.rows * W.cols / cfg->w_group;
        L.tile_begin = tiles;
        L.inv_n = 1.0 / ((double)W.rows * (double)W.cols);
        tiles += (L.n_groups + gpt - 1) / gpt;
    }
    const long long tpc = (tiles + grid - 1) / grid;
    long long slot = 0;
    for (int i = 0; i < n_layers; ++i) {
        MtLayer &L = table[(size_t)i];
        const long long end = (i + 1 < n_layers ? table[(size_t)i + 1].tile_begin : tiles) - 1;
        L.first_cta = (int)(L.tile_begin / tpc);
        L.n_slots = (int)(end / tpc - L.first_cta + 1) * kConsumerWarps;
        L.slot_off = (int)slot;
        slot += L.n_slots;
    }
    char *base = static_cast<char *>(ws);
    MtLayer *d_table = reinterpret_cast<MtLayer *>(base);
    double *d_partials = reinterpret_cast<double *>(base + align256(sizeof(MtLayer) * (size_t)n_layers));
    int32_t *d_status = reinterpret_cast<int32_t *>(reinterpret_cast<char *>(d_partials) +
                                                    align256(((size_t)grid + (size_t)n_layers) * kConsumerWarps * kMaxAcc * sizeof(double)));
    for (int i = 0; i < n_layers; i += kUploadChunk) {
        TableChunk chunk;
        const int n = std::min(kUploadChunk, n_layers - i);
        for (int k = 0; k < n; ++k) chunk.e[k] = table[(size_t)(i + k)];
        kq_mt_upload<<<1, kUploadChunk, 0, st>>>(chunk, d_table + i, n);
        if (cudaGetLastError() != cudaSuccess) return MOFQ_ERR_CUDA;
    }
    if (cudaMemsetAsync(d_status, 0, sizeof(int32_t) * ((size_t)n_layers + 1), st) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    MtParams p{};
    p.layers = d_table;
    p.n_layers = n_layers;
    p.total_tiles = tiles;
    p.tiles_per_cta = tpc;
    p.group = cfg->w_group;
    if (cs.n_int) p.q[0] = cs.int_q;
    for (int f = 0; f < cs.n_fp; ++f) p.q[cs.n_int + f] = cs.fp_q[f];
    for (int j = 0; j < 3; ++j) p.rq[j] = p.q[j] > 0.0f ? 1.0f / p.q[j] : 0.0f;
    p.partials = d_partials;
    p.status = d_status;
    p.timeout = d_status + n_layers;
    const int k0 = cs.n_fp > 0 ? fp_kind(fp_formats[0]) : -1, k1 = cs.n_fp > 1 ? fp_kind(fp_formats[1]) : -1;
    const int used = (int)std::min<long long>(grid, (tiles + tpc - 1) / tpc);
    int rc;
    if (bs) {
        p.bs = *bs;
        rc = layers[0].W.dtype == MOFQ_F16 ? dispatch_blocks<MOFQ_F16>(cs.n_int, k0, k1, &p, used, st)
                                           : dispatch_blocks<MOFQ_BF16>(cs.n_int, k0, k1, &p, used, st);
    } else {
        rc = layers[0].W.dtype == MOFQ_F16 ? dispatch<MOFQ_F16>(cs.n_int, k0, k1, p, used, st)
                                           : dispatch<MOFQ_BF16>(cs.n_int, k0, k1, p, used, st);
    }
    if (rc) return rc;
    Finalize fin{};
    fin.n_cand = cfg->n_candidates;
    fin.n_sets = 1;
    fin.nc = nc;
    fin.mse_out = mse_out;
    fin.status_out = status_out;
    for (int i = 0; i < MOFQ_MAX_CAND; ++i) fin.perm[i] = perm[i];
    if (bs) {   // the candidates in the caller's order, then the mixture (accumulator nc)
        if (fin.n_cand + 1 > MOFQ_MAX_CAND) return MOFQ_ERR_UNSUPPORTED;
        fin.perm[fin.n_cand] = fin.nc;
        fin.n_cand += 1;
        fin.nc += 1;
    }
    kq_mt_finalize<<<n_layers, 128, 0, st>>>(d_table, d_partials, d_status, d_status + n_layers, fin, results);
    if (cudaGetLastError() != cudaSuccess) return MOFQ_ERR_CUDA;
    return MOFQ_OK;
}

}  // namespace mofq
