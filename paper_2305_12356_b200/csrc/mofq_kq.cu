// Quantise / score kernels: abs-max scale -> round to the INT-k and FP-k grids -> dequantise ->
// squared error -> block reduce, for all candidates from one read of the tensor.
//
// The arithmetic follows the contract in mofq.h: scale = RN32(a/Q), inv = RN32(Q/a),
// t = RN32(x*inv), INT: RNE(t); FP: RNE of |t| onto the spacing 2^(e-M) of its binade, e clamped
// at the smallest normal exponent (gradual underflow).  Both roundings use the add-and-subtract
// of a power of two whose ulp equals the wanted spacing, which is an exact RNE in binary32.
// Every grid is symmetric, (x - v*s)^2 = (|x| - |v|*s)^2: the scalar kernels score magnitudes, the packed ones
// (kq_math.cuh) keep the signs through sign-symmetric roundings; signs matter only when codes are written out.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>
#include <type_traits>

#include "kq_finish.cuh"
#include "kq_math.cuh"
#include "kq_pipe.cuh"
#include "mofq_internal.h"

namespace mofq {
namespace {

using kqfin::write_outputs;

constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds |t| < 2^22 to an integer (RNE)

// ---- small device helpers --------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ void unpack2(uint32_t w, float &lo, float &hi)
{
    if (DT == MOFQ_F16) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w));
        lo = f.x;
        hi = f.y;
    } else {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xFFFF0000u);
    }
}

using kqmath::fold16;
using kqmath::mag16_nonfinite;
using kqmath::mag16_to_float;
using kqmath::scale_pair;

// running abs-max over packed 16-bit magnitude patterns (integer order == magnitude order; Inf/NaN sort on top)
__device__ __forceinline__ uint32_t absmax_chunk(const uint4 v, uint32_t m)
{
    m = __vmaxu2(m, v.x & 0x7FFF7FFFu);
    m = __vmaxu2(m, v.y & 0x7FFF7FFFu);
    m = __vmaxu2(m, v.z & 0x7FFF7FFFu);
    m = __vmaxu2(m, v.w & 0x7FFF7FFFu);
    return m;
}

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

// |t| -> nearest FP grid magnitude (RNE), no saturation (|t| <= Q(1+2^-23) under abs-max scales)
__device__ __forceinline__ float fp_grid_round(float t, uint32_t eminb, uint32_t kadd)
{
    const uint32_t eb = max(__float_as_uint(t) & 0x7F800000u, eminb);
    const float c = __uint_as_float(eb + kadd);
    return __fsub_rn(__fadd_rn(t, c), c);
}


// ---- block reductions and the last-block-done finish -------------------------------------------------
__device__ __forceinline__ uint32_t block_max_u32(uint32_t v, uint32_t *red /* >= 33 words */)
{
#pragma unroll
    for (int o = 16; o; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    if (warp == 0) {
        uint32_t r = lane < nw ? red[lane] : 0u;
#pragma unroll
        for (int o = 16; o; o >>= 1) r = max(r, __shfl_xor_sync(0xffffffffu, r, o));
        if (lane == 0) red[32] = r;
    }
    __syncthreads();
    return red[32];
}

// Sum NA doubles per thread over the block in a fixed order; the totals land in red[0..NA).
template <int NA>
__device__ __forceinline__ void block_sum(double *acc, double *red /* >= 32*NA + NA doubles */)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
#pragma unroll
    for (int j = 0; j < NA; ++j)
#pragma unroll
        for (int o = 16; o; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
    __syncthreads();
    if (lane == 0)
        for (int j = 0; j < NA; ++j) red[NA + warp * NA + j] = acc[j];
    __syncthreads();
    if (threadIdx.x < NA) {
        double s = 0.0;
        for (int w = 0; w < nw; ++w) s += red[NA + w * NA + threadIdx.x];
        red[threadIdx.x] = s;
    }
    __syncthreads();
}

// Every block deposits its partial sums; the block that arrives last adds them in slot order.
template <int NA>
__device__ void block_finish(double *acc, int status, WsHeader *hdr, double *partials, const Finalize &fin, double *red)
{
    __shared__ int is_last;
    if (status) atomicOr(&hdr->status, status);
    block_sum<NA>(acc, red);
    if (threadIdx.x == 0) {
        for (int j = 0; j < NA; ++j) partials[(size_t)blockIdx.x * kMaxAcc + j] = red[j];
        __threadfence();
        const uint32_t ticket = atomicAdd(&hdr->counter, 1u);
        is_last = (ticket == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double tot[NA];
#pragma unroll
    for (int j = 0; j < NA; ++j) tot[j] = 0.0;
    for (int slot = threadIdx.x; slot < (int)gridDim.x; slot += blockDim.x)
#pragma unroll
        for (int j = 0; j < NA; ++j) tot[j] += __ldcg(&partials[(size_t)slot * kMaxAcc + j]);
    block_sum<NA>(tot, red);
    if (threadIdx.x == 0) {
        hdr->counter = 0;
        write_outputs(red, fin, hdr);
    }
}

// ---- scoring kernel 2: one row per block; per-channel and/or per-group scales ---------------------------
// The row is staged in shared memory so that the abs-max pass and the scoring pass cost one HBM read.
// Work is chunk-strided (a chunk = 8 elements = 16 bytes), so every thread stays busy whatever the row
// length: pass 1 leaves one abs-max per chunk; the first `groups per row` threads fold 16-byte chunk maxima
// into group maxima and derive the group scales; a block reduction gives the row scale; pass 2 scores each
// chunk against its group's scales and/or the row's scales from the same registers.
// Arithmetic: packed f32x2 and hardware FP converts (kq_math.cuh).  Accumulator order: [first set][second
// set]; `grp_first` says whether the group set comes first.
constexpr int kRowThreads = 256;

template <int DT, int NI, int K0, int K1, bool CH, bool GRP>
__global__ void __launch_bounds__(kRowThreads)
kq_score_rows(const uint16_t *__restrict__ x, long long rows, int cols, long long ld, int group, int grp_first, RowQ rq,
              WsHeader *hdr, double *partials, Finalize fin)
{
    using S = kqmath::Scorer<DT, NI, K0, K1>;
    constexpr int NC = S::NC;
    constexpr int NA = NC * ((CH ? 1 : 0) + (GRP ? 1 : 0));
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ double red[33 * NA];
    __shared__ uint32_t mred[34];
    __shared__ kqmath::Sc<NC> row_sc;
    __shared__ int row_status;
    const int chunks = cols >> 3;
    const int cpg_shift = GRP ? 31 - __clz(group >> 3) : 0;  // chunks per group is a power of two
    const int gpr = GRP ? cols / group : 0;
    const uint4 *row4 = reinterpret_cast<const uint4 *>(smem);
    uint16_t *cmax = reinterpret_cast<uint16_t *>(smem + (size_t)cols * 2);                               // per-chunk abs-max
    kqmath::Sc<NC> *gsc = reinterpret_cast<kqmath::Sc<NC> *>(smem + (size_t)cols * 2 + (((size_t)chunks * 2 + 15) & ~(size_t)15));
    double dacc[NA];
#pragma unroll
    for (int j = 0; j < NA; ++j) dacc[j] = 0.0;
    int status = 0;

    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const unsigned char *src = reinterpret_cast<const unsigned char *>(x + row * ld);
        for (int q = threadIdx.x; q < chunks; q += kRowThreads) cp_async16(smem + q * 16, src + (size_t)q * 16);
        cp_async_wait_all();
        __syncthreads();
        // pass 1: abs-max per chunk
        uint32_t m16 = 0;
        for (int q = threadIdx.x; q < chunks; q += kRowThreads) {
            const uint32_t c16 = fold16(kqmath::absmax_chunk<DT>(row4[q], 0u));
            if (GRP) cmax[q] = (uint16_t)c16;
            m16 = max(m16, c16);
        }
        if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
        if (GRP) {
            __syncthreads();
            for (int g = threadIdx.x; g < gpr; g += kRowThreads) {
                uint32_t gm = 0;
                for (int j = 0; j < (1 << cpg_shift); ++j) gm = max(gm, (uint32_t)cmax[(g << cpg_shift) + j]);
                const float a = mag16_to_float<DT>(gm);
                kqmath::Sc<NC> sc;
#pragma unroll
                for (int j = 0; j < NC; ++j) scale_pair(a, rq.q[j], sc.s[j], sc.inv[j], status);
                gsc[g] = sc;
            }
        }
        if (CH) {
            const uint32_t rm = block_max_u32(m16, mred);
            if (threadIdx.x == 0) {
                int st = 0;
                kqmath::Sc<NC> sc;
#pragma unroll
                for (int j = 0; j < NC; ++j) scale_pair(mag16_to_float<DT>(rm), rq.q[j], sc.s[j], sc.inv[j], st);
                row_sc = sc;
                row_status = st;
            }
            __syncthreads();
            status |= row_status;
        } else {
            __syncthreads();
        }
        // pass 2: score
        S sg;                                            // group scales change from chunk to chunk: unscaled accumulation
        kqmath::Scorer<DT, NI, K0, K1, true> sc;         // the row's scales are fixed: scaled accumulation
        sg.clear();
        sc.clear();
        if (CH) sc.set_scales(row_sc);
        for (int q = threadIdx.x; q < chunks; q += kRowThreads) {
            const uint4 v = row4[q];
            if (GRP) {
                sg.set_scales(gsc[q >> cpg_shift]);
                sg.chunk(v);
            }
            if (CH) sc.chunk(v);
        }
        double a_g[NC], a_c[NC];
#pragma unroll
        for (int j = 0; j < NC; ++j) a_g[j] = a_c[j] = 0.0;
        if (GRP) sg.end(a_g);
        if (CH) sc.end(a_c);
        if (CH && GRP) {
#pragma unroll
            for (int j = 0; j < NC; ++j) {
                dacc[j] += grp_first ? a_g[j] : a_c[j];
                dacc[NC + j] += grp_first ? a_c[j] : a_g[j];
            }
        } else {
#pragma unroll
            for (int j = 0; j < NC; ++j) dacc[j] += GRP ? a_g[j] : a_c[j];
        }
        __syncthreads();
    }
    block_finish<NA>(dacc, status, hdr, partials, fin, red);
}

// ---- block-wise selection: one winner per scale block (row or group) ---------------------------------------
// A team of T lanes (a quarter of the block's chunks when that is a power of two <= 32, else a whole warp) owns one
// block at a time, up to four chunks per lane held in registers: abs-max by shuffles, scales, then every candidate's squared error from the same registers; lane 0
// of the team applies Algorithm 1's rule (strictly smaller, caller's order) to the block's errors.  Accumulators:
// [canonical slots][mixture].
template <int DT, int NI, int K0, int K1>
__global__ void __launch_bounds__(256)
kq_select_blocks(const uint16_t *__restrict__ x, long long rows, int cols, long long ld, int width, int team, RowQ rq,
                 BlockSel bs, WsHeader *hdr, double *partials, Finalize fin)
{
    // unscaled accumulation: a block can be as small as 8 elements, where the scaled form's rounding of x * inv
    // (relative to x, not to the error) would show in the block's own sum
    using S = kqmath::Scorer<DT, NI, K0, K1, false>;
    constexpr int NC = S::NC;
    constexpr int NA = NC + 1;
    __shared__ double red[33 * NA];
    const int lane = threadIdx.x & 31;
    const int tl = lane & (team - 1);                       // lane within the team
    const int teams_per_warp = 32 / team;
    const int cpb = width >> 3;                             // 16-byte chunks per block
    const int per_row = cols / width;
    const long long n_blocks = rows * per_row;
    const long long warp_id = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * (blockDim.x >> 5);
    constexpr int KPL = 4;                                  // chunks a lane can keep in registers
    const bool one_pass = cpb <= KPL * team;                // the block is read once; else twice (second read from cache)
    double dacc[NA];
#pragma unroll
    for (int j = 0; j < NA; ++j) dacc[j] = 0.0;
    int status = 0;

    for (long long b0 = warp_id * teams_per_warp; b0 < n_blocks; b0 += n_warps * teams_per_warp) {
        const long long b = b0 + lane / team;
        const bool live = b < n_blocks;                     // whole teams are live or not; shuffles stay warp-wide
        const long long r = live ? b / per_row : 0;
        const uint4 *blk = reinterpret_cast<const uint4 *>(x + r * ld + (live ? (b - r * per_row) * width : 0));
        uint4 v[KPL];
        uint32_t m = 0;
        if (one_pass) {
#pragma unroll
            for (int k = 0; k < KPL; ++k) {
                const int q = tl + k * team;
                v[k] = (live && q < cpb) ? __ldg(blk + q) : make_uint4(0, 0, 0, 0);
                m = kqmath::absmax_chunk<DT>(v[k], m);
            }
        } else if (live) {
            for (int q = tl; q < cpb; q += team) m = kqmath::absmax_chunk<DT>(__ldg(blk + q), m);
        }
        uint32_t m16 = fold16(m);
        for (int o = team >> 1; o; o >>= 1) m16 = max(m16, __shfl_xor_sync(0xffffffffu, m16, o));
        if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
        const float a = mag16_to_float<DT>(m16);
        kqmath::Sc<NC> sc;
#pragma unroll
        for (int j = 0; j < NC; ++j) {
            // binary16 abs-max values cannot overflow the reciprocal: the short division-free sequence is exact there
            if (DT == MOFQ_F16) kqmath::scale_pair_fast(a, rq.q[j], rq.rq[j], sc.s[j], sc.inv[j]);
            else scale_pair(a, rq.q[j], sc.s[j], sc.inv[j], status);
        }
        S scorer;
        scorer.begin(sc);
        if (one_pass) {
#pragma unroll
            for (int k = 0; k < KPL; ++k) scorer.chunk(v[k]);   // zeros (idle slots) add nothing
        } else if (live) {
            for (int q = tl; q < cpb; q += team) scorer.chunk(__ldg(blk + q));
        }
        float e[NC];
#pragma unroll
        for (int j = 0; j < NC; ++j) {
            float lo, hi;
            kqmath::upk(scorer.acc2[j], lo, hi);
            e[j] = lo + hi;
            for (int o = team >> 1; o; o >>= 1) e[j] += __shfl_xor_sync(0xffffffffu, e[j], o);
        }
        if (live && tl == 0) {
            float best = INFINITY;
            int pick = 0;
            for (int i = 0; i < bs.n_cand; ++i) {
                float ei = e[0];
#pragma unroll
                for (int j = 1; j < NC; ++j)
                    if (bs.perm[i] == j) ei = e[j];
                if (bs.block_sse) bs.block_sse[b * bs.n_cand + i] = ei;
                if (ei < best) {                            // strictly smaller: the first candidate keeps a tie
                    best = ei;
                    pick = i;
                }
            }
            if (bs.choice) bs.choice[b] = (uint8_t)pick;
#pragma unroll
            for (int j = 0; j < NC; ++j) dacc[j] += (double)e[j];
            dacc[NC] += (double)best;
        }
    }
    block_finish<NA>(dacc, status, hdr, partials, fin, red);
}

// ---- per-tensor scale: abs-max kernel, then a streaming scoring kernel -----------------------------------
template <int DT>
__global__ void __launch_bounds__(256)
kq_absmax(const uint16_t *__restrict__ x, long long rows, int chunks_per_row, long long ld, WsHeader *hdr)
{
    chain_enter();
    uint32_t m = 0;
    const long long total = rows * chunks_per_row;
    const long long stride = (long long)gridDim.x * blockDim.x;
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (rows == 1) {  // dense: no row arithmetic, four independent loads in flight per thread
        const uint4 *p = reinterpret_cast<const uint4 *>(x);
        for (; i + 3 * stride < total; i += 4 * stride) {
            const uint4 v0 = __ldg(p + i), v1 = __ldg(p + i + stride), v2 = __ldg(p + i + 2 * stride), v3 = __ldg(p + i + 3 * stride);
            m = absmax_chunk(v0, m);
            m = absmax_chunk(v1, m);
            m = absmax_chunk(v2, m);
            m = absmax_chunk(v3, m);
        }
    }
    for (; i < total; i += stride) {
        const long long r = i / chunks_per_row;
        const int c = (int)(i - r * chunks_per_row);
        m = absmax_chunk(__ldg(reinterpret_cast<const uint4 *>(x + r * ld) + c), m);
    }
    __shared__ uint32_t mred[34];
    const uint32_t m16 = block_max_u32(fold16(m), mred);   // one atomic per block: they all go to one address
    if (threadIdx.x == 0 && m16) atomicMax(&hdr->absmax_bits, m16);
}

// The scale pairs are the same for every element, so the packed scorer runs in its scaled form; its binary32 chains
// are folded into double every 16 chunks (128 terms).
template <int DT, int NI, int K0, int K1>
__global__ void __launch_bounds__(256)
kq_score_uniform(const uint16_t *__restrict__ x, long long rows, int chunks_per_row, long long ld, RowQ rq,
                 WsHeader *hdr, double *partials, Finalize fin)
{
    using S = kqmath::Scorer<DT, NI, K0, K1, true>;
    constexpr int NC = S::NC;
    __shared__ double red[33 * NC];
    int status = 0;
    const uint32_t m16 = *reinterpret_cast<volatile uint32_t *>(&hdr->absmax_bits);
    if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
    kqmath::Sc<NC> sc;
#pragma unroll
    for (int j = 0; j < NC; ++j) scale_pair(mag16_to_float<DT>(m16), rq.q[j], sc.s[j], sc.inv[j], status);
    S scorer;
    scorer.begin(sc);
    double dacc[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) dacc[j] = 0.0;
    const long long total = rows * chunks_per_row;
    const long long stride = (long long)gridDim.x * blockDim.x;
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    int n = 0;
    if (rows == 1) {  // dense: no row arithmetic, the next pair of chunks is loaded while this pair is scored
        const uint4 *p = reinterpret_cast<const uint4 *>(x);
        for (; i + stride < total; i += 2 * stride) {
            const uint4 v0 = __ldg(p + i), v1 = __ldg(p + i + stride);
            scorer.chunk(v0);
            scorer.chunk(v1);
            if ((n += 2) >= 16) {
                scorer.end(dacc);
                scorer.clear();
                n = 0;
            }
        }
    }
    for (; i < total; i += stride) {
        const long long r = i / chunks_per_row;
        const int c = (int)(i - r * chunks_per_row);
        scorer.chunk(__ldg(reinterpret_cast<const uint4 *>(x + r * ld) + c));
        if (++n >= 16) {
            scorer.end(dacc);
            scorer.clear();
            n = 0;
        }
    }
    scorer.end(dacc);
    block_finish<NC>(dacc, status, hdr, partials, fin, red);
}

// ---- caller-supplied per-tensor scales (calibration, Section 3.2 dynamic tensor analysis): saturating scorer -------
// scales[i] belongs to the caller's candidate i; inv = RN32(1/scale); out-of-range values clip to the grid ends.
template <int DT, int NI, int NFP>
__global__ void __launch_bounds__(256)
kq_score_supplied(const uint16_t *__restrict__ x, long long rows, int chunks_per_row, long long ld, CandSet cs,
                  const float *__restrict__ scales, WsHeader *hdr, double *partials, Finalize fin)
{
    constexpr int NC = NI + NFP;
    __shared__ double red[33 * NC];
    float s[NC], inv[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        s[j] = 1.0f;
        for (int i = fin.n_cand - 1; i >= 0; --i)
            if (fin.perm[i] == j) s[j] = scales[i];
        inv[j] = __fdiv_rn(1.0f, s[j]);
    }
    double dacc[NC];
    float acc[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        dacc[j] = 0.0;
        acc[j] = 0.0f;
    }
    int status = 0, n = 0;
    const long long total = rows * chunks_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / chunks_per_row;
        const int c = (int)(i - r * chunks_per_row);
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(x + r * ld) + c);
        if (mag16_nonfinite<DT>(fold16(absmax_chunk(v, 0)))) status |= MOFQ_STATUS_NONFINITE_INPUT;
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float xv[2];
            unpack2<DT>(w[k], xv[0], xv[1]);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (NI) {
                    const float t = fminf(fmaxf(__fmul_rn(xv[h], inv[0]), -1024.0f), 1024.0f);
                    float q = __fsub_rn(__fadd_rn(t, kMagic), kMagic);
                    q = fminf(fmaxf(q, -cs.int_q - 1.0f), cs.int_q);
                    const float e = __fmaf_rn(-q, s[0], xv[h]);
                    acc[0] = __fmaf_rn(e, e, acc[0]);
                }
#pragma unroll
                for (int f = 0; f < NFP; ++f) {
                    const float a = fabsf(xv[h]);
                    const float t = fminf(__fmul_rn(a, inv[NI + f]), 2.0f * cs.fp_q[f]);
                    const float q = fminf(fp_grid_round(t, cs.fp_eminb[f], cs.fp_kadd[f]), cs.fp_q[f]);
                    const float e = __fmaf_rn(-q, s[NI + f], a);
                    acc[NI + f] = __fmaf_rn(e, e, acc[NI + f]);
                }
            }
        }
        if (++n == 16) {
#pragma unroll
            for (int j = 0; j < NC; ++j) {
                dacc[j] += (double)acc[j];
                acc[j] = 0.0f;
            }
            n = 0;
        }
    }
#pragma unroll
    for (int j = 0; j < NC; ++j) dacc[j] += (double)acc[j];
    block_finish<NC>(dacc, status, hdr, partials, fin, red);
}

// running abs-max over calibration batches: *absmax_inout = max(*absmax_inout, max |x|) (non-negative floats order like uints)
template <int DT>
__global__ void __launch_bounds__(256)
kq_absmax_update(const uint16_t *__restrict__ x, long long rows, int chunks_per_row, long long ld, float *absmax_inout)
{
    uint32_t m = 0;
    const long long total = rows * chunks_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / chunks_per_row;
        const int c = (int)(i - r * chunks_per_row);
        m = absmax_chunk(__ldg(reinterpret_cast<const uint4 *>(x + r * ld) + c), m);
    }
    uint32_t m16 = fold16(m);
#pragma unroll
    for (int o = 16; o; o >>= 1) m16 = max(m16, __shfl_xor_sync(0xffffffffu, m16, o));
    if ((threadIdx.x & 31) == 0 && m16)
        atomicMax(reinterpret_cast<uint32_t *>(absmax_inout), __float_as_uint(mag16_to_float<DT>(m16)));
}

// ---- emit kernel: codes / scales / dequantised values for ONE format ---------------------------------------
// One row per block.  GRAN selects where the scale of a 16-byte chunk comes from.
__device__ __forceinline__ uint32_t fp_code_from_mag(float r, const FmtDesc &f)
{
    // below the smallest normal, adding it puts the subnormal step count into the mantissa field
    uint32_t rb = (r < f.min_normal) ? __float_as_uint(__fadd_rn(r, f.min_normal)) - (1u << 23) : __float_as_uint(r);
    return (rb >> (23 - f.M)) - ((uint32_t)(127 - f.bias) << f.M);
}

template <int DT>
__device__ __forceinline__ uint16_t to_storage(float v)
{
    if (DT == MOFQ_F16) return __half_as_ushort(__float2half_rn(v));
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
}

template <int DT, int GRAN>
__global__ void __launch_bounds__(kRowThreads)
kq_emit(const uint16_t *__restrict__ x, long long rows, int cols, long long ld, FmtDesc f, int group,
        const float *__restrict__ scales_in, unsigned char *codes_out, float *scales_out, uint16_t *dequant_out,
        uint16_t *values_out, int values_dtype, WsHeader *hdr, const EmitSel sel)
{
    __shared__ uint32_t mred[34];
    // When the host launched this kernel as the next layer of one emission call, the launch after it may start as
    // soon as every block of this one is running: the layers read and write disjoint buffers.  The wait at the end
    // keeps the launches completing in stream order.
    asm volatile("griddepcontrol.launch_dependents;");
    if (sel.res) {  // the winner of the selection record decides the grid
        const int c = min(max(sel.res->chosen, 0), MOFQ_MAX_CAND - 1);
        f = sel.cand[c];
        if (sel.tag_out && blockIdx.x == 0 && threadIdx.x == 0) *sel.tag_out = sel.format[c];
    }
    const int chunks = cols >> 3;
    const int lanes_per_group = GRAN == MOFQ_PER_GROUP ? (group >> 3) : 1;  // power of two <= 32
    const int gpr = GRAN == MOFQ_PER_GROUP ? cols / group : 1;
    int status = 0;
    const float int_lo = -f.Q - 1.0f;

    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4 *xr = reinterpret_cast<const uint4 *>(x + row * ld);
        float s = 1.0f, inv = 1.0f;
        if (GRAN == MOFQ_PER_TENSOR || GRAN == MOFQ_PER_CHANNEL) {
            if (scales_in) {
                s = scales_in[GRAN == MOFQ_PER_TENSOR ? 0 : row];
                inv = __fdiv_rn(1.0f, s);
            } else {
                uint32_t m16;
                if (GRAN == MOFQ_PER_TENSOR) {
                    m16 = *reinterpret_cast<volatile uint32_t *>(&hdr->absmax_bits);
                } else {
                    uint32_t m = 0;
                    for (int q = threadIdx.x; q < chunks; q += kRowThreads) m = absmax_chunk(__ldg(xr + q), m);
                    m16 = block_max_u32(fold16(m), mred);
                }
                if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
                scale_pair(mag16_to_float<DT>(m16), f.Q, s, inv, status);
            }
            if (scales_out && threadIdx.x == 0 && (GRAN == MOFQ_PER_CHANNEL || row == 0))
                scales_out[GRAN == MOFQ_PER_TENSOR ? 0 : row] = s;
        }
        const int iters = (chunks + kRowThreads - 1) / kRowThreads;
        for (int it = 0; it < iters; ++it) {
            const int q = it * kRowThreads + threadIdx.x;
            const bool active = q < chunks;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (active) v = __ldg(xr + q);
            if (GRAN == MOFQ_PER_GROUP) {
                const int g = q / lanes_per_group;
                if (scales_in) {
                    if (active) {
                        s = scales_in[row * gpr + g];
                        inv = __fdiv_rn(1.0f, s);
                    }
                } else {
                    uint32_t m16 = fold16(absmax_chunk(v, 0));
                    for (int o = lanes_per_group >> 1; o; o >>= 1) m16 = max(m16, __shfl_xor_sync(0xffffffffu, m16, o));
                    if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
                    scale_pair(mag16_to_float<DT>(m16), f.Q, s, inv, status);
                }
                if (scales_out && active && (q & (lanes_per_group - 1)) == 0) scales_out[row * gpr + g] = s;
            }
            if (!active) continue;
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            uint32_t code[8];
            float val[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float xv[2];
                unpack2<DT>(w[i], xv[0], xv[1]);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float t = __fmul_rn(xv[h], inv);
                    const uint32_t neg = __float_as_uint(xv[h]) >> 31;
                    float value;
                    uint32_t c;
                    if (f.is_fp) {
                        float r = fp_grid_round(fminf(fabsf(t), 2.0f * f.Q), f.eminb, f.kadd);
                        r = fminf(r, f.Q);
                        c = fp_code_from_mag(r, f) | (neg << (f.bits - 1));
                        value = neg ? -r : r;
                    } else {
                        float r = __fsub_rn(__fadd_rn(fminf(fmaxf(t, -1024.0f), 1024.0f), kMagic), kMagic);
                        r = fminf(fmaxf(r, int_lo), f.Q);
                        c = (uint32_t)((int)r) & ((1u << f.bits) - 1u);
                        value = r;
                    }
                    code[2 * i + h] = c;
                    val[2 * i + h] = value;
                }
            }
            const size_t e0 = (size_t)row * cols + (size_t)q * 8;
            if (codes_out) {
                if (f.bits == 8) {
                    uint2 o;
                    o.x = code[0] | (code[1] << 8) | (code[2] << 16) | (code[3] << 24);
                    o.y = code[4] | (code[5] << 8) | (code[6] << 16) | (code[7] << 24);
                    *reinterpret_cast<uint2 *>(codes_out + e0) = o;
                } else {
                    uint32_t o = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) o |= code[i] << (4 * i);
                    *reinterpret_cast<uint32_t *>(codes_out + (e0 >> 1)) = o;
                }
            }
            if (dequant_out) {
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    o[i] = (uint32_t)to_storage<DT>(__fmul_rn(val[2 * i], s)) |
                           ((uint32_t)to_storage<DT>(__fmul_rn(val[2 * i + 1], s)) << 16);
                *reinterpret_cast<uint4 *>(dequant_out + e0) = make_uint4(o[0], o[1], o[2], o[3]);
            }
            if (values_out) {  // unscaled grid values (exact in fp16 and bf16 for every format here)
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (values_dtype == MOFQ_F16)
                        o[i] = (uint32_t)to_storage<MOFQ_F16>(val[2 * i]) | ((uint32_t)to_storage<MOFQ_F16>(val[2 * i + 1]) << 16);
                    else
                        o[i] = (uint32_t)to_storage<MOFQ_BF16>(val[2 * i]) | ((uint32_t)to_storage<MOFQ_BF16>(val[2 * i + 1]) << 16);
                }
                *reinterpret_cast<uint4 *>(values_out + e0) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
    if (status) atomicOr(&hdr->status, status);
}

// ---- fused code emission: per-channel scales, every requested format from ONE read of the row --------------------
// Used for the tensor-core operands of the layer-output metric and for plain per-channel quantisation.
// The FP codes come from the hardware converts (round-to-nearest-even, saturating, sign kept on zero), which
// produce the same codes as the add/subtract rounding above; INT codes are the low bits of t + 1.5*2^23.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi)
{
    uint32_t d;
    asm("{ .reg .b16 t; cvt.rn.satfinite.e4m3x2.f32 t, %2, %1; cvt.u32.u16 %0, t; }" : "=r"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ uint32_t cvt_e5m2x2(float lo, float hi)
{
    uint32_t d;
    asm("{ .reg .b16 t; cvt.rn.satfinite.e5m2x2.f32 t, %2, %1; cvt.u32.u16 %0, t; }" : "=r"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi)
{
    uint32_t d;
    asm("{ .reg .b8 t; .reg .b16 w; cvt.rn.satfinite.e2m1x2.f32 t, %2, %1; mov.b16 w, {t, 0}; cvt.u32.u16 %0, w; }" : "=r"(d) : "f"(lo), "f"(hi));
    return d & 0xFFu;
}

// ---- fast code emission for group and per-tensor scales (codes + scales only, abs-max scales) -------------------
// A team of lanes owns one scale block (a group; for a per-tensor scale a run of 32 elements), each lane four
// consecutive 16-byte chunks held in registers: abs-max by shuffles inside the team, the scale pair, then the codes
// through packed f32x2 arithmetic and the hardware converts, stored as contiguous runs per lane.  The format is
// decoded once per kernel (it may have been picked on the device), not per element.
enum { CLS_INT4 = 0, CLS_INT8 = 1, CLS_E2M1 = 2, CLS_E4M3 = 3, CLS_E5M2 = 4 };

// code(s) of one pair of elements (already widened to packed binary32); 8-bit classes: 16 bits, 4-bit classes: 8 bits
template <int CLS>
__device__ __forceinline__ uint32_t pair_code(uint64_t a2, uint64_t inv2)
{
    float lo, hi;
    kqmath::upk(kqmath::mul2(a2, inv2), lo, hi);   // t = RN32(x * inv) first: the code is decided on the rounded t
    if (CLS == CLS_INT4 || CLS == CLS_INT8) {
        // the low mantissa bits of t + 1.5 * 2^23 are the two's-complement code
        // (the add stays scalar: a packed multiply followed by a packed add came out as one fused operation,
        // which rounds the exact product instead of t and breaks ties differently)
        lo = __fadd_rn(lo, kMagic);
        hi = __fadd_rn(hi, kMagic);
        uint32_t t = __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x0040);
        if (CLS == CLS_INT4) {
            t &= 0x0F0Fu;
            t = (t | (t >> 4)) & 0xFFu;
        }
        return t;
    }
    return CLS == CLS_E2M1 ? cvt_e2m1x2(lo, hi) : CLS == CLS_E4M3 ? cvt_e4m3x2(lo, hi) : cvt_e5m2x2(lo, hi);
}

// four pair codes -> the chunk's codes, little-endian (8-bit classes: 64 bits, 4-bit classes: 32 bits in .x)
template <int CLS>
__device__ __forceinline__ uint2 pack_codes(const uint32_t (&c)[4])
{
    uint2 o;
    if (CLS == CLS_INT4 || CLS == CLS_E2M1) {
        o.x = __byte_perm(__byte_perm(c[0], c[1], 0x0040), __byte_perm(c[2], c[3], 0x0040), 0x5410);
        o.y = 0;
    } else {
        o.x = __byte_perm(c[0], c[1], 0x5410);
        o.y = __byte_perm(c[2], c[3], 0x5410);
    }
    return o;
}

template <int DT, int CLS>
__device__ __forceinline__ uint2 chunk_codes(const uint4 v, uint64_t inv2)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = pair_code<CLS>(kqmath::unpack2<DT>(w[i]), inv2);
    return pack_codes<CLS>(c);
}

// the codes of up to three formats (classes C0, C1, C2; -1 = absent) from one widening of the chunk
template <int DT, int C0, int C1, int C2>
__device__ __forceinline__ void chunk_codes3(const uint4 v, const uint64_t (&inv2)[3], uint2 (&o)[3])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t c0[4], c1[4], c2[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint64_t a2 = kqmath::unpack2<DT>(w[i]);
        c0[i] = pair_code<C0>(a2, inv2[0]);
        if (C1 >= 0) c1[i] = pair_code<(C1 >= 0 ? C1 : 0)>(a2, inv2[1]);
        if (C2 >= 0) c2[i] = pair_code<(C2 >= 0 ? C2 : 0)>(a2, inv2[2]);
    }
    o[0] = pack_codes<C0>(c0);
    if (C1 >= 0) o[1] = pack_codes<(C1 >= 0 ? C1 : 0)>(c1);
    if (C2 >= 0) o[2] = pack_codes<(C2 >= 0 ? C2 : 0)>(c2);
}

template <int CLS>
__device__ __forceinline__ void store_codes(unsigned char *base, size_t chunk, const uint2 o)
{
    if (CLS == CLS_INT4 || CLS == CLS_E2M1) reinterpret_cast<uint32_t *>(base)[chunk] = o.x;
    else reinterpret_cast<uint2 *>(base)[chunk] = o;
}

template <int DT, int CLS>
__device__ __forceinline__ void emit_blocks(const uint16_t *__restrict__ x, long long rows, int cols, long long ld, float Q, int width,
                                            bool uniform, unsigned char *codes_out, float *scales_out, WsHeader *hdr, int &status)
{
    constexpr int KPL = 4;
    constexpr bool kFour = CLS == CLS_INT4 || CLS == CLS_E2M1;
    const int lane = threadIdx.x & 31;
    const int cpb = width >> 3;                             // chunks per block: 1, 2, 4, ..., 32
    const int n_k = min(KPL, cpb);                          // chunks per lane
    const int team = max(1, cpb / KPL);
    const int tl = lane & (team - 1);
    const int teams_per_warp = 32 / team;
    const int per_row = cols / width;
    const long long n_blocks = rows * per_row;
    const long long warp_id = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * (blockDim.x >> 5);
    const float rQ = 1.0f / Q;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(codes_out) & 15) == 0;   // blocks of >= 32 elements start on 32-element boundaries
    float s_u = 1.0f, inv_u = 1.0f;
    if (uniform) {
        const uint32_t m16 = *reinterpret_cast<volatile uint32_t *>(&hdr->absmax_bits);
        if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
        scale_pair(mag16_to_float<DT>(m16), Q, s_u, inv_u, status);
        if (scales_out && blockIdx.x == 0 && threadIdx.x == 0) scales_out[0] = s_u;
    }
    for (long long b0 = warp_id * teams_per_warp; b0 < n_blocks; b0 += n_warps * teams_per_warp) {
        const long long b = b0 + lane / team;
        const bool live = b < n_blocks;                     // whole teams are live or not; shuffles stay warp-wide
        const long long r = live ? b / per_row : 0;
        const long long c0 = live ? (b - r * per_row) * width : 0;
        const uint4 *blk = reinterpret_cast<const uint4 *>(x + r * ld + c0);
        uint4 v[KPL];
        uint32_t m = 0;
#pragma unroll
        for (int k = 0; k < KPL; ++k) {
            v[k] = (live && k < n_k) ? __ldg(blk + tl * n_k + k) : make_uint4(0, 0, 0, 0);
            m = kqmath::absmax_chunk<DT>(v[k], m);
        }
        float s = s_u, inv = inv_u;
        if (!uniform) {
            uint32_t m16 = fold16(m);
            for (int o = team >> 1; o; o >>= 1) m16 = max(m16, __shfl_xor_sync(0xffffffffu, m16, o));
            if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
            const float a = mag16_to_float<DT>(m16);
            if (DT == MOFQ_F16) kqmath::scale_pair_fast(a, Q, rQ, s, inv);
            else scale_pair(a, Q, s, inv, status);
            if (live && tl == 0 && scales_out) scales_out[b] = s;
        }
        if (!live) continue;
        const uint64_t inv2 = kqmath::pk(inv, inv);
        const size_t e0 = (size_t)r * cols + (size_t)c0 + (size_t)(tl * n_k) * 8;   // first element of this lane's run
        if (n_k == KPL && vec_ok) {
            // a lane's four chunks are one aligned run of 16 (4-bit) or 32 (8-bit) bytes of codes
            uint2 o[KPL];
#pragma unroll
            for (int k = 0; k < KPL; ++k) o[k] = chunk_codes<DT, CLS>(v[k], inv2);
            if (kFour) {
                *reinterpret_cast<uint4 *>(codes_out + (e0 >> 1)) = make_uint4(o[0].x, o[1].x, o[2].x, o[3].x);
            } else {
                reinterpret_cast<uint4 *>(codes_out + e0)[0] = make_uint4(o[0].x, o[0].y, o[1].x, o[1].y);
                reinterpret_cast<uint4 *>(codes_out + e0)[1] = make_uint4(o[2].x, o[2].y, o[3].x, o[3].y);
            }
            continue;
        }
#pragma unroll
        for (int k = 0; k < KPL; ++k) {
            if (k < n_k) {
                const uint2 o = chunk_codes<DT, CLS>(v[k], inv2);
                if (kFour) reinterpret_cast<uint32_t *>(codes_out + (e0 >> 1))[k] = o.x;
                else reinterpret_cast<uint2 *>(codes_out + e0)[k] = o;
            }
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(256)
kq_emit_blocks(const uint16_t *__restrict__ x, long long rows, int cols, long long ld, FmtDesc f, int width, int uniform,
               unsigned char *codes_out, float *scales_out, WsHeader *hdr, const EmitSel sel)
{
    // When the host launched this kernel as the next layer of one emission call, the launch after it may start as
    // soon as every block of this one is running: the layers read and write disjoint buffers.  The wait at the end
    // keeps the launches completing in stream order.
    asm volatile("griddepcontrol.launch_dependents;");
    if (sel.res) {  // the winner of the selection record decides the grid
        const int c = min(max(sel.res->chosen, 0), MOFQ_MAX_CAND - 1);
        f = sel.cand[c];
        if (sel.tag_out && blockIdx.x == 0 && threadIdx.x == 0) *sel.tag_out = sel.format[c];
    }
    int status = 0;
    const int cls = !f.is_fp ? (f.bits == 4 ? CLS_INT4 : CLS_INT8) : f.M == 1 ? CLS_E2M1 : f.M == 3 ? CLS_E4M3 : CLS_E5M2;
    switch (cls) {
    case CLS_INT4: emit_blocks<DT, CLS_INT4>(x, rows, cols, ld, f.Q, width, uniform != 0, codes_out, scales_out, hdr, status); break;
    case CLS_INT8: emit_blocks<DT, CLS_INT8>(x, rows, cols, ld, f.Q, width, uniform != 0, codes_out, scales_out, hdr, status); break;
    case CLS_E2M1: emit_blocks<DT, CLS_E2M1>(x, rows, cols, ld, f.Q, width, uniform != 0, codes_out, scales_out, hdr, status); break;
    case CLS_E4M3: emit_blocks<DT, CLS_E4M3>(x, rows, cols, ld, f.Q, width, uniform != 0, codes_out, scales_out, hdr, status); break;
    default: emit_blocks<DT, CLS_E5M2>(x, rows, cols, ld, f.Q, width, uniform != 0, codes_out, scales_out, hdr, status); break;
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");   // a no-op unless this launch was started early
    if (status) atomicOr(&hdr->status, status);
}

struct EmitSet {
    int n;
    float Q[3];                // formats in the kernel's class order C0, C1, C2
    unsigned char *codes[3];
    float *scales[3];
    uint16_t *x16;     // per-tensor variant, bf16 input: the tensor as binary16 times a power of two (nullable)
    float *alpha;      // 1 / that power of two
};

// Per-channel scales, codes of up to three formats (classes C0..C2 fixed at compile time, -1 = absent) from one staged
// read of each row: one block per row at a time.
template <int DT, int C0, int C1, int C2>
__global__ void __launch_bounds__(kRowThreads)
kq_emit_codes_rows(const uint16_t *__restrict__ x, long long rows, int cols, long long ld, EmitSet es, WsHeader *hdr)
{
    chain_enter();
    constexpr int N = 1 + (C1 >= 0) + (C2 >= 0);
    constexpr bool four = C0 == CLS_INT4 || C0 == CLS_E2M1;   // the classes of one launch share a code width
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint32_t mred[34];
    __shared__ float inv_s[3];
    const int chunks = cols >> 3;
    const uint4 *row4 = reinterpret_cast<const uint4 *>(smem);
    int status = 0;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const unsigned char *src = reinterpret_cast<const unsigned char *>(x + row * ld);
        for (int q = threadIdx.x; q < chunks; q += kRowThreads) cp_async16(smem + q * 16, src + (size_t)q * 16);
        cp_async_wait_all();
        __syncthreads();
        uint32_t m = 0;
        for (int q = threadIdx.x; q < chunks; q += kRowThreads) m = absmax_chunk(row4[q], m);
        const uint32_t m16 = block_max_u32(fold16(m), mred);
        if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
        if ((int)threadIdx.x < N) {
            float sc, inv;
            scale_pair(mag16_to_float<DT>(m16), threadIdx.x == 0 ? es.Q[0] : threadIdx.x == 1 ? es.Q[1] : es.Q[2], sc, inv, status);
            inv_s[threadIdx.x] = inv;
            float *sp = threadIdx.x == 0 ? es.scales[0] : threadIdx.x == 1 ? es.scales[1] : es.scales[2];
            if (sp) sp[row] = sc;
        }
        __syncthreads();
        const uint64_t inv2[3] = {kqmath::pk(inv_s[0], inv_s[0]), kqmath::pk(inv_s[1], inv_s[1]), kqmath::pk(inv_s[2], inv_s[2])};
        const size_t row_off = four ? ((size_t)row * cols >> 1) : (size_t)row * cols;
        unsigned char *out0 = es.codes[0] + row_off, *out1 = N > 1 ? es.codes[1] + row_off : nullptr,
                      *out2 = N > 2 ? es.codes[2] + row_off : nullptr;
#pragma unroll 2
        for (int q = threadIdx.x; q < chunks; q += kRowThreads) {
            uint2 o[3];
            chunk_codes3<DT, C0, C1, C2>(row4[q], inv2, o);
            store_codes<C0>(out0, q, o[0]);
            if (C1 >= 0) store_codes<(C1 >= 0 ? C1 : 0)>(out1, q, o[1]);
            if (C2 >= 0) store_codes<(C2 >= 0 ? C2 : 0)>(out2, q, o[2]);
        }
        __syncthreads();
    }
    if (status) atomicOr(&hdr->status, status);
}

// per-tensor variant: the abs-max is already in the workspace header; codes of every requested format from one read
template <int DT, int C0, int C1, int C2>
__global__ void __launch_bounds__(256)
kq_emit_codes_uniform(const uint16_t *__restrict__ x, long long rows, int chunks_per_row, long long ld, EmitSet es, WsHeader *hdr)
{
    chain_enter();
    constexpr int N = 1 + (C1 >= 0) + (C2 >= 0);
    __shared__ float inv_s[3];
    int status = 0;
    const uint32_t m16 = *reinterpret_cast<volatile uint32_t *>(&hdr->absmax_bits);
    if (mag16_nonfinite<DT>(m16)) status |= MOFQ_STATUS_NONFINITE_INPUT;
    // binary16 copy of a bfloat16 tensor for the reference product: scaled by the power of two that puts the abs-max in
    // [2^13, 2^14), which keeps every value exact unless it is more than 2^27 times smaller than the abs-max
    float mult = 1.0f;
    if (DT == MOFQ_BF16 && es.x16) {
        const int e = (int)(m16 >> 7) - 127;
        const int pw = m16 ? 13 - e : 0;
        mult = exp2f((float)max(min(pw, 126), -126));
        if (blockIdx.x == 0 && threadIdx.x == 0) *es.alpha = exp2f((float)-max(min(pw, 126), -126));
    }
    if ((int)threadIdx.x < N) {   // thread f forms format f's scale pair for the block
        float sc, inv;
        scale_pair(mag16_to_float<DT>(m16), threadIdx.x == 0 ? es.Q[0] : threadIdx.x == 1 ? es.Q[1] : es.Q[2], sc, inv, status);
        inv_s[threadIdx.x] = inv;
        float *sp = threadIdx.x == 0 ? es.scales[0] : threadIdx.x == 1 ? es.scales[1] : es.scales[2];
        if (blockIdx.x == 0 && sp) sp[0] = sc;
    }
    __syncthreads();
    const uint64_t inv2[3] = {kqmath::pk(inv_s[0], inv_s[0]), kqmath::pk(inv_s[N > 1 ? 1 : 0], inv_s[N > 1 ? 1 : 0]),
                              kqmath::pk(inv_s[N > 2 ? 2 : 0], inv_s[N > 2 ? 2 : 0])};
    const long long total = rows * chunks_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = rows == 1 ? 0 : i / chunks_per_row;
        const int c = (int)(i - r * chunks_per_row);
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(x + r * ld) + c);
        if (DT == MOFQ_BF16 && es.x16) {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            uint32_t o[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float lo = __uint_as_float(w[k] << 16) * mult, hi = __uint_as_float(w[k] & 0xFFFF0000u) * mult;
                o[k] = (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
            }
            reinterpret_cast<uint4 *>(es.x16)[i] = make_uint4(o[0], o[1], o[2], o[3]);
        }
        uint2 o[3];
        chunk_codes3<DT, C0, C1, C2>(v, inv2, o);
        store_codes<C0>(es.codes[0], (size_t)i, o[0]);
        if (C1 >= 0) store_codes<(C1 >= 0 ? C1 : 0)>(es.codes[1], (size_t)i, o[1]);
        if (C2 >= 0) store_codes<(C2 >= 0 ? C2 : 0)>(es.codes[2], (size_t)i, o[2]);
    }
    if (status) atomicOr(&hdr->status, status);
}

// ---- host-side dispatch ----------------------------------------------------------------------------------
#define MOFQ_CUDA_OK(expr)                      \
    do {                                        \
        if ((expr) != cudaSuccess) {            \
            (void)cudaGetLastError();           \
            return MOFQ_ERR_CUDA;               \
        }                                       \
    } while (0)

template <typename F>
int dispatch_cands(int dt, int ni, int nfp, F &&f)
{
#define MOFQ_CASE(DT_, NI_, NFP_) \
    if (dt == DT_ && ni == NI_ && nfp == NFP_) return f(std::integral_constant<int, DT_>(), std::integral_constant<int, NI_>(), std::integral_constant<int, NFP_>());
    MOFQ_CASE(0, 1, 0) MOFQ_CASE(0, 0, 1) MOFQ_CASE(0, 1, 1) MOFQ_CASE(0, 0, 2) MOFQ_CASE(0, 1, 2)
    MOFQ_CASE(1, 1, 0) MOFQ_CASE(1, 0, 1) MOFQ_CASE(1, 1, 1) MOFQ_CASE(1, 0, 2) MOFQ_CASE(1, 1, 2)
#undef MOFQ_CASE
    return MOFQ_ERR_UNSUPPORTED;
}

// Canonical candidate set -> compile-time (dtype, INT present, FP kind of slot 0, FP kind of slot 1); kinds are
// kqmath::FPK_* or -1.  Only the combinations one bit-width allows exist.
template <typename F>
int dispatch_kinds(int dt, int ni, int k0, int k1, F &&f)
{
#define MOFQ_KIND(DT_, NI_, K0_, K1_)                                                                    \
    if (dt == DT_ && ni == NI_ && k0 == K0_ && k1 == K1_)                                                \
        return f(std::integral_constant<int, DT_>(), std::integral_constant<int, NI_>(), std::integral_constant<int, K0_>(), \
                 std::integral_constant<int, K1_>());
#define MOFQ_KIND_DT(DT_)                                                                                             \
    MOFQ_KIND(DT_, 1, -1, -1) MOFQ_KIND(DT_, 0, 0, -1) MOFQ_KIND(DT_, 1, 0, -1) MOFQ_KIND(DT_, 0, 0, 0) MOFQ_KIND(DT_, 1, 0, 0) \
    MOFQ_KIND(DT_, 0, 1, -1) MOFQ_KIND(DT_, 1, 1, -1) MOFQ_KIND(DT_, 0, 2, -1) MOFQ_KIND(DT_, 1, 2, -1)                         \
    MOFQ_KIND(DT_, 0, 1, 2) MOFQ_KIND(DT_, 1, 1, 2) MOFQ_KIND(DT_, 0, 2, 1) MOFQ_KIND(DT_, 1, 2, 1)
    MOFQ_KIND_DT(0)
    MOFQ_KIND_DT(1)
#undef MOFQ_KIND_DT
#undef MOFQ_KIND
    return MOFQ_ERR_UNSUPPORTED;
}

int fp_kind_of(int format)
{
    return format == MOFQ_FP8_E4M3 ? (int)kqmath::FPK_E4M3 : format == MOFQ_FP8_E5M2 ? (int)kqmath::FPK_E5M2 : (int)kqmath::FPK_E2M1;
}

RowQ job_rowq(const ScoreJob &job) { return candset_rowq(job.cs); }

int blocks_per_sm(const void *kernel, int threads, size_t smem)
{
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

template <typename K>
int set_smem(K kernel, size_t smem)
{
    if (smem > 48 * 1024) MOFQ_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    return MOFQ_OK;
}

}  // namespace

int sm_count()
{
    static int cached = 0;
    if (!cached) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return 148;
        }
        cached = n;
    }
    return cached;
}

int launch_absmax_update(const mofq_tensor &x, float *absmax_inout, cudaStream_t st)
{
    if (x.cols / 8 > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    const long long total = x.rows * (x.cols / 8);
    const int grid = (int)std::min<long long>((total + 255) / 256, (long long)sm_count() * 8);
    if (x.dtype == MOFQ_F16)
        kq_absmax_update<0><<<grid, 256, 0, st>>>(xp, x.rows, (int)(x.cols / 8), x.ld, absmax_inout);
    else
        kq_absmax_update<1><<<grid, 256, 0, st>>>(xp, x.rows, (int)(x.cols / 8), x.ld, absmax_inout);
    MOFQ_CUDA_OK(cudaGetLastError());
    return MOFQ_OK;
}

// tensor error of every candidate under caller-supplied per-tensor scales (job.gran is ignored)
int launch_score_supplied(const ScoreJob &job, const float *scales, cudaStream_t st)
{
    const mofq_tensor &x = job.x;
    if (x.cols / 8 > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    const long long total = x.rows * (x.cols / 8);
    const int grid = (int)std::min<long long>((total + 255) / 256, (long long)sm_count() * 8);
    return dispatch_cands(x.dtype, job.cs.n_int, job.cs.n_fp, [&](auto DT, auto NI, auto NFP) {
        kq_score_supplied<DT(), NI(), NFP()><<<grid, 256, 0, st>>>(xp, x.rows, (int)(x.cols / 8), x.ld, job.cs, scales, job.hdr,
                                                                    job.partials, job.fin);
        MOFQ_CUDA_OK(cudaGetLastError());
        return MOFQ_OK;
    });
}

// abs-max of the whole tensor into hdr->absmax_bits (the caller has cleared that word)
int launch_select_blocks(const ScoreJob &job, uint8_t *choice, float *block_sse, cudaStream_t st)
{
    const mofq_tensor &x = job.x;
    if (job.gran != MOFQ_PER_CHANNEL && job.gran != MOFQ_PER_GROUP) return MOFQ_ERR_UNSUPPORTED;
    const bool with_map = choice != nullptr;   // without a format map this is plain per-block-scale scoring
    if (x.cols > 0x7fffffffLL || (with_map && job.fin.n_cand + 1 > MOFQ_MAX_CAND)) return MOFQ_ERR_UNSUPPORTED;
    const int width = job.gran == MOFQ_PER_GROUP ? job.group : (int)x.cols;
    const int cpb = width >> 3;
    const int team = (cpb <= 128 && (cpb & (cpb - 1)) == 0) ? std::max(1, cpb / 4) : 32;
    const long long n_blocks = x.rows * (x.cols / width);
    const long long warps = (n_blocks + (32 / team) - 1) / (32 / team);
    const int grid = (int)std::min<long long>((warps + 7) / 8, std::min<long long>((long long)sm_count() * 8, kMaxSlots));
    const RowQ rq = job_rowq(job);
    const int k0 = job.cs.n_fp > 0 ? fp_kind_of(job.fp_formats[0]) : -1, k1 = job.cs.n_fp > 1 ? fp_kind_of(job.fp_formats[1]) : -1;
    BlockSel bs{};
    bs.choice = choice;
    bs.block_sse = block_sse;
    bs.n_cand = job.fin.n_cand;
    std::memcpy(bs.perm, job.fin.perm, sizeof(bs.perm));
    // the finalize step reports the candidates in the caller's order and then the mixture (accumulator nc)
    Finalize fin = job.fin;
    if (with_map) {
        fin.perm[fin.n_cand] = fin.nc;
        fin.n_cand += 1;
    }
    fin.nc += 1;
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    return dispatch_kinds(x.dtype, job.cs.n_int, k0, k1, [&](auto DT, auto NI, auto K0, auto K1) {
        kq_select_blocks<DT(), NI(), K0(), K1()><<<grid, 256, 0, st>>>(xp, x.rows, (int)x.cols, x.ld, width, team, rq, bs, job.hdr,
                                                                       job.partials, fin);
        MOFQ_CUDA_OK(cudaGetLastError());
        return MOFQ_OK;
    });
}

int launch_absmax(const mofq_tensor &x, WsHeader *hdr, cudaStream_t st, bool chained)
{
    if (x.cols / 8 > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    const long long total = x.rows * (x.cols / 8);
    const int grid = (int)std::max<long long>(1, std::min<long long>((total + 1023) / 1024, (long long)sm_count() * 8));   // four loads in flight per thread
    // a dense tensor is one long row for the kernel: no per-chunk row arithmetic, independent loads
    const bool flat = x.ld == x.cols && total <= 0x7fffffffLL;
    const long long rows = flat ? 1 : x.rows;
    const int cpr = flat ? (int)total : (int)(x.cols / 8);
    if (x.dtype == MOFQ_F16)
        MOFQ_CUDA_OK(launch_chained(kq_absmax<0>, dim3(grid), dim3(256), 0, st, chained, xp, rows, cpr, (long long)x.ld, hdr));
    else
        MOFQ_CUDA_OK(launch_chained(kq_absmax<1>, dim3(grid), dim3(256), 0, st, chained, xp, rows, cpr, (long long)x.ld, hdr));
    return MOFQ_OK;
}

int launch_score(const ScoreJob &job, cudaStream_t st)
{
    const mofq_tensor &x = job.x;
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    const bool dense = (x.ld == x.cols);
    const bool has_ch = job.gran == MOFQ_PER_CHANNEL || job.gran2 == MOFQ_PER_CHANNEL;
    const bool has_grp = job.gran == MOFQ_PER_GROUP || job.gran2 == MOFQ_PER_GROUP;
    const bool has_tensor = job.gran == MOFQ_PER_TENSOR || job.gran2 == MOFQ_PER_TENSOR;
    const int nsm = sm_count();
    const bool rows_route = !has_tensor && has_ch && x.cols <= (1 << 20) && rows_single_applicable(job);
    if (job.clear_header && !rows_route) MOFQ_CUDA_OK(cudaMemsetAsync(job.hdr, 0, sizeof(WsHeader), st));

    if (has_tensor) {
        if (job.gran2 != MOFQ_GRAN_NONE) return MOFQ_ERR_UNSUPPORTED;  // per-tensor cannot share a read
        MOFQ_CUDA_OK(cudaMemsetAsync(&job.hdr->absmax_bits, 0, sizeof(uint32_t), st));
        const long long rows = dense ? 1 : x.rows;
        const long long cpr = dense ? x.rows * x.cols / 8 : x.cols / 8;
        if (cpr > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
        const long long total = rows * cpr;
        const int grid = (int)std::min<long long>((total + 255) / 256, (long long)nsm * 8);
        if (x.dtype == MOFQ_F16)
            kq_absmax<0><<<grid, 256, 0, st>>>(xp, rows, (int)cpr, x.ld, job.hdr);
        else
            kq_absmax<1><<<grid, 256, 0, st>>>(xp, rows, (int)cpr, x.ld, job.hdr);
        MOFQ_CUDA_OK(cudaGetLastError());
        const RowQ rq = job_rowq(job);
        const int k0 = job.cs.n_fp > 0 ? fp_kind_of(job.fp_formats[0]) : -1, k1 = job.cs.n_fp > 1 ? fp_kind_of(job.fp_formats[1]) : -1;
        return dispatch_kinds(x.dtype, job.cs.n_int, k0, k1, [&](auto DT, auto NI, auto K0, auto K1) {
            kq_score_uniform<DT(), NI(), K0(), K1()><<<grid, 256, 0, st>>>(xp, rows, (int)cpr, x.ld, rq, job.hdr, job.partials, job.fin);
            MOFQ_CUDA_OK(cudaGetLastError());
            return MOFQ_OK;
        });
    }

    // group scales only (dense or strided): the register-resident team kernel, without a format map
    if (has_grp && !has_ch) return launch_select_blocks(job, nullptr, nullptr, st);

    // row kernels: per-channel scales, alone or with group scales from the same read
    if (x.cols > (1 << 20)) return MOFQ_ERR_UNSUPPORTED;
    if (rows_route) return rows_single_run(job, st);
    const int chunks = (int)(x.cols / 8);
    const int gpr = has_grp ? (int)(x.cols / job.group) : 0;
    const size_t smem = (size_t)x.cols * 2 + (((size_t)chunks * 2 + 15) & ~(size_t)15) + (size_t)gpr * 8 * 3 + 16;
    if (smem > 200 * 1024) return MOFQ_ERR_UNSUPPORTED;
    const int grp_first = (job.gran == MOFQ_PER_GROUP) ? 1 : 0;
    const RowQ rq = job_rowq(job);
    const int k0 = job.cs.n_fp > 0 ? fp_kind_of(job.fp_formats[0]) : -1, k1 = job.cs.n_fp > 1 ? fp_kind_of(job.fp_formats[1]) : -1;
    auto launch = [&](auto kernel) {
        if (int rc = set_smem(kernel, smem)) return rc;
        const int occ = std::max(1, blocks_per_sm((const void *)kernel, kRowThreads, smem));
        const int grid = (int)std::min<long long>(x.rows, std::min<long long>((long long)nsm * occ, kMaxSlots));
        kernel<<<grid, kRowThreads, smem, st>>>(xp, x.rows, (int)x.cols, x.ld, has_grp ? job.group : 8, grp_first, rq, job.hdr,
                                                job.partials, job.fin);
        MOFQ_CUDA_OK(cudaGetLastError());
        return MOFQ_OK;
    };
    return dispatch_kinds(x.dtype, job.cs.n_int, k0, k1, [&](auto DT, auto NI, auto K0, auto K1) {
        if (has_ch && has_grp) return launch(kq_score_rows<DT(), NI(), K0(), K1(), true, true>);
        return launch(kq_score_rows<DT(), NI(), K0(), K1(), true, false>);
    });
}

namespace {

int emit_class(int format)
{
    switch (format) {
    case MOFQ_INT4: return CLS_INT4;
    case MOFQ_INT8: return CLS_INT8;
    case MOFQ_FP8_E4M3: return CLS_E4M3;
    case MOFQ_FP8_E5M2: return CLS_E5M2;
    default: return CLS_E2M1;   // both E2M1 variants: same spacing below the IEEE maximum 3 (their Q differ)
    }
}

// The emission kernels are instantiated for single classes and for the 8-bit class pairs and triple, classes in
// ascending order; any other list is emitted one format per launch.
template <typename F>
int dispatch_classes(int dt, int c0, int c1, int c2, F &&f)
{
#define MOFQ_CLS(C0_, C1_, C2_)                                                                                     \
    if (c0 == C0_ && c1 == C1_ && c2 == C2_)                                                                         \
        return dt == MOFQ_F16 ? f(std::integral_constant<int, 0>(), std::integral_constant<int, C0_>(), std::integral_constant<int, C1_>(), std::integral_constant<int, C2_>()) \
                              : f(std::integral_constant<int, 1>(), std::integral_constant<int, C0_>(), std::integral_constant<int, C1_>(), std::integral_constant<int, C2_>());
    MOFQ_CLS(CLS_INT4, -1, -1) MOFQ_CLS(CLS_E2M1, -1, -1)   // (4-bit codes are emitted one format at a time: no caller asks for more)
    MOFQ_CLS(CLS_INT8, -1, -1) MOFQ_CLS(CLS_E4M3, -1, -1) MOFQ_CLS(CLS_E5M2, -1, -1) MOFQ_CLS(CLS_INT8, CLS_E4M3, -1)
    MOFQ_CLS(CLS_INT8, CLS_E5M2, -1) MOFQ_CLS(CLS_E4M3, CLS_E5M2, -1) MOFQ_CLS(CLS_INT8, CLS_E4M3, CLS_E5M2)
#undef MOFQ_CLS
    return MOFQ_ERR_UNSUPPORTED;
}

// The formats of one emission call sorted by class (stable), their buffers following; cls[] padded with -1.
struct EmitPlan {
    EmitSet es;
    int cls[3];
    bool has_kernel;   // an instantiation exists for the triple
};
int make_emit_plan(int n, const int *formats, void *const *codes, float *const *scales, EmitPlan *plan)
{
    if (n < 1 || n > 3) return MOFQ_ERR_UNSUPPORTED;
    int order[3] = {0, 1, 2};
    for (int i = 1; i < n; ++i)
        for (int k = i; k > 0 && emit_class(formats[order[k]]) < emit_class(formats[order[k - 1]]); --k) std::swap(order[k], order[k - 1]);
    plan->es = EmitSet{};
    plan->es.n = n;
    for (int i = 0; i < 3; ++i) plan->cls[i] = -1;
    int bits = 0;
    for (int i = 0; i < n; ++i) {
        FmtDesc d;
        if (!describe_format(formats[order[i]], &d)) return MOFQ_ERR_INVALID_ARG;
        if (bits && d.bits != bits) return MOFQ_ERR_INVALID_ARG;   // one code width per call
        bits = d.bits;
        plan->cls[i] = emit_class(formats[order[i]]);
        plan->es.Q[i] = d.Q;
        plan->es.codes[i] = static_cast<unsigned char *>(codes[order[i]]);
        plan->es.scales[i] = scales ? scales[order[i]] : nullptr;
    }
    plan->has_kernel = dispatch_classes(MOFQ_F16, plan->cls[0], plan->cls[1], plan->cls[2], [](auto, auto, auto, auto) { return MOFQ_OK; }) == MOFQ_OK;
    return MOFQ_OK;
}

}  // namespace

// Per-tensor scale from the abs-max already stored in hdr->absmax_bits (launch_absmax); codes of n formats from one read.
int launch_emit_codes_uniform(const mofq_tensor &x, int n, const int *formats, void *const *codes, float *const *scales,
                              WsHeader *hdr, cudaStream_t st, uint16_t *x16_out, float *alpha_out, bool chained)
{
    if (x.cols / 8 > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
    if (x16_out && (x.dtype != MOFQ_BF16 || !alpha_out)) return MOFQ_ERR_INVALID_ARG;
    EmitPlan plan;
    if (int rc = make_emit_plan(n, formats, codes, scales, &plan)) return rc;
    if (!plan.has_kernel) {   // a class twice: one launch per format (the binary16 copy with the first)
        for (int i = 0; i < n; ++i)
            if (int rc = launch_emit_codes_uniform(x, 1, formats + i, codes + i, scales ? scales + i : nullptr, hdr, st,
                                                   i == 0 ? x16_out : nullptr, i == 0 ? alpha_out : nullptr, chained || i > 0))
                return rc;
        return MOFQ_OK;
    }
    plan.es.x16 = x16_out;
    plan.es.alpha = alpha_out;
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    const long long total = x.rows * (x.cols / 8);
    const int grid = (int)std::max<long long>(1, std::min<long long>((total + 1023) / 1024, (long long)sm_count() * 8));   // >= 4 chunks per thread
    // a dense tensor is one long row for this kernel (the codes are dense either way): no per-chunk row arithmetic
    const bool flat = x.ld == x.cols && total <= 0x7fffffffLL;
    const long long rows = flat ? 1 : x.rows;
    const int cpr = flat ? (int)total : (int)(x.cols / 8);
    return dispatch_classes(x.dtype, plan.cls[0], plan.cls[1], plan.cls[2], [&](auto DT, auto C0, auto C1, auto C2) {
        MOFQ_CUDA_OK(launch_chained(kq_emit_codes_uniform<DT(), C0(), C1(), C2()>, dim3(grid), dim3(256), 0, st, chained, xp, rows, cpr,
                                    (long long)x.ld, plan.es, hdr));
        return MOFQ_OK;
    });
}

// Per-channel abs-max scales; codes (and scales) of n formats from one read.  formats[i] is a mofq_format.
int launch_emit_codes_rows(const mofq_tensor &x, int n, const int *formats, void *const *codes, float *const *scales,
                           WsHeader *hdr, cudaStream_t st, bool chained)
{
    if (x.cols > (1 << 20)) return MOFQ_ERR_UNSUPPORTED;
    const size_t smem = (size_t)x.cols * 2;
    if (smem > 200 * 1024) return MOFQ_ERR_UNSUPPORTED;
    EmitPlan plan;
    if (int rc = make_emit_plan(n, formats, codes, scales, &plan)) return rc;
    if (!plan.has_kernel) {   // a class twice: one launch per format
        for (int i = 0; i < n; ++i)
            if (int rc = launch_emit_codes_rows(x, 1, formats + i, codes + i, scales ? scales + i : nullptr, hdr, st, chained || i > 0)) return rc;
        return MOFQ_OK;
    }
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    return dispatch_classes(x.dtype, plan.cls[0], plan.cls[1], plan.cls[2], [&](auto DT, auto C0, auto C1, auto C2) {
        auto kernel = kq_emit_codes_rows<DT(), C0(), C1(), C2()>;
        if (int rc = set_smem(kernel, smem)) return rc;
        const int occ = std::max(1, blocks_per_sm((const void *)kernel, kRowThreads, smem));
        const int grid = (int)std::min<long long>(x.rows, (long long)sm_count() * occ);
        MOFQ_CUDA_OK(launch_chained(kernel, dim3(grid), dim3(kRowThreads), smem, st, chained, xp, (long long)x.rows, (int)x.cols, (long long)x.ld,
                                    plan.es, hdr));
        return MOFQ_OK;
    });
}

int launch_emit(const mofq_tensor &x, const FmtDesc &f, int gran, int group, const float *scales_in, void *codes_out,
                float *scales_out, void *dequant_out, void *values_out, int values_dtype, WsHeader *hdr, cudaStream_t st,
                int format_id, const EmitSel *sel, bool overlap_prev)
{
    EmitSel es{};
    if (sel) {
        es = *sel;
        format_id = -1;  // the fused code kernel needs the format on the host
    }
    const uint16_t *xp = static_cast<const uint16_t *>(x.data);
    const int nsm = sm_count();
    if (x.cols > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
    if (gran == MOFQ_PER_CHANNEL && !scales_in && codes_out && !dequant_out && !values_out && x.cols * 2 <= 200 * 1024 &&
        format_id >= 0) {
        void *c[1] = {codes_out};
        float *sc[1] = {scales_out};
        return launch_emit_codes_rows(x, 1, &format_id, c, sc, hdr, st);
    }
    if (gran == MOFQ_PER_TENSOR && !scales_in) {
        MOFQ_CUDA_OK(cudaMemsetAsync(&hdr->absmax_bits, 0, sizeof(uint32_t), st));
        const long long total = x.rows * (x.cols / 8);
        const int grid = (int)std::min<long long>((total + 255) / 256, (long long)nsm * 8);
        if (x.dtype == MOFQ_F16)
            kq_absmax<0><<<grid, 256, 0, st>>>(xp, x.rows, (int)(x.cols / 8), x.ld, hdr);
        else
            kq_absmax<1><<<grid, 256, 0, st>>>(xp, x.rows, (int)(x.cols / 8), x.ld, hdr);
        MOFQ_CUDA_OK(cudaGetLastError());
    }
    if ((gran == MOFQ_PER_GROUP || gran == MOFQ_PER_TENSOR) && !scales_in && codes_out && !dequant_out && !values_out &&
        (gran == MOFQ_PER_GROUP || x.cols % 32 == 0)) {
        // codes + scales under abs-max scales: the register-resident team kernel
        const int width = gran == MOFQ_PER_GROUP ? group : 32;
        const int team = std::max(1, (width >> 3) / 4);
        const long long n_blocks = x.rows * (x.cols / width);
        const long long warps = (n_blocks + (32 / team) - 1) / (32 / team);
        const int g = (int)std::min<long long>((warps + 7) / 8, (long long)nsm * 8);
        // group scales, after the previous layer's launch of the same emission call: may start while that one drains
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3((unsigned)g);
        lc.blockDim = dim3(256);
        lc.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at;
        lc.numAttrs = (overlap_prev && gran == MOFQ_PER_GROUP) ? 1 : 0;
        const int uniform = gran == MOFQ_PER_TENSOR ? 1 : 0;
        if (x.dtype == MOFQ_F16)
            MOFQ_CUDA_OK(cudaLaunchKernelEx(&lc, kq_emit_blocks<0>, xp, (long long)x.rows, (int)x.cols, (long long)x.ld, f, width, uniform,
                                            (unsigned char *)codes_out, scales_out, hdr, es));
        else
            MOFQ_CUDA_OK(cudaLaunchKernelEx(&lc, kq_emit_blocks<1>, xp, (long long)x.rows, (int)x.cols, (long long)x.ld, f, width, uniform,
                                            (unsigned char *)codes_out, scales_out, hdr, es));
        return MOFQ_OK;
    }
    const int grid = (int)std::min<long long>(x.rows, (long long)nsm * 8);
#define MOFQ_EMIT(DT_, G_)                                                                                                   \
    if (x.dtype == DT_ && gran == G_) {                                                                                      \
        kq_emit<DT_, G_><<<grid, kRowThreads, 0, st>>>(xp, x.rows, (int)x.cols, x.ld, f, group, scales_in,                   \
                                                       (unsigned char *)codes_out, scales_out, (uint16_t *)dequant_out,      \
                                                       (uint16_t *)values_out, values_dtype, hdr, es);                       \
        MOFQ_CUDA_OK(cudaGetLastError());                                                                                    \
        return MOFQ_OK;                                                                                                      \
    }
    MOFQ_EMIT(0, MOFQ_PER_TENSOR) MOFQ_EMIT(0, MOFQ_PER_CHANNEL) MOFQ_EMIT(0, MOFQ_PER_GROUP)
    MOFQ_EMIT(1, MOFQ_PER_TENSOR) MOFQ_EMIT(1, MOFQ_PER_CHANNEL) MOFQ_EMIT(1, MOFQ_PER_GROUP)
#undef MOFQ_EMIT
    return MOFQ_ERR_INVALID_ARG;
}

}  // namespace mofq
