// Layer-output metric (Section 3.2, layer analysis): error of Y = X W^T when W (and X) are quantised.
//
//   reference pass : Y[t,o] = sum_i X[t,i] W[o,i]            (fp32 accumulation of the exact operands), sum Y^2
//   per format f   : Yq = a_f * s_w[o] * (A_f B_f^T),  sum (Y - Yq)^2
//                    WA     : A_f = grid values of X, B_f = grid values of W, a_f = s_x
//                    W-only : A_f = X,                B_f = grid values of W, a_f = 1
// The grid values of INT8 / E4M3 / E5M2 / INT4 / E2M1 are exactly representable in fp16 and bf16, so every
// product below is exact and only the fp32 accumulation rounds.
//
// One GEMM kernel serves all passes: tcgen05.mma (kind::f16, M=128, N=128, K=16) issued by one
// thread, operands staged by TMA (128-byte swizzle, K-major, no multicast) through a 6-stage
// shared-memory ring, two 128-column fp32 accumulators in tensor memory so that the epilogue of one
// tile overlaps the main loop of the next.  The epilogue reads the accumulator with tcgen05.ld,
// applies the scales, forms Y (stored once, fp32) or the difference to the stored Y, and reduces the
// squares; per-CTA partial sums are added in a fixed order by a small finalize kernel.
// Every mbarrier wait is bounded: on expiry the CTA records MOFQ_STATUS_TIMEOUT, frees its tensor
// memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <type_traits>

#include "mofq_internal.h"

namespace mofq {
namespace {

constexpr int BM = 128;
constexpr int kRowBytes = 128;  // bytes of K per tile row: 64 16-bit or 128 8-bit elements (one 128-byte swizzle row)
constexpr int kABytes = BM * kRowBytes;
constexpr int kRingBytes = 192 * 1024;
constexpr int kEpiWarps = 8;        // two per tensor-memory lane quarter, each on half of the tile's columns
constexpr int kStageTile = 32 * 32 * 4;  // one epilogue warp's 32 x 32 fp32 staging tile for the TMA store of Y
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;  // warp 0: TMA, warp 1: MMA + tensor-memory owner, warps 2..: epilogue
// Tile width BN is 128 or 256: the wider tile moves 25% fewer operand bytes per flop (the main loop is bound by
// L2 -> shared-memory traffic), the narrower one quantises better onto 148 SMs.  Two accumulators of BN columns.
// CG = 2: a cluster of two CTAs computes a 256 x BN tile; each CTA stages its own 128 rows of A and BN/2 rows of B
// (32 KB per k-block for BN = 256 instead of 48 KB), the leader CTA issues M = 256 MMAs that read both CTAs' shared
// memory and write both CTAs' tensor memory.
// KA = K atoms (128-byte swizzle rows) per stage: with KA = 2 one barrier wait and one commit serve 8 MMAs instead of
// 4, which halves the per-stage overhead of the issuing thread (measured: ~400 cycles per stage that tensor execution
// does not hide).
template <int BN, int CG = 1> struct TileCfg {
    static constexpr int kBRows = BN / CG;                    // rows of B staged by one CTA
    static constexpr int kBBytes = kBRows * kRowBytes;        // one K atom of B
    static constexpr int KA = (kABytes + kBBytes) <= 32 * 1024 ? 2 : 1;
    static constexpr int kStageBytes = KA * (kABytes + kBBytes);
    static constexpr int kStages = kRingBytes / kStageBytes;  // 3 (64 KB stages) or 4 (48 KB stages)
    static constexpr int kTmemCols = 2 * BN;
};
constexpr long long kWaitCycles = 4000000000LL;
constexpr int kMaxGemmCtas = 148 * 2;

// ---- PTX wrappers ----------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, int count) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count)); }
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *err)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*err || clock64() - t0 > kWaitCycles) {
            *err = 1;
            return false;
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p; }"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p; }"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// ---- two-CTA (cta_group::2) forms: a pair of CTAs in a cluster shares one 256-row MMA ----------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t mapa_u32(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion bytes are counted on the LEADER CTA's barrier (cluster address); no multicast
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, int c0, int c1, uint32_t leader_bar)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(leader_bar) : "memory");
}
// TMA store of a shared-memory box to global memory (bulk group completion), and the two waits on the group:
// "read" = the shared memory may be overwritten, full = the data is in global memory
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, const void *src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(smem_u32(src)) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void sts128(uint32_t addr, float4 v)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
// arrive on the barrier at this offset in both CTAs of the pair once the MMAs issued so far have completed
__device__ __forceinline__ void tc_commit_pair(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
template <int KIND>
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    if (KIND == 0)
        asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p; }"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    else if (KIND == 1)
        asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p; }"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p; }"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i receives row (lane base + i)
// issues the load; the data is valid after tc_ld_wait
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                   "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
                   "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                   "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
// completes every tensor-memory load this thread has issued; the registers are operands so that no use of them can
// be scheduled ahead of the wait
__device__ __forceinline__ void tc_ld_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                   "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
                   "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                   "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :
                 : "memory");
}

// Shared-memory matrix descriptor for a K-major tile whose rows are 128 bytes (64 16-bit elements) written
// by TMA with the 128-byte swizzle: 8-row atoms of 1024 bytes, stacked along M/N.
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) /* leading offset: unused with a swizzle */ |
           ((uint64_t)(1024 >> 4) << 32) /* stride between 8-row atoms */ | (1ull << 46) /* descriptor version */ |
           (2ull << 61) /* 128-byte swizzle */;
}

constexpr int kMaxProb = 3;     // products of one shape that one launch can carry (the candidates of a layer)
struct GemmParams {
    int M, N, K;              // Y is M x N, contraction over K
    int mode;                 // 0: reference (write Y, sum Y^2); 1: quantised (sum (Y - alpha*col*acc)^2)
    int n_prob;               // products in this launch; their tiles form one list, so the waves are shared
    float *Y;                 // [M, N] fp32, dense
    const float *alpha[kMaxProb];      // device scalar per product
    const float *col_scale[kMaxProb];  // device [N] or nullptr (treated as 1)
    double *partials[kMaxProb];        // one double per CTA and product
    int32_t *status;          // device status word (timeout)
    uint32_t idesc[kMaxProb];
    int kind[kMaxProb];       // operand kind of the MMA: KIND_F16 (fp16/bf16), KIND_I8 (int8 -> int32), KIND_F8 (e4m3/e5m2)
    int bk;                   // elements of K per tile row (64 or 128), the same for every product of a launch
    int y_tma;                // mode 0: Y is written by TMA stores through map_y
};
struct GemmMaps {             // operand tensor maps of the products
    CUtensorMap a[kMaxProb], b[kMaxProb];
};
enum { KIND_F16 = 0, KIND_I8 = 1, KIND_F8 = 2 };

template <int BN, int CG>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_err_kernel(const __grid_constant__ GemmMaps maps, const __grid_constant__ CUtensorMap map_y, const GemmParams p)
{
    using Cfg = TileCfg<BN, CG>;
    constexpr int kStages = Cfg::kStages, kStageBytes = Cfg::kStageBytes, kTmemCols = Cfg::kTmemCols;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages], empty_bar[kStages], tfull_bar[2], tempty_bar[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int err_flag;
    __shared__ double red[kEpiWarps][kMaxProb];
    volatile int *const perr = &err_flag;
#define err (*perr)

    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = CG == 2 ? (int)cluster_ctarank() : 0;            // 0 = leader of the pair
    const int unit = (int)blockIdx.x / CG, n_units = (int)gridDim.x / CG;  // a unit (CTA or pair) owns whole tiles
    const int tiles_m = (p.M + BM * CG - 1) / (BM * CG), tiles_n = (p.N + BN - 1) / BN;
    const int n_tiles = tiles_m * tiles_n;          // per product
    const int all_tiles = n_tiles * p.n_prob;       // the launch's tile list: product-major
    constexpr int KA = Cfg::KA;
    const int kblocks = (p.K + p.bk * KA - 1) / (p.bk * KA);  // a k-block is one stage: KA atoms of K

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tfull_bar[b], 1);
            mbar_init(&tempty_bar[b], kEpiWarps * CG);  // the epilogue warps of every CTA of the unit release the leader
        }
        err = 0;
        for (int i = 0; i < kEpiWarps; ++i)
            for (int j = 0; j < kMaxProb; ++j) red[i][j] = 0.0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // the MMA warp owns the tensor-memory allocation
        if (CG == 2) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    if (CG == 2) cluster_sync();  // the peer's barriers are initialised before anything signals them
    else __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&tmem_base_slot);
    chain_enter();   // barriers, tensor memory and descriptors are set up while the previous kernel of the call drains

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int it = 0;
            for (int gt = unit; gt < all_tiles && !err; gt += n_units) {
                const int prob = gt / n_tiles, tile = gt - prob * n_tiles;
                const CUtensorMap *map_a = &maps.a[prob], *map_b = &maps.b[prob];
                // m fastest: co-running tiles share a B tile.  This CTA's rows of A and of B inside the unit's tile:
                const int m0 = (tile % tiles_m) * BM * CG + rank * BM, n0 = (tile / tiles_m) * BN + rank * Cfg::kBRows;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % kStages;
                    if (!mbar_wait(&empty_bar[s], ((it / kStages) & 1) ^ 1, perr)) break;
                    unsigned char *st = smem + (size_t)s * kStageBytes;
                    // stage layout: KA atoms of A (16 KB each), then KA atoms of B
                    if (CG == 2) {  // both CTAs' bytes are counted on the leader's barrier
                        if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * kStageBytes);
                        const uint32_t leader_bar = mapa_u32(smem_u32(&full_bar[s]), 0);
#pragma unroll
                        for (int a = 0; a < KA; ++a) {
                            tma_load_2d_pair(st + a * kABytes, map_a, (kb * KA + a) * p.bk, m0, leader_bar);
                            tma_load_2d_pair(st + KA * kABytes + a * Cfg::kBBytes, map_b, (kb * KA + a) * p.bk, n0, leader_bar);
                        }
                    } else {
                        mbar_expect_tx(&full_bar[s], kStageBytes);
#pragma unroll
                        for (int a = 0; a < KA; ++a) {
                            tma_load_2d(st + a * kABytes, map_a, (kb * KA + a) * p.bk, m0, &full_bar[s]);
                            tma_load_2d(st + KA * kABytes + a * Cfg::kBBytes, map_b, (kb * KA + a) * p.bk, n0, &full_bar[s]);
                        }
                    }
                }
            }
            if (err && rank == 0) {  // let copies that are still in flight land before the shared memory is given back
                for (int s = 0; s < kStages; ++s) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full_bar[s], 0) && !mbar_try_wait(&full_bar[s], 1) && clock64() - t0 < kWaitCycles) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // The tensor pipe takes an MMA only when it can start it, so whatever else this thread does between MMAs is
        // a bubble: the loop is kept to a barrier wait, KA*4 MMAs whose descriptors are one 64-bit add away, a commit.
        if (lane == 0 && rank == 0) {
            const uint64_t a_desc0 = smem_desc_k_major_sw128(smem_u32(smem));
            const uint64_t b_desc0 = smem_desc_k_major_sw128(smem_u32(smem + KA * kABytes));
            int s = 0;
            uint32_t ph = 0;
            uint64_t a_desc = a_desc0, b_desc = b_desc0;  // descriptors of the current stage (address field in 16-byte units)
            // the main loop of one tile for one operand kind; false = a bounded wait expired
            auto tile_mmas = [&](auto kind_tag, uint32_t idesc, uint32_t d_tmem) -> bool {
                constexpr int KIND = decltype(kind_tag)::value;
                uint32_t acc = 0;
                for (int kb = 0; kb < kblocks; ++kb) {
                    // (no tcgen05 fence here: the mbarrier orders the TMA data for the MMAs)
                    if (!mbar_wait(&full_bar[s], ph, perr)) return false;
#pragma unroll
                    for (int k = 0; k < KA * (kRowBytes / 32); ++k) {  // one MMA consumes 32 bytes of K
                        constexpr int per = kRowBytes / 32;
                        const uint64_t ad = a_desc + (uint64_t)((k / per) * (kABytes >> 4) + 2 * (k % per));
                        const uint64_t bd = b_desc + (uint64_t)((k / per) * (Cfg::kBBytes >> 4) + 2 * (k % per));
                        if (CG == 2) tc_mma_pair<KIND>(d_tmem, ad, bd, idesc, acc);
                        else if (KIND == KIND_F16) tc_mma_f16(d_tmem, ad, bd, idesc, acc);
                        else if (KIND == KIND_I8) tc_mma_i8(d_tmem, ad, bd, idesc, acc);
                        else tc_mma_f8(d_tmem, ad, bd, idesc, acc);
                        acc = 1;
                    }
                    // the stage is free (in every CTA of the unit) once these MMAs have read it
                    if (CG == 2) tc_commit_pair(&empty_bar[s]);
                    else tc_commit(&empty_bar[s]);
                    if (++s == kStages) {
                        s = 0;
                        ph ^= 1u;
                        a_desc = a_desc0;
                        b_desc = b_desc0;
                    } else {
                        a_desc += (uint64_t)(kStageBytes >> 4);
                        b_desc += (uint64_t)(kStageBytes >> 4);
                    }
                }
                return true;
            };
            int local = 0;
            for (int gt = unit; gt < all_tiles && !err; gt += n_units, ++local) {
                const int prob = gt / n_tiles;
                const int buf = local & 1;
                if (!mbar_wait(&tempty_bar[buf], ((local >> 1) & 1) ^ 1, perr)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                const uint32_t idesc = p.idesc[prob];
                const int kind = p.kind[prob];
                const bool ok = kind == KIND_F16  ? tile_mmas(std::integral_constant<int, KIND_F16>(), idesc, d_tmem)
                                : kind == KIND_I8 ? tile_mmas(std::integral_constant<int, KIND_I8>(), idesc, d_tmem)
                                                  : tile_mmas(std::integral_constant<int, KIND_F8>(), idesc, d_tmem);
                if (!ok) break;
                if (CG == 2) tc_commit_pair(&tfull_bar[buf]);  // accumulator complete
                else tc_commit(&tfull_bar[buf]);
            }
        }
    } else {
        // ---------------- epilogue: warps 2..5 read the lane quarter (warp % 4) of the accumulator ----------------
        // The epilogue is bound by the latency of its tensor-memory and global loads, not by arithmetic: eight warps
        // keep twice as many of them in flight as four would.
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;                 // which half of the tile's columns this warp handles
        constexpr int kChunks = BN / 32 / (kEpiWarps / 4);
        const uint32_t stage = smem_u32(smem + kRingBytes + (warp - 2) * kStageTile);
        double dsum0 = 0.0, dsum1 = 0.0, dsum2 = 0.0;    // one running sum per product
        int local = 0;
        for (int gt = unit; gt < all_tiles; gt += n_units, ++local) {
            const int prob = gt / n_tiles, tile = gt - prob * n_tiles;
            const float alpha = __ldg(p.alpha[prob]);
            const float *col_scale = p.col_scale[prob];
            const int kind = p.kind[prob];
            const int buf = local & 1;
            const int m0 = (tile % tiles_m) * BM * CG + rank * BM, n0 = (tile / tiles_m) * BN;
            const int row = m0 + q * 32 + lane;
            float fsum = 0.0f;
            // the stored Y of the next 32-column chunk is fetched while the current chunk is processed; the first
            // chunk's is requested before the accumulator is waited for
            const bool vec = (p.N & 3) == 0;
            float4 ycur[8], ynext[8];
            auto prefetch_y = [&](int c, float4 (&y)[8]) {
                const int pc0 = n0 + c * 32;
                if (p.mode == 1 && row < p.M && vec && pc0 + 32 <= p.N) {
                    const float4 *src = reinterpret_cast<const float4 *>(p.Y + (size_t)row * p.N + pc0);
#pragma unroll
                    for (int j = 0; j < 8; ++j) y[j] = __ldg(src + j);
                }
            };
            prefetch_y(half * kChunks, ycur);
            if (!mbar_wait(&tfull_bar[buf], (local >> 1) & 1, perr)) break;
            tc_fence_after();
            // two register sets: the tensor-memory load of chunk c+1 is in flight while chunk c is processed
            uint32_t ra[32], rb[32];
            const uint32_t t0 = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN);
            tc_ld_32x32(t0 + (uint32_t)(half * kChunks * 32), ra);
#pragma unroll
            for (int ci = 0; ci < kChunks; ++ci) {
                const int c = half * kChunks + ci;
                uint32_t(&r)[32] = (ci & 1) ? rb : ra;
                uint32_t(&rn)[32] = (ci & 1) ? ra : rb;
                if (ci + 1 < kChunks) prefetch_y(c + 1, ynext);
                tc_ld_wait(r);
                if (ci + 1 < kChunks) tc_ld_32x32(t0 + (uint32_t)((c + 1) * 32), rn);
                const int col0 = n0 + c * 32;
                if (kind == KIND_I8) {  // exact integer dot products -> float
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint((float)(int)r[j]);
                }
                if (p.mode == 0 && p.y_tma) {
                    // Y leaves through shared memory: each thread's 32 values go into the warp's 32 x 32 staging tile
                    // in the 128-byte-swizzle layout (conflict-free 16-byte stores), one TMA store writes the tile
                    // as full rows and clips what lies beyond M or N
                    if (lane == 0) tma_store_wait_read();   // the previous chunk's store has read the tile
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float4 v;
                        v.x = __uint_as_float(r[j]) * alpha;
                        v.y = __uint_as_float(r[j + 1]) * alpha;
                        v.z = __uint_as_float(r[j + 2]) * alpha;
                        v.w = __uint_as_float(r[j + 3]) * alpha;
                        sts128(stage + (uint32_t)(lane * 128 + (((j >> 2) ^ (lane & 7)) << 4)), v);
                        if (row < p.M) {
                            if (col0 + j < p.N) fsum = fmaf(v.x, v.x, fsum);
                            if (col0 + j + 1 < p.N) fsum = fmaf(v.y, v.y, fsum);
                            if (col0 + j + 2 < p.N) fsum = fmaf(v.z, v.z, fsum);
                            if (col0 + j + 3 < p.N) fsum = fmaf(v.w, v.w, fsum);
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && col0 < p.N && m0 + q * 32 < p.M) tma_store_2d(&map_y, smem + kRingBytes + (warp - 2) * kStageTile, col0, m0 + q * 32);
                } else if (row < p.M) {
                    float *yrow = p.Y + (size_t)row * p.N + col0;
                    if (col0 + 32 <= p.N && vec) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 v;
                            if (p.mode == 0) {
                                v.x = __uint_as_float(r[j]) * alpha;
                                v.y = __uint_as_float(r[j + 1]) * alpha;
                                v.z = __uint_as_float(r[j + 2]) * alpha;
                                v.w = __uint_as_float(r[j + 3]) * alpha;
                                *reinterpret_cast<float4 *>(yrow + j) = v;
                                fsum = fmaf(v.x, v.x, fsum);
                                fsum = fmaf(v.y, v.y, fsum);
                                fsum = fmaf(v.z, v.z, fsum);
                                fsum = fmaf(v.w, v.w, fsum);
                            } else {
                                const float4 y = ycur[j >> 2];
                                float4 cs = make_float4(1.f, 1.f, 1.f, 1.f);
                                if (col_scale) cs = __ldg(reinterpret_cast<const float4 *>(col_scale + col0 + j));
                                const float d0 = y.x - __uint_as_float(r[j]) * (alpha * cs.x);
                                const float d1 = y.y - __uint_as_float(r[j + 1]) * (alpha * cs.y);
                                const float d2 = y.z - __uint_as_float(r[j + 2]) * (alpha * cs.z);
                                const float d3 = y.w - __uint_as_float(r[j + 3]) * (alpha * cs.w);
                                fsum = fmaf(d0, d0, fsum);
                                fsum = fmaf(d1, d1, fsum);
                                fsum = fmaf(d2, d2, fsum);
                                fsum = fmaf(d3, d3, fsum);
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {  // ragged right edge (static indices keep r in registers)
                            if (col0 + j >= p.N) continue;
                            const float a = __uint_as_float(r[j]);
                            if (p.mode == 0) {
                                const float v = a * alpha;
                                yrow[j] = v;
                                fsum = fmaf(v, v, fsum);
                            } else {
                                const float cs = col_scale ? col_scale[col0 + j] : 1.0f;
                                const float d = yrow[j] - a * (alpha * cs);
                                fsum = fmaf(d, d, fsum);
                            }
                        }
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) ycur[j] = ynext[j];
            }
            if (prob == 0) dsum0 += (double)fsum;
            else if (prob == 1) dsum1 += (double)fsum;
            else dsum2 += (double)fsum;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 2 && rank != 0) mbar_arrive_cluster(mapa_u32(smem_u32(&tempty_bar[buf]), 0));
                else mbar_arrive(&tempty_bar[buf]);
            }
        }
        if (p.mode == 0 && p.y_tma && lane == 0) tma_store_wait_all();   // Y is in global memory before the block leaves
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            dsum0 += __shfl_xor_sync(0xffffffffu, dsum0, o);
            dsum1 += __shfl_xor_sync(0xffffffffu, dsum1, o);
            dsum2 += __shfl_xor_sync(0xffffffffu, dsum2, o);
        }
        if (lane == 0) {
            red[warp - 2][0] = dsum0;
            red[warp - 2][1] = dsum1;
            red[warp - 2][2] = dsum2;
        }
    }
    tc_fence_before();
    if (CG == 2) cluster_sync();  // no CTA leaves while its peer may still touch its shared or tensor memory
    else __syncthreads();
    if (threadIdx.x == 0) {
        for (int j = 0; j < p.n_prob; ++j) {
            double tot = 0.0;
            for (int i = 0; i < kEpiWarps; ++i) tot += red[i][j];
            p.partials[j][blockIdx.x] = tot;
        }
        if (err) atomicOr(p.status, MOFQ_STATUS_TIMEOUT);
    }
    if (warp == 1) {
        tc_fence_after();
        if (CG == 2) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
#undef err
}

// ---- helper kernels -------------------------------------------------------------------------------------------
// bf16 activations -> fp16 operand: scaled by the power of two that puts the tensor's abs-max in [2^13, 2^14), which
// keeps every bf16 value exact in fp16 unless it is more than 2^27 times smaller than the abs-max.
__global__ void __launch_bounds__(256)
x_bf16_to_f16(const uint16_t *__restrict__ x, long long rows, int cols, long long ld, const WsHeader *hdr, uint16_t *out, float *alpha_out)
{
    chain_enter();
    const uint32_t m16 = hdr->absmax_bits;
    const int e = (int)(m16 >> 7) - 127;  // bf16 exponent of the abs-max (0 -> treated as tiny)
    const int pw = m16 ? 13 - e : 0;
    const float mult = exp2f((float)max(min(pw, 126), -126));
    if (blockIdx.x == 0 && threadIdx.x == 0) *alpha_out = exp2f((float)-max(min(pw, 126), -126));
    const int cpr = cols >> 3;
    const long long total = rows * cpr;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / cpr;
        const int c = (int)(i - r * cpr);
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(x + r * ld) + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = __uint_as_float(w[k] << 16) * mult, hi = __uint_as_float(w[k] & 0xFFFF0000u) * mult;
            o[k] = (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
        }
        *reinterpret_cast<uint4 *>(out + r * cols + (long long)c * 8) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

__global__ void set_scalar(float *p, float v)
{
    chain_enter();
    *p = v;
}

struct LayerFinalize {
    const double *partials;  // [(1 + n_cand)][stride]
    int stride, n_cand;
    int n_ctas[1 + MOFQ_MAX_CAND];  // blocks that wrote each entry's partial sums (launch grids can differ)
    double inv_n;
    mofq_result *res;
    float *mse_out, *nsr_out;
    int32_t *status;         // device status word: cleared after it is read when a record is written
    uint32_t *absmax_bits;   // the header's activation abs-max: left zero for the next layer of the call
};

// Warp k adds entry k's partial sums (the reference's, then one per candidate) in a fixed order: lane l takes blocks
// l, l + 32, ..., eight of them fetched per trip, then the lanes' sums are folded.
constexpr int kFinalizeThreads = 32 * (1 + MOFQ_MAX_CAND);
__global__ void __launch_bounds__(kFinalizeThreads)
layer_finalize(const LayerFinalize f)
{
    chain_enter();
    __shared__ double tot[1 + MOFQ_MAX_CAND];
    const int k = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) *f.absmax_bits = 0;
    if (k <= f.n_cand) {
        double s = 0.0;
        for (int c0 = lane; c0 < f.n_ctas[k]; c0 += 32 * 8) {
            double v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = c0 + 32 * j < f.n_ctas[k] ? __ldcg(&f.partials[(size_t)k * f.stride + c0 + 32 * j]) : 0.0;
#pragma unroll
            for (int j = 0; j < 8; ++j) s += v[j];
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) tot[k] = s;
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    double best = INFINITY, second = INFINITY;
    int chosen = -1;
    mofq_result r;
    for (int i = 0; i < MOFQ_MAX_CAND; ++i) r.error[i] = r.nsr[i] = 0.0f;
    for (int i = 0; i < f.n_cand; ++i) {
        const double mse = tot[1 + i] * f.inv_n, nsr = tot[0] > 0.0 ? tot[1 + i] / tot[0] : 0.0;
        r.error[i] = (float)mse;
        r.nsr[i] = (float)nsr;
        if (f.mse_out) f.mse_out[i] = (float)mse;
        if (f.nsr_out) f.nsr_out[i] = (float)nsr;
        // Algorithm 1: strict '<' in the caller's candidate order
        if (mse < best) {
            second = best;
            best = mse;
            chosen = i;
        } else if (mse < second) {
            second = mse;
        }
    }
    if (f.res) {
        r.chosen = chosen;
        r.status = atomicExch(f.status, 0);
        r.rel_margin = best > 0.0 ? (float)((second - best) / best) : INFINITY;
        r.reserved = 0;
        *f.res = r;
    }
}

// ---- host side ---------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [rows, cols] 16-bit row-major tensor with leading dimension ld -> map with a {BK, box_rows} box and the 128-byte swizzle
// elem: MOFQ_F16, MOFQ_BF16 or kElemU8
constexpr int kElemU8 = 2;
int make_map(CUtensorMap *map, const void *base, int elem, long long rows, long long cols, long long ld, int box_rows)
{
    EncodeTiledFn fn = encode_tiled();
    if (!fn) return MOFQ_ERR_CUDA;
    const int esize = elem == kElemU8 ? 1 : 2;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * esize};
    const cuuint32_t box[2] = {(cuuint32_t)(kRowBytes / esize), (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = elem == kElemU8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                   : elem == MOFQ_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult rc = fn(map, dt, 2,
                           const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? MOFQ_OK : MOFQ_ERR_CUDA;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// Workspace of the layer metric, after the scoring workspace:
struct LayerWs {
    size_t x16, cx, cw, y, sw, scal, partials, total;
};
LayerWs layer_ws_layout(long long T, long long n_in, long long n_out)
{
    LayerWs w{};
    size_t off = 0;
    w.x16 = off; off += align256((size_t)T * n_in * 2);
    w.cx = off;  off += 3 * align256((size_t)T * n_in);        // 8-bit codes of up to 3 formats, or 16-bit values of one
    w.cw = off;  off += 3 * align256((size_t)n_out * n_in);   // 8-bit codes of up to 3 formats, or 16-bit values of one
    w.y = off;   off += align256((size_t)T * n_out * 4);
    w.sw = off;  off += 3 * align256((size_t)n_out * 4);
    w.scal = off; off += 256;  // [0] reference alpha, [1] activation scale of the current format
    w.partials = off; off += align256(sizeof(double) * (1 + MOFQ_MAX_CAND) * kMaxGemmCtas);
    w.total = off;
    return w;
}

// op: MOFQ_F16 / MOFQ_BF16 (16-bit operands), or an 8-bit mofq_format (MOFQ_INT8, MOFQ_FP8_E4M3, MOFQ_FP8_E5M2) + 100
constexpr int kOp8 = 100;
// One launch over n products of the same shape (the candidates of a layer): their tiles form one list, so the last
// wave is shared instead of paid once per product.  n = 1 for the reference pass.
int run_gemm_n(int n, const void *const *a, long long a_rows, const long long *a_ld, const void *const *b, long long b_rows,
               long long b_ld, long long K, const int *op, int mode, float *Y, const float *const *alpha,
               const float *const *col_scale, double *const *partials, int32_t *status, int *grid_out, cudaStream_t st,
               bool chained = false)
{
    if (n < 1 || n > kMaxProb) return MOFQ_ERR_INVALID_ARG;
    // tile shape: waves x relative tile cost.  Operand bytes per CTA and k-block: 32 KB for a 128x128 tile, 48 KB for
    // 128x256, and 32 KB per CTA for a CTA pair sharing a 256x256 tile (cost per 128x128 of output: 1, 0.75, 0.5).
    const int nsm = sm_count();
    const long long mt = (a_rows + BM - 1) / BM;
    const long long t128 = n * mt * ((b_rows + 127) / 128), t256 = n * mt * ((b_rows + 255) / 256);
    const long long tpair = n * ((a_rows + 2 * BM - 1) / (2 * BM)) * ((b_rows + 255) / 256);
    const int npair = std::max(1, nsm / 2);
    const double c128 = (double)((t128 + nsm - 1) / nsm) * 1.0, c256 = (double)((t256 + nsm - 1) / nsm) * 1.5;
    const double cpair = (double)((tpair + npair - 1) / npair) * 1.0;
    const int cg = cpair < std::min(c128, c256) ? 2 : 1;
    const int bn = cg == 2 ? 256 : (c256 < c128 ? 256 : 128);
    GemmMaps maps;
    GemmParams p{};
    p.n_prob = n;
    for (int i = 0; i < kMaxProb; ++i) {
        const int j = i < n ? i : 0;  // unused slots repeat product 0 so that every map is a valid object
        const int elem = op[j] >= kOp8 ? kElemU8 : op[j];
        if ((op[j] >= kOp8) != (op[0] >= kOp8)) return MOFQ_ERR_INVALID_ARG;  // one K-atom width per launch
        if (int rc = make_map(&maps.a[i], a[j], elem, a_rows, K, a_ld[j], BM)) return rc;
        if (int rc = make_map(&maps.b[i], b[j], elem, b_rows, K, b_ld, bn / cg)) return rc;
        p.alpha[i] = alpha[j];
        p.col_scale[i] = col_scale[j];
        p.partials[i] = partials[j];
        // instruction descriptor: accumulator type [4,6), A type [7,10), B type [10,13), both K-major, N/8 at [17,23), M/16 at [24,29)
        uint32_t cfmt, abfmt;
        if (op[j] == kOp8 + MOFQ_INT8) {
            p.kind[i] = KIND_I8; cfmt = 2u /* s32 */; abfmt = 1u /* signed 8-bit */;
        } else if (op[j] >= kOp8) {
            p.kind[i] = KIND_F8; cfmt = 1u /* f32 */; abfmt = op[j] == kOp8 + MOFQ_FP8_E4M3 ? 0u : 1u /* e4m3 : e5m2 */;
        } else {
            p.kind[i] = KIND_F16; cfmt = 1u; abfmt = op[j] == MOFQ_F16 ? 0u : 1u /* f16 : bf16 */;
        }
        p.idesc[i] = (cfmt << 4) | (abfmt << 7) | (abfmt << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)((BM * cg) >> 4) << 24);
    }
    const CUtensorMap &map_a = maps.a[0];
    p.M = (int)a_rows;
    p.N = (int)b_rows;
    p.K = (int)K;
    p.mode = mode;
    p.Y = Y;
    p.status = status;
    p.bk = op[0] >= kOp8 ? kRowBytes : kRowBytes / 2;
    const int tiles = cg == 2 ? (int)tpair : (int)(n * ((a_rows + BM - 1) / BM) * ((b_rows + bn - 1) / bn));
    const int grid = cg * std::min(tiles, std::min(nsm, kMaxGemmCtas) / cg);
    // the staging tiles are only needed (and only touched) by the reference pass; the candidate passes keep the
    // smaller request so that more of the SM's unified memory stays level-1 cache for their reads of Y
    const size_t smem = (size_t)kRingBytes + (mode == 0 ? (size_t)kEpiWarps * kStageTile : 0) + 1024;
    // the reference pass stores Y through a tensor map (fp32, 32 x 32 boxes, 128-byte swizzle) when its rows are 16-byte multiples
    CUtensorMap map_y = map_a;
    p.y_tma = 0;
    if (p.mode == 0 && (p.N & 3) == 0 && (reinterpret_cast<uintptr_t>(p.Y) & 15) == 0) {
        EncodeTiledFn fn = encode_tiled();
        if (!fn) return MOFQ_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)p.N, (cuuint64_t)p.M};
        const cuuint64_t strides[1] = {(cuuint64_t)p.N * 4};
        const cuuint32_t box[2] = {32, 32};
        const cuuint32_t estr[2] = {1, 1};
        if (fn(&map_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, p.Y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return MOFQ_ERR_CUDA;
        p.y_tma = 1;
    }
    auto launch = [&](auto kernel) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return MOFQ_ERR_CUDA;
        }
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3((unsigned)grid);
        lc.blockDim = dim3(kGemmThreads);
        lc.dynamicSmemBytes = smem;
        lc.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cg;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see chain_enter()
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = chained ? 2 : 1;
        if (cudaLaunchKernelEx(&lc, kernel, maps, map_y, p) != cudaSuccess) {
            (void)cudaGetLastError();
            return MOFQ_ERR_CUDA;
        }
        return MOFQ_OK;
    };
    if (int rc = cg == 2 ? launch(gemm_err_kernel<256, 2>)
                         : (bn == 256 ? launch(gemm_err_kernel<256, 1>) : launch(gemm_err_kernel<128, 1>)))
        return rc;
    *grid_out = grid;
    return MOFQ_OK;
}

int run_gemm(const void *a, long long a_rows, long long a_ld, const void *b, long long b_rows, long long b_ld, long long K,
             int op, int mode, float *Y, const float *alpha, const float *col_scale, double *partials, int32_t *status,
             int *grid_out, cudaStream_t st, bool chained = false)
{
    return run_gemm_n(1, &a, a_rows, &a_ld, &b, b_rows, b_ld, K, &op, mode, Y, &alpha, &col_scale, &partials, status, grid_out, st, chained);
}

}  // namespace

size_t layer_metric_ws_bytes(const mofq_layer *layers, int n_layers, const mofq_config *)
{
    size_t need = 0;
    for (int i = 0; i < n_layers; ++i)
        need = std::max(need, layer_ws_layout(layers[i].X.rows, layers[i].W.cols, layers[i].W.rows).total);
    return need;
}

int layer_metric_check(const mofq_layer &L, const mofq_config *cfg)
{
    const mofq_tensor &W = L.W, &X = L.X;
    if (X.cols != W.cols) return MOFQ_ERR_INVALID_ARG;
    if (cfg->w_gran != MOFQ_PER_CHANNEL) return MOFQ_ERR_UNSUPPORTED;               // scales must factor out of the contraction
    if (!cfg->is_w_only && cfg->a_gran != MOFQ_PER_TENSOR) return MOFQ_ERR_UNSUPPORTED;
    if (X.dtype == MOFQ_F16 && W.dtype == MOFQ_BF16) return MOFQ_ERR_UNSUPPORTED;    // no exact common 16-bit operand type
    if (W.rows > 0x7fffffffLL || X.rows > 0x7fffffffLL || W.cols > 0x7fffffffLL) return MOFQ_ERR_UNSUPPORTED;
    if (!cfg->is_w_only && cfg->bit_width == 8 && W.cols * 2 > 200 * 1024) return MOFQ_ERR_UNSUPPORTED;  // the code emission stages a weight row in shared memory
    for (int i = 0; i < cfg->n_candidates; ++i) {
        FmtDesc fd;
        if (!describe_format(cfg->candidates[i], &fd)) return MOFQ_ERR_INVALID_ARG;
        if (fd.bits != cfg->bit_width) return MOFQ_ERR_UNSUPPORTED;
    }
    return MOFQ_OK;
}

int layer_metric_run(const mofq_layer &L, const mofq_config *cfg, mofq_result *res, float *mse_out, float *nsr_out,
                     void *workspace, size_t workspace_bytes, cudaStream_t st, bool after_own)
{
    const mofq_tensor &W = L.W, &X = L.X;
    if (int rc = layer_metric_check(L, cfg)) return rc;
    FmtDesc fd[MOFQ_MAX_CAND];
    for (int i = 0; i < cfg->n_candidates; ++i) describe_format(cfg->candidates[i], &fd[i]);
    const long long T = X.rows, n_in = W.cols, n_out = W.rows;
    const LayerWs lw = layer_ws_layout(T, n_in, n_out);
    const size_t base_off = align256(score_ws_bytes());
    if (workspace_bytes < base_off + lw.total) return MOFQ_ERR_WORKSPACE_TOO_SMALL;
    char *base = static_cast<char *>(workspace) + base_off;
    WsHeader *hdr = static_cast<WsHeader *>(workspace);
    uint16_t *x16 = reinterpret_cast<uint16_t *>(base + lw.x16), *cx = reinterpret_cast<uint16_t *>(base + lw.cx);
    uint16_t *cw = reinterpret_cast<uint16_t *>(base + lw.cw);
    float *Y = reinterpret_cast<float *>(base + lw.y), *sw = reinterpret_cast<float *>(base + lw.sw);
    float *scal = reinterpret_cast<float *>(base + lw.scal);
    double *partials = reinterpret_cast<double *>(base + lw.partials);
    const int op_dtype = W.dtype;  // operand type of every GEMM of this layer

    // reference operand for X (and its abs-max, which also serves the per-tensor activation scale)
    const void *xa = X.data;
    long long xa_ld = X.ld;
    const bool native8 = !cfg->is_w_only && cfg->bit_width == 8 && (n_in % 16) == 0;
    const bool fused = native8 && cfg->n_candidates <= 3;
    // The header's abs-max word is zero here: the entry points clear the header and every layer's finalize kernel leaves
    // the word zero again.  Kernels of this layer after the first, and the first one after another layer of the same
    // call, are chained launches (see chain_enter()).
    bool chained = after_own;
    if (X.dtype != op_dtype || fused) {  // one abs-max of X serves the exact fp16 copy and the per-tensor activation scales
        if (int rc = launch_absmax(X, hdr, st, chained)) return rc;
        chained = true;
    }
    const bool x16_with_codes = fused && X.dtype == MOFQ_BF16 && op_dtype == MOFQ_F16;   // written by the code-emission kernel below
    if (X.dtype != op_dtype) {  // bf16 activations with fp16 weights
        if (!x16_with_codes) {
            const long long total = T * (n_in / 8);
            const int grid = (int)std::min<long long>((total + 255) / 256, (long long)sm_count() * 8);
            if (launch_chained(x_bf16_to_f16, dim3(grid), dim3(256), 0, st, chained, static_cast<const uint16_t *>(X.data), T, (int)n_in,
                               (long long)X.ld, (const WsHeader *)hdr, x16, scal) != cudaSuccess) {
                (void)cudaGetLastError();
                return MOFQ_ERR_CUDA;
            }
            chained = true;
        }
        xa = x16;
        xa_ld = n_in;
    } else {
        if (launch_chained(set_scalar, dim3(1), dim3(1), 0, st, chained, scal, 1.0f) != cudaSuccess) {
            (void)cudaGetLastError();
            return MOFQ_ERR_CUDA;
        }
        chained = true;
    }
    // WA with 8-bit candidates: the codes themselves are the tensor-core operands (int8 / e4m3 / e5m2 kinds)
    // native path: the codes of every candidate from one read of W (one byte per element and format)
    const bool fused_w = fused;
    const size_t cx_stride = align256((size_t)T * n_in);
    const size_t cw_stride = align256((size_t)n_out * n_in), sw_stride = align256((size_t)n_out * 4) / 4;
    if (fused_w) {
        void *cptr[3];
        float *sptr[3];
        int fmts[3];
        for (int i = 0; i < cfg->n_candidates; ++i) {
            cptr[i] = reinterpret_cast<unsigned char *>(cw) + (size_t)i * cw_stride;
            sptr[i] = sw + (size_t)i * sw_stride;
            fmts[i] = cfg->candidates[i];
        }
        if (int rc = launch_emit_codes_rows(W, cfg->n_candidates, fmts, cptr, sptr, hdr, st, chained)) return rc;
        chained = true;
        for (int i = 0; i < cfg->n_candidates; ++i) {  // activations: codes of every candidate, scales in scal[1 + i]
            cptr[i] = reinterpret_cast<unsigned char *>(cx) + (size_t)i * cx_stride;
            sptr[i] = scal + 1 + i;
        }
        // the same read of X also leaves its binary16 copy for the reference product
        if (int rc = launch_emit_codes_uniform(X, cfg->n_candidates, fmts, cptr, sptr, hdr, st, x16_with_codes ? x16 : nullptr,
                                               x16_with_codes ? scal : nullptr, chained))
            return rc;
    }
    int grid_used = 0;
    int grids[1 + MOFQ_MAX_CAND] = {0};
    if (int rc = run_gemm(xa, T, xa_ld, W.data, n_out, W.ld, n_in, op_dtype, 0, Y, scal, nullptr, partials, &hdr->status, &grid_used, st, chained))
        return rc;
    chained = true;
    grids[0] = grid_used;
    if (fused && cfg->n_candidates <= kMaxProb) {
        // every candidate's operands exist already: one launch carries all their products (Algorithm 1's loop over the
        // formats becomes the product index of the tile list), so the partly filled last wave is paid once
        const void *ga[kMaxProb], *gb[kMaxProb];
        long long gld[kMaxProb];
        int gop[kMaxProb];
        const float *galpha[kMaxProb], *gcs[kMaxProb];
        double *gpart[kMaxProb];
        for (int i = 0; i < cfg->n_candidates; ++i) {
            ga[i] = reinterpret_cast<unsigned char *>(cx) + (size_t)i * cx_stride;
            gb[i] = reinterpret_cast<unsigned char *>(cw) + (size_t)i * cw_stride;
            gld[i] = n_in;
            gop[i] = kOp8 + cfg->candidates[i];
            galpha[i] = scal + 1 + i;
            gcs[i] = sw + (size_t)i * sw_stride;
            gpart[i] = partials + (size_t)(1 + i) * kMaxGemmCtas;
        }
        if (int rc = run_gemm_n(cfg->n_candidates, ga, T, gld, gb, n_out, n_in, n_in, gop, 1, Y, galpha, gcs, gpart, &hdr->status,
                                &grid_used, st, true))
            return rc;
        for (int i = 0; i < cfg->n_candidates; ++i) grids[1 + i] = grid_used;
    } else {
    for (int i = 0; i < cfg->n_candidates; ++i) {  // Algorithm 1: for format in format_candidates
        const void *bw = cw;
        const float *bsw = sw;
        if (fused_w) {
            bw = reinterpret_cast<unsigned char *>(cw) + (size_t)i * cw_stride;
            bsw = sw + (size_t)i * sw_stride;
        } else if (int rc = launch_emit(W, fd[i], MOFQ_PER_CHANNEL, 0, nullptr, native8 ? cw : nullptr, sw, nullptr,
                                        native8 ? nullptr : cw, op_dtype, hdr, st))
            return rc;
        const void *a = xa;
        long long a_ld = xa_ld;
        const float *alpha = scal;
        if (fused) {
            a = reinterpret_cast<unsigned char *>(cx) + (size_t)i * cx_stride;
            a_ld = n_in;
            alpha = scal + 1 + i;
        } else if (!cfg->is_w_only) {
            if (int rc = launch_emit(X, fd[i], MOFQ_PER_TENSOR, 0, nullptr, native8 ? cx : nullptr, scal + 1, nullptr,
                                     native8 ? nullptr : cx, op_dtype, hdr, st))
                return rc;
            a = cx;
            a_ld = n_in;
            alpha = scal + 1;
        }
        const int op = native8 ? kOp8 + cfg->candidates[i] : op_dtype;
        if (int rc = run_gemm(a, T, a_ld, bw, n_out, n_in, n_in, op, 1, Y, alpha, bsw, partials + (size_t)(1 + i) * kMaxGemmCtas,
                              &hdr->status, &grid_used, st))
            return rc;
        grids[1 + i] = grid_used;
    }
    }
    LayerFinalize f{};
    f.partials = partials;
    f.stride = kMaxGemmCtas;
    for (int k = 0; k <= cfg->n_candidates; ++k) f.n_ctas[k] = grids[k];
    f.n_cand = cfg->n_candidates;
    f.inv_n = 1.0 / ((double)T * (double)n_out);
    f.res = res;
    f.mse_out = mse_out;
    f.nsr_out = nsr_out;
    f.status = &hdr->status;
    f.absmax_bits = &hdr->absmax_bits;
    // (after the per-candidate loop of the general path the previous launch may be a memset-preceded kernel of the
    // emission path: a chained launch behind a kernel that never signals simply starts when that kernel has finished)
    if (launch_chained(layer_finalize, dim3(1), dim3(kFinalizeThreads), 0, st, true, f) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    return MOFQ_OK;
}

}  // namespace mofq
