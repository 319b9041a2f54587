// Persistent scoring kernel for per-channel scales (optionally group-128 scales from the same read): one launch
// scores every layer of a model, or one tensor.
//
// Section 3.2 quantises weights with one scale per output channel, so every element of a row waits for the row's
// abs-max.  Work = the concatenation of all layers' tiles; a tile is a few WHOLE rows (at most 72 KB), so that a
// row's abs-max is complete as soon as its tile is in shared memory.  One CTA per SM owns a contiguous range of
// tiles, balanced by bytes.  A producer warp streams tiles into a shared-memory ring with bulk asynchronous copies
// (TMA, 1-D) that complete on mbarriers.  The consumer warps work in "rounds" of 32 consecutive 128-element
// segments, one segment per lane:
//   pass 1 of a tile: abs-max of the lane's segment -> segmax[stage][segment], folded into rowmax[stage][row];
//   pass 2 of a tile: scales from rowmax (and segmax when group scales are scored too), then every candidate's
//                     squared error from one walk over the segment's 16-byte chunks.
// Pass 1 runs one tile AHEAD of pass 2, so the "every warp has finished pass 1 of this tile" barrier has normally
// completed long before anyone waits on it, and the copies of the tiles after that are in flight meanwhile (the ring
// holds three to six tiles, depending on the layer's tile size).  Rounds are dealt to the warps round-robin over the CTA's whole tile sequence (a fixed function
// of the launch geometry, so sums are formed in the same order on every run), which keeps all lanes busy whatever
// the number of segments per tile.  Per (layer, CTA, warp) partial sums go to the workspace and are added in slot
// order: by a small finalize kernel for a layer list, by the last CTA to finish for a single tensor.
// Every wait is bounded; on expiry the CTA records MOFQ_STATUS_TIMEOUT and drains.
// The arithmetic per element is the packed scorer of kq_math.cuh in its scaled form (see mofq_kq_mt.cu).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <utility>
#include <vector>

#include "kq_finish.cuh"
#include "kq_math.cuh"
#include "kq_pipe.cuh"
#include "mofq_internal.h"

namespace mofq {
namespace {

using namespace kqmath;
using namespace kqpipe;

constexpr int kRmConsumerWarps = 12;                       // warps 0..11: pass 2 (scoring), three per scheduler
constexpr int kRmScoutWarps = 4;                           // warps 12..15: pass 1 (abs-max), one per scheduler
constexpr int kRmThreads = (kRmConsumerWarps + kRmScoutWarps + 1) * 32;    // + the producer warp
constexpr int kRmTileCap = 70 * 1024;                      // most bytes of one tile (two rows of 17920 fp16)
constexpr int kRmMaxSeg = kRmTileCap / 256;                // segments (= most rows) of one tile
constexpr int kRmSlots = 6;                                // tiles in flight: barrier sets and per-tile tables
constexpr int kRmRingBytes = 3 * kRmTileCap;               // shared-memory ring: 3 tiles of 70 KB, 5 of 40 KB, 6 of <= 35 KB
constexpr int kRmSlotMeta = 2 * kRmMaxSeg * 4;             // per slot: abs-max pattern of every segment and of every row
constexpr int kRmSmemBytes = kRmRingBytes + kRmSlots * kRmSlotMeta + 1024;   // + slack to align the ring

// One layer of the work table (device memory, or inline in the parameters for a single tensor).
struct RmLayer {
    const uint16_t *x;
    long long rows, ld;
    long long tile_begin;     // index of the layer's first tile in the concatenated tile list
    long long w_begin;        // segments before this layer in the concatenated list (the balancing weight)
    long long n_tiles;
    double inv_n;             // 1 / element count
    int cols;                 // elements per row: a multiple of 128
    int rows_per_tile;
    int segs_per_row;
    uint32_t row_magic;       // segment index -> row within the tile: (q * row_magic) >> 16
    int stage_bytes, stages;  // how this layer's tiles divide the ring
    int first_cta, n_slots, slot_off, pad;
};

struct RmTileInfo {           // what the producer publishes with each tile
    int nseg, nrows, layer;
    uint32_t row_magic, smem_off;
};

struct RmParams {
    const RmLayer *layers;    // nullptr: `one` is the only layer
    RmLayer one;
    int n_layers, grp_first;
    long long total_tiles, total_w;
    RowQ rq;
    double *partials;         // [slot][kMaxAcc]
    int32_t *status;          // [layer] (layer list) or the header's status word (single tensor)
    int32_t *timeout;         // one word: set if a bounded wait expired
    WsHeader *hdr;            // single tensor: the finish happens in this kernel
    Finalize fin;
};

// First tile of CTA c out of g: the first tile that begins at or after the c-th of g equal shares of the weight.
// The same integer arithmetic runs on the host (slot bookkeeping) and on the device (each CTA's own range).
__host__ __device__ inline long long rm_first_tile(const RmLayer *layers, int n_layers, long long total_tiles, long long total_w, int c, int g)
{
    if (c >= g) return total_tiles;
    const long long target = (long long)(((unsigned long long)c * (unsigned long long)total_w) / (unsigned long long)g);
    int lo = 0, hi = n_layers - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (layers[mid].w_begin <= target) lo = mid;
        else hi = mid - 1;
    }
    const RmLayer &L = layers[lo];
    const long long tile_w = (long long)L.rows_per_tile * L.segs_per_row;
    const long long j = (target - L.w_begin + tile_w - 1) / tile_w;
    return L.tile_begin + (j < L.n_tiles ? j : L.n_tiles);
}

__device__ __forceinline__ int find_layer(const RmLayer *layers, int n, long long tile)
{
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (layers[mid].tile_begin <= tile) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

// The CTA's tiles are numbered it = 0, 1, ...; tile `it` uses barrier set and tables it % kRmSlots, in phase it / kRmSlots.
__device__ __forceinline__ uint32_t slot_parity(int it) { return (uint32_t)(it / kRmSlots) & 1u; }

template <int DT, int NI, int K0, int K1, bool GRP>
__global__ void __launch_bounds__(kRmThreads, 1)
kq_score_rows_mt(const __grid_constant__ RmParams p)
{
    using S = Scorer<DT, NI, K0, K1, true>;      // the scales are fixed over a segment: scaled accumulation
    constexpr int NC = S::NC;
    constexpr int NA = NC * (GRP ? 2 : 1);
    extern __shared__ __align__(16) unsigned char smem[];   // aligned by hand below
    __shared__ __align__(8) uint64_t full_bar[kRmSlots], empty_bar[kRmSlots], row_bar[kRmSlots];
    __shared__ RmTileInfo tinfo[kRmSlots];
    __shared__ int err;
    __shared__ int is_last;
    __shared__ double red[kRmConsumerWarps][kMaxAcc];   // single tensor: the consumer warps' sums, then the last CTA's totals
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem) + 1023u) & ~1023u;
    unsigned char *const smem_al = smem + (smem_base - smem_u32(smem));
    // behind the ring: per slot the segments' abs-max patterns and the rows' abs-max patterns
    uint32_t *const segmax = reinterpret_cast<uint32_t *>(smem_al + kRmRingBytes);
    uint32_t *const rowmax = segmax + kRmSlots * kRmMaxSeg;
    const RmLayer *const layers = p.layers ? p.layers : &p.one;
    if (tid == 0) {
        for (int s = 0; s < kRmSlots; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kRmConsumerWarps);
            mbar_init(&row_bar[s], kRmScoutWarps);
        }
        err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const long long t_begin = rm_first_tile(layers, p.n_layers, p.total_tiles, p.total_w, (int)blockIdx.x, (int)gridDim.x);
    const long long t_end = rm_first_tile(layers, p.n_layers, p.total_tiles, p.total_w, (int)blockIdx.x + 1, (int)gridDim.x);
    const int n_it = (int)(t_end - t_begin);
    double dacc[NA];
#pragma unroll
    for (int j = 0; j < NA; ++j) dacc[j] = 0.0;
    int status = 0;

    if (warp == kRmConsumerWarps + kRmScoutWarps) {
        // ---------------- producer warp: lane 0 issues the copies, all lanes clear the tile's row maxima ----------------
        // A layer's tiles cycle through `stages` (>= 3) equal parts of the ring (its own division: small tiles get
        // more parts).  Tiles are released in order, so "tile it - stages has been released" frees the part tile `it`
        // takes.  A new layer's first tile does not wait for the last tile of the layer before it (that would leave the
        // ring empty at every change of layer): it goes to a part of the new division that does not touch that tile's
        // bytes, and the new division's other parts are used once that tile, too, has been released.
        int layer = n_it > 0 ? find_layer(layers, p.n_layers, t_begin) : 0;
        RmLayer L = layers[layer];
        int run = 0;          // tiles issued under the current division of the ring
        int first_part = 0;   // part of the current division that its first tile took
        uint32_t prev_off = 0, prev_bytes = 0;   // where the tile issued last sits
        bool ok = true;
        for (int it = 0; it < n_it && ok; ++it) {
            const long long t = t_begin + it;
            if (t >= L.tile_begin + L.n_tiles) {
                while (t >= L.tile_begin + L.n_tiles) L = layers[++layer];
                run = 0;
                first_part = 0;
                while (first_part + 1 < L.stages && (uint32_t)first_part * (uint32_t)L.stage_bytes < prev_off + prev_bytes &&
                       (uint32_t)(first_part + 1) * (uint32_t)L.stage_bytes > prev_off)
                    ++first_part;
            }
            // The tiles whose release frees this tile's place.  The groups release their tiles in any order, so every
            // tile that must be gone is waited for by name: the one that had this tile's barrier set and tables, and
            // then either the tile that had its part of the ring or, after a change of layer, every tile of the old
            // division (all but the last one before the new division's first tile, the last one too after that).
            if (it >= kRmSlots) ok = mbar_wait(&empty_bar[it % kRmSlots], slot_parity(it - kRmSlots), &err);
            if (run == 0) {
                for (int k = max(0, it - kRmSlots + 1); k <= it - 2 && ok; ++k) ok = mbar_wait(&empty_bar[k % kRmSlots], slot_parity(k), &err);
            } else {
                const int need = run < L.stages ? it - run - 1 : it - L.stages;
                if (need >= 0 && ok) ok = mbar_wait(&empty_bar[need % kRmSlots], slot_parity(need), &err);
            }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int slot = it % kRmSlots;
            const long long r0 = (t - L.tile_begin) * L.rows_per_tile;
            const int nr = (int)min((long long)L.rows_per_tile, L.rows - r0);
            for (int r = lane; r < nr; r += 32) rowmax[slot * kRmMaxSeg + r] = 0;
            __syncwarp();
            const uint32_t off = (uint32_t)((first_part + run) % L.stages) * (uint32_t)L.stage_bytes;
            prev_off = off;
            prev_bytes = (uint32_t)L.stage_bytes;
            if (lane == 0) {
                tinfo[slot].nseg = nr * L.segs_per_row;
                tinfo[slot].nrows = nr;
                tinfo[slot].layer = layer;
                tinfo[slot].row_magic = L.row_magic;
                tinfo[slot].smem_off = off;
                const uint32_t row_bytes = (uint32_t)L.cols * 2u;
                mbar_expect_tx(&full_bar[slot], (uint32_t)nr * row_bytes);   // (release: the stores above are visible to the waiters)
                unsigned char *dst = smem_al + off;
                if (L.ld == L.cols) {
                    bulk_load(dst, L.x + r0 * L.ld, (uint32_t)nr * row_bytes, &full_bar[slot]);
                } else {
                    for (int r = 0; r < nr; ++r) bulk_load(dst + (size_t)r * row_bytes, L.x + (r0 + r) * L.ld, row_bytes, &full_bar[slot]);
                }
            }
            ++run;
        }
        if (!ok && lane == 0) {
            // give copies already issued a bounded chance to land before the shared memory is released
            for (int k = 0; k < kRmSlots; ++k) {
                const long long t0 = clock64();
                while (!mbar_try_wait(&full_bar[k], 0) && !mbar_try_wait(&full_bar[k], 1) && clock64() - t0 < kWaitCycles) {}
            }
            chain_leave();
            atomicOr(p.timeout, MOFQ_STATUS_TIMEOUT);
        }
    } else if (warp >= kRmConsumerWarps) {
        // ---------------- scout warps: pass 1 of every tile as soon as it has landed ----------------
        // The maxima do not depend on who forms them or in which order, and this pass is bound by the latency of its
        // chain of maxima, not by issue slots: one light warp per scheduler does it for all, so that the scoring
        // warps never wait for one another's pass 1.
        const int sid = warp - kRmConsumerWarps;
        bool ok = true;
        for (int it = 0; it < n_it && ok; ++it) {
            const int slot = it % kRmSlots;
            ok = mbar_wait(&full_bar[slot], slot_parity(it), &err);
            if (!ok) break;
            const RmTileInfo ti = tinfo[slot];
            const int rounds = (ti.nseg + 31) >> 5;
            const uint32_t tile = smem_base + ti.smem_off;
            for (int r = (sid + it) % kRmScoutWarps; r < rounds; r += kRmScoutWarps) {   // rotated: no scout gets the extra round every time
                const int q = r * 32 + lane;
                const bool live = q < ti.nseg;
                uint32_t m16 = 0;
                if (live) {
                    const uint32_t a0 = tile + (uint32_t)q * 256u + (uint32_t)((q & 15) << 4);
                    uint32_t m[4] = {0, 0, 0, 0};   // four independent chains
#pragma unroll
                    for (int k = 0; k < 16; ++k) m[k & 3] = absmax_chunk<DT>(lds128(a0 ^ (uint32_t)(k << 4)), m[k & 3]);
                    m16 = max(max(fold16(m[0]), fold16(m[1])), max(fold16(m[2]), fold16(m[3])));
                    segmax[slot * kRmMaxSeg + q] = m16;
                }
                // the round's segments lie in one or two rows unless rows are shorter than a round: one shared-memory
                // update per row instead of one per lane
                const uint32_t row = ((uint32_t)min(q, ti.nseg - 1) * ti.row_magic) >> 16;
                const uint32_t row0 = __shfl_sync(0xffffffffu, row, 0);
                if (__all_sync(0xffffffffu, row - row0 <= 1u)) {
                    const uint32_t m0 = __reduce_max_sync(0xffffffffu, row == row0 ? m16 : 0u);
                    const uint32_t m1 = __reduce_max_sync(0xffffffffu, row != row0 ? m16 : 0u);
                    if (lane == 0) {
                        atomicMax(&rowmax[slot * kRmMaxSeg + row0], m0);
                        if (m1) atomicMax(&rowmax[slot * kRmMaxSeg + row0 + 1], m1);
                    }
                } else if (live) {
                    atomicMax(&rowmax[slot * kRmMaxSeg + row], m16);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&row_bar[slot]);     // (release: the maxima above are visible to whoever waits)
        }
        if (!ok && lane == 0) {
            chain_leave();
            atomicOr(p.timeout, MOFQ_STATUS_TIMEOUT);
        }
    } else {
        // ---------------- consumer warps: pass 2 ----------------
        // The rounds of the CTA's tile sequence are numbered consecutively and warp w takes the rounds congruent to w:
        // a fixed function of the launch geometry, so sums are formed in the same order on every run.  A warp waits
        // only for the scouts' pass 1 of the tile at hand; the warps drift apart by as many tiles as the ring holds,
        // which evens out the rounds that do not divide among them tile by tile.
        int off2 = warp;      // this warp's first round inside the next tile
        int cur_layer = -1;
        RmLayer L = layers[0];

        auto flush = [&]() __attribute__((always_inline)) {
            // this warp's partial sums of the finished layer -> its slot; the slots are added in order later
#pragma unroll
            for (int j = 0; j < NA; ++j)
#pragma unroll
                for (int o = 16; o; o >>= 1) dacc[j] += __shfl_xor_sync(0xffffffffu, dacc[j], o);
            if (lane == 0) {
                if (p.hdr) {      // single tensor: the CTA adds its warps' sums itself (below) and deposits one slot
#pragma unroll
                    for (int j = 0; j < NA; ++j) red[warp][j] = dacc[j];
                } else {
                    const long long slot = L.slot_off + (long long)((int)blockIdx.x - L.first_cta) * kRmConsumerWarps + warp;
#pragma unroll
                    for (int j = 0; j < NA; ++j) p.partials[slot * kMaxAcc + j] = dacc[j];
                }
            }
            status = __reduce_or_sync(0xffffffffu, status);
            if (status && lane == 0) {
                chain_leave();
                atomicOr(&p.status[p.layers ? cur_layer : 0], status);
            }
#pragma unroll
            for (int j = 0; j < NA; ++j) dacc[j] = 0.0;
            status = 0;
        };

        bool ok = true;
        for (int it = 0; it < n_it; ++it) {
            const int slot = it % kRmSlots;
            ok = mbar_wait(&row_bar[slot], slot_parity(it), &err) && ok;   // the scouts have finished pass 1 of this tile
            if (ok) {
                const RmTileInfo ti = tinfo[slot];
                if (ti.layer != cur_layer) {
                    if (cur_layer >= 0) flush();
                    cur_layer = ti.layer;
                    L = layers[cur_layer];
                }
                const int rounds = (ti.nseg + 31) >> 5;
                const uint32_t tile = smem_base + ti.smem_off;
                for (int r = off2; r < rounds; r += kRmConsumerWarps) {
                    const int q = r * 32 + lane;
                    if (q < ti.nseg) {
                        const uint32_t a0 = tile + (uint32_t)q * 256u + (uint32_t)((q & 15) << 4);
                        const uint32_t rm = rowmax[slot * kRmMaxSeg + ((q * ti.row_magic) >> 16)];
                        if (mag16_nonfinite<DT>(rm)) status |= MOFQ_STATUS_NONFINITE_INPUT;
                        Sc<NC> sc;
                        S s_c, s_g;
#pragma unroll
                        for (int j = 0; j < NC; ++j) {
                            if (DT == MOFQ_F16) scale_pair_fast(mag16_to_float<DT>(rm), p.rq.q[j], p.rq.rq[j], sc.s[j], sc.inv[j]);
                            else scale_pair(mag16_to_float<DT>(rm), p.rq.q[j], sc.s[j], sc.inv[j], status);
                        }
                        s_c.begin(sc);
                        if (GRP) {
                            const uint32_t gm = segmax[slot * kRmMaxSeg + q];
#pragma unroll
                            for (int j = 0; j < NC; ++j) {
                                if (DT == MOFQ_F16) scale_pair_fast(mag16_to_float<DT>(gm), p.rq.q[j], p.rq.rq[j], sc.s[j], sc.inv[j]);
                                else scale_pair(mag16_to_float<DT>(gm), p.rq.q[j], sc.s[j], sc.inv[j], status);
                            }
                            s_g.begin(sc);
                        }
                        // with four candidates per element the fully unrolled loop no longer fits the instruction cache
                        // close to the schedulers (a fifth of the issue slots went to instruction fetch stalls)
#pragma unroll (GRP ? 4 : 16)
                        for (int j = 0; j < 16; ++j) {
                            const uint4 v = lds128(a0 ^ (uint32_t)(j << 4));
                            s_c.chunk(v);
                            if (GRP) s_g.chunk(v);
                        }
                        if (GRP) {      // accumulator order: [first set][second set]
                            double a_c[NC], a_g[NC];
#pragma unroll
                            for (int j = 0; j < NC; ++j) a_c[j] = a_g[j] = 0.0;
                            s_c.end(a_c);
                            s_g.end(a_g);
#pragma unroll
                            for (int j = 0; j < NC; ++j) {
                                dacc[j] += p.grp_first ? a_g[j] : a_c[j];
                                dacc[NC + j] += p.grp_first ? a_c[j] : a_g[j];
                            }
                        } else {
                            s_c.end(dacc);
                        }
                    }
                }
                off2 -= rounds % kRmConsumerWarps;
                if (off2 < 0) off2 += kRmConsumerWarps;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[slot]);
        }
        if (cur_layer >= 0) flush();
        if (!ok && lane == 0) {   // a wait expired: the sums are incomplete
            chain_leave();
            atomicOr(p.timeout, MOFQ_STATUS_TIMEOUT);
        }
    }
    if (!p.hdr) return;
    // A single tensor's launch may have started beside the kernel that clears the workspace header (see
    // kq_header_clear): the header is first touched below, or just above where a status bit is recorded.
    chain_leave();

    // ---------------- single tensor: each CTA deposits the sum of its warps; the last CTA to finish adds the CTAs' sums in
    // order and writes the outputs ----------------
    if (n_it == 0 && warp < kRmConsumerWarps && lane < NA) red[warp][lane] = 0.0;   // (cannot happen: every CTA has a tile)
    __syncthreads();
    if (tid < NA) {
        double t = 0.0;
        for (int w = 0; w < kRmConsumerWarps; ++w) t += red[w][tid];
        p.partials[(size_t)blockIdx.x * kMaxAcc + tid] = t;
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const uint32_t ticket = atomicAdd(&p.hdr->counter, 1u);
        is_last = (ticket == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last || warp != 0) return;
    __threadfence();
    double tot[NA];
#pragma unroll
    for (int j = 0; j < NA; ++j) tot[j] = 0.0;
    // lane l: CTAs l, l + 32, ... in that order; eight CTAs' slots are fetched before the first is added, so that the
    // reduction costs one trip to the level-2 cache per 256 CTAs instead of one per 32
    for (int c0 = lane; c0 < (int)gridDim.x; c0 += 32 * 8) {
        double v[8][NA];
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
            for (int j = 0; j < NA; ++j)
                v[k][j] = c0 + 32 * k < (int)gridDim.x ? __ldcg(&p.partials[(size_t)(c0 + 32 * k) * kMaxAcc + j]) : 0.0;
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
            for (int j = 0; j < NA; ++j) tot[j] += v[k][j];
    }
#pragma unroll
    for (int j = 0; j < NA; ++j)
#pragma unroll
        for (int o = 16; o; o >>= 1) tot[j] += __shfl_xor_sync(0xffffffffu, tot[j], o);
    if (lane == 0) {
        p.hdr->counter = 0;
        const int t = *reinterpret_cast<volatile int32_t *>(p.timeout);
        if (t) atomicOr(&p.hdr->status, t);
        kqfin::write_outputs(tot, p.fin, p.hdr);
    }
}

// ---- finalize of a layer list: one block per layer ---------------------------------------------------------------
__global__ void __launch_bounds__(128)
kq_rows_finalize(const RmLayer *layers, const double *partials, const int32_t *status, const int32_t *timeout, Finalize fin,
                 mofq_result *results)
{
    __shared__ double red[4][kMaxAcc];
    const RmLayer L = layers[blockIdx.x];
    const int na = fin.nc * fin.n_sets;
    double tot[kMaxAcc];
#pragma unroll
    for (int j = 0; j < kMaxAcc; ++j) tot[j] = 0.0;
    for (int slot = threadIdx.x; slot < L.n_slots; slot += blockDim.x)
        for (int j = 0; j < na; ++j) tot[j] += partials[(size_t)(L.slot_off + slot) * kMaxAcc + j];
    for (int j = 0; j < na; ++j)
#pragma unroll
        for (int o = 16; o; o >>= 1) tot[j] += __shfl_xor_sync(0xffffffffu, tot[j], o);
    if ((threadIdx.x & 31) == 0)
        for (int j = 0; j < na; ++j) red[threadIdx.x >> 5][j] = tot[j];
    __syncthreads();
    if (threadIdx.x != 0) return;
    for (int s = 0; s < fin.n_sets; ++s) {
        double err[MOFQ_MAX_CAND];
        double best = INFINITY, second = INFINITY;
        int chosen = -1;
        for (int i = 0; i < fin.n_cand; ++i) {
            const int j = s * fin.nc + fin.perm[i];
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
        results[(size_t)blockIdx.x * fin.n_sets + s] = r;
    }
}

// The work table travels to the device as kernel arguments, 256 entries (26 KB of the 32 KB a launch may carry) per
// launch: fully stream-ordered, no pageable-memory copy (which would synchronise the stream) and nothing for the caller
// to keep alive.
constexpr int kRmUploadChunk = 256;
static_assert(sizeof(RmLayer) * kRmUploadChunk + 64 <= 32764, "the chunk must fit a launch's parameter space");
struct RmTableChunk {
    RmLayer e[kRmUploadChunk];
};
__global__ void kq_rows_upload(const RmTableChunk chunk, RmLayer *dst, int n)
{
    if ((int)threadIdx.x < n) dst[threadIdx.x] = chunk.e[threadIdx.x];
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

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

// Rows per tile: the whole rows (within the cap) that leave the fewest idle lanes in a tile's last round.  Among equally
// well filled shapes the tile grows up to 48 KB (fewer barrier rounds per byte); a single tensor keeps at least eight
// tiles per SM so that the CTAs' shares stay even.
int rows_per_tile(long long rows, int cols, bool single)
{
    const int row_bytes = cols * 2, spr = cols / 128;
    const long long min_tiles = single ? 8LL * sm_count() : 1;
    int best = 1;
    double best_fill = 0.0;
    for (int k = 1; k <= kRmMaxSeg && (long long)k * row_bytes <= kRmTileCap && k <= rows; ++k) {
        if (k > 1 && (rows + k - 1) / k < min_tiles) break;
        const int nseg = k * spr;
        const double fill = (double)nseg / (double)(32 * ((nseg + 31) / 32));
        if (fill > best_fill + 1e-9 || (fill > best_fill - 1e-9 && k * row_bytes <= 48 * 1024)) {
            best_fill = std::max(fill, best_fill);
            best = k;
        }
    }
    return best;
}

// Fills the geometry of one layer; false if the kernel cannot take the tensor.
bool describe_layer(const mofq_tensor &W, RmLayer *L, bool single = false)
{
    if (W.cols % 128 != 0 || W.cols * 2 > kRmTileCap || W.cols <= 0 || W.rows <= 0) return false;
    L->x = static_cast<const uint16_t *>(W.data);
    L->rows = W.rows;
    L->ld = W.ld;
    L->cols = (int)W.cols;
    L->segs_per_row = (int)(W.cols / 128);
    L->rows_per_tile = rows_per_tile(W.rows, (int)W.cols, single);
    L->n_tiles = (W.rows + L->rows_per_tile - 1) / L->rows_per_tile;
    L->inv_n = 1.0 / ((double)W.rows * (double)W.cols);
    L->stage_bytes = (L->rows_per_tile * (int)W.cols * 2 + 1023) & ~1023;
    L->stages = std::min(kRmSlots, kRmRingBytes / L->stage_bytes);   // >= 3: a tile is at most a third of the ring
    // q / segs_per_row for q < kRmMaxSeg through a multiply and a shift (checked here for every q)
    L->row_magic = (65536u + (uint32_t)L->segs_per_row - 1u) / (uint32_t)L->segs_per_row;
    for (uint32_t q = 0; q < (uint32_t)kRmMaxSeg; ++q)
        if (((q * L->row_magic) >> 16) != q / (uint32_t)L->segs_per_row) return false;
    return true;
}

struct RmPlan {
    std::vector<RmLayer> table;
    long long total_tiles = 0, total_w = 0;
    int grid = 1;
    long long slots = 0;
};

bool make_plan(const mofq_tensor *const *tensors, int n, RmPlan *plan)
{
    plan->table.resize((size_t)n);
    long long tiles = 0, w = 0;
    for (int i = 0; i < n; ++i) {
        RmLayer &L = plan->table[(size_t)i];
        std::memset(&L, 0, sizeof(L));
        if (!describe_layer(*tensors[i], &L, n == 1)) return false;
        L.tile_begin = tiles;
        L.w_begin = w;
        tiles += L.n_tiles;
        w += L.n_tiles * L.rows_per_tile * L.segs_per_row;   // the last tile of a layer counts as a full one
    }
    plan->total_tiles = tiles;
    plan->total_w = w;
    // every CTA's share of the weight holds at least one tile begin, so that no CTA between two others is idle
    const long long by_weight = std::max<long long>(1, w / kRmMaxSeg);
    plan->grid = (int)std::max<long long>(1, std::min<long long>(std::min<long long>(sm_count(), tiles), by_weight));
    std::vector<long long> first((size_t)plan->grid + 1);
    for (int c = 0; c <= plan->grid; ++c) first[(size_t)c] = rm_first_tile(plan->table.data(), n, tiles, w, c, plan->grid);
    long long slot = 0;
    int c0 = 0;
    for (int i = 0; i < n; ++i) {
        RmLayer &L = plan->table[(size_t)i];
        const long long b = L.tile_begin, e = L.tile_begin + L.n_tiles;
        while (c0 + 1 <= plan->grid && first[(size_t)c0 + 1] <= b) ++c0;   // first CTA whose range reaches past b
        int c1 = c0;
        while (c1 + 1 < plan->grid && first[(size_t)c1 + 1] < e) ++c1;    // last CTA whose range starts before e
        L.first_cta = c0;
        L.n_slots = (c1 - c0 + 1) * kRmConsumerWarps;
        L.slot_off = (int)slot;
        slot += L.n_slots;
    }
    plan->slots = slot;
    return true;
}

// The kernel always asks for the same amount of dynamic shared memory, so the opt-in is made once per (device, kernel)
// and remembered: a single small tensor's call is short enough for the repeated attribute call to show.
int smem_opt_in(const void *kernel)
{
    static std::mutex mu;
    static std::vector<std::pair<int, const void *>> done;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(mu);
    for (const auto &d : done)
        if (d.first == dev && d.second == kernel) return MOFQ_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRmSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    done.emplace_back(dev, kernel);
    return MOFQ_OK;
}

template <typename K>
int launch_kernel(K kernel, const RmPlan &plan, const RmParams &p, cudaStream_t st, bool chained)
{
    const size_t smem = kRmSmemBytes;
    if (int rc = smem_opt_in(reinterpret_cast<const void *>(kernel))) return rc;
    if (launch_chained(kernel, dim3((unsigned)plan.grid), dim3(kRmThreads), smem, st, chained, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    return MOFQ_OK;
}

// Clears a workspace header.  A single tensor's scoring launch is chained behind it and starts at once: that kernel
// touches the header only after its chain_leave().
__global__ void kq_header_clear(WsHeader *hdr)
{
    chain_enter_early();
    reinterpret_cast<uint32_t *>(hdr)[threadIdx.x] = 0u;
}

int launch_plan(const RmPlan &plan, RmParams &p, int dtype, const CandSet &cs, const int *fp_formats, bool has_grp, cudaStream_t st,
                bool chained = false)
{
    p.n_layers = (int)plan.table.size();
    p.total_tiles = plan.total_tiles;
    p.total_w = plan.total_w;
    p.rq = candset_rowq(cs);
    const int k0 = cs.n_fp > 0 ? fp_kind(fp_formats[0]) : -1, k1 = cs.n_fp > 1 ? fp_kind(fp_formats[1]) : -1;
    return dispatch_kinds(dtype, cs.n_int, k0, k1, [&](auto DT, auto NI, auto K0, auto K1) {
        if (has_grp) return launch_kernel(kq_score_rows_mt<DT(), NI(), K0(), K1(), true>, plan, p, st, chained);
        return launch_kernel(kq_score_rows_mt<DT(), NI(), K0(), K1(), false>, plan, p, st, chained);
    });
}

bool grans_ok(int gran, int gran2, int group)
{
    const bool has_ch = gran == MOFQ_PER_CHANNEL || gran2 == MOFQ_PER_CHANNEL;
    const bool has_grp = gran == MOFQ_PER_GROUP || gran2 == MOFQ_PER_GROUP;
    if (!has_ch || gran == MOFQ_PER_TENSOR || gran2 == MOFQ_PER_TENSOR) return false;
    return !has_grp || group == 128;
}

}  // namespace

// One tensor with per-channel scales (optionally group-128 scales as the other set): true if the streamed-rows
// kernel takes it.
bool rows_single_applicable(const ScoreJob &job)
{
    RmLayer L;
    return grans_ok(job.gran, job.gran2, job.group) && describe_layer(job.x, &L);
}

int rows_single_run(const ScoreJob &job, cudaStream_t st)
{
    RmPlan plan;
    const mofq_tensor *t = &job.x;
    if (!make_plan(&t, 1, &plan)) return MOFQ_ERR_UNSUPPORTED;
    if (plan.slots > kMaxSlots) return MOFQ_ERR_UNSUPPORTED;
    if (job.clear_header) {
        kq_header_clear<<<1, (unsigned)(sizeof(WsHeader) / sizeof(uint32_t)), 0, st>>>(job.hdr);
        if (cudaGetLastError() != cudaSuccess) return MOFQ_ERR_CUDA;
    }
    RmParams p{};
    p.layers = nullptr;
    p.one = plan.table[0];
    p.grp_first = job.gran == MOFQ_PER_GROUP ? 1 : 0;
    p.partials = job.partials;
    p.status = &job.hdr->status;
    p.timeout = reinterpret_cast<int32_t *>(&job.hdr->pad[0]);   // cleared with the header
    p.hdr = job.hdr;
    p.fin = job.fin;
    const bool has_grp = job.gran == MOFQ_PER_GROUP || job.gran2 == MOFQ_PER_GROUP;
    return launch_plan(plan, p, job.x.dtype, job.cs, job.fp_formats, has_grp, st, job.clear_header);
}

// A layer list under the tensor metric with per-channel scales (optionally group-128 scales as the other set) on
// tensors of one dtype whose rows are multiples of 128 elements and at most 72 KB long.
bool rows_mt_applicable(const mofq_layer *layers, int n_layers, const mofq_config *cfg)
{
    if (cfg->metric != MOFQ_TENSOR_MSE || n_layers < 2 || !grans_ok(cfg->w_gran, cfg->w_gran2, cfg->w_group)) return false;
    for (int i = 0; i < n_layers; ++i) {
        RmLayer L;
        if (layers[i].W.dtype != layers[0].W.dtype || !describe_layer(layers[i].W, &L)) return false;
    }
    return true;
}

size_t rows_mt_ws_bytes(int n_layers)
{
    const size_t slots = ((size_t)sm_count() + (size_t)n_layers) * kRmConsumerWarps;
    return align256(sizeof(RmLayer) * (size_t)n_layers) + align256(slots * kMaxAcc * sizeof(double)) +
           align256(sizeof(int32_t) * ((size_t)n_layers + 1));
}

int rows_mt_run(const mofq_layer *layers, int n_layers, const mofq_config *cfg, const CandSet &cs, const int *perm, int nc,
                const int *fp_formats, mofq_result *results, void *ws, cudaStream_t st)
{
    std::vector<const mofq_tensor *> tensors((size_t)n_layers);
    for (int i = 0; i < n_layers; ++i) tensors[(size_t)i] = &layers[i].W;
    RmPlan plan;
    if (!make_plan(tensors.data(), n_layers, &plan)) return MOFQ_ERR_UNSUPPORTED;
    char *base = static_cast<char *>(ws);
    RmLayer *d_table = reinterpret_cast<RmLayer *>(base);
    double *d_partials = reinterpret_cast<double *>(base + align256(sizeof(RmLayer) * (size_t)n_layers));
    const size_t slots_cap = ((size_t)sm_count() + (size_t)n_layers) * kRmConsumerWarps;
    if ((size_t)plan.slots > slots_cap) return MOFQ_ERR_WORKSPACE_TOO_SMALL;
    int32_t *d_status = reinterpret_cast<int32_t *>(reinterpret_cast<char *>(d_partials) + align256(slots_cap * kMaxAcc * sizeof(double)));
    for (int i = 0; i < n_layers; i += kRmUploadChunk) {
        RmTableChunk chunk;
        const int n = std::min(kRmUploadChunk, n_layers - i);
        for (int k = 0; k < n; ++k) chunk.e[k] = plan.table[(size_t)(i + k)];
        kq_rows_upload<<<1, kRmUploadChunk, 0, st>>>(chunk, d_table + i, n);
        if (cudaGetLastError() != cudaSuccess) return MOFQ_ERR_CUDA;
    }
    if (cudaMemsetAsync(d_status, 0, sizeof(int32_t) * ((size_t)n_layers + 1), st) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    RmParams p{};
    p.layers = d_table;
    p.grp_first = cfg->w_gran == MOFQ_PER_GROUP ? 1 : 0;
    p.partials = d_partials;
    p.status = d_status;
    p.timeout = d_status + n_layers;
    p.hdr = nullptr;
    const bool has_grp = cfg->w_gran == MOFQ_PER_GROUP || cfg->w_gran2 == MOFQ_PER_GROUP;
    if (int rc = launch_plan(plan, p, layers[0].W.dtype, cs, fp_formats, has_grp, st)) return rc;
    Finalize fin{};
    fin.n_cand = cfg->n_candidates;
    fin.n_sets = cfg->w_gran2 != MOFQ_GRAN_NONE ? 2 : 1;
    fin.nc = nc;
    for (int i = 0; i < MOFQ_MAX_CAND; ++i) fin.perm[i] = perm[i];
    kq_rows_finalize<<<n_layers, 128, 0, st>>>(d_table, d_partials, d_status, d_status + n_layers, fin, results);
    if (cudaGetLastError() != cudaSuccess) return MOFQ_ERR_CUDA;
    return MOFQ_OK;
}

}  // namespace mofq
