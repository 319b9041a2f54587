// Seeded synthetic tensors on the device (separate shared library: input generation only, no
// quantisation arithmetic).  Counter-based Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel
// random numbers: as easy as 1, 2, 3", SC'11): key = seed, counter = (element pair, tensor, layer),
// so any layer of a model can be produced on its own.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace {

enum { KIND_GAUSS_OUTLIER = 0, KIND_STUDENT_T = 1, KIND_LAPLACE = 2, KIND_ACTIVATION = 3 };
constexpr int kMaxChannels = 16;

struct Channels {
    int32_t idx[kMaxChannels];
    int n;
};

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

// (0,1]: never zero, so logs and inverse roots stay finite
__device__ __forceinline__ float u01(uint32_t r) { return ((float)(r >> 8) + 1.0f) * (1.0f / 16777216.0f); }

__device__ __forceinline__ void normal_pair(uint32_t a, uint32_t b, float &z0, float &z1)
{
    const float r = sqrtf(-2.0f * __logf(u01(a)));
    float s, c;
    __sincosf(6.28318530718f * u01(b), &s, &c);
    z0 = r * c;
    z1 = r * s;
}

template <int DT>
__device__ __forceinline__ uint32_t pack2(float a, float b)
{
    if (DT == 0) return (uint32_t)__half_as_ushort(__float2half_rn(a)) | ((uint32_t)__half_as_ushort(__float2half_rn(b)) << 16);
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(b)) << 16);
}

template <int DT>
__global__ void __launch_bounds__(256)
synth_fill(uint16_t *out, long long rows, int cols, long long ld, int kind, uint2 key, uint32_t layer, uint32_t tensor_id,
           float p0, float p1, float p2, Channels ch)
{
    const int cpr = cols >> 3;
    const long long total = rows * cpr;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long row = i / cpr;
        const int c8 = (int)(i - row * cpr);
        float row_gain = 1.0f;
        if (kind == KIND_ACTIVATION && p1 > 0.0f) {  // token-wise spikes: a per-row draw
            const uint4 r = philox4x32_10(make_uint4((uint32_t)row, (uint32_t)(row >> 32), tensor_id ^ 0x80000000u, layer), key);
            if (u01(r.x) <= p1) row_gain = p2;
        }
        uint32_t w[4];
#pragma unroll
        for (int pi = 0; pi < 4; ++pi) {
            const long long pair = (row * (long long)cols + (long long)c8 * 8 + pi * 2) >> 1;
            const uint4 r = philox4x32_10(make_uint4((uint32_t)pair, (uint32_t)(pair >> 32), tensor_id, layer), key);
            float v0, v1;
            if (kind == KIND_GAUSS_OUTLIER) {  // N(0,std^2), replaced with prob. p1 by N(0,(p2*std)^2)
                normal_pair(r.x, r.y, v0, v1);
                v0 *= p0 * (u01(r.z) <= p1 ? p2 : 1.0f);
                v1 *= p0 * (u01(r.w) <= p1 ? p2 : 1.0f);
            } else if (kind == KIND_STUDENT_T) {  // Bailey's polar form for Student-t, nu = 4
                v0 = p0 * sqrtf(4.0f * (rsqrtf(u01(r.x)) - 1.0f)) * __cosf(6.28318530718f * u01(r.y));
                v1 = p0 * sqrtf(4.0f * (rsqrtf(u01(r.z)) - 1.0f)) * __cosf(6.28318530718f * u01(r.w));
            } else if (kind == KIND_LAPLACE) {  // inverse CDF; sign from the top bit; x10 with prob. p1
                const float m0 = -p0 * __logf(u01(r.x << 1)), m1 = -p0 * __logf(u01(r.y << 1));
                v0 = ((r.x >> 31) ? -m0 : m0) * (u01(r.z) <= p1 ? p2 : 1.0f);
                v1 = ((r.y >> 31) ? -m1 : m1) * (u01(r.w) <= p1 ? p2 : 1.0f);
            } else {  // activations: N(0,1), outlier channels x p0, spiky rows x p2
                normal_pair(r.x, r.y, v0, v1);
                const int col = c8 * 8 + pi * 2;
                for (int k = 0; k < ch.n; ++k) {
                    if (ch.idx[k] == col) v0 *= p0;
                    if (ch.idx[k] == col + 1) v1 *= p0;
                }
                v0 *= row_gain;
                v1 *= row_gain;
            }
            w[pi] = pack2<DT>(v0, v1);
        }
        *reinterpret_cast<uint4 *>(out + row * ld + (long long)c8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

}  // namespace

// out: device, [rows, cols] with leading dimension ld (elements), 16-byte aligned, cols % 8 == 0.
// channels: host array of n_channels (<= 16) outlier channel indices (activation kind only).
// Returns 0, -1 for a bad argument, -5 for a launch failure.
extern "C" int mofq_synth_fill(void *out, int dtype, int64_t rows, int64_t cols, int64_t ld, int kind, uint64_t seed,
                               uint32_t layer, uint32_t tensor_id, float p0, float p1, float p2, float p3,
                               const int32_t *channels, int n_channels, void *stream)
{
    (void)p3;
    if (!out || rows <= 0 || cols <= 0 || (cols & 7) || (ld & 7) || ld < cols || (reinterpret_cast<uintptr_t>(out) & 15)) return -1;
    if (kind < 0 || kind > 3 || (dtype != 0 && dtype != 1) || n_channels < 0 || n_channels > kMaxChannels) return -1;
    Channels ch{};
    ch.n = n_channels;
    for (int i = 0; i < n_channels; ++i) ch.idx[i] = channels[i];
    const long long total = rows * (cols / 8);
    const long long blocks = (total + 255) / 256;
    const int grid = (int)(blocks > 148 * 16 ? 148 * 16 : blocks);
    const uint2 key = make_uint2((uint32_t)seed, (uint32_t)(seed >> 32));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == 0)
        synth_fill<0><<<grid, 256, 0, st>>>((uint16_t *)out, rows, (int)cols, ld, kind, key, layer, tensor_id, p0, p1, p2, ch);
    else
        synth_fill<1><<<grid, 256, 0, st>>>((uint16_t *)out, rows, (int)cols, ld, kind, key, layer, tensor_id, p0, p1, p2, ch);
    return cudaGetLastError() == cudaSuccess ? 0 : -5;
}
