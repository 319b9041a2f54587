// Diagnostic entry point: exposes the grid rounding that the scoring kernels perform with the hardware
// converts, so that a test can compare it value by value with the definition (nearest grid point, ties to even).
#include "kq_math.cuh"
#include "kq_pipe.cuh"
#include "mofq_internal.h"

namespace {

template <int KIND>
__global__ void diag_round(const float *__restrict__ t, float *__restrict__ out, long long n)
{
    const long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 2;
    if (i >= n) return;
    const float a = t[i], b = i + 1 < n ? t[i + 1] : 0.0f;
    const uint32_t h2 = mofq::kqmath::fp_round_trip<KIND>(fabsf(a), fabsf(b));
    const float2 r = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    out[i] = copysignf(r.x, a);
    if (i + 1 < n) out[i + 1] = copysignf(r.y, b);
}

__global__ void diag_scale_pair(const float *__restrict__ a, float Q, float rQ, float *__restrict__ s, float *__restrict__ inv, long long n)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) mofq::kqmath::scale_pair_fast(a[i], Q, rQ, s[i], inv[i]);
}

// waits, with the library's bounded wait, on a barrier that nothing ever arrives on
__global__ void diag_wait_expiry(int32_t *status_out)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int err;
    if (threadIdx.x == 0) {
        mofq::kqpipe::mbar_init(&bar, 1);
        err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool ok = mofq::kqpipe::mbar_wait(&bar, 0, &err);
        *status_out = ok ? 0 : MOFQ_STATUS_TIMEOUT;
    }
}

}  // namespace

extern "C" int mofq_diag_wait_expiry(int32_t *status_out, void *stream)
{
    if (!status_out) return MOFQ_ERR_INVALID_ARG;
    diag_wait_expiry<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status_out);
    return cudaGetLastError() == cudaSuccess ? MOFQ_OK : MOFQ_ERR_CUDA;
}

extern "C" int mofq_diag_scale_pair(int format, const float *absmax, float *scale_out, float *inv_out, int64_t n, void *stream)
{
    mofq::FmtDesc d;
    if (!absmax || !scale_out || !inv_out || n <= 0 || !mofq::describe_format(format, &d)) return MOFQ_ERR_INVALID_ARG;
    diag_scale_pair<<<(int)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(absmax, d.Q, 1.0f / d.Q, scale_out, inv_out, n);
    return cudaGetLastError() == cudaSuccess ? MOFQ_OK : MOFQ_ERR_CUDA;
}

extern "C" int mofq_diag_fp_round(int format, const float *t, float *out, int64_t n, void *stream)
{
    if (!t || !out || n <= 0) return MOFQ_ERR_INVALID_ARG;
    const int grid = (int)((n / 2 + 1 + 255) / 256);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (format) {
    case MOFQ_FP4_E2M1: diag_round<mofq::kqmath::FPK_E2M1><<<grid, 256, 0, st>>>(t, out, n); break;
    case MOFQ_FP8_E4M3: diag_round<mofq::kqmath::FPK_E4M3><<<grid, 256, 0, st>>>(t, out, n); break;
    case MOFQ_FP8_E5M2: diag_round<mofq::kqmath::FPK_E5M2><<<grid, 256, 0, st>>>(t, out, n); break;
    default: return MOFQ_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? MOFQ_OK : MOFQ_ERR_CUDA;
}
