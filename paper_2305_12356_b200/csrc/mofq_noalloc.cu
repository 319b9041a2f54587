// mofq_tensor_error_noalloc: the tensor-error entry point for callers that cannot allocate.
//
// Some users of this library run where cudaMalloc is off the table: inside a process whose whole
// device memory was handed to another allocator up front, in a plug-in that is forbidden to grow
// the process's footprint, or at a point of a serving loop where an allocation would stall every
// stream.  mofq_tensor_error asks such a caller for a workspace it cannot produce.  This variant
// keeps the workspace in a fixed array inside the library image instead.
#include <mutex>

#include "mofq_internal.h"

namespace {

// The scratch lives in every CUDA context that loads this library, until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[MOFQ_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices];  // device address of the array, per device ordinal
std::mutex g_setup_mutex;

// The array's name is only a host-side handle; kernels need its address on the current device.
int scratch_for_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return MOFQ_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return MOFQ_OK;
}

}  // namespace

extern "C" size_t mofq_noalloc_scratch_bytes(void) { return MOFQ_NOALLOC_SCRATCH_BYTES; }

extern "C" int mofq_tensor_error_noalloc(const mofq_tensor *x, const int32_t *formats, int n, int gran, int gran2,
                                         int group, float *mse_out, int32_t *status_out, void *stream)
{
    if (!x) return MOFQ_ERR_INVALID_ARG;
    // the fixed array must cover what this tensor's scoring pass needs
    if (mofq_tensor_workspace_bytes(x) > (size_t)MOFQ_NOALLOC_SCRATCH_BYTES) return MOFQ_ERR_SCRATCH_LIMIT;
    if ((int64_t)x->rows * (int64_t)x->cols > (int64_t)MOFQ_NOALLOC_MAX_ELEMENTS) return MOFQ_ERR_SCRATCH_LIMIT;
    void *scratch = nullptr;
    if (int rc = scratch_for_current_device(&scratch)) return rc;
    // mofq_tensor_error clears the header of its workspace itself, so the previous call's status,
    // block counter and abs-max never leak into this one; the partial sums are overwritten before use.
    const int rc = mofq_tensor_error(x, formats, n, gran, gran2, group, mse_out, scratch, MOFQ_NOALLOC_SCRATCH_BYTES, stream);
    if (rc != MOFQ_OK) return rc;
    if (status_out &&
        cudaMemcpyAsync(status_out, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return MOFQ_ERR_CUDA;
    }
    return MOFQ_OK;
}
