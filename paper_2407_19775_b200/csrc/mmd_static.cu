// mmd_static.cu -- mmd_linear_static: the decomposed linear layer for callers that cannot
// obtain device memory, with its scratch in a fixed array that is part of the library image.
//
// The array below is device memory that every GPU which loads the library holds until the
// process exits.  In host code its name stands for the symbol, not for a device address, so
// the address is looked up once per device (cudaGetSymbolAddress, with that device current)
// and that pointer is what the kernels receive.
#include "../../include/mmd.h"
#include "bq_error.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[MMD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_lock;
void* g_scratch_of_device[kMaxDevices] = {};

// The device address of the array on the current device; looked up on the first call per device.
cudaError_t scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> guard(g_lock);
    if (!g_scratch_of_device[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_of_device[dev] = p;
    }
    *out = g_scratch_of_device[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int mmd_linear_static(const mmd_weights* w, const void* X, int M, void* Y, bq_dtype ydt, int path, void* cuda_stream) {
    if (!w) return BQ_ERR_NULL;
    if (M < 0) return BQ_ERR_SIZE;
    // A call of mmd_linear with zero rows checks the element type and the path and launches nothing:
    // both entry points then answer a bad argument with the same code, whatever M is.
    const int checked = mmd_linear(w, X, 0, Y, ydt, nullptr, 0, path, cuda_stream);
    if (checked != BQ_OK || M == 0) return checked;
    size_t need = 0;
    const int rc = mmd_workspace_layout(w, M, nullptr, &need);
    if (rc != BQ_OK) return rc;
    if (need > size_t(MMD_STATIC_SCRATCH_BYTES)) {
        char text[160];
        std::snprintf(text, sizeof(text), "mmd_linear_static: %d rows need %zu bytes of scratch, the static array holds %u", M, need,
                      unsigned(MMD_STATIC_SCRATCH_BYTES));
        bql::set_last_cuda_error(text);
        return MMD_ERR_STATIC_LIMIT;
    }
    void* scratch = nullptr;
    const cudaError_t e = scratch_address(&scratch);
    if (e != cudaSuccess) {
        bql::set_last_cuda_error(cudaGetErrorString(e));
        return BQ_ERR_CUDA;
    }
    // Nothing in the array has to start at zero: the row kernel writes every byte of it that
    // the product kernel reads (codes, scales and the zero padding of the side columns), so
    // what an earlier call left behind is never seen.
    return mmd_linear(w, X, M, Y, ydt, scratch, size_t(MMD_STATIC_SCRATCH_BYTES), path, cuda_stream);
}
