// bq_api.cu -- the C ABI of libbq (see include/bq.h): argument checks, codebook handles and
// the choice of kernel.  Kernel instantiations live in bq_inst_*.cu so that they compile in
// parallel; this file only calls their launchers.
#include "../../include/mmd.h"
#include "bq_debug.h"
#include "bq_error.h"
#include "bq_launch.h"

#include <atomic>
#include <cstring>
#include <new>

namespace {

thread_local char g_last_error[256] = "";

int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}

bool known_dtype(int dt) { return dt == BQ_F32 || dt == BQ_F16 || dt == BQ_BF16; }
size_t elem_bytes(int dt) { return dt == BQ_F32 ? 4 : 2; }

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int log2_exact(size_t v) {
    int l = 0;
    while ((size_t(1) << l) < v) ++l;
    return ((size_t(1) << l) == v) ? l : -1;
}

bool tuned_block(int block) {
    switch (block) {
        case 64: case 128: case 256: case 512: case 1024: case 2048: case 4096: return true;
        default: return false;
    }
}

constexpr size_t kMaxElems = size_t(1) << 40;

std::atomic<int> g_staging{0};      // bq_set_staging: blocks of 2048 / 4096 through the shared-memory-staged kernel

}  // namespace

void bql::set_last_cuda_error(const char* text) { std::strncpy(g_last_error, text, sizeof(g_last_error) - 1); }

struct bq_codebook {
    bqt::Tables host;
    bqk::DeviceTables dev;
    void* blob;
    int* status;              // device word set by a kernel whose bounded wait ran out
    int device;
    int sm_count;
};

static bool on_codebook_device_c(const bq_codebook* cb);

extern "C" {

const char* bq_status_string(int status) {
    switch (status) {
        case BQ_OK: return "ok";
        case BQ_ERR_NULL: return "a required pointer is NULL";
        case BQ_ERR_DTYPE: return "unknown element type";
        case BQ_ERR_BLOCK: return "block size must be at least 1";
        case BQ_ERR_SIZE: return "element count out of range";
        case BQ_ERR_CODEBOOK: return "invalid codebook kind, values or handle";
        case BQ_ERR_CUDA: return "CUDA runtime error (see bq_last_cuda_error)";
        case BQ_ERR_ASSERT: return "an assertion of the debug build failed (see bq_last_cuda_error)";
        case MMD_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case MMD_ERR_FEATURES: return "feature list not ascending, out of range or too long";
        case MMD_ERR_PATH: return "the requested kernel path cannot take this shape";
        case MMD_ERR_STATIC_LIMIT: return "the call needs more scratch than the library's static array holds (see bq_last_cuda_error)";
        default: return "unknown status";
    }
}

const char* bq_last_cuda_error(void) { return g_last_error; }

int bq_make_codebook(int kind, const float* user_values256, float* host_values_out256, bq_codebook** out) {
    if (!out) return BQ_ERR_NULL;
    *out = nullptr;
    bq_codebook* cb = new (std::nothrow) bq_codebook();
    if (!cb) return BQ_ERR_CUDA;
    if (kind == BQ_CODEBOOK_DYNAMIC_TREE) {
        if (user_values256) { delete cb; return BQ_ERR_CODEBOOK; }
        bqt::dynamic_tree_values(cb->host.values);
    } else if (kind == BQ_CODEBOOK_USER) {
        if (!user_values256) { delete cb; return BQ_ERR_NULL; }
        if (!bqt::valid_user_values(user_values256)) { delete cb; return BQ_ERR_CODEBOOK; }
        std::memcpy(cb->host.values, user_values256, 256 * sizeof(float));
    } else {
        delete cb;
        return BQ_ERR_CODEBOOK;
    }
    bqt::build(cb->host);
    if (host_values_out256) std::memcpy(host_values_out256, cb->host.values, 256 * sizeof(float));

    // one device allocation: values | thr_down | tk | cmag | guess  (the kernels rely on guess following cmag directly)
    const size_t words = 256 + 256 + 128 + 132 + bqt::kCells + 4;      // the last four words: the kernels' status word (zero)
    cudaError_t e = cudaGetDevice(&cb->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&cb->sm_count, cudaDevAttrMultiProcessorCount, cb->device);
    if (e == cudaSuccess) e = cudaMalloc(&cb->blob, words * 4);
    if (e != cudaSuccess) { delete cb; return cuda_fail(e); }
    uint32_t* stage = new (std::nothrow) uint32_t[words]();
    if (!stage) { cudaFree(cb->blob); delete cb; return BQ_ERR_CUDA; }
    size_t o = 0;
    std::memcpy(stage + o, cb->host.values, 256 * 4);   const size_t o_val = o; o += 256;
    std::memcpy(stage + o, cb->host.thr_down, 256 * 4); const size_t o_thr = o; o += 256;
    std::memcpy(stage + o, cb->host.tk, 128 * 4);       const size_t o_tk = o;  o += 128;
    std::memcpy(stage + o, cb->host.cmag, 132 * 4);     const size_t o_cm = o;  o += 132;
    std::memcpy(stage + o, cb->host.guess, bqt::kCells * 4); const size_t o_gs = o;
    e = cudaMemcpy(cb->blob, stage, words * 4, cudaMemcpyHostToDevice);
    delete[] stage;
    if (e != cudaSuccess) { cudaFree(cb->blob); delete cb; return cuda_fail(e); }
    const uint32_t* base = static_cast<const uint32_t*>(cb->blob);
    cb->dev.values = reinterpret_cast<const float*>(base + o_val);
    cb->dev.thr_down = reinterpret_cast<const float*>(base + o_thr);
    cb->dev.tk = base + o_tk;
    cb->dev.cmag = reinterpret_cast<const float*>(base + o_cm);
    cb->dev.guess = base + o_gs;
    cb->dev.neg_limit = cb->host.folded ? cb->host.neg_limit : 0.0f;
    cb->status = reinterpret_cast<int*>(cb->blob) + (words - 4);
    *out = cb;
    return BQ_OK;
}

int bq_free_codebook(bq_codebook* cb) {
    if (!cb) return BQ_OK;
    cudaError_t e = cudaFree(cb->blob);
    delete cb;
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bq_codebook_is_folded(const bq_codebook* cb) { return (cb && cb->host.folded) ? 1 : 0; }

int bq_debug_build(void) { return bqd::kOn ? 1 : 0; }

int bq_set_staging(int on) { return g_staging.exchange(on ? 1 : 0); }

int bq_kernel_status(const bq_codebook* cb, int* status_out) {
    if (!cb || !status_out) return BQ_ERR_NULL;
    if (!on_codebook_device_c(cb)) return BQ_ERR_CODEBOOK;
    int host[2] = {0, 0};
    cudaError_t e = cudaMemcpy(host, cb->status, sizeof(int), cudaMemcpyDeviceToHost);      // waits for the device's earlier work
    if (e == cudaSuccess && host[0] != 0) e = cudaMemset(cb->status, 0, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    *status_out = host[0];
    return BQ_OK;
}

}  // extern "C"

namespace {

// The handle's tables live on the device that was current when it was made; a call from
// another current device would hand the kernels pointers they cannot reach.
bool on_codebook_device(const bq_codebook* cb) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == cb->device;
}

// Shared body of bq_quantize and bq_roundtrip.
int forward(const void* x, int xdt, size_t n, int block, const bq_codebook* cb, void* y, int ydt, bool write_y,
            uint8_t* codes, float* absmax, bool write_q, cudaStream_t stream) {
    const size_t B = size_t(block);
    size_t done = 0;        // elements covered by the tuned kernel
    {
        const size_t xs = n * elem_bytes(xdt), ys = write_y ? n * elem_bytes(ydt) : 0, cs = write_q ? n : 0;
        const size_t as = write_q ? ((n + B - 1) / B) * sizeof(float) : 0;
        BQ_ASSERT(!write_y || y == x || bqd::disjoint(x, xs, y, ys));          // in place, or apart
        BQ_ASSERT(!write_y || y != x || xdt == ydt);
        BQ_ASSERT(bqd::disjoint(x, xs, codes, cs) && bqd::disjoint(x, xs, absmax, as));
        BQ_ASSERT(bqd::disjoint(y, ys, codes, cs) && bqd::disjoint(y, ys, absmax, as) && bqd::disjoint(codes, cs, absmax, as));
    }
    const bool can_tune = cb->host.folded && tuned_block(block) && aligned(x, 16) && (!write_y || (aligned(y, 16) && ydt == xdt)) &&
                          (!write_q || (aligned(codes, 8) && aligned(absmax, 4)));
    if (can_tune && n >= B && g_staging.load() && (block == 2048 || block == 4096)) {
        // the staged kernel takes every whole block; the short last block, if any, goes to the general kernel below
        bool taken = false;
        cudaError_t e = bql::launch_fwd_staged(xdt, block, write_y, write_q, x, y, codes, absmax, n / B, cb->dev, cb->sm_count, cb->device,
                                               cb->status, stream, &taken);
        if (e != cudaSuccess) return cuda_fail(e);
        if (taken) done = (n / B) * B;
    }
    if (can_tune && n >= B && done == 0) {
        const size_t n_full = (n / B) * B;
        cudaError_t e = bql::launch_fwd_fast(xdt, block, write_y, write_q, x, y, codes, absmax, n_full, cb->dev, cb->sm_count, cb->device, stream,
                                             &done);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    BQ_ASSERT(done % B == 0 && done <= n);                                   // the general kernel starts on a block border
    if (done < n) {
        cudaError_t e = bql::launch_fwd_general(xdt, ydt, write_y, write_q, x, y, codes, absmax, n, B, done / B, cb->dev, cb->sm_count, stream);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return BQ_OK;
}

}  // namespace

extern "C" {

int bq_quantize(const void* x, bq_dtype xdt, size_t n, int block, const bq_codebook* cb, uint8_t* codes_out, float* absmax_out,
                void* cuda_stream) {
    if (!known_dtype(xdt)) return BQ_ERR_DTYPE;
    if (block < 1) return BQ_ERR_BLOCK;
    if (n >= kMaxElems) return BQ_ERR_SIZE;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (n == 0) return BQ_OK;
    if (!x || !codes_out || !absmax_out) return BQ_ERR_NULL;
    if (!on_codebook_device(cb)) return BQ_ERR_CODEBOOK;
    return forward(x, xdt, n, block, cb, nullptr, xdt, false, codes_out, absmax_out, true, static_cast<cudaStream_t>(cuda_stream));
}

int bq_roundtrip(const void* x, bq_dtype xdt, size_t n, int block, const bq_codebook* cb, void* y_out, bq_dtype ydt, uint8_t* codes_out,
                 float* absmax_out, void* cuda_stream) {
    if (!known_dtype(xdt) || !known_dtype(ydt)) return BQ_ERR_DTYPE;
    if (block < 1) return BQ_ERR_BLOCK;
    if (n >= kMaxElems) return BQ_ERR_SIZE;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (n == 0) return BQ_OK;
    if (!x || !y_out) return BQ_ERR_NULL;
    if ((codes_out == nullptr) != (absmax_out == nullptr)) return BQ_ERR_NULL;
    if (!on_codebook_device(cb)) return BQ_ERR_CODEBOOK;
    return forward(x, xdt, n, block, cb, y_out, ydt, true, codes_out, absmax_out, codes_out != nullptr,
                   static_cast<cudaStream_t>(cuda_stream));
}

int bq_dequantize(const uint8_t* codes, const float* absmax, size_t n, int block, const bq_codebook* cb, void* y_out, bq_dtype ydt,
                  void* cuda_stream) {
    if (!known_dtype(ydt)) return BQ_ERR_DTYPE;
    if (block < 1) return BQ_ERR_BLOCK;
    if (n >= kMaxElems) return BQ_ERR_SIZE;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (n == 0) return BQ_OK;
    if (!codes || !absmax || !y_out) return BQ_ERR_NULL;
    if (!on_codebook_device(cb)) return BQ_ERR_CODEBOOK;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t B = size_t(block);
    size_t done = 0;
    {
        const size_t ys = n * elem_bytes(ydt), as = ((n + B - 1) / B) * sizeof(float);
        BQ_ASSERT(bqd::disjoint(y_out, ys, codes, n) && bqd::disjoint(y_out, ys, absmax, as));
    }
    const int l2 = log2_exact(B);
    if (l2 >= 4 && aligned(codes, 16) && aligned(y_out, 16) && n >= 16) {
        const size_t n16 = n / 16;
        cudaError_t e = bql::launch_deq_fast(ydt, codes, absmax, y_out, n16, l2, cb->dev, cb->sm_count, cb->device, stream);
        if (e != cudaSuccess) return cuda_fail(e);
        done = n16 * 16;
    }
    BQ_ASSERT(done % 16 == 0 && done <= n);
    if (done < n) {
        cudaError_t e = bql::launch_deq_general(ydt, codes, absmax, y_out, n, B, done, cb->dev, cb->sm_count, stream);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return BQ_OK;
}

}  // extern "C"

static bool on_codebook_device_c(const bq_codebook* cb) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == cb->device;
}
