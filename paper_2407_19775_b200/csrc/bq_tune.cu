// Block-size selection (include/bq_tune.h): the reconstruction error of the 8-bit roundtrip for
// a list of candidate block sizes, and the host rule that picks one.
//
// Per candidate: bq_roundtrip into the scratch copy, then sq_sums (1024 CTAs, each thread sums
// its grid-stride share in fp64, a shared-memory tree per CTA) and sq_final (one CTA adds the 1024
// partial sums in a fixed tree).  HBM-bound: the roundtrip moves 2 n s bytes, the sums read 2 n s.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "bq_error.h"
#include "bq_tune.h"

namespace {

constexpr int kGrid = 1024;                                      // fixed: the summation order must not depend on the device
constexpr int kThreads = 256;
constexpr size_t kPartialBytes = size_t(kGrid) * 2 * sizeof(double);

__host__ __device__ inline size_t round_up_256(size_t v) { return (v + 255) & ~size_t(255); }

template <int DT> struct Elem;
template <> struct Elem<BQ_F32> { using type = float; static constexpr int kPerVec = 4; };
template <> struct Elem<BQ_F16> { using type = __half; static constexpr int kPerVec = 8; };
template <> struct Elem<BQ_BF16> { using type = __nv_bfloat16; static constexpr int kPerVec = 8; };

template <int DT>
__device__ __forceinline__ double widen_d(const typename Elem<DT>::type& v) {
    if constexpr (DT == BQ_F32) return double(v);
    else if constexpr (DT == BQ_F16) return double(__half2float(v));
    else return double(__bfloat162float(v));
}

template <int DT>
__device__ __forceinline__ void add_terms(const typename Elem<DT>::type& xv, const typename Elem<DT>::type& yv, double& err, double& norm) {
    const double xd = widen_d<DT>(xv), d = xd - widen_d<DT>(yv);  // the difference of two such values is exact in fp64
    err = __fma_rn(d, d, err);
    norm = __fma_rn(xd, xd, norm);
}

// partial[2 b] = this CTA's share of sum (x - y)^2, partial[2 b + 1] = its share of sum x^2
template <int DT, bool VEC>
__global__ void __launch_bounds__(kThreads)
sq_sums(const void* __restrict__ xp, const void* __restrict__ yp, size_t n, double* __restrict__ partial) {
    using T = typename Elem<DT>::type;
    constexpr int V = Elem<DT>::kPerVec;
    const T* x = static_cast<const T*>(xp);
    const T* y = static_cast<const T*>(yp);
    double err = 0.0, norm = 0.0;
    const size_t tid = size_t(blockIdx.x) * kThreads + threadIdx.x, stride = size_t(kGrid) * kThreads;
    if constexpr (VEC) {
        const size_t nvec = n / V;
        for (size_t c = tid; c < nvec; c += stride) {
            const uint4 xw = __ldg(reinterpret_cast<const uint4*>(x) + c), yw = __ldg(reinterpret_cast<const uint4*>(y) + c);
            const T* xe = reinterpret_cast<const T*>(&xw);
            const T* ye = reinterpret_cast<const T*>(&yw);
#pragma unroll
            for (int i = 0; i < V; ++i) add_terms<DT>(xe[i], ye[i], err, norm);
        }
        for (size_t i = nvec * V + tid; i < n; i += stride) add_terms<DT>(x[i], y[i], err, norm);
    } else {
        for (size_t i = tid; i < n; i += stride) add_terms<DT>(x[i], y[i], err, norm);
    }
    __shared__ double se[kThreads], sn[kThreads];
    se[threadIdx.x] = err;
    sn[threadIdx.x] = norm;
    __syncthreads();
    for (int s = kThreads / 2; s >= 1; s >>= 1) {
        if (threadIdx.x < s) {
            se[threadIdx.x] += se[threadIdx.x + s];
            sn[threadIdx.x] += sn[threadIdx.x + s];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        partial[2 * blockIdx.x] = se[0];
        partial[2 * blockIdx.x + 1] = sn[0];
    }
}

__global__ void __launch_bounds__(kThreads)
sq_final(const double* __restrict__ partial, double* __restrict__ err_out, double* __restrict__ norm_out /* may be null */) {
    __shared__ double se[kThreads], sn[kThreads];
    double err = 0.0, norm = 0.0;
    for (int b = threadIdx.x; b < kGrid; b += kThreads) {
        err += partial[2 * b];
        norm += partial[2 * b + 1];
    }
    se[threadIdx.x] = err;
    sn[threadIdx.x] = norm;
    __syncthreads();
    for (int s = kThreads / 2; s >= 1; s >>= 1) {
        if (threadIdx.x < s) {
            se[threadIdx.x] += se[threadIdx.x + s];
            sn[threadIdx.x] += sn[threadIdx.x + s];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        *err_out = se[0];
        if (norm_out) *norm_out = sn[0];
    }
}

template <int DT>
cudaError_t launch_sums(const void* x, const void* y, size_t n, double* partial, double* err_out, double* norm_out, cudaStream_t s) {
    const bool vec = (reinterpret_cast<uintptr_t>(x) % 16 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    if (vec) sq_sums<DT, true><<<kGrid, kThreads, 0, s>>>(x, y, n, partial);
    else sq_sums<DT, false><<<kGrid, kThreads, 0, s>>>(x, y, n, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    sq_final<<<1, kThreads, 0, s>>>(partial, err_out, norm_out);
    return cudaGetLastError();
}

int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}

size_t elem_bytes(bq_dtype dt) { return dt == BQ_F32 ? 4 : ((dt == BQ_F16 || dt == BQ_BF16) ? 2 : 0); }

}  // namespace

extern "C" {

size_t bqt_workspace_bytes(bq_dtype xdt, size_t n) {
    const size_t eb = elem_bytes(xdt);
    return eb ? round_up_256(n * eb) + kPartialBytes : 0;
}

int bqt_block_errors(const void* x, bq_dtype xdt, size_t n, const bq_codebook* cb, const int* blocks, int n_blocks,
                     void* workspace, size_t workspace_bytes, double* sums_out, void* cuda_stream) {
    if (elem_bytes(xdt) == 0) return BQ_ERR_DTYPE;
    if (!blocks || !sums_out) return BQ_ERR_NULL;
    if (n_blocks < 1 || n_blocks > BQT_MAX_CANDIDATES) return BQ_ERR_BLOCK;
    for (int c = 0; c < n_blocks; ++c)
        if (blocks[c] < 1) return BQ_ERR_BLOCK;
    if (!cb) return BQ_ERR_CODEBOOK;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (n == 0) {
        const cudaError_t e = cudaMemsetAsync(sums_out, 0, size_t(n_blocks + 1) * sizeof(double), s);
        return e == cudaSuccess ? BQ_OK : cuda_fail(e);
    }
    if (!x || !workspace) return BQ_ERR_NULL;
    if (workspace_bytes < bqt_workspace_bytes(xdt, n) || reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return BQ_ERR_SIZE;
    void* y = workspace;
    double* partial = reinterpret_cast<double*>(static_cast<unsigned char*>(workspace) + round_up_256(n * elem_bytes(xdt)));
    for (int c = 0; c < n_blocks; ++c) {
        const int rc = bq_roundtrip(x, xdt, n, blocks[c], cb, y, xdt, nullptr, nullptr, cuda_stream);
        if (rc != BQ_OK) return rc;
        double* norm_out = (c == 0) ? sums_out + n_blocks : nullptr;
        cudaError_t e;
        switch (xdt) {
            case BQ_F32: e = launch_sums<BQ_F32>(x, y, n, partial, sums_out + c, norm_out, s); break;
            case BQ_F16: e = launch_sums<BQ_F16>(x, y, n, partial, sums_out + c, norm_out, s); break;
            default: e = launch_sums<BQ_BF16>(x, y, n, partial, sums_out + c, norm_out, s); break;
        }
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return BQ_OK;
}

int bqt_pick_block(const int* blocks, const double* sums, int n_blocks, double max_rel_rms, int* block_out) {
    if (!blocks || !sums || !block_out) return BQ_ERR_NULL;
    if (n_blocks < 1 || n_blocks > BQT_MAX_CANDIDATES) return BQ_ERR_BLOCK;
    for (int c = 0; c < n_blocks; ++c)
        if (blocks[c] < 1) return BQ_ERR_BLOCK;
    if (!(max_rel_rms >= 0.0) || !std::isfinite(max_rel_rms)) return BQ_ERR_SIZE;
    const double bound = max_rel_rms * max_rel_rms * sums[n_blocks];
    int best = -1;
    for (int c = 0; c < n_blocks; ++c)
        if (sums[c] <= bound && (best < 0 || blocks[c] > blocks[best])) best = c;
    if (best < 0) {
        best = 0;
        for (int c = 1; c < n_blocks; ++c)
            if (sums[c] < sums[best] || (sums[c] == sums[best] && blocks[c] > blocks[best])) best = c;
    }
    *block_out = blocks[best];
    return BQ_OK;
}

}  // extern "C"
