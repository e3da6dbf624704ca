// bq_launch.h -- launchers of the kernel instantiations (internal to libbq).
#pragma once

#include <cuda_runtime.h>

#include <mutex>

#include "../../include/bq.h"
#include "bq_kernels.cuh"
#include "bq_tables.h"

namespace bql {

// Tuned forward kernels, one translation unit per element type.  n_full is a whole number of
// blocks; *done receives how many leading elements were handled (whole tiles only).
cudaError_t launch_fwd_fast_f32(int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax,
                                size_t n_full, const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream, size_t* done);
cudaError_t launch_fwd_fast_f16(int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax,
                                size_t n_full, const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream, size_t* done);
cudaError_t launch_fwd_fast_bf16(int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax,
                                 size_t n_full, const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream, size_t* done);

inline cudaError_t launch_fwd_fast(int xdt, int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes,
                                   float* absmax, size_t n_full, const bqk::DeviceTables& tab, int sm_count, int device,
                                   cudaStream_t stream, size_t* done) {
    switch (xdt) {
        case BQ_F32: return launch_fwd_fast_f32(block, write_y, write_q, x, y, codes, absmax, n_full, tab, sm_count, device, stream, done);
        case BQ_F16: return launch_fwd_fast_f16(block, write_y, write_q, x, y, codes, absmax, n_full, tab, sm_count, device, stream, done);
        default: return launch_fwd_fast_bf16(block, write_y, write_q, x, y, codes, absmax, n_full, tab, sm_count, device, stream, done);
    }
}

// The shared-memory-staged forward kernel (blocks of 2048 and 4096 elements whose ring fits beside the tables): all
// `nblocks` whole blocks; *taken says whether this shape has such a kernel.  `status` is the codebook's device word that a
// wait which ran out sets.
cudaError_t launch_fwd_staged(int xdt, int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax,
                              size_t nblocks, const bqk::DeviceTables& tab, int sm_count, int device, int* status, cudaStream_t stream,
                              bool* taken);

// The forward kernel's 4-bit flavour on the leading whole tiles of n_full elements (whole blocks; 16-bit inputs, blocks of
// 64 .. 4096): packed receives two codes per byte, absmax one float per block (with scale16: one bf16, the absmax rounded
// up, in 16-bit words); *done = elements covered (0: not taken).
cudaError_t launch_fwd4_fast(int xdt, int block, bool scale16, const void* x, uint8_t* packed, float* absmax, size_t n_full,
                             const bqk::Tables4Fast& tab, int sm_count, int device, cudaStream_t stream, size_t* done);

cudaError_t launch_fwd_general(int xdt, int ydt, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax,
                               size_t n, size_t block, size_t first_block, const bqk::DeviceTables& tab, int sm_count,
                               cudaStream_t stream);
cudaError_t launch_deq_fast(int ydt, const uint8_t* codes, const float* absmax, void* y, size_t n16, int log2_block,
                            const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream);
cudaError_t launch_deq_general(int ydt, const uint8_t* codes, const float* absmax, void* y, size_t n, size_t block, size_t first_elem,
                               const bqk::DeviceTables& tab, int sm_count, cudaStream_t stream);

// Kernels that need more than 48 KB of dynamic shared memory must opt in once per device.
// The per-device "already done" table is written under a lock (two host threads may make their
// first call together); a device beyond the table simply opts in on every call.
template <auto Kernel>
inline cudaError_t allow_smem(int bytes, int device) {
    static std::mutex lock;
    static bool done[64] = {};
    const bool tracked = device >= 0 && device < 64;
    std::lock_guard<std::mutex> guard(lock);
    if (tracked && done[device]) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && tracked) done[device] = true;
    return e;
}

}  // namespace bql
