// Instantiations and launcher of the shared-memory-staged forward kernel (blocks of 2048 and 4096).
#include "bq_launch.h"
#include "bq_staged.cuh"

namespace bql {
namespace {

// Teams and stages per block size: the rings take what the per-lane tables leave of a CTA's
// shared memory (about 32 KB): 2048-element blocks of a 16-bit type are 4 KB each.
template <int XDT, int B> struct StagedShape {
    static constexpr int kBlockBytes = B * bqk::Elem<XDT>::kBytes;
    static constexpr int TEAMS = (kBlockBytes <= 4096) ? 3 : 2;
    static constexpr int STAGES = (32 * 1024) / (TEAMS * kBlockBytes) >= 2 ? (32 * 1024) / (TEAMS * kBlockBytes) : 0;
    static constexpr bool kFits = STAGES >= 2;
};

template <int XDT, int B, bool WY, bool WQ>
cudaError_t go(const void* x, void* y, uint8_t* codes, float* absmax, size_t nblocks, const bqk::DeviceTables& tab, int sm_count, int device,
               int* status, cudaStream_t stream, bool* taken) {
    using S = StagedShape<XDT, B>;
    if constexpr (!S::kFits) {
        *taken = false;                                          // fp32 blocks of 4096 elements: two stages per team do not fit
        return cudaSuccess;
    } else {
        constexpr int STAGES = S::STAGES > 4 ? 4 : S::STAGES;
        using Cfg = bqk::StagedCfg<XDT, B, S::TEAMS, STAGES>;
        constexpr auto kernel = bqk::fwd_staged<XDT, B, S::TEAMS, STAGES, WY, WQ>;
        cudaError_t e = allow_smem<kernel>(int(Cfg::kSmemBytes), device);
        if (e != cudaSuccess) return e;
        size_t grid = (nblocks + S::TEAMS - 1) / S::TEAMS;
        if (grid > size_t(sm_count)) grid = size_t(sm_count);
        kernel<<<unsigned(grid), S::TEAMS * bqk::kTeamThreads, Cfg::kSmemBytes, stream>>>(x, y, codes, absmax, nblocks, tab, status);
        *taken = true;
        return cudaGetLastError();
    }
}

template <int XDT, int B>
cudaError_t by_mode(bool wy, bool wq, const void* x, void* y, uint8_t* codes, float* absmax, size_t nblocks, const bqk::DeviceTables& tab,
                    int sm_count, int device, int* status, cudaStream_t stream, bool* taken) {
    if (wy && wq) return go<XDT, B, true, true>(x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
    if (wy) return go<XDT, B, true, false>(x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
    return go<XDT, B, false, true>(x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
}

template <int XDT>
cudaError_t by_block(int block, bool wy, bool wq, const void* x, void* y, uint8_t* codes, float* absmax, size_t nblocks,
                     const bqk::DeviceTables& tab, int sm_count, int device, int* status, cudaStream_t stream, bool* taken) {
    if (block == 2048) return by_mode<XDT, 2048>(wy, wq, x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
    if (block == 4096) return by_mode<XDT, 4096>(wy, wq, x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
    *taken = false;
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_fwd_staged(int xdt, int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax,
                              size_t nblocks, const bqk::DeviceTables& tab, int sm_count, int device, int* status, cudaStream_t stream,
                              bool* taken) {
    switch (xdt) {
        case BQ_F32: return by_block<bqk::kF32>(block, write_y, write_q, x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
        case BQ_F16: return by_block<bqk::kF16>(block, write_y, write_q, x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
        default: return by_block<bqk::kBF16>(block, write_y, write_q, x, y, codes, absmax, nblocks, tab, sm_count, device, status, stream, taken);
    }
}

}  // namespace bql
