// bq_fwd_inst.cuh -- body shared by the per-type instantiation files of the tuned forward
// kernel.  Each including file defines BQ_INST_DT and BQ_INST_NAME first.
#include "bq_launch.h"

namespace bql {
namespace {

#ifndef BQ_NT
#define BQ_NT 512
#endif
#ifndef BQ_RMAX
#define BQ_RMAX 4
#endif
constexpr int kNT = BQ_NT;

// Tile shape per block size: R chunks per thread, TW warps per block.
template <int XDT, int B> struct Shape {
    static constexpr int ROW = 32 * bqk::Elem<XDT>::kPerChunk;
    static constexpr bool IN_ROW = B <= ROW;
    static constexpr int ROWS = IN_ROW ? BQ_RMAX : B / ROW;    // rows one tile must cover
    static constexpr int R = ROWS <= BQ_RMAX ? ROWS : BQ_RMAX;
    static constexpr int TW = IN_ROW ? 1 : ROWS / R;
};

template <int XDT, int B, bool WY, bool WQ>
cudaError_t go(const void* x, void* y, uint8_t* codes, float* absmax, size_t n_full, const bqk::DeviceTables& tab, int sm_count,
               int device, cudaStream_t stream) {
    using S = Shape<XDT, B>;
    constexpr auto kernel = bqk::fwd_fast<XDT, B, S::R, S::TW, WY, WQ, kNT>;
    cudaError_t e = allow_smem<kernel>(int(bqk::kFwdSmemBytes), device);
    if (e != cudaSuccess) return e;
    const size_t tile = size_t(S::TW) * S::R * S::ROW;
    const size_t ntiles = (n_full + tile - 1) / tile;
    const size_t teams = (kNT / 32) / S::TW;
    size_t grid = (ntiles + teams - 1) / teams;
    if (grid > size_t(sm_count)) grid = size_t(sm_count);
    kernel<<<unsigned(grid), kNT, bqk::kFwdSmemBytes, stream>>>(x, y, codes, absmax, n_full, tab);
    return cudaGetLastError();
}

template <int XDT, int B>
cudaError_t by_mode(bool wy, bool wq, const void* x, void* y, uint8_t* codes, float* absmax, size_t n_full,
                    const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream) {
    if (wy && wq) return go<XDT, B, true, true>(x, y, codes, absmax, n_full, tab, sm_count, device, stream);
    if (wy) return go<XDT, B, true, false>(x, y, codes, absmax, n_full, tab, sm_count, device, stream);
    return go<XDT, B, false, true>(x, y, codes, absmax, n_full, tab, sm_count, device, stream);
}

}  // namespace

cudaError_t BQ_INST_NAME(int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax, size_t n_full,
                         const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream) {
    switch (block) {
#define BQ_CASE(BB) case BB: return by_mode<BQ_INST_DT, BB>(write_y, write_q, x, y, codes, absmax, n_full, tab, sm_count, device, stream);
        BQ_CASE(64) BQ_CASE(128) BQ_CASE(256) BQ_CASE(512) BQ_CASE(1024) BQ_CASE(2048) BQ_CASE(4096)
#undef BQ_CASE
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace bql
