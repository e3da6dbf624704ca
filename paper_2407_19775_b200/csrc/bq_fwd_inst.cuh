// bq_fwd_inst.cuh -- body shared by the per-type instantiation files of the tuned forward
// kernel.  Each including file defines BQ_INST_DT and BQ_INST_NAME first.
#include "bq_launch.h"

namespace bql {
namespace {

#ifndef BQ_NT
#define BQ_NT 384
#endif
#ifndef BQ_RMAX
#define BQ_RMAX 8
#endif
constexpr int kNT = BQ_NT;

// Tile shape per block size: R chunks per thread, TW warps per block.
template <int XDT, int B, int RMAX> struct Shape {
    static constexpr int ROW = 32 * bqk::Elem<XDT>::kPerChunk;
    static constexpr bool IN_ROW = B <= ROW;
    static constexpr int ROWS = IN_ROW ? RMAX : B / ROW;       // rows of one block (any number when blocks fit in a row)
    static constexpr int R = RMAX;                             // a warp holds RMAX rows: several blocks, one, or a share of one
    static constexpr int TW = (IN_ROW || ROWS <= RMAX) ? 1 : ROWS / RMAX;
};

// Below this many elements the per-CTA table set-up of the tuned kernel (193 KB of shared
// memory to fill) costs more than it saves; the LITE kernels read the tables through L1.
#ifndef BQ_LITE_MAX_LOG2
#define BQ_LITE_MAX_LOG2 23
#endif
constexpr size_t kLiteMaxElems = size_t(1) << BQ_LITE_MAX_LOG2;

// Launches the tuned kernel on the leading whole tiles and reports how many elements it covered.
template <int XDT, int B, bool WY, bool WQ>
cudaError_t go(const void* x, void* y, uint8_t* codes, float* absmax, size_t n_full, const bqk::DeviceTables& tab, int sm_count,
               int device, cudaStream_t stream, size_t* done) {
    if (n_full <= kLiteMaxElems) {
        // small tiles and small CTAs, so that even a decode-step tensor spreads over all SMs
        using S = Shape<XDT, B, (B <= 32 * bqk::Elem<XDT>::kPerChunk) ? 2 : 4>;
        constexpr int kLiteNT = 32 * (S::TW > 4 ? S::TW : 4);
        const size_t tile = size_t(S::TW) * S::R * S::ROW;
        const size_t ntiles = n_full / tile;
        *done = ntiles * tile;
        if (ntiles == 0) return cudaSuccess;
        constexpr auto kernel = bqk::fwd_fast<XDT, B, S::R, S::TW, WY, WQ, kLiteNT, true>;
        const size_t teams = (kLiteNT / 32) / S::TW;
        const size_t grid = (ntiles + teams - 1) / teams;
        kernel<<<unsigned(grid), kLiteNT, bqk::kFwdLiteSmemBytes, stream>>>(x, y, codes, absmax, ntiles, tab);
        return cudaGetLastError();
    }
    using S = Shape<XDT, B, BQ_RMAX>;
    const size_t tile = size_t(S::TW) * S::R * S::ROW;
    const size_t ntiles = n_full / tile;
    *done = ntiles * tile;
    if (ntiles == 0) return cudaSuccess;
    constexpr auto kernel = bqk::fwd_fast<XDT, B, S::R, S::TW, WY, WQ, kNT, false>;
    cudaError_t e = allow_smem<kernel>(int(bqk::kFwdSmemBytes), device);
    if (e != cudaSuccess) return e;
    const size_t teams = (kNT / 32) / S::TW;
    size_t grid = (ntiles + teams - 1) / teams;
    if (grid > size_t(sm_count)) grid = size_t(sm_count);
    kernel<<<unsigned(grid), kNT, bqk::kFwdSmemBytes, stream>>>(x, y, codes, absmax, ntiles, tab);
    return cudaGetLastError();
}

template <int XDT, int B>
cudaError_t by_mode(bool wy, bool wq, const void* x, void* y, uint8_t* codes, float* absmax, size_t n_full,
                    const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream, size_t* done) {
    if (wy && wq) return go<XDT, B, true, true>(x, y, codes, absmax, n_full, tab, sm_count, device, stream, done);
    if (wy) return go<XDT, B, true, false>(x, y, codes, absmax, n_full, tab, sm_count, device, stream, done);
    return go<XDT, B, false, true>(x, y, codes, absmax, n_full, tab, sm_count, device, stream, done);
}

}  // namespace

cudaError_t BQ_INST_NAME(int block, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax, size_t n_full,
                         const bqk::DeviceTables& tab, int sm_count, int device, cudaStream_t stream, size_t* done) {
    switch (block) {
#define BQ_CASE(BB) case BB: return by_mode<BQ_INST_DT, BB>(write_y, write_q, x, y, codes, absmax, n_full, tab, sm_count, device, stream, done);
        BQ_CASE(64) BQ_CASE(128) BQ_CASE(256) BQ_CASE(512) BQ_CASE(1024) BQ_CASE(2048) BQ_CASE(4096)
#undef BQ_CASE
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace bql
