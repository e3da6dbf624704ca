// The forward kernel in its 4-bit flavour (16 codes, two per byte): instantiations for 16-bit inputs and the launcher
// the 4-bit calls use for large tensors.
#include "bq_launch.h"

namespace bql {
namespace {

constexpr int kNT = 384;
constexpr int kR = 8;

template <int XDT, int B, bool S16>
cudaError_t go(const void* x, uint8_t* packed, float* absmax, size_t n_full, const bqk::Tables4Fast& tab, int sm_count, int device,
               cudaStream_t stream, size_t* done) {
    constexpr int ROW = 32 * bqk::Elem<XDT>::kPerChunk;
    constexpr bool IN_ROW = B <= ROW;                           // tile shape only: a one-row block and an in-row block both take kR rows per warp
    constexpr int ROWS = IN_ROW ? kR : B / ROW;
    constexpr int TW = (IN_ROW || ROWS <= kR) ? 1 : ROWS / kR;
    const size_t tile = size_t(TW) * kR * ROW;
    const size_t ntiles = n_full / tile;
    *done = ntiles * tile;
    if (ntiles == 0) return cudaSuccess;
    constexpr auto kernel = bqk::fwd_fast<XDT, B, kR, TW, false, true, kNT, false, 4, S16>;
    const size_t teams = (kNT / 32) / TW;
    size_t grid = (ntiles + teams - 1) / teams;
    if (grid > size_t(sm_count)) grid = size_t(sm_count);
    (void)device;                                                // 10 KB of shared memory: no opt-in needed
    kernel<<<unsigned(grid), kNT, bqk::kFwd4SmemBytes, stream>>>(x, nullptr, packed, absmax, ntiles, tab);
    return cudaGetLastError();
}

template <int XDT, bool S16>
cudaError_t by_block(int block, const void* x, uint8_t* packed, float* absmax, size_t n_full, const bqk::Tables4Fast& tab, int sm_count,
                     int device, cudaStream_t stream, size_t* done) {
    switch (block) {
#define BQ_CASE(BB) case BB: return go<XDT, BB, S16>(x, packed, absmax, n_full, tab, sm_count, device, stream, done);
        BQ_CASE(64) BQ_CASE(128) BQ_CASE(256) BQ_CASE(512) BQ_CASE(1024) BQ_CASE(2048) BQ_CASE(4096)
#undef BQ_CASE
        default: *done = 0; return cudaSuccess;
    }
}

}  // namespace

cudaError_t launch_fwd4_fast(int xdt, int block, bool scale16, const void* x, uint8_t* packed, float* absmax, size_t n_full,
                             const bqk::Tables4Fast& tab, int sm_count, int device, cudaStream_t stream, size_t* done) {
    *done = 0;
    if (xdt == BQ_F16) return scale16 ? by_block<bqk::kF16, true>(block, x, packed, absmax, n_full, tab, sm_count, device, stream, done)
                                      : by_block<bqk::kF16, false>(block, x, packed, absmax, n_full, tab, sm_count, device, stream, done);
    if (xdt == BQ_BF16) return scale16 ? by_block<bqk::kBF16, true>(block, x, packed, absmax, n_full, tab, sm_count, device, stream, done)
                                       : by_block<bqk::kBF16, false>(block, x, packed, absmax, n_full, tab, sm_count, device, stream, done);
    return cudaSuccess;                                          // fp32 inputs stay with the 4-bit kernels of their own
}

}  // namespace bql
