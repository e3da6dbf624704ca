// General (any block / alignment / codebook) kernels and the tuned dequantize kernel.
#include "bq_launch.h"

namespace bql {
namespace {

template <int XDT, int YDT>
cudaError_t fwd_general_mode(bool wy, bool wq, const void* x, void* y, uint8_t* codes, float* absmax, size_t n, size_t block,
                             size_t first_block, const bqk::DeviceTables& tab, unsigned grid, cudaStream_t stream) {
    if (wy && wq) bqk::fwd_general<XDT, YDT, true, true><<<grid, 256, 0, stream>>>(x, y, codes, absmax, n, block, first_block, tab);
    else if (wy) bqk::fwd_general<XDT, YDT, true, false><<<grid, 256, 0, stream>>>(x, y, codes, absmax, n, block, first_block, tab);
    else bqk::fwd_general<XDT, YDT, false, true><<<grid, 256, 0, stream>>>(x, y, codes, absmax, n, block, first_block, tab);
    return cudaGetLastError();
}

template <int XDT>
cudaError_t fwd_general_y(int ydt, bool wy, bool wq, const void* x, void* y, uint8_t* codes, float* absmax, size_t n, size_t block,
                          size_t first_block, const bqk::DeviceTables& tab, unsigned grid, cudaStream_t stream) {
    switch (ydt) {
        case BQ_F32: return fwd_general_mode<XDT, bqk::kF32>(wy, wq, x, y, codes, absmax, n, block, first_block, tab, grid, stream);
        case BQ_F16: return fwd_general_mode<XDT, bqk::kF16>(wy, wq, x, y, codes, absmax, n, block, first_block, tab, grid, stream);
        default: return fwd_general_mode<XDT, bqk::kBF16>(wy, wq, x, y, codes, absmax, n, block, first_block, tab, grid, stream);
    }
}

#ifndef BQ_LITE_MAX_LOG2
#define BQ_LITE_MAX_LOG2 21
#endif
#ifndef BQ_DEQ_NT
#define BQ_DEQ_NT 512
#endif
#ifndef BQ_DEQ_U
#define BQ_DEQ_U 2
#endif
#ifndef BQ_DEQ_CTAS
#define BQ_DEQ_CTAS 3
#endif
constexpr int kDeqNT = BQ_DEQ_NT;
constexpr int kDeqU = BQ_DEQ_U;

template <int YDT, bool WIDE>
cudaError_t deq_fast_go(const uint8_t* codes, const float* absmax, void* y, size_t n16, int log2_block, const bqk::DeviceTables& tab,
                        int sm_count, cudaStream_t stream) {
    if (n16 <= (size_t(1) << (BQ_LITE_MAX_LOG2 + 2 - 4))) {      // up to 8 Mi elements: one plain copy of the values, one chunk per thread
        const size_t grid = (n16 + 255) / 256;
        bqk::deq_fast<YDT, 256, 1, true, WIDE><<<unsigned(grid), 256, bqk::kDeqLiteSmemBytes, stream>>>(codes, absmax, y, n16, log2_block, tab);
        return cudaGetLastError();
    }
    const size_t tile = size_t(kDeqNT) * kDeqU;
    size_t grid = (n16 + tile - 1) / tile;
    const size_t cap = size_t(sm_count) * BQ_DEQ_CTAS;
    if (grid > cap) grid = cap;
    bqk::deq_fast<YDT, kDeqNT, kDeqU, false, WIDE><<<unsigned(grid), kDeqNT, bqk::kDeqSmemBytes, stream>>>(codes, absmax, y, n16, log2_block, tab);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_general(int xdt, int ydt, bool write_y, bool write_q, const void* x, void* y, uint8_t* codes, float* absmax,
                               size_t n, size_t block, size_t first_block, const bqk::DeviceTables& tab, int sm_count,
                               cudaStream_t stream) {
    const size_t nb = (n + block - 1) / block - first_block;
    size_t grid = (nb + 7) / 8;
    const size_t cap = size_t(sm_count) * 8;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    switch (xdt) {
        case BQ_F32: return fwd_general_y<bqk::kF32>(ydt, write_y, write_q, x, y, codes, absmax, n, block, first_block, tab, unsigned(grid), stream);
        case BQ_F16: return fwd_general_y<bqk::kF16>(ydt, write_y, write_q, x, y, codes, absmax, n, block, first_block, tab, unsigned(grid), stream);
        default: return fwd_general_y<bqk::kBF16>(ydt, write_y, write_q, x, y, codes, absmax, n, block, first_block, tab, unsigned(grid), stream);
    }
}

cudaError_t launch_deq_fast(int ydt, const uint8_t* codes, const float* absmax, void* y, size_t n16, int log2_block,
                            const bqk::DeviceTables& tab, int sm_count, int /*device*/, cudaStream_t stream) {
    // the 256-bit stores of the kernel need y on a 32-byte boundary; a y that is only 16-byte
    // aligned (a tensor sliced at 8 16-bit elements, say) takes the variant with 128-bit stores
    const bool wide = (reinterpret_cast<uintptr_t>(y) & 31u) == 0;
    switch (ydt) {
#define BQ_DEQ_CASE(DT) (wide ? deq_fast_go<DT, true>(codes, absmax, y, n16, log2_block, tab, sm_count, stream) \
                              : deq_fast_go<DT, false>(codes, absmax, y, n16, log2_block, tab, sm_count, stream))
        case BQ_F32: return BQ_DEQ_CASE(bqk::kF32);
        case BQ_F16: return BQ_DEQ_CASE(bqk::kF16);
        default: return BQ_DEQ_CASE(bqk::kBF16);
#undef BQ_DEQ_CASE
    }
}

cudaError_t launch_deq_general(int ydt, const uint8_t* codes, const float* absmax, void* y, size_t n, size_t block, size_t first_elem,
                               const bqk::DeviceTables& tab, int sm_count, cudaStream_t stream) {
    size_t grid = (n - first_elem + 255) / 256;
    const size_t cap = size_t(sm_count) * 8;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    switch (ydt) {
        case BQ_F32: bqk::deq_general<bqk::kF32><<<unsigned(grid), 256, 0, stream>>>(codes, absmax, y, n, block, first_elem, tab); break;
        case BQ_F16: bqk::deq_general<bqk::kF16><<<unsigned(grid), 256, 0, stream>>>(codes, absmax, y, n, block, first_elem, tab); break;
        default: bqk::deq_general<bqk::kBF16><<<unsigned(grid), 256, 0, stream>>>(codes, absmax, y, n, block, first_elem, tab); break;
    }
    return cudaGetLastError();
}

}  // namespace bql
