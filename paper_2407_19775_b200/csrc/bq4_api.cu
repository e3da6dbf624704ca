// bq4_api.cu -- the C ABI of the 4-bit variant (see include/bq4.h): argument checks, the
// codebook handle (host memory only: the tables travel as a kernel parameter) and the choice
// of kernel.
#include "../../include/bq4.h"
#include "bq4_kernels.cuh"
#include "bq_debug.h"
#include "bq_launch.h"
#include "bq_error.h"

#include <cmath>
#include <cstring>
#include <limits>
#include <new>

struct bq4_codebook {
    bq4k::Tables4 tab;
};

namespace {

constexpr size_t kMaxElems = size_t(1) << 40;

bool known_dtype(int dt) { return dt == BQ_F32 || dt == BQ_F16 || dt == BQ_BF16; }
bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
int log2_exact(size_t v) {
    int l = 0;
    while ((size_t(1) << l) < v) ++l;
    return ((size_t(1) << l) == v) ? l : -1;
}
int cuda_fail(cudaError_t e) {
    bql::set_last_cuda_error(cudaGetErrorString(e));
    return BQ_ERR_CUDA;
}

// The 4-bit dynamic-tree map: decade k = 0..2 holds the midpoints of 2^k equal bins of [0.1, 1]
// scaled by 10^(k-2): (2^(k+1) + 9 (2j+1)) / (2^(k+1) 10^(3-k)), one double division of exact
// integers rounded once to fp32.  Plus 0 and 1.  They come out ascending decade by decade.
void dynamic_tree_values16(float out[16]) {
    float mags[7];
    int cnt = 0;
    double p10 = 1e3;
    for (int k = 0; k <= 2; ++k, p10 /= 10.0) {
        const double two = double(1 << (k + 1));
        for (int j = 0; j < (1 << k); ++j) mags[cnt++] = float((two + 9.0 * double(2 * j + 1)) / (two * p10));
    }
    for (int p = 0; p < 7; ++p) { out[8 + p] = mags[p]; out[6 - p] = -mags[p]; }
    out[7] = 0.0f;
    out[15] = 1.0f;
}

bool valid_user_values16(const float* v) {
    for (int i = 0; i < 16; ++i) {
        if (!std::isfinite(v[i]) || v[i] < -1.0f || v[i] > 1.0f) return false;
        if (i && !(v[i] > v[i - 1])) return false;
        if (v[i] != 0.0f && std::fabs(v[i]) < 5.9604644775390625e-8f) return false;      // 2^-24: keeps every midpoint exact in double
    }
    return true;
}

// Midpoints rounded toward -inf: for an fp32 xhat, t < xhat holds exactly when round_down(t) < xhat.
void build_thresholds(bq4k::Tables4& t) {
    for (int j = 0; j < 15; ++j) {
        const double mid = (double(t.val[j]) + double(t.val[j + 1])) / 2.0;               // exact
        float f = float(mid);
        if (double(f) > mid) f = std::nextafterf(f, -std::numeric_limits<float>::infinity());
        t.thr[j] = f;
    }
    t.thr[15] = std::numeric_limits<float>::infinity();
}

uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }

// The folded search tables (see Tables4); left invalid when the codebook does not mirror or two thresholds share a cell.
void build_folded(bq4k::Tables4& t) {
    t.folded = 0;
    std::memset(t.entry, 0, sizeof t.entry);
    t.neg_limit = 0.0f;
    if (t.val[7] != 0.0f) return;
    for (int j = 0; j < 7; ++j)
        if (t.val[j] != -t.val[14 - j]) return;
    uint32_t tk[8];
    for (int p = 0; p < 8; ++p) {
        const double mid = (double(t.val[7 + p]) + double(t.val[8 + p])) / 2.0;            // exact
        float f = float(mid);
        if (double(f) > mid) f = std::nextafterf(f, 0.0f);                                 // positive: toward zero = toward -inf
        tk[p] = 2u * f2u(f) + ((double(f) != mid) ? 1u : 0u);
        if (tk[p] <= bq4k::kFoldKeyLow || tk[p] >= 0x7F000000u) return;                    // must lie inside the table's span
    }
    for (int i = 0; i < bq4k::kFoldCells; ++i) {
        const uint32_t S = (bq4k::kFoldCellBase + uint32_t(i)) << 21;
        uint32_t p0 = 0, inside = 0, off = 0x1FFFFFu;
        for (int p = 0; p < 8; ++p) {
            if (tk[p] < S) ++p0;
            else if (tk[p] - S < (1u << 21)) { ++inside; off = tk[p] - S; }
        }
        if (inside > 1) return;
        if (inside == 1 && off == 0x1FFFFFu) return;                                       // would look like an empty cell
        t.entry[i] = (((7u + p0) << 24) | 0xE00000u | (0x1FFFFFu - off)) - S;
    }
    // negative side: P must not count the top midpoint (there is no code below -val[14]); xhat is clamped to the largest
    // magnitude whose odd key does not pass it
    {
        const uint32_t bits = (tk[7] - 1u) >> 1;
        float m;
        std::memcpy(&m, &bits, 4);
        t.neg_limit = -m;
    }
    t.folded = 1;
}

int sm_count_of_current(int* sms) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

unsigned capped(size_t want, size_t cap) { return unsigned(want < 1 ? 1 : (want > cap ? cap : want)); }

template <int DT, bool FOLDED, bool S16>
void launch_q4_fast_f(int log2_lpb, unsigned grid, cudaStream_t s, const void* x, uint8_t* packed, float* absmax, size_t nchunks,
                      const bq4k::Tables4& tab) {
    switch (log2_lpb) {
        case 0: bq4k::q4_fast<DT, FOLDED, 0, S16><<<grid, 256, 0, s>>>(x, packed, absmax, nchunks, tab); break;
        case 1: bq4k::q4_fast<DT, FOLDED, 1, S16><<<grid, 256, 0, s>>>(x, packed, absmax, nchunks, tab); break;
        case 2: bq4k::q4_fast<DT, FOLDED, 2, S16><<<grid, 256, 0, s>>>(x, packed, absmax, nchunks, tab); break;
        case 3: bq4k::q4_fast<DT, FOLDED, 3, S16><<<grid, 256, 0, s>>>(x, packed, absmax, nchunks, tab); break;
        case 4: bq4k::q4_fast<DT, FOLDED, 4, S16><<<grid, 256, 0, s>>>(x, packed, absmax, nchunks, tab); break;
        default: bq4k::q4_fast<DT, FOLDED, 5, S16><<<grid, 256, 0, s>>>(x, packed, absmax, nchunks, tab); break;
    }
}

template <int DT, bool S16>
void launch_q4_fast(int log2_lpb, bool folded, unsigned grid, cudaStream_t s, const void* x, uint8_t* packed, float* absmax, size_t nchunks,
                    const bq4k::Tables4& tab) {
    if (folded) launch_q4_fast_f<DT, true, S16>(log2_lpb, grid, s, x, packed, absmax, nchunks, tab);
    else launch_q4_fast_f<DT, false, S16>(log2_lpb, grid, s, x, packed, absmax, nchunks, tab);
}

// Above this many elements the 8-bit path's persistent forward kernel, in its 4-bit flavour, takes the whole tiles (its
// per-block scalars are computed once per block and its tiles keep eight chunks per thread in flight).
constexpr size_t kFwd4MinElems = size_t(1) << 23;

template <int DT, bool S16 = false>
cudaError_t quantize_t(const void* x, size_t n, size_t B, const bq4k::Tables4& tab, uint8_t* packed, float* absmax, int sms, cudaStream_t s) {
    size_t done = 0;
    const int l2 = log2_exact(B);
    constexpr size_t EB = (DT == bq4k::kF32) ? 4 : 2;
    if (l2 >= 3 && l2 <= 16 && aligned(x, 16) && aligned(packed, 4) && n >= B) {
        const size_t nblocks = n / B, n_full = nblocks * B;
        if (DT != bq4k::kF32 && tab.folded && l2 >= 6 && l2 <= 12 && n_full > kFwd4MinElems && aligned(absmax, S16 ? 2 : 4)) {
            bqk::Tables4Fast fast;
            std::memcpy(fast.entry, tab.entry, sizeof fast.entry);
            fast.neg_limit = tab.neg_limit;
            int dev = 0;
            cudaError_t e = cudaGetDevice(&dev);
            if (e == cudaSuccess) e = bql::launch_fwd4_fast(DT == bq4k::kF16 ? BQ_F16 : BQ_BF16, int(B), S16, x, packed, absmax, n_full, fast, sms, dev, s, &done);
            if (e != cudaSuccess) return e;
        }
        if (done < n_full) {                                      // the whole blocks the tiles did not cover (all of them for small tensors)
            const char* xr = static_cast<const char*>(x) + done * EB;
            uint8_t* pr = packed + done / 2;
            float* ar = S16 ? reinterpret_cast<float*>(reinterpret_cast<uint16_t*>(absmax) + done / B) : absmax + done / B;
            const size_t rblocks = (n_full - done) / B;
            if (l2 <= 8) {
                const size_t nchunks = (n_full - done) / 8;
                const unsigned grid = capped((nchunks + 511) / 512, size_t(sms) * 8);
                launch_q4_fast<DT, S16>(l2 - 3, tab.folded != 0, grid, s, xr, pr, ar, nchunks, tab);
            } else {
                const unsigned grid = capped((rblocks + 7) / 8, size_t(sms) * 8);
                if (tab.folded) bq4k::q4_wide<DT, true, S16><<<grid, 256, 0, s>>>(xr, pr, ar, rblocks, int(B / 8), tab);
                else bq4k::q4_wide<DT, false, S16><<<grid, 256, 0, s>>>(xr, pr, ar, rblocks, int(B / 8), tab);
            }
            cudaError_t e = cudaGetLastError();
            if (e != cudaSuccess) return e;
        }
        done = n_full;
    }
    if (done < n) {
        const size_t nb = (n + B - 1) / B, first_block = done / B;
        bq4k::q4_general_absmax<DT, S16><<<capped((nb - first_block + 7) / 8, size_t(sms) * 8), 256, 0, s>>>(x, absmax, n, B, first_block);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        const size_t nbytes = (n + 1) / 2, first_byte = done / 2;
        bq4k::q4_general_codes<DT, S16><<<capped((nbytes - first_byte + 255) / 256, size_t(sms) * 8), 256, 0, s>>>(x, absmax, packed, n, B, first_byte, tab);
        return cudaGetLastError();
    }
    return cudaSuccess;
}

template <int DT, bool S16 = false>
cudaError_t dequantize_t(const uint8_t* packed, const float* absmax, size_t n, size_t B, const bq4k::Tables4& tab, void* y, int sms, cudaStream_t s) {
    size_t done = 0;
    const int l2 = log2_exact(B);
    if (l2 >= 4 && aligned(packed, 8) && aligned(y, 32) && n >= 16) {
        const size_t n16 = n / 16;
        bq4k::dq4_fast<DT, S16><<<capped((n16 + 255) / 256, size_t(sms) * 16), 256, 0, s>>>(packed, absmax, y, n16, l2, tab);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        done = n16 * 16;
    }
    if (done < n) {
        bq4k::dq4_general<DT, S16><<<capped((n - done + 255) / 256, size_t(sms) * 8), 256, 0, s>>>(packed, absmax, y, n, B, done, tab);
        return cudaGetLastError();
    }
    return cudaSuccess;
}

}  // namespace

extern "C" {

int bq4_make_codebook(int kind, const float* user_values16, float* host_values_out16, bq4_codebook** out) {
    if (!out) return BQ_ERR_NULL;
    *out = nullptr;
    bq4_codebook* cb = new (std::nothrow) bq4_codebook();
    if (!cb) return BQ_ERR_CUDA;
    if (kind == BQ_CODEBOOK_DYNAMIC_TREE) {
        if (user_values16) { delete cb; return BQ_ERR_CODEBOOK; }
        dynamic_tree_values16(cb->tab.val);
    } else if (kind == BQ_CODEBOOK_USER) {
        if (!user_values16) { delete cb; return BQ_ERR_NULL; }
        if (!valid_user_values16(user_values16)) { delete cb; return BQ_ERR_CODEBOOK; }
        std::memcpy(cb->tab.val, user_values16, 16 * sizeof(float));
    } else {
        delete cb;
        return BQ_ERR_CODEBOOK;
    }
    build_thresholds(cb->tab);
    build_folded(cb->tab);
    if (host_values_out16) std::memcpy(host_values_out16, cb->tab.val, 16 * sizeof(float));
    *out = cb;
    return BQ_OK;
}

int bq4_free_codebook(bq4_codebook* cb) {
    delete cb;
    return BQ_OK;
}

int bq4_quantize(const void* x, bq_dtype xdt, size_t n, int block, const bq4_codebook* cb, uint8_t* packed_out, float* absmax_out,
                 void* cuda_stream) {
    if (!known_dtype(xdt)) return BQ_ERR_DTYPE;
    if (block < 1) return BQ_ERR_BLOCK;
    if (n >= kMaxElems) return BQ_ERR_SIZE;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (n == 0) return BQ_OK;
    if (!x || !packed_out || !absmax_out) return BQ_ERR_NULL;
    {
        const size_t xs = n * (xdt == BQ_F32 ? 4 : 2), ps = (n + 1) / 2, as = ((n + size_t(block) - 1) / size_t(block)) * sizeof(float);
        BQ_ASSERT(bqd::disjoint(x, xs, packed_out, ps) && bqd::disjoint(x, xs, absmax_out, as) && bqd::disjoint(packed_out, ps, absmax_out, as));
    }
    int sms = 0;
    const int rc = sm_count_of_current(&sms);
    if (rc != BQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    switch (xdt) {
        case BQ_F32: e = quantize_t<bq4k::kF32>(x, n, size_t(block), cb->tab, packed_out, absmax_out, sms, s); break;
        case BQ_F16: e = quantize_t<bq4k::kF16>(x, n, size_t(block), cb->tab, packed_out, absmax_out, sms, s); break;
        default: e = quantize_t<bq4k::kBF16>(x, n, size_t(block), cb->tab, packed_out, absmax_out, sms, s); break;
    }
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bq4_dequantize(const uint8_t* packed, const float* absmax, size_t n, int block, const bq4_codebook* cb, void* y_out, bq_dtype ydt,
                   void* cuda_stream) {
    if (!known_dtype(ydt)) return BQ_ERR_DTYPE;
    if (block < 1) return BQ_ERR_BLOCK;
    if (n >= kMaxElems) return BQ_ERR_SIZE;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (n == 0) return BQ_OK;
    if (!packed || !absmax || !y_out) return BQ_ERR_NULL;
    {
        const size_t ys = n * (ydt == BQ_F32 ? 4 : 2), ps = (n + 1) / 2, as = ((n + size_t(block) - 1) / size_t(block)) * sizeof(float);
        BQ_ASSERT(bqd::disjoint(y_out, ys, packed, ps) && bqd::disjoint(y_out, ys, absmax, as));
    }
    int sms = 0;
    const int rc = sm_count_of_current(&sms);
    if (rc != BQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    switch (ydt) {
        case BQ_F32: e = dequantize_t<bq4k::kF32>(packed, absmax, n, size_t(block), cb->tab, y_out, sms, s); break;
        case BQ_F16: e = dequantize_t<bq4k::kF16>(packed, absmax, n, size_t(block), cb->tab, y_out, sms, s); break;
        default: e = dequantize_t<bq4k::kBF16>(packed, absmax, n, size_t(block), cb->tab, y_out, sms, s); break;
    }
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bq4_quantize_s16(const void* x, bq_dtype xdt, size_t n, int block, const bq4_codebook* cb, uint8_t* packed_out, uint16_t* scale_out,
                     void* cuda_stream) {
    if (!known_dtype(xdt)) return BQ_ERR_DTYPE;
    if (block < 1) return BQ_ERR_BLOCK;
    if (n >= kMaxElems) return BQ_ERR_SIZE;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (n == 0) return BQ_OK;
    if (!x || !packed_out || !scale_out) return BQ_ERR_NULL;
    {
        const size_t xs = n * (xdt == BQ_F32 ? 4 : 2), ps = (n + 1) / 2, ss = ((n + size_t(block) - 1) / size_t(block)) * sizeof(uint16_t);
        BQ_ASSERT(bqd::disjoint(x, xs, packed_out, ps) && bqd::disjoint(x, xs, scale_out, ss) && bqd::disjoint(packed_out, ps, scale_out, ss));
    }
    int sms = 0;
    const int rc = sm_count_of_current(&sms);
    if (rc != BQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    float* scales = reinterpret_cast<float*>(scale_out);          // the S16 kernels address it as 16-bit words
    cudaError_t e;
    switch (xdt) {
        case BQ_F32: e = quantize_t<bq4k::kF32, true>(x, n, size_t(block), cb->tab, packed_out, scales, sms, s); break;
        case BQ_F16: e = quantize_t<bq4k::kF16, true>(x, n, size_t(block), cb->tab, packed_out, scales, sms, s); break;
        default: e = quantize_t<bq4k::kBF16, true>(x, n, size_t(block), cb->tab, packed_out, scales, sms, s); break;
    }
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

int bq4_dequantize_s16(const uint8_t* packed, const uint16_t* scale, size_t n, int block, const bq4_codebook* cb, void* y_out, bq_dtype ydt,
                       void* cuda_stream) {
    if (!known_dtype(ydt)) return BQ_ERR_DTYPE;
    if (block < 1) return BQ_ERR_BLOCK;
    if (n >= kMaxElems) return BQ_ERR_SIZE;
    if (!cb) return BQ_ERR_CODEBOOK;
    if (n == 0) return BQ_OK;
    if (!packed || !scale || !y_out) return BQ_ERR_NULL;
    {
        const size_t ys = n * (ydt == BQ_F32 ? 4 : 2), ps = (n + 1) / 2, ss = ((n + size_t(block) - 1) / size_t(block)) * sizeof(uint16_t);
        BQ_ASSERT(bqd::disjoint(y_out, ys, packed, ps) && bqd::disjoint(y_out, ys, scale, ss));
    }
    int sms = 0;
    const int rc = sm_count_of_current(&sms);
    if (rc != BQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const float* scales = reinterpret_cast<const float*>(scale);
    cudaError_t e;
    switch (ydt) {
        case BQ_F32: e = dequantize_t<bq4k::kF32, true>(packed, scales, n, size_t(block), cb->tab, y_out, sms, s); break;
        case BQ_F16: e = dequantize_t<bq4k::kF16, true>(packed, scales, n, size_t(block), cb->tab, y_out, sms, s); break;
        default: e = dequantize_t<bq4k::kBF16, true>(packed, scales, n, size_t(block), cb->tab, y_out, sms, s); break;
    }
    return e == cudaSuccess ? BQ_OK : cuda_fail(e);
}

}  // extern "C"
