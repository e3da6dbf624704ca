// bq_oracle.cpp -- CPU oracle (test infrastructure only; see bq_oracle.h).
//
// Plain C++17, single-threaded, no blocking, no vectorisation, no tables beyond the
// codebook itself.  Build with -O2 -ffp-contract=off and without -ffast-math so that
// every float operation below is one IEEE-754 binary32 operation, round-to-nearest-even,
// subnormals honoured.
//
// Readings of the method (the paper, section "Compression techniques" item 1, names
// "dynamic blockwise quantization" of the exchanged hidden states and fixes nothing else):
//   * codebook      : dynamic-tree 8-bit map over [-1, 1]: a sign bit, an exponent field
//                     whose length selects one of 7 decades, and a linear fraction that
//                     takes the remaining bits; plus the two end values 0 and 1.
//   * block scale   : absmax of the block in fp32, stored as is (not itself quantised).
//   * normalisation : a true fp32 division by the absmax (by 1 when the block is all zero).
//   * nearest code  : least |xhat - c_j| measured in double; equal distances go to the
//                     smaller index.
//   * inverse       : one fp32 multiply c[q] * absmax, then round-to-nearest-even to the
//                     output type.
#include "bq_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

namespace {

inline uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float u2f(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// bf16 is the upper half of an fp32.
float widen_bf16(uint16_t b) { return u2f(uint32_t(b) << 16); }

// fp16: 1 sign, 5 exponent (bias 15), 10 fraction bits.
float widen_f16(uint16_t h) {
    const int sign = (h >> 15) & 1;
    const int e = (h >> 10) & 0x1f;
    const int frac = h & 0x3ff;
    float mag;
    if (e == 0) {
        mag = std::ldexp(float(frac), -24);                  // zero and subnormals: frac * 2^-24
    } else if (e == 31) {
        mag = frac ? std::nanf("") : INFINITY;
    } else {
        mag = std::ldexp(float(1024 + frac), e - 25);        // (1 + frac/1024) * 2^(e-15)
    }
    return sign ? -mag : mag;
}

// Round-to-nearest-even of an fp32 to bf16.
uint16_t narrow_bf16(float v) {
    uint32_t u = f2u(v);
    if ((u & 0x7fffffffu) > 0x7f800000u) return uint16_t((u >> 16) | 0x0040u);   // NaN stays NaN
    const uint32_t lower = u & 0xffffu;
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1;       // carry may reach Inf
    return uint16_t(upper);
}

// Round-to-nearest-even of an fp32 to fp16, subnormal results included.
uint16_t narrow_f16(float v) {
    const uint32_t u = f2u(v);
    const uint16_t sign = uint16_t((u >> 16) & 0x8000u);
    const uint32_t absu = u & 0x7fffffffu;
    if (absu > 0x7f800000u) return uint16_t(sign | 0x7e00u);                     // NaN
    if (absu == 0x7f800000u) return uint16_t(sign | 0x7c00u);                    // Inf
    const double a = std::fabs(double(v));
    if (a == 0.0) return sign;
    // Spacing of fp16 values around a: 2^-24 below 2^-14, else 2^(floor(log2 a) - 10).
    int ex;
    std::frexp(a, &ex);                     // a = m * 2^ex with m in [0.5, 1)  =>  floor(log2 a) = ex - 1
    int e2 = ex - 1;
    if (e2 < -14) e2 = -14;
    const double ulp = std::ldexp(1.0, e2 - 10);
    const double scaled = a / ulp;          // exact: a power-of-two scaling of a value with <= 24 bits
    double r = std::floor(scaled);
    const double rem = scaled - r;
    if (rem > 0.5 || (rem == 0.5 && std::fmod(r, 2.0) == 1.0)) r += 1.0;
    const double rounded = r * ulp;
    if (rounded >= 65520.0) return uint16_t(sign | 0x7c00u);                     // overflows to Inf
    if (rounded < std::ldexp(1.0, -14)) return uint16_t(sign | uint16_t(r));     // subnormal: r = frac
    int ex2;
    const double m = std::frexp(rounded, &ex2);                                  // rounded = m * 2^ex2
    const int be = ex2 - 1 + 15;
    const int frac = int(std::ldexp(m, 11)) - 1024;                              // (2m - 1) * 1024
    return uint16_t(sign | uint16_t(be << 10) | uint16_t(frac));
}

float load_elem(const void* x, int dt, size_t i) {
    switch (dt) {
        case BQ_ORACLE_F32:  return static_cast<const float*>(x)[i];
        case BQ_ORACLE_F16:  return widen_f16(static_cast<const uint16_t*>(x)[i]);
        default:             return widen_bf16(static_cast<const uint16_t*>(x)[i]);
    }
}

void store_elem(void* y, int dt, size_t i, float v) {
    switch (dt) {
        case BQ_ORACLE_F32:  static_cast<float*>(y)[i] = v; break;
        case BQ_ORACLE_F16:  static_cast<uint16_t*>(y)[i] = narrow_f16(v); break;
        default:             static_cast<uint16_t*>(y)[i] = narrow_bf16(v); break;
    }
}

bool known_dtype(int dt) { return dt == BQ_ORACLE_F32 || dt == BQ_ORACLE_F16 || dt == BQ_ORACLE_BF16; }

}  // namespace

extern "C" {

float bq_oracle_widen(uint16_t bits, int dt) {
    return dt == BQ_ORACLE_F16 ? widen_f16(bits) : widen_bf16(bits);
}

uint16_t bq_oracle_narrow(float v, int dt) {
    return dt == BQ_ORACLE_F16 ? narrow_f16(v) : narrow_bf16(v);
}

// Dynamic-tree codebook.  Of the 8 bits one is the sign.  In the other 7, the position
// of the first set bit is the exponent field: it picks decade k = 0..6 (scale 10^(k-6))
// and leaves k bits of linear fraction, so decade k has 2^k magnitudes, the midpoints of
// 2^k equal bins of [0.1, 1]:
//     m(k, j) = 10^(k-6) * (0.1 + 0.9 * (2j + 1) / 2^(k+1)),   j = 0 .. 2^k - 1.
// That gives 127 magnitudes with both signs (254 values); 0 and 1 complete the 256.
// Each magnitude is evaluated as one ratio of two exact integers,
//     m = (2^(k+1) + 9 (2j + 1)) / (2^(k+1) * 10^(7-k)),
// divided in double and rounded once to fp32.  Sorted ascending; the code is the index.
int bq_oracle_make_codebook(float values_out[256]) {
    if (!values_out) return 1;
    std::vector<float> v;
    for (int k = 0; k <= 6; ++k) {
        const long bins2 = 1L << (k + 1);                 // 2^(k+1)
        long pow10 = 1;
        for (int t = 0; t < 7 - k; ++t) pow10 *= 10;      // 10^(7-k)
        for (long j = 0; j < (1L << k); ++j) {
            const double num = double(bins2 + 9 * (2 * j + 1));
            const double den = double(bins2 * pow10);
            const float m = float(num / den);
            v.push_back(m);
            v.push_back(-m);
        }
    }
    v.push_back(0.0f);
    v.push_back(1.0f);
    std::sort(v.begin(), v.end());
    for (int i = 0; i < 256; ++i) values_out[i] = v[size_t(i)];
    return 0;
}

// Linear scan for the nearest code; strict "<" keeps the first (smallest) index on ties.
int bq_oracle_nearest(float xhat, const float codebook[256]) {
    int best = 0;
    double best_dist = std::fabs(double(xhat) - double(codebook[0]));
    for (int j = 1; j < 256; ++j) {
        const double dist = std::fabs(double(xhat) - double(codebook[j]));
        if (dist < best_dist) { best_dist = dist; best = j; }
    }
    return best;
}

int bq_oracle_quantize(const void* x, int xdt, size_t n, int block, const float codebook[256],
                       uint8_t* codes_out, float* absmax_out) {
    if (n == 0) return 0;
    if (!x || !codebook || !codes_out || !absmax_out || block < 1 || !known_dtype(xdt)) return 1;
    const size_t B = size_t(block);
    const size_t nb = (n + B - 1) / B;
    for (size_t b = 0; b < nb; ++b) {
        const size_t lo = b * B;
        const size_t hi = std::min(n, lo + B);
        float a = 0.0f;                                    // absmax over the block's real elements
        for (size_t i = lo; i < hi; ++i) {
            const float v = std::fabs(load_elem(x, xdt, i));
            a = (v > a) ? v : a;
        }
        absmax_out[b] = a;
        const float d = (a != 0.0f) ? a : 1.0f;            // an all-zero block divides by 1
        for (size_t i = lo; i < hi; ++i) {
            const float xhat = load_elem(x, xdt, i) / d;   // one fp32 division
            codes_out[i] = uint8_t(bq_oracle_nearest(xhat, codebook));
        }
    }
    return 0;
}

int bq_oracle_dequantize(const uint8_t* codes, const float* absmax, size_t n, int block,
                         const float codebook[256], void* y_out, int ydt) {
    if (n == 0) return 0;
    if (!codes || !absmax || !codebook || !y_out || block < 1 || !known_dtype(ydt)) return 1;
    const size_t B = size_t(block);
    for (size_t i = 0; i < n; ++i) {
        const float v = codebook[codes[i]] * absmax[i / B];   // one fp32 multiply
        store_elem(y_out, ydt, i, v);
    }
    return 0;
}

int bq_oracle_roundtrip(const void* x, int xdt, size_t n, int block, const float codebook[256],
                        void* y_out, int ydt, uint8_t* codes_out, float* absmax_out) {
    if (n == 0) return 0;
    if (!x || !codebook || !y_out || block < 1 || !known_dtype(xdt) || !known_dtype(ydt)) return 1;
    const size_t B = size_t(block);
    std::vector<uint8_t> codes(n);
    std::vector<float> absmax((n + B - 1) / B);
    int rc = bq_oracle_quantize(x, xdt, n, block, codebook, codes.data(), absmax.data());
    if (rc) return rc;
    rc = bq_oracle_dequantize(codes.data(), absmax.data(), n, block, codebook, y_out, ydt);
    if (rc) return rc;
    if (codes_out) std::memcpy(codes_out, codes.data(), n);
    if (absmax_out) std::memcpy(absmax_out, absmax.data(), absmax.size() * sizeof(float));
    return 0;
}

}  // extern "C"
