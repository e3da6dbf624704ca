// bq_tables.h -- host-side construction of the codebook and of the search tables the
// kernels use.  Plain C++ (no CUDA), so that it can be exercised without a device.
//
// Search tables.  The nearest-code rule (least |xhat - c_j|, equal distances to the
// smaller index) is the step function  q(xhat) = #{ j : t_j < xhat }  over the exact
// midpoints t_j = (c_j + c_j+1) / 2.  Because xhat is an fp32, comparing against t_j
// rounded toward -inf to fp32 gives the same answer, so the search needs no wider type.
//
// For a codebook that mirrors (c_j = -c_254-j, zero at 127) the search is folded onto
// magnitudes.  Let theta_p (p = 0..127) be the positive midpoints and m = |xhat|.  With
//     key(xhat) = rotate-left-by-one of xhat's bits = 2 * bits(m) + sign
//     TK[p]     = 2 * bits(round_down(theta_p)) + (theta_p is not an fp32 ? 1 : 0)
// the count P = #{ p : TK[p] < key } equals #{theta_p < m} for xhat >= 0 and
// #{theta_p <= m} for xhat < 0, which is what the tie rule needs on each side:
//     code = 127 + P (xhat >= 0),  127 - min(P, 127) (xhat < 0).
//
// P comes from ONE table lookup and one addition.  Keys are clamped from below to
// kKeyLow (the key of 2^-22, below the smallest threshold) and cut into cells of 2^18
// consecutive keys (exponent plus 6 fraction bits of m); no cell holds more than one
// threshold.  For the cell that starts at key S, with P0 thresholds below S and (at most)
// one threshold TK inside it, the entry is
//     E = ((127 + P0) << 24 | 0xFC0000 | (0x3FFFF - (TK - S))) - S        (mod 2^32)
// so that E + key = (127 + P0) << 24 | 0xFC0000 | ... plus a carry out of bit 17 exactly when
// key > TK; the six set bits pass that carry on into the top byte: (E + key) >> 24 = 127 + P,
// which is the code itself for xhat >= 0.
// A cell without a threshold uses TK - S = 0x3FFFF, which never carries.
#pragma once

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace bqt {

constexpr uint32_t kKeyLow = 0x69000000u;               // key of +2^-22
constexpr int kCellShift = 18;
constexpr uint32_t kCellBase = kKeyLow >> kCellShift;    // index of the first cell
constexpr int kCells = int((0x7F000001u >> kCellShift) - kCellBase) + 1;    // up to the key of -1.0: 1409 cells

inline uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float u2f(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

struct Tables {
    float values[256];        // the codebook, ascending
    float thr_down[256];      // [0..254] midpoints rounded toward -inf; [255] = +inf sentinel
    bool folded;              // true when the magnitude-folded tables below are valid
    uint32_t tk[128];         // folded threshold keys
    float cmag[132];          // cmag[p] = values[127 + p], p = 0..128 (padded)
    uint32_t guess[kCells];   // per cell: the entry E described above
    float neg_limit;          // xhat is clamped from below to this before the folded search
};

// Dynamic-tree map: sign bit, decade chosen by the exponent field, linear fraction.
// Decade k = 0..6 holds the midpoints of 2^k equal bins of [0.1, 1] scaled by 10^(k-6);
// each magnitude is (2^(k+1) + 9 (2j+1)) / (2^(k+1) 10^(7-k)), one double division of
// exact integers rounded once to fp32.  Plus 0 and 1.
inline void dynamic_tree_values(float out[256]) {
    float mags[127];
    int cnt = 0;
    double p10 = 1e7;
    for (int k = 0; k <= 6; ++k, p10 /= 10.0) {          // p10 = 10^(7-k), exact in double
        const double two = double(1 << (k + 1));
        for (int j = 0; j < (1 << k); ++j)
            mags[cnt++] = float((two + 9.0 * double(2 * j + 1)) / (two * p10));
    }
    // the magnitudes come out ascending (decade by decade), so the table can be laid out directly
    for (int p = 0; p < 127; ++p) {
        out[128 + p] = mags[p];
        out[126 - p] = -mags[p];
    }
    out[127] = 0.0f;
    out[255] = 1.0f;
}

inline bool valid_user_values(const float* v) {
    bool has_zero = false;
    for (int i = 0; i < 256; ++i) {
        if (!std::isfinite(v[i]) || v[i] < -1.0f || v[i] > 1.0f) return false;
        if (i && !(v[i] > v[i - 1])) return false;
        if (v[i] == 0.0f) has_zero = true;
        else if (std::fabs(v[i]) < 5.9604644775390625e-08f) return false;     // 2^-24
    }
    return has_zero;
}

inline float round_down_to_float(double t) {
    float g = float(t);
    if (double(g) > t) g = std::nextafterf(g, -INFINITY);
    return g;
}

inline void build(Tables& T) {
    for (int j = 0; j < 255; ++j) {
        const double t = (double(T.values[j]) + double(T.values[j + 1])) * 0.5;   // exact (see header)
        T.thr_down[j] = round_down_to_float(t);
    }
    T.thr_down[255] = INFINITY;

    T.folded = (T.values[127] == 0.0f);
    for (int j = 0; j <= 254 && T.folded; ++j) T.folded = (T.values[j] == -T.values[254 - j]);
    if (!T.folded) return;

    for (int p = 0; p <= 128; ++p) T.cmag[p] = T.values[127 + p];
    for (int p = 129; p < 132; ++p) T.cmag[p] = 1.0f;
    for (int p = 0; p < 128; ++p) {
        const double t = (double(T.values[127 + p]) + double(T.values[128 + p])) * 0.5;
        const float d = round_down_to_float(t);
        T.tk[p] = 2u * f2u(d) + (double(d) == t ? 0u : 1u);
    }
    // negative side: P must not count theta_127 (there is no code below -c_254)
    T.neg_limit = -u2f((T.tk[127] - 1u) >> 1);

    if (T.tk[0] <= kKeyLow) { T.folded = false; return; }          // clamped keys must sit below every threshold
    int p = 0;                                                       // thresholds below the current cell
    for (int c = 0; c < kCells; ++c) {
        const uint32_t start = (kCellBase + uint32_t(c)) << kCellShift;
        const uint64_t end = uint64_t(start) + (1u << kCellShift);
        uint32_t inside = 0x3FFFFu;
        int count = 0;
        while (p + count < 128 && uint64_t(T.tk[p + count]) < end) {
            inside = T.tk[p + count] - start;
            ++count;
        }
        if (count > 1) { T.folded = false; return; }
        T.guess[c] = ((uint32_t(127 + p) << 24) | 0xFC0000u | (0x3FFFFu - inside)) - start;
        p += count;
    }
}

}  // namespace bqt
