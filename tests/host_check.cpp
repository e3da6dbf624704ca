// host_check.cpp -- host-side restatement of the tuned kernels' arithmetic, for CPU tests.
//
// The CUDA library builds its search tables on the host (bq_tables.h) and its kernels use
// them with a handful of fp32 / integer operations.  This file repeats exactly those
// operations in plain C++ so that, without a GPU, the tests can check (a) that the folded
// search returns the nearest code for any xhat and (b) that the reciprocal-based quotient
// used for 16-bit inputs equals the IEEE quotient wherever a code depends on it.
#include <cmath>
#include <cstdint>
#include <cstring>

#include "../paper_2407_19775_b200/csrc/bq_tables.h"

namespace {
bqt::Tables g_tab;
bool g_ready = false;
void ensure() {
    if (g_ready) return;
    bqt::dynamic_tree_values(g_tab.values);
    bqt::build(g_tab);
    g_ready = true;
}

struct Found { uint32_t count; uint32_t bits; };

Found search_folded(float xhat) {
    Found f;
    xhat = std::fmax(xhat, g_tab.neg_limit);
    f.bits = bqt::f2u(xhat);
    uint32_t key = (f.bits << 1) | (f.bits >> 31);
    if (key < bqt::kKeyLow) key = bqt::kKeyLow;
    const uint32_t cell = (key >> 18) - bqt::kCellBase;
    f.count = ((g_tab.guess[cell] + key) >> 24) - 127u;
    return f;
}
}  // namespace

extern "C" {

int hc_tables(float* values, float* thr_down, uint32_t* tk, float* cmag, uint32_t* guess, float* neg_limit) {
    ensure();
    std::memcpy(values, g_tab.values, sizeof g_tab.values);
    std::memcpy(thr_down, g_tab.thr_down, sizeof g_tab.thr_down);
    std::memcpy(tk, g_tab.tk, sizeof g_tab.tk);
    std::memcpy(cmag, g_tab.cmag, sizeof g_tab.cmag);
    std::memcpy(guess, g_tab.guess, sizeof g_tab.guess);
    *neg_limit = g_tab.neg_limit;
    return g_tab.folded ? 1 : 0;
}

int hc_user_tables_folded(const float* values) {
    bqt::Tables t;
    if (!bqt::valid_user_values(values)) return -1;
    std::memcpy(t.values, values, sizeof t.values);
    bqt::build(t);
    return t.folded ? 1 : 0;
}

int hc_code_folded(float xhat) {
    ensure();
    const Found f = search_folded(xhat);
    const uint32_t sm = uint32_t(int32_t(f.bits) >> 31);
    return int(127u + ((f.count ^ sm) - sm));
}

float hc_value_folded(float xhat, float absmax) {
    ensure();
    const Found f = search_folded(xhat);
    const float cm = g_tab.cmag[f.count];
    const float as = bqt::u2f(bqt::f2u(absmax) | (f.bits & 0x80000000u));
    return std::fmaf(cm, as, 0.0f);
}

int hc_code_general(float xhat) {
    ensure();
    int q = 0;
    for (int s = 128; s >= 1; s >>= 1) q += (g_tab.thr_down[q + s - 1] < xhat) ? s : 0;
    return q;
}

// All codes over a range of bit patterns: out[i] = folded code of the float with bits lo + i.
void hc_codes_of_bits(uint32_t lo, uint32_t count, uint8_t* out_folded, uint8_t* out_general) {
    for (uint32_t i = 0; i < count; ++i) {
        const float x = bqt::u2f(lo + i);
        out_folded[i] = uint8_t(hc_code_folded(x));
        out_general[i] = uint8_t(hc_code_general(x));
    }
}

// Exhaustive check of the reciprocal-based quotient (reciprocal perturbed by -2..+2 ulp) for inputs with `sig_bits`-bit
// significands: d = (2^(sig_bits-1) + md) * 2^ed and x = (2^(sig_bits-1) + mx) * 2^(ed - gap ...)
// for every pair of significands and every exponent gap 0..max_gap with |x| <= d.
// Returns the number of pairs whose quotient differs from x / d; *code_mismatch counts
// those whose nearest code differs too.
long hc_check_quick_division(int sig_bits, int max_gap, int d_exp, long* code_mismatch, long* checked) {
    ensure();
    const int half = 1 << (sig_bits - 1);
    long bad = 0, bad_code = 0, cnt = 0;
    for (int md = 0; md < half; ++md) {
        const float d = std::ldexp(float(half + md), d_exp - (sig_bits - 1));
        for (int dr = -2; dr <= 2; ++dr) {
        // any reciprocal within 2 ulp of the correctly rounded one (the kernel uses the
        // hardware's approximate reciprocal, whose last bits are not specified)
        const float r = bqt::u2f(bqt::f2u(1.0f / d) + uint32_t(dr));
        for (int gap = 0; gap <= max_gap; ++gap) {
            for (int mx = 0; mx < half; ++mx) {
                const float x = std::ldexp(float(half + mx), d_exp - gap - (sig_bits - 1));
                if (x > d) continue;
                for (int sgn = 0; sgn < 2; ++sgn) {
                    const float xs = sgn ? -x : x;
                    const float q0 = xs * r;
                    const float e = std::fmaf(-d, q0, xs);
                    const float q = std::fmaf(e, r, q0);
                    const float ref = xs / d;
                    ++cnt;
                    if (bqt::f2u(q) != bqt::f2u(ref)) {
                        ++bad;
                        if (hc_code_general(q) != hc_code_general(ref)) ++bad_code;
                    }
                }
            }
        }
        }
    }
    *code_mismatch = bad_code;
    *checked = cnt;
    return bad;
}

// The row kernel of the mixed matrix decomposition needs t = RN32(127 x / d) for 16-bit x and d
// with |x| <= d.  It computes n = 127 x (exact), q0 = RN(n r), e = n - d q0 (one fma, exact),
// t = RN(q0 + e r) from an approximate reciprocal r.  Same exhaustive check as above with the
// 18-bit numerators 127 x: returns how many t differ in any bit from n / d; *int_mismatch
// counts those whose rounding to an integer (ties to even) differs too.
long hc_check_rowquant_division(int sig_bits, int max_gap, int d_exp, long* int_mismatch, long* checked) {
    const int half = 1 << (sig_bits - 1);
    long bad = 0, bad_int = 0, cnt = 0;
    for (int md = 0; md < half; ++md) {
        const float d = std::ldexp(float(half + md), d_exp - (sig_bits - 1));
        for (int dr = -2; dr <= 2; ++dr) {
            const float r = bqt::u2f(bqt::f2u(1.0f / d) + uint32_t(dr));
            for (int gap = 0; gap <= max_gap; ++gap) {
                for (int mx = 0; mx < half; ++mx) {
                    const float x = std::ldexp(float(half + mx), d_exp - gap - (sig_bits - 1));
                    if (x > d) continue;
                    for (int sgn = 0; sgn < 2; ++sgn) {
                        const float n = (sgn ? -x : x) * 127.0f;
                        const float q0 = n * r;
                        const float e = std::fmaf(-d, q0, n);
                        const float t = std::fmaf(e, r, q0);
                        const float ref = n / d;
                        ++cnt;
                        if (bqt::f2u(t) != bqt::f2u(ref)) {
                            ++bad;
                            if (std::nearbyintf(t) != std::nearbyintf(ref)) ++bad_int;
                        }
                    }
                }
            }
        }
    }
    *int_mismatch = bad_int;
    *checked = cnt;
    return bad;
}

}  // extern "C"
