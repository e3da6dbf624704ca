// bq_kernels.cuh -- device code of libbq (sm_100a).
//
// Three kernels:
//   fwd_fast     : quantize, or the fused quantize->dequantize roundtrip, for power-of-two
//                  blocks on 16-byte aligned tensors.  One pass over HBM: a tile of the
//                  input sits in registers between the absmax reduction and the search.
//                  Built in two flavours: persistent CTAs with the search tables replicated
//                  per lane in shared memory (large tensors), and LITE, which reads the
//                  tables through L1 and has no set-up (small tensors).
//   deq_fast     : dequantize, 16 codes per 128-bit load, one 256-bit store per 16 outputs;
//                  the same two flavours (its LITE one keeps one plain 1 KB copy of the
//                  values in shared memory: a word per thread to fill).
//   *_general    : any block size, any alignment, any codebook; one warp per block.
//
// Arithmetic contract shared by all of them (it is what makes the results bit-identical
// to the plain definition): absmax is an exact fp32 max; xhat is the correctly rounded
// fp32 quotient x / absmax; the code is #{ j : t_j < xhat } over the exact midpoints; the
// inverse is one fp32 multiply followed by a round-to-nearest-even conversion.  No fused
// contraction, fast division or flush-to-zero is allowed to change any of these.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bqk {

enum { kF32 = 0, kF16 = 1, kBF16 = 2 };

constexpr uint32_t kKeyLow = 0x69000000u;              // key of +2^-22: keys are clamped to it from below
constexpr uint32_t kCellBase = kKeyLow >> 18;
constexpr int kCells = int((0x7F000001u >> 18) - kCellBase) + 1;      // 1409

// Shared-memory image of the folded search tables.  Every entry is replicated 32 times,
// one copy per lane in that lane's own bank (entry e, lane l at byte e*128 + l*4), so a
// data-dependent lookup by 32 lanes never has a bank conflict.
constexpr uint32_t kCmOff = 0;                          // 129 magnitudes (132 rows reserved)
constexpr uint32_t kGuessOff = kCmOff + 132u * 128u;    // kCells count entries
constexpr uint32_t kRedOff = kGuessOff + uint32_t(kCells) * 128u;   // cross-warp partial maxima
constexpr uint32_t kFwdSmemBytes = kRedOff + 2u * 32u * 4u + 128u;    // + slack to align the base to 128 bytes
constexpr uint32_t kFwdLiteSmemBytes = 2u * 32u * 4u + 128u;

constexpr uint32_t kDeqSmemBytes = 256u * 128u;         // signed code values, replicated per lane
constexpr uint32_t kDeqLiteSmemBytes = 256u * 4u;       // LITE: one plain copy

struct DeviceTables {
    const float* values;        // [256]
    const float* thr_down;      // [256], last = +inf
    const uint32_t* tk;         // [128]
    const float* cmag;          // [132]; guess follows it directly in memory
    const uint32_t* guess;      // [kCells]
    float neg_limit;            // -(largest |xhat| whose negative key does not pass the last threshold)
};

// The 4-bit variant of the path (16 codes, two per byte) runs through the same forward kernel.  Its
// folded table is small enough to travel in the kernel's parameters: cells of 2^21 keys from the
// key of 2^-9 up, entry ((7 + P0) << 24 | 0xE00000 | (0x1FFFFF - (TK - S))) - S, so that the top byte
// of entry + key is 7 + P (see bq4_kernels.cuh for the map and the table's construction).
constexpr uint32_t kKeyLow4 = 0x76000000u;             // key of +2^-9
constexpr uint32_t kCellBase4 = kKeyLow4 >> 21;
constexpr int kCells4 = 73;
struct Tables4Fast {
    uint32_t entry[kCells4];
    float neg_limit;
};
constexpr uint32_t kFwd4SmemBytes = uint32_t(kCells4) * 128u + 2u * 32u * 4u + 128u;
constexpr uint32_t kRedOff4 = uint32_t(kCells4) * 128u;
template <int BITS> struct TabArg { using type = DeviceTables; };
template <> struct TabArg<4> { using type = Tables4Fast; };

// ------------------------------------------------------------------------------------------
// small helpers

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// Streaming accesses.  Loads skip L1 allocation (every byte is used once) but are not
// marked read-only, so bq_roundtrip may run in place; stores are evict-first.  Of the
// cache-operator combinations tried on a 1 GiB tensor this one was the fastest by 1-3 %.
__device__ __forceinline__ uint4 ldg_stream_16(const void* p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void stg_stream_16(void* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// 32 contiguous bytes per thread as one 256-bit store: a warp then writes whole 128-byte lines
__device__ __forceinline__ void stg_stream_32(void* p, uint4 a, uint4 b) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}
// 32 contiguous bytes: one 256-bit store when p is 32-byte aligned (WIDE), else two 128-bit ones
template <bool WIDE>
__device__ __forceinline__ void store_32(void* p, uint4 a, uint4 b) {
    if constexpr (WIDE) {
        stg_stream_32(p, a, b);
    } else {
        stg_stream_16(p, a);
        stg_stream_16(static_cast<char*>(p) + 16, b);
    }
}
__device__ __forceinline__ void stg_stream_8(void* p, uint2 v) {
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
}
__device__ __forceinline__ void stg_stream_4(void* p, uint32_t v) {
    asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

template <int DT> struct Elem;
template <> struct Elem<kF32> { static constexpr int kBytes = 4; static constexpr int kPerChunk = 4; };
template <> struct Elem<kF16> { static constexpr int kBytes = 2; static constexpr int kPerChunk = 8; };
template <> struct Elem<kBF16> { static constexpr int kBytes = 2; static constexpr int kPerChunk = 8; };

// Widen the elements of one 16-byte chunk to fp32 (exact).
template <int DT, int N>
__device__ __forceinline__ void widen_chunk(const uint4& w, float (&f)[N]) {
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
    if constexpr (DT == kF32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) f[i] = __uint_as_float(u[i]);
    } else if constexpr (DT == kBF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(u[i] << 16);
            f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&u[i]));
            f[2 * i] = p.x;
            f[2 * i + 1] = p.y;
        }
    }
}

// Round-to-nearest-even narrowing of one chunk's worth of fp32 values.
template <int DT, int N>
__device__ __forceinline__ uint4 narrow_chunk(const float (&v)[N]) {
    uint32_t u[4];
    if constexpr (DT == kF32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) u[i] = __float_as_uint(v[i]);
    } else if constexpr (DT == kBF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 p = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            u[i] = *reinterpret_cast<const uint32_t*>(&p);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __half2 p = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
            u[i] = *reinterpret_cast<const uint32_t*>(&p);
        }
    }
    return make_uint4(u[0], u[1], u[2], u[3]);
}

template <int DT>
__device__ __forceinline__ float load_elem(const void* x, size_t i) {
    if constexpr (DT == kF32) return static_cast<const float*>(x)[i];
    else if constexpr (DT == kBF16) return __uint_as_float(uint32_t(static_cast<const uint16_t*>(x)[i]) << 16);
    else return __half2float(static_cast<const __half*>(x)[i]);
}

template <int DT>
__device__ __forceinline__ void store_elem(void* y, size_t i, float v) {
    if constexpr (DT == kF32) static_cast<float*>(y)[i] = v;
    else if constexpr (DT == kBF16) static_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
    else static_cast<__half*>(y)[i] = __float2half_rn(v);
}

// ------------------------------------------------------------------------------------------
// Folded search (see bq_tables.h): one lookup of the cell's entry, one addition, and the
// count of thresholds below the key sits in the top byte.

struct Found {
    uint32_t sum;          // entry + key: its top byte is 127 + P, the code of a non-negative xhat
    uint32_t bits;         // bit pattern of the clamped xhat
};

// Where the two tables are read from.  The tuned kernels keep them in shared memory, one
// copy per lane (built once per CTA: worth it when the CTA then streams megabytes); the
// LITE kernels, used for small tensors where that set-up would dominate, read the 6 KB of
// tables straight from global memory through L1.
template <bool LITE> struct TabRef;
template <> struct TabRef<false> {
    static constexpr uint32_t kLow = kKeyLow;
    uint32_t guess_lane;   // this lane's column of the entry table, rebased by the index of the first cell
    uint32_t cm_lane;      // this lane's column of the magnitude table, rebased by -127 rows
    __device__ __forceinline__ TabRef(const DeviceTables&, uint32_t sm_lane)
        : guess_lane(sm_lane + kGuessOff - kCellBase * 128u), cm_lane(sm_lane + kCmOff - 127u * 128u) {}
    // index * 128 + base as one multiply-add (the fp32 multiplier pipe has room; the integer
    // ALU is the busiest unit of these kernels)
    __device__ __forceinline__ uint32_t entry(uint32_t key) const {
        uint32_t ga;
        asm("mad.lo.u32 %0, %1, 128, %2;" : "=r"(ga) : "r"(key >> 18), "r"(guess_lane));
        return lds_u32(ga);
    }
    __device__ __forceinline__ float magnitude(uint32_t sum) const {
        uint32_t va;
        asm("mad.lo.u32 %0, %1, 128, %2;" : "=r"(va) : "r"(sum >> 24), "r"(cm_lane));
        return __uint_as_float(lds_u32(va));
    }
};
template <> struct TabRef<true> {
    static constexpr uint32_t kLow = kKeyLow;
    const uint32_t* guess;
    const float* cmag;
    __device__ __forceinline__ TabRef(const DeviceTables& t, uint32_t) : guess(t.guess - kCellBase), cmag(t.cmag - 127) {}
    __device__ __forceinline__ uint32_t entry(uint32_t key) const { return __ldg(guess + (key >> 18)); }
    __device__ __forceinline__ float magnitude(uint32_t sum) const { return __ldg(cmag + (sum >> 24)); }
};

// the 4-bit table: per-lane copies in shared memory only (large tensors)
struct TabRef4 {
    static constexpr uint32_t kLow = kKeyLow4;
    uint32_t guess_lane;
    __device__ __forceinline__ TabRef4(uint32_t sm_lane) : guess_lane(sm_lane - kCellBase4 * 128u) {}
    __device__ __forceinline__ uint32_t entry(uint32_t key) const {
        uint32_t ga;
        asm("mad.lo.u32 %0, %1, 128, %2;" : "=r"(ga) : "r"(key >> 21), "r"(guess_lane));
        return lds_u32(ga);
    }
};

template <class Tab>
__device__ __forceinline__ Found search_folded(float xhat, float neg_limit, const Tab& tab) {
    Found f;
    xhat = fmaxf(xhat, neg_limit);
    f.bits = __float_as_uint(xhat);
    const uint32_t key = max(__funnelshift_l(f.bits, f.bits, 1), Tab::kLow);
    f.sum = tab.entry(key) + key;
    return f;
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Four codes as one word.  The top bytes of the four sums are the codes for non-negative
// values, c = 127 + P; a negative value takes 127 - P = (c ^ 0xFF) - 1.  `neg` holds 0xFF in
// the bytes of negative elements (sign_mask_* below: byte-permutes that replicate a sign bit
// over its byte; taken from the inputs, whose signs the quotients share); the subtraction
// cannot borrow between bytes because c ^ 0xFF >= 1 wherever 1 is subtracted (the clamp in
// search_folded keeps c <= 254 on the negative side).  The "1 in every negative byte" is never
// formed: neg = 255 * (neg & 0x01010101) and 255 * 0x01010101 = -1 (mod 2^32), so
// neg * 0x01010101 = -(neg & 0x01010101), and the subtraction is one multiply-add.
__device__ __forceinline__ uint32_t pack_codes(const Found& f0, const Found& f1, const Found& f2, const Found& f3, uint32_t neg) {
    const uint32_t c = prmt(prmt(f0.sum, f1.sum, 0x0073u), prmt(f2.sum, f3.sum, 0x0073u), 0x5410u);
    uint32_t out;
    asm("mad.lo.u32 %0, %1, 0x01010101, %2;" : "=r"(out) : "r"(neg), "r"(c ^ neg));
    return out;
}
// sign bytes of four 16-bit elements held in two words (element sign bits sit in bytes 1, 3, 5, 7)
__device__ __forceinline__ uint32_t sign_mask_16(uint32_t w0, uint32_t w1) { return prmt(w0, w1, 0xFDB9u); }
// sign bytes of four fp32 elements
__device__ __forceinline__ uint32_t sign_mask_32(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return prmt(prmt(a, b, 0x00FBu), prmt(c, d, 0x00FBu), 0x5410u);
}

// Eight 4-bit codes as eight nibbles (element 2i in the low nibble of byte i).  The top bytes c = 7 + P of the
// sums are gathered four to a word; negative elements (0xFF in `neg0` / `neg1`) take 7 - P = (c ^ 0xF) - 1, which
// cannot borrow between bytes because c <= 14 there (the clamp keeps P <= 7 on that side), and the "-1 in every
// negative byte" is neg * 0x01010101 as in pack_codes; then byte pairs fold into nibble pairs: x | x >> 4 leaves
// [q1 q0] in byte 0 and [q3 q2] in byte 2.
__device__ __forceinline__ uint32_t pack_nibbles8(const uint32_t (&sum)[8], uint32_t neg0, uint32_t neg1) {
    uint32_t c0 = prmt(prmt(sum[0], sum[1], 0x0073u), prmt(sum[2], sum[3], 0x0073u), 0x5410u);
    uint32_t c1 = prmt(prmt(sum[4], sum[5], 0x0073u), prmt(sum[6], sum[7], 0x0073u), 0x5410u);
    asm("mad.lo.u32 %0, %1, 0x01010101, %2;" : "=r"(c0) : "r"(neg0), "r"(c0 ^ (neg0 & 0x0F0F0F0Fu)));
    asm("mad.lo.u32 %0, %1, 0x01010101, %2;" : "=r"(c1) : "r"(neg1), "r"(c1 ^ (neg1 & 0x0F0F0F0Fu)));
    return prmt(c0 | (c0 >> 4), c1 | (c1 >> 4), 0x6420u);
}

// Two fp32 lanes per instruction (sm_100 packed fp32 arithmetic).
__device__ __forceinline__ uint64_t pack2(float a, float b) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(a), "f"(b));
    return v;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// c[code] * absmax as one rounding: the magnitude times the signed absmax, plus +0.0 so
// that a zero magnitude gives +0.0 whatever the sign.
template <bool LITE>
__device__ __forceinline__ void values_of(const Found& f0, const Found& f1, float absmax, const TabRef<LITE>& tab, float& v0, float& v1) {
    const float c0 = tab.magnitude(f0.sum), c1 = tab.magnitude(f1.sum);
    const float a0 = __uint_as_float(__float_as_uint(absmax) | (f0.bits & 0x80000000u));
    const float a1 = __uint_as_float(__float_as_uint(absmax) | (f1.bits & 0x80000000u));
    unpack2(fma2(pack2(c0, c1), pack2(a0, a1), 0ull), v0, v1);         // two products per instruction; +0.0 addend
}

// Builds the per-lane copies.  The magnitude rows and the entry rows are consecutive both in
// the device blob (cmag | guess) and in shared memory, so row i is word i of one array.  Each
// warp first loads its rows coalesced (one word per lane, all loads in flight together), then
// hands every word round with a shuffle so that all 32 lanes store it into their own column.
template <int NT>
__device__ __forceinline__ void fill_fwd_tables(const DeviceTables& t, uint32_t sm_base) {
    constexpr int NROWS = 132 + kCells;
    constexpr int NWARPS = NT / 32;
    constexpr int ITERS = (NROWS + NWARPS * 32 - 1) / (NWARPS * 32);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t sm_lane = sm_base + uint32_t(lane) * 4u + kCmOff;
    const uint32_t* src = reinterpret_cast<const uint32_t*>(t.cmag);
    uint32_t v[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        const int row = (it * NWARPS + warp) * 32 + lane;
        v[it] = row < NROWS ? __ldg(src + row) : 0u;
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        const int row0 = (it * NWARPS + warp) * 32;
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            const uint32_t word = __shfl_sync(0xffffffffu, v[it], k);
            if (row0 + k < NROWS) sts_u32(sm_lane + uint32_t(row0 + k) * 128u, word);
        }
    }
}

__device__ __forceinline__ float max3_abs(float a, float b, float c) {      // max(|a|, |b|, |c|)
    float d;
    asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float rcp_approx(float d) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(d));
    return r;
}

// ------------------------------------------------------------------------------------------
// fwd_fast
//
//   XDT          element type of x (and of y: the fused kernel keeps the type)
//   B            block size, a power of two, >= 64
//   R            16-byte chunks ("rows") each thread keeps in registers per tile
//   TW           warps that share one block (1 unless B > R * 32 * elements-per-chunk)
//   WRITE_Y      store the dequantised tensor
//   WRITE_Q      store codes and absmax
//
// A row is 32 consecutive chunks, one per lane (512 contiguous bytes).  Blocks no longer
// than a row occupy B / kPerChunk consecutive lanes of one row and are reduced with
// segmented shuffles; longer blocks take R rows of TW warps.  Only whole tiles are handled
// (the host sends the remainder to the general kernel).  The loads of the next tile
// are issued as soon as the current one has been widened, so they fly during the search.
//
// Normalisation.  The contract is the correctly rounded quotient x / d.  For 16-bit inputs
// (significands of at most 11 bits) and d within [2^-64, 2^64] it is computed as
//     q0 = RN(x r);  e = x - d q0 (exact in one fma);  q = RN(q0 + e r)
// from any r within 2^-22 (relative) of 1/d, here the hardware's approximate reciprocal:
// q0 + e r differs from x/d by a relative 2^-44 at most, while a quotient of two 11-bit
// significands that is not itself an fp32 stays at least a relative 2^-36 away from every
// rounding boundary, and never sits on one.  The CPU tests check every significand pair
// with r perturbed by +-2 ulp.  Outside that window, and for fp32 inputs, the IEEE division
// is used.
//   BITS         8: the 256-entry codebook, one code per byte.  4: the 16-entry codebook of the 4-bit variant, two
//                codes per byte (quantize only, 16-bit inputs, the shared-memory flavour); everything up to
//                the search is the same code.
//   S16          (4-bit flavour only) the block's scale is its absmax rounded toward +infinity to a bf16, never above the
//                largest finite bf16; x is divided by that scale and its two bytes are what absmax_out receives.
template <int XDT, int B, int R, int TW, bool WRITE_Y, bool WRITE_Q, int NT, bool LITE, int BITS = 8, bool S16 = false>
__global__ void __launch_bounds__(NT, 1)
fwd_fast(const void* __restrict__ x, void* __restrict__ y, uint8_t* __restrict__ codes, float* __restrict__ absmax_out,
         size_t ntiles, const __grid_constant__ typename TabArg<BITS>::type tab) {
    static_assert(BITS == 8 || (BITS == 4 && !WRITE_Y && WRITE_Q && !LITE && Elem<XDT>::kPerChunk == 8), "the 4-bit flavour: quantize, 16-bit inputs, tables in shared memory");
    static_assert(!S16 || BITS == 4, "the 16-bit scale belongs to the 4-bit flavour");
    // the scale a block is divided by, from its absmax
    auto scale_of = [](float a) -> float {
        if constexpr (S16) return __uint_as_float(min((__float_as_uint(a) + 0xFFFFu) & 0xFFFF0000u, 0x7F7F0000u));
        else return a;
    };
    auto store_scale = [&](size_t i, float s) {
        if constexpr (S16) reinterpret_cast<uint16_t*>(absmax_out)[i] = uint16_t(__float_as_uint(s) >> 16);
        else absmax_out[i] = s;
    };
    constexpr int EPC = Elem<XDT>::kPerChunk;
    constexpr int EB = Elem<XDT>::kBytes;
    constexpr int ROW = 32 * EPC;
    constexpr bool IN_ROW = (B < ROW);                         // a block of exactly one row is a whole-warp reduction: the paths below
    constexpr int LPB = IN_ROW ? B / EPC : 32;                 // lanes per block inside a row
    constexpr int RPB = IN_ROW ? 1 : (B / ROW) / TW;           // rows of one warp that belong to one block
    constexpr int NBLK = R / RPB;                              // blocks per tile when blocks span rows
    static_assert(IN_ROW ? (TW == 1) : (RPB >= 1 && R % RPB == 0 && (TW == 1 || NBLK == 1)), "a tile holds whole blocks");
    constexpr int WARPS = NT / 32;
    static_assert(WARPS % TW == 0 && TW <= 15, "teams must tile the CTA, one named barrier each");

    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t sm_base = (uint32_t(__cvta_generic_to_shared(smem_raw)) + 127u) & ~127u;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t sm_lane = sm_base + uint32_t(lane) * 4u;
    auto make_tref = [&]() {
        if constexpr (BITS == 4) return TabRef4(sm_lane);
        else return TabRef<LITE>(tab, sm_lane);
    };
    const auto tref = make_tref();
    constexpr uint32_t RED = (BITS == 4) ? kRedOff4 : (LITE ? 0u : kRedOff);

    if constexpr (BITS == 4) {
        for (int i = threadIdx.x; i < kCells4 * 32; i += NT) sts_u32(sm_base + uint32_t(i) * 4u, tab.entry[i >> 5]);     // every entry once per lane
        __syncthreads();
    } else if constexpr (!LITE) {
        fill_fwd_tables<NT>(tab, sm_base);
        __syncthreads();
    }

    const float neg_limit = tab.neg_limit;
    const char* xb = static_cast<const char*>(x);
    char* yb = static_cast<char*>(y);

    constexpr size_t TILE = size_t(TW) * R * ROW;
    const size_t team = size_t(blockIdx.x) * (WARPS / TW) + size_t(warp / TW);
    const size_t nteams = size_t(gridDim.x) * (WARPS / TW);
    const int wt = warp % TW;
    const size_t lane_off = size_t(wt) * R * ROW + size_t(lane) * EPC;
    int parity = 0;

    uint4 w[R];
    auto load_tile = [&](size_t t) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            w[r] = ldg_stream_16(xb + (t * TILE + lane_off + size_t(r) * ROW) * EB);
        }
    };
    if (team < ntiles) load_tile(team);

    for (size_t t = team; t < ntiles; t += nteams) {
        const size_t base = t * TILE + lane_off;
        float f[R][EPC];
        float amax[R];
        uint32_t neg[R][2];                                        // sign bytes, taken before w is reused
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if constexpr (WRITE_Q) {
                if constexpr (EPC == 8) {
                    neg[r][0] = sign_mask_16(w[r].x, w[r].y);
                    neg[r][1] = sign_mask_16(w[r].z, w[r].w);
                } else {
                    neg[r][0] = sign_mask_32(w[r].x, w[r].y, w[r].z, w[r].w);
                }
            }
            widen_chunk<XDT>(w[r], f[r]);
            float a = 0.0f;
#pragma unroll
            for (int i = 0; i < EPC; i += 2) a = max3_abs(a, f[r][i], f[r][i + 1]);
            amax[r] = a;
        }
        if (t + nteams < ntiles) load_tile(t + nteams);          // in flight during everything below

        float d[R], rcv[R];                                        // divisor and its reciprocal, per row
        bool quick = false;                                        // warp-uniform: reciprocal route for the whole tile
        constexpr bool QUICK_OK = (XDT != kF32);
        if constexpr (IN_ROW) {
            // The tile holds R x (32 / LPB) blocks, at most one per lane.  A butterfly that hands
            // half of the rows to the partner lane at each of its first log2(R) steps leaves every
            // lane with the maximum of ONE row of its group (row rho below); the per-block scalars
            // (divisor, window test, reciprocal) are then computed once, by that lane, and handed
            // back with one shuffle per row, instead of by every lane for every row.
            constexpr int LOGR = (R == 8) ? 3 : (R == 4) ? 2 : (R == 2) ? 1 : 0;
            static_assert((1 << LOGR) == R && LPB >= R, "row-halving butterfly needs R a power of two and LPB >= R");
            float v[R];
#pragma unroll
            for (int r = 0; r < R; ++r) v[r] = amax[r];
#pragma unroll
            for (int s = 0; s < LOGR; ++s) {
                const bool up = (lane >> s) & 1;
                const int half = R >> (s + 1);
#pragma unroll
                for (int i = 0; i < half; ++i) {
                    const float keep = up ? v[i + half] : v[i];
                    const float send = up ? v[i] : v[i + half];
                    v[i] = fmaxf(keep, __shfl_xor_sync(0xffffffffu, send, 1 << s));
                }
            }
            float m = v[0];
#pragma unroll
            for (int s = R; s < LPB; s <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
            m = scale_of(m);
            // this lane's block: row rho = sum_s bit_s(lane) * (R >> (s+1)), group lane / LPB
            const float dm = (m != 0.0f) ? m : 1.0f;
            const float rm = QUICK_OK ? rcp_approx(dm) : 0.0f;
            if constexpr (QUICK_OK)
                quick = __all_sync(0xffffffffu, (dm >= 5.421010862427522e-20f) && (dm <= 1.8446744073709552e19f));    // 2^-64 .. 2^64
            if constexpr (WRITE_Q) {
                int rho = 0;
#pragma unroll
                for (int s = 0; s < LOGR; ++s) rho += ((lane >> s) & 1) * (R >> (s + 1));
                if ((lane % LPB) < R) store_scale((base + size_t(rho) * ROW) / B, m);
            }
            const int group_base = lane & ~(LPB - 1);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                int src = 0;                                        // the lane of the group that holds row r
#pragma unroll
                for (int s = 0; s < LOGR; ++s) src |= ((r >> (LOGR - 1 - s)) & 1) << s;
                amax[r] = __shfl_sync(0xffffffffu, m, group_base + src);
                d[r] = __shfl_sync(0xffffffffu, dm, group_base + src);
                if constexpr (QUICK_OK) rcv[r] = __shfl_sync(0xffffffffu, rm, group_base + src);
            }
        } else if constexpr (TW == 1) {
            // NBLK whole blocks of RPB rows each inside this warp
#pragma unroll
            for (int k = 0; k < NBLK; ++k) {
                float a = amax[k * RPB];
#pragma unroll
                for (int r = 1; r < RPB; ++r) a = fmaxf(a, amax[k * RPB + r]);
                a = scale_of(__uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(a))));
#pragma unroll
                for (int r = 0; r < RPB; ++r) amax[k * RPB + r] = a;
            }
        } else {
            float a = amax[0];
#pragma unroll
            for (int r = 1; r < R; ++r) a = fmaxf(a, amax[r]);
            a = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(a)));
            // partial maxima of the team's warps meet in shared memory; two slots alternate so
            // that one barrier per tile is enough
            const uint32_t slot = sm_base + RED + uint32_t(parity) * 128u + uint32_t(warp / TW) * TW * 4u;
            if (lane == 0) sts_u32(slot + uint32_t(wt) * 4u, __float_as_uint(a));
            asm volatile("bar.sync %0, %1;" ::"r"(1 + warp / TW), "r"(TW * 32) : "memory");
#pragma unroll
            for (int k = 0; k < TW; ++k) {
                uint32_t v;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(slot + uint32_t(k) * 4u) : "memory");
                a = fmaxf(a, __uint_as_float(v));
            }
            parity ^= 1;
            a = scale_of(a);
#pragma unroll
            for (int r = 0; r < R; ++r) amax[r] = a;
        }

        // normalise the whole tile in place; one warp-uniform choice between the reciprocal
        // route and the IEEE division keeps the per-element code free of branches
        if constexpr (!IN_ROW) {
            bool ok = QUICK_OK;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                d[r] = (amax[r] != 0.0f) ? amax[r] : 1.0f;
                ok = ok && (d[r] >= 5.421010862427522e-20f) && (d[r] <= 1.8446744073709552e19f);      // 2^-64 .. 2^64
                rcv[r] = QUICK_OK ? rcp_approx(d[r]) : 0.0f;
            }
            if constexpr (QUICK_OK) quick = __all_sync(0xffffffffu, ok);
        }
        if (quick) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const uint64_t r2 = pack2(rcv[r], rcv[r]), nd2 = pack2(-d[r], -d[r]);
#pragma unroll
                for (int i = 0; i < EPC; i += 2) {
                    const uint64_t x2 = pack2(f[r][i], f[r][i + 1]);
                    const uint64_t q0 = mul2(x2, r2);
                    const uint64_t e = fma2(nd2, q0, x2);
                    unpack2(fma2(e, r2, q0), f[r][i], f[r][i + 1]);
                }
            }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < EPC; ++i) f[r][i] = __fdiv_rn(f[r][i], d[r]);
        }

#pragma unroll
        for (int r = 0; r < R; ++r) {
            float out[EPC];
            Found fd[EPC];
#pragma unroll
            for (int i = 0; i < EPC; i += 2) {
                fd[i] = search_folded(f[r][i], neg_limit, tref);
                fd[i + 1] = search_folded(f[r][i + 1], neg_limit, tref);
                if constexpr (WRITE_Y) values_of(fd[i], fd[i + 1], amax[r], tref, out[i], out[i + 1]);
            }
            const size_t off = base + size_t(r) * ROW;
            {
                if constexpr (WRITE_Y) stg_stream_16(yb + off * EB, narrow_chunk<XDT>(out));
                if constexpr (WRITE_Q) {
                    if constexpr (BITS == 4) {
                        const uint32_t sums[8] = {fd[0].sum, fd[1].sum, fd[2].sum, fd[3].sum, fd[4].sum, fd[5].sum, fd[6].sum, fd[7].sum};
                        stg_stream_4(codes + off / 2, pack_nibbles8(sums, neg[r][0], neg[r][1]));
                    } else if constexpr (EPC == 8) {
                        stg_stream_8(codes + off, make_uint2(pack_codes(fd[0], fd[1], fd[2], fd[3], neg[r][0]), pack_codes(fd[4], fd[5], fd[6], fd[7], neg[r][1])));
                    } else {
                        stg_stream_4(codes + off, pack_codes(fd[0], fd[1], fd[2], fd[3], neg[r][0]));
                    }
                }
            }
        }
        if constexpr (WRITE_Q && !IN_ROW) {
            if (lane == 0 && wt == 0) {
#pragma unroll
                for (int k = 0; k < NBLK; ++k) store_scale(t * NBLK + k, amax[k * RPB]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// deq_fast: 16 codes per 128-bit load, U loads per thread per tile, signed code values
// replicated per lane in shared memory.  The loads of the next tile (codes and the blocks'
// absmax) are issued before the current tile is expanded.
#ifndef BQ_DEQ_MINB
#define BQ_DEQ_MINB 3
#endif
// WIDE: y is 32-byte aligned, so 16 outputs of a 16-bit type (8 of fp32) go out as one 256-bit
// store; otherwise (y only 16-byte aligned) the same bytes leave as two 128-bit stores.
template <int YDT, int NT, int U, bool LITE, bool WIDE>
__global__ void __launch_bounds__(NT, LITE ? 1 : BQ_DEQ_MINB)
deq_fast(const uint8_t* __restrict__ codes, const float* __restrict__ absmax, void* __restrict__ y, size_t n16 /* n / 16 */,
         int log2_block, DeviceTables tab) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t sm_base = uint32_t(__cvta_generic_to_shared(smem_raw));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t sm_lane = sm_base + uint32_t(lane) * 4u;
    if constexpr (!LITE) {
        // one coalesced load of 32 values per warp, then a shuffle hands each value to all lanes
        for (int row0 = warp * 32; row0 < 256; row0 += NT) {
            const uint32_t mine = __float_as_uint(__ldg(tab.values + row0 + lane));
#pragma unroll
            for (int k = 0; k < 32; ++k) sts_u32(sm_lane + uint32_t(row0 + k) * 128u, __shfl_sync(0xffffffffu, mine, k));
        }
        __syncthreads();
    } else {
        // one plain copy of the 256 values (kDeqLiteSmemBytes)
        for (int i = threadIdx.x; i < 256; i += NT) sts_u32(sm_base + uint32_t(i) * 4u, __float_as_uint(__ldg(tab.values + i)));
        __syncthreads();
    }
    // value of one code byte sitting at bit `shift` of a packed word
    auto value = [&](uint32_t word, int shift) -> float {
        if constexpr (LITE) {
            const uint32_t off = (shift >= 2 ? (word >> (shift - 2)) : (word << (2 - shift))) & 0x3fcu;
            return __uint_as_float(lds_u32(sm_base + off));
        } else {
            const uint32_t row = (shift >= 7 ? (word >> (shift - 7)) : (word << (7 - shift))) & 0x7f80u;
            return __uint_as_float(lds_u32(sm_lane + row));
        }
    };

    char* yb = static_cast<char*>(y);
    constexpr int EB = Elem<YDT>::kBytes;
    constexpr size_t TILE = size_t(NT) * U;                      // chunks per tile
    const size_t ntiles = (n16 + TILE - 1) / TILE;
    const int log2_chunks = log2_block - 4;                      // chunks per block

    uint4 w[U];
    float a[U];
    auto load_tile = [&](size_t t) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t c = t * TILE + size_t(u) * NT + threadIdx.x;
            const bool ok = c < n16;
            w[u] = ok ? ldg_stream_16(codes + c * 16) : make_uint4(0, 0, 0, 0);
            a[u] = ok ? __ldg(absmax + (c >> log2_chunks)) : 0.0f;
        }
    };
    if (blockIdx.x < ntiles) load_tile(blockIdx.x);
    for (size_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        uint4 cw[U];
        float ca[U];
#pragma unroll
        for (int u = 0; u < U; ++u) { cw[u] = w[u]; ca[u] = a[u]; }
        if (t + gridDim.x < ntiles) load_tile(t + gridDim.x);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t c = t * TILE + size_t(u) * NT + threadIdx.x;
            if (c >= n16) continue;
            const uint32_t q[4] = {cw[u].x, cw[u].y, cw[u].z, cw[u].w};
            float v[16];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                v[4 * k + 0] = __fmul_rn(value(q[k], 0), ca[u]);
                v[4 * k + 1] = __fmul_rn(value(q[k], 8), ca[u]);
                v[4 * k + 2] = __fmul_rn(value(q[k], 16), ca[u]);
                v[4 * k + 3] = __fmul_rn(value(q[k], 24), ca[u]);
            }
            char* out = yb + c * 16 * EB;
            if constexpr (YDT == kF32) {
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const float t0[4] = {v[8 * k], v[8 * k + 1], v[8 * k + 2], v[8 * k + 3]};
                    const float t1[4] = {v[8 * k + 4], v[8 * k + 5], v[8 * k + 6], v[8 * k + 7]};
                    store_32<WIDE>(out + 32 * k, narrow_chunk<kF32>(t0), narrow_chunk<kF32>(t1));
                }
            } else {
                const float t0[8] = {v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]};
                const float t1[8] = {v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15]};
                store_32<WIDE>(out, narrow_chunk<YDT>(t0), narrow_chunk<YDT>(t1));
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// General kernels: any block, any alignment, any valid codebook.  One warp per block, two
// passes over the block (the second pass hits L1/L2), 8-step branch-free binary search over
// the 255 round-down midpoints in shared memory.

__device__ __forceinline__ int search_general(const float* thr /* shared, 256 entries */, float xhat) {
    int q = 0;
#pragma unroll
    for (int s = 128; s >= 1; s >>= 1) q += (thr[q + s - 1] < xhat) ? s : 0;
    return q;
}

template <int XDT, int YDT, bool WRITE_Y, bool WRITE_Q>
__global__ void __launch_bounds__(256)
fwd_general(const void* __restrict__ x, void* __restrict__ y, uint8_t* __restrict__ codes, float* __restrict__ absmax_out,
            size_t n, size_t block, size_t first_block, DeviceTables tab) {
    __shared__ float thr[256];
    __shared__ float val[256];
    thr[threadIdx.x] = tab.thr_down[threadIdx.x];
    val[threadIdx.x] = tab.values[threadIdx.x];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const size_t nb = (n + block - 1) / block;
    const size_t wstride = size_t(gridDim.x) * 8;
    for (size_t b = first_block + size_t(blockIdx.x) * 8 + (threadIdx.x >> 5); b < nb; b += wstride) {
        const size_t lo = b * block;
        const size_t hi = (lo + block < n) ? lo + block : n;
        float a = 0.0f;
        for (size_t i = lo + lane; i < hi; i += 32) a = fmaxf(a, fabsf(load_elem<XDT>(x, i)));
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, s));
        const float d = (a != 0.0f) ? a : 1.0f;
        for (size_t i = lo + lane; i < hi; i += 32) {
            const float xhat = __fdiv_rn(load_elem<XDT>(x, i), d);
            const int q = search_general(thr, xhat);
            if constexpr (WRITE_Q) codes[i] = uint8_t(q);
            if constexpr (WRITE_Y) store_elem<YDT>(y, i, __fmul_rn(val[q], a));
        }
        if constexpr (WRITE_Q) {
            if (lane == 0) absmax_out[b] = a;
        }
    }
}

template <int YDT>
__global__ void __launch_bounds__(256)
deq_general(const uint8_t* __restrict__ codes, const float* __restrict__ absmax, void* __restrict__ y, size_t n, size_t block,
            size_t first_elem, DeviceTables tab) {
    __shared__ float val[256];
    val[threadIdx.x] = tab.values[threadIdx.x];
    __syncthreads();
    const size_t stride = size_t(gridDim.x) * 256;
    for (size_t i = first_elem + size_t(blockIdx.x) * 256 + threadIdx.x; i < n; i += stride)
        store_elem<YDT>(y, i, __fmul_rn(val[codes[i]], absmax[i / block]));
}

}  // namespace bqk
