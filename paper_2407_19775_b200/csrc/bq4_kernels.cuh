// bq4_kernels.cuh -- device code of the 4-bit variant (sm_100a).
//
//   q4_fast    : power-of-two blocks of 8..256 elements.  One thread per 8 elements (one or two
//                128-bit loads), block absmax by a segmented shuffle over block / 8 lanes, codes
//                by a 4-step branch-free search over the 15 thresholds in shared memory, eight
//                nibbles per 32-bit store.  Two chunks per thread and trip, persistent grid.
//   q4_wide    : power-of-two blocks of 512..65536: one warp per block, two passes over it (the
//                second hits L1 / L2).
//   dq4_fast   : 16 codes per 64-bit load, values from shared memory, 256-bit or 2 x 256-bit stores.
//   *_general  : any block, any alignment: absmax per block, then one thread per byte.
//
// Arithmetic contract, as for the 8-bit kernels: exact fp32 absmax; the correctly rounded
// quotient (for 16-bit inputs and divisors within [2^-64, 2^64] through the reciprocal route
// whose exactness the CPU tests check over every pair of significands; IEEE division
// otherwise); code = #{ j : t_j < xhat } over midpoints rounded toward -inf; one fp32 multiply
// and a round-to-nearest-even narrowing on the way back.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bq4k {

enum { kF32 = 0, kF16 = 1, kBF16 = 2 };

constexpr int kFoldCells = 73;          // cells of 2^21 keys from the key of 2^-9 up to the key of -1.0
constexpr uint32_t kFoldKeyLow = 0x76000000u;      // key of +2^-9 (twice its bit pattern)
constexpr uint32_t kFoldCellBase = kFoldKeyLow >> 21;

struct Tables4 {
    float thr[16];      // [0..14] midpoints rounded toward -inf, [15] = +inf
    float val[16];      // the codebook
    // Folded search, valid when `folded` is set (a codebook that mirrors around code 7 with one extra top value, such as
    // the dynamic tree).  key = rotate-left-by-one of xhat's bits = 2 bits(|xhat|) + sign.  With the threshold keys
    // TK[p] = 2 bits(round_down(theta_p)) + (theta_p is not an fp32) of the positive midpoints, P = #{TK[p] < key} is
    // #{theta_p < |xhat|} for xhat >= 0 and #{theta_p <= |xhat|} for xhat < 0: the tie rule on either side.  Keys are
    // clamped from below to kFoldKeyLow and cut into cells of 2^21 keys (exponent and 3 fraction bits); no cell holds
    // two thresholds.  For the cell that starts at key S, with P0 thresholds below S and the threshold TK in it:
    //     E = ((7 + P0) << 24 | 0xE00000 | (0x1FFFFF - (TK - S))) - S, and (E + key) >> 24 = 7 + P0 + [key > TK]:
    // the low 21 bits carry through the three set bits into the top byte, which is the code of a non-negative xhat.
    // (No threshold in the cell: TK - S = 0x1FFFFF, which never carries.)  A negative xhat takes 7 - P = (c ^ 0xF) - 1
    // from the same byte c, applied to four elements at a time once the bytes are gathered in a word; xhat is clamped
    // from below to neg_limit first, so that P <= 7 there (there is no code for -1.0).
    uint32_t entry[kFoldCells];
    float neg_limit;                    // -(largest |xhat| whose negative key does not pass the top threshold)
    int folded;
};

template <int DT>
__device__ __forceinline__ float load1(const void* x, size_t i) {
    if constexpr (DT == kF32) return static_cast<const float*>(x)[i];
    else if constexpr (DT == kBF16) return __uint_as_float(uint32_t(static_cast<const uint16_t*>(x)[i]) << 16);
    else return __half2float(static_cast<const __half*>(x)[i]);
}
template <int DT>
__device__ __forceinline__ void store1(void* y, size_t i, float v) {
    if constexpr (DT == kF32) static_cast<float*>(y)[i] = v;
    else if constexpr (DT == kBF16) static_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
    else static_cast<__half*>(y)[i] = __float2half_rn(v);
}

// eight consecutive elements starting at element 8 c
template <int DT>
__device__ __forceinline__ void load8(const void* x, size_t c, float (&f)[8]) {
    if constexpr (DT == kF32) {
        const float4* p = reinterpret_cast<const float4*>(x) + 2 * c;
        const float4 a = p[0], b = p[1];
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    } else {
        const uint4 w = reinterpret_cast<const uint4*>(x)[c];
        const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (DT == kBF16) {
                f[2 * i] = __uint_as_float(u[i] << 16);
                f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
            } else {
                const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&u[i]));
                f[2 * i] = p.x;
                f[2 * i + 1] = p.y;
            }
        }
    }
}

// the same eight elements from the raw 128-bit words of a chunk (one word for 16-bit types, two for fp32)
template <int DT, int W>
__device__ __forceinline__ void widen_chunk(const uint4 (&w)[W], float (&f)[8]) {
    if constexpr (DT == kF32) {
        f[0] = __uint_as_float(w[0].x); f[1] = __uint_as_float(w[0].y); f[2] = __uint_as_float(w[0].z); f[3] = __uint_as_float(w[0].w);
        f[4] = __uint_as_float(w[1].x); f[5] = __uint_as_float(w[1].y); f[6] = __uint_as_float(w[1].z); f[7] = __uint_as_float(w[1].w);
    } else {
        const uint32_t u[4] = {w[0].x, w[0].y, w[0].z, w[0].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (DT == kBF16) {
                f[2 * i] = __uint_as_float(u[i] << 16);
                f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
            } else {
                const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&u[i]));
                f[2 * i] = p.x;
                f[2 * i + 1] = p.y;
            }
        }
    }
}

__device__ __forceinline__ uint32_t search16(const float* thr, float xhat) {
    uint32_t q = 0;
#pragma unroll
    for (int s = 8; s >= 1; s >>= 1) q += (thr[q + s - 1] < xhat) ? s : 0;
    return q;
}

// xhat = RN32(x / d).  16-bit inputs with d in [2^-64, 2^64]: q0 = RN(x r), e = x - d q0 (exact
// in one fma), q = RN(q0 + e r) from the approximate reciprocal r; otherwise the IEEE division.
template <int DT>
__device__ __forceinline__ float quotient(float x, float d, float r, bool quick) {
    if (DT != kF32 && quick) {
        const float q0 = __fmul_rn(x, r);
        const float e = __fmaf_rn(-d, q0, x);
        return __fmaf_rn(e, r, q0);
    }
    return __fdiv_rn(x, d);
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// 0xFF in the byte of every negative element: four fp32 values, or four 16-bit elements held in two words (the
// permute's sign-replicate mode copies a sign bit over a whole byte)
__device__ __forceinline__ uint32_t sign_bytes_32(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return prmt(prmt(a, b, 0x00FBu), prmt(c, d, 0x00FBu), 0x5410u);
}
__device__ __forceinline__ uint32_t sign_bytes_16(uint32_t w0, uint32_t w1) { return prmt(w0, w1, 0xFDB9u); }

// entry + key of one xhat through the folded table: the top byte of the result is 7 + P.  `ent_lane` is this lane's column
// of the per-lane replicated entries, rebased by the index of the first cell.  The address step is a multiply-add on
// purpose: the integer ALU is the busiest pipe of these kernels, the fp32 pipe has room.
__device__ __forceinline__ uint32_t folded_sum16(uint32_t ent_lane, float xhat, float neg_limit) {
    const uint32_t b = __float_as_uint(fmaxf(xhat, neg_limit));
    const uint32_t key = max(__funnelshift_l(b, b, 1), kFoldKeyLow);
    uint32_t addr, e;
    asm("mad.lo.u32 %0, %1, 128, %2;" : "=r"(addr) : "r"(key >> 21), "r"(ent_lane));
    asm("ld.shared.u32 %0, [%1];" : "=r"(e) : "r"(addr));
    return e + key;
}
// Eight codes as eight nibbles.  The top bytes c = 7 + P of the sums are gathered four to a word; negative elements
// (0xFF in `neg0` / `neg1`) take 7 - P = (c ^ 0xF) - 1, which cannot borrow between bytes because c <= 14 there, and the
// "-1 in every negative byte" is neg * 0x01010101 (neg = 255 * (neg & 0x01010101), and 255 * 0x01010101 = -1 mod 2^32);
// then byte pairs fold into nibble pairs: x | x >> 4 leaves [q1 q0] in byte 0 and [q3 q2] in byte 2.
__device__ __forceinline__ uint32_t pack_nibbles8(const uint32_t (&sum)[8], uint32_t neg0, uint32_t neg1) {
    uint32_t c0 = prmt(prmt(sum[0], sum[1], 0x0073u), prmt(sum[2], sum[3], 0x0073u), 0x5410u);
    uint32_t c1 = prmt(prmt(sum[4], sum[5], 0x0073u), prmt(sum[6], sum[7], 0x0073u), 0x5410u);
    asm("mad.lo.u32 %0, %1, 0x01010101, %2;" : "=r"(c0) : "r"(neg0), "r"(c0 ^ (neg0 & 0x0F0F0F0Fu)));
    asm("mad.lo.u32 %0, %1, 0x01010101, %2;" : "=r"(c1) : "r"(neg1), "r"(c1 ^ (neg1 & 0x0F0F0F0Fu)));
    return prmt(c0 | (c0 >> 4), c1 | (c1 >> 4), 0x6420u);
}
// the codes of eight normalised values as one word of nibbles: the folded table, or the 4-step search over the thresholds
template <bool FOLDED>
__device__ __forceinline__ uint32_t codes8(const float (&xh)[8], uint32_t ent_lane, float neg_limit, const float* thr, uint32_t neg0, uint32_t neg1) {
    if constexpr (FOLDED) {
        uint32_t sum[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) sum[i] = folded_sum16(ent_lane, xh[i], neg_limit);
        return pack_nibbles8(sum, neg0, neg1);
    } else {
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) word |= search16(thr, xh[i]) << (4 * i);
        return word;
    }
}

// two fp32 lanes per instruction (sm_100 packed fp32 arithmetic)
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

// xhat of eight elements by one route for all of them (`quick` is uniform over the warp): the reciprocal route two
// quotients per instruction (q0 = x r; e = x - d q0; q = q0 + e r), or the IEEE division.
__device__ __forceinline__ void quotients8(const float (&f)[8], float d, float r, bool quick, float (&xh)[8]) {
    if (quick) {
        const uint64_t r2 = pack2(r, r), nd2 = pack2(-d, -d);
#pragma unroll
        for (int i = 0; i < 8; i += 2) {
            const uint64_t x2 = pack2(f[i], f[i + 1]);
            const uint64_t q0 = mul2(x2, r2);
            const uint64_t e = fma2(nd2, q0, x2);
            unpack2(fma2(e, r2, q0), xh[i], xh[i + 1]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) xh[i] = __fdiv_rn(f[i], d);
    }
}

// The scale of a block.  Plain form: its absmax as an fp32.  S16 form: the absmax rounded toward +infinity to a bf16 (so
// that no |x| / scale exceeds 1), never above the largest finite bf16; the two stored bytes are the bf16 itself.  The
// `absmax` arguments of the kernels point at floats or, with S16, at 16-bit words.
template <bool S16>
__device__ __forceinline__ float block_scale(float a /* >= 0 */) {
    if constexpr (!S16) return a;
    else return __uint_as_float(min((__float_as_uint(a) + 0xFFFFu) & 0xFFFF0000u, 0x7F7F0000u));
}
template <bool S16>
__device__ __forceinline__ void store_scale(float* p, size_t i, float s) {
    if constexpr (!S16) p[i] = s;
    else reinterpret_cast<uint16_t*>(p)[i] = uint16_t(__float_as_uint(s) >> 16);
}
template <bool S16>
__device__ __forceinline__ float load_scale(const float* p, size_t i) {
    if constexpr (!S16) return __ldg(p + i);
    else return __uint_as_float(uint32_t(__ldg(reinterpret_cast<const uint16_t*>(p) + i)) << 16);
}

__device__ __forceinline__ void fill_tables(const Tables4& tab, float* thr, float* val) {
    if (threadIdx.x < 16) { thr[threadIdx.x] = tab.thr[threadIdx.x]; val[threadIdx.x] = tab.val[threadIdx.x]; }
    __syncthreads();
}

template <int DT, bool FOLDED, int LOG2_LPB /* log2 of the lanes per block = log2(block / 8) */, bool S16 = false>
__global__ void __launch_bounds__(256)
q4_fast(const void* __restrict__ x, uint8_t* __restrict__ packed, float* __restrict__ absmax, size_t nchunks, const __grid_constant__ Tables4 tab) {
    constexpr int lpb = 1 << LOG2_LPB;
    constexpr int log2_lpb = LOG2_LPB;
    __shared__ float thr[16], val[16];
    __shared__ __align__(128) uint32_t ent[FOLDED ? kFoldCells * 32 : 1];      // every entry once per lane, in that lane's bank
    fill_tables(tab, thr, val);
    uint32_t ent_lane = 0;
    if constexpr (FOLDED) {
        for (int i = threadIdx.x; i < kFoldCells * 32; i += 256) ent[i] = tab.entry[i >> 5];
        __syncthreads();
        ent_lane = uint32_t(__cvta_generic_to_shared(ent)) + (threadIdx.x & 31) * 4u - kFoldCellBase * 128u;
    }
    const float neg_limit = tab.neg_limit;
    const size_t stride = size_t(gridDim.x) * 256;
    // Two chunks per trip; the loads of the next trip are issued before this trip's arithmetic.  The trip count is the
    // same for the whole warp because chunk indices start at a multiple of 32 and the shuffles need every lane.
    const size_t first = size_t(blockIdx.x) * 256 + threadIdx.x;
    const size_t warp_first = first - (threadIdx.x & 31);
    constexpr int W = (DT == kF32) ? 2 : 1;                      // 128-bit loads per chunk
    uint4 nxt[2][W];
    auto fetch = [&](size_t c0) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const size_t c = c0 + size_t(u) * stride;
#pragma unroll
            for (int k = 0; k < W; ++k)
                nxt[u][k] = (c < nchunks) ? __ldg(reinterpret_cast<const uint4*>(x) + c * W + k) : make_uint4(0, 0, 0, 0);
        }
    };
    if (warp_first < nchunks) fetch(first);
    for (size_t c0 = first, w0 = warp_first; w0 < nchunks; c0 += 2 * stride, w0 += 2 * stride) {
        float f[2][8];
        uint32_t neg[2][2];                                         // sign bytes of the eight elements, taken before the words are reused
        const size_t c[2] = {c0, c0 + stride};
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if constexpr (DT == kF32) {
                neg[u][0] = sign_bytes_32(nxt[u][0].x, nxt[u][0].y, nxt[u][0].z, nxt[u][0].w);
                neg[u][1] = sign_bytes_32(nxt[u][W - 1].x, nxt[u][W - 1].y, nxt[u][W - 1].z, nxt[u][W - 1].w);
            } else {
                neg[u][0] = sign_bytes_16(nxt[u][0].x, nxt[u][0].y);
                neg[u][1] = sign_bytes_16(nxt[u][0].z, nxt[u][0].w);
            }
            widen_chunk<DT>(nxt[u], f[u]);
        }
        if (w0 + 2 * stride < nchunks) fetch(c0 + 2 * stride);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            float a = 0.0f;
#pragma unroll
            for (int i = 0; i < 8; i += 2) asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(a) : "f"(a), "f"(f[u][i]), "f"(f[u][i + 1]));     // max(|a|, |x|, |y|)
#pragma unroll
            for (int s = 1; s < lpb; s <<= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, s));
            a = block_scale<S16>(a);
            const float d = (a != 0.0f) ? a : 1.0f;
            // one choice of route for the whole warp keeps the per-element code free of branches
            const bool quick = (DT != kF32) && __all_sync(0xffffffffu, (d >= 5.421010862427522e-20f) && (d <= 1.8446744073709552e19f));
            float r;
            asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(d));
            float xh[8];
            quotients8(f[u], d, r, quick, xh);
            const uint32_t word = codes8<FOLDED>(xh, ent_lane, neg_limit, thr, neg[u][0], neg[u][1]);
            if (c[u] < nchunks) {
                reinterpret_cast<uint32_t*>(packed)[c[u]] = word;
                if ((c[u] & size_t(lpb - 1)) == 0) store_scale<S16>(absmax, c[u] >> log2_lpb, a);
            }
        }
    }
}

template <int DT, bool FOLDED, bool S16 = false>
__global__ void __launch_bounds__(256)
q4_wide(const void* __restrict__ x, uint8_t* __restrict__ packed, float* __restrict__ absmax, size_t nblocks, int chunks_per_block,
        const __grid_constant__ Tables4 tab) {
    __shared__ float thr[16], val[16];
    __shared__ __align__(128) uint32_t ent[FOLDED ? kFoldCells * 32 : 1];
    fill_tables(tab, thr, val);
    uint32_t ent_lane = 0;
    if constexpr (FOLDED) {
        for (int i = threadIdx.x; i < kFoldCells * 32; i += 256) ent[i] = tab.entry[i >> 5];
        __syncthreads();
        ent_lane = uint32_t(__cvta_generic_to_shared(ent)) + (threadIdx.x & 31) * 4u - kFoldCellBase * 128u;
    }
    const float neg_limit = tab.neg_limit;
    const int lane = threadIdx.x & 31;
    const size_t wstride = size_t(gridDim.x) * 8;
    for (size_t b = size_t(blockIdx.x) * 8 + (threadIdx.x >> 5); b < nblocks; b += wstride) {
        const size_t cbase = b * size_t(chunks_per_block);
        float a = 0.0f;
        for (int k = lane; k < chunks_per_block; k += 32) {
            float f[8];
            load8<DT>(x, cbase + k, f);
#pragma unroll
            for (int i = 0; i < 8; ++i) a = fmaxf(a, fabsf(f[i]));
        }
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, s));
        a = block_scale<S16>(a);
        const float d = (a != 0.0f) ? a : 1.0f;
        const bool quick = (DT != kF32) && (d >= 5.421010862427522e-20f) && (d <= 1.8446744073709552e19f);      // one block per warp: uniform
        float r;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(d));
        for (int k = lane; k < chunks_per_block; k += 32) {
            float f[8], xh[8];
            load8<DT>(x, cbase + k, f);
            quotients8(f, d, r, quick, xh);
            // the quotients carry the signs of the inputs
            const uint32_t neg0 = sign_bytes_32(__float_as_uint(xh[0]), __float_as_uint(xh[1]), __float_as_uint(xh[2]), __float_as_uint(xh[3]));
            const uint32_t neg1 = sign_bytes_32(__float_as_uint(xh[4]), __float_as_uint(xh[5]), __float_as_uint(xh[6]), __float_as_uint(xh[7]));
            reinterpret_cast<uint32_t*>(packed)[cbase + k] = codes8<FOLDED>(xh, ent_lane, neg_limit, thr, neg0, neg1);
        }
        if (lane == 0) store_scale<S16>(absmax, b, a);
    }
}

// General quantize, step 1: absmax of blocks first_block .. (one warp per block).
template <int DT, bool S16 = false>
__global__ void __launch_bounds__(256)
q4_general_absmax(const void* __restrict__ x, float* __restrict__ absmax, size_t n, size_t block, size_t first_block) {
    const int lane = threadIdx.x & 31;
    const size_t nb = (n + block - 1) / block;
    for (size_t b = first_block + size_t(blockIdx.x) * 8 + (threadIdx.x >> 5); b < nb; b += size_t(gridDim.x) * 8) {
        const size_t lo = b * block, hi = (lo + block < n) ? lo + block : n;
        float a = 0.0f;
        for (size_t i = lo + lane; i < hi; i += 32) a = fmaxf(a, fabsf(load1<DT>(x, i)));
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, s));
        if (lane == 0) store_scale<S16>(absmax, b, block_scale<S16>(a));
    }
}

// General quantize, step 2: one thread per output byte from byte first_byte on.
template <int DT, bool S16 = false>
__global__ void __launch_bounds__(256)
q4_general_codes(const void* __restrict__ x, const float* __restrict__ absmax, uint8_t* __restrict__ packed, size_t n, size_t block,
                 size_t first_byte, const __grid_constant__ Tables4 tab) {
    __shared__ float thr[16], val[16];
    fill_tables(tab, thr, val);
    const size_t nbytes = (n + 1) / 2;
    for (size_t j = first_byte + size_t(blockIdx.x) * 256 + threadIdx.x; j < nbytes; j += size_t(gridDim.x) * 256) {
        uint32_t byte = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const size_t i = 2 * j + h;
            if (i < n) {
                const float a = load_scale<S16>(absmax, i / block);
                const float d = (a != 0.0f) ? a : 1.0f;
                byte |= search16(thr, __fdiv_rn(load1<DT>(x, i), d)) << (4 * h);
            }
        }
        packed[j] = uint8_t(byte);
    }
}

__device__ __forceinline__ void st32(void* p, const uint32_t (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]),
                 "r"(w[6]), "r"(w[7]) : "memory");
}

// 16 elements per thread; block is a power of two >= 16, so the 16 share one absmax.
template <int DT, bool S16 = false>
__global__ void __launch_bounds__(256)
dq4_fast(const uint8_t* __restrict__ packed, const float* __restrict__ absmax, void* __restrict__ y, size_t n16, int log2_block,
         const __grid_constant__ Tables4 tab) {
    __shared__ float thr[16], val[16];
    fill_tables(tab, thr, val);
    for (size_t c = size_t(blockIdx.x) * 256 + threadIdx.x; c < n16; c += size_t(gridDim.x) * 256) {
        const uint2 w = reinterpret_cast<const uint2*>(packed)[c];
        const float a = load_scale<S16>(absmax, (c * 16) >> log2_block);
        float v[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            v[i] = __fmul_rn(val[(w.x >> (4 * i)) & 15u], a);
            v[8 + i] = __fmul_rn(val[(w.y >> (4 * i)) & 15u], a);
        }
        if constexpr (DT == kF32) {
            uint32_t lo[8], hi[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { lo[i] = __float_as_uint(v[i]); hi[i] = __float_as_uint(v[8 + i]); }
            st32(static_cast<char*>(y) + c * 64, lo);
            st32(static_cast<char*>(y) + c * 64 + 32, hi);
        } else {
            uint32_t pk[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if constexpr (DT == kBF16) {
                    const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                    pk[i] = *reinterpret_cast<const uint32_t*>(&h);
                } else {
                    const __half2 h = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
                    pk[i] = *reinterpret_cast<const uint32_t*>(&h);
                }
            }
            st32(static_cast<char*>(y) + c * 32, pk);
        }
    }
}

template <int DT, bool S16 = false>
__global__ void __launch_bounds__(256)
dq4_general(const uint8_t* __restrict__ packed, const float* __restrict__ absmax, void* __restrict__ y, size_t n, size_t block, size_t first_elem,
            const __grid_constant__ Tables4 tab) {
    __shared__ float thr[16], val[16];
    fill_tables(tab, thr, val);
    for (size_t i = first_elem + size_t(blockIdx.x) * 256 + threadIdx.x; i < n; i += size_t(gridDim.x) * 256) {
        const uint32_t code = (packed[i >> 1] >> (4 * (i & 1))) & 15u;
        store1<DT>(y, i, __fmul_rn(val[code], load_scale<S16>(absmax, i / block)));
    }
}

}  // namespace bq4k
