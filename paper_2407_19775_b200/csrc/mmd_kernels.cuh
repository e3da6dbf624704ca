// mmd_kernels.cuh -- device code of the mixed matrix decomposition (sm_100a).
//
//   rowquant      : per row absmax over the regular features, int8 codes, row scale and the
//                   16-bit side columns of the critical features.  One CTA per row.
//   gemm_general  : Y = fma(fp32(qx qw^T), sx sw, sidex sidew^T) with integer dot products
//                   (dp4a) for any M and N; the correctness path and the fallback.
//   gemm_tc       : the same on the 5th-generation tensor cores: TMA loads 128-byte-swizzled
//                   tiles into a 4-stage shared-memory ring, one thread issues tcgen05.mma
//                   (kind::i8 into an int32 accumulator in tensor memory, then kind::f16 for
//                   the side columns into a second, fp32 accumulator), four warps read both
//                   accumulators back with tcgen05.ld and apply the scales.
//
// Arithmetic contract (it is what makes the integer part bit-identical to the plain
// definition): 127 v is exact in fp32 for 16-bit v; one IEEE division; cvt.rni (ties to
// even); int32 sums are exact; the output is one fma and one round-to-nearest-even narrowing.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mmdk {

enum { kF32 = 0, kF16 = 1, kBF16 = 2 };

constexpr int kSidePad = 64;

template <int DT>
__device__ __forceinline__ float widen16(uint32_t bits16) {
    if constexpr (DT == kBF16) return __uint_as_float(bits16 << 16);
    else return __half2float(__ushort_as_half(static_cast<unsigned short>(bits16)));
}

template <int DT>
__device__ __forceinline__ void widen8(const uint4& w, float (&f)[8]) {
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = widen16<DT>(u[i] & 0xffffu);
        f[2 * i + 1] = widen16<DT>(u[i] >> 16);
    }
}

// ------------------------------------------------------------------------------------------
// rowquant: one CTA of 256 threads per row.  A bit mask of the critical features sits in
// shared memory, one byte per 16-byte chunk of the row, so the regular path costs one byte
// load per eight elements.  The row is read twice (the second pass hits L1 / L2).
//
// The kernel is bound by instruction issue, so both passes are written for few instructions:
// the absmax pass works on the packed 16-bit patterns (the magnitudes of finite fp16 / bf16
// values order like their bit patterns: one mask and one two-lane unsigned max per pair), the
// code pass does its fp32 arithmetic two elements per instruction, rounds to an integer by
// adding 1.5 * 2^23 (round-to-nearest-even, the low byte of the sum's bit pattern is the int8
// code) and gathers the four low bytes of a word with byte permutes.  A chunk that holds a
// critical feature (rare) takes a slower masked path.
__device__ __forceinline__ uint64_t rq_pack2(float a, float b) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(a), "f"(b));
    return v;
}
__device__ __forceinline__ uint64_t rq_mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t rq_fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t rq_add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t rq_prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// per-halfword unsigned maximum
__device__ __forceinline__ uint32_t rq_max_u16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// 0xffff in the halves of word j (elements 2j, 2j + 1 of the chunk) whose mask bit is clear
__device__ __forceinline__ uint32_t rq_keep_halves(uint32_t mk, int j) {
    return (((mk >> (2 * j)) & 1u) ? 0u : 0x0000ffffu) | (((mk >> (2 * j + 1)) & 1u) ? 0u : 0xffff0000u);
}
// 0xff in the bytes of code word h (elements 4h .. 4h + 3 of the chunk) whose mask bit is clear
__device__ __forceinline__ uint32_t rq_keep_bytes(uint32_t mk, int h) {
    uint32_t keep = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) keep |= ((mk >> (4 * h + i)) & 1u) ? 0u : (0xffu << (8 * i));
    return keep;
}

template <int DT>
__global__ void __launch_bounds__(256, 6)                        // six CTAs per SM: the row's second read then mostly hits L1 / L2 while others load
rowquant(const void* __restrict__ v, int R, int K, const int32_t* __restrict__ idx, int ko, int side_cols,
         int8_t* __restrict__ q_out, float* __restrict__ scale_out, void* __restrict__ side_out,
         int* __restrict__ zero_words, int n_zero_words /* counters of the product kernel that follows; may be none */) {
    extern __shared__ __align__(16) unsigned char mask[];       // K / 8 bytes
    __shared__ uint32_t red[8];
    // A product kernel launched behind this one with programmatic stream serialization may start its set-up and its
    // weight loads now; it waits (griddepcontrol.wait) for this grid's results before it reads them.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int nchunks = K / 8;
    for (int c = threadIdx.x; c < (nchunks + 3) / 4; c += 256) reinterpret_cast<uint32_t*>(mask)[c] = 0u;
    // This kernel is itself launched with programmatic stream serialization: behind a product kernel that lets its
    // dependents start early (a chain of layers) its CTAs are already resident when that kernel ends.  Everything it reads
    // from or writes to global memory comes after this wait for the kernels before it (the product kernel of the previous
    // call may still be reading the buffers written below).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();
    if (blockIdx.x == 0)
        for (int j = threadIdx.x; j < n_zero_words; j += 256) zero_words[j] = 0;
    for (int j = threadIdx.x; j < ko; j += 256) {
        const int k = idx[j];
        atomicOr(reinterpret_cast<uint32_t*>(mask) + (k >> 5), 1u << (k & 31));
    }
    __syncthreads();

    for (int r = blockIdx.x; r < R; r += gridDim.x) {
        const uint4* row = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(v) + size_t(r) * K);
        uint32_t m2 = 0u;                                                       // two running maxima of 15-bit magnitudes
        for (int c0 = threadIdx.x; c0 < nchunks; c0 += 256 * 4) {               // four loads in flight per thread
            uint4 w[4];
            uint32_t mk[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = c0 + 256 * u;
                const bool in = c < nchunks;
                w[u] = in ? row[c] : make_uint4(0, 0, 0, 0);
                mk[u] = in ? uint32_t(mask[c]) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint32_t x[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
                if (mk[u] != 0u) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) x[j] &= rq_keep_halves(mk[u], j);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) m2 = rq_max_u16x2(m2, x[j] & 0x7fff7fffu);
            }
        }
        m2 = max(m2 & 0xffffu, m2 >> 16);
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) m2 = max(m2, __shfl_xor_sync(0xffffffffu, m2, s));
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m2;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 8; ++i) m2 = max(m2, red[i]);
        const float a = widen16<DT>(m2);
        const float d = (a != 0.0f) ? a : 1.0f;
        if (threadIdx.x == 0) scale_out[r] = __fdiv_rn(a, 127.0f);
        // t = RN32(127 v / d).  n = 127 v is exact; for d within [2^-64, 2^64]: q0 = RN(n rc), e = n - d q0 (exact in one
        // fma), t = RN(q0 + e rc) from the approximate reciprocal rc (within 1 ulp of 1 / d).  q0 + e rc is within a relative
        // 2^-44 of n / d while a quotient with an 11-bit divisor that is not itself an fp32 stays a relative 2^-36 away from
        // every rounding boundary, so t is the IEEE quotient (the CPU tests check every pair of 16-bit significands with rc
        // off by up to 2 ulp).  Outside the window: the IEEE division.  d is the same for the whole CTA.
        const bool quick = (d >= 5.421010862427522e-20f) && (d <= 1.8446744073709552e19f);
        float rc;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc) : "f"(d));
        constexpr float kMagic = 12582912.0f;                                   // 1.5 * 2^23: t + kMagic rounds t to an integer, ties to even
        const uint64_t c127 = rq_pack2(127.0f, 127.0f), rc2 = rq_pack2(rc, rc), nd2 = rq_pack2(-d, -d), magic2 = rq_pack2(kMagic, kMagic);

        uint2* qrow = reinterpret_cast<uint2*>(q_out + size_t(r) * K);
        for (int c = threadIdx.x; c < nchunks; c += 256) {
            const uint4 w = row[c];
            const uint32_t mk = mask[c];
            float f[8];
            widen8<DT>(w, f);
            uint32_t b[8];                                                      // bit patterns whose low byte is the code
            if (quick) {
#pragma unroll
                for (int i = 0; i < 8; i += 2) {
                    const uint64_t n2 = rq_mul2(rq_pack2(f[i], f[i + 1]), c127);
                    const uint64_t q0 = rq_mul2(n2, rc2);
                    const uint64_t t2 = rq_fma2(rq_fma2(nd2, q0, n2), rc2, q0);
                    const uint64_t s2 = rq_add2(t2, magic2);
                    b[i] = uint32_t(s2);
                    b[i + 1] = uint32_t(s2 >> 32);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) b[i] = __float_as_uint(__fadd_rn(__fdiv_rn(__fmul_rn(f[i], 127.0f), d), kMagic));
            }
            uint32_t lo = rq_prmt(rq_prmt(b[0], b[1], 0x0040u), rq_prmt(b[2], b[3], 0x0040u), 0x5410u);
            uint32_t hi = rq_prmt(rq_prmt(b[4], b[5], 0x0040u), rq_prmt(b[6], b[7], 0x0040u), 0x5410u);
            if (mk != 0u) {                                                     // critical features hold no code
                lo &= rq_keep_bytes(mk, 0);
                hi &= rq_keep_bytes(mk, 1);
            }
            qrow[c] = make_uint2(lo, hi);
        }
        uint16_t* srow = static_cast<uint16_t*>(side_out) + size_t(r) * side_cols;
        const uint16_t* vrow = static_cast<const uint16_t*>(v) + size_t(r) * K;
        for (int j = threadIdx.x; j < side_cols; j += 256) srow[j] = (j < ko) ? vrow[idx[j]] : uint16_t(0);
        __syncthreads();                                         // red[] is reused by the next row
    }
}

// ------------------------------------------------------------------------------------------
// output of one element: the single fma of the definition and the narrowing
template <int YDT>
__device__ __forceinline__ void store_y(void* y, size_t i, float v) {
    if constexpr (YDT == kF32) static_cast<float*>(y)[i] = v;
    else if constexpr (YDT == kBF16) static_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
    else static_cast<__half*>(y)[i] = __float2half_rn(v);
}

// ------------------------------------------------------------------------------------------
// gemm_general: 64 x 64 outputs per CTA of 256 threads, 4 x 4 per thread (rows ty + 16 i,
// columns tx + 16 j), 64 features per step through shared memory, four int8 products per dp4a.
template <int XDT, int YDT>
__global__ void __launch_bounds__(256)
gemm_general(const int8_t* __restrict__ qx, const int8_t* __restrict__ qw, const float* __restrict__ sx, const float* __restrict__ sw,
             const void* __restrict__ sidex, const void* __restrict__ sidew, int side_cols, void* __restrict__ y, int M, int N, int K) {
    __shared__ uint32_t xs[64][17];
    __shared__ uint32_t ws[64][17];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    int acc[4][4];
    float part[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j] = 0; part[i][j] = 0.0f; }

    const int lr = threadIdx.x >> 2, lc = threadIdx.x & 3;       // this thread's 16-byte piece of the 64 x 64-byte tiles
    for (int k0 = 0; k0 < K; k0 += 64) {
        uint4 a = make_uint4(0, 0, 0, 0), b = make_uint4(0, 0, 0, 0);
        const int kk = k0 + lc * 16;
        if (kk < K) {
            if (m0 + lr < M) a = *reinterpret_cast<const uint4*>(qx + size_t(m0 + lr) * K + kk);
            if (n0 + lr < N) b = *reinterpret_cast<const uint4*>(qw + size_t(n0 + lr) * K + kk);
        }
        __syncthreads();
        xs[lr][lc * 4 + 0] = a.x; xs[lr][lc * 4 + 1] = a.y; xs[lr][lc * 4 + 2] = a.z; xs[lr][lc * 4 + 3] = a.w;
        ws[lr][lc * 4 + 0] = b.x; ws[lr][lc * 4 + 1] = b.y; ws[lr][lc * 4 + 2] = b.z; ws[lr][lc * 4 + 3] = b.w;
        __syncthreads();
#pragma unroll
        for (int kw = 0; kw < 16; ++kw) {
            int av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = int(xs[ty + 16 * i][kw]); bv[i] = int(ws[tx + 16 * i][kw]); }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(av[i], bv[j], acc[i][j]);
        }
    }
    // side columns: 16 per step, widened to fp32 in shared memory
    float* xf = reinterpret_cast<float*>(&xs[0][0]);
    float* wf = reinterpret_cast<float*>(&ws[0][0]);
    for (int k0 = 0; k0 < side_cols; k0 += 16) {
        __syncthreads();
        {
            const int row = threadIdx.x >> 2, c4 = (threadIdx.x & 3) * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int col = k0 + c4 + e;
                float xv = 0.0f, wv = 0.0f;
                if (m0 + row < M) xv = mmdk::widen16<XDT>(static_cast<const uint16_t*>(sidex)[size_t(m0 + row) * side_cols + col]);
                if (n0 + row < N) wv = mmdk::widen16<XDT>(static_cast<const uint16_t*>(sidew)[size_t(n0 + row) * side_cols + col]);
                xf[row * 17 + c4 + e] = xv;
                wf[row * 17 + c4 + e] = wv;
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = xf[(ty + 16 * i) * 17 + k]; bv[i] = wf[(tx + 16 * i) * 17 + k]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) part[i][j] = __fmaf_rn(av[i], bv[j], part[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 16 * i;
        if (m >= M) continue;
        const float sxm = sx[m];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx + 16 * j;
            if (n >= N) continue;
            const float s = __fmul_rn(sxm, sw[n]);
            store_y<YDT>(y, size_t(m) * N + n, __fmaf_rn(float(acc[i][j]), s, part[i][j]));
        }
    }
}

// ------------------------------------------------------------------------------------------
// gemm_tc: tensor-core kernel.
//
// One CTA computes a 128 x BN tile of Y.  192 threads: warp 0 issues the TMA loads, warp 1
// allocates tensor memory and issues the MMAs, warps 2-5 are the epilogue (warp w reads the
// 32 accumulator lanes of its quarter, w % 4).  A stage of the ring holds a 128-row tile of
// the activations and a BN-row tile of the weights, each row 128 bytes (128 int8 features,
// or 64 side columns of 16 bits), written by TMA with the 128-byte swizzle that the MMA's
// shared-memory descriptors name.  The int8 steps accumulate into columns [0, BN) of tensor
// memory as int32; the side steps into columns [BN, 2 BN) as fp32.
//
// Every wait is bounded: a wait that runs out records a code in *status, raises the CTA's
// abort flag and the kernel winds down (no further stores, tensor memory freed).
//
// Split K.  A call with one row of tiles over a narrow layer (a decode step) has fewer tiles
// than the GPU has SMs, and an SM streams weights from DRAM only as fast as the bytes it can
// keep in flight.  Such calls are launched in clusters of 2-4 CTAs along z: the CTAs of a
// cluster work on the same tile, each on its own share of the K steps (the side steps go to
// rank 0), and afterwards ranks 1.. write their int32 accumulators into rank 0's ring memory
// (distributed shared memory; the ring is free by then, which the first cluster barrier
// establishes), a second cluster barrier publishes them, and rank 0 adds them to its own and
// runs the epilogue.  Integer sums do not depend on the order, so the result is the same bits.

constexpr int kTcThreads = 192;
constexpr int kTcBM = 128;
constexpr int kTcRowBytes = 128;
constexpr long long kWaitLimitCycles = 4000000000ll;            // about two seconds

// BM = rows of the MMA: 128, or 64 for calls with at most 64 activation rows (a decode step), whose ring stages then
// spend 8 KB instead of 16 KB on activations and hold more steps of the weight stream in flight.
// KPB = K blocks of 128 features one ring step (one TMA load per operand) brings: 1, or 2 for decode-size calls, where
// the pace is set by the number of loads rather than by their bytes.
template <int BN, int BM = kTcBM, int KPB = 1> struct TcCfg {
    static constexpr uint32_t kASlabBytes = BM * kTcRowBytes;                   // one K block of the activation tile
    static constexpr uint32_t kBSlabBytes = BN * kTcRowBytes;
    static constexpr uint32_t kABytes = KPB * kASlabBytes;
    static constexpr uint32_t kBBytes = KPB * kBSlabBytes;
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = (196608u / kStageBytes) > 12u ? 12 : int(196608u / kStageBytes);
    static constexpr uint32_t kTmemCols = (2 * BN <= 32) ? 32 : 2 * BN;          // a power of two >= 32
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 2048 /* barriers, scales */;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int code,
                                          long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) {
                *abort_flag = 1;
                atomicCAS(status, 0, code);
                return false;
            }
        }
    }
}

// a [K blocks][rows][128 bytes] box from a map that views the matrix as (128 bytes, rows, K / 128)
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int row, int kblock, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(kblock), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// K-major operand tile with 128-byte rows and the 128-byte swizzle: 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t addr) {
    return uint64_t((addr & 0x3FFFFu) >> 4) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) | (uint64_t(2) << 61);
}
// instruction descriptor: D format (1 = fp32, 2 = int32), A / B format, both K-major, N / 8, M / 16
__host__ __device__ constexpr uint32_t umma_idesc(uint32_t dfmt, uint32_t abfmt, uint32_t M, uint32_t N) {
    return (dfmt << 4) | (abfmt << 7) | (abfmt << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the address, in the cluster's shared window, of this CTA's shared address `addr` in CTA `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}

template <int XDT, int YDT, int BN, int BM, int KPB>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc(const __grid_constant__ CUtensorMap map_qx, const __grid_constant__ CUtensorMap map_qw,
        const __grid_constant__ CUtensorMap map_sidex, const __grid_constant__ CUtensorMap map_sidew,
        const float* __restrict__ sx, const float* __restrict__ sw, void* __restrict__ y,
        int M, int N, int kblocks_all /* K blocks of 128 int8 features */, int sblocks_all /* side steps of 64 columns */,
        int n_tile_base /* first column tile of this launch */, int* status) {
    using Cfg = TcCfg<BN, BM, KPB>;
    constexpr uint32_t kTxMain = Cfg::kStageBytes;                              // bytes of an int8 step's two loads (boxes of BM and BN rows)
    constexpr uint32_t kTxSide = Cfg::kASlabBytes + Cfg::kBSlabBytes;           // bytes of a side step's two loads
    constexpr int S = Cfg::kStages;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;               // swizzled tiles need 1024-byte alignment
    unsigned char* ctrl = smem_raw + (tiles - smem_u32(smem_raw)) + S * Cfg::kStageBytes;
    const uint32_t full0 = smem_u32(ctrl);                                      // S barriers: tile landed
    const uint32_t empty0 = full0 + 8u * S;                                     // S barriers: tile consumed
    const uint32_t accbar = empty0 + 8u * S;                                    // accumulators complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 8 * (2 * S + 1));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 1) + 8);
    volatile int* peer_gave_up = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 1) + 12);   // split K: set in rank 0 by a rank that ran out of a wait
    static_assert(8 * (2 * S + 1) + 16 <= 256, "control words end before the column scales");
    float* sw_s = reinterpret_cast<float*>(ctrl + 256);                         // BN scales of this tile's columns

    // Kernels launched behind this one with programmatic stream serialization (the row kernel of the next call, or this
    // call's second launch for the tiles left over) may become resident as SMs free up; each waits for this grid to
    // complete before it touches global memory that this grid reads or writes.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM, n0 = (n_tile_base + int(blockIdx.y)) * BN;
    const uint32_t nsplit = cluster_size(), rank = cluster_rank();              // 1 and 0 without a cluster launch
    const int ksteps_all = (kblocks_all + KPB - 1) / KPB;                       // int8 ring steps of KPB K blocks each
    const int kb_lo = int((long(ksteps_all) * rank) / nsplit), kb_hi = int((long(ksteps_all) * (rank + 1)) / nsplit);
    const int kblocks = kb_hi - kb_lo;                                          // this CTA's share of the int8 steps
    const int sblocks = (rank == 0) ? sblocks_all : 0;
    const int steps = kblocks + sblocks;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
        mbar_init(accbar, 1);
        *abort_flag = 0;
        *peer_gave_up = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(Cfg::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;
    // the load of one int8 step of one operand: KPB K blocks of `rows` rows from K block `step * KPB` on
    auto load_main = [&](uint32_t dst, const CUtensorMap* map, int row0, int step, uint32_t bar) {
        if constexpr (KPB == 1) tma_load_2d(dst, map, step * 128, row0, bar);
        else tma_load_3d(dst, map, row0, step * KPB, bar);                      // a K block past the end reads as zeros
    };

    if (warp == 0) {
        if (lane == 0) {
            // The first ring-full of weight tiles does not depend on the row kernel that runs before this one: their loads
            // go out at once; the activation tiles of those stages follow when that kernel's results are visible.
            const int pre = steps < S ? steps : S;
            for (int i = 0; i < pre; ++i) {
                const uint32_t b_dst = tiles + uint32_t(i) * Cfg::kStageBytes + Cfg::kABytes;
                mbar_expect_tx(full0 + 8u * i, i < kblocks ? kTxMain : kTxSide);
                if (i < kblocks) load_main(b_dst, &map_qw, n0, kb_lo + i, full0 + 8u * i);
                else tma_load_2d(b_dst, &map_sidew, (i - kblocks) * 64, n0, full0 + 8u * i);
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int i = 0; i < pre; ++i) {
                const uint32_t a_dst = tiles + uint32_t(i) * Cfg::kStageBytes;
                if (i < kblocks) load_main(a_dst, &map_qx, m0, kb_lo + i, full0 + 8u * i);
                else tma_load_2d(a_dst, &map_sidex, (i - kblocks) * 64, m0, full0 + 8u * i);
            }
            for (int i = pre; i < steps; ++i) {
                const int s = i % S;
                const uint32_t round = uint32_t(i / S);
                if (!mbar_wait(empty0 + 8u * s, (round & 1u) ^ 1u, abort_flag, status, 1)) break;
                const uint32_t a_dst = tiles + uint32_t(s) * Cfg::kStageBytes, b_dst = a_dst + Cfg::kABytes;
                mbar_expect_tx(full0 + 8u * s, i < kblocks ? kTxMain : kTxSide);
                if (i < kblocks) {
                    load_main(a_dst, &map_qx, m0, kb_lo + i, full0 + 8u * s);
                    load_main(b_dst, &map_qw, n0, kb_lo + i, full0 + 8u * s);
                } else {
                    tma_load_2d(a_dst, &map_sidex, (i - kblocks) * 64, m0, full0 + 8u * s);
                    tma_load_2d(b_dst, &map_sidew, (i - kblocks) * 64, n0, full0 + 8u * s);
                }
            }
        }
        __syncwarp();
        if (nsplit > 1) { cluster_sync_all(); cluster_sync_all(); }              // the two barriers of the exchange (see the epilogue)
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_i8 = umma_idesc(2, 1, BM, BN);                      // int32 <- int8 x int8
            constexpr uint32_t idesc_16 = umma_idesc(1, XDT == kBF16 ? 1u : 0u, BM, BN);        // fp32 <- 16-bit x 16-bit
            bool ok = true;
            for (int i = 0; i < steps && ok; ++i) {
                const int s = i % S;
                const uint32_t round = uint32_t(i / S);
                ok = mbar_wait(full0 + 8u * s, round & 1u, abort_flag, status, 2);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_src = tiles + uint32_t(s) * Cfg::kStageBytes, b_src = a_src + Cfg::kABytes;
                const uint64_t adesc = umma_smem_desc(a_src), bdesc = umma_smem_desc(b_src);
                if (i < kblocks) {
#pragma unroll
                    for (int j = 0; j < KPB; ++j) {
                        const uint64_t aj = umma_smem_desc(a_src + uint32_t(j) * Cfg::kASlabBytes), bj = umma_smem_desc(b_src + uint32_t(j) * Cfg::kBSlabBytes);
#pragma unroll
                        for (int k = 0; k < 4; ++k)                   // 32 int8 features = 32 bytes per MMA
                            umma_i8(tmem, aj + uint64_t(2 * k), bj + uint64_t(2 * k), idesc_i8, (i > 0 || j > 0 || k > 0) ? 1u : 0u);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)                       // 16 side columns = 32 bytes per MMA
                        umma_f16(tmem + uint32_t(BN), adesc + uint64_t(2 * k), bdesc + uint64_t(2 * k), idesc_16, (i > kblocks || k > 0) ? 1u : 0u);
                }
                umma_commit(empty0 + 8u * s);                         // the stage is free once these MMAs have read it
            }
            if (ok) umma_commit(accbar);
        }
        __syncwarp();
        if (nsplit > 1) { cluster_sync_all(); cluster_sync_all(); }
    } else {
        // epilogue: 128 threads, one accumulator row each
        const int et = threadIdx.x - 64;
        for (int c = et; c < BN; c += 128) sw_s[c] = (n0 + c < N) ? sw[n0 + c] : 0.0f;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");       // the activations' row scales come from the kernel before this one
        const int quarter = warp & 3;
        // a 128-row accumulator has row r in lane r; a 64-row one keeps rows 16 q .. 16 q + 15 in the first 16 lanes of
        // quarter q (the other lanes of the quarter hold nothing of it)
        const bool row_lane = (BM == 128) || lane < 16;
        const int m = row_lane ? m0 + quarter * (BM / 4) + lane : M;
        const float sxm = (m < M) ? sx[m] : 0.0f;
        bool ok = true;
        if (lane == 0) ok = mbar_wait(accbar, 0, abort_flag, status, 3);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t lane_base = tmem + (uint32_t(quarter * 32) << 16);
        const uint32_t row_in_tile = uint32_t(quarter * (BM / 4) + lane);       // meaningful where row_lane holds
        constexpr uint32_t kPartBytes = uint32_t(BM) * BN * 4u;                  // one rank's accumulator, stored [column][row]
        if (nsplit > 1) {
            cluster_sync_all();                                                  // every CTA of the cluster is through its main loop: rank 0's ring is free
            if (rank > 0) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t ai[32];
                    tmem_ld32(lane_base + uint32_t(c0), ai);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (ok && row_lane) {
                        const uint32_t dst = map_to_cta(tiles + (rank - 1u) * kPartBytes + uint32_t(c0) * BM * 4u + row_in_tile * 4u, 0);
#pragma unroll
                        for (int j = 0; j < 32; ++j) st_cluster_u32(dst + uint32_t(j) * BM * 4u, ai[j]);
                    }
                }
                // a rank whose wait ran out has no sums to give: it says so, and rank 0 then stores nothing for this tile
                if (!ok && lane == 0) st_cluster_u32(map_to_cta(smem_u32(const_cast<int*>(peer_gave_up)), 0), 1u);
            }
            cluster_sync_all();                                                  // the partial sums are in rank 0's shared memory
            if (rank == 0 && *peer_gave_up) ok = false;
        }
        if (ok && rank == 0) {
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t ai[32], af[32];
                tmem_ld32(lane_base + uint32_t(c0), ai);
                if (sblocks > 0) tmem_ld32(lane_base + uint32_t(BN + c0), af);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (nsplit > 1 && row_lane) {
                    for (uint32_t r = 1; r < nsplit; ++r) {
                        const uint32_t src = tiles + (r - 1u) * kPartBytes + uint32_t(c0) * BM * 4u + row_in_tile * 4u;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            uint32_t v;
                            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(src + uint32_t(j) * BM * 4u) : "memory");
                            ai[j] += v;
                        }
                    }
                }
                float out[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float s = __fmul_rn(sxm, sw_s[c0 + j]);
                    const float p = (sblocks > 0) ? __uint_as_float(af[j]) : 0.0f;
                    out[j] = __fmaf_rn(float(int(ai[j])), s, p);
                }
                if (m < M) {
                    const int n = n0 + c0;
                    if constexpr (YDT == kF32) {
                        float* dst = static_cast<float*>(y) + size_t(m) * N + n;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (n + j < N) *reinterpret_cast<float4*>(dst + j) = make_float4(out[j], out[j + 1], out[j + 2], out[j + 3]);
                    } else {
                        uint16_t* dst = static_cast<uint16_t*>(y) + size_t(m) * N + n;
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            uint32_t pk[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                if constexpr (YDT == kBF16) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                                    pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                                } else {
                                    const __half2 h = __floats2half2_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                                    pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                                }
                            }
                            if (n + j < N) *reinterpret_cast<uint4*>(dst + j) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    }
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }

    __syncthreads();
    if (*abort_flag) {
        // copies that were issued but never waited for may still be landing in this CTA's
        // shared memory: give them time before the memory is handed to another CTA
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(Cfg::kTmemCols) : "memory");
    }
}


// ------------------------------------------------------------------------------------------
// gemm_sk: one row of tiles (a decode step, at most 64 activation rows) with the K steps of ALL
// tiles dealt out evenly over the CTAs of one launch ("stream K").
//
// gemm_tc gives every 128-column tile to one CTA, or to a cluster of 2-4 CTAs that share its K
// steps; with 64 tiles on 148 SMs either 84 SMs stream weights or 128 do.  Here the units of
// work (per tile: its int8 steps of two K blocks, then one unit for all of its side steps) are
// numbered across the tiles and CTA c takes units [c T / G, (c + 1) T / G): every SM streams the
// same number of bytes, whatever the number of tiles.  A CTA's range touches at most two tiles
// (the host launches at least as many CTAs as tiles); the part of a tile that a CTA computes is a
// "segment", accumulated in its own half of tensor memory, so the epilogue of the first segment
// runs under the loads and MMAs of the second.
//
// Tiles that several CTAs share are put together without anybody waiting: a CTA writes its
// segment's int32 sums (and, if it holds the tile's side unit, the fp32 side sums) to a slot of
// global scratch, fences, and takes a ticket from the tile's counter; the CTA whose ticket is
// the last one adds the other slots to its own sums, which are still in its tensor memory, and
// runs the epilogue.  Integer sums do not depend on the order and the side sums come from one
// CTA, so the result is the same bits as gemm_tc's.  The counters are zeroed by the row kernel
// that runs before every product.  Waits are bounded as in gemm_tc.
constexpr int kSkBN = 128, kSkBM = 64, kSkKPB = 2;

template <int XDT, int YDT>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_sk(const __grid_constant__ CUtensorMap map_qx, const __grid_constant__ CUtensorMap map_qw,
        const __grid_constant__ CUtensorMap map_sidex, const __grid_constant__ CUtensorMap map_sidew,
        const float* __restrict__ sx, const float* __restrict__ sw, void* __restrict__ y,
        int M, int N, int kblocks_all, int sblocks_all, int n_tiles, int maxparts,
        int* __restrict__ counters, int* __restrict__ part_acc, float* __restrict__ part_side, int* status) {
    using Cfg = TcCfg<kSkBN, kSkBM, kSkKPB>;
    constexpr int BN = kSkBN, BM = kSkBM, KPB = kSkKPB, S = Cfg::kStages;
    constexpr uint32_t kTxMain = Cfg::kStageBytes;
    constexpr uint32_t kTxSide = Cfg::kASlabBytes + Cfg::kBSlabBytes;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* ctrl = smem_raw + (tiles - smem_u32(smem_raw)) + S * Cfg::kStageBytes;
    const uint32_t full0 = smem_u32(ctrl);                                      // S barriers: tile landed
    const uint32_t empty0 = full0 + 8u * S;                                     // S barriers: tile consumed
    const uint32_t accbar0 = empty0 + 8u * S;                                   // 2 barriers: a segment's accumulators complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 8 * (2 * S + 2));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 2) + 8);
    volatile int* ticket = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 2) + 12);
    static_assert(8 * (2 * S + 2) + 16 <= 256, "control words end before the column scales");
    float* sw_s = reinterpret_cast<float*>(ctrl + 256);                         // 2 x BN scales: one set per segment

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ksteps = (kblocks_all + KPB - 1) / KPB;
    const int upt = ksteps + (sblocks_all > 0 ? 1 : 0);                         // units per tile
    const long long total = (long long)n_tiles * upt;
    const long long G = gridDim.x, c = blockIdx.x;
    const long long lo = total * c / G, hi = total * (c + 1) / G;               // this CTA's units
    const int t_first = int(lo / upt), t_last = int((hi - 1) / upt);
    const int nseg = (hi > lo) ? t_last - t_first + 1 : 0;                      // 0, 1 or 2

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
        mbar_init(accbar0, 1);
        mbar_init(accbar0 + 8u, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    // ring steps of a unit: an int8 unit is one step, the side unit is sblocks_all steps
    auto steps_of = [&](long long g) -> int { return (int(g % upt) < ksteps) ? 1 : sblocks_all; };

    if (warp == 0) {
        if (lane == 0) {
            // The loads of one ring step: `side` < 0 is int8 step `kstep` of tile `t`, otherwise side step `side`.
            auto issue_b = [&](int s, int t, int kstep, int side) {
                const uint32_t b_dst = tiles + uint32_t(s) * Cfg::kStageBytes + Cfg::kABytes;
                if (side < 0) tma_load_3d(b_dst, &map_qw, t * BN, kstep * KPB, full0 + 8u * s);
                else tma_load_2d(b_dst, &map_sidew, side * 64, t * BN, full0 + 8u * s);
            };
            auto issue_a = [&](int s, int kstep, int side) {
                const uint32_t a_dst = tiles + uint32_t(s) * Cfg::kStageBytes;
                if (side < 0) tma_load_3d(a_dst, &map_qx, 0, kstep * KPB, full0 + 8u * s);
                else tma_load_2d(a_dst, &map_sidex, side * 64, 0, full0 + 8u * s);
            };
            // The first ring-full of weight tiles does not depend on the row kernel before this one.
            int it = 0;
            bool waited = false, ok = true;
            int pre_t[S], pre_k[S], pre_side[S], npre = 0;
            for (long long g = lo; g < hi && ok; ++g) {
                const int t = int(g / upt), u = int(g % upt);
                const int nst = steps_of(g);
                for (int j = 0; j < nst && ok; ++j, ++it) {
                    const int s = it % S;
                    const int kstep = (u < ksteps) ? u : 0, side = (u < ksteps) ? -1 : j;
                    if (it < S) {                                                    // ring not yet wrapped: weights now, activations after the wait
                        mbar_expect_tx(full0 + 8u * s, side < 0 ? kTxMain : kTxSide);
                        issue_b(s, t, kstep, side);
                        pre_t[npre] = t; pre_k[npre] = kstep; pre_side[npre] = side; ++npre;
                        continue;
                    }
                    if (!waited) {
                        asm volatile("griddepcontrol.wait;" ::: "memory");
                        for (int q = 0; q < npre; ++q) issue_a(q, pre_k[q], pre_side[q]);
                        waited = true;
                    }
                    ok = mbar_wait(empty0 + 8u * s, ((uint32_t(it / S) & 1u) ^ 1u), abort_flag, status, 1);
                    if (!ok) break;
                    mbar_expect_tx(full0 + 8u * s, side < 0 ? kTxMain : kTxSide);
                    issue_a(s, kstep, side);
                    issue_b(s, t, kstep, side);
                }
            }
            if (!waited) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                for (int q = 0; q < npre; ++q) issue_a(q, pre_k[q], pre_side[q]);
            }
            (void)pre_t;
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_i8 = umma_idesc(2, 1, BM, BN);
            constexpr uint32_t idesc_16 = umma_idesc(1, XDT == kBF16 ? 1u : 0u, BM, BN);
            int it = 0;
            bool ok = true;
            for (int seg = 0; seg < nseg && ok; ++seg) {
                const int t = t_first + seg;
                const long long a = (lo > (long long)t * upt) ? lo : (long long)t * upt;
                const long long b = (hi < (long long)(t + 1) * upt) ? hi : (long long)(t + 1) * upt;
                const uint32_t tm = tmem + uint32_t(seg & 1) * 256u;
                bool first_i8 = true, first_side = true;
                for (long long g = a; g < b && ok; ++g) {
                    const int u = int(g % upt);
                    const int nst = steps_of(g);
                    for (int j = 0; j < nst && ok; ++j, ++it) {
                        const int s = it % S;
                        ok = mbar_wait(full0 + 8u * s, uint32_t(it / S) & 1u, abort_flag, status, 2);
                        if (!ok) break;
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t a_src = tiles + uint32_t(s) * Cfg::kStageBytes, b_src = a_src + Cfg::kABytes;
                        if (u < ksteps) {
#pragma unroll
                            for (int jj = 0; jj < KPB; ++jj) {
                                const uint64_t aj = umma_smem_desc(a_src + uint32_t(jj) * Cfg::kASlabBytes), bj = umma_smem_desc(b_src + uint32_t(jj) * Cfg::kBSlabBytes);
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    umma_i8(tm, aj + uint64_t(2 * k), bj + uint64_t(2 * k), idesc_i8, (first_i8 && jj == 0 && k == 0) ? 0u : 1u);
                            }
                            first_i8 = false;
                        } else {
                            const uint64_t adesc = umma_smem_desc(a_src), bdesc = umma_smem_desc(b_src);
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_f16(tm + uint32_t(BN), adesc + uint64_t(2 * k), bdesc + uint64_t(2 * k), idesc_16, (first_side && k == 0) ? 0u : 1u);
                            first_side = false;
                        }
                        umma_commit(empty0 + 8u * s);
                    }
                }
                if (ok) umma_commit(accbar0 + 8u * uint32_t(seg & 1));
            }
        }
        __syncwarp();
    } else {
        // epilogue: 128 threads; a 64-row accumulator keeps rows 16 q .. 16 q + 15 in the first 16 lanes of quarter q
        const int et = threadIdx.x - 64;
        const int quarter = warp & 3;
        const bool row_lane = lane < 16;
        const int m = row_lane ? quarter * 16 + lane : M;
        asm volatile("griddepcontrol.wait;" ::: "memory");       // row scales and the zeroed counters come from the kernel before this one
        const float sxm = (m < M) ? sx[m] : 0.0f;
        const uint32_t row_in_tile = uint32_t(quarter * 16 + lane);
        constexpr size_t kPart = size_t(BM) * BN;                                // values of one partial tile, stored [row][column]
        for (int seg = 0; seg < nseg; ++seg) {
            const int t = t_first + seg;
            const int n0 = t * BN;
            const long long ta = (long long)t * upt, tb = (long long)(t + 1) * upt;
            const long long a = lo > ta ? lo : ta, b = hi < tb ? hi : tb;
            const bool has_side = sblocks_all > 0 && b == tb;                    // the side unit is the tile's last
            const bool has_i8 = a < ta + ksteps;                                 // a segment of the side unit alone has no integer sums
            const int c_first = int(((ta + 1) * G + total - 1) / total) - 1, c_last = int((tb * G + total - 1) / total) - 1;
            const int parts = c_last - c_first + 1, mypart = int(c) - c_first;
            float* sws = sw_s + (seg & 1) * BN;
            for (int cc = et; cc < BN; cc += 128) sws[cc] = (n0 + cc < N) ? sw[n0 + cc] : 0.0f;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            bool ok = true;
            if (lane == 0) ok = mbar_wait(accbar0 + 8u * uint32_t(seg & 1), 0, abort_flag, status, 3);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t lane_base = tmem + uint32_t(seg & 1) * 256u + (uint32_t(quarter * 32) << 16);
            bool last = true;
            if (parts > 1) {
                // this segment's sums into its slot, then a ticket: the last one to arrive finishes the tile
                if (ok) {
#pragma unroll 1
                    for (int c0 = 0; c0 < BN; c0 += 32) {
                        uint32_t ai[32], af[32];
                        tmem_ld32(lane_base + uint32_t(c0), ai);
                        if (has_side) tmem_ld32(lane_base + uint32_t(BN + c0), af);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (!has_i8) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) ai[j] = 0u;
                        }
                        if (row_lane) {
                            int* dst = part_acc + (size_t(t) * maxparts + mypart) * kPart + size_t(row_in_tile) * BN + c0;
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *reinterpret_cast<uint4*>(dst + j) = make_uint4(ai[j], ai[j + 1], ai[j + 2], ai[j + 3]);
                            if (has_side) {
                                float* ds = part_side + size_t(t) * kPart + size_t(row_in_tile) * BN + c0;
#pragma unroll
                                for (int j = 0; j < 32; j += 4) *reinterpret_cast<uint4*>(ds + j) = make_uint4(af[j], af[j + 1], af[j + 2], af[j + 3]);
                            }
                        }
                    }
                    __threadfence();
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) *ticket = ok ? atomicAdd(counters + t, 1) : -1;      // a segment that gave up takes no ticket: the tile is then never finished
                asm volatile("bar.sync 1, 128;" ::: "memory");
                last = (*ticket == parts - 1);
                __threadfence();
            }
            if (ok && last) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t ai[32], af[32];
                    tmem_ld32(lane_base + uint32_t(c0), ai);
                    if (has_side) tmem_ld32(lane_base + uint32_t(BN + c0), af);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (!has_i8) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) ai[j] = 0u;
                    }
                    if (parts > 1 && row_lane) {
                        for (int pp = 0; pp < parts; ++pp) {
                            if (pp == mypart) continue;
                            const int* src = part_acc + (size_t(t) * maxparts + pp) * kPart + size_t(row_in_tile) * BN + c0;
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                const uint4 v = __ldcg(reinterpret_cast<const uint4*>(src + j));
                                ai[j] += v.x; ai[j + 1] += v.y; ai[j + 2] += v.z; ai[j + 3] += v.w;
                            }
                        }
                        if (sblocks_all > 0 && !has_side) {
                            const float* ss = part_side + size_t(t) * kPart + size_t(row_in_tile) * BN + c0;
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                const uint4 v = __ldcg(reinterpret_cast<const uint4*>(ss + j));
                                af[j] = v.x; af[j + 1] = v.y; af[j + 2] = v.z; af[j + 3] = v.w;
                            }
                        }
                    }
                    float out[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float sc = __fmul_rn(sxm, sws[c0 + j]);
                        const float pside = (sblocks_all > 0) ? __uint_as_float(af[j]) : 0.0f;
                        out[j] = __fmaf_rn(float(int(ai[j])), sc, pside);
                    }
                    if (m < M) {
                        const int n = n0 + c0;
                        if constexpr (YDT == kF32) {
                            float* dst = static_cast<float*>(y) + size_t(m) * N + n;
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                if (n + j < N) *reinterpret_cast<float4*>(dst + j) = make_float4(out[j], out[j + 1], out[j + 2], out[j + 3]);
                        } else {
                            uint16_t* dst = static_cast<uint16_t*>(y) + size_t(m) * N + n;
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                uint32_t pk[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    if constexpr (YDT == kBF16) {
                                        const __nv_bfloat162 h = __floats2bfloat162_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                                        pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                                    } else {
                                        const __half2 h = __floats2half2_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                                        pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                                    }
                                }
                                if (n + j < N) *reinterpret_cast<uint4*>(dst + j) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            }
                        }
                    }
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }

    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// ------------------------------------------------------------------------------------------
// gemm_tcp: persistent tensor-core kernel for large products with at most kTcpSide critical
// features.
//
// One CTA per SM walks over 128 x 256 tiles (M-tile index fastest, so CTAs that run together
// share weight tiles in L2).  Tensor memory holds TWO int32 accumulators (2 x 256 columns):
// while the epilogue warps drain the accumulator of tile i, the MMA thread is already
// accumulating tile i + 1 into the other one, and the TMA thread runs ahead through the
// 4-stage ring, so set-up, the first load round trip and the epilogue no longer stop the
// tensor pipe between tiles.  With both accumulators taken by integer sums the side columns
// cannot use the tensor cores here; they are few, so the epilogue adds them with fp32 FMAs
// in ascending feature order (the same order as gemm_general), hidden under the next tile's
// MMAs.  Waits are bounded as in gemm_tc.

constexpr int kTcpBN = 256;
constexpr int kTcpStages = 4;
constexpr int kTcpSide = 16;                                   // most critical features this kernel takes
constexpr uint32_t kTcpStageBytes = (kTcBM + kTcpBN) * kTcRowBytes;
constexpr uint32_t kTcpCtrlBytes = 512;
constexpr uint32_t kTcpSwBytes = 2 * kTcpBN * 4;               // column scales, one copy per accumulator
constexpr uint32_t kTcpWoBytes = kTcpBN * kTcpSide * 4;        // side columns of the tile's weight rows, fp32
constexpr uint32_t kTcpSmemBytes = kTcpStages * kTcpStageBytes + 1024 + kTcpCtrlBytes + kTcpSwBytes + kTcpWoBytes;

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int XDT, int YDT>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tcp(const __grid_constant__ CUtensorMap map_qx, const __grid_constant__ CUtensorMap map_qw,
         const float* __restrict__ sx, const float* __restrict__ sw, const void* __restrict__ sidex, const void* __restrict__ sidew,
         int side_cols /* row pitch of the side matrices */, int ko /* critical features, <= kTcpSide */,
         void* __restrict__ y, int M, int N, int kblocks, int mtiles, int ntiles, int* status) {
    constexpr int S = kTcpStages;
    constexpr int BN = kTcpBN;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t tiles_sm = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* ctrl = smem_raw + (tiles_sm - smem_u32(smem_raw)) + S * kTcpStageBytes;
    const uint32_t full0 = smem_u32(ctrl);                                      // S: tile landed
    const uint32_t empty0 = full0 + 8u * S;                                     // S: tile consumed
    const uint32_t accf0 = empty0 + 8u * S;                                     // 2: accumulator complete
    const uint32_t acce0 = accf0 + 16u;                                         // 2: accumulator drained
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 8 * (2 * S + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 4) + 8);
    volatile int* epi_ok = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 4) + 12);     // what the epilogue thread that waited found, for the other 127
    float* sw_s = reinterpret_cast<float*>(ctrl + kTcpCtrlBytes);               // [2][BN]
    float* wo_s = sw_s + 2 * BN;                                                // [BN][kTcpSide]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = mtiles * ntiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8u * b, 1); mbar_init(acce0 + 8u * b, 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const int m0 = (t % mtiles) * kTcBM, n0 = (t / mtiles) * BN;
                for (int i = 0; i < kblocks; ++i, ++it) {
                    const uint32_t s = it % S, round = it / S;
                    ok = mbar_wait(empty0 + 8u * s, (round & 1u) ^ 1u, abort_flag, status, 1);
                    if (!ok) break;
                    const uint32_t a_dst = tiles_sm + s * kTcpStageBytes, b_dst = a_dst + kTcBM * kTcRowBytes;
                    mbar_expect_tx(full0 + 8u * s, kTcpStageBytes);
                    tma_load_2d(a_dst, &map_qx, i * 128, m0, full0 + 8u * s);
                    tma_load_2d(b_dst, &map_qw, i * 128, n0, full0 + 8u * s);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_i8 = umma_idesc(2, 1, kTcBM, BN);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++lt) {
                const uint32_t buf = lt & 1u;
                ok = mbar_wait(acce0 + 8u * buf, ((lt >> 1) & 1u) ^ 1u, abort_flag, status, 4);    // the epilogue has drained this accumulator
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem + buf * uint32_t(BN);
                for (int i = 0; i < kblocks; ++i, ++it) {
                    const uint32_t s = it % S, round = it / S;
                    ok = mbar_wait(full0 + 8u * s, round & 1u, abort_flag, status, 2);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_src = tiles_sm + s * kTcpStageBytes, b_src = a_src + kTcBM * kTcRowBytes;
                    const uint64_t adesc = umma_smem_desc(a_src), bdesc = umma_smem_desc(b_src);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_i8(d_tmem, adesc + uint64_t(2 * k), bdesc + uint64_t(2 * k), idesc_i8, (i > 0 || k > 0) ? 1u : 0u);
                    umma_commit(empty0 + 8u * s);
                }
                if (ok) umma_commit(accf0 + 8u * buf);
            }
        }
        __syncwarp();
    } else {
        const int et = threadIdx.x - 64;
        const int quarter = warp & 3;
        const uint16_t* sxo = static_cast<const uint16_t*>(sidex);
        const uint16_t* swo = static_cast<const uint16_t*>(sidew);
        uint32_t lt = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++lt) {
            const uint32_t buf = lt & 1u;
            const int m0 = (t % mtiles) * kTcBM, n0 = (t / mtiles) * BN;
            const int m = m0 + quarter * 32 + lane;
            // this tile's column scales and side columns; they are read while the MMAs of the tile still run
            float* sws = sw_s + buf * BN;
            for (int c = et; c < BN; c += 128) sws[c] = (n0 + c < N) ? sw[n0 + c] : 0.0f;
            float xo[kTcpSide];
#pragma unroll
            for (int j = 0; j < kTcpSide; ++j) xo[j] = 0.0f;
            if (ko > 0) {
                // side rows are at least 64 columns wide (128 bytes), so the first 16 columns are two aligned 16-byte loads
                for (int c = et; c < BN; c += 128) {
                    const int n = n0 + c;
                    float f[kTcpSide];
                    if (n < N) {
                        const uint4* src = reinterpret_cast<const uint4*>(swo + size_t(n) * side_cols);
                        float lo[8], hi[8];
                        widen8<XDT>(src[0], lo);
                        widen8<XDT>(src[1], hi);
#pragma unroll
                        for (int j = 0; j < 8; ++j) { f[j] = lo[j]; f[8 + j] = hi[j]; }
                    } else {
#pragma unroll
                        for (int j = 0; j < kTcpSide; ++j) f[j] = 0.0f;
                    }
#pragma unroll
                    for (int j = 0; j < kTcpSide; j += 4)
                        *reinterpret_cast<float4*>(wo_s + c * kTcpSide + j) = make_float4(f[j], f[j + 1], f[j + 2], f[j + 3]);
                }
                if (m < M) {
                    const uint4* src = reinterpret_cast<const uint4*>(sxo + size_t(m) * side_cols);
                    float lo[8], hi[8];
                    widen8<XDT>(src[0], lo);
                    widen8<XDT>(src[1], hi);
#pragma unroll
                    for (int j = 0; j < 8; ++j) { xo[j] = lo[j]; xo[8 + j] = hi[j]; }
                }
            }
            const float sxm = (m < M) ? sx[m] : 0.0f;
            // one thread waits for the accumulator, with the bound; what it found reaches the other 127 through the
            // barrier that also publishes the scales above, so the four warps always take the same way
            if (et == 0) *epi_ok = mbar_wait(accf0 + 8u * buf, (lt >> 1) & 1u, abort_flag, status, 3) ? 1 : 0;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            ok = (*epi_ok != 0);
            if (ok) (void)mbar_try(accf0 + 8u * buf, (lt >> 1) & 1u);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (ok) {
                const uint32_t lane_base = tmem + (uint32_t(quarter * 32) << 16) + buf * uint32_t(BN);
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t ai[32];
                    tmem_ld32(lane_base + uint32_t(c0), ai);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    float out[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float p = 0.0f;
                        if (ko > 0) {
                            const float4* wrow = reinterpret_cast<const float4*>(wo_s + (c0 + j) * kTcpSide);
#pragma unroll
                            for (int q = 0; q < kTcpSide / 4; ++q) {
                                if (q * 4 < ko) {
                                    const float4 wv = wrow[q];
                                    p = __fmaf_rn(xo[4 * q + 0], wv.x, p);
                                    p = __fmaf_rn(xo[4 * q + 1], wv.y, p);
                                    p = __fmaf_rn(xo[4 * q + 2], wv.z, p);
                                    p = __fmaf_rn(xo[4 * q + 3], wv.w, p);
                                }
                            }
                        }
                        out[j] = __fmaf_rn(float(int(ai[j])), __fmul_rn(sxm, sws[c0 + j]), p);
                    }
                    if (m < M) {
                        const int n = n0 + c0;
                        if constexpr (YDT == kF32) {
                            float* dst = static_cast<float*>(y) + size_t(m) * N + n;
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                if (n + j < N) *reinterpret_cast<float4*>(dst + j) = make_float4(out[j], out[j + 1], out[j + 2], out[j + 3]);
                        } else {
                            uint16_t* dst = static_cast<uint16_t*>(y) + size_t(m) * N + n;
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                uint32_t pk[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    if constexpr (YDT == kBF16) {
                                        const __nv_bfloat162 h = __floats2bfloat162_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                                        pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                                    } else {
                                        const __half2 h = __floats2half2_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                                        pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                                    }
                                }
                                if (n + j < N) *reinterpret_cast<uint4*>(dst + j) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            }
                        }
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(acce0 + 8u * buf);         // this warp's quarter of the accumulator is free again
            }
            asm volatile("bar.sync 2, 128;" ::: "memory");             // wo_s is rewritten for the next tile
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }

    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * BN) : "memory");
    }
}


// ------------------------------------------------------------------------------------------
// gemm_tc2: persistent kernel on CTA pairs (clusters of two, tcgen05 cta_group::2).
//
// The two SMs of a TPC share a 256 x 256 tile: each CTA loads its own 128 activation rows and
// only HALF of the weight rows (32 KB per K step of 128 features instead of 48 KB), and one
// thread of the even CTA issues MMAs of shape 256 x 256 x 32 that read both halves from the
// two shared memories and write each CTA's 128 rows into that CTA's own tensor memory.
// Otherwise as gemm_tcp: a ring (6 stages here), two accumulators per CTA, epilogue under the
// next tile's MMAs, side features by ordered fp32 FMAs.
//
// Barriers: "tile landed" lives in the even CTA and counts the bytes of both CTAs' loads (the
// odd CTA's TMA loads name the even CTA's barrier); "stage free" and "accumulator complete"
// are signalled in both CTAs by one multicast tcgen05.commit; "accumulator drained" lives in
// the even CTA and takes one arrival per epilogue warp of both CTAs.  No load is multicast.

constexpr int kPairStages = 3;
constexpr int kPairStepBlocks = 2;                                            // K blocks of 128 features one TMA load brings
constexpr uint32_t kPairSlabBytes = 128 * kTcRowBytes;                        // 128 rows x 128 features
constexpr uint32_t kPairHalfBytes = kPairStepBlocks * kPairSlabBytes;         // a stage's activations, or its weights
constexpr uint32_t kPairStageBytes = 2 * kPairHalfBytes;
constexpr uint32_t kPairSmemBytes = kPairStages * kPairStageBytes + 1024 + kTcpCtrlBytes + kTcpSwBytes + kTcpWoBytes;

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// one load of a [K blocks][rows][128 bytes] box from a map that views the matrix as (128 bytes, rows, K / 128)
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int row, int kblock, uint32_t bar_cluster_addr) {
    asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(kblock), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives on the barrier at this shared address in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(uint16_t(3)) : "memory");
}

// Scales and side columns of one tile's 256 weight rows into shared memory, and this thread's
// own activation row's side values into registers (epilogue threads, et = 0..127).
template <int XDT>
__device__ __forceinline__ void stage_tile_side(int et, int n0, int N, int m, int M, int ko, int side_cols, const float* __restrict__ sw,
                                                const uint16_t* __restrict__ sxo, const uint16_t* __restrict__ swo, float* sws, float* wo_s,
                                                float (&xo)[kTcpSide]) {
    for (int c = et; c < kTcpBN; c += 128) sws[c] = (n0 + c < N) ? sw[n0 + c] : 0.0f;
#pragma unroll
    for (int j = 0; j < kTcpSide; ++j) xo[j] = 0.0f;
    if (ko > 0) {
        for (int c = et; c < kTcpBN; c += 128) {
            const int n = n0 + c;
            float f[kTcpSide];
            if (n < N) {
                const uint4* src = reinterpret_cast<const uint4*>(swo + size_t(n) * side_cols);
                float lo[8], hi[8];
                widen8<XDT>(src[0], lo);
                widen8<XDT>(src[1], hi);
#pragma unroll
                for (int j = 0; j < 8; ++j) { f[j] = lo[j]; f[8 + j] = hi[j]; }
            } else {
#pragma unroll
                for (int j = 0; j < kTcpSide; ++j) f[j] = 0.0f;
            }
#pragma unroll
            for (int j = 0; j < kTcpSide; j += 4)
                *reinterpret_cast<float4*>(wo_s + c * kTcpSide + j) = make_float4(f[j], f[j + 1], f[j + 2], f[j + 3]);
        }
        if (m < M) {
            const uint4* src = reinterpret_cast<const uint4*>(sxo + size_t(m) * side_cols);
            float lo[8], hi[8];
            widen8<XDT>(src[0], lo);
            widen8<XDT>(src[1], hi);
#pragma unroll
            for (int j = 0; j < 8; ++j) { xo[j] = lo[j]; xo[8 + j] = hi[j]; }
        }
    }
}

// One accumulator row of 256 int32 sums -> scaled, side part added, narrowed, stored.
template <int YDT>
__device__ __forceinline__ void drain_row(uint32_t lane_base, float sxm, const float* sws, const float* wo_s, const float (&xo)[kTcpSide], int ko,
                                          void* __restrict__ y, int m, int M, int n0, int N) {
#pragma unroll 1
    for (int c0 = 0; c0 < kTcpBN; c0 += 32) {
        uint32_t ai[32];
        tmem_ld32(lane_base + uint32_t(c0), ai);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        float out[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            float p = 0.0f;
            if (ko > 0) {
                const float4* wrow = reinterpret_cast<const float4*>(wo_s + (c0 + j) * kTcpSide);
#pragma unroll
                for (int q = 0; q < kTcpSide / 4; ++q) {
                    if (q * 4 < ko) {
                        const float4 wv = wrow[q];
                        p = __fmaf_rn(xo[4 * q + 0], wv.x, p);
                        p = __fmaf_rn(xo[4 * q + 1], wv.y, p);
                        p = __fmaf_rn(xo[4 * q + 2], wv.z, p);
                        p = __fmaf_rn(xo[4 * q + 3], wv.w, p);
                    }
                }
            }
            out[j] = __fmaf_rn(float(int(ai[j])), __fmul_rn(sxm, sws[c0 + j]), p);
        }
        if (m < M) {
            const int n = n0 + c0;
            if constexpr (YDT == kF32) {
                float* dst = static_cast<float*>(y) + size_t(m) * N + n;
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    if (n + j < N) *reinterpret_cast<float4*>(dst + j) = make_float4(out[j], out[j + 1], out[j + 2], out[j + 3]);
            } else {
                uint16_t* dst = static_cast<uint16_t*>(y) + size_t(m) * N + n;
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    uint32_t pk[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if constexpr (YDT == kBF16) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                            pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                        } else {
                            const __half2 h = __floats2half2_rn(out[j + 2 * e], out[j + 2 * e + 1]);
                            pk[e] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                    }
                    if (n + j < N) *reinterpret_cast<uint4*>(dst + j) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
        }
    }
}

template <int XDT, int YDT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTcThreads, 1)
gemm_tc2(const __grid_constant__ CUtensorMap map_qx, const __grid_constant__ CUtensorMap map_qw /* boxes of 128 weight rows */,
         const float* __restrict__ sx, const float* __restrict__ sw, const void* __restrict__ sidex, const void* __restrict__ sidew,
         int side_cols, int ko, void* __restrict__ y, int M, int N, int kblocks, int mpairs /* tiles of 256 rows */, int ntiles, int* status) {
    constexpr int S = kPairStages;
    constexpr int BN = kTcpBN;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t tiles_sm = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* ctrl = smem_raw + (tiles_sm - smem_u32(smem_raw)) + S * kPairStageBytes;
    const uint32_t full0 = smem_u32(ctrl);                                      // S: tile landed (used in the even CTA)
    const uint32_t empty0 = full0 + 8u * S;                                     // S: stage free
    const uint32_t accf0 = empty0 + 8u * S;                                     // 2: accumulator complete
    const uint32_t acce0 = accf0 + 16u;                                         // 2: accumulator drained (used in the even CTA)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 8 * (2 * S + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 4) + 8);
    volatile int* epi_ok = reinterpret_cast<volatile int*>(ctrl + 8 * (2 * S + 4) + 12);
    float* sw_s = reinterpret_cast<float*>(ctrl + kTcpCtrlBytes);               // [2][BN]
    float* wo_s = sw_s + 2 * BN;                                                // [BN][kTcpSide]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int total_tiles = mpairs * ntiles;
    const int ksteps = (kblocks + kPairStepBlocks - 1) / kPairStepBlocks;      // ring steps per tile

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8u * b, 1); mbar_init(acce0 + 8u * b, 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                                          // both CTAs' barriers exist before either signals the other
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += npairs) {
                const int m0 = (t % mpairs) * 256 + int(rank) * 128;             // this CTA's activation rows
                const int nb0 = (t / mpairs) * BN + int(rank) * 128;             // this CTA's half of the weight rows
                for (int i = 0; i < ksteps; ++i, ++it) {
                    const uint32_t s = it % S, round = it / S;
                    ok = mbar_wait(empty0 + 8u * s, (round & 1u) ^ 1u, abort_flag, status, 1);
                    if (!ok) break;
                    const uint32_t a_dst = tiles_sm + s * kPairStageBytes, b_dst = a_dst + kPairHalfBytes;
                    const uint32_t full_even = map_to_cta(full0 + 8u * s, 0);
                    if (rank == 0) mbar_expect_tx(full0 + 8u * s, 2 * kPairStageBytes);      // both CTAs' bytes
                    tma_load_3d_pair(a_dst, &map_qx, m0, i * kPairStepBlocks, full_even);     // a K block past the end reads as zeros
                    tma_load_3d_pair(b_dst, &map_qw, nb0, i * kPairStepBlocks, full_even);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc_i8 = umma_idesc(2, 1, 256, BN);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += npairs, ++lt) {
                const uint32_t buf = lt & 1u;
                ok = mbar_wait(acce0 + 8u * buf, ((lt >> 1) & 1u) ^ 1u, abort_flag, status, 4);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem + buf * uint32_t(BN);
                for (int i = 0; i < ksteps; ++i, ++it) {
                    const uint32_t s = it % S, round = it / S;
                    ok = mbar_wait(full0 + 8u * s, round & 1u, abort_flag, status, 2);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_src = tiles_sm + s * kPairStageBytes, b_src = a_src + kPairHalfBytes;
#pragma unroll
                    for (int j = 0; j < kPairStepBlocks; ++j) {
                        const uint64_t adesc = umma_smem_desc(a_src + uint32_t(j) * kPairSlabBytes), bdesc = umma_smem_desc(b_src + uint32_t(j) * kPairSlabBytes);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_i8_pair(d_tmem, adesc + uint64_t(2 * k), bdesc + uint64_t(2 * k), idesc_i8, (i > 0 || j > 0 || k > 0) ? 1u : 0u);
                    }
                    umma_commit_pair(empty0 + 8u * s);
                }
                if (ok) umma_commit_pair(accf0 + 8u * buf);
            }
        }
        __syncwarp();
    } else {
        const int et = threadIdx.x - 64;
        const int quarter = warp & 3;
        const uint16_t* sxo = static_cast<const uint16_t*>(sidex);
        const uint16_t* swo = static_cast<const uint16_t*>(sidew);
        uint32_t lt = 0;
        bool ok = true;
        for (int t = pair; t < total_tiles && ok; t += npairs, ++lt) {
            const uint32_t buf = lt & 1u;
            const int m0 = (t % mpairs) * 256 + int(rank) * 128, n0 = (t / mpairs) * BN;
            const int m = m0 + quarter * 32 + lane;
            float* sws = sw_s + buf * BN;
            float xo[kTcpSide];
            stage_tile_side<XDT>(et, n0, N, m, M, ko, side_cols, sw, sxo, swo, sws, wo_s, xo);
            const float sxm = (m < M) ? sx[m] : 0.0f;
            if (et == 0) *epi_ok = mbar_wait(accf0 + 8u * buf, (lt >> 1) & 1u, abort_flag, status, 3) ? 1 : 0;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            ok = (*epi_ok != 0);
            if (ok) (void)mbar_try(accf0 + 8u * buf, (lt >> 1) & 1u);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (ok) {
                drain_row<YDT>(tmem + (uint32_t(quarter * 32) << 16) + buf * uint32_t(BN), sxm, sws, wo_s, xo, ko, y, m, M, n0, N);
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(acce0 + 8u * buf, 0));
            }
            asm volatile("bar.sync 2, 128;" ::: "memory");
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }

    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    cluster_sync_all();                                                          // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * BN) : "memory");
    }
}


// ------------------------------------------------------------------------------------------
// wait_selftest: the give-up path of the tensor-core kernels on its own, with a short limit.
//
// One CTA with the roles of gemm_tc: warp 1 allocates tensor memory; thread 0 (the "MMA
// thread") waits, through the same bounded routine as the product kernels, for a barrier that
// nothing ever arms; the epilogue warps wait for an "accumulator complete" barrier that, as in
// a product kernel whose MMA thread gave up, is never committed.  The first wait to run out
// records `code` and raises the CTA's abort flag, the other waiters see the flag and leave,
// every thread meets at the barrier, the tensor memory is given back and the kernel returns.
// No copy is in flight and nothing is stored besides the status word and the `left` counter
// (how many threads left through the give-up path).
__global__ void __launch_bounds__(kTcThreads, 1)
wait_selftest(int* status, int code, long long limit_cycles, int* left) {
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t never = smem_u32(&bars[0]), accbar = smem_u32(&bars[1]);
    if (threadIdx.x == 0) {
        mbar_init(never, 1);
        mbar_init(accbar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(32) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_slot;
    bool ok = true;
    if (warp == 0) {
        if (lane == 0) ok = mbar_wait(never, 0, abort_flag, status, code, limit_cycles);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else if (warp >= 2) {
        // a limit of its own, far longer: these warps leave because of the abort flag, not their own clock
        if (lane == 0) ok = mbar_wait(accbar, 0, abort_flag, status, code + 1, limit_cycles * 64);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }
    if (!ok) atomicAdd(left, 1);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(32) : "memory");
    }
}

}  // namespace mmdk
