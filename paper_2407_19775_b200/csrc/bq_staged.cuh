// bq_staged.cuh -- fwd_staged: quantize / fused roundtrip for blocks of 2048 and 4096 elements
// with the input staged through shared memory by bulk asynchronous copies.
//
// A CTA is a few teams of 256 threads.  A team owns a ring of stages in shared memory, one
// quantization block per stage; one elected thread keeps the ring full with
// cp.async.bulk.shared::cta.global copies (this GPU's memory only, no multicast) that complete
// on an mbarrier per stage.  Per block: the elected thread waits for the stage (a bounded
// wait), the team meets at a named barrier, every thread takes its 16-byte chunks out of the
// stage into registers and reduces the block's absmax (warp redux, 8 partials in shared
// memory, a second named barrier); after that barrier nobody reads the stage any more, so the
// elected thread refills it at once with the block `stages` rounds ahead, and the team
// normalises, searches and stores from registers exactly as fwd_fast does (same helpers, same
// bits).  Compared with fwd_fast the copies are in flight independently of what the warps are
// doing and a thread holds one or two chunks instead of eight, so more warps fit; against that,
// the per-lane search tables leave about 32 KB of shared memory for the rings, fewer bytes in
// flight per SM than fwd_fast keeps in registers.
//
// A wait that runs out (about 2 s) records a code in the status word, the team stops taking
// blocks, every stage's outstanding copy is waited for (again bounded) and the kernel returns;
// the blocks the team did not reach keep whatever the output buffers held.
#pragma once

#include "bq_kernels.cuh"

namespace bqk {

constexpr int kTeamThreads = 256;
constexpr uint32_t kStagedCtrlBytes = 512;          // mbarriers, partial maxima, flags
// the rings start after the tables and the control words
constexpr uint32_t kStagedRingOff = kRedOff + 128u + kStagedCtrlBytes;

template <int XDT, int B, int TEAMS, int STAGES>
struct StagedCfg {
    static constexpr uint32_t kBlockBytes = uint32_t(B) * Elem<XDT>::kBytes;
    static constexpr uint32_t kRingBytes = uint32_t(TEAMS) * STAGES * kBlockBytes;
    static constexpr uint32_t kSmemBytes = kStagedRingOff + kRingBytes + 128u;
    static_assert(kSmemBytes <= 227u * 1024u, "tables and rings fit one CTA's shared memory");
    static_assert(TEAMS * (STAGES * 8 + 48) <= int(kStagedCtrlBytes), "control words fit");
};

__device__ __forceinline__ void mbar_init_cta(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cta(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cta(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// Waits for a phase of the barrier for at most about two seconds.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait_cta(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait_cta(bar, parity)) {
        if (clock64() - t0 > 4000000000LL) return false;
    }
    return true;
}
// One contiguous piece of this GPU's global memory into this CTA's shared memory; both addresses
// 16-byte aligned, the size a multiple of 16.  Completion is counted in bytes on `bar`.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds_16(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

template <int XDT, int B, int TEAMS, int STAGES, bool WRITE_Y, bool WRITE_Q>
__global__ void __launch_bounds__(TEAMS* kTeamThreads, 1)
fwd_staged(const void* __restrict__ x, void* __restrict__ y, uint8_t* __restrict__ codes, float* __restrict__ absmax_out,
           size_t nblocks, DeviceTables tab, int* __restrict__ status) {
    using Cfg = StagedCfg<XDT, B, TEAMS, STAGES>;
    constexpr int EPC = Elem<XDT>::kPerChunk;
    constexpr int EB = Elem<XDT>::kBytes;
    constexpr int CHUNKS = B / EPC;                          // 16-byte chunks of one block
    constexpr int R = CHUNKS / kTeamThreads;                 // chunks per thread
    static_assert(CHUNKS % kTeamThreads == 0 && R >= 1 && R <= 4, "a block is a whole number of chunks per thread");
    constexpr int NT = TEAMS * kTeamThreads;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t sm_base = (uint32_t(__cvta_generic_to_shared(smem_raw)) + 127u) & ~127u;
    const int lane = threadIdx.x & 31;
    const int team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads, tw = tt >> 5;
    const uint32_t sm_lane = sm_base + uint32_t(lane) * 4u;
    const TabRef<false> tref(tab, sm_lane);
    const uint32_t ctrl = sm_base + kRedOff + 128u + uint32_t(team) * (STAGES * 8u + 48u);
    const uint32_t full0 = ctrl;                                            // STAGES mbarriers
    const uint32_t part0 = ctrl + STAGES * 8u;                              // 8 partial maxima
    const uint32_t flag = part0 + 32u;                                      // what the elected thread's wait came to
    const uint32_t ring = sm_base + kStagedRingOff + uint32_t(team) * STAGES * Cfg::kBlockBytes;

    fill_fwd_tables<NT>(tab, sm_base);
    if (tt == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init_cta(full0 + 8u * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const float neg_limit = tab.neg_limit;
    const char* xb = static_cast<const char*>(x);
    char* yb = static_cast<char*>(y);
    const size_t first = size_t(blockIdx.x) * TEAMS + size_t(team);
    const size_t stride = size_t(gridDim.x) * TEAMS;
    const int bar_id = 1 + team;

    // the ring starts full
    if (tt == 0) {
        for (int s = 0; s < STAGES; ++s) {
            const size_t b = first + size_t(s) * stride;
            if (b < nblocks) {
                mbar_expect_tx_cta(full0 + 8u * s, Cfg::kBlockBytes);
                bulk_load(ring + uint32_t(s) * Cfg::kBlockBytes, xb + b * size_t(B) * EB, Cfg::kBlockBytes, full0 + 8u * s);
            }
        }
    }

    size_t it = 0;
    bool ok = true;
    for (size_t b = first; b < nblocks; b += stride, ++it) {
        const int s = int(it % STAGES);
        const uint32_t parity = uint32_t(it / STAGES) & 1u;
        if (tt == 0) {
            const bool landed = mbar_wait_bounded(full0 + 8u * s, parity);
            if (!landed) atomicExch(status, 1);
            sts_u32(flag, landed ? 1u : 0u);
        }
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(kTeamThreads) : "memory");
        {
            uint32_t v;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(flag) : "memory");
            ok = v != 0;
        }
        if (!ok) break;

        // the block out of the stage: chunk c of the block belongs to thread c mod 256
        uint4 w[R];
        float f[R][EPC];
        uint32_t neg[R][2];
        float a = 0.0f;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            w[r] = lds_16(ring + uint32_t(s) * Cfg::kBlockBytes + uint32_t(r * kTeamThreads + tt) * 16u);
            if constexpr (WRITE_Q) {
                if constexpr (EPC == 8) {
                    neg[r][0] = sign_mask_16(w[r].x, w[r].y);
                    neg[r][1] = sign_mask_16(w[r].z, w[r].w);
                } else {
                    neg[r][0] = sign_mask_32(w[r].x, w[r].y, w[r].z, w[r].w);
                }
            }
            widen_chunk<XDT>(w[r], f[r]);
#pragma unroll
            for (int i = 0; i < EPC; i += 2) a = max3_abs(a, f[r][i], f[r][i + 1]);
        }
        a = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(a)));
        const uint32_t slot = part0;                                        // one set of slots: the first barrier of the next block separates reuse
        if (lane == 0) sts_u32(slot + uint32_t(tw) * 4u, __float_as_uint(a));
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(kTeamThreads) : "memory");
        // every thread holds its chunks in registers: the stage is free for the block STAGES rounds ahead
        if (tt == 0) {
            const size_t nb = b + size_t(STAGES) * stride;
            if (nb < nblocks) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the generic-proxy reads of the stage come before the async-proxy write
                mbar_expect_tx_cta(full0 + 8u * s, Cfg::kBlockBytes);
                bulk_load(ring + uint32_t(s) * Cfg::kBlockBytes, xb + nb * size_t(B) * EB, Cfg::kBlockBytes, full0 + 8u * s);
            }
        }
#pragma unroll
        for (int k = 0; k < kTeamThreads / 32; ++k) {
            uint32_t v;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(slot + uint32_t(k) * 4u) : "memory");
            a = fmaxf(a, __uint_as_float(v));
        }

        const float d = (a != 0.0f) ? a : 1.0f;
        constexpr bool QUICK_OK = (XDT != kF32);
        const bool quick = QUICK_OK && (d >= 5.421010862427522e-20f) && (d <= 1.8446744073709552e19f);     // 2^-64 .. 2^64; the same for the whole team
        if (quick) {
            const float rc = rcp_approx(d);
            const uint64_t r2 = pack2(rc, rc), nd2 = pack2(-d, -d);
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < EPC; i += 2) {
                    const uint64_t x2 = pack2(f[r][i], f[r][i + 1]);
                    const uint64_t q0 = mul2(x2, r2);
                    const uint64_t e = fma2(nd2, q0, x2);
                    unpack2(fma2(e, r2, q0), f[r][i], f[r][i + 1]);
                }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < EPC; ++i) f[r][i] = __fdiv_rn(f[r][i], d);
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float out[EPC];
            Found fd[EPC];
#pragma unroll
            for (int i = 0; i < EPC; i += 2) {
                fd[i] = search_folded(f[r][i], neg_limit, tref);
                fd[i + 1] = search_folded(f[r][i + 1], neg_limit, tref);
                if constexpr (WRITE_Y) values_of(fd[i], fd[i + 1], a, tref, out[i], out[i + 1]);
            }
            const size_t off = b * size_t(B) + size_t(r * kTeamThreads + tt) * EPC;
            if constexpr (WRITE_Y) stg_stream_16(yb + off * EB, narrow_chunk<XDT>(out));
            if constexpr (WRITE_Q) {
                if constexpr (EPC == 8) {
                    stg_stream_8(codes + off, make_uint2(pack_codes(fd[0], fd[1], fd[2], fd[3], neg[r][0]), pack_codes(fd[4], fd[5], fd[6], fd[7], neg[r][1])));
                } else {
                    stg_stream_4(codes + off, pack_codes(fd[0], fd[1], fd[2], fd[3], neg[r][0]));
                }
            }
        }
        if constexpr (WRITE_Q) {
            if (tt == 0) absmax_out[b] = a;
        }
    }

    if (!ok && tt == 0) {
        // copies that were issued and not consumed may still be landing: wait for each stage's current phase (bounded) so that
        // the shared memory is quiet before the CTA ends.  Stage s was last armed for iteration j with j mod STAGES == s.
        for (int s = 0; s < STAGES; ++s) {
            for (size_t j = it; j < it + STAGES; ++j) {
                if (int(j % STAGES) == s && first + j * stride < nblocks) mbar_wait_bounded(full0 + 8u * s, uint32_t(j / STAGES) & 1u);
            }
        }
    }
    __syncthreads();
}

}  // namespace bqk
