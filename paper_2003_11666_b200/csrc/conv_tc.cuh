// Tensor-core (tcgen05) implicit GEMM for the bfloat16 convolution path.
//
// The three GEMMs of a convolution stage run on the 5th-generation tensor
// cores: 128 x BN tiles of D accumulate in tensor memory (fp32), operands are
// bfloat16 and are gathered straight from the NHWC activation ring / gradient
// scratch / KRSC weight copies into 128-byte-swizzled shared-memory tiles by
// the block's threads (implicit im2col: no staging buffer in global memory).
//   fprop  D[c_out, pixel]      A = predicted weights (K-major)   B = im2col(x)      (K-major)
//   dgrad  D[c_in, in pixel]    A = weights, read transposed (MN-major)  B = scattered dz (K-major)
//   wgrad  D[c_out, (r,s,c_in)] A = dz (MN-major)                 B = im2col(x)      (MN-major)
// with K ordered (r, s, channel) so that 8 consecutive K (one 16-byte unit)
// are 8 consecutive channels of one pixel.  The gather uses 16-byte asynchronous
// copies (cp.async, zero-filled outside the image) into a three-stage ring: two
// K-chunks of 64 are in flight while the tensor core works on a third.
// Every mbarrier wait is bounded; on expiry the block records an error, skips
// its stores, frees its tensor memory and returns.
#pragma once
#include <cuda_bf16.h>

#include "conv_types.h"

namespace pb {

constexpr int kTcChunk = 64;                  // K elements per shared-memory stage
constexpr int kTcThreads = 256;                // 8 warps gather; warps 0-3 / 4-7 split the columns in the epilogue
constexpr int kTcRowsPerPass = kTcThreads / 8; // K-major tiles: rows filled per pass (8 units of 16 bytes per row)
constexpr int kTcPasses = 128 / kTcRowsPerPass;
constexpr int kTcKPerPass = kTcThreads / 16;   // MN-major tiles of width 128: k rows filled per pass
constexpr int kTcKPasses = kTcChunk / kTcKPerPass;
constexpr int kTcBM = 128;
constexpr int kTcStageBytes = 16384 * 2;      // A tile + B tile
constexpr int kTcStages = 3;                  // shared-memory stages of the operand pipeline
constexpr int kTcSmemBytes = kTcStages * kTcStageBytes + 1024;
constexpr int kTcWaitLimit = 1 << 22;
constexpr int kTcMaxK = 3072;                 // longest K loop of one tile before K is sliced

struct ConvGemmTC {
    int mode, M, N, K;
    int ci, co, k, stride, pad, ih, iw, oh, ow;
    int s, bn;                    // stage index; N-tile width (64 or 128)
    int nsplit, k_per_split;      // k_per_split is a multiple of kTcChunk
    const __nv_bfloat16* a;       // fprop: predicted weights; dgrad: weights; wgrad: dz (NHWC)
    const __nv_bfloat16* b;       // fprop/wgrad: NHWC activation ring; dgrad: dz (NHWC)
    int b_slots, b_elems;
    float* c;                     // [c_slots][nsplit][M*N]
    int c_slots;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptor: start address, leading/stride byte offsets
// (all >> 4), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor of kind::f16: fp32 accumulator, bf16 x bf16, operand
// majorness, N >> 3 and M >> 4.
__device__ __forceinline__ uint32_t tc_idesc(int M, int N, int a_mn, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ uint32_t kmajor_off(int row, int unit) {
    return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((unit ^ (row & 7)) << 4));
}
__device__ __forceinline__ uint32_t mnmajor_off(int k, int mu) {
    return (uint32_t)((mu >> 3) * 8192 + (k >> 3) * 1024 + (k & 7) * 128 + (((mu & 7) ^ (k & 7)) << 4));
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    uint32_t done = 0;
    for (int it = 0; it < kTcWaitLimit && !done; ++it) {
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    }
    return done != 0;
}

// 16-byte asynchronous global -> shared copy; with ok == false the destination is zero-filled
__device__ __forceinline__ void cp_async16(unsigned char* dst, const __nv_bfloat16* src, bool ok) {
    const int sz = ok ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(sz) : "memory");
}

__global__ void __launch_bounds__(kTcThreads)
conv_tc_kernel(const ConvGemmTC* __restrict__ gemms, const GemmTile* __restrict__ tiles, TickState* ts, int S, int par) {
    extern __shared__ unsigned char tc_smem_raw[];
    __shared__ uint64_t mbar[kTcStages];
    __shared__ uint32_t tmem_base_sh;
    __shared__ ConvGemmTC G;                               // descriptor copy (no re-reads through global memory)
    const GemmTile tl = tiles[blockIdx.x];
    {
        const int* s_ = reinterpret_cast<const int*>(&gemms[tl.gemm]);
        int* d_ = reinterpret_cast<int*>(&G);
        for (int k = threadIdx.x; k < (int)(sizeof(ConvGemmTC) / 4); k += kTcThreads) d_[k] = s_[k];
    }
    __syncthreads();
    const long long t = ts->cnt[par];
    const long long smp = (G.mode == kFprop) ? t - G.s : t - 2LL * (S - 1) + G.s;
    if (!sample_live(ts, smp)) return;                                   // uniform: before any allocation
    unsigned char* smem = (unsigned char*)(((uintptr_t)tc_smem_raw + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int M = G.M, N = G.N, BN = G.bn;
    const int kb = tl.split * G.k_per_split, ke = min(G.K, kb + G.k_per_split);
    const int nchunks = (ke - kb + kTcChunk - 1) / kTcChunk;
    const __nv_bfloat16* __restrict__ A = G.a;
    const __nv_bfloat16* __restrict__ B = G.b + (size_t)(smp % G.b_slots) * G.b_elems;
    float* __restrict__ Cp = G.c + ((size_t)(smp % G.c_slots) * G.nsplit + tl.split) * ((size_t)M * N);
    const int CI = G.ci, CO = G.co, ksz = G.k, st = G.stride, pad = G.pad, ih = G.ih, iw = G.iw, oh = G.oh, ow = G.ow;
    // the gathers divide by these for every 16-byte unit: reciprocals once per block
    const float inv_ci = 1.f / (float)CI, inv_co = 1.f / (float)CO, inv_ksz = 1.f / (float)ksz,
                inv_st = 1.f / (float)st, inv_ow = 1.f / (float)ow;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)), "r"(128) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int q = 0; q < kTcStages; ++q)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&mbar[q])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base_sh;
    const int a_mn = G.mode != kFprop, b_mn = G.mode == kWgrad;
    const uint32_t idesc = tc_idesc(kTcBM, BN, a_mn, b_mn);

    // ---- per-thread invariants of the gathers
    // K-major tiles: this thread fills unit (tid & 7) of rows (tid >> 3) + kTcRowsPerPass i
    // MN-major tiles of width 128: unit (tid & 15) of k-rows (tid >> 4) + kTcKPerPass i
    const int ku = tid & 7, krow0 = tid >> 3;
    int bp[kTcPasses], bq[kTcPasses];   // K-major B rows: pixel coordinates (fprop: output pixel; dgrad: input pixel)
    bool bok[kTcPasses];
    if (G.mode != kWgrad) {
        const int wdt = (G.mode == kFprop) ? ow : iw;
        const float inv_wdt = 1.f / (float)wdt;
#pragma unroll
        for (int i = 0; i < kTcPasses; ++i) {
            const int n = tl.n0 + krow0 + kTcRowsPerPass * i;
            bok[i] = (krow0 + kTcRowsPerPass * i) < BN && n < N;
            bp[i] = quot(n, inv_wdt); bq[i] = n - bp[i] * wdt;
        }
    }
    // wgrad B: this thread's 8 consecutive n = (r, s, ci..ci+7)
    const int b_units_per_k = BN >> 3;                      // 16 or 8
    const int bshift = BN == 128 ? 4 : 3;                   // log2 of b_units_per_k
    const int bmu = tid & (b_units_per_k - 1), bk0 = tid >> bshift, bkstep = kTcThreads >> bshift;
    int wr = 0, wsx = 0, wci = 0;
    bool wok = false;
    if (G.mode == kWgrad) {
        const int n = tl.n0 + bmu * 8;
        wok = n < N;
        const int rs = quot(n, inv_ci); wci = n - rs * CI; wr = quot(rs, inv_ksz); wsx = rs - wr * ksz;
    }
    const int amu = tid & 15, ak0 = tid >> 4;               // MN-major A (width 128)
    const bool a_m_ok = (tl.m0 + amu * 8) < M;

    // gather of K-chunk c into its stage (every unit is written: data or zeros)
    auto gather = [&](int c) {
        unsigned char* sA = smem + (c % kTcStages) * kTcStageBytes;
        unsigned char* sB = sA + 16384;
        const int k0 = kb + c * kTcChunk;
        // ---------------- A tile
        if (G.mode == kFprop) {
            const int k = k0 + ku * 8;
#pragma unroll
            for (int i = 0; i < kTcPasses; ++i) {
                const int row = krow0 + kTcRowsPerPass * i, m = tl.m0 + row;
                const bool ok = m < M && k < ke;
                cp_async16(sA + kmajor_off(row, ku), ok ? A + (size_t)m * G.K + k : A, ok);
            }
        } else if (G.mode == kDgrad) {
#pragma unroll
            for (int i = 0; i < kTcKPasses; ++i) {
                const int kl = ak0 + kTcKPerPass * i, k = k0 + kl;          // k = rs * CO + co
                const bool ok = a_m_ok && k < ke;
                const int rs = quot(k, inv_co), co = k - rs * CO;
                cp_async16(sA + mnmajor_off(kl, amu), ok ? A + ((size_t)co * (ksz * ksz) + rs) * CI + tl.m0 + amu * 8 : A, ok);
            }
        } else {
#pragma unroll
            for (int i = 0; i < kTcKPasses; ++i) {
                const int kl = ak0 + kTcKPerPass * i, k = k0 + kl;          // k = output pixel
                const bool ok = a_m_ok && k < ke;
                cp_async16(sA + mnmajor_off(kl, amu), ok ? A + (size_t)k * CO + tl.m0 + amu * 8 : A, ok);
            }
        }
        // ---------------- B tile
        if (G.mode == kFprop) {
            const int k = k0 + ku * 8;
            const int rs = quot(k, inv_ci), ci = k - rs * CI, r = quot(rs, inv_ksz), s = rs - r * ksz;
#pragma unroll
            for (int i = 0; i < kTcPasses; ++i) {
                const int row = krow0 + kTcRowsPerPass * i;
                if (row >= BN) break;
                const int y = bp[i] * st + r - pad, x = bq[i] * st + s - pad;
                const bool ok = bok[i] && k < ke && y >= 0 && y < ih && x >= 0 && x < iw;
                cp_async16(sB + kmajor_off(row, ku), ok ? B + ((size_t)y * iw + x) * CI + ci : B, ok);
            }
        } else if (G.mode == kDgrad) {
            const int k = k0 + ku * 8;
            const int rs = quot(k, inv_co), co = k - rs * CO, r = quot(rs, inv_ksz), s = rs - r * ksz;
#pragma unroll
            for (int i = 0; i < kTcPasses; ++i) {
                const int row = krow0 + kTcRowsPerPass * i;
                if (row >= BN) break;
                const int ty = bp[i] + pad - r, tx = bq[i] + pad - s;
                const int p = quot(ty, inv_st), q = quot(tx, inv_st);
                const bool ok = bok[i] && k < ke && ty >= 0 && tx >= 0 && p * st == ty && q * st == tx && p < oh && q < ow;
                cp_async16(sB + kmajor_off(row, ku), ok ? B + ((size_t)p * ow + q) * CO + co : B, ok);
            }
        } else {
            for (int kl = bk0; kl < kTcChunk; kl += bkstep) {
                const int k = k0 + kl;
                const int p = quot(k, inv_ow), q = k - p * ow;
                const int y = p * st + wr - pad, x = q * st + wsx - pad;
                const bool ok = wok && k < ke && y >= 0 && y < ih && x >= 0 && x < iw;
                cp_async16(sB + mnmajor_off(kl, bmu), ok ? B + ((size_t)y * iw + x) * CI + wci : B, ok);
            }
        }
    };

    bool failed = false;
    for (int c = 0; c < kTcStages - 1; ++c) {
        if (c < nchunks) gather(c);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int c = 0; c < nchunks; ++c) {
        const int stg = c % kTcStages;
        unsigned char* sA = smem + stg * kTcStageBytes;
        unsigned char* sB = sA + 16384;
        // this thread's copies of chunk c have landed; make them visible to the tensor core
        asm volatile("cp.async.wait_group %0;" ::"n"(kTcStages - 2) : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (__syncthreads_or(failed)) { failed = true; break; }
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int j = 0; j < kTcChunk / 16; ++j) {
                const uint64_t da = a_mn ? tc_desc(smem_u32(sA) + j * 2048, 8192, 1024) : tc_desc(smem_u32(sA) + j * 32, 16, 1024);
                const uint64_t db = b_mn ? tc_desc(smem_u32(sB) + j * 2048, 8192, 1024) : tc_desc(smem_u32(sB) + j * 32, 16, 1024);
                const uint32_t acc = (c > 0 || j > 0) ? 1u : 0u;
                asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                             ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&mbar[stg])) : "memory");
        }
        // refill the stage that chunk c-1 used, once its MMAs have read it
        const int nxt = c + kTcStages - 1;
        if (nxt < nchunks) {
            if (c >= 1 && !mbar_wait(smem_u32(&mbar[(c - 1) % kTcStages]), (uint32_t)(((c - 1) / kTcStages) & 1))) failed = true;
            gather(nxt);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    // the last commit covers every MMA issued before it
    if (!failed && nchunks > 0) {
        const int last = nchunks - 1;
        if (!mbar_wait(smem_u32(&mbar[last % kTcStages]), (uint32_t)((last / kTcStages) & 1))) failed = true;
    }
    failed = __syncthreads_or(failed);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (!failed) {
        // epilogue: warp w reads lanes 32w..32w+31 (rows of D), 32 columns per load
        // (a warp may only touch the TMEM lanes of its quarter, warp % 4; the two warps of a
        //  quarter take one half of the columns each)
        const int quarter = warp & 3, half = warp >> 2;
        const int m = tl.m0 + quarter * 32 + lane;
        for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
            if (tl.n0 + c0 >= N) break;                         // uniform
            uint32_t r[32];
            const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                         "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                         : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
                           "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
                           "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
                           "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                         : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (m < M) {
                float* dst = Cp + (size_t)m * N + tl.n0 + c0;
                const int nleft = N - (tl.n0 + c0);
                if (nleft >= 32 && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        reinterpret_cast<float4*>(dst)[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                                                        __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
                } else {
#pragma unroll
                    for (int q = 0; q < 32; ++q)
                        if (q < nleft) dst[q] = __uint_as_float(r[q]);
                }
            }
        }
    } else if (tid == 0) {
        ts->error = kErrWait;
        ts->error_info = tl.gemm;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128) : "memory");
}

}  // namespace pb
