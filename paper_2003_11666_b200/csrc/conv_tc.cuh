// Tensor-core (tcgen05) implicit GEMM for the bfloat16 convolution path.
//
// The three GEMMs of a convolution stage run on the 5th-generation tensor
// cores: 128 x BN tiles of D accumulate in tensor memory (fp32), operands are
// bfloat16 in 128-byte-swizzled shared-memory tiles.
//   fprop  D[c_out, pixel]      A = predicted weights (K-major)   B = im2col(x)      (K-major)
//   dgrad  D[c_in, in pixel]    A = weights, read transposed (MN-major)  B = scattered dz (K-major)
//   wgrad  D[c_out, (r,s,c_in)] A = dz (MN-major)                 B = im2col(x)      (MN-major)
// with K ordered (r, s, channel) so that 8 consecutive K (one 16-byte unit)
// are 8 consecutive channels of one pixel.
//
// Two persistent blocks per SM work through lists of tiles (all stages of the
// tick, balanced on the host by their number of K chunks) with three kinds of warps:
//   * producer warps (4) fill a three-stage ring of K chunks of 64.  An operand
//     that is a plain matrix in memory (the weights in all three GEMMs, dz as
//     the A operand of wgrad, and the activations / dz of 1x1 stride-1
//     convolutions) is fetched by ONE thread with a bulk tensor copy (TMA, 2-D
//     or 3-D tiles, 128-byte swizzle, zero fill outside the matrix) that
//     completes on the stage's "full" barrier; an operand that needs the
//     implicit im2col (3x3 taps, strides, padding) is gathered by all producer
//     threads with 16-byte cp.async copies, zero-filled outside the image;
//   * one MMA warp: a single thread waits for "full", issues four
//     tcgen05.mma (K = 16 each) per chunk and commits them to the stage's
//     "empty" barrier, and after a tile's last chunk to the accumulator's barrier;
//   * epilogue warps (4, one per quarter of the tensor-memory lanes) drain the
//     accumulator with tcgen05.ld while the MMA warp already works on the next
//     tile in the second accumulator (2 x 128 columns of tensor memory).
// The forward GEMM of a stage whose K fits one slice also produces what the
// normalisation needs: it writes the conv output straight into its ring slot and,
// per channel and column tile, count / mean / M2 of the values it has in registers.
// Every barrier wait is bounded; on expiry the block records an error, stops
// issuing work, waits for its copies in flight, frees its tensor memory and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "conv_types.h"

namespace pb {

constexpr int kTcChunk = 64;                  // K elements per shared-memory stage
constexpr int kTcBM = 128;
constexpr int kTcStageBytes = 16384 * 2;      // A tile + B tile
constexpr int kTcStages = 3;                  // shared-memory stages of the operand pipeline (97 KB: two blocks per SM)
constexpr int kTcEpiPitch = 20;               // floats between rows of an epilogue warp's staging buffer (16-byte aligned, conflict-free 128-bit writes)
constexpr int kTcEpiBufFloats = 32 * kTcEpiPitch;   // per epilogue warp: a 32 x 16 piece of D on its way to coalesced stores
constexpr int kTcSmemBytes = kTcStages * kTcStageBytes + 4 * kTcEpiBufFloats * 4 + 1024;
constexpr int kTcEpiWarps = 4;                // warps 0-3: quarter q of the tensor-memory lanes belongs to warp q
constexpr int kTcProdWarps = 4;               // warps 4-7
constexpr int kTcProducers = 32 * kTcProdWarps;
constexpr int kTcRowStep = kTcProducers / 8;  // K-major tiles: rows between two units of one thread (8 units per row)
constexpr int kTcRowIters = 128 / kTcRowStep;
constexpr int kTcKStep = kTcProducers / 16;   // MN-major tiles of width 128: k rows between two units of one thread
constexpr int kTcKIters = kTcChunk / kTcKStep;
constexpr int kTcLag = 1;                     // chunks a producer thread keeps in flight behind the one it is issuing (< kTcStages - 1)
constexpr int kTcMmaWarp = kTcEpiWarps + kTcProdWarps;
constexpr int kTcTmaWarp = kTcMmaWarp + 1;    // one thread of it issues every bulk tensor copy
constexpr int kTcThreads = 32 * (kTcTmaWarp + 1);
constexpr int kTcTmemCols = 256;              // two accumulators of 128 columns
constexpr long long kTcWaitNs = 200LL * 1000 * 1000;   // a barrier wait gives up after 0.2 s
constexpr int kTcMaxK = 3072;                 // longest K loop of one dgrad / wgrad tile before K is sliced
constexpr int kTcMaxKFprop = 1152;            // ... of a forward tile: the few deep stages with a longer K (3x3 on 256 or 512 channels, 1x1 on 2048)
                                              // would otherwise be the tail of the whole launch; their statistics then come from the first normalisation step

struct ConvGemmTC {
    int mode, M, N, K;
    int ci, co, k, stride, pad, ih, iw, oh, ow;
    int s, bn;                    // stage index; N-tile width (64 or 128)
    int nsplit, k_per_split;      // k_per_split is a multiple of kTcChunk
    const __nv_bfloat16* a;       // fprop: predicted weights; dgrad: weights; wgrad: dz (NHWC)
    int a_slots, a_elems;         // ring geometry of a: 1 slot, or the stashed forward weights of dgrad (then gathered, no tensor map)
    const __nv_bfloat16* b;       // fprop/wgrad: NHWC activation ring; dgrad: dz (NHWC)
    int b_slots, b_elems;
    float* c;                     // [c_slots][nsplit][M*N]
    int c_slots;
    int a_tmap, b_tmap;           // index of the operand's tensor map (bulk tensor copy), or -1: gathered
    int b_rect, b_bytes;          // B of a 3x3 stride-1 convolution fetched as boxes of whole image rows, one tap per K chunk
                                  // (b_rect = image width of the boxed tensor); bytes of one B box
    // forward GEMMs that also finish the statistics (nsplit == 1): c is then the conv-output ring
    int fuse, cpg, ntn;           // channels per normalisation group; column tiles per row of D
    float* fstat;                 // [groups][cpg * ntn][3]: count, mean, M2 of (channel, column tile)
};

// One thread block's tiles are tiles[begin[b] .. begin[b+1]).
struct TcLaunch {
    const GemmTile* tiles;
    const int* begin;
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

// Bounded wait on an mbarrier phase; gives up early once another warp has reported a failure.
__device__ __forceinline__ long long global_ns() {
    long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int* fail) {
    uint32_t done = 0;
    long long t0 = 0;
    for (int it = 0; !done; ++it) {
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (!done && (it & 63) == 63) {
            if (*fail) return false;
            const long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kTcWaitNs) return false;
        }
    }
    return true;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// Bulk tensor copies (tiles of a matrix described by a tensor map) that complete on an mbarrier.
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}

__device__ __forceinline__ void tma_4d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                 ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}

// 16-byte asynchronous global -> shared copy; with ok == false the destination is zero-filled
__device__ __forceinline__ void cp_async16(unsigned char* dst, const __nv_bfloat16* src, bool ok) {
    const int sz = ok ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(sz) : "memory");
}

struct TcShared {
    uint64_t full[kTcStages];     // a stage's operands have landed (one arrival per producer warp + 1 with the bulk copies' bytes)
    uint64_t empty[kTcStages];    // the MMAs that read a stage have completed
    uint64_t acc_full[2];         // a tile's accumulator is complete
    uint64_t acc_empty[2];        // the epilogue warps have drained an accumulator
    uint32_t tmem_base;
    int fail;
};

__device__ __forceinline__ long long tc_sample(const ConvGemmTC& G, long long t, int S) {
    return (G.mode == kFprop) ? t - G.s : t - 2LL * (S - 1) + G.s;
}

// ------------------------------------------------------------------ producer warps
__device__ void tc_producer(const ConvGemmTC* __restrict__ gemms, const GemmTile* __restrict__ tiles, int q0, int q1,
                            const TickState* ts, long long t, int S, unsigned char* smem, TcShared& sh) {
    const int ptid = threadIdx.x - 32 * kTcEpiWarps;          // 0 .. kTcProducers - 1
    const int lane = threadIdx.x & 31;
    int it = 0;                                               // chunks issued so far (all tiles)
    bool ok_all = true;
    for (int q = q0; q < q1 && ok_all; ++q) {
        const GemmTile tl = tiles[q];
        const ConvGemmTC& G = gemms[tl.gemm];
        const long long smp = tc_sample(G, t, S);
        if (!sample_live(ts, smp)) continue;
        const int mode = G.mode, M = G.M, N = G.N, BN = G.bn;
        const int kb = tl.split * G.k_per_split, ke = min(G.K, kb + G.k_per_split);
        const int nchunks = (ke - kb + kTcChunk - 1) / kTcChunk;
        const int slot = (int)(smp % G.b_slots);
        const __nv_bfloat16* __restrict__ A = G.a + (size_t)(smp % G.a_slots) * G.a_elems;
        const __nv_bfloat16* __restrict__ B = G.b + (size_t)slot * G.b_elems;
        const int CI = G.ci, CO = G.co, ksz = G.k, st = G.stride, pad = G.pad, ih = G.ih, iw = G.iw, oh = G.oh, ow = G.ow;
        const bool tmA = G.a_tmap >= 0, tmB = G.b_tmap >= 0;      // operands the bulk-copy thread fetches
        // the gathers divide by these for every 16-byte unit: reciprocals once per tile
        const float inv_ci = 1.f / (float)CI, inv_co = 1.f / (float)CO, inv_ksz = 1.f / (float)ksz,
                    inv_st = 1.f / (float)st, inv_ow = 1.f / (float)ow;
        // ---- per-thread invariants of the gathers
        // K-major tiles (rows of 8 units): unit ku of rows krow0 + kTcRowStep i
        const int ku = ptid & 7, krow0 = ptid >> 3;
        int bp[kTcRowIters], bq[kTcRowIters];               // K-major B rows: pixel coordinates (fprop: output pixel; dgrad: input pixel)
        bool bok[kTcRowIters];
        if (!tmB && mode != kWgrad) {
            const int wdt = (mode == kFprop) ? ow : iw;
            const float inv_wdt = 1.f / (float)wdt;
#pragma unroll
            for (int i = 0; i < kTcRowIters; ++i) {
                const int row = krow0 + kTcRowStep * i, n = tl.n0 + row;
                bok[i] = row < BN && n < N;
                bp[i] = quot(n, inv_wdt); bq[i] = n - bp[i] * wdt;
            }
        }
        // MN-major tiles: unit mu of k-rows k0 + step i
        const int b_units = BN >> 3;                          // 16 or 8 units per k-row of B
        const int bshift = BN == 128 ? 4 : 3;
        const int bmu = ptid & (b_units - 1), bk0 = ptid >> bshift, bkstep = kTcProducers >> bshift;
        int wr = 0, wsx = 0, wci = 0;
        bool wok = false;
        if (!tmB && mode == kWgrad) {
            const int n = tl.n0 + bmu * 8;                    // this thread's 8 consecutive n = (r, s, ci..ci+7)
            wok = n < N;
            const int rs = quot(n, inv_ci); wci = n - rs * CI; wr = quot(rs, inv_ksz); wsx = rs - wr * ksz;
        }
        const int amu = ptid & 15, ak0 = ptid >> 4;           // MN-major A (width 128): k-rows ak0 + kTcKStep i
        const bool a_m_ok = (tl.m0 + amu * 8) < M;

        for (int c = 0; c < nchunks; ++c, ++it) {
            const int stg = it % kTcStages;
            // (the verdict is taken by the whole warp, so that its lanes stay together for the warp-level arrival below)
            if (it >= kTcStages && !__all_sync(0xffffffffu, mbar_wait(smem_u32(&sh.empty[stg]), (uint32_t)(((it / kTcStages) & 1) ^ 1), &sh.fail))) { ok_all = false; break; }
            unsigned char* sA = smem + stg * kTcStageBytes;
            unsigned char* sB = sA + 16384;
            const int k0 = kb + c * kTcChunk;
            // ---------------- gathered A tile
            if (!tmA) {
                if (mode == kFprop) {
                    const int k = k0 + ku * 8;
#pragma unroll
                    for (int i = 0; i < kTcRowIters; ++i) {
                        const int row = krow0 + kTcRowStep * i, m = tl.m0 + row;
                        const bool ok = m < M && k < ke;
                        cp_async16(sA + kmajor_off(row, ku), ok ? A + (size_t)m * G.K + k : A, ok);
                    }
                } else if (mode == kDgrad) {
#pragma unroll
                    for (int i = 0; i < kTcKIters; ++i) {
                        const int kl = ak0 + kTcKStep * i, k = k0 + kl;                    // k = rs * CO + co
                        const bool ok = a_m_ok && k < ke;
                        const int rs = quot(k, inv_co), co = k - rs * CO;
                        cp_async16(sA + mnmajor_off(kl, amu), ok ? A + ((size_t)co * (ksz * ksz) + rs) * CI + tl.m0 + amu * 8 : A, ok);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < kTcKIters; ++i) {
                        const int kl = ak0 + kTcKStep * i, k = k0 + kl;                    // k = output pixel
                        const bool ok = a_m_ok && k < ke;
                        cp_async16(sA + mnmajor_off(kl, amu), ok ? A + (size_t)k * CO + tl.m0 + amu * 8 : A, ok);
                    }
                }
            }
            // ---------------- gathered B tile
            if (!tmB) {
                if (mode == kFprop) {
                    const int k = k0 + ku * 8;
                    const int rs = quot(k, inv_ci), ci = k - rs * CI, r = quot(rs, inv_ksz), s = rs - r * ksz;
#pragma unroll
                    for (int i = 0; i < kTcRowIters; ++i) {
                        const int row = krow0 + kTcRowStep * i;
                        if (row >= BN) break;
                        const int y = bp[i] * st + r - pad, x = bq[i] * st + s - pad;
                        const bool ok = bok[i] && k < ke && y >= 0 && y < ih && x >= 0 && x < iw;
                        cp_async16(sB + kmajor_off(row, ku), ok ? B + ((size_t)y * iw + x) * CI + ci : B, ok);
                    }
                } else if (mode == kDgrad) {
                    const int k = k0 + ku * 8;
                    const int rs = quot(k, inv_co), co = k - rs * CO, r = quot(rs, inv_ksz), s = rs - r * ksz;
#pragma unroll
                    for (int i = 0; i < kTcRowIters; ++i) {
                        const int row = krow0 + kTcRowStep * i;
                        if (row >= BN) break;
                        const int ty = bp[i] + pad - r, tx = bq[i] + pad - s;
                        const int p = quot(ty, inv_st), qq = quot(tx, inv_st);
                        const bool ok = bok[i] && k < ke && ty >= 0 && tx >= 0 && p * st == ty && qq * st == tx && p < oh && qq < ow;
                        cp_async16(sB + kmajor_off(row, ku), ok ? B + ((size_t)p * ow + qq) * CO + co : B, ok);
                    }
                } else {
                    for (int kl = bk0; kl < kTcChunk; kl += bkstep) {
                        const int k = k0 + kl;
                        const int p = quot(k, inv_ow), qq = k - p * ow;
                        const int y = p * st + wr - pad, x = qq * st + wsx - pad;
                        const bool ok = wok && k < ke && y >= 0 && y < ih && x >= 0 && x < iw;
                        cp_async16(sB + mnmajor_off(kl, bmu), ok ? B + ((size_t)y * iw + x) * CI + wci : B, ok);
                    }
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            // this thread's copies of the chunk issued kTcLag iterations ago have landed: make them
            // visible to the tensor core (async proxy); once the whole warp has done so, one lane
            // counts the warp in at that chunk's barrier.  The copies of the kTcLag chunks issued
            // since stay in flight meanwhile.
            if (it >= kTcLag) {
                asm volatile("cp.async.wait_group %0;" ::"n"(kTcLag) : "memory");
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.full[(it - kTcLag) % kTcStages]));
            }
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (ok_all) {
        // the chunks still owed an arrival, oldest first
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0)
            for (int c = max(0, it - kTcLag); c < it; ++c) mbar_arrive(smem_u32(&sh.full[c % kTcStages]));
    }
    if (!ok_all) sh.fail = 1;
}

// ------------------------------------------------------------------ bulk-copy thread
// Issues every bulk tensor copy of the block's tiles, chunk by chunk, as soon as the chunk's stage
// is free, and counts in at the stage's barrier with the bytes to expect.  It runs apart from the
// gathering warps, whose every iteration waits for their own copies of the chunk before: issued
// from there, the bulk copies of a chunk would start one memory latency after those of the last.
__device__ void tc_tma(const ConvGemmTC* __restrict__ gemms, const GemmTile* __restrict__ tiles, int q0, int q1,
                       const CUtensorMap* __restrict__ tmaps, const TickState* ts, long long t, int S,
                       unsigned char* smem, TcShared& sh) {
    // the descriptors of all this block's tiles on their way into the descriptor cache (a tile
    // switch would otherwise wait for them, one memory latency each)
    for (int q = q0; q < q1; ++q) {
        const ConvGemmTC& G = gemms[tiles[q].gemm];
        if (G.a_tmap >= 0) asm volatile("prefetch.tensormap [%0];" ::"l"(tmaps + G.a_tmap) : "memory");
        if (G.b_tmap >= 0) asm volatile("prefetch.tensormap [%0];" ::"l"(tmaps + G.b_tmap) : "memory");
    }
    int it = 0;
    for (int q = q0; q < q1; ++q) {
        const GemmTile tl = tiles[q];
        const ConvGemmTC& G = gemms[tl.gemm];
        const long long smp = tc_sample(G, t, S);
        if (!sample_live(ts, smp)) continue;
        const int mode = G.mode, M = G.M, N = G.N, BN = G.bn;
        const int kb = tl.split * G.k_per_split, ke = min(G.K, kb + G.k_per_split);
        const int nchunks = (ke - kb + kTcChunk - 1) / kTcChunk;
        const int slot = (int)(smp % G.b_slots);
        const int CI = G.ci, CO = G.co, ksz = G.k, pad = G.pad, b_rect = G.b_rect;
        const CUtensorMap* tmA = G.a_tmap >= 0 ? tmaps + G.a_tmap : nullptr;
        const CUtensorMap* tmB = G.b_tmap >= 0 ? tmaps + G.b_tmap : nullptr;
        // MN-major tiles arrive as boxes of 64 columns: a second box that would lie wholly outside
        // the matrix is not fetched (its rows / columns of D are never stored)
        const bool a2 = mode != kFprop && tl.m0 + 64 < M;
        const bool b2 = mode == kWgrad && BN == 128 && tl.n0 + 64 < N;
        const uint32_t tx_bytes = (tmA ? (mode == kFprop ? 16384u : (a2 ? 16384u : 8192u)) : 0u) +
                                  (tmB ? (mode == kWgrad ? (b2 ? 16384u : 8192u) : (uint32_t)G.b_bytes) : 0u);
        for (int c = 0; c < nchunks; ++c, ++it) {
            const int stg = it % kTcStages;
            if (it >= kTcStages && !mbar_wait(smem_u32(&sh.empty[stg]), (uint32_t)(((it / kTcStages) & 1) ^ 1), &sh.fail)) { sh.fail = 1; return; }
            unsigned char* sA = smem + stg * kTcStageBytes;
            unsigned char* sB = sA + 16384;
            const int k0 = kb + c * kTcChunk;
            const uint32_t fullb = smem_u32(&sh.full[stg]);
            {
                // the extra arrival of the stage, carrying the bytes of this chunk's bulk copies
                if (tx_bytes) mbar_arrive_tx(fullb, tx_bytes); else mbar_arrive(fullb);
                if (tmA) {
                    if (mode == kFprop) {
                        tma_2d(smem_u32(sA), tmA, k0, tl.m0, fullb);
                    } else if (mode == kDgrad) {
                        const int rs = k0 / CO, co0 = k0 - rs * CO;       // a chunk is 64 output channels of one tap
                        tma_3d(smem_u32(sA), tmA, tl.m0, rs, co0, fullb);
                        if (a2) tma_3d(smem_u32(sA) + 8192, tmA, tl.m0 + 64, rs, co0, fullb);
                    } else {
                        tma_2d(smem_u32(sA), tmA, tl.m0, k0, fullb);
                        if (a2) tma_2d(smem_u32(sA) + 8192, tmA, tl.m0 + 64, k0, fullb);
                    }
                }
                if (tmB) {
                    if (b_rect) {
                        // 3x3, stride 1: the chunk is 64 channels of ONE tap (r, s); the tile's pixels are whole
                        // image rows, so its operand is the same box of the image shifted by the tap
                        // (rows and columns outside the image arrive as zeros)
                        const int C = mode == kFprop ? CI : CO;
                        const int rs = k0 / C, c0 = k0 - rs * C, r = rs / ksz, sx = rs - r * ksz;
                        const int row0 = tl.n0 / b_rect;
                        if (mode == kFprop) tma_4d(smem_u32(sB), tmB, c0, sx - pad, row0 + r - pad, slot, fullb);
                        else tma_3d(smem_u32(sB), tmB, c0, pad - sx, row0 + pad - r, fullb);
                    } else if (mode == kFprop) {
                        tma_3d(smem_u32(sB), tmB, k0, tl.n0, slot, fullb);
                    } else if (mode == kDgrad) {
                        tma_2d(smem_u32(sB), tmB, k0, tl.n0, fullb);
                    } else {
                        tma_3d(smem_u32(sB), tmB, tl.n0, k0, slot, fullb);
                        if (b2) tma_3d(smem_u32(sB) + 8192, tmB, tl.n0 + 64, k0, slot, fullb);
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------ MMA warp (one thread)
__device__ void tc_mma(const ConvGemmTC* __restrict__ gemms, const GemmTile* __restrict__ tiles, int q0, int q1,
                       const TickState* ts, long long t, int S, unsigned char* smem, TcShared& sh) {
    const uint32_t tmem = sh.tmem_base;
    int it = 0, lt = 0;
    for (int q = q0; q < q1; ++q) {
        const GemmTile tl = tiles[q];
        const ConvGemmTC& G = gemms[tl.gemm];
        if (!sample_live(ts, tc_sample(G, t, S))) continue;
        const int kb = tl.split * G.k_per_split, ke = min(G.K, kb + G.k_per_split);
        const int nchunks = (ke - kb + kTcChunk - 1) / kTcChunk;
        const int a_mn = G.mode != kFprop, b_mn = G.mode == kWgrad;
        const uint32_t idesc = tc_idesc(kTcBM, G.bn, a_mn, b_mn);
        const int buf = lt & 1;
        if (lt >= 2 && !mbar_wait(smem_u32(&sh.acc_empty[buf]), (uint32_t)(((lt >> 1) & 1) ^ 1), &sh.fail)) { sh.fail = 1; return; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t dcol = tmem + (uint32_t)(buf * 128);
        for (int c = 0; c < nchunks; ++c, ++it) {
            const int stg = it % kTcStages;
            if (!mbar_wait(smem_u32(&sh.full[stg]), (uint32_t)((it / kTcStages) & 1), &sh.fail)) { sh.fail = 1; return; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sA = smem_u32(smem + stg * kTcStageBytes), sB = sA + 16384;
#pragma unroll
            for (int j = 0; j < kTcChunk / 16; ++j) {
                const uint64_t da = a_mn ? tc_desc(sA + j * 2048, 8192, 1024) : tc_desc(sA + j * 32, 16, 1024);
                const uint64_t db = b_mn ? tc_desc(sB + j * 2048, 8192, 1024) : tc_desc(sB + j * 32, 16, 1024);
                const uint32_t acc = (c > 0 || j > 0) ? 1u : 0u;
                asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                             ::"r"(dcol), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
            }
            // frees the stage once these MMAs (and all before them) have read it
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&sh.empty[stg])) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&sh.acc_full[buf])) : "memory");
        ++lt;
    }
}

// ------------------------------------------------------------------ epilogue warps
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
                   "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
                   "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
                   "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ void tc_epilogue(const ConvGemmTC* __restrict__ gemms, const GemmTile* __restrict__ tiles, int q0, int q1,
                            const TickState* ts, long long t, int S, unsigned char* smem, TcShared& sh) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;      // warp = quarter of the tensor-memory lanes
    const uint32_t tmem = sh.tmem_base;
    // A thread holds one ROW of D (32 consecutive columns per load).  Stored as they are, a warp's
    // store instruction would touch 32 rows at once (32 half-used sectors); instead 16 columns at a
    // time go through a shared-memory buffer, from which four lanes write the 64 contiguous bytes of
    // one row with 128-bit stores (eight rows per instruction), or, where rows of D do not start on
    // 16-byte boundaries (N not a multiple of 4), half a warp writes them with 32-bit stores.
    float* tb = reinterpret_cast<float*>(smem + kTcStages * kTcStageBytes) + warp * kTcEpiBufFloats;
    const int sub = lane >> 4, col = lane & 15;
    const int rsub = lane >> 2, c4 = (lane & 3) * 4;
    int lt = 0;
    for (int q = q0; q < q1; ++q) {
        const GemmTile tl = tiles[q];
        const ConvGemmTC& G = gemms[tl.gemm];
        const long long smp = tc_sample(G, t, S);
        if (!sample_live(ts, smp)) continue;
        const int M = G.M, N = G.N, BN = G.bn;
        const int buf = lt & 1;
        if (!mbar_wait(smem_u32(&sh.acc_full[buf]), (uint32_t)((lt >> 1) & 1), &sh.fail)) { sh.fail = 1; return; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float* __restrict__ Cp = G.fuse ? G.c + (size_t)(smp % G.c_slots) * ((size_t)M * N)
                                        : G.c + ((size_t)(smp % G.c_slots) * G.nsplit + tl.split) * ((size_t)M * N);
        const int m = tl.m0 + warp * 32 + lane;                     // row of D held by this thread
        const bool vec = (N & 3) == 0;
        float cnt = 0.f, mean = 0.f, m2 = 0.f;                      // statistics of this row's columns (forward, fused)
        for (int c0 = 0; c0 < BN; c0 += 32) {
            if (tl.n0 + c0 >= N) break;                             // uniform
            uint32_t r[32];
            tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * 128 + c0), r);
            const int nleft = min(N - (tl.n0 + c0), BN - c0);          // columns of this tile that exist (a tile may be narrower than 32 k)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                __syncwarp();
                float4* trow = reinterpret_cast<float4*>(tb + lane * kTcEpiPitch);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    trow[j] = make_float4(__uint_as_float(r[half * 16 + 4 * j]), __uint_as_float(r[half * 16 + 4 * j + 1]),
                                          __uint_as_float(r[half * 16 + 4 * j + 2]), __uint_as_float(r[half * 16 + 4 * j + 3]));
                __syncwarp();
                if (vec) {
                    // n0, c0 and the tile widths are multiples of 16, so nleft is a multiple of 4 here
                    const int cg = half * 16 + c4;
                    if (cg < nleft) {
                        float* dst = Cp + (size_t)(tl.m0 + warp * 32 + rsub) * N + tl.n0 + c0 + cg;
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (tl.m0 + warp * 32 + 8 * i + rsub < M)
                                *reinterpret_cast<float4*>(dst + (size_t)(8 * i) * N) = *reinterpret_cast<const float4*>(tb + (8 * i + rsub) * kTcEpiPitch + c4);
                    }
                } else {
                    const int cg = half * 16 + col;
                    if (cg < nleft) {
                        float* dst = Cp + (size_t)(tl.m0 + warp * 32 + sub) * N + tl.n0 + c0 + cg;
#pragma unroll
                        for (int rr = 0; rr < 16; ++rr)
                            if (tl.m0 + warp * 32 + 2 * rr + sub < M) dst[(size_t)(2 * rr) * N] = tb[(2 * rr + sub) * kTcEpiPitch + col];
                    }
                }
            }
            if (m < M) {
                if (G.fuse) {
                    // count / mean / M2 of these (up to) 32 values, merged into the row's running triple
                    const int nv = min(32, nleft);
                    float s = 0.f;
#pragma unroll
                    for (int u = 0; u < 32; ++u) s += (u < nv) ? __uint_as_float(r[u]) : 0.f;
                    const float mg = s / (float)nv;
                    float q2 = 0.f;
#pragma unroll
                    for (int u = 0; u < 32; ++u) { const float d = __uint_as_float(r[u]) - mg; q2 = (u < nv) ? fmaf(d, d, q2) : q2; }
                    const float tot = cnt + (float)nv, dl = mg - mean;
                    mean += dl * ((float)nv / tot);
                    m2 += q2 + dl * dl * (cnt * (float)nv / tot);
                    cnt = tot;
                }
            }
        }
        if (G.fuse && m < M) {
            const int grp = m / G.cpg, cl = m - grp * G.cpg;
            float* f = G.fstat + (((size_t)grp * G.cpg + cl) * G.ntn + tl.n0 / BN) * 3;
            f[0] = cnt; f[1] = mean; f[2] = m2;
        }
        // the accumulator may be overwritten once all four epilogue warps have read it
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.acc_empty[buf]));
        ++lt;
    }
}

__global__ void __launch_bounds__(kTcThreads, 2)
conv_tc_kernel(const ConvGemmTC* __restrict__ gemms, TcLaunch L, const CUtensorMap* __restrict__ tmaps,
               TickState* ts, int S, int par) {
    extern __shared__ unsigned char tc_smem_raw[];
    __shared__ TcShared sh;
    unsigned char* smem = (unsigned char*)(((uintptr_t)tc_smem_raw + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int q0 = L.begin[blockIdx.x], q1 = L.begin[blockIdx.x + 1];
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(kTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 32) {
        for (int q = 0; q < kTcStages; ++q) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&sh.full[q])), "r"(kTcProdWarps + 1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh.empty[q])) : "memory");
        }
        for (int q = 0; q < 2; ++q) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh.acc_full[q])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&sh.acc_empty[q])), "r"(kTcEpiWarps) : "memory");
        }
        sh.fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const long long t = ts->cnt[par];
    if (warp < kTcEpiWarps) tc_epilogue(gemms, L.tiles, q0, q1, ts, t, S, smem, sh);
    else if (warp < kTcMmaWarp) tc_producer(gemms, L.tiles, q0, q1, ts, t, S, smem, sh);
    else if (tid == 32 * kTcMmaWarp) tc_mma(gemms, L.tiles, q0, q1, ts, t, S, smem, sh);
    else if (tid == 32 * kTcTmaWarp) tc_tma(gemms, L.tiles, q0, q1, tmaps, ts, t, S, smem, sh);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (sh.fail) {
        // a wait ran out: report it and give bulk copies still in flight time to land before
        // the shared memory they write goes back to the SM
        if (tid == 0) { ts->error = kErrWait; ts->error_info = (int)blockIdx.x; }
        for (int k = 0; k < 512; ++k) __nanosleep(200);
    }
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh.tmem_base), "r"(kTcTmemCols) : "memory");
}

}  // namespace pb
