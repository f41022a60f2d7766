// Group-resident normalisation kernels for tensor-core stages of large networks.
//
// GroupNorm needs a whole group before any element can be normalised (forward)
// or differentiated (backward).  For the stages of a deep bottleneck network a
// group - and even a bundle of groups that together span 8 channels, the unit
// of the bfloat16 [pixel][channel] copies - is at most a hundred kilobytes, so
// a CLUSTER of four thread blocks takes a bundle through both steps with the
// intermediate in shared memory, in one launch and with one pass over memory per
// direction; each block of the cluster owns a quarter of the pixels (so that many
// blocks fit on an SM) and the per-channel sums cross the cluster through
// distributed shared memory:
//   forward   merge the (channel, column tile) statistics that the GEMM epilogue
//             left (or, where the GEMM left K slices, sum them and take the
//             statistics of the sum) -> group mean and 1/std -> normalise, add the skip input,
//             ReLU -> float32 output (only where somebody reads it), ReLU mask,
//             and the bfloat16 copy, transposed through shared memory;
//   backward  gradient at the normalised activation (consumers' partial rows
//             summed, gated by the mask) into shared memory, per-channel sums
//             by one warp per channel -> scale / shift gradients and the two
//             group means -> gradient at the conv output, written as the
//             bfloat16 [pixel][channel] operand of dgrad / wgrad (these stages
//             need no float32 copy), and the skip input's gradient.
// Reductions have a fixed order (lanes over pixels, then a warp shuffle tree), so
// results do not depend on scheduling.
#pragma once
#include <cooperative_groups.h>

#include "conv_stage.cuh"

namespace pb {

constexpr int kGroupThreads = 256;
constexpr int kGroupWarps = kGroupThreads / 32;
constexpr int kGroupMaxElems = 25088;          // elements of a bundle that stay in shared memory (98 KB as float32)
constexpr int kGroupMaxChannels = 256;        // channels of a bundle
constexpr int kGroupTargetElems = 12544;       // small groups are bundled up to about this many elements (one block then has a few thousand)
constexpr int kGroupSliceElems = 6272;         // a bundle whose forward GEMM left K slices also keeps their float32 sum in shared memory: at most this many elements
constexpr int kGroupSliceTarget = 3136;        // ... and such groups are bundled only up to this many
constexpr int kGroupMaxRows = kMaxDeltaSrc * 16;   // partial rows of all consumers of one stage (a consumer's dgrad has at most 16 K slices)
constexpr int kGroupSplit = 4;                 // blocks (one cluster) that share a bundle's pixels

// One block's bundle: groups [grp0, grp0 + ngrp) of one stage.
struct GroupBlock { int stage, grp0, ngrp; };

struct GroupShared {
    float gs[kGroupMaxChannels], bb[kGroupMaxChannels];       // per channel: scale * rstd and shift (forward), gamma (backward)
    float mean[kGroupMaxChannels], rstd[kGroupMaxChannels];   // per channel copy of its group's statistics
    float s1[kGroupMaxChannels], s2[kGroupMaxChannels];       // per channel sums of dn and dn * zhat
    float m1[kGroupMaxChannels], m2[kGroupMaxChannels];       // per channel copy of its group's means
    float t1[kGroupMaxChannels], t2[kGroupMaxChannels];       // the sums over the whole cluster
    const float* rows[kGroupMaxRows];                         // backward: the consumers' partial rows for this sample, in summation order
    int nrows;
    float part[kGroupWarps][3];                               // forward: a warp's share of a group's statistics
};

// Pixel units [lo, hi) of block `rank` of a bundle's cluster (npu units of VEC pixels per channel).
__device__ __forceinline__ void group_range(int npu, int rank, int& lo, int& hi) {
    lo = (int)((long long)npu * rank / kGroupSplit);
    hi = (int)((long long)npu * (rank + 1) / kGroupSplit);
}

// ---------------------------------------------------------------- forward
template <int VEC>
__device__ void group_forward(const ConvStage& st, const GroupBlock gb, int rank, long long t, float* buf, GroupShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long i = t - st.s;
    const int slot = slot_of(i, st.slots);
    const int hw = st.oh * st.ow, cpg = st.cpg, c0 = gb.grp0 * cpg, nch = gb.ngrp * cpg;
    const size_t zelems = (size_t)st.co * hw;
    const int npu = hw / VEC;
    int u_lo, u_hi;
    group_range(npu, rank, u_lo, u_hi);
    const int p_lo = u_lo * VEC, np = (u_hi - u_lo) * VEC;               // this block's pixels
    // ---- group statistics (every block of the bundle computes the same numbers)
    __nv_bfloat16* t16 = reinterpret_cast<__nv_bfloat16*>(buf);          // [nch][np + 2]
    const int rs = np + 2;
    float* zs = buf + ((nch * rs * 2 + 15) / 16) * 4;                    // [nch][hw]: sum of the K slices (only where the GEMM left slices)
    if (st.fused) {
        // From the GEMM epilogue's partials (count, mean, M2 per channel and column tile).  A bundle
        // of few groups gives each group several warps: wpg warps fold the entries k = sub * 32 + lane,
        // + 32 wpg, ... of a group into one triple per lane (independent loads), merge them along a
        // fixed shuffle tree, and one thread merges the warps' triples in warp order.
        int wpg = 1;
        while (2 * wpg * gb.ngrp <= kGroupWarps) wpg *= 2;
        const int gpp = kGroupWarps / wpg;                               // groups per pass
        const int nidx = st.fstat_stride;
        for (int g0 = 0; g0 < gb.ngrp; g0 += gpp) {
            const int g = g0 + warp / wpg, sub = warp % wpg;
            float n = 0.f, mean = 0.f, m2 = 0.f;
            if (g < gb.ngrp) {
                const float* f = st.fstat + (size_t)(gb.grp0 + g) * nidx * 3;
                for (int k = sub * 32 + lane; k < nidx; k += 32 * wpg) {
                    const float nb = f[3 * k], mb = f[3 * k + 1], qb = f[3 * k + 2];
                    const float tot = n + nb, dl = mb - mean;
                    if (tot > 0.f) { mean += dl * (nb / tot); m2 += qb + dl * dl * (n * nb / tot); }
                    n = tot;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float nb = __shfl_xor_sync(0xffffffffu, n, o), mb = __shfl_xor_sync(0xffffffffu, mean, o), qb = __shfl_xor_sync(0xffffffffu, m2, o);
                // (both partners compute the same merged triple: a and b enter symmetrically up to the sign of dl)
                const bool low = (lane & o) == 0;
                const float na = low ? n : nb, ma = low ? mean : mb, qa = low ? m2 : qb;
                const float nc = low ? nb : n, mc = low ? mb : mean, qc = low ? qb : m2;
                const float tot = na + nc, dl = mc - ma;
                if (tot > 0.f) { mean = ma + dl * (nc / tot); m2 = qa + qc + dl * dl * (na * nc / tot); } else { mean = 0.f; m2 = 0.f; }
                n = tot;
            }
            if (lane == 0) { sh.part[warp][0] = n; sh.part[warp][1] = mean; sh.part[warp][2] = m2; }
            __syncthreads();
            if (tid < gpp && g0 + tid < gb.ngrp) {
                float na = sh.part[tid * wpg][0], ma = sh.part[tid * wpg][1], qa = sh.part[tid * wpg][2];
                for (int w = 1; w < wpg; ++w) {
                    const float nc = sh.part[tid * wpg + w][0], mc = sh.part[tid * wpg + w][1], qc = sh.part[tid * wpg + w][2];
                    const float tot = na + nc, dl = mc - ma;
                    if (tot > 0.f) { ma += dl * (nc / tot); qa += qc + dl * dl * (na * nc / tot); }
                    na = tot;
                }
                const float rstd = rsqrtf(qa / na + kGnEps);
                const int gg = g0 + tid, grp = gb.grp0 + gg;
                sh.m1[gg] = ma; sh.m2[gg] = rstd;
                if (rank == 0) {
                    st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0] = ma;
                    st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1] = rstd;
                }
            }
            __syncthreads();
        }
    } else {
        // The forward GEMM left K slices: the conv output is their sum in slice order, kept in shared
        // memory for the whole bundle (this block files its own pixels in the ring for the backward);
        // then mean and squared deviations of every group, a warp per group.
        const int ne = nch * hw;
        const float inv_hw = 1.f / (float)hw;
        const float* __restrict__ zp = st.zpart + (size_t)c0 * hw;
        float* __restrict__ zr = st.z_ring + (size_t)slot * zelems + (size_t)c0 * hw;
        for (int e0 = tid; e0 < ne; e0 += 4 * kGroupThreads) {
            float v[4] = {0.f, 0.f, 0.f, 0.f};                  // four elements of a thread in flight (loads before any store)
            for (int q = 0; q < st.z_nsplit; ++q)
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int e = e0 + k * kGroupThreads;
                    if (e < ne) v[k] += zp[(size_t)q * zelems + e];
                }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int e = e0 + k * kGroupThreads;
                if (e < ne) {
                    zs[e] = v[k];
                    const int p = e - quot(e, inv_hw) * hw;
                    if (p >= p_lo && p < p_lo + np) zr[e] = v[k];
                }
            }
        }
        __syncthreads();
        const int gne = cpg * hw;
        for (int g = warp; g < gb.ngrp; g += kGroupWarps) {
            const float* zg = zs + g * gne;
            float s1 = 0.f;
            for (int e = lane; e < gne; e += 32) s1 += zg[e];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s1 += __shfl_xor_sync(0xffffffffu, s1, o);
            const float mean = s1 / (float)gne;
            float s2 = 0.f;
            for (int e = lane; e < gne; e += 32) { const float d = zg[e] - mean; s2 = fmaf(d, d, s2); }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o);
            if (lane == 0) {
                const float rstd = rsqrtf(s2 / (float)gne + kGnEps);
                const int grp = gb.grp0 + g;
                sh.m1[g] = mean; sh.m2[g] = rstd;
                if (rank == 0) {
                    st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0] = mean;
                    st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1] = rstd;
                }
            }
        }
        __syncthreads();
    }
    for (int cl = tid; cl < nch; cl += kGroupThreads) {
        const int g = cl / cpg, c = c0 + cl;
        sh.gs[cl] = st.wh[st.nw + c] * sh.m2[g];
        sh.bb[cl] = st.wh[st.nw + st.co + c];
        sh.mean[cl] = sh.m1[g];
    }
    __syncthreads();
    const float* __restrict__ z = st.z_ring + (size_t)slot * zelems;
    const float* __restrict__ sk = st.skip_ring
        ? st.skip_ring + (size_t)slot_of(i, st.skip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w) : nullptr;
    unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems;
    float* __restrict__ out = st.out_ring + (size_t)slot * zelems;
    // ---- normalise, skip, ReLU: the bundle's (channel, pixel unit) pairs spread flat over the
    // block, four units of a thread in flight at a time (a channel's share of the pixels can be
    // a dozen pixels: per-channel loops would wait one memory latency per channel)
    const int upc = u_hi - u_lo, total = nch * upc;
    const float inv_upc = 1.f / (float)max(upc, 1);
    // (explicit batches of U units: all loads of a batch are issued before any is used, whatever the
    //  branches on the kind of skip input do to the compiler's own unrolling)
    constexpr int U = VEC == 4 ? 4 : 8;
    const bool fused = st.fused != 0, relu = st.relu != 0, out32 = st.need_out32 != 0;
    const int skip_kind = !sk ? 0 : (st.skip_mode == 0 ? 1 : 2);
    for (int i0 = tid; i0 < total; i0 += U * kGroupThreads) {
        int cl[U], p[U];
        float zv[U][VEC], sv[U][VEC];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int idx = min(i0 + k * kGroupThreads, total - 1);      // (a unit beyond the end repeats the last one and is not stored)
            cl[k] = quot(idx, inv_upc);
            p[k] = (u_lo + idx - cl[k] * upc) * VEC;
            const size_t base = (size_t)(c0 + cl[k]) * hw;
            if (fused) {
                vload<VEC>(zv[k], z + base + p[k]);
            } else {
#pragma unroll
                for (int e = 0; e < VEC; ++e) zv[k][e] = zs[cl[k] * hw + p[k] + e];
            }
            if (skip_kind == 1) {
                vload<VEC>(sv[k], sk + base + p[k]);
            } else if (skip_kind == 2) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) sv[k][e] = skip_value(st, sk, c0 + cl[k], (p[k] + e) / st.ow, (p[k] + e) % st.ow);
            } else {
#pragma unroll
                for (int e = 0; e < VEC; ++e) sv[k][e] = 0.f;
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (i0 + k * kGroupThreads >= total) break;
            const float gs = sh.gs[cl[k]], bb = sh.bb[cl[k]], mean = sh.mean[cl[k]];
            const size_t base = (size_t)(c0 + cl[k]) * hw;
            float a[VEC];
            unsigned char cd[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                const float v = fmaf(gs, zv[k][e] - mean, bb) + sv[k][e];
                const bool pass = relu ? v > 0.f : true;
                cd[e] = pass ? 1 : 0;
                a[e] = pass ? v : 0.f;
                t16[cl[k] * rs + p[k] - p_lo + e] = __float2bfloat16_rn(a[e]);
            }
            stb<VEC>(code + base + p[k], cd);
            if (out32) vstore<VEC>(out + base + p[k], a);
        }
    }
    __syncthreads();
    // ---- bfloat16 [pixel][channel] copy: 16-byte runs of 8 channels (bundles span multiples of 8 channels)
    __nv_bfloat16* __restrict__ out16 = st.out16 + (size_t)slot * zelems;
    const int ng = nch >> 3;
    const unsigned short* s16 = reinterpret_cast<const unsigned short*>(t16);
    for (int idx = tid; idx < ng * np; idx += kGroupThreads) {
        const int u = idx / np, p = idx - u * np;           // pixels fastest: conflict-free shared-memory reads
        const unsigned short* src = s16 + (size_t)(u * 8) * rs + p;
        uint4 v;
        v.x = src[0] | ((unsigned)src[rs] << 16);
        v.y = src[2 * rs] | ((unsigned)src[3 * rs] << 16);
        v.z = src[4 * rs] | ((unsigned)src[5 * rs] << 16);
        v.w = src[6 * rs] | ((unsigned)src[7 * rs] << 16);
        *reinterpret_cast<uint4*>(out16 + (size_t)(p_lo + p) * st.co + c0 + u * 8) = v;
    }
}

__global__ void __launch_bounds__(kGroupThreads, 4)
conv_group_fwd_kernel(const ConvStage* __restrict__ stages, const GroupBlock* __restrict__ blocks, int nblocks,
                      const TickState* __restrict__ ts, int S, int par) {
    extern __shared__ __align__(16) float group_buf[];
    __shared__ GroupShared sh;
    __shared__ ConvStage st;
    (void)S;
    if ((int)blockIdx.x >= nblocks * kGroupSplit) return;
    const GroupBlock gb = blocks[blockIdx.x / kGroupSplit];
    const int rank = blockIdx.x % kGroupSplit;
    {
        const int* s_ = reinterpret_cast<const int*>(&stages[gb.stage]);
        int* d_ = reinterpret_cast<int*>(&st);
        for (int k = threadIdx.x; k < (int)(sizeof(ConvStage) / 4); k += kGroupThreads) d_[k] = s_[k];
    }
    __syncthreads();
    const long long t = ts->cnt[par];
    if (!sample_live(ts, t - st.s)) return;
    if (st.vec4) group_forward<4>(st, gb, rank, t, group_buf, sh);
    else group_forward<1>(st, gb, rank, t, group_buf, sh);
}

// ---------------------------------------------------------------- backward
template <int VEC>
__device__ void group_backward(const ConvStage& st, const GroupBlock gb, long long j, float* dn, GroupShared& sh) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slot = slot_of(j, st.slots);
    const int hw = st.oh * st.ow, cpg = st.cpg, c0 = gb.grp0 * cpg, nch = gb.ngrp * cpg;
    const size_t zelems = (size_t)st.co * hw;
    const float* __restrict__ z = st.z_ring + (size_t)slot * zelems;
    const unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems;
    const float* __restrict__ gam = st.gstash ? st.gstash + (size_t)slot_of(j, st.gstash_slots) * st.co : st.w + st.nw;
    const int npu = hw / VEC;
    int u_lo, u_hi;
    group_range(npu, rank, u_lo, u_hi);
    const int p_lo = u_lo * VEC, np = (u_hi - u_lo) * VEC;   // this block's pixels
    const int rs = np <= 16 ? ((np + 4) | 1) : np + 4;       // row pitch of dn and zhat in shared memory (odd where a thread walks a row)
    float* zh = dn + (size_t)nch * rs;                       // normalised conv output, kept beside dn
    for (int cl = tid; cl < nch; cl += kGroupThreads) {
        const int grp = (c0 + cl) / cpg;
        sh.mean[cl] = st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0];
        sh.rstd[cl] = st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1];
        sh.gs[cl] = gam[c0 + cl];
    }
    // the consumers' partial rows for this sample, flat and in summation order (consumer, then K slice)
    if (tid == 0) {
        int nr = 0;
        for (int q = 0; q < st.n_dsrc; ++q) {
            const float* p0 = st.dsrc[q].ptr + (size_t)slot_of(j, st.dsrc[q].slots) * st.dsrc[q].nparts * zelems;
            for (int kp = 0; kp < st.dsrc[q].nparts && nr < kGroupMaxRows; ++kp) sh.rows[nr++] = p0 + (size_t)kp * zelems;
        }
        sh.nrows = nr;
    }
    __syncthreads();
    const int nrows = sh.nrows;
    // ---- gradient at the normalised activation, and the normalised conv output, into shared
    // memory: the bundle's (channel, pixel unit) pairs spread flat over the block, several units
    // of a thread in flight at a time
    const int upc = u_hi - u_lo, total = nch * upc;
    const float inv_upc = 1.f / (float)max(upc, 1);
    // (explicit batches of U units x 4 rows: all loads of a batch are issued before any is used)
    constexpr int U = VEC == 4 ? 2 : 4;
    for (int i0 = tid; i0 < total; i0 += U * kGroupThreads) {
        int cl[U], p[U];
        size_t off[U];
        float d[U][VEC], zv[U][VEC];
        unsigned char cd[U][VEC];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int idx = min(i0 + k * kGroupThreads, total - 1);      // (a unit beyond the end repeats the last one and is not stored)
            cl[k] = quot(idx, inv_upc);
            p[k] = (u_lo + idx - cl[k] * upc) * VEC;
            off[k] = (size_t)(c0 + cl[k]) * hw + p[k];
            vload<VEC>(zv[k], z + off[k]);
            ldb<VEC>(cd[k], code + off[k]);
#pragma unroll
            for (int e = 0; e < VEC; ++e) d[k][e] = 0.f;
        }
        // the consumers' rows in summation order, four rows in flight per unit (a row beyond the list
        // re-reads row 0 and counts as zero)
        for (int r0 = 0; r0 < nrows; r0 += 4) {
            float r[U][4][VEC];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float* rp = sh.rows[r0 + j < nrows ? r0 + j : 0];
#pragma unroll
                for (int k = 0; k < U; ++k) vload<VEC>(r[k][j], rp + off[k]);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int k = 0; k < U; ++k)
#pragma unroll
                    for (int e = 0; e < VEC; ++e) d[k][e] += (r0 + j < nrows) ? r[k][j][e] : 0.f;
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (i0 + k * kGroupThreads >= total) break;
            const float mean = sh.mean[cl[k]], rstd = sh.rstd[cl[k]];
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                dn[cl[k] * rs + p[k] - p_lo + e] = cd[k][e] ? d[k][e] : 0.f;
                zh[cl[k] * rs + p[k] - p_lo + e] = (zv[k][e] - mean) * rstd;
            }
        }
    }
    __syncthreads();
    // ---- per-channel sums of dn and dn * zhat over this block's pixels, from shared memory: a thread
    // per channel where a block has at most 16 pixels of each (odd pitch: no bank conflicts), else a
    // warp per channel
    if (np <= 16) {
        for (int cl = tid; cl < nch; cl += kGroupThreads) {
            float a1 = 0.f, a2 = 0.f;
            for (int p = 0; p < np; ++p) {
                const float d = dn[cl * rs + p];
                a1 += d;
                a2 = fmaf(d, zh[cl * rs + p], a2);
            }
            sh.s1[cl] = a1; sh.s2[cl] = a2;                  // this block's pixels only
        }
    } else {
        for (int cl = warp; cl < nch; cl += kGroupWarps) {
            float a1 = 0.f, a2 = 0.f;
            for (int p = lane; p < np; p += 32) {
                const float d = dn[cl * rs + p];
                a1 += d;
                a2 = fmaf(d, zh[cl * rs + p], a2);
            }
            a1 = warp_sum(a1);
            a2 = warp_sum(a2);
            if (lane == 0) { sh.s1[cl] = a1; sh.s2[cl] = a2; }
        }
    }
    // ---- the cluster's blocks add their sums up in rank order (distributed shared memory)
    cluster.sync();
    for (int cl = tid; cl < nch; cl += kGroupThreads) {
        float a1 = 0.f, a2 = 0.f;
        for (int r = 0; r < kGroupSplit; ++r) {
            const GroupShared* peer = cluster.map_shared_rank(&sh, r);
            a1 += peer->s1[cl]; a2 += peer->s2[cl];
        }
        sh.t1[cl] = a1; sh.t2[cl] = a2;
        if (rank == 0) {
            st.g[st.nw + c0 + cl] = a2;                      // gradient of the scale
            st.g[st.nw + st.co + c0 + cl] = a1;              // gradient of the shift
        }
    }
    __syncthreads();
    // ---- the two means of every group (with the scale in use), in channel order
    for (int g = tid; g < gb.ngrp; g += kGroupThreads) {
        float m1 = 0.f, m2 = 0.f;
        for (int cl = 0; cl < cpg; ++cl) {
            m1 = fmaf(sh.gs[g * cpg + cl], sh.t1[g * cpg + cl], m1);
            m2 = fmaf(sh.gs[g * cpg + cl], sh.t2[g * cpg + cl], m2);
        }
        m1 /= (float)(cpg * hw); m2 /= (float)(cpg * hw);
        for (int cl = 0; cl < cpg; ++cl) { sh.m1[g * cpg + cl] = m1; sh.m2[g * cpg + cl] = m2; }
    }
    __syncthreads();
    // ---- gradient at the conv output (kept in place of dn), gradient of the skip input
    float* __restrict__ dsk = st.dskip
        ? st.dskip + (size_t)slot_of(j, st.dskip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w) : nullptr;
#pragma unroll(VEC == 4 ? 2 : 8)
    for (int idx = tid; idx < total; idx += kGroupThreads) {
        const int cl = quot(idx, inv_upc), u = u_lo + idx - cl * upc;
        const int c = c0 + cl, p = u * VEC;
        const size_t base = (size_t)c * hw;
        const float rstd = sh.rstd[cl], gv = sh.gs[cl], m1 = sh.m1[cl], m2 = sh.m2[cl];
        float d[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) d[e] = dn[cl * rs + p - p_lo + e];
        if (dsk) {
            // the skip input joined after the normalisation: it receives dn itself
            if (st.skip_mode == 0) {
                vstore<VEC>(dsk + base + p, d);
            } else if (c < st.skip_c) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    const int y = (p + e) / st.ow, x = (p + e) % st.ow;
                    for (int dy = 0; dy < 2; ++dy)
                        for (int dx = 0; dx < 2; ++dx) {
                            const int ys = 2 * y + dy, xs = 2 * x + dx;
                            if (ys < st.skip_h && xs < st.skip_w)
                                dsk[((size_t)c * st.skip_h + ys) * st.skip_w + xs] = (dy | dx) ? 0.f : d[e];
                        }
                }
            }
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e)
            dn[cl * rs + p - p_lo + e] = rstd * (fmaf(d[e], gv, -m1) - zh[cl * rs + p - p_lo + e] * m2);
    }
    __syncthreads();
    // ---- bfloat16 [pixel][channel] operand of dgrad / wgrad
    const int ng = nch >> 3;
    for (int idx = tid; idx < ng * np; idx += kGroupThreads) {
        const int u = idx / np, p = idx - u * np;
        const float* src = dn + (size_t)(u * 8) * rs + p;
        __nv_bfloat162 b0 = __floats2bfloat162_rn(src[0], src[rs]), b1 = __floats2bfloat162_rn(src[2 * rs], src[3 * rs]);
        __nv_bfloat162 b2 = __floats2bfloat162_rn(src[4 * rs], src[5 * rs]), b3 = __floats2bfloat162_rn(src[6 * rs], src[7 * rs]);
        uint4 v;
        v.x = *reinterpret_cast<unsigned*>(&b0); v.y = *reinterpret_cast<unsigned*>(&b1);
        v.z = *reinterpret_cast<unsigned*>(&b2); v.w = *reinterpret_cast<unsigned*>(&b3);
        *reinterpret_cast<uint4*>(st.dz16 + (size_t)(p_lo + p) * st.co + c0 + u * 8) = v;
    }
    cluster.sync();          // no block leaves while another may still read its sums
}

__global__ void __cluster_dims__(kGroupSplit, 1, 1) __launch_bounds__(kGroupThreads, 3)
conv_group_bwd_kernel(const ConvStage* __restrict__ stages, const GroupBlock* __restrict__ blocks, int nblocks,
                      const TickState* __restrict__ ts, int S, int par) {
    extern __shared__ __align__(16) float group_buf[];
    __shared__ GroupShared sh;
    __shared__ ConvStage st;
    if ((int)blockIdx.x >= nblocks * kGroupSplit) return;       // (uniform over a cluster: the grid is nblocks clusters)
    const GroupBlock gb = blocks[blockIdx.x / kGroupSplit];
    {
        const int* s_ = reinterpret_cast<const int*>(&stages[gb.stage]);
        int* d_ = reinterpret_cast<int*>(&st);
        for (int k = threadIdx.x; k < (int)(sizeof(ConvStage) / 4); k += kGroupThreads) d_[k] = s_[k];
    }
    __syncthreads();
    const long long j = ts->cnt[par] - 2LL * (S - 1) + st.s;
    if (!sample_live(ts, j)) return;
    if (st.vec4) group_backward<4>(st, gb, j, group_buf, sh);
    else group_backward<1>(st, gb, j, group_buf, sh);
}

}  // namespace pb
