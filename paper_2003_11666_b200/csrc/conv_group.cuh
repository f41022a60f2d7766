// Group-resident normalisation kernels for tensor-core stages of large networks.
//
// GroupNorm needs a whole group before any element can be normalised (forward)
// or differentiated (backward).  For the stages of a deep bottleneck network a
// group - and even a bundle of groups that together span 8 channels, the unit
// of the bfloat16 [pixel][channel] copies - is at most a hundred kilobytes, so
// ONE thread block takes a bundle through both steps with the intermediate in
// shared memory, in one launch and with one pass over memory per direction:
//   forward   merge the (channel, column tile) statistics that the GEMM epilogue
//             left -> group mean and 1/std -> normalise, add the skip input,
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
#include "conv_stage.cuh"

namespace pb {

constexpr int kGroupThreads = 256;
constexpr int kGroupWarps = kGroupThreads / 32;
constexpr int kGroupMaxElems = 25088;          // elements of a bundle that stay in shared memory (98 KB as float32)
constexpr int kGroupMaxChannels = 64;

// One block's bundle: groups [grp0, grp0 + ngrp) of one stage.
struct GroupBlock { int stage, grp0, ngrp; };

struct GroupShared {
    float gs[kGroupMaxChannels], bb[kGroupMaxChannels];       // per channel: scale * rstd and shift (forward), gamma (backward)
    float mean[kGroupMaxChannels], rstd[kGroupMaxChannels];   // per channel copy of its group's statistics
    float s1[kGroupMaxChannels], s2[kGroupMaxChannels];       // per channel sums of dn and dn * zhat
    float m1[kGroupMaxChannels], m2[kGroupMaxChannels];       // per channel copy of its group's means
};

// ---------------------------------------------------------------- forward
template <int VEC>
__device__ void group_forward(const ConvStage& st, const GroupBlock gb, long long t, float* buf, GroupShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long i = t - st.s;
    const int slot = slot_of(i, st.slots);
    const int hw = st.oh * st.ow, cpg = st.cpg, c0 = gb.grp0 * cpg, nch = gb.ngrp * cpg;
    const size_t zelems = (size_t)st.co * hw;
    // ---- group statistics from the GEMM epilogue's partials (count, mean, M2 per channel and column tile)
    for (int g = warp; g < gb.ngrp; g += kGroupWarps) {
        const int grp = gb.grp0 + g, nidx = st.fstat_stride;
        const float* f = st.fstat + (size_t)grp * nidx * 3;
        float tot = 0.f, wsum = 0.f;
        for (int k = lane; k < nidx; k += 32) { const float n = f[3 * k]; tot += n; wsum = fmaf(n, f[3 * k + 1], wsum); }
        tot = warp_sum(tot);
        const float mean = warp_sum(wsum) / tot;
        float m2 = 0.f;
        for (int k = lane; k < nidx; k += 32) { const float d = f[3 * k + 1] - mean; m2 += f[3 * k + 2] + f[3 * k] * d * d; }
        const float rstd = rsqrtf(warp_sum(m2) / tot + kGnEps);
        if (lane == 0) {
            st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0] = mean;
            st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1] = rstd;
        }
        for (int cl = lane; cl < cpg; cl += 32) {
            const int c = c0 + g * cpg + cl;
            sh.gs[g * cpg + cl] = st.wh[st.nw + c] * rstd;
            sh.bb[g * cpg + cl] = st.wh[st.nw + st.co + c];
            sh.mean[g * cpg + cl] = mean;
        }
    }
    __syncthreads();
    const float* __restrict__ z = st.z_ring + (size_t)slot * zelems;
    const float* __restrict__ sk = st.skip_ring
        ? st.skip_ring + (size_t)slot_of(i, st.skip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w) : nullptr;
    unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems;
    float* __restrict__ out = st.out_ring + (size_t)slot * zelems;
    __nv_bfloat16* t16 = reinterpret_cast<__nv_bfloat16*>(buf);          // [nch][hw + 2]
    const int rs = hw + 2;
    const int npu = hw / VEC;
    // ---- normalise, skip, ReLU: a warp per channel, lanes over the pixels
    for (int cl = warp; cl < nch; cl += kGroupWarps) {
        const int c = c0 + cl;
        const float gs = sh.gs[cl], bb = sh.bb[cl], mean = sh.mean[cl];
        const size_t base = (size_t)c * hw;
        for (int u = lane; u < npu; u += 32) {
            const int p = u * VEC;
            float zv[VEC], sv[VEC], a[VEC];
            unsigned char cd[VEC];
            vload<VEC>(zv, z + base + p);
            if (!sk) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) sv[e] = 0.f;
            } else if (st.skip_mode == 0) {
                vload<VEC>(sv, sk + base + p);
            } else {
#pragma unroll
                for (int e = 0; e < VEC; ++e) sv[e] = skip_value(st, sk, c, (p + e) / st.ow, (p + e) % st.ow);
            }
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                const float v = fmaf(gs, zv[e] - mean, bb) + sv[e];
                const bool pass = st.relu ? v > 0.f : true;
                cd[e] = pass ? 1 : 0;
                a[e] = pass ? v : 0.f;
                t16[cl * rs + p + e] = __float2bfloat16_rn(a[e]);
            }
            stb<VEC>(code + base + p, cd);
            if (st.need_out32) vstore<VEC>(out + base + p, a);
        }
    }
    __syncthreads();
    // ---- bfloat16 [pixel][channel] copy: 16-byte runs of 8 channels (bundles span multiples of 8 channels)
    __nv_bfloat16* __restrict__ out16 = st.out16 + (size_t)slot * zelems;
    const int ng = nch >> 3;
    const unsigned short* s16 = reinterpret_cast<const unsigned short*>(t16);
    for (int idx = tid; idx < ng * hw; idx += kGroupThreads) {
        const int u = idx / hw, p = idx - u * hw;           // pixels fastest: conflict-free shared-memory reads
        const unsigned short* src = s16 + (size_t)(u * 8) * rs + p;
        uint4 v;
        v.x = src[0] | ((unsigned)src[rs] << 16);
        v.y = src[2 * rs] | ((unsigned)src[3 * rs] << 16);
        v.z = src[4 * rs] | ((unsigned)src[5 * rs] << 16);
        v.w = src[6 * rs] | ((unsigned)src[7 * rs] << 16);
        *reinterpret_cast<uint4*>(out16 + (size_t)p * st.co + c0 + u * 8) = v;
    }
}

__global__ void __launch_bounds__(kGroupThreads, 2)
conv_group_fwd_kernel(const ConvStage* __restrict__ stages, const GroupBlock* __restrict__ blocks, int nblocks,
                      const TickState* __restrict__ ts, int S, int par) {
    extern __shared__ __align__(16) float group_buf[];
    __shared__ GroupShared sh;
    __shared__ ConvStage st;
    (void)S;
    if ((int)blockIdx.x >= nblocks) return;
    const GroupBlock gb = blocks[blockIdx.x];
    {
        const int* s_ = reinterpret_cast<const int*>(&stages[gb.stage]);
        int* d_ = reinterpret_cast<int*>(&st);
        for (int k = threadIdx.x; k < (int)(sizeof(ConvStage) / 4); k += kGroupThreads) d_[k] = s_[k];
    }
    __syncthreads();
    const long long t = ts->cnt[par];
    if (!sample_live(ts, t - st.s)) return;
    if (st.vec4) group_forward<4>(st, gb, t, group_buf, sh);
    else group_forward<1>(st, gb, t, group_buf, sh);
}

// ---------------------------------------------------------------- backward
template <int VEC>
__device__ void group_backward(const ConvStage& st, const GroupBlock gb, long long j, float* dn, GroupShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slot = slot_of(j, st.slots);
    const int hw = st.oh * st.ow, cpg = st.cpg, c0 = gb.grp0 * cpg, nch = gb.ngrp * cpg;
    const size_t zelems = (size_t)st.co * hw;
    const float* __restrict__ z = st.z_ring + (size_t)slot * zelems;
    const unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems;
    const float* __restrict__ gam = st.gstash ? st.gstash + (size_t)slot_of(j, st.gstash_slots) * st.co : st.w + st.nw;
    const int rs = hw + 4;                                   // row pitch of dn in shared memory (a multiple of 4 when hw is)
    const int npu = hw / VEC;
    for (int cl = tid; cl < nch; cl += kGroupThreads) {
        const int grp = (c0 + cl) / cpg;
        sh.mean[cl] = st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0];
        sh.rstd[cl] = st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1];
        sh.gs[cl] = gam[c0 + cl];
    }
    __syncthreads();
    // ---- gradient at the normalised activation and its per-channel sums: a warp per channel
    for (int cl = warp; cl < nch; cl += kGroupWarps) {
        const size_t base = (size_t)(c0 + cl) * hw;
        const float mean = sh.mean[cl], rstd = sh.rstd[cl];
        float a1 = 0.f, a2 = 0.f;
        for (int u = lane; u < npu; u += 32) {
            const int p = u * VEC;
            float d[VEC], zv[VEC];
            unsigned char cd[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) d[e] = 0.f;
            vload<VEC>(zv, z + base + p);
            ldb<VEC>(cd, code + base + p);
            for (int q = 0; q < st.n_dsrc; ++q) {
                const float* bp = st.dsrc[q].ptr + (size_t)slot_of(j, st.dsrc[q].slots) * st.dsrc[q].nparts * zelems + base + p;
                for (int kp = 0; kp < st.dsrc[q].nparts; ++kp, bp += zelems) {
                    float r[VEC];
                    vload<VEC>(r, bp);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) d[e] += r[e];
                }
            }
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                d[e] = cd[e] ? d[e] : 0.f;
                a1 += d[e];
                a2 = fmaf(d[e], (zv[e] - mean) * rstd, a2);
                dn[cl * rs + p + e] = d[e];
            }
        }
        a1 = warp_sum(a1);
        a2 = warp_sum(a2);
        if (lane == 0) {
            sh.s1[cl] = a1; sh.s2[cl] = a2;
            st.g[st.nw + c0 + cl] = a2;                      // gradient of the scale
            st.g[st.nw + st.co + c0 + cl] = a1;              // gradient of the shift
        }
    }
    __syncthreads();
    // ---- the two means of every group (with the scale in use), in channel order
    for (int g = tid; g < gb.ngrp; g += kGroupThreads) {
        float m1 = 0.f, m2 = 0.f;
        for (int cl = 0; cl < cpg; ++cl) {
            m1 = fmaf(sh.gs[g * cpg + cl], sh.s1[g * cpg + cl], m1);
            m2 = fmaf(sh.gs[g * cpg + cl], sh.s2[g * cpg + cl], m2);
        }
        m1 /= (float)(cpg * hw); m2 /= (float)(cpg * hw);
        for (int cl = 0; cl < cpg; ++cl) { sh.m1[g * cpg + cl] = m1; sh.m2[g * cpg + cl] = m2; }
    }
    __syncthreads();
    // ---- gradient at the conv output (kept in place of dn), gradient of the skip input
    float* __restrict__ dsk = st.dskip
        ? st.dskip + (size_t)slot_of(j, st.dskip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w) : nullptr;
    for (int cl = warp; cl < nch; cl += kGroupWarps) {
        const int c = c0 + cl;
        const size_t base = (size_t)c * hw;
        const float mean = sh.mean[cl], rstd = sh.rstd[cl], gv = sh.gs[cl], m1 = sh.m1[cl], m2 = sh.m2[cl];
        for (int u = lane; u < npu; u += 32) {
            const int p = u * VEC;
            float zv[VEC], d[VEC];
            vload<VEC>(zv, z + base + p);
#pragma unroll
            for (int e = 0; e < VEC; ++e) d[e] = dn[cl * rs + p + e];
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
            for (int e = 0; e < VEC; ++e) {
                const float zh = (zv[e] - mean) * rstd;
                dn[cl * rs + p + e] = rstd * (fmaf(d[e], gv, -m1) - zh * m2);
            }
        }
    }
    __syncthreads();
    // ---- bfloat16 [pixel][channel] operand of dgrad / wgrad
    const int ng = nch >> 3;
    for (int idx = tid; idx < ng * hw; idx += kGroupThreads) {
        const int u = idx / hw, p = idx - u * hw;
        const float* src = dn + (size_t)(u * 8) * rs + p;
        __nv_bfloat162 b0 = __floats2bfloat162_rn(src[0], src[rs]), b1 = __floats2bfloat162_rn(src[2 * rs], src[3 * rs]);
        __nv_bfloat162 b2 = __floats2bfloat162_rn(src[4 * rs], src[5 * rs]), b3 = __floats2bfloat162_rn(src[6 * rs], src[7 * rs]);
        uint4 v;
        v.x = *reinterpret_cast<unsigned*>(&b0); v.y = *reinterpret_cast<unsigned*>(&b1);
        v.z = *reinterpret_cast<unsigned*>(&b2); v.w = *reinterpret_cast<unsigned*>(&b3);
        *reinterpret_cast<uint4*>(st.dz16 + (size_t)p * st.co + c0 + u * 8) = v;
    }
}

__global__ void __launch_bounds__(kGroupThreads, 2)
conv_group_bwd_kernel(const ConvStage* __restrict__ stages, const GroupBlock* __restrict__ blocks, int nblocks,
                      const TickState* __restrict__ ts, int S, int par) {
    extern __shared__ __align__(16) float group_buf[];
    __shared__ GroupShared sh;
    __shared__ ConvStage st;
    if ((int)blockIdx.x >= nblocks) return;
    const GroupBlock gb = blocks[blockIdx.x];
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
