// Per-stage normalisation / activation / pooling kernels and the fused update.
//
// A convolution stage is  conv -> GroupNorm -> (+skip) -> ReLU -> (max-pool |
// global average pool).  One thread block owns one normalisation group of one
// stage, so every reduction (group statistics, per-channel gradient sums)
// stays inside the block and has a fixed order.
#pragma once
#include "conv_types.h"
#include "fc_kernels.cuh"   // ring_slot, warp_sum

namespace pb {

constexpr float kGnEps = 1e-5f;

struct GroupShared {
    float red[kGroupThreads / 32];
    float wp1[kGroupThreads / 32], wp2[kGroupThreads / 32];
    float s1[kMaxGroupChannels], s2[kMaxGroupChannels];
    float bc[4];
};

__device__ __forceinline__ float block_sum(float x, GroupShared& sh) {
    x = warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = x;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int k = 0; k < kGroupThreads / 32; ++k) tot += sh.red[k];
    return tot;
}

__device__ __forceinline__ float skip_value(const ConvStage& st, const float* __restrict__ sk, int c, int y, int x) {
    if (st.skip_mode == 0) return sk[((size_t)c * st.skip_h + y) * st.skip_w + x];
    return c < st.skip_c ? sk[((size_t)c * st.skip_h + 2 * y) * st.skip_w + 2 * x] : 0.f;
}

// ---------------------------------------------------------------- forward
// grid: one block per (stage, group); `map` gives (stage, group) per block.
__global__ void __launch_bounds__(kGroupThreads)
conv_post_fwd_kernel(const ConvStage* __restrict__ stages, const int2* __restrict__ map,
                     const TickState* __restrict__ ts, int par) {
    __shared__ GroupShared sh;
    const ConvStage& st = stages[map[blockIdx.x].x];
    const int grp = map[blockIdx.x].y;
    const long long i = ts->cnt[par] - st.s;
    if (i < 0) return;
    const int slot = ring_slot(i, st.slots);
    const int hw = st.oh * st.ow, cpg = st.cpg, n = cpg * hw, c0 = grp * cpg;
    const size_t zelems = (size_t)st.co * hw;
    float* __restrict__ z = st.z_ring + (size_t)slot * zelems + (size_t)c0 * hw;
    const float* __restrict__ zp = st.zpart + (size_t)c0 * hw;
    const int tid = threadIdx.x;

    // 1. add the K-slices of the convolution, keep z, group mean
    float sum = 0.f;
    for (int e = tid; e < n; e += kGroupThreads) {
        float v = 0.f;
        for (int q = 0; q < st.z_nsplit; ++q) v += zp[(size_t)q * zelems + e];
        z[e] = v;
        sum += v;
    }
    const float mean = block_sum(sum, sh) / (float)n;
    // 2. biased variance about the mean
    float sq = 0.f;
    for (int e = tid; e < n; e += kGroupThreads) { const float d = z[e] - mean; sq = fmaf(d, d, sq); }
    const float var = block_sum(sq, sh) / (float)n;
    const float rstd = rsqrtf(var + kGnEps);
    if (tid == 0) {
        st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0] = mean;
        st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1] = rstd;
    }
    // 3. normalise with the predicted scale/shift, add the skip input, activate
    const float* __restrict__ gam = st.wh + st.nw;
    const float* __restrict__ bet = gam + st.co;
    const float* __restrict__ sk = st.skip_ring
        ? st.skip_ring + (size_t)ring_slot(i, st.skip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w) : nullptr;
    unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems + (size_t)c0 * hw;
    const bool pooled = st.pool_k > 0 || st.avgpool;
    const size_t oelems = (size_t)st.co * st.out_h * st.out_w;
    float* __restrict__ out = st.out_ring + (size_t)slot * oelems;
    __nv_bfloat16* __restrict__ out16 = st.out16 ? st.out16 + (size_t)slot * oelems : nullptr;
    auto act = [&](int e) -> float {
        const int c = c0 + e / hw, p = e % hw;
        float v = fmaf(gam[c] * rstd, z[e] - mean, bet[c]);
        if (sk) v += skip_value(st, sk, c, p / st.ow, p % st.ow);
        return v;
    };
    for (int e = tid; e < n; e += kGroupThreads) {
        const float v = act(e);
        const bool pass = st.relu ? v > 0.f : true;
        code[e] = pass ? 1 : 0;
        if (!pooled) {
            const float a = pass ? v : 0.f;
            out[(size_t)c0 * hw + e] = a;
            if (out16) out16[(size_t)(e % hw) * st.co + c0 + e / hw] = __float2bfloat16_rn(a);
        }
    }
    if (st.pool_k > 0) {
        // 4a. max-pool: first maximum in row-major window order; padding never wins
        const int ohw = st.out_h * st.out_w, k = st.pool_k;
        unsigned char* __restrict__ arg = st.arg_ring + (size_t)slot * oelems + (size_t)c0 * ohw;
        for (int o = tid; o < cpg * ohw; o += kGroupThreads) {
            const int cl = o / ohw, op = o % ohw, py = op / st.out_w, px = op % st.out_w;
            float best = -INFINITY;
            int bpos = 0;
            for (int r = 0; r < k; ++r)
                for (int s = 0; s < k; ++s) {
                    const int y = py * st.pool_stride + r - st.pool_pad, x = px * st.pool_stride + s - st.pool_pad;
                    if (y < 0 || y >= st.oh || x < 0 || x >= st.ow) continue;
                    float v = act(cl * hw + y * st.ow + x);
                    if (st.relu) v = fmaxf(v, 0.f);
                    if (v > best) { best = v; bpos = r * k + s; }
                }
            out[(size_t)c0 * ohw + o] = best;
            if (out16) out16[(size_t)op * st.co + c0 + cl] = __float2bfloat16_rn(best);
            arg[o] = (unsigned char)bpos;
        }
    } else if (st.avgpool) {
        // 4b. global average per channel: one warp per channel, fixed order
        const int lane = tid & 31, warp = tid >> 5;
        for (int cl = warp; cl < cpg; cl += kGroupThreads / 32) {
            float a = 0.f;
            for (int p = lane; p < hw; p += 32) {
                float v = act(cl * hw + p);
                if (st.relu) v = fmaxf(v, 0.f);
                a += v;
            }
            a = warp_sum(a);
            if (lane == 0) out[c0 + cl] = a / (float)hw;
        }
    }
}

// ---------------------------------------------------------------- backward
// Gradient w.r.t. the stage output element `o` for backward sample j.
__device__ __forceinline__ float gather_out_delta(const ConvStage& st, size_t oelems, size_t o, long long j) {
    float d = 0.f;
    for (int q = 0; q < st.n_dsrc; ++q) {
        const DeltaSrc& ds = st.dsrc[q];
        const float* p = ds.ptr + ((size_t)ring_slot(j, ds.slots) * ds.nparts) * oelems + o;
        for (int k = 0; k < ds.nparts; ++k) d += p[(size_t)k * oelems];
    }
    return d;
}

__global__ void __launch_bounds__(kGroupThreads)
conv_post_bwd_kernel(const ConvStage* __restrict__ stages, const int2* __restrict__ map,
                     const TickState* __restrict__ ts, int S, int par) {
    __shared__ GroupShared sh;
    const ConvStage& st = stages[map[blockIdx.x].x];
    const int grp = map[blockIdx.x].y;
    const long long j = ts->cnt[par] - 2LL * (S - 1) + st.s;
    if (j < 0) return;
    const int slot = ring_slot(j, st.slots);
    const int hw = st.oh * st.ow, cpg = st.cpg, n = cpg * hw, c0 = grp * cpg;
    const size_t zelems = (size_t)st.co * hw;
    const size_t oelems = (size_t)st.co * st.out_h * st.out_w;
    const float* __restrict__ z = st.z_ring + (size_t)slot * zelems + (size_t)c0 * hw;
    const unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems + (size_t)c0 * hw;
    const float mean = st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0];
    const float rstd = st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1];
    float* __restrict__ dz = st.dz + (size_t)c0 * hw;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ohw = st.out_h * st.out_w;
    const unsigned char* __restrict__ arg = st.pool_k > 0 ? st.arg_ring + (size_t)slot * oelems + (size_t)c0 * ohw : nullptr;

    // 1. gradient w.r.t. the normalised activation and per-channel sums.  All warps
    //    stay busy: a channel is shared by `wpc` warps when there are fewer channels
    //    than warps; their partial sums are combined in a fixed order.
    constexpr int kWarps = kGroupThreads / 32;
    const int wpc = cpg < kWarps ? kWarps / cpg : 1;
    const int cpp = kWarps / wpc;                        // channels per pass
    for (int base = 0; base < cpg; base += cpp) {
        const int cl = base + warp / wpc, sub = warp % wpc;
        float a1 = 0.f, a2 = 0.f;
        if (cl < cpg && warp < cpp * wpc) {
            const int c = c0 + cl;
            const float davg = st.avgpool ? gather_out_delta(st, oelems, c, j) / (float)hw : 0.f;
            for (int p = sub * 32 + lane; p < hw; p += 32 * wpc) {
                const int e = cl * hw + p;
                float d;
                if (st.avgpool) {
                    d = davg;
                } else if (st.pool_k > 0) {
                    // every pooling window that contains this element and chose it
                    const int y = p / st.ow, x = p % st.ow, k = st.pool_k, ps = st.pool_stride, pp = st.pool_pad;
                    d = 0.f;
                    for (int r = 0; r < k; ++r) {
                        const int ty = y + pp - r;
                        if (ty < 0 || ty % ps) continue;
                        const int py = ty / ps;
                        if (py >= st.out_h) continue;
                        for (int s = 0; s < k; ++s) {
                            const int tx = x + pp - s;
                            if (tx < 0 || tx % ps) continue;
                            const int px = tx / ps;
                            if (px >= st.out_w) continue;
                            const int o = cl * ohw + py * st.out_w + px;
                            if (arg[o] == r * k + s) d += gather_out_delta(st, oelems, (size_t)c0 * ohw + o, j);
                        }
                    }
                } else {
                    d = gather_out_delta(st, oelems, (size_t)c0 * hw + e, j);
                }
                d = code[e] ? d : 0.f;
                dz[e] = d;
                a1 += d;
                a2 = fmaf(d, (z[e] - mean) * rstd, a2);
            }
        }
        a1 = warp_sum(a1);
        a2 = warp_sum(a2);
        if (lane == 0) { sh.wp1[warp] = a1; sh.wp2[warp] = a2; }
        __syncthreads();
        if (tid < cpp && base + tid < cpg) {
            float t1 = 0.f, t2 = 0.f;
            for (int q = 0; q < wpc; ++q) { t1 += sh.wp1[tid * wpc + q]; t2 += sh.wp2[tid * wpc + q]; }
            sh.s1[base + tid] = t1;
            sh.s2[base + tid] = t2;
        }
        __syncthreads();
    }
    // 2. gradients of scale and shift; group means with the CURRENT scale
    const float* __restrict__ gam = st.w + st.nw;
    if (tid < cpg) {
        st.g[st.nw + c0 + tid] = sh.s2[tid];
        st.g[st.nw + st.co + c0 + tid] = sh.s1[tid];
    }
    if (tid == 0) {
        float m1 = 0.f, m2 = 0.f;
        for (int cl = 0; cl < cpg; ++cl) { m1 = fmaf(gam[c0 + cl], sh.s1[cl], m1); m2 = fmaf(gam[c0 + cl], sh.s2[cl], m2); }
        sh.bc[0] = m1 / (float)n;
        sh.bc[1] = m2 / (float)n;
    }
    __syncthreads();
    const float m1 = sh.bc[0], m2 = sh.bc[1];
    // 3. skip gradient (taken before normalisation) and gradient w.r.t. the conv output
    if (st.dskip) {
        float* __restrict__ dsk = st.dskip + (size_t)ring_slot(j, st.dskip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w);
        if (st.skip_mode == 0) {
            for (int e = tid; e < n; e += kGroupThreads) dsk[(size_t)c0 * hw + e] = dz[e];
        } else {
            const int shw = st.skip_h * st.skip_w;
            for (int cl = 0; cl < cpg; ++cl) {
                const int c = c0 + cl;
                if (c >= st.skip_c) break;
                for (int p = tid; p < shw; p += kGroupThreads) {
                    const int y = p / st.skip_w, x = p % st.skip_w;
                    dsk[(size_t)c * shw + p] = ((y | x) & 1) ? 0.f : dz[cl * hw + (y >> 1) * st.ow + (x >> 1)];
                }
            }
        }
        __syncthreads();
    }
    for (int e = tid; e < n; e += kGroupThreads) {
        const int c = c0 + e / hw;
        const float zh = (z[e] - mean) * rstd;
        const float d = rstd * (fmaf(dz[e], gam[c], -m1) - zh * m2);
        dz[e] = d;
        if (st.dz16) st.dz16[(size_t)(e % hw) * st.co + c] = __float2bfloat16_rn(d);
    }
}

// ---------------------------------------------------------------- update
// Fused SC + LWP step for materialised gradients (convolution stages):
// reads w, v and the gradient slices once, writes w, v and the predicted
// weights the next forward will use.
__global__ void __launch_bounds__(256)
update_kernel(const UpdRange* __restrict__ ranges, const UpdChunk* __restrict__ chunks,
              const TickState* __restrict__ ts, int S, int par) {
    const UpdChunk ch = chunks[blockIdx.x];
    const UpdRange& R = ranges[ch.range];
    const long long j = ts->cnt[par] - 2LL * (S - 1) + R.s;
    if (j < 0) return;
    const int end = min(R.n, ch.start + kUpdChunk);
    for (int e = ch.start + threadIdx.x; e < end; e += 256) {
        float g = 0.f;
        for (int q = 0; q < R.nparts; ++q) g += R.g[(size_t)q * R.part_stride + e];
        const float w = R.w[e], v = R.v[e];
        const float vn = fmaf(R.m, v, g);
        const float wn = fmaf(R.neg_lr_a, vn, fmaf(R.neg_lr_b, g, w));
        const float wh = fmaf(R.neg_lr_T, vn, wn);
        R.v[e] = vn;
        R.w[e] = wn;
        R.wh[e] = wh;
        if (R.w16) { R.w16[e] = __float2bfloat16_rn(wn); R.wh16[e] = __float2bfloat16_rn(wh); }
    }
}

// bfloat16 copies of freshly loaded weights (w_hat = w while the velocity is zero)
__global__ void __launch_bounds__(256)
cast_weights_kernel(const UpdRange* __restrict__ ranges, const UpdChunk* __restrict__ chunks) {
    const UpdChunk ch = chunks[blockIdx.x];
    const UpdRange& R = ranges[ch.range];
    if (!R.w16) return;
    const int end = min(R.n, ch.start + kUpdChunk);
    for (int e = ch.start + threadIdx.x; e < end; e += 256) {
        const __nv_bfloat16 b = __float2bfloat16_rn(R.w[e]);
        R.w16[e] = b;
        R.wh16[e] = b;
    }
}

}  // namespace pb
