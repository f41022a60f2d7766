// Per-stage normalisation / activation / pooling kernels and the fused update.
//
// A convolution stage is  conv -> GroupNorm -> (+skip) -> ReLU -> (max-pool |
// global average pool).  The elements of a normalisation group are cut into
// chunks of at most kPostChunk elements that are contiguous in memory (whole
// channels when the image is small, a piece of one channel when it is large)
// and ONE BLOCK owns a chunk: every thread holds kPostPer elements, all its
// loads are issued before anything is used, and a resident SM keeps six to eight
// such blocks in flight.  Whatever needs the whole group goes through small
// partial tables that are combined in a fixed order.  Both directions are ONE launch:
// the groups of a stage are bundled (whole groups, at least 8 channels where bfloat16
// copies are written); every block does the first step for its chunk, then counts
// itself in at the bundle's counter, and the block that arrives last - by then all
// partials of the bundle are in memory - merges them and does the second step for the
// bundle's tiles.  Nobody waits for anybody, and the merge order is the table's, not
// the arrival order, so results do not depend on scheduling.
//   forward  (conv_fwd_post_kernel): conv_stats_chunk (sum the K-slices, keep z, chunk
//             mean / M2) -> group_merge_fwd (group mean and 1/std) -> conv_apply_fwd_chunk
//             (normalise, skip, ReLU, pool)
//   backward (conv_bwd_post_kernel): conv_bwd_dn_chunk (gradient at the normalised
//             activation, channel sums per chunk) -> group_merge_bwd (scale/shift
//             gradients, group means) -> conv_bwd_dz_chunk (gradient at the conv output)
#pragma once
#include "conv_types.h"
#include "fc_kernels.cuh"   // ring_slot, warp_sum

namespace pb {

constexpr float kGnEps = 1e-5f;
constexpr int kPostPer = kPostChunk / kPostThreads;       // elements per thread
constexpr int kPostWarps = kPostThreads / 32;

__device__ __forceinline__ float skip_value(const ConvStage& st, const float* __restrict__ sk, int c, int y, int x) {
    if (st.skip_mode == 0) return sk[((size_t)c * st.skip_h + y) * st.skip_w + x];
    return c < st.skip_c ? sk[((size_t)c * st.skip_h + 2 * y) * st.skip_w + 2 * x] : 0.f;
}

__device__ __forceinline__ int slot_of(long long sample, int slots) { return (int)((unsigned)sample % (unsigned)slots); }

// Loads of data that OTHER blocks of the same launch have written (read by the block
// that closes a bundle): served by the L2 cache, never by a non-coherent path.
template <int VEC> __device__ __forceinline__ void vload_cg(float (&r)[VEC], const float* p);
template <> __device__ __forceinline__ void vload_cg<4>(float (&r)[4], const float* p) {
    const float4 q = __ldcg(reinterpret_cast<const float4*>(p));
    r[0] = q.x; r[1] = q.y; r[2] = q.z; r[3] = q.w;
}
template <> __device__ __forceinline__ void vload_cg<1>(float (&r)[1], const float* p) { r[0] = __ldcg(p); }

template <int VEC> __device__ __forceinline__ void ldb(unsigned char (&r)[VEC], const unsigned char* p);
template <> __device__ __forceinline__ void ldb<4>(unsigned char (&r)[4], const unsigned char* p) {
    const uchar4 q = *reinterpret_cast<const uchar4*>(p); r[0] = q.x; r[1] = q.y; r[2] = q.z; r[3] = q.w;
}
template <> __device__ __forceinline__ void ldb<1>(unsigned char (&r)[1], const unsigned char* p) { r[0] = *p; }
template <int VEC> __device__ __forceinline__ void stb(unsigned char* p, const unsigned char (&r)[VEC]);
template <> __device__ __forceinline__ void stb<4>(unsigned char* p, const unsigned char (&r)[4]) {
    *reinterpret_cast<uchar4*>(p) = make_uchar4(r[0], r[1], r[2], r[3]);
}
template <> __device__ __forceinline__ void stb<1>(unsigned char* p, const unsigned char (&r)[1]) { *p = r[0]; }

// Sum over the block, returned to every thread (two barriers; `red` holds kPostWarps floats).
__device__ __forceinline__ float block_sum(float x, float* red) {
    x = warp_sum(x);
    __syncthreads();                       // `red` may still be read from the previous call
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    float a = 0.f;
#pragma unroll
    for (int k = 0; k < kPostWarps; ++k) a += red[k];
    return a;
}

// A chunk is the contiguous range [base, base + n) of the stage's [channel][pixel] tensor:
// unit q (VEC consecutive pixels of one channel) of thread `tid` is unit u*kPostThreads + tid.
struct ChunkGeom {
    int hw, n, nunits, base, c_first;
    __device__ __forceinline__ ChunkGeom(const ConvStage& st, const PostChunk& ch, int vec) {
        hw = st.oh * st.ow;
        n = ch.ncl * ch.np;
        nunits = n / vec;
        c_first = ch.grp * st.cpg + ch.cl0;
        base = c_first * hw + ch.p0;
    }
};

// ---------------------------------------------------------------- forward, step 1
template <int VEC>
__device__ void conv_stats_chunk(const ConvStage& st, const PostChunk& ch, long long t, const TickState* ts, float* red) {
    constexpr int U = kPostPer / VEC;
    const long long i = t - st.s;
    if (!sample_live(ts, i)) return;
    const int tid = threadIdx.x;
    const int slot = slot_of(i, st.slots);
    const ChunkGeom cg(st, ch, VEC);
    const size_t zelems = (size_t)st.co * cg.hw;
    float* __restrict__ z = st.z_ring + (size_t)slot * zelems + cg.base;
    const float* __restrict__ zp = st.zpart + cg.base;
    float vals[U][VEC];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int e = 0; e < VEC; ++e) vals[u][e] = 0.f;
    // the K-slice loop is outside so that each step issues U independent loads
    for (int q = 0; q < st.z_nsplit; ++q) {
        const float* __restrict__ zq = zp + (size_t)q * zelems;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int unit = u * kPostThreads + tid;
            if (unit < cg.nunits) {
                float r[VEC];
                vload<VEC>(r, zq + unit * VEC);
#pragma unroll
                for (int e = 0; e < VEC; ++e) vals[u][e] += r[e];
            }
        }
    }
    if (st.skip_ring && st.skip_pre) {
        // pre-activation network: the source stage's running sum (its own conv output after such an
        // addition, same sample) joins before the statistics are taken
        const float* __restrict__ sk = st.skip_ring + (size_t)slot_of(i, st.skip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int unit = u * kPostThreads + tid;
            if (unit >= cg.nunits) continue;
            const int flat = cg.base + unit * VEC;              // index in this stage's [channel][pixel] tensor
            if (st.skip_mode == 0) {
                float r[VEC];
                vload<VEC>(r, sk + flat);
#pragma unroll
                for (int e = 0; e < VEC; ++e) vals[u][e] += r[e];
            } else {
                const int c = flat / cg.hw, p = flat - c * cg.hw;
#pragma unroll
                for (int e = 0; e < VEC; ++e) vals[u][e] += skip_value(st, sk, c, (p + e) / st.ow, (p + e) % st.ow);
            }
        }
    }
    float sum = 0.f;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int unit = u * kPostThreads + tid;
        if (unit < cg.nunits) {
            vstore<VEC>(z + unit * VEC, vals[u]);
#pragma unroll
            for (int e = 0; e < VEC; ++e) sum += vals[u][e];
        }
    }
    const float mean = block_sum(sum, red) / (float)cg.n;
    float sq = 0.f;
#pragma unroll
    for (int u = 0; u < U; ++u)
        if (u * kPostThreads + tid < cg.nunits) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) { const float d = vals[u][e] - mean; sq = fmaf(d, d, sq); }
        }
    const float m2 = block_sum(sq, red);
    if (tid == 0) {
        float* f = st.fstat + ((size_t)ch.grp * st.fstat_stride + ch.idx) * 3;
        f[0] = (float)cg.n; f[1] = mean; f[2] = m2;
    }
}

// ---------------------------------------------------------------- forward, step 2
// Elementwise over a TILE: channels [cl0, cl0+ncl) (absolute) x pixels [p0, p0+np).  Plain
// stages are tiled as (a multiple of 8 channels) x (up to 128 pixels), so that the bfloat16
// [pixel][channel] copy can be written as whole 16-byte runs of 8 channels after a transpose
// through shared memory; stages that pool keep their group chunks as tiles.
__device__ __forceinline__ void store_nhwc_tile(const __nv_bfloat16* t16, int rs, const PostChunk& ch, int co,
                                                __nv_bfloat16* __restrict__ dst) {
    const int ng = ch.ncl >> 3;
    for (int idx = threadIdx.x; idx < ch.np * ng; idx += kPostThreads) {
        const int pix = idx / ng, cgp = idx - pix * ng;
        const unsigned short* src = reinterpret_cast<const unsigned short*>(t16) + (size_t)(cgp * 8) * rs + pix;
        uint4 v;
        v.x = src[0] | ((unsigned)src[rs] << 16);
        v.y = src[2 * rs] | ((unsigned)src[3 * rs] << 16);
        v.z = src[4 * rs] | ((unsigned)src[5 * rs] << 16);
        v.w = src[6 * rs] | ((unsigned)src[7 * rs] << 16);
        *reinterpret_cast<uint4*>(dst + (size_t)(ch.p0 + pix) * co + ch.cl0 + cgp * 8) = v;
    }
}

// CG: the tile's inputs were written by other blocks of the SAME launch (the caller is the
// block that closes a bundle): they are then loaded through the L2 cache.
template <int VEC, bool CG>
__device__ void conv_apply_fwd_chunk(const ConvStage& st, const PostChunk& ch, long long t, const TickState* ts, __nv_bfloat16* t16) {
    constexpr int U = kPostPer / VEC;
    const long long i = t - st.s;
    if (!sample_live(ts, i)) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slot = slot_of(i, st.slots);
    const int hw = st.oh * st.ow, npu = ch.np / VEC, nunits = ch.ncl * npu, rs = ch.np + 2;
    const size_t zelems = (size_t)st.co * hw;
    const float* z = st.z_ring + (size_t)slot * zelems;
    const float* __restrict__ gam = st.wh + st.nw;
    const float* __restrict__ bet = gam + st.co;
    const float* stat = st.stat_ring + (size_t)slot * st.groups * 2;     // may have been written by this very block
    const float* __restrict__ sk = (st.skip_ring && !st.skip_pre)      // (a pre-normalisation skip is already part of z)
        ? st.skip_ring + (size_t)slot_of(i, st.skip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w) : nullptr;
    unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems;
    const bool pooled = st.pool_k > 0 || st.avgpool;
    const size_t oelems = (size_t)st.co * st.out_h * st.out_w;
    float* __restrict__ out = st.out_ring + (size_t)slot * oelems;
    __nv_bfloat16* __restrict__ out16 = st.out16 ? st.out16 + (size_t)slot * oelems : nullptr;
    const bool transposed = out16 && !pooled && (ch.ncl & 7) == 0 && ch.ncl <= kPostTileChannels && (ch.cl0 & 7) == 0 && (st.co & 7) == 0;
    // all loads of the thread's units first
    int cc[U], pp[U];
    bool ok[U];
    float zv[U][VEC], sv[U][VEC], gs[U], bb[U], mean[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int unit = u * kPostThreads + tid;
        ok[u] = unit < nunits;
        const int uu = ok[u] ? unit : 0;
        const int cl = uu / npu;
        cc[u] = ch.cl0 + cl;
        pp[u] = ch.p0 + (uu - cl * npu) * VEC;
        const size_t idx = (size_t)cc[u] * hw + pp[u];
        const int grp = cc[u] / st.cpg;
        if (CG) vload_cg<VEC>(zv[u], z + idx); else vload<VEC>(zv[u], z + idx);
        mean[u] = stat[2 * grp];
        gs[u] = gam[cc[u]] * stat[2 * grp + 1];
        bb[u] = bet[cc[u]];
        if (!sk) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) sv[u][e] = 0.f;
        } else if (st.skip_mode == 0) {
            vload<VEC>(sv[u], sk + idx);            // identity skips share this stage's indexing
        } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e) sv[u][e] = skip_value(st, sk, cc[u], (pp[u] + e) / st.ow, (pp[u] + e) % st.ow);
        }
    }
    auto act = [&](int c, int p) -> float {
        const int grp = c / st.cpg;
        const float zc = CG ? __ldcg(z + (size_t)c * hw + p) : z[(size_t)c * hw + p];
        float v = fmaf(gam[c] * stat[2 * grp + 1], zc - stat[2 * grp], bet[c]);
        if (sk) v += skip_value(st, sk, c, p / st.ow, p % st.ow);
        return v;
    };
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!ok[u]) continue;
        const int c = cc[u], p = pp[u];
        float a[VEC];
        unsigned char cd[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const float v = fmaf(gs[u], zv[u][e] - mean[u], bb[u]) + sv[u][e];
            const bool pass = st.relu ? v > 0.f : true;
            cd[e] = pass ? 1 : 0;
            a[e] = pass ? v : 0.f;
        }
        stb<VEC>(code + (size_t)c * hw + p, cd);
        if (!pooled) {
            vstore<VEC>(out + (size_t)c * hw + p, a);
            if (transposed) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) t16[(c - ch.cl0) * rs + (p - ch.p0) + e] = __float2bfloat16_rn(a[e]);
            } else if (out16) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) out16[(size_t)(p + e) * st.co + c] = __float2bfloat16_rn(a[e]);
            }
        }
    }
    if (transposed) {
        __syncthreads();
        store_nhwc_tile(t16, rs, ch, st.co, out16);
    }
    if (st.pool_k > 0) {
        // max-pool: this tile owns the pooled pixels [p0*ohw/hw, (p0+np)*ohw/hw) of its channels;
        // first maximum in row-major window order, padding never wins
        const int ohw = st.out_h * st.out_w, k = st.pool_k;
        const int o0 = (int)((long long)ch.p0 * ohw / hw), o1 = (int)((long long)(ch.p0 + ch.np) * ohw / hw);
        const int no = o1 - o0;
        unsigned char* __restrict__ arg = st.arg_ring + (size_t)slot * oelems;
        for (int e = tid; e < ch.ncl * no; e += kPostThreads) {
            const int c = ch.cl0 + e / no, op = o0 + e % no, py = op / st.out_w, px = op % st.out_w;
            float best = -INFINITY;
            int bpos = 0;
            for (int r = 0; r < k; ++r)
                for (int s = 0; s < k; ++s) {
                    const int y = py * st.pool_stride + r - st.pool_pad, x = px * st.pool_stride + s - st.pool_pad;
                    if (y < 0 || y >= st.oh || x < 0 || x >= st.ow) continue;
                    float v = act(c, y * st.ow + x);
                    if (st.relu) v = fmaxf(v, 0.f);
                    if (v > best) { best = v; bpos = r * k + s; }
                }
            out[(size_t)c * ohw + op] = best;
            if (out16) out16[(size_t)op * st.co + c] = __float2bfloat16_rn(best);
            arg[(size_t)c * ohw + op] = (unsigned char)bpos;
        }
    } else if (st.avgpool) {
        // global average per channel (tiles of such stages hold whole channels): a warp per channel
        for (int cl = warp; cl < ch.ncl; cl += kPostWarps) {
            const int c = ch.cl0 + cl;
            float a = 0.f;
            for (int p = lane; p < hw; p += 32) {
                float v = act(c, p);
                if (st.relu) v = fmaxf(v, 0.f);
                a += v;
            }
            a = warp_sum(a);
            if (lane == 0) out[c] = a / (float)hw;
        }
    }
}

// ---------------------------------------------------------------- backward, step 1
// Gradient w.r.t. the stage output element `o` for backward sample j.
__device__ __forceinline__ float gather_out_delta(const ConvStage& st, size_t oelems, size_t o, long long j) {
    float d = 0.f;
    for (int q = 0; q < st.n_dsrc; ++q) {
        const DeltaSrc& ds = st.dsrc[q];
        const float* p = ds.ptr + ((size_t)slot_of(j, ds.slots) * ds.nparts) * oelems + o;
        for (int k = 0; k < ds.nparts; ++k) d += p[(size_t)k * oelems];
    }
    return d;
}

template <int VEC>
__device__ void conv_bwd_dn_chunk(const ConvStage& st, const PostChunk& ch, long long t, const TickState* ts, int S, float* red, float* usum) {
    constexpr int U = kPostPer / VEC;
    const long long j = t - 2LL * (S - 1) + st.s;
    if (!sample_live(ts, j)) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slot = slot_of(j, st.slots);
    const ChunkGeom cg(st, ch, VEC);
    const int hw = cg.hw, npu = ch.np / VEC;
    const size_t zelems = (size_t)st.co * hw;
    const size_t oelems = (size_t)st.co * st.out_h * st.out_w;
    const float* __restrict__ z = st.z_ring + (size_t)slot * zelems + cg.base;
    const unsigned char* __restrict__ code = st.code_ring + (size_t)slot * zelems + cg.base;
    const float mean = st.stat_ring[((size_t)slot * st.groups + ch.grp) * 2 + 0];
    const float rstd = st.stat_ring[((size_t)slot * st.groups + ch.grp) * 2 + 1];
    float* __restrict__ dz = st.dz + cg.base;
    const int ohw = st.out_h * st.out_w;
    bool ok[U];
    float d[U][VEC], zv[U][VEC];
    unsigned char cd[U][VEC];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int unit = u * kPostThreads + tid;
        ok[u] = unit < cg.nunits;
#pragma unroll
        for (int e = 0; e < VEC; ++e) { d[u][e] = 0.f; zv[u][e] = 0.f; cd[u][e] = 0; }
        if (ok[u]) {
            vload<VEC>(zv[u], z + unit * VEC);
            ldb<VEC>(cd[u], code + unit * VEC);
        }
    }
    if (!st.avgpool && st.pool_k == 0) {
        // plain stage: the consumers' partial rows line up with this stage's elements
        for (int q = 0; q < st.n_dsrc; ++q) {
            const float* bp = st.dsrc[q].ptr + (size_t)slot_of(j, st.dsrc[q].slots) * st.dsrc[q].nparts * oelems + cg.base;
            const int np_ = st.dsrc[q].nparts;
            for (int kp = 0; kp < np_; ++kp, bp += oelems) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (!ok[u]) continue;
                    float r[VEC];
                    vload<VEC>(r, bp + (u * kPostThreads + tid) * VEC);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) d[u][e] += r[e];
                }
            }
        }
    } else if (st.avgpool) {
        // every pixel of a channel receives the same value: a warp gathers it once per
        // channel (lanes over the consumers' partial rows) and hands it on through shared memory
        __syncthreads();
        for (int cl = warp; cl < ch.ncl; cl += kPostWarps) {
            float a = 0.f;
            for (int q = 0; q < st.n_dsrc; ++q) {
                const DeltaSrc& ds = st.dsrc[q];
                const float* p = ds.ptr + ((size_t)slot_of(j, ds.slots) * ds.nparts) * oelems + cg.c_first + cl;
                for (int k = lane; k < ds.nparts; k += 32) a += p[(size_t)k * oelems];
            }
            a = warp_sum(a);
            if (lane == 0) usum[cl] = a / (float)hw;
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!ok[u]) continue;
            const float a = usum[(u * kPostThreads + tid) / npu];
#pragma unroll
            for (int e = 0; e < VEC; ++e) d[u][e] = a;
        }
    } else {
        // max-pool: every window that contains the element and chose it
        const unsigned char* __restrict__ arg = st.arg_ring + (size_t)slot * oelems;
        const int kk = st.pool_k, ps = st.pool_stride, pp = st.pool_pad;
#pragma unroll 1
        for (int u = 0; u < U; ++u) {
            if (!ok[u]) continue;
            const int unit = u * kPostThreads + tid, cl = unit / npu;
            const int c = cg.c_first + cl, p0 = ch.p0 + (unit - cl * npu) * VEC;
#pragma unroll 1
            for (int e = 0; e < VEC; ++e) {
                const int p = p0 + e;
                const int y = p / st.ow, x = p % st.ow;
                float a = 0.f;
                // only window offsets congruent to the element's position modulo the stride can hold it
                for (int r = (y + pp) % ps; r < kk; r += ps) {
                    const int ty = y + pp - r;
                    if (ty < 0) break;
                    const int py = ty / ps;
                    if (py >= st.out_h) continue;
                    for (int s = (x + pp) % ps; s < kk; s += ps) {
                        const int tx = x + pp - s;
                        if (tx < 0) break;
                        const int px = tx / ps;
                        if (px >= st.out_w) continue;
                        const size_t o = (size_t)c * ohw + py * st.out_w + px;
                        if (arg[o] == r * kk + s) a += gather_out_delta(st, oelems, o, j);
                    }
                }
                d[u][e] = a;
            }
        }
    }
    float s1[U], s2[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        s1[u] = 0.f; s2[u] = 0.f;
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            d[u][e] = (ok[u] && cd[u][e]) ? d[u][e] : 0.f;
            s1[u] += d[u][e];
            s2[u] = fmaf(d[u][e], (zv[u][e] - mean) * rstd, s2[u]);      // d * zhat
        }
        if (ok[u]) vstore<VEC>(dz + (u * kPostThreads + tid) * VEC, d[u]);
    }
    // per-channel sums of d and d*zhat over this chunk's pixels
    const int piece = ch.p0 / kPostChunk;
    if (ch.ncl == 1) {
        float a1 = 0.f, a2 = 0.f;
#pragma unroll
        for (int u = 0; u < U; ++u) { a1 += s1[u]; a2 += s2[u]; }
        a1 = block_sum(a1, red);
        a2 = block_sum(a2, red);
        if (tid == 0) {
            float* b = st.bsum + ((size_t)cg.c_first * st.npieces + piece) * 2;
            b[0] = a1; b[1] = a2;
        }
    } else {
        // several whole channels: unit sums go through shared memory, then a warp per channel
        __syncthreads();
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int unit = u * kPostThreads + tid;
            if (unit < cg.nunits) { usum[2 * unit] = s1[u]; usum[2 * unit + 1] = s2[u]; }
        }
        __syncthreads();
        for (int cl = warp; cl < ch.ncl; cl += kPostWarps) {
            float a1 = 0.f, a2 = 0.f;
            for (int q = lane; q < npu; q += 32) { a1 += usum[2 * (cl * npu + q)]; a2 += usum[2 * (cl * npu + q) + 1]; }
            a1 = warp_sum(a1);
            a2 = warp_sum(a2);
            if (lane == 0) {
                float* b = st.bsum + ((size_t)(cg.c_first + cl) * st.npieces + piece) * 2;
                b[0] = a1; b[1] = a2;
            }
        }
    }
}

// ---------------------------------------------------------------- backward, step 2
// Elementwise over a tile (see the forward step 2).
template <int VEC, bool CG>
__device__ void conv_bwd_dz_chunk(const ConvStage& st, const PostChunk& ch, long long t, const TickState* ts, int S, __nv_bfloat16* t16) {
    constexpr int U = kPostPer / VEC;
    const long long j = t - 2LL * (S - 1) + st.s;
    if (!sample_live(ts, j)) return;
    const int tid = threadIdx.x;
    const int slot = slot_of(j, st.slots);
    const int hw = st.oh * st.ow, npu = ch.np / VEC, nunits = ch.ncl * npu, rs = ch.np + 2;
    const size_t zelems = (size_t)st.co * hw;
    const float* __restrict__ z = st.z_ring + (size_t)slot * zelems;
    const float* __restrict__ stat = st.stat_ring + (size_t)slot * st.groups * 2;
    // the CURRENT scale (with weight stashing: the one the sample's forward used)
    const float* __restrict__ gam = st.gstash ? st.gstash + (size_t)slot_of(j, st.gstash_slots) * st.co : st.w + st.nw;
    float* __restrict__ dz = st.dz;
    const bool transposed = st.dz16 && (ch.ncl & 7) == 0 && ch.ncl <= kPostTileChannels && (ch.cl0 & 7) == 0 && (st.co & 7) == 0;
    int cc[U], pp[U];
    bool ok[U];
    float dnv[U][VEC], zv[U][VEC], gv[U], mean[U], rstd[U], m1[U], m2[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {                     // all loads of the thread's units first
        const int unit = u * kPostThreads + tid;
        ok[u] = unit < nunits;
        const int uu = ok[u] ? unit : 0;
        const int cl = uu / npu;
        cc[u] = ch.cl0 + cl;
        pp[u] = ch.p0 + (uu - cl * npu) * VEC;
        const size_t idx = (size_t)cc[u] * hw + pp[u];
        const int grp = cc[u] / st.cpg;
        if (CG) vload_cg<VEC>(dnv[u], dz + idx); else vload<VEC>(dnv[u], dz + idx);
        vload<VEC>(zv[u], z + idx);
        gv[u] = gam[cc[u]];
        mean[u] = stat[2 * grp]; rstd[u] = stat[2 * grp + 1];
        m1[u] = st.gsum[2 * grp]; m2[u] = st.gsum[2 * grp + 1];
    }
    float* __restrict__ dsk = st.dskip
        ? st.dskip + (size_t)slot_of(j, st.dskip_slots) * ((size_t)st.skip_c * st.skip_h * st.skip_w) : nullptr;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!ok[u]) continue;
        const int c = cc[u], p = pp[u];
        const size_t idx = (size_t)c * hw + p;
        float dd[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const float zh = (zv[u][e] - mean[u]) * rstd[u];
            dd[e] = rstd[u] * (fmaf(dnv[u][e], gv[u], -m1[u]) - zh * m2[u]);
        }
        // later stages that added this stage's pre-normalisation sum to theirs send their gradient straight here
        for (int q = 0; q < st.n_rsrc; ++q) {
            float r[VEC];
            vload<VEC>(r, st.rsrc[q].ptr + (size_t)slot_of(j, st.rsrc[q].slots) * zelems + idx);
#pragma unroll
            for (int e = 0; e < VEC; ++e) dd[e] += r[e];
        }
        // a skip input that joined after the normalisation receives dn itself, one that joined before it dz
        if (dsk) {
            const float* src = st.skip_pre ? dd : dnv[u];
            if (st.skip_mode == 0) {
                float tmp[VEC];
#pragma unroll
                for (int e = 0; e < VEC; ++e) tmp[e] = src[e];
                vstore<VEC>(dsk + idx, tmp);
            } else if (c < st.skip_c) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    const int y = (p + e) / st.ow, x = (p + e) % st.ow;
                    for (int dy = 0; dy < 2; ++dy)
                        for (int dx = 0; dx < 2; ++dx) {
                            const int ys = 2 * y + dy, xs = 2 * x + dx;
                            if (ys < st.skip_h && xs < st.skip_w)
                                dsk[((size_t)c * st.skip_h + ys) * st.skip_w + xs] = (dy | dx) ? 0.f : src[e];
                        }
                }
            }
        }
        vstore<VEC>(dz + idx, dd);
        if (transposed) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) t16[(c - ch.cl0) * rs + (p - ch.p0) + e] = __float2bfloat16_rn(dd[e]);
        } else if (st.dz16) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) st.dz16[(size_t)(p + e) * st.co + c] = __float2bfloat16_rn(dd[e]);
        }
    }
    if (transposed) {
        __syncthreads();
        store_nhwc_tile(t16, rs, ch, st.co, st.dz16);
    }
}

// ---------------------------------------------------------------- group merges
// forward: chunk statistics (count, mean, M2) -> group mean and 1/std, kept for the backward.
__device__ __forceinline__ void group_merge_fwd(const ConvStage& st, int grp, long long t, int lane) {
    const int slot = slot_of(t - st.s, st.slots), nidx = st.fstat_stride;
    const float* f = st.fstat + (size_t)grp * st.fstat_stride * 3;
    float tot = 0.f, wsum = 0.f;
    for (int k = lane; k < nidx; k += 32) { const float n = __ldcg(f + 3 * k); tot += n; wsum = fmaf(n, __ldcg(f + 3 * k + 1), wsum); }
    tot = warp_sum(tot);
    const float mean = warp_sum(wsum) / tot;
    float m2 = 0.f;
    for (int k = lane; k < nidx; k += 32) { const float d = __ldcg(f + 3 * k + 1) - mean; m2 += __ldcg(f + 3 * k + 2) + __ldcg(f + 3 * k) * d * d; }
    const float rstd = rsqrtf(warp_sum(m2) / tot + kGnEps);
    if (lane == 0) {
        st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 0] = mean;
        st.stat_ring[((size_t)slot * st.groups + grp) * 2 + 1] = rstd;
    }
}

// backward: per-chunk channel sums -> gradients of scale and shift, and the two group
// means the gradient at the conv output needs (with the CURRENT scale).
__device__ __forceinline__ void group_merge_bwd(const ConvStage& st, int grp, int lane, long long j) {
    const int hw = st.oh * st.ow, cpg = st.cpg, c0 = grp * cpg;
    const float* __restrict__ gam = st.gstash ? st.gstash + (size_t)slot_of(j, st.gstash_slots) * st.co : st.w + st.nw;
    const int np = st.npieces;
    float m1 = 0.f, m2 = 0.f;
    if (np >= 8) {
        // few channels, many pieces: lanes over the pieces of one channel at a time
        for (int cl = 0; cl < cpg; ++cl) {
            const float* b = st.bsum + (size_t)(c0 + cl) * np * 2;
            float t1 = 0.f, t2 = 0.f;
            for (int q = lane; q < np; q += 32) { t1 += __ldcg(b + 2 * q); t2 += __ldcg(b + 2 * q + 1); }
            t1 = warp_sum(t1); t2 = warp_sum(t2);
            if (lane == 0) {
                st.g[st.nw + c0 + cl] = t2;
                st.g[st.nw + st.co + c0 + cl] = t1;
            }
            m1 = fmaf(gam[c0 + cl], t1, m1);
            m2 = fmaf(gam[c0 + cl], t2, m2);
        }
    } else {
        for (int cl = lane; cl < cpg; cl += 32) {
            const float* b = st.bsum + (size_t)(c0 + cl) * np * 2;
            float t1 = 0.f, t2 = 0.f;
            for (int q = 0; q < np; ++q) { t1 += __ldcg(b + 2 * q); t2 += __ldcg(b + 2 * q + 1); }
            st.g[st.nw + c0 + cl] = t2;
            st.g[st.nw + st.co + c0 + cl] = t1;
            m1 = fmaf(gam[c0 + cl], t1, m1);
            m2 = fmaf(gam[c0 + cl], t2, m2);
        }
        m1 = warp_sum(m1); m2 = warp_sum(m2);
    }
    if (lane == 0) {
        st.gsum[2 * grp] = m1 / (float)(cpg * hw);
        st.gsum[2 * grp + 1] = m2 / (float)(cpg * hw);
    }
}

// ---------------------------------------------------------------- the two launches
// Counts this block in at its bundle; true (for every thread) in the block that arrives
// last, which also clears the counter for the next launch.  Every thread's stores of
// the first step are fenced before the count, so the last block sees all of them.
__device__ __forceinline__ bool bundle_closed_by_me(int* counter, int nchunks, int* flag) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int old = atomicAdd(counter, 1);
        const int last = old == nchunks - 1;
        if (last) *counter = 0;
        *flag = last;
        __threadfence();
    }
    __syncthreads();
    return *flag != 0;
}

// What the closing block does: merge the bundle's groups, then its tiles of the second
// step.  Kept out of line so that its registers do not weigh on the first step, which
// every block runs.
__device__ __noinline__ void close_bundle_fwd(const ConvStage* __restrict__ stages, const PostBundle* __restrict__ bundles, int bundle,
                                              const PostChunk* __restrict__ tiles, long long t, const TickState* ts, __nv_bfloat16* t16) {
    const PostBundle bd = bundles[bundle];
    const ConvStage& st = stages[bd.stage];
    for (int g = threadIdx.x >> 5; g < bd.ngrp; g += kPostWarps) group_merge_fwd(st, bd.grp0 + g, t, threadIdx.x & 31);
    __syncthreads();
    for (int q = 0; q < bd.nftiles; ++q) {
        const PostChunk tl = tiles[bd.ftile0 + q];
        if (st.vec4) conv_apply_fwd_chunk<4, true>(st, tl, t, ts, t16);
        else conv_apply_fwd_chunk<1, true>(st, tl, t, ts, t16);
        __syncthreads();                                     // t16 is reused by the next tile
    }
}

__device__ __noinline__ void close_bundle_bwd(const ConvStage* __restrict__ stages, const PostBundle* __restrict__ bundles, int bundle,
                                              const PostChunk* __restrict__ tiles, long long t, const TickState* ts, int S, __nv_bfloat16* t16) {
    const PostBundle bd = bundles[bundle];
    const ConvStage& st = stages[bd.stage];
    for (int g = threadIdx.x >> 5; g < bd.ngrp; g += kPostWarps) group_merge_bwd(st, bd.grp0 + g, threadIdx.x & 31, t - 2LL * (S - 1) + st.s);
    __syncthreads();
    for (int q = 0; q < bd.nbtiles; ++q) {
        const PostChunk tl = tiles[bd.btile0 + q];
        if (st.vec4) conv_bwd_dz_chunk<4, true>(st, tl, t, ts, S, t16);
        else conv_bwd_dz_chunk<1, true>(st, tl, t, ts, S, t16);
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kPostThreads, 4)
conv_fwd_post_kernel(const ConvStage* __restrict__ stages, const PostChunk* __restrict__ chunks, int nchunks,
                     const PostBundle* __restrict__ bundles, const PostChunk* __restrict__ tiles, int* __restrict__ counters,
                     const TickState* __restrict__ ts, int S, int par) {
    __shared__ float red[kPostWarps];
    __shared__ __align__(16) __nv_bfloat16 t16[kPostChunk + 2 * kPostTileChannels];
    __shared__ int last_flag;
    (void)S;
    if ((int)blockIdx.x >= nchunks) return;
    const PostChunk ch = chunks[blockIdx.x];
    const long long t = ts->cnt[par];
    const ConvStage& st = stages[ch.stage];
    if (!sample_live(ts, t - st.s)) return;                 // uniform over the bundle: nobody counts in
    if (st.vec4) conv_stats_chunk<4>(st, ch, t, ts, red);
    else conv_stats_chunk<1>(st, ch, t, ts, red);
    const int bundle = chunks[blockIdx.x].bundle;
    if (bundle < 0) return;                                 // merged and finished by the launches that follow
    if (!bundle_closed_by_me(counters + bundle, bundles[bundle].nchunks, &last_flag)) return;
    close_bundle_fwd(stages, bundles, bundle, tiles, ts->cnt[par], ts, t16);
}

__global__ void __launch_bounds__(kPostThreads, 4)
conv_bwd_post_kernel(const ConvStage* __restrict__ stages, const PostChunk* __restrict__ chunks, int nchunks,
                     const PostBundle* __restrict__ bundles, const PostChunk* __restrict__ tiles, int* __restrict__ counters,
                     const TickState* __restrict__ ts, int S, int par) {
    __shared__ float red[kPostWarps];
    __shared__ __align__(16) float usum[2 * kPostChunk];
    __shared__ int last_flag;
    if ((int)blockIdx.x >= nchunks) return;
    const PostChunk ch = chunks[blockIdx.x];
    const long long t = ts->cnt[par];
    const ConvStage& st = stages[ch.stage];
    if (!sample_live(ts, t - 2LL * (S - 1) + st.s)) return;
    if (st.vec4) conv_bwd_dn_chunk<4>(st, ch, t, ts, S, red, usum);
    else conv_bwd_dn_chunk<1>(st, ch, t, ts, S, red, usum);
    const int bundle = chunks[blockIdx.x].bundle;
    if (bundle < 0) return;
    if (!bundle_closed_by_me(counters + bundle, bundles[bundle].nchunks, &last_flag)) return;
    // the transposing tile of the second step lives in the space of the first step's sums
    close_bundle_bwd(stages, bundles, bundle, tiles, ts->cnt[par], ts, S, reinterpret_cast<__nv_bfloat16*>(usum));
}

// Stages that are not fused: one warp per group merges the partials ...
__global__ void __launch_bounds__(256)
conv_group_merge_kernel(const ConvStage* __restrict__ stages, const GroupRef* __restrict__ groups, int ngroups,
                        const TickState* __restrict__ ts, int S, int par, int mode) {
    const int gi = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (gi >= ngroups) return;
    const GroupRef gr = groups[gi];
    const ConvStage& st = stages[gr.stage];
    const long long t = ts->cnt[par];
    if (mode == 0) {
        if (sample_live(ts, t - st.s)) group_merge_fwd(st, gr.grp, t, threadIdx.x & 31);
    } else {
        if (sample_live(ts, t - 2LL * (S - 1) + st.s)) group_merge_bwd(st, gr.grp, threadIdx.x & 31, t - 2LL * (S - 1) + st.s);
    }
}

// ... and the second step runs one block per tile.
__global__ void __launch_bounds__(kPostThreads, 4)
conv_apply_fwd_kernel(const ConvStage* __restrict__ stages, const PostChunk* __restrict__ tiles, int ntiles,
                      const TickState* __restrict__ ts, int S, int par) {
    __shared__ __align__(16) __nv_bfloat16 t16[kPostChunk + 2 * kPostTileChannels];
    (void)S;
    if ((int)blockIdx.x >= ntiles) return;
    const PostChunk tl = tiles[blockIdx.x];
    const long long t = ts->cnt[par];
    const ConvStage& st = stages[tl.stage];
    if (st.vec4) conv_apply_fwd_chunk<4, false>(st, tl, t, ts, t16);
    else conv_apply_fwd_chunk<1, false>(st, tl, t, ts, t16);
}

__global__ void __launch_bounds__(kPostThreads, 4)
conv_bwd_dz_kernel(const ConvStage* __restrict__ stages, const PostChunk* __restrict__ tiles, int ntiles,
                   const TickState* __restrict__ ts, int S, int par) {
    __shared__ __align__(16) __nv_bfloat16 t16[kPostChunk + 2 * kPostTileChannels];
    if ((int)blockIdx.x >= ntiles) return;
    const PostChunk tl = tiles[blockIdx.x];
    const long long t = ts->cnt[par];
    const ConvStage& st = stages[tl.stage];
    if (st.vec4) conv_bwd_dz_chunk<4, false>(st, tl, t, ts, S, t16);
    else conv_bwd_dz_chunk<1, false>(st, tl, t, ts, S, t16);
}

// ---------------------------------------------------------------- update
// Fused SC + LWP step for materialised gradients (convolution stages):
// reads w, v and the gradient slices once, writes w, v and the predicted
// weights the next forward will use.
__global__ void __launch_bounds__(256, 6)
update_kernel(const UpdRange* __restrict__ ranges, const UpdChunk* __restrict__ chunks,
              const TickState* __restrict__ ts, int S, int par) {
    const UpdChunk ch = chunks[blockIdx.x];
    const UpdRange& R = ranges[ch.range];
    const long long j = ts->cnt[par] - 2LL * (S - 1) + R.s;
    if (!sample_live(ts, j)) return;
    float m_eff, nla, gsc;
    step_coefficients(ts, j, R.m, R.neg_lr_a, m_eff, nla, gsc);
    const int end = min(R.n, ch.start + kUpdChunk);
    const bool vec = ((reinterpret_cast<uintptr_t>(R.w) | reinterpret_cast<uintptr_t>(R.v) | reinterpret_cast<uintptr_t>(R.wh) |
                       reinterpret_cast<uintptr_t>(R.g)) & 15) == 0 && (R.part_stride & 3) == 0 && (R.n & 3) == 0 &&
                     (!R.w16 || ((reinterpret_cast<uintptr_t>(R.w16) | reinterpret_cast<uintptr_t>(R.wh16)) & 7) == 0);
    if (vec) {
        // four parameters per thread and step (kUpdChunk and ch.start are multiples of 4)
        for (int e = ch.start + 4 * threadIdx.x; e < end; e += 4 * 256) {
            // the K slices of the gradient, summed in slice order, four loads in flight at a time
            // (a slice beyond the last re-reads slice 0 and counts as zero)
            float4 g = *reinterpret_cast<const float4*>(R.g + e);
            for (int q0 = 1; q0 < R.nparts; q0 += 4) {
                float4 p[4];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    p[k] = *reinterpret_cast<const float4*>(R.g + (size_t)(q0 + k < R.nparts ? q0 + k : 0) * R.part_stride + e);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (q0 + k < R.nparts) { g.x += p[k].x; g.y += p[k].y; g.z += p[k].z; g.w += p[k].w; }
            }
            g.x *= gsc; g.y *= gsc; g.z *= gsc; g.w *= gsc;
            const float4 w = *reinterpret_cast<const float4*>(R.w + e), v = *reinterpret_cast<const float4*>(R.v + e);
            float4 vn, wn, wh;
            vn.x = fmaf(m_eff, v.x, g.x); vn.y = fmaf(m_eff, v.y, g.y); vn.z = fmaf(m_eff, v.z, g.z); vn.w = fmaf(m_eff, v.w, g.w);
            wn.x = fmaf(nla, vn.x, fmaf(R.neg_lr_b, g.x, w.x)); wn.y = fmaf(nla, vn.y, fmaf(R.neg_lr_b, g.y, w.y));
            wn.z = fmaf(nla, vn.z, fmaf(R.neg_lr_b, g.z, w.z)); wn.w = fmaf(nla, vn.w, fmaf(R.neg_lr_b, g.w, w.w));
            if (R.wform) {
                wh.x = fmaf(R.T_w, wn.x - w.x, wn.x); wh.y = fmaf(R.T_w, wn.y - w.y, wn.y);
                wh.z = fmaf(R.T_w, wn.z - w.z, wn.z); wh.w = fmaf(R.T_w, wn.w - w.w, wn.w);
            } else {
                wh.x = fmaf(R.neg_lr_T, vn.x, wn.x); wh.y = fmaf(R.neg_lr_T, vn.y, wn.y);
                wh.z = fmaf(R.neg_lr_T, vn.z, wn.z); wh.w = fmaf(R.neg_lr_T, vn.w, wn.w);
            }
            *reinterpret_cast<float4*>(R.v + e) = vn;
            *reinterpret_cast<float4*>(R.w + e) = wn;
            if (R.w16) {
                // tensor-core stages read only the bfloat16 copies of the conv weights
                __nv_bfloat162 a0 = __floats2bfloat162_rn(wn.x, wn.y), a1 = __floats2bfloat162_rn(wn.z, wn.w);
                __nv_bfloat162 b0 = __floats2bfloat162_rn(wh.x, wh.y), b1 = __floats2bfloat162_rn(wh.z, wh.w);
                uint2 ua, ub;
                ua.x = *reinterpret_cast<unsigned*>(&a0); ua.y = *reinterpret_cast<unsigned*>(&a1);
                ub.x = *reinterpret_cast<unsigned*>(&b0); ub.y = *reinterpret_cast<unsigned*>(&b1);
                *reinterpret_cast<uint2*>(R.w16 + e) = ua;
                *reinterpret_cast<uint2*>(R.wh16 + e) = ub;
            } else {
                *reinterpret_cast<float4*>(R.wh + e) = wh;
            }
        }
        return;
    }
    for (int e = ch.start + threadIdx.x; e < end; e += 256) {
        float g = 0.f;
        for (int q = 0; q < R.nparts; ++q) g += R.g[(size_t)q * R.part_stride + e];
        g *= gsc;
        const float w = R.w[e], v = R.v[e];
        const float vn = fmaf(m_eff, v, g);
        const float wn = fmaf(nla, vn, fmaf(R.neg_lr_b, g, w));
        const float wh = R.wform ? fmaf(R.T_w, wn - w, wn) : fmaf(R.neg_lr_T, vn, wn);
        R.v[e] = vn;
        R.w[e] = wn;
        if (R.w16) { R.w16[e] = __float2bfloat16_rn(wn); R.wh16[e] = __float2bfloat16_rn(wh); }
        else R.wh[e] = wh;
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

// Weight stashing: files the weights (and normalisation scale) that this tick's forward
// of every stage has used under the forward sample's ring slot, before the update
// overwrites them.  16-byte copies where source, ring and slot stride allow, else word by word.
__global__ void __launch_bounds__(256)
stash_copy_kernel(const StashRange* __restrict__ ranges, const StashChunk* __restrict__ chunks,
                  const TickState* __restrict__ ts, int par) {
    const StashChunk ch = chunks[blockIdx.x];
    const StashRange R = ranges[ch.range];
    const long long i = ts->cnt[par] - R.s;
    if (!sample_live(ts, i)) return;
    const long long bytes = R.n * R.esize;
    const char* src = static_cast<const char*>(R.src);
    char* dst = static_cast<char*>(R.ring) + (size_t)slot_of(i, R.slots) * (size_t)R.stride;
    const long long end = min(bytes, ch.start + (long long)kStashChunkBytes);
    const bool wide = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0;
    long long b = ch.start;                       // chunk starts are multiples of 16 bytes
    if (wide) {
        const long long full = ch.start + (end - ch.start) / 16 * 16;
        for (long long q = b + 16LL * threadIdx.x; q < full; q += 16LL * 256)
            *reinterpret_cast<uint4*>(dst + q) = *reinterpret_cast<const uint4*>(src + q);
        b = full;
    }
    // the rest (everything when not 16-byte aligned) in elements of 2 or 4 bytes
    if (R.esize == 4)
        for (long long q = b + 4LL * threadIdx.x; q < end; q += 4LL * 256) *reinterpret_cast<float*>(dst + q) = *reinterpret_cast<const float*>(src + q);
    else
        for (long long q = b + 2LL * threadIdx.x; q < end; q += 2LL * 256) *reinterpret_cast<unsigned short*>(dst + q) = *reinterpret_cast<const unsigned short*>(src + q);
}

// Predicted weights re-made from the current state, w_hat = w - lr T v (LWP, velocity
// form), after the horizon T of the stages has been changed between ticks.
__global__ void __launch_bounds__(256)
repredict_kernel(const UpdRange* __restrict__ ranges, const UpdChunk* __restrict__ chunks) {
    const UpdChunk ch = chunks[blockIdx.x];
    const UpdRange& R = ranges[ch.range];
    const int end = min(R.n, ch.start + kUpdChunk);
    for (int e = ch.start + threadIdx.x; e < end; e += 256) {
        const float wh = fmaf(R.neg_lr_T, R.v[e], R.w[e]);
        if (R.wh16) R.wh16[e] = __float2bfloat16_rn(wh);
        else R.wh[e] = wh;
    }
}

}  // namespace pb
