// Fused tick of 3x3 convolution stages on tiny images (4x4 or 2x2 pixels).
//
// With 4 to 16 output pixels a convolution is a matrix-vector product in all
// but name: every weight is used a handful of times, so the stage is bound by
// streaming its weights, exactly like a fully connected stage ("weight
// bandwidth without reuse", Appendix "GPU Bottlenecks for Fine-Grained Pipelined
// Training").  It therefore gets the treatment of the FC tick kernel: ONE pass
// over (w, v) serves the forward of the sample that has arrived (with the
// predicted weights w_hat = w - lr T v formed in registers), the data gradient
// of the sample whose gradient has come back (with the current w), the weight
// gradient (never written to memory) and the SC + LWP update: 16 bytes per
// parameter and tick.
//
// Work split: a block owns kGemvRows output channels of one stage.  Lanes own
// input channels (32 per step, a warp takes every 8th step), so one lane reads
// the 9 taps of (c_out, c_in) as 36 contiguous bytes and holds that channel's
// 16 (or 4) forward and backward input pixels in registers.  Forward sums over
// input channels are reduced in the warp and kept per warp in shared memory;
// input gradients stay in registers across the block's output channels and
// leave as one partial row per block, added up by the reader in table order.
// The 3x3 / pad 1 neighbourhoods are compile-time patterns: the tap loops unroll
// completely and taps that fall outside the image vanish.
#pragma once
#include "conv_types.h"
#include "fc_kernels.cuh"

namespace pb {

constexpr int kGemvRows = 8;          // output channels per block
constexpr int kGemvThreads = 256;
constexpr int kGemvWarps = kGemvThreads / 32;

// Sums of P per-lane values over the warp with P shuffles instead of 5 P: at every halving
// step a lane keeps one half of its values and hands the other half to its partner.  On
// return every lane holds the warp total of value `idx` (pairs of lanes hold the same one).
template <int P>
__device__ __forceinline__ float warp_sum_vec(float (&f)[P], int lane, int& idx) {
    static_assert(P == 16 || P == 4, "tiny images of 4x4 or 2x2 pixels");
    idx = 0;
    if (P == 16) {
        float a[8], b[4], c[2];
        const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4, h2 = lane & 2;
#pragma unroll
        for (int q = 0; q < 8; ++q) a[q] = (h16 ? f[q + 8] : f[q]) + __shfl_xor_sync(0xffffffffu, h16 ? f[q] : f[q + 8], 16);
#pragma unroll
        for (int q = 0; q < 4; ++q) b[q] = (h8 ? a[q + 4] : a[q]) + __shfl_xor_sync(0xffffffffu, h8 ? a[q] : a[q + 4], 8);
#pragma unroll
        for (int q = 0; q < 2; ++q) c[q] = (h4 ? b[q + 2] : b[q]) + __shfl_xor_sync(0xffffffffu, h4 ? b[q] : b[q + 2], 4);
        float d = (h2 ? c[1] : c[0]) + __shfl_xor_sync(0xffffffffu, h2 ? c[0] : c[1], 2);
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        idx = (h16 ? 8 : 0) + (h8 ? 4 : 0) + (h4 ? 2 : 0) + (h2 ? 1 : 0);
        return d;
    } else {
        float a[2];
        const bool h16 = lane & 16, h8 = lane & 8;
#pragma unroll
        for (int q = 0; q < 2; ++q) a[q] = (h16 ? f[q + 2] : f[q]) + __shfl_xor_sync(0xffffffffu, h16 ? f[q] : f[q + 2], 16);
        float d = (h8 ? a[1] : a[0]) + __shfl_xor_sync(0xffffffffu, h8 ? a[0] : a[1], 8);
        d += __shfl_xor_sync(0xffffffffu, d, 4);
        d += __shfl_xor_sync(0xffffffffu, d, 2);
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        idx = (h16 ? 2 : 0) + (h8 ? 1 : 0);
        return d;
    }
}

struct ConvGemvStage {
    float* w;                 // [co][ci][3][3] master weights
    float* v;                 // velocity, same layout
    int ci, co, hw;           // image side is hw (4 or 2); P = hw*hw pixels in and out
    int s;                    // stage index
    const float* xin; int xin_slots;     // producer's output ring [slots][ci*P]
    const float* dz;          // gradient at the conv output of the backward sample [co*P]
    float* z;                 // conv output of the forward sample [co*P] (read by the normalisation kernel)
    float* dx; int dx_slots, dx_nparts;  // input-gradient hand-off [slots][nparts][ci*P]
    float neg_lr_T, m, neg_lr_a, neg_lr_b;
};
struct GemvBlock { int stage, row0, part; };

template <int HW>
__device__ void conv_gemv_block(const ConvGemvStage& st, const GemvBlock gb, long long t, int S, const TickState* ts, float* smem) {
    constexpr int P = HW * HW;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long i = t - st.s, j = t - 2LL * (S - 1) + st.s;
    const bool do_fwd = sample_live(ts, i), do_bwd = sample_live(ts, j);
    if (!do_fwd && !do_bwd) return;
    const int CI = st.ci, rows = min(kGemvRows, st.co - gb.row0);
    float* xf = smem;                               // [CI][P + 1]
    float* xb = xf + (size_t)CI * (P + 1);          // [CI][P + 1]
    float* dzs = xb + (size_t)CI * (P + 1);         // [kGemvRows][P]
    float* zsum = dzs + kGemvRows * P;              // [warps][kGemvRows][P]
    // per warp: the 32 x 9 weights and velocities of one (output channel, 32 input channels) item,
    // moved with 16-byte accesses (a lane's own 9 taps are 36 bytes: not a vector access)
    float* wst = zsum + kGemvWarps * kGemvRows * P + (size_t)warp * 576;
    float* vst = wst + 288;
    const float* __restrict__ xfg = st.xin + (size_t)ring_slot(i < 0 ? 0 : i, st.xin_slots) * CI * P;
    const float* __restrict__ xbg = st.xin + (size_t)ring_slot(j < 0 ? 0 : j, st.xin_slots) * CI * P;
    for (int e = tid; e < CI * P; e += kGemvThreads) {
        const int c = e / P, p = e - c * P;
        xf[c * (P + 1) + p] = do_fwd ? xfg[e] : 0.f;
        xb[c * (P + 1) + p] = do_bwd ? xbg[e] : 0.f;
    }
    for (int e = tid; e < kGemvRows * P; e += kGemvThreads) {
        const int r = e / P;
        dzs[e] = (do_bwd && r < rows) ? st.dz[(size_t)(gb.row0 + r) * P + (e - r * P)] : 0.f;
    }
    for (int e = tid; e < kGemvWarps * kGemvRows * P; e += kGemvThreads) zsum[e] = 0.f;
    __syncthreads();
    float m_eff, nla, gsc;
    step_coefficients(ts, j, st.m, st.neg_lr_a, m_eff, nla, gsc);
    const float nlT = st.neg_lr_T, nlb = st.neg_lr_b;
    float* __restrict__ dxrow = st.dx ? st.dx + ((size_t)ring_slot(j < 0 ? 0 : j, st.dx_slots) * st.dx_nparts + gb.part) * ((size_t)CI * P) : nullptr;

    for (int c0 = warp * 32; c0 < CI; c0 += kGemvWarps * 32) {
        const int ci = c0 + lane;                   // CI is a multiple of 32
        float xfr[P], xbr[P], dxacc[P];
#pragma unroll
        for (int p = 0; p < P; ++p) { xfr[p] = xf[ci * (P + 1) + p]; xbr[p] = xb[ci * (P + 1) + p] * gsc; dxacc[p] = 0.f; }
        // software pipeline: the next item's 288 + 288 floats are in flight (3 + 3 float4 per lane,
        // the last one only in lanes 0-7) while the current item is computed
        float4 pw[3], pv[3];
        auto fetch = [&](int r) {
            const float4* wg = reinterpret_cast<const float4*>(st.w + ((size_t)(gb.row0 + r) * CI + c0) * 9);
            const float4* vg = reinterpret_cast<const float4*>(st.v + ((size_t)(gb.row0 + r) * CI + c0) * 9);
#pragma unroll
            for (int u = 0; u < 3; ++u)
                if (lane + 32 * u < 72) { pw[u] = __ldcs(wg + lane + 32 * u); pv[u] = __ldcs(vg + lane + 32 * u); }
        };
        if (rows > 0) fetch(0);
        for (int r = 0; r < rows; ++r) {
            const size_t off0 = ((size_t)(gb.row0 + r) * CI + c0) * 9;
            __syncwarp();
#pragma unroll
            for (int u = 0; u < 3; ++u)
                if (lane + 32 * u < 72) { reinterpret_cast<float4*>(wst)[lane + 32 * u] = pw[u]; reinterpret_cast<float4*>(vst)[lane + 32 * u] = pv[u]; }
            __syncwarp();
            if (r + 1 < rows) fetch(r + 1);
            float w[9], v[9];
#pragma unroll
            for (int k = 0; k < 9; ++k) { w[k] = wst[lane * 9 + k]; v[k] = vst[lane * 9 + k]; }
            // ---- forward: z[co][p] += sum over taps of w_hat * x_fwd (this input channel's share)
            float f[P];
#pragma unroll
            for (int p = 0; p < P; ++p) f[p] = 0.f;
            float g[9];
#pragma unroll
            for (int k = 0; k < 9; ++k) g[k] = 0.f;
            float d[P];
#pragma unroll
            for (int p = 0; p < P; ++p) d[p] = dzs[r * P + p];
#pragma unroll
            for (int ky = 0; ky < 3; ++ky)
#pragma unroll
                for (int kx = 0; kx < 3; ++kx) {
                    const int k = ky * 3 + kx;
                    const float what = fmaf(nlT, v[k], w[k]);            // w_hat = w - lr T v
#pragma unroll
                    for (int py = 0; py < HW; ++py)
#pragma unroll
                        for (int px = 0; px < HW; ++px) {
                            const int qy = py + ky - 1, qx = px + kx - 1;      // input pixel under this tap (pad 1)
                            if (qy >= 0 && qy < HW && qx >= 0 && qx < HW) {
                                const int p = py * HW + px, q = qy * HW + qx;
                                f[p] = fmaf(what, xfr[q], f[p]);                // forward
                                dxacc[q] = fmaf(w[k], d[p], dxacc[q]);          // data gradient with the current weights
                                g[k] = fmaf(d[p], xbr[q], g[k]);                // weight gradient (xbr carries the 1/N of a mini-batch mean)
                            }
                        }
                }
            // ---- update: v <- m v + g ; w <- w - lr (a v + b g)
            if (do_bwd) {
#pragma unroll
                for (int k = 0; k < 9; ++k) {
                    const float vn = fmaf(m_eff, v[k], g[k]);
                    vst[lane * 9 + k] = vn;
                    wst[lane * 9 + k] = fmaf(nla, vn, fmaf(nlb, g[k], w[k]));
                }
                __syncwarp();
                float4* wg = reinterpret_cast<float4*>(st.w + off0);
                float4* vg = reinterpret_cast<float4*>(st.v + off0);
#pragma unroll
                for (int u = 0; u < 3; ++u)
                    if (lane + 32 * u < 72) {
                        __stcs(wg + lane + 32 * u, reinterpret_cast<const float4*>(wst)[lane + 32 * u]);
                        __stcs(vg + lane + 32 * u, reinterpret_cast<const float4*>(vst)[lane + 32 * u]);
                    }
            }
            // ---- forward sums over the 32 input channels of this step, into the warp's table
            if (do_fwd) {
                int idx;
                const float sum = warp_sum_vec<P>(f, lane, idx);
                if ((lane & 1) == 0 && (P == 16 || (lane & 7) == 0)) zsum[(warp * kGemvRows + r) * P + idx] += sum;
            }
        }
        if (do_bwd && dxrow) {
#pragma unroll
            for (int p = 0; p < P; ++p) dxrow[(size_t)ci * P + p] = dxacc[p];
        }
    }
    __syncthreads();
    if (do_fwd) {
        for (int e = tid; e < rows * P; e += kGemvThreads) {
            float a = 0.f;
            for (int q = 0; q < kGemvWarps; ++q) a += zsum[q * kGemvRows * P + e];          // warps in order
            st.z[(size_t)gb.row0 * P + e] = a;
        }
    }
}

__global__ void __launch_bounds__(kGemvThreads, 2)
conv_gemv_kernel(const ConvGemvStage* __restrict__ stages, const GemvBlock* __restrict__ blocks,
                 const TickState* __restrict__ ts, int S, int par) {
    extern __shared__ __align__(16) float gemv_smem[];
    __shared__ ConvGemvStage st;
    const GemvBlock gb = blocks[blockIdx.x];
    {
        const int* s_ = reinterpret_cast<const int*>(&stages[gb.stage]);
        int* d_ = reinterpret_cast<int*>(&st);
        for (int k = threadIdx.x; k < (int)(sizeof(ConvGemvStage) / 4); k += kGemvThreads) d_[k] = s_[k];
    }
    __syncthreads();
    const long long t = ts->cnt[par];
    if (st.hw == 4) conv_gemv_block<4>(st, gb, t, S, ts, gemv_smem);
    else conv_gemv_block<2>(st, gb, t, S, ts, gemv_smem);
}

}  // namespace pb
