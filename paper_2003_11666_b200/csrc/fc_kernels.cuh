// Fully connected stages of a Pipelined Backpropagation tick.
//
// For an FC stage everything a tick needs from the weights can be served by
// ONE pass over (w, v): the forward of the sample that has just arrived uses
// the predicted weights w_hat = w - lr*T*v (LWP, velocity form), the backward
// of the sample whose gradient has come back uses w itself, and the update
// v <- m v + g, w <- w - lr (a v + b g) (combined SC + LWP step) needs only the
// rank-1 gradient g = delta x^T, which is formed on the fly.  So the kernel
// reads w and v once, writes them once (16 bytes per parameter) and never
// materialises w_hat or g.
//
// Work split: a thread block owns a band of rows [row0, row1) of one stage.
// Each warp owns a set of 128-column chunks ("column group") and a subset of
// the band's rows ("row split").  Row sums (the forward GEMV) are reduced with
// warp shuffles and a small shared-memory table; column sums (the data
// gradient W^T delta) stay in registers across the band and leave as one
// partial row per band that the consumer adds up in a fixed order, so results
// do not depend on scheduling.
#pragma once
#include "pb_internal.h"

namespace pb {

template <int VEC> struct VecT;
template <> struct VecT<4> { using type = float4; };
template <> struct VecT<1> { using type = float; };

template <int VEC> __device__ __forceinline__ void vload(float (&r)[VEC], const float* p);
template <> __device__ __forceinline__ void vload<4>(float (&r)[4], const float* p) {
    float4 q = *reinterpret_cast<const float4*>(p);
    r[0] = q.x; r[1] = q.y; r[2] = q.z; r[3] = q.w;
}
template <> __device__ __forceinline__ void vload<1>(float (&r)[1], const float* p) { r[0] = *p; }

// streaming load: the weights are touched once per tick
template <int VEC> __device__ __forceinline__ void vload_stream(float (&r)[VEC], const float* p);
template <> __device__ __forceinline__ void vload_stream<4>(float (&r)[4], const float* p) {
    float4 q = __ldcs(reinterpret_cast<const float4*>(p));
    r[0] = q.x; r[1] = q.y; r[2] = q.z; r[3] = q.w;
}
template <> __device__ __forceinline__ void vload_stream<1>(float (&r)[1], const float* p) { r[0] = __ldcs(p); }

template <int VEC> __device__ __forceinline__ void vstore(float* p, const float (&r)[VEC]);
template <> __device__ __forceinline__ void vstore<4>(float* p, const float (&r)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(r[0], r[1], r[2], r[3]);
}
template <> __device__ __forceinline__ void vstore<1>(float* p, const float (&r)[1]) { *p = r[0]; }

// streaming store: updated weights are not read again before the next tick
template <int VEC> __device__ __forceinline__ void vstore_stream(float* p, const float (&r)[VEC]);
template <> __device__ __forceinline__ void vstore_stream<4>(float* p, const float (&r)[4]) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(r[0], r[1], r[2], r[3]));
}
template <> __device__ __forceinline__ void vstore_stream<1>(float* p, const float (&r)[1]) { __stcs(p, r[0]); }

__device__ __forceinline__ int ring_slot(long long sample, int slots) {
    return (int)((unsigned)sample % (unsigned)slots);   // samples stay far below 2^32
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Sum of four per-lane values over the warp with 6 shuffles instead of 20:
// after the exchange steps lane l holds the total of value (l>>3)&3... every
// lane ends with the total of value q = ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1).
__device__ __forceinline__ float warp_sum4(float a0, float a1, float a2, float a3, int lane) {
    const bool hi16 = lane & 16;
    float keep0 = hi16 ? a2 : a0, send0 = hi16 ? a0 : a2;
    float keep1 = hi16 ? a3 : a1, send1 = hi16 ? a1 : a3;
    keep0 += __shfl_xor_sync(0xffffffffu, send0, 16);
    keep1 += __shfl_xor_sync(0xffffffffu, send1, 16);
    const bool hi8 = lane & 8;
    float keep = hi8 ? keep1 : keep0, send = hi8 ? keep0 : keep1;
    keep += __shfl_xor_sync(0xffffffffu, send, 8);
    keep += __shfl_xor_sync(0xffffffffu, keep, 4);
    keep += __shfl_xor_sync(0xffffffffu, keep, 2);
    keep += __shfl_xor_sync(0xffffffffu, keep, 1);
    return keep;
}

struct FcShared {
    float rowpart[kFcWarps][kFcMaxSegRows];               // forward partial sums per column group
    float delta[kFcMaxSegRows];                           // gradient w.r.t. the band's pre-activations
    float colpart[kFcWarps][kFcChunksPerSweep * 128];     // column partials across row splits
    float red[kFcWarps];
    int redi[kFcWarps];
    float bcast[2];
};

// Gradient of the loss w.r.t. the pre-activation of row `r` for the backward
// sample: sum of the consumers' partial rows, gated by the ReLU that followed.
__device__ __forceinline__ float gather_delta(const FcStage& st, int r, long long j) {
    float d = 0.f;
    for (int q = 0; q < st.n_dsrc; ++q) {
        const DeltaSrc& ds = st.dsrc[q];
        const float* p = ds.ptr + ((size_t)ring_slot(j, ds.slots) * ds.nparts) * st.out_dim + r;
        for (int k = 0; k < ds.nparts; ++k) d += p[(size_t)k * st.out_dim];
    }
    if (st.relu) {
        const float y = st.out[(size_t)ring_slot(j, st.out_slots) * st.out_dim + r];
        d = y > 0.f ? d : 0.f;
    }
    return d;
}

// phase 0: every stage's forward, and backward + update of every stage but the
//          last (whose gradient only exists once its own forward is done);
// phase 1: the last stage's loss, backward and update.
// ST: weight stashing (the comparison mode of Appendix "Pipelined Backpropagation",
//     Eq. W_{i+1} = W_i - eta grad L(x_i; F_i)): the forward files the weights it used in
//     a ring slot of its sample, and the data gradient of the backward sample is taken
//     with the weights filed at THAT sample's forward instead of the current ones.
template <int VEC, bool WF, bool ST>
__device__ void fc_segment(const FcStage& st, const FcSeg& seg, long long t, int S, int phase,
                           const int* __restrict__ label_ring, float* __restrict__ loss_out,
                           FcShared& sh, TickState* ts, const float* __restrict__ x_now, int label_now) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long i = t - st.s;                        // forward sample
    const long long j = t - 2LL * (S - 1) + st.s;        // backward sample
    const bool live_j = sample_live(ts, j);
    const bool do_fwd = phase == 0 && sample_live(ts, i);
    const bool do_bwd = live_j && (st.is_last ? phase == 1 : phase == 0);
    if (phase == 1 && seg.row0 == 0 && tid == 0 && !live_j && loss_out) *loss_out = __int_as_float(0x7fc00000);
    if (!do_fwd && !do_bwd) return;
    const int rows = seg.row1 - seg.row0;
    if (rows > kFcMaxSegRows || rows <= 0) {
        if (tid == 0) { ts->error = kErrSegRows; ts->error_info = seg.stage; }
        return;
    }
    const int in = st.in_dim, out = st.out_dim;
    const float* __restrict__ xf = st.xin + (size_t)ring_slot(i < 0 ? 0 : i, st.xin_slots) * in;
    const float* __restrict__ xb = st.xin + (size_t)ring_slot(j < 0 ? 0 : j, st.xin_slots) * in;
    // when this launch also ingests the sample, the input ring slot of tick t is being
    // written by other blocks: read the caller's copy of the current sample instead
    if (x_now && st.s == 0) {
        xf = x_now;
        if (j == t) xb = x_now;
    }

    // ---- gradient w.r.t. this band's pre-activations
    __syncthreads();   // shared memory may still be in use by the previous segment
    if (do_bwd) {
        if (st.is_last) {
            // softmax over all logits (every block repeats it; n_classes is small).
            // The term of the first maximum (exp(0) = 1) is kept out of the sum so
            // that a confident prediction's loss, log1p(rest), keeps its digits.
            const float* lg = st.out + (size_t)ring_slot(j, st.out_slots) * out;
            float mx = -INFINITY;
            int amx = 0x7fffffff;
            for (int k = tid; k < out; k += kFcThreads) {
                const float x = lg[k];
                if (x > mx) { mx = x; amx = k; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float om = __shfl_xor_sync(0xffffffffu, mx, o);
                const int oa = __shfl_xor_sync(0xffffffffu, amx, o);
                if (om > mx || (om == mx && oa < amx)) { mx = om; amx = oa; }
            }
            if (lane == 0) { sh.red[warp] = mx; sh.redi[warp] = amx; }
            __syncthreads();
            mx = sh.red[0]; amx = sh.redi[0];
            for (int k = 1; k < kFcWarps; ++k)
                if (sh.red[k] > mx || (sh.red[k] == mx && sh.redi[k] < amx)) { mx = sh.red[k]; amx = sh.redi[k]; }
            __syncthreads();
            float rest = 0.f;
            for (int k = tid; k < out; k += kFcThreads) rest += (k == amx) ? 0.f : expf(lg[k] - mx);
            rest = warp_sum(rest);
            if (lane == 0) sh.red[warp] = rest;
            __syncthreads();
            rest = 0.f;
            for (int k = 0; k < kFcWarps; ++k) rest += sh.red[k];
            const float sum = 1.f + rest;
            int label = (x_now && j == t) ? label_now : label_ring[ring_slot(j, S)];
            if (label < 0 || label >= out) {
                if (tid == 0) { ts->error = kErrLabel; ts->error_info = label; }
                label = 0;
            }
            if (seg.row0 == 0 && tid == 0 && loss_out) *loss_out = log1pf(rest) - (lg[label] - mx);
            const float inv = 1.f / sum;
            for (int r = tid; r < rows; r += kFcThreads) {
                const int row = seg.row0 + r;
                sh.delta[r] = expf(lg[row] - mx) * inv - (row == label ? 1.f : 0.f);
            }
        } else {
            for (int r = tid; r < rows; r += kFcThreads) sh.delta[r] = gather_delta(st, seg.row0 + r, j);
        }
    }
    __syncthreads();

    // ---- warp roles
    constexpr int CW = 32 * VEC;                          // columns per chunk
    const int nchunks = ceil_div(in, CW);
    int ncg = 1;
    while (ncg * 2 <= nchunks && ncg * 2 <= kFcWarps) ncg *= 2;
    const int nrs = kFcWarps / ncg;
    const int cg = warp % ncg, rs = warp / ncg;
    const float nlT = st.neg_lr_T, nlb = st.neg_lr_b, Tw = st.T_w;
    float m, nla, gsc;
    step_coefficients(ts, j, st.m, st.neg_lr_a, m, nla, gsc);
    const bool want_dx = do_bwd && st.need_dx;
    const size_t wcount = (size_t)out * in;
    float* __restrict__ stash_f = ST ? st.stash + (size_t)ring_slot(i < 0 ? 0 : i, st.stash_slots) * wcount : nullptr;
    const float* __restrict__ stash_b = ST ? st.stash + (size_t)ring_slot(j < 0 ? 0 : j, st.stash_slots) * wcount : nullptr;

    for (int c0 = 0; c0 < nchunks; c0 += ncg * kFcChunksPerSweep) {
        int col[kFcChunksPerSweep];
        bool cok[kFcChunksPerSweep];
        float xfr[kFcChunksPerSweep][VEC], xbr[kFcChunksPerSweep][VEC], cacc[kFcChunksPerSweep][VEC];
#pragma unroll
        for (int c = 0; c < kFcChunksPerSweep; ++c) {
            col[c] = (c0 + cg + c * ncg) * CW + lane * VEC;
            cok[c] = col[c] < in;            // in % VEC == 0, so a vector is all in or all out
#pragma unroll
            for (int e = 0; e < VEC; ++e) { xfr[c][e] = 0.f; xbr[c][e] = 0.f; cacc[c][e] = 0.f; }
            if (cok[c]) {
                if (do_fwd) vload<VEC>(xfr[c], xf + col[c]);
                if (do_bwd) {
                    vload<VEC>(xbr[c], xb + col[c]);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) xbr[c][e] *= gsc;
                }
            }
        }
        // Rows of this row split, two at a time, software-pipelined: the loads of the
        // next pair are issued before the current pair is used, so a warp always has a
        // full set of loads in flight while it computes and stores.
        const int step = nrs * 2;
        // (WF: the weight-difference form keeps its predicted weights in memory; they ride
        //  in the slot of the velocity operand's twin `hv`)
        // (ST: the stashed weights of the backward sample ride in `sv`)
        auto load_pair = [&](float (&wv)[2][kFcChunksPerSweep][VEC], float (&vv)[2][kFcChunksPerSweep][VEC],
                             float (&hv)[2][kFcChunksPerSweep][VEC], float (&sv)[2][kFcChunksPerSweep][VEC], int r0) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int r = r0 + u;
#pragma unroll
                for (int c = 0; c < kFcChunksPerSweep; ++c) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) { wv[u][c][e] = 0.f; vv[u][c][e] = 0.f; if (WF) hv[u][c][e] = 0.f; if (ST) sv[u][c][e] = 0.f; }
                    if (r < rows && cok[c]) {
                        const size_t off = (size_t)(seg.row0 + r) * in + col[c];
                        vload_stream<VEC>(wv[u][c], st.w + off);
                        if (do_bwd) vload_stream<VEC>(vv[u][c], st.v + off);
                        if (WF && do_fwd) vload_stream<VEC>(hv[u][c], st.wh + off);
                        if (ST && want_dx) vload_stream<VEC>(sv[u][c], stash_b + off);
                    }
                }
            }
        };
        auto use_pair = [&](float (&wv)[2][kFcChunksPerSweep][VEC], float (&vv)[2][kFcChunksPerSweep][VEC],
                            float (&hv)[2][kFcChunksPerSweep][VEC], float (&sv)[2][kFcChunksPerSweep][VEC], int r0) {
            float facc[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int r = r0 + u;
                facc[u] = 0.f;
                const float d = (do_bwd && r < rows) ? sh.delta[r] : 0.f;
#pragma unroll
                for (int c = 0; c < kFcChunksPerSweep; ++c) {
                    float wn[VEC], vn[VEC], hn[VEC], wf[VEC];
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        const float w = wv[u][c][e], v = vv[u][c][e];
                        const float what = WF ? hv[u][c][e] : fmaf(nlT, v, w);   // w_hat = w - lr T v (or the stored prediction)
                        wf[e] = what;
                        facc[u] = fmaf(what, xfr[c][e], facc[u]);     // forward  (W_hat x)
                        cacc[c][e] = fmaf(ST ? sv[u][c][e] : w, d, cacc[c][e]);   // backward (W^T delta; stashed forward weights when ST)
                        const float g = d * xbr[c][e];                // rank-1 gradient (xbr carries the 1/N of a mini-batch mean)
                        vn[e] = fmaf(m, v, g);                        // v <- m v + g
                        wn[e] = fmaf(nla, vn[e], fmaf(nlb, g, w));    // w <- w - lr (a v + b g)
                        hn[e] = fmaf(Tw, wn[e] - w, wn[e]);           // w_hat = w_new + T (w_new - w_old)
                    }
                    if (ST && do_fwd && r < rows && cok[c])
                        vstore_stream<VEC>(stash_f + (size_t)(seg.row0 + r) * in + col[c], wf);
                    if (do_bwd && r < rows && cok[c]) {
                        const size_t off = (size_t)(seg.row0 + r) * in + col[c];
                        vstore_stream<VEC>(st.w + off, wn);
                        vstore_stream<VEC>(st.v + off, vn);
                        if (WF) vstore_stream<VEC>(st.wh + off, hn);
                    }
                }
            }
            if (do_fwd && r0 < rows) {
                // two row sums with 5 shuffles: lanes 0-15 end with row r0, lanes 16-31 with row r0+1
                const bool hi = lane & 16;
                float keep = hi ? facc[1] : facc[0];
                const float send = hi ? facc[0] : facc[1];
                keep += __shfl_xor_sync(0xffffffffu, send, 16);
                keep += __shfl_xor_sync(0xffffffffu, keep, 8);
                keep += __shfl_xor_sync(0xffffffffu, keep, 4);
                keep += __shfl_xor_sync(0xffffffffu, keep, 2);
                keep += __shfl_xor_sync(0xffffffffu, keep, 1);
                const int q = lane >> 4;
                if ((lane & 15) == 0 && r0 + q < rows) {
                    float* slot = &sh.rowpart[cg][r0 + q];
                    *slot = (c0 == 0 ? 0.f : *slot) + keep;
                }
            }
        };
        {
            // (ha / hb are only touched when WF is set; otherwise they cost nothing)
            float wa[2][kFcChunksPerSweep][VEC], va[2][kFcChunksPerSweep][VEC], ha[2][kFcChunksPerSweep][VEC], sa[2][kFcChunksPerSweep][VEC];
            float wb[2][kFcChunksPerSweep][VEC], vb[2][kFcChunksPerSweep][VEC], hb[2][kFcChunksPerSweep][VEC], sb[2][kFcChunksPerSweep][VEC];
            int r0 = rs * 2;
            load_pair(wa, va, ha, sa, r0);
            for (; r0 < rows; r0 += 2 * step) {
                load_pair(wb, vb, hb, sb, r0 + step);
                use_pair(wa, va, ha, sa, r0);
                load_pair(wa, va, ha, sa, r0 + 2 * step);
                use_pair(wb, vb, hb, sb, r0 + step);
            }
        }
        // column partials: combine the row splits in a fixed order, then store
        if (want_dx) {
            if (nrs > 1) {
#pragma unroll
                for (int c = 0; c < kFcChunksPerSweep; ++c)
#pragma unroll
                    for (int e = 0; e < VEC; ++e) sh.colpart[warp][c * 128 + lane * VEC + e] = cacc[c][e];
                __syncthreads();
                if (rs == 0) {
#pragma unroll
                    for (int c = 0; c < kFcChunksPerSweep; ++c)
#pragma unroll
                        for (int e = 0; e < VEC; ++e) {
                            float a = cacc[c][e];
                            for (int k = 1; k < nrs; ++k) a += sh.colpart[k * ncg + cg][c * 128 + lane * VEC + e];
                            cacc[c][e] = a;
                        }
                }
                __syncthreads();
            }
            if (rs == 0) {
                float* dst = st.dx + ((size_t)ring_slot(j, st.dx_slots) * st.dx_nparts + seg.part) * in;
#pragma unroll
                for (int c = 0; c < kFcChunksPerSweep; ++c)
                    if (cok[c]) vstore<VEC>(dst + col[c], cacc[c]);
            }
        }
    }
    __syncthreads();

    // ---- finish rows: bias, activation, bias update
    float* bias = st.w + (size_t)out * in;
    float* vbias = st.v + (size_t)out * in;
    for (int r = tid; r < rows; r += kFcThreads) {
        const int row = seg.row0 + r;
        const float b = bias[row];
        const float vb = do_bwd ? vbias[row] : 0.f;
        if (do_fwd) {
            float y = 0.f;
            for (int k = 0; k < ncg; ++k) y += sh.rowpart[k][r];
            y += WF ? st.wh[(size_t)out * in + row] : fmaf(nlT, vb, b);
            if (st.relu) y = fmaxf(y, 0.f);
            st.out[(size_t)ring_slot(i, st.out_slots) * out + row] = y;
        }
        if (do_bwd) {
            const float g = sh.delta[r] * gsc;
            const float vn = fmaf(m, vb, g);
            const float bn = fmaf(nla, vn, fmaf(nlb, g, b));
            vbias[row] = vn;
            bias[row] = bn;
            if (WF) st.wh[(size_t)out * in + row] = fmaf(Tw, bn - b, bn);
        }
    }
}

// One launch per tick for fully connected pipelines: phase 0 of every stage, the
// fused last stage, and (ingest != 0) the copy of the new sample and label into
// their rings.  When the last stage is too large for one block it gets its own
// phase-1 launch; `publish` marks the launch that ends the tick.
__global__ void __launch_bounds__(kFcThreads, kFcBlocksPerSM)
fc_tick_kernel(const FcStage* __restrict__ stages, const FcSeg* __restrict__ segs,
               const int* __restrict__ cta_seg_begin, TickState* ts, int S, int phase, int par, int publish,
               int* __restrict__ label_ring, float* __restrict__ losses, long long t_base,
               const float* __restrict__ xs, const int* __restrict__ labels, int label_value,
               float* __restrict__ in_ring, int in_slots, int elems) {
    __shared__ FcShared sh;
    __shared__ FcStage sst;
    // Programmatic dependent launch: when the host launches consecutive ticks with that
    // attribute, the next tick's blocks may become resident as soon as every block of
    // this one has started, and they stop here until this grid has finished and its
    // stores are visible.  Only the constant tables are read before the wait.  (Without
    // the attribute both instructions do nothing.)
    if (kFcEarlyTrigger) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int seg_begin = cta_seg_begin[blockIdx.x], seg_end = cta_seg_begin[blockIdx.x + 1];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long t = ts->cnt[par];
    float* loss_out = losses ? losses + (t - t_base) : nullptr;
    const float* x_now = nullptr;
    int label_now = 0;
    if (xs) {
        // ingest: every block copies a slice of the sample; block 0 files the label
        x_now = xs + (size_t)(t - t_base) * elems;
        label_now = labels ? labels[t - t_base] : label_value;
        float* dst = in_ring + (size_t)(t % in_slots) * elems;
        for (int k = blockIdx.x * kFcThreads + threadIdx.x; k < elems; k += gridDim.x * kFcThreads) dst[k] = x_now[k];
        if (blockIdx.x == 0 && threadIdx.x == 0) label_ring[t % S] = label_now;
    }
    for (int q = seg_begin; q < seg_end; ++q) {
        const FcSeg seg = segs[q];
        // the stage descriptor goes through shared memory: the kernel stores to global
        // memory in its loops, so fields behind a global reference would be re-read
        __syncthreads();
        {
            const int* s_ = reinterpret_cast<const int*>(&stages[seg.stage]);
            int* d_ = reinterpret_cast<int*>(&sst);
            for (int k = threadIdx.x; k < (int)(sizeof(FcStage) / 4); k += kFcThreads) d_[k] = s_[k];
        }
        __syncthreads();
        const FcStage& st = sst;
        const int nph = seg.fused ? 2 : 1;
        for (int ph = 0; ph < nph; ++ph) {
            const int phs = seg.fused ? ph : phase;
            if (st.stash) {
                // the comparison mode: scalar or vector, both prediction forms, in one instantiation each
                if (st.wh) {
                    if (st.vec == 4) fc_segment<4, true, true>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
                    else fc_segment<1, true, true>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
                } else {
                    if (st.vec == 4) fc_segment<4, false, true>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
                    else fc_segment<1, false, true>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
                }
            } else if (st.wh) {
                if (st.vec == 4) fc_segment<4, true, false>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
                else fc_segment<1, true, false>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
            } else {
                if (st.vec == 4) fc_segment<4, false, false>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
                else fc_segment<1, false, false>(st, seg, t, S, phs, label_ring, loss_out, sh, ts, x_now, label_now);
            }
            __syncthreads();      // the logits written by phase 0 are read by phase 1
        }
    }
    if (publish && blockIdx.x == 0 && threadIdx.x == 0) ts->cnt[par ^ 1] = t + 1;
}

}  // namespace pb
