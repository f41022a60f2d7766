// Grouped implicit-GEMM kernel for the float32 convolution path.
//
// One launch covers the forward convolutions of every stage (fprop), or the
// data gradients (dgrad), or the weight gradients (wgrad): a tile table maps
// each thread block to (problem, tile, K-slice).  Operands are gathered
// straight from the activation rings / gradient scratch (no im2col buffer) into
// shared memory; 256 threads form a 16 x 16 grid and each owns a TM x TN patch
// of a (16 TM) x (16 TN) tile.  TM and TN are 1 or 4 per problem, so that a
// layer with 16 channels or a 2x2 image does not pay for a 64 x 64 tile.
#pragma once
#include <cuda_bf16.h>

#include "conv_types.h"

namespace pb {

__device__ __forceinline__ float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

template <int KS> struct KDiv {
    __device__ __forceinline__ static void split(int kk, int k, int& c, int& r, int& s) {
        c = kk / (KS * KS); const int rs = kk - c * (KS * KS); r = rs / KS; s = rs - r * KS;
    }
};
template <> struct KDiv<0> {
    __device__ __forceinline__ static void split(int kk, int k, int& c, int& r, int& s) {
        const int k2 = k * k; c = kk / k2; const int rs = kk - c * k2; r = rs / k; s = rs - r * k;
    }
};

template <int KS, int TM, int TN>
__device__ void gemm_tile(const ConvGemm& G, const GemmTile& tl, long long smp, float* __restrict__ smem) {
    constexpr int BM = 16 * TM, BN = 16 * TN;
    float (*As)[BM + 4] = reinterpret_cast<float (*)[BM + 4]>(smem);
    float (*Bs)[BN + 4] = reinterpret_cast<float (*)[BN + 4]>(smem + kBK * (BM + 4));
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int M = G.M, N = G.N;
    const int kb = tl.split * G.k_per_split;
    const int ke = min(G.K, kb + G.k_per_split);
    const float* __restrict__ A = G.a + (size_t)(smp % G.a_slots) * G.a_elems;
    const float* __restrict__ B = G.b + (size_t)(smp % G.b_slots) * G.b_elems;
    float* __restrict__ Cp = G.c + ((size_t)(smp % G.c_slots) * G.nsplit + tl.split) * ((size_t)M * N);
    const int ksz = G.k, st = G.stride, pad = G.pad, ih = G.ih, iw = G.iw, oh = G.oh, ow = G.ow;
    const bool bf = G.bf16 != 0;
    const float inv_st = 1.f / (float)st, inv_ow = 1.f / (float)ow;     // see quot()

    float acc[TM][TN];
#pragma unroll
    for (int a = 0; a < TM; ++a)
#pragma unroll
        for (int b = 0; b < TN; ++b) acc[a][b] = 0.f;

    // Loader maps.  Element e = tid + 256 q of a tile:
    //   A, K contiguous in memory (fprop, wgrad): kk = e & 15, m = e >> 4        (q < TM)
    //   A, M fastest (dgrad):                      m = e % BM, kk = e / BM        (q < TM)
    //   B, N fastest (fprop, dgrad):               n = e % BN, kk = e / BN        (q < TN)
    //   B, K fastest (wgrad):                      kk = e & 15, n = e >> 4        (q < TN)
    const int lo16 = tid & 15, hi16 = tid >> 4;
    const int a_m = tid % BM, a_k0 = tid / BM, a_kstep = 256 / BM;      // dgrad A
    const int b_n = tid % BN, b_k0 = tid / BN, b_kstep = 256 / BN;      // fprop / dgrad B
    int n_p = 0, n_q = 0;                            // fprop/dgrad: pixel of column n0 + b_n
    bool n_ok = false;
    int wc[TN], wr[TN], ws[TN];                      // wgrad: (ci, r, s) of columns n0 + hi16 + 16 q
    bool w_ok[TN];
    if (G.mode == kFprop) {
        const int n = tl.n0 + b_n; n_ok = n < N; n_p = n / ow; n_q = n - n_p * ow;
    } else if (G.mode == kDgrad) {
        const int n = tl.n0 + b_n; n_ok = n < N; n_p = n / iw; n_q = n - n_p * iw;
    } else {
#pragma unroll
        for (int q = 0; q < TN; ++q) {
            const int n = tl.n0 + hi16 + 16 * q;
            w_ok[q] = n < N;
            KDiv<KS>::split(n, ksz, wc[q], wr[q], ws[q]);
        }
    }

    // gather of one K step into registers (ra: this thread's elements of the A tile, rb: of the B tile)
    auto fetch = [&](int k0, float (&ra)[TM], float (&rb)[TN]) {
        if (G.mode == kFprop) {
            // A[m, kk] = w_hat[m*K + kk]: 16 consecutive kk per row
            const int kk = k0 + lo16;
#pragma unroll
            for (int q = 0; q < TM; ++q) {
                const int m = tl.m0 + hi16 + 16 * q;
                ra[q] = (m < M && kk < ke) ? A[(size_t)m * G.K + kk] : 0.f;
            }
            // B[kk, n] = x[ci, p*st + r - pad, q*st + s - pad]
#pragma unroll
            for (int q = 0; q < TN; ++q) {
                const int kq = k0 + b_k0 + b_kstep * q;
                int c, r, s;
                KDiv<KS>::split(kq, ksz, c, r, s);
                const int y = n_p * st + r - pad, x = n_q * st + s - pad;
                rb[q] = (n_ok && kq < ke && y >= 0 && y < ih && x >= 0 && x < iw) ? B[((size_t)c * ih + y) * iw + x] : 0.f;
            }
        } else if (G.mode == kDgrad) {
            // A[m = ci, kk = (co, r, s)] = w[co, ci, r, s];  B[kk, n = (y, x)] = dz[co, (y+pad-r)/st, (x+pad-s)/st]
#pragma unroll
            for (int q = 0; q < TM; ++q) {
                const int kq = k0 + a_k0 + a_kstep * q;
                int c, r, s;
                KDiv<KS>::split(kq, ksz, c, r, s);
                const int m = tl.m0 + a_m;
                ra[q] = (m < M && kq < ke) ? A[(((size_t)c * G.ci + m) * ksz + r) * ksz + s] : 0.f;
            }
#pragma unroll
            for (int q = 0; q < TN; ++q) {
                const int kq = k0 + b_k0 + b_kstep * q;
                int c, r, s;
                KDiv<KS>::split(kq, ksz, c, r, s);
                const int ty_ = n_p + pad - r, tx_ = n_q + pad - s;
                float v = 0.f;
                if (n_ok && kq < ke && ty_ >= 0 && tx_ >= 0) {
                    const int p = quot(ty_, inv_st), qq = quot(tx_, inv_st);
                    if (p * st == ty_ && qq * st == tx_ && p < oh && qq < ow) v = B[((size_t)c * oh + p) * ow + qq];
                }
                rb[q] = v;
            }
        } else {
            // A[m = co, kk = pixel] = dz[m*K + kk];  B[kk = (p, q), n = (ci, r, s)] = x[ci, p*st+r-pad, q*st+s-pad]
            const int kk = k0 + lo16;
            const int p = quot(kk, inv_ow), qq = kk - p * ow;
#pragma unroll
            for (int q = 0; q < TM; ++q) {
                const int m = tl.m0 + hi16 + 16 * q;
                ra[q] = (m < M && kk < ke) ? A[(size_t)m * G.K + kk] : 0.f;
            }
#pragma unroll
            for (int q = 0; q < TN; ++q) {
                const int y = p * st + wr[q] - pad, x = qq * st + ws[q] - pad;
                rb[q] = (w_ok[q] && kk < ke && y >= 0 && y < ih && x >= 0 && x < iw) ? B[((size_t)wc[q] * ih + y) * iw + x] : 0.f;
            }
        }
        if (bf) {
#pragma unroll
            for (int q = 0; q < TM; ++q) ra[q] = round_bf16(ra[q]);
#pragma unroll
            for (int q = 0; q < TN; ++q) rb[q] = round_bf16(rb[q]);
        }
    };
    // Software pipeline: the gather of step k+1 is in flight while step k is multiplied.
    float ra[TM], rb[TN];
    fetch(kb, ra, rb);
    for (int k0 = kb; k0 < ke; k0 += kBK) {
        __syncthreads();
        if (G.mode == kDgrad) {
#pragma unroll
            for (int q = 0; q < TM; ++q) As[a_k0 + a_kstep * q][a_m] = ra[q];
        } else {
#pragma unroll
            for (int q = 0; q < TM; ++q) As[lo16][hi16 + 16 * q] = ra[q];
        }
        if (G.mode == kWgrad) {
#pragma unroll
            for (int q = 0; q < TN; ++q) Bs[lo16][hi16 + 16 * q] = rb[q];
        } else {
#pragma unroll
            for (int q = 0; q < TN; ++q) Bs[b_k0 + b_kstep * q][b_n] = rb[q];
        }
        __syncthreads();
        if (k0 + kBK < ke) fetch(k0 + kBK, ra, rb);
#pragma unroll
        for (int kk = 0; kk < kBK; ++kk) {
            float av[TM], bv[TN];
#pragma unroll
            for (int a = 0; a < TM; ++a) av[a] = As[kk][ty * TM + a];
#pragma unroll
            for (int b = 0; b < TN; ++b) bv[b] = Bs[kk][tx * TN + b];
#pragma unroll
            for (int a = 0; a < TM; ++a)
#pragma unroll
                for (int b = 0; b < TN; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
        }
    }
#pragma unroll
    for (int a = 0; a < TM; ++a) {
        const int m = tl.m0 + ty * TM + a;
        if (m >= M) continue;
#pragma unroll
        for (int b = 0; b < TN; ++b) {
            const int n = tl.n0 + tx * TN + b;
            if (n < N) Cp[(size_t)m * N + n] = acc[a][b];
        }
    }
}

template <int TM, int TN>
__device__ __forceinline__ void gemm_dispatch_k(const ConvGemm& G, const GemmTile& tl, long long smp, float* smem) {
    switch (G.k) {
        case 1: gemm_tile<1, TM, TN>(G, tl, smp, smem); break;
        case 3: gemm_tile<3, TM, TN>(G, tl, smp, smem); break;
        case 7: gemm_tile<7, TM, TN>(G, tl, smp, smem); break;
        default: gemm_tile<0, TM, TN>(G, tl, smp, smem); break;
    }
}

__global__ void __launch_bounds__(kGemmThreads)
conv_gemm_kernel(const ConvGemm* __restrict__ gemms, const GemmTile* __restrict__ tiles,
                 const TickState* __restrict__ ts, int S, int par) {
    __shared__ __align__(16) float smem[2 * kBK * (kBM + 4)];
    __shared__ ConvGemm G;                                 // descriptor copy (no re-reads through global memory)
    const GemmTile tl = tiles[blockIdx.x];
    {
        const int* s_ = reinterpret_cast<const int*>(&gemms[tl.gemm]);
        int* d_ = reinterpret_cast<int*>(&G);
        for (int k = threadIdx.x; k < (int)(sizeof(ConvGemm) / 4); k += kGemmThreads) d_[k] = s_[k];
    }
    __syncthreads();
    const long long t = ts->cnt[par];
    const long long smp = (G.mode == kFprop) ? t - G.s : t - 2LL * (S - 1) + G.s;
    if (!sample_live(ts, smp)) return;
    if (G.tm == 4) {
        if (G.tn == 4) gemm_dispatch_k<4, 4>(G, tl, smp, smem);
        else gemm_dispatch_k<4, 1>(G, tl, smp, smem);
    } else {
        if (G.tn == 4) gemm_dispatch_k<1, 4>(G, tl, smp, smem);
        else gemm_dispatch_k<1, 1>(G, tl, smp, smem);
    }
}

}  // namespace pb
