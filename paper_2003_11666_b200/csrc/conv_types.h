// Device-side descriptors of convolution stages.
#pragma once
#include <cuda_bf16.h>

#include "pb_internal.h"

namespace pb {

constexpr int kGemmThreads = 256;
constexpr int kBM = 64, kBN = 64, kBK = 16;
constexpr int kSimtMaxK = 192;             // longest K loop of one float32 tile before K is sliced
constexpr int kPostThreads = 256;         // normalisation / activation kernels
constexpr int kPostChunk = 2048;          // elements per block of those kernels
constexpr int kPostTilePixels = 128;       // pixels of a tile of the elementwise kernels
constexpr int kPostTileChannels = 64;      // most channels of such a tile
constexpr int kPostFuseTiles = 4;           // a bundle with at most this many second-step tiles is finished by its closing block
constexpr int kMaxGroupChannels = 64;      // channels per normalisation group

enum GemmMode { kFprop = 0, kDgrad = 1, kWgrad = 2 };

// One implicit GEMM  C[M,N] = sum_k A[m,k] B[k,n]  of a convolution stage.
//   fprop: M = c_out, N = out pixels, K = c_in*k*k    A = predicted weights, B = im2col(x_fwd)
//   dgrad: M = c_in,  N = in pixels,  K = c_out*k*k   A = weights (transposed view), B = scattered dz
//   wgrad: M = c_out, N = c_in*k*k,   K = out pixels  A = dz, B = im2col(x_bwd)^T
// K is cut into nsplit slices; slice q writes its own partial result
// c + q*M*N, and the reader adds the slices in order (deterministic split-K).
struct ConvGemm {
    int mode, M, N, K;
    int ci, co, k, stride, pad, ih, iw, oh, ow;
    int s;                       // stage index (for the tick arithmetic)
    int bf16;                    // round both operands to bfloat16 before multiplying
    int tm, tn;                  // per-thread patch (1 or 4): the tile is (16 tm) x (16 tn)
    int nsplit, k_per_split;
    const float* a;              // fprop: w_hat; dgrad: w (or the ring of stashed forward weights); wgrad: dz
    int a_slots, a_elems;        // ring geometry of a (1 slot unless the weights are stashed per sample)
    const float* b;              // fprop/wgrad: ring of the input activations; dgrad: dz
    int b_slots, b_elems;        // ring geometry of b (1 slot for dz)
    float* c;                    // [c_slots][nsplit][M*N]
    int c_slots;
};

struct GemmTile { int gemm, m0, n0, split; };

// Everything the normalisation / activation / pooling kernels need for one stage.
struct ConvStage {
    int s;
    int co, oh, ow;              // conv output (z) shape
    int groups, cpg;             // GroupNorm groups, channels per group
    int relu, avgpool;
    int need_out32;              // somebody reads the float32 output ring (a skip add, a CUDA-core or FC consumer)
    int vec4;                    // oh*ow is a multiple of 4: the element kernels use 4-wide accesses
    int pool_k, pool_stride, pool_pad;   // pool_k == 0: no max-pool
    int out_h, out_w;            // stage output spatial shape (after pooling)
    // forward
    const float* zpart; int z_nsplit;    // fprop partial sums [nsplit][co*oh*ow]
    float* z_ring;               // [slots][co*oh*ow] conv output, kept for the backward
    float* stat_ring;            // [slots][2*groups] mean, rstd
    float* fstat; int fstat_stride;      // forward chunk partials [groups][fstat_stride][3]: count, mean, M2
    int fused;                           // the forward GEMM wrote z_ring and fstat itself (one K slice)
    float* bsum; int npieces;            // backward channel partials [co][npieces][2]
    float* gsum;                 // backward group means [groups][2] (of d*gamma and d*gamma*zhat)
    unsigned char* code_ring;    // [slots][co*oh*ow] bit0: ReLU passed
    unsigned char* arg_ring;     // [slots][co*out_h*out_w] max-pool winner position in its window
    float* out_ring;             // [slots][co*out_h*out_w]
    __nv_bfloat16* out16;        // [slots][out_h*out_w][co] bfloat16 NHWC copy for the tensor-core path (or nullptr)
    int slots;                   // D_s + 1 (all the rings above)
    const float* wh;             // predicted parameters: weights, then gamma, then beta
    const float* w;              // current parameters
    float* g;                    // gradient buffer, same layout
    int nw;                      // number of conv weights (offset of gamma)
    // skip input
    const float* skip_ring; int skip_slots, skip_mode, skip_c, skip_h, skip_w;   // skip_ring == nullptr: none
    int skip_pre;                // the skip input joins the convolution output BEFORE the normalisation and is the source
                                 // stage's own such sum (skip_ring is then that stage's z_ring): pre-activation networks
    int n_rsrc; DeltaSrc rsrc[kMaxDeltaSrc];   // later stages that added this stage's sum to theirs: their gradients join dz
    float* dskip; int dskip_slots;       // gradient handed to the skip source [slots][skip elems]
    // backward
    int n_dsrc; DeltaSrc dsrc[kMaxDeltaSrc];
    const float* gstash; int gstash_slots;   // weight stashing: ring [slots][co] of the scale each forward used (or nullptr)
    float* dz;                   // scratch [co*oh*ow]
    __nv_bfloat16* dz16;         // scratch [oh*ow][co] bfloat16 NHWC copy (or nullptr)
};

// A range of parameters updated together: v <- m v + g, w <- w - lr (a v + b g),
// w_hat <- w - lr T v, with g the sum of nparts partial gradients.
struct UpdRange {
    float *w, *v, *wh;
    __nv_bfloat16 *w16, *wh16;   // bfloat16 copies of w and w_hat in the same order (or nullptr)
    const float* g; int nparts; long long part_stride;
    int n;
    int s;
    float neg_lr_T, m, neg_lr_a, neg_lr_b;
    float T_w; int wform;        // weight-difference form: w_hat = w_new + T (w_new - w_old)
};
struct UpdChunk { int range, start; };
// Weight stashing: one tensor whose forward copy (src) is filed under the forward sample's
// slot of a ring, n elements of esize bytes each.
struct StashRange { const void* src; void* ring; int slots, s, esize; long long n, stride; };   // stride: bytes between ring slots
struct StashChunk { int range; long long start; };
constexpr int kStashChunkBytes = 32768;

// One block's share of the normalisation kernels: channels [cl0, cl0+ncl) of group `grp`
// (relative to the group), pixels [p0, p0+np); chunk `idx` of `nidx` in its group.
// The same record describes a tile of the elementwise kernels: there cl0 is an absolute
// channel and grp is not used.
// Either ncl >= 1 whole channels (p0 = 0, np = all pixels) or a piece of one channel.
struct PostChunk { int stage, grp, cl0, ncl, p0, np, idx, nidx, bundle; };   // bundle < 0: the stage is not fused
// A bundle: groups [grp0, grp0 + ngrp) of one stage, whose nchunks chunks are closed by
// one block that then works through the bundle's tiles of the second step.
// One normalisation group of a stage that is not fused (a warp of the merge kernel).
struct GroupRef { int stage, grp; };
struct PostBundle { int stage, grp0, ngrp, nchunks, ftile0, nftiles, btile0, nbtiles; };
constexpr int kUpdChunk = 4096;
constexpr bool kEarlyIngest = true;        // conv networks: the sample of tick t+1 is copied in beside the update of tick t
constexpr bool kEarlyBackward = true;      // large networks: the first backward step of tick t+1 runs beside the update of tick t
// stream priorities of a conv tick's side chains (1 = the device's highest, 0 = default)
constexpr int kPrioBwd = 1, kPrioAux = 1, kPrioSide = 0;

#ifdef __CUDACC__
// Quotient a / b for 0 <= a < 2^21 and b <= 2^13 from the float reciprocal of b: the
// product (a + 0.5) / b is at least 0.5 / b away from every integer, far more than its
// rounding error (about 2e-7 a / b), so rounding down gives the exact quotient.  A
// negative a gives a negative result (only ever used to reject the element).
__device__ __forceinline__ int quot(int a, float inv_b) { return __float2int_rd(((float)a + 0.5f) * inv_b); }
#endif

}  // namespace pb
