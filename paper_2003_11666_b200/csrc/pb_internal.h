// Internal descriptors shared by the host-side engine and its kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace pb {

constexpr int kMaxDeltaSrc = 4;     // consumers feeding one stage's output gradient
constexpr int kFcThreads = 256;
constexpr int kFcWarps = kFcThreads / 32;
constexpr int kFcMaxSegRows = 256;  // rows of one FC segment (bounds shared memory)
constexpr int kFcChunksPerSweep = 2;
// FC tick kernel: signal the next tick's launch at the START of this one (its blocks then wait
// resident) instead of at block exit.  Measured slower on the 4-stage MLP (14.7 vs 13.2 us/tick),
// equal on the deep one: off.
constexpr bool kFcEarlyTrigger = false;
constexpr int kFcBlocksPerSM = 2;         // resident blocks per SM of the FC tick kernel (register budget) = blocks of the first wave
constexpr double kFcTailFraction = 0.10;  // share of a large stage's rows left to short second-wave blocks
constexpr int kFcTailRows = 16;           // rows of one such block

// Where a stage finds the gradient w.r.t. its output: a consumer's hand-off
// buffer laid out [slots][nparts][elems]; the reader sums the nparts rows.
struct DeltaSrc {
    const float* ptr;
    int slots;
    int nparts;
};

// Device-side description of one fully connected stage.
struct FcStage {
    float* w;              // [out, in] master weights; bias [out] follows at w + out*in
    float* v;              // velocity, same layout
    int in_dim, out_dim;
    int s;                 // stage index
    int relu;              // ReLU follows
    int is_last;           // softmax cross-entropy follows
    int need_dx;           // 0 for the first stage
    int vec;               // 4 when rows are 16-byte aligned, else 1
    const float* xin;      // producer's output ring (or the input ring) [xin_slots][in_dim]
    int xin_slots;
    float* out;            // own output ring [out_slots][out_dim]
    int out_slots;
    float* dx;             // own hand-off buffer [dx_slots][dx_nparts][in_dim]
    int dx_slots, dx_nparts;
    int n_dsrc;
    DeltaSrc dsrc[kMaxDeltaSrc];
    float neg_lr_T;        // -lr * T      (LWP horizon)
    float T_w;             // T itself, for the weight-difference form
    float* wh;             // stored predicted weights (weight-difference form only), else nullptr
    float* stash;          // weight stashing: ring [stash_slots][out*in] of the weights each forward used, else nullptr
    int stash_slots;
    float m;               // momentum
    float neg_lr_a;        // -lr * a      (spike compensation)
    float neg_lr_b;        // -lr * b
};

// One thread block's share of one FC stage: rows [row0, row1).
struct FcSeg {
    int stage;             // index into the FcStage table
    int row0, row1;
    int part;              // which partial row of the stage's dx buffer it writes
    int fused;             // last stage, whole in this block: loss, backward and update follow its forward here
};

// Tick state that lives on the device so that launches need no per-tick
// arguments besides a parity bit.  Every kernel of tick t is launched with
// par = t & 1 and reads cnt[par]; the last kernel of the tick writes
// cnt[par ^ 1] = t + 1.  No kernel reads a field that another block of the
// same launch writes.
struct TickState {
    long long cnt[2];
    int error;             // first failed index check (0 = none)
    int error_info;
    int fd_n;              // fill-and-drain mode: samples per update (0 = pipelined backpropagation)
    int fd_cycle;          // ... and ticks per update, fd_n + 2 (S - 1)
};

enum ErrorCode { kErrNone = 0, kErrSegRows = 1, kErrLabel = 2, kErrSlot = 3, kErrWait = 4 };

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

#ifdef __CUDACC__
// Samples are named by the tick at which they entered.  In pipelined backpropagation
// one enters at every tick; when the pipeline is filled and drained for every update
// (mini-batch SGD, Section 1), only at the first fd_n ticks of a cycle.
__device__ __forceinline__ bool sample_live(const TickState* ts, long long i) {
    if (i < 0) return false;
    const int n = ts->fd_n;
    return n == 0 || (int)((unsigned)i % (unsigned)ts->fd_cycle) < n;      // ticks stay far below 2^32
}

// Coefficients of the update that backward sample j triggers:
//   v <- m_eff v + gscale g ;  w <- w + nla_eff v + neg_lr_b (gscale g).
// Pipelined backpropagation: the stage's own constants.  Fill and drain: the velocity
// collects the mean gradient of the cycle (decayed once, at the cycle's first sample)
// and the weights move once, at its last sample, so that every sample of the cycle
// sees the same weights; the stage tables then hold a = 1, b = 0, T = 0.
__device__ __forceinline__ void step_coefficients(const TickState* ts, long long j, float m, float neg_lr_a,
                                                  float& m_eff, float& nla_eff, float& gscale) {
    const int n = ts->fd_n;
    m_eff = m; nla_eff = neg_lr_a; gscale = 1.f;
    if (n > 0 && j >= 0) {
        const int pos = (int)((unsigned)j % (unsigned)ts->fd_cycle);
        m_eff = pos == 0 ? m : 1.f;
        nla_eff = pos == n - 1 ? neg_lr_a : 0.f;
        gscale = 1.f / (float)n;
    }
}
#endif

}  // namespace pb
