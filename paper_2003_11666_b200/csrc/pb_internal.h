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
};

enum ErrorCode { kErrNone = 0, kErrSegRows = 1, kErrLabel = 2, kErrSlot = 3, kErrWait = 4 };

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace pb
