// Stage split over several GPUs (Section 2.1: stages split over GPUs, one host
// thread per GPU; Appendix "Batch Parallel vs Pipeline Parallel Computation":
// a worker only exchanges one activation forward and one gradient backward with
// its neighbours).  Every rank owns a contiguous range of stages.  At the end
// of its tick t a rank stores, with plain stores, the output its last stage made
// for the sample it forwarded into the NEXT rank's copy of that stage's output
// ring, and the input gradient its first stage made into the PREVIOUS rank's
// copy of that hand-off buffer, each followed by a tick stamp (t + 1) in the
// receiver's memory.  What a rank consumes at tick t was produced by its
// neighbours at tick t - 1 at the latest, so before its own kernels of tick t
// it waits until both stamps have reached t; the wait is bounded and reports
// through the engine's error word.  No bulk tensor copy and no collective is
// involved: the receiver's memory is written through ordinary peer stores.
#pragma once
#include "fc_kernels.cuh"

namespace pb {

constexpr long long kSplitWaitNs = 1000LL * 1000 * 1000;     // a neighbour has one second to deliver

struct SplitLinks {
    // receive side (this rank's own memory, written by the neighbours)
    volatile long long* act_stamp;     // ticks of the previous rank whose activation has landed
    volatile long long* grad_stamp;    // ticks of the next rank whose gradient has landed
    // send side
    const float* act_src; int act_slots, act_dim, act_stage;      // own last stage: output ring
    float* act_dst; volatile long long* act_dst_stamp;            // next rank's copy and stamp (nullptr: no next rank)
    const float* grad_src; int grad_slots, grad_nparts, grad_dim, grad_stage;   // own first stage: input-gradient hand-off
    float* grad_dst; volatile long long* grad_dst_stamp;          // previous rank's copy and stamp (nullptr: no previous rank)
};

__device__ __forceinline__ long long split_now_ns() {
    long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Start of a tick: wait for the neighbours' previous tick and file the label.
__global__ void split_wait_kernel(SplitLinks L, TickState* ts, int par, int* __restrict__ label_ring, int S,
                                  const int* __restrict__ labels, int label_value, long long t_base,
                                  float* __restrict__ nan_losses) {
    if (threadIdx.x != 0) return;
    const long long t = ts->cnt[par];
    if (nan_losses) nan_losses[t - t_base] = __int_as_float(0x7fc00000);      // this rank has no loss: the last stage is elsewhere
    if (label_ring) label_ring[t % S] = labels ? labels[t - t_base] : label_value;
    const long long t0 = split_now_ns();
    bool ok = true;
    if (L.act_stamp) while (*L.act_stamp < t) { if (split_now_ns() - t0 > kSplitWaitNs) { ok = false; break; } }
    if (ok && L.grad_stamp) while (*L.grad_stamp < t) { if (split_now_ns() - t0 > kSplitWaitNs) { ok = false; break; } }
    if (!ok) { ts->error = kErrWait; ts->error_info = -1; }
    __threadfence_system();
}

// End of a tick: hand this tick's boundary activation and gradient to the neighbours.
// Launched after the tick counter has advanced: `par` is the parity of the tick that just ran.
__global__ void __launch_bounds__(256)
split_handoff_kernel(SplitLinks L, const TickState* __restrict__ ts, int par, int S) {
    const long long t = ts->cnt[par ^ 1] - 1;            // the tick that has just been computed
    if (L.act_dst) {
        const long long i = t - L.act_stage;              // sample forwarded by the last own stage
        if (sample_live(ts, i)) {
            const size_t off = (size_t)ring_slot(i, L.act_slots) * L.act_dim;
            for (int k = threadIdx.x; k < L.act_dim; k += blockDim.x) L.act_dst[off + k] = L.act_src[off + k];
        }
    }
    if (L.grad_dst) {
        const long long j = t - 2LL * (S - 1) + L.grad_stage;      // sample back-propagated by the first own stage
        if (sample_live(ts, j)) {
            const size_t slot = (size_t)ring_slot(j, L.grad_slots);
            const float* src = L.grad_src + slot * L.grad_nparts * L.grad_dim;
            for (int k = threadIdx.x; k < L.grad_dim; k += blockDim.x) {
                float a = 0.f;
                for (int q = 0; q < L.grad_nparts; ++q) a += src[(size_t)q * L.grad_dim + k];    // partial rows in table order
                L.grad_dst[slot * L.grad_dim + k] = a;
            }
        }
    }
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x == 0) {
        if (L.act_dst_stamp) *L.act_dst_stamp = t + 1;
        if (L.grad_dst_stamp) *L.grad_dst_stamp = t + 1;
        __threadfence_system();
    }
}

}  // namespace pb
