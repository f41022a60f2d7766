// Two small measurement kernels that give the roofline denominators which a plain
// HBM copy does not: the bandwidth of a read-modify-write sweep over a buffer that
// stays in the L2 cache (the regime of networks whose weights and velocities fit
// there), and the float32 fused-multiply-add rate of the CUDA cores (the bound of
// the float32 convolutions).
#pragma once
#include <cuda_runtime.h>

namespace pb {

// x <- a x + b over n float4: one 16-byte load and one 16-byte store per element,
// the access pattern of the update kernels.
__global__ void __launch_bounds__(256)
l2_sweep_kernel(float4* __restrict__ x, size_t n, float a, float b) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float4 v = x[i];
        v.x = fmaf(a, v.x, b); v.y = fmaf(a, v.y, b); v.z = fmaf(a, v.z, b); v.w = fmaf(a, v.w, b);
        x[i] = v;
    }
}

// 16 independent fused-multiply-add chains per thread, `iters` links each.
__global__ void __launch_bounds__(256)
fma_chain_kernel(float* __restrict__ out, int iters, float a, float b) {
    float r[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) r[k] = (float)(threadIdx.x + k) * 1e-3f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int k = 0; k < 16; ++k) r[k] = fmaf(r[k], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < 16; ++k) s += r[k];
    if (s == 123.456f) out[blockIdx.x * blockDim.x + threadIdx.x] = s;     // keeps the chains alive
}

}  // namespace pb
