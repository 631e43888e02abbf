// The K-reduction on its own: sum, dot product and mean squared error of fp32 vectors
// (the paper's Prompts appendix, tasks 14, 15 and 7), as single-pass streaming kernels.
//
// One pass over HBM: every thread walks the vectors with 128-bit loads in a grid-stride
// loop, eight float4 in flight, sixteen or more independent fp32 accumulators per
// thread (so no accumulator sees more than about n / (threads * 16) terms); they are
// folded in fp64, lanes are combined with warp shuffles, warps through shared memory, and
// each CTA parks one fp64 partial in the handle's scratch.  The CTA that arrives last on
// the counter (nobody waits) adds the partials in CTA order and writes the fp32 result.
// Every order is fixed, so the result is reproducible for a given n and device.
#pragma once

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

enum : int { kReduceSum = 0, kReduceDot = 1, kReduceMse = 2 };
constexpr int kReduceThreads = 256;
constexpr int kReduceCtasPerSm = 4;    // 64 registers per thread: the accumulators and 8 loads in flight stay in registers

template <int KIND>
__device__ __forceinline__ float reduce_term(float x, float y) {
    if (KIND == kReduceSum) return x;
    if (KIND == kReduceDot) return x * y;
    const float d = x - y;
    return d * d;
}

template <int KIND>
__global__ void __launch_bounds__(kReduceThreads, kReduceCtasPerSm)
reduce_f32_kernel(const float* __restrict__ x, const float* __restrict__ y, int64_t n, float* __restrict__ out,
                  double* __restrict__ partials, unsigned int* __restrict__ counter) {
    __shared__ double warp_sums[kReduceThreads / 32];
    __shared__ int s_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    ptx::griddep_wait();                      // launched as a programmatic dependent
    ptx::griddep_launch_dependents();

    // loads in flight per thread and trip: 8 float4 either way (one vector: 8, two vectors: 4 + 4)
    constexpr int U = KIND == kReduceSum ? 8 : 4;
    float acc[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[u][j] = 0.0f;

    // body: whole float4s (the pointers are 16-byte aligned), four per thread per trip
    const int64_t n4 = n / 4;
    const int64_t stride = (int64_t)gridDim.x * kReduceThreads;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const float4* y4 = reinterpret_cast<const float4*>(y);
    for (int64_t i = (int64_t)blockIdx.x * kReduceThreads + threadIdx.x; i < n4; i += U * stride) {
        float4 vx[U], vy[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t k = i + u * stride;
            vx[u] = k < n4 ? __ldcs(x4 + k) : make_float4(0, 0, 0, 0);
            if (KIND != kReduceSum) vy[u] = k < n4 ? __ldcs(y4 + k) : make_float4(0, 0, 0, 0);
            else vy[u] = make_float4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            acc[u][0] += reduce_term<KIND>(vx[u].x, vy[u].x);
            acc[u][1] += reduce_term<KIND>(vx[u].y, vy[u].y);
            acc[u][2] += reduce_term<KIND>(vx[u].z, vy[u].z);
            acc[u][3] += reduce_term<KIND>(vx[u].w, vy[u].w);
        }
    }
    double s = 0.0;
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int j = 0; j < 4; ++j) s += (double)acc[u][j];
    // tail: the last n % 4 elements, by the first threads of CTA 0
    if (blockIdx.x == 0 && threadIdx.x < (int)(n - n4 * 4)) {
        const int64_t k = n4 * 4 + threadIdx.x;
        s += (double)reduce_term<KIND>(x[k], KIND == kReduceSum ? 0.0f : y[k]);
    }

    // lanes -> warp (shuffles), warps -> CTA (shared memory), fixed order
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_down_sync(0xffffffffu, s, off);
    if (lane == 0) warp_sums[warp] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double c = 0.0;
#pragma unroll
        for (int w = 0; w < kReduceThreads / 32; ++w) c += warp_sums[w];
        partials[blockIdx.x] = c;
        __threadfence();
        const unsigned int prev = atomicAdd(counter, 1u);
        s_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // last CTA: partials in CTA order, 256 at a time
    double t = 0.0;
    for (unsigned int b = threadIdx.x; b < gridDim.x; b += kReduceThreads) t += __ldcg(partials + b);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_down_sync(0xffffffffu, t, off);
    if (lane == 0) warp_sums[warp] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        double c = 0.0;
#pragma unroll
        for (int w = 0; w < kReduceThreads / 32; ++w) c += warp_sums[w];
        if (KIND == kReduceMse) c /= (double)n;
        *out = (float)c;
        *counter = 0u;                        // re-armed for the next call
    }
}

}  // namespace optiml
