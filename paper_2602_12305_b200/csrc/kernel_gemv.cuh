// GEMV / very skinny variant (bf16, M <= 4): the problem is a stream over B, so the
// kernel is organised around HBM: every lane issues 128-bit non-allocating loads of B
// (8 bf16 columns), a warp covers one 512-byte row segment per load, eight warps take
// interleaved rows, and kGemvUnroll independent loads per thread are in flight before the
// first FMA.  K is split across gridDim.y CTAs so that the grid fills every SM once
// (gemv_ctas_per_sm CTAs per SM).
//
// Reduction of the K slices: warps -> shared memory (fixed order) -> CTA partial in the
// handle's scratch; the CTA that arrives last on a column block (atomic counter, no
// waiting anywhere) sums the slices in slice order, applies bias + activation in
// registers and stores Y once.  The order is fixed, so results are reproducible.
#pragma once

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

constexpr int kGemvCols = 256;     // columns per CTA: 32 lanes x 8 bf16
constexpr int kGemvWarps = 8;
constexpr int kGemvThreads = kGemvWarps * 32;
// Measured on B200 (1 x 8192 x 8192): many resident warps with few loads each beat few
// warps with deep unrolling -- 4 loads in flight per thread and 5 CTAs per SM (40 warps)
// stream at 5.5 TB/s, 8 loads and 2 CTAs at 4.5 TB/s.
constexpr int kGemvUnroll = 4;
// resident CTAs per SM: M = 1 needs few registers; 2-4 rows of A need more accumulators
constexpr int gemv_ctas_per_sm(int mr) { return mr == 1 ? 5 : 2; }

template <int MR>
__global__ void __launch_bounds__(kGemvThreads, gemv_ctas_per_sm(MR))
gemv_splitk_kernel(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ B,
                   const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ Y,
                   int M, int N, int K, int act, float* __restrict__ partials, unsigned int* __restrict__ counters) {
    __shared__ float red[kGemvWarps][MR][kGemvCols];
    __shared__ int s_last;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cb = blockIdx.x, slice = blockIdx.y, S = gridDim.y;
    const int64_t n = (int64_t)cb * kGemvCols + lane * 8;
    const bool n_ok = n < N;                                   // N % 8 == 0: all 8 columns or none
    const int k_begin = (int)((int64_t)K * slice / S);
    const int k_end = (int)((int64_t)K * (slice + 1) / S);

    float acc[MR][8];
#pragma unroll
    for (int m = 0; m < MR; ++m)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[m][j] = 0.0f;

    // launched as a programmatic dependent: wait for the previous kernel before touching memory
    ptx::griddep_wait();
    ptx::griddep_launch_dependents();

    const __nv_bfloat16* bp = B + n;
    for (int kb = k_begin + warp; kb < k_end; kb += kGemvWarps * kGemvUnroll) {
        uint4 v[kGemvUnroll];
        float a[kGemvUnroll][MR];
#pragma unroll
        for (int u = 0; u < kGemvUnroll; ++u) {
            const int k = kb + u * kGemvWarps;
            const bool ok = n_ok && k < k_end;
            v[u] = ok ? ld_stream_v4(bp + (int64_t)k * N) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int m = 0; m < MR; ++m)
                a[u][m] = (k < k_end && m < M) ? __bfloat162float(A[(int64_t)m * K + k]) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < kGemvUnroll; ++u) {
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float b0 = bf16lo_to_f32(w[q]), b1 = bf16hi_to_f32(w[q]);
#pragma unroll
                for (int m = 0; m < MR; ++m) {
                    acc[m][2 * q] = fmaf(a[u][m], b0, acc[m][2 * q]);
                    acc[m][2 * q + 1] = fmaf(a[u][m], b1, acc[m][2 * q + 1]);
                }
            }
        }
    }

    // warps -> shared memory
#pragma unroll
    for (int m = 0; m < MR; ++m)
#pragma unroll
        for (int j = 0; j < 8; ++j) red[warp][m][lane * 8 + j] = acc[m][j];
    __syncthreads();

    const int t = threadIdx.x;                 // one output column per thread from here on
    const int64_t col = (int64_t)cb * kGemvCols + t;
    float sum[MR];
#pragma unroll
    for (int m = 0; m < MR; ++m) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < kGemvWarps; ++w) s += red[w][m][t];
        sum[m] = s;
    }

    if (S > 1) {
        float* mine = partials + ((size_t)cb * S + slice) * (MR * kGemvCols);
#pragma unroll
        for (int m = 0; m < MR; ++m) mine[m * kGemvCols + t] = sum[m];
        __threadfence();
        __syncthreads();
        if (t == 0) {
            const unsigned int prev = atomicAdd(&counters[cb], 1u);
            s_last = (prev == (unsigned int)(S - 1));
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        const float* all = partials + (size_t)cb * S * (MR * kGemvCols);
        // slices in order, eight loads in flight at a time (one dependent chain of L2 round
        // trips per slice would cost more than the whole stream over B)
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            float s = 0.0f;
            for (int q0 = 0; q0 < S; q0 += 8) {
                float v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    v[i] = (q0 + i < S) ? __ldcg(all + (size_t)(q0 + i) * (MR * kGemvCols) + m * kGemvCols + t) : 0.0f;
#pragma unroll
                for (int i = 0; i < 8; ++i) s += v[i];
            }
            sum[m] = s;
        }
        if (t == 0) counters[cb] = 0u;         // ready for the next call on this stream
    }

    if (col < N) {
        const float bv = bias ? __bfloat162float(bias[col]) : 0.0f;
#pragma unroll
        for (int m = 0; m < MR; ++m)
            if (m < M) Y[(int64_t)m * N + col] = __float2bfloat16_rn(epilogue_rt<true>(sum[m], bv, act));
    }
}

}  // namespace optiml
