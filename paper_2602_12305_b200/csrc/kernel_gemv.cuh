// GEMV / very skinny variant (M <= 4; bf16 or fp32): the problem is a stream over B, so
// the kernel is organised around HBM: every lane issues 128-bit non-allocating loads of B
// (8 bf16 or 4 fp32 columns), a warp covers one 512-byte row segment per load, eight warps
// take interleaved rows, and kGemvUnroll independent loads per thread are in flight before
// the first FMA.  K is split across gridDim.y CTAs so that the grid fills every SM once
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

constexpr int kGemvWarps = 8;
constexpr int kGemvThreads = kGemvWarps * 32;
// Measured on B200 (1 x 8192 x 8192 bf16): many resident warps with few loads each beat few
// warps with deep unrolling -- 4 loads in flight per thread and 5 CTAs per SM (40 warps)
// stream at 5.5 TB/s, 8 loads and 2 CTAs at 4.5 TB/s.
constexpr int kGemvUnroll = 4;
// resident CTAs per SM: M = 1 needs few registers; 2-4 rows of A need more accumulators
constexpr int gemv_ctas_per_sm(int mr) { return mr == 1 ? 5 : 2; }

// columns per 16-byte load and per CTA (32 lanes)
template <typename T> struct GemvVec { static constexpr int V = 16 / (int)sizeof(T); static constexpr int kCols = 32 * V; };
constexpr int kGemvCols = GemvVec<__nv_bfloat16>::kCols;       // 256 (bf16); fp32: 128

__device__ __forceinline__ void gemv_unpack(const uint4& v, float (&b)[8], __nv_bfloat16) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        b[2 * q] = bf16lo_to_f32(w[q]);
        b[2 * q + 1] = bf16hi_to_f32(w[q]);
    }
}
__device__ __forceinline__ void gemv_unpack(const uint4& v, float (&b)[4], float) {
    b[0] = __uint_as_float(v.x);
    b[1] = __uint_as_float(v.y);
    b[2] = __uint_as_float(v.z);
    b[3] = __uint_as_float(v.w);
}

template <typename T, int MR>
__global__ void __launch_bounds__(kGemvThreads, gemv_ctas_per_sm(MR))
gemv_splitk_kernel(const T* __restrict__ A, const T* __restrict__ B, const T* __restrict__ bias, T* __restrict__ Y,
                   int M, int N, int K, int act, float* __restrict__ partials, unsigned int* __restrict__ counters,
                   int prefetch_rows) {
    constexpr int V = GemvVec<T>::V, kCols = GemvVec<T>::kCols;
    __shared__ float red[kGemvWarps][MR][kCols];
    __shared__ int s_last;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cb = blockIdx.x, slice = blockIdx.y, S = gridDim.y;
    const int64_t n = (int64_t)cb * kCols + lane * V;
    const bool n_ok = n < N;                                   // N % V == 0: all V columns or none
    const int k_begin = (int)((int64_t)K * slice / S);
    const int k_end = (int)((int64_t)K * (slice + 1) / S);

    float acc[MR][V];
#pragma unroll
    for (int m = 0; m < MR; ++m)
#pragma unroll
        for (int j = 0; j < V; ++j) acc[m][j] = 0.0f;

    // Launched as a programmatic dependent, this CTA may be running while the previous kernel
    // still drains.  Nothing may be read or written before the wait below, but the first rows of
    // this CTA's slice of B can be pulled from DRAM into L2 meanwhile (one 512-byte row segment
    // per thread and instruction), so that HBM does not idle across the kernel boundary.
    if (prefetch_rows > 0 && (int64_t)cb * kCols < N) {
        const int64_t n0 = (int64_t)cb * kCols;
        const uint32_t seg = (uint32_t)((N - n0 < kCols ? N - n0 : kCols) * (int64_t)sizeof(T));   // multiple of 16
        const int rows = k_end - k_begin < prefetch_rows ? k_end - k_begin : prefetch_rows;
        for (int r = threadIdx.x; r < rows; r += kGemvThreads)
            ptx::prefetch_l2_bulk(B + (int64_t)(k_begin + r) * N + n0, seg);
    }
    ptx::griddep_wait();
    ptx::griddep_launch_dependents();

    const T* bp = B + n;
    for (int kb = k_begin + warp; kb < k_end; kb += kGemvWarps * kGemvUnroll) {
        uint4 v[kGemvUnroll];
        float a[kGemvUnroll][MR];
#pragma unroll
        for (int u = 0; u < kGemvUnroll; ++u) {
            const int k = kb + u * kGemvWarps;
            const bool ok = n_ok && k < k_end;
            v[u] = ok ? ld_stream_v4(bp + (int64_t)k * N) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int m = 0; m < MR; ++m) a[u][m] = (k < k_end && m < M) ? to_f32(A[(int64_t)m * K + k]) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < kGemvUnroll; ++u) {
            float b[V];
            gemv_unpack(v[u], b, T());
#pragma unroll
            for (int j = 0; j < V; ++j)
#pragma unroll
                for (int m = 0; m < MR; ++m) acc[m][j] = fmaf(a[u][m], b[j], acc[m][j]);
        }
    }

    // warps -> shared memory
#pragma unroll
    for (int m = 0; m < MR; ++m)
#pragma unroll
        for (int j = 0; j < V; ++j) red[warp][m][lane * V + j] = acc[m][j];
    __syncthreads();

    const int t = threadIdx.x;                 // one output column per thread from here on
    const bool has_col = t < kCols;            // fp32: the upper half of the CTA has no column
    const int64_t col = (int64_t)cb * kCols + t;
    float sum[MR];
#pragma unroll
    for (int m = 0; m < MR; ++m) {
        float s = 0.0f;
        if (has_col) {
#pragma unroll
            for (int w = 0; w < kGemvWarps; ++w) s += red[w][m][t];
        }
        sum[m] = s;
    }

    if (S > 1) {
        float* mine = partials + ((size_t)cb * S + slice) * (MR * kCols);
        if (has_col) {
#pragma unroll
            for (int m = 0; m < MR; ++m) mine[m * kCols + t] = sum[m];
        }
        __threadfence();
        __syncthreads();
        if (t == 0) {
            const unsigned int prev = atomicAdd(&counters[cb], 1u);
            s_last = (prev == (unsigned int)(S - 1));
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        const float* all = partials + (size_t)cb * S * (MR * kCols);
        // slices in order, kBatch loads in flight at a time (one dependent chain of L2 round
        // trips per slice would cost more than the whole stream over B; a single row of A leaves
        // the registers for 24 at once, which covers the 23 slices of 1 x 8192 x 8192 in one trip)
        constexpr int kBatch = MR == 1 ? 24 : 8;
        if (has_col) {
#pragma unroll
            for (int m = 0; m < MR; ++m) {
                float s = 0.0f;
                for (int q0 = 0; q0 < S; q0 += kBatch) {
                    float v[kBatch];
#pragma unroll
                    for (int i = 0; i < kBatch; ++i)
                        v[i] = (q0 + i < S) ? __ldcg(all + (size_t)(q0 + i) * (MR * kCols) + m * kCols + t) : 0.0f;
#pragma unroll
                    for (int i = 0; i < kBatch; ++i) s += v[i];
                }
                sum[m] = s;
            }
        }
        if (t == 0) counters[cb] = 0u;         // ready for the next call on this stream
    }

    if (has_col && col < N) {
        const float bv = bias ? to_f32(bias[col]) : 0.0f;
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            if (m >= M) continue;
            // tanhf / expf for fp32 output, the hardware approximations for bf16 output
            const float y = sizeof(T) == 4 ? epilogue_rt<false>(sum[m], bv, act) : epilogue_rt<true>(sum[m], bv, act);
            Y[(int64_t)m * N + col] = from_f32<T>(y);
        }
    }
}

}  // namespace optiml
