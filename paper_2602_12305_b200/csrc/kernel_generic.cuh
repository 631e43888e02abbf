// Generic variant: fully predicated 64x64 FMA tiles for any shape, alignment and dtype.
// It is the catch-all behind the fast variants (ragged or unaligned problems) and an
// on-device cross-check for them; correctness first, speed second.
#pragma once

#include "common.cuh"

namespace optiml {

constexpr int kGenBM = 64, kGenBN = 64, kGenBK = 16, kGenThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kGenThreads)
gemm_generic_kernel(const T* __restrict__ A, const T* __restrict__ B, const T* __restrict__ bias,
                    T* __restrict__ Y, int M, int N, int K, int act) {
    // As is stored k-major (transposed) so the inner product reads both operands as float4.
    __shared__ __align__(16) float As[kGenBK][kGenBM + 4];
    __shared__ __align__(16) float Bs[kGenBK][kGenBN];

    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    // 1-D grid, N tiles fastest
    const int tiles_n = (N + kGenBN - 1) / kGenBN;
    const int64_t m0 = (int64_t)(blockIdx.x / tiles_n) * kGenBM;
    const int64_t n0 = (int64_t)(blockIdx.x % tiles_n) * kGenBN;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

    for (int64_t k0 = 0; k0 < K; k0 += kGenBK) {
#pragma unroll
        for (int e = tid; e < kGenBM * kGenBK; e += kGenThreads) {
            const int r = e / kGenBK, c = e % kGenBK;
            const int64_t m = m0 + r, k = k0 + c;
            As[c][r] = (m < M && k < K) ? to_f32(A[m * K + k]) : 0.0f;
        }
#pragma unroll
        for (int e = tid; e < kGenBK * kGenBN; e += kGenThreads) {
            const int r = e / kGenBN, c = e % kGenBN;
            const int64_t k = k0 + r, n = n0 + c;
            Bs[r][c] = (k < K && n < N) ? to_f32(B[k * N + n]) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kGenBK; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w};
            const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t n = n0 + tx * 4 + j;
            if (n >= N) continue;
            const float bv = bias ? to_f32(bias[n]) : 0.0f;
            // tanhf for fp32 output, hardware tanh for bf16 output
            const float y = sizeof(T) == 4 ? epilogue_rt<false>(acc[i][j], bv, act)
                                           : epilogue_rt<true>(acc[i][j], bv, act);
            Y[m * N + n] = from_f32<T>(y);
        }
    }
}

}  // namespace optiml
