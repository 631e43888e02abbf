// fp32 variant: FMA-pipe tiles (no tensor cores, so no TF32 anywhere), 128-bit global
// loads, double-buffered shared memory with register prefetch, epilogue fused in
// registers.  Needs N % 4 == 0, K % 4 == 0 and 16-byte aligned pointers so that every
// float4 lies wholly inside or wholly outside the matrices; ragged tile edges in M, N
// and K are predicated per float4.
//
// Small problems (few tiles) additionally split K across kKS thread groups of one CTA
// and sum the groups through shared memory in a fixed order, which shortens the serial
// K loop when the grid cannot fill the machine.
#pragma once

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

constexpr int kF32BK = 16;

template <int BM, int BN, int TM, int TN, int KS>
struct F32Cfg {
    static constexpr int kGroup = (BM / TM) * (BN / TN);   // threads working on one K slice
    static constexpr int kThreads = kGroup * KS;
    static constexpr int kLdA = BM + 4;                    // padded, keeps float4 alignment
    static constexpr int kStage = kF32BK * kLdA + kF32BK * BN;   // floats per K-slice stage
    static constexpr int kSmemFloats = 2 * KS * kStage;
    // A thread's TM rows (TN columns) are TM / 4 (TN / 4) groups of four, the groups spread evenly
    // over the tile: neighbouring threads then read neighbouring float4s of a stage (no bank
    // conflict), where one block of 8 consecutive columns per thread made every other thread of a
    // quarter-warp hit the same banks.
    static constexpr int kRowGroupStride = BM / (TM / 4), kColGroupStride = BN / (TN / 4);
    // two CTAs per SM for the large tile (the compiler keeps it within 128 registers)
    static constexpr int kMinCtas = (BM == 128 && BN == 128 && KS == 1) ? 2 : 1;
    __host__ __device__ static constexpr int row_of(int ty, int i) { return (i / 4) * kRowGroupStride + ty * 4 + i % 4; }
    __host__ __device__ static constexpr int col_of(int tx, int j) { return (j / 4) * kColGroupStride + tx * 4 + j % 4; }
};

template <int BM, int BN, int TM, int TN, int KS, int ACT>
__global__ void __launch_bounds__(F32Cfg<BM, BN, TM, TN, KS>::kThreads, F32Cfg<BM, BN, TM, TN, KS>::kMinCtas)
gemm_f32_tiled_kernel(const float* __restrict__ A, const float* __restrict__ B, const float* __restrict__ bias,
                      float* __restrict__ Y, int M, int N, int K) {
    using C = F32Cfg<BM, BN, TM, TN, KS>;
    static_assert(TM % 4 == 0 && TN % 4 == 0, "micro-tile must be float4-sized");
    static_assert((BM * kF32BK / 4) % C::kGroup == 0 && (kF32BK * BN / 4) % C::kGroup == 0, "load split");
    constexpr int kAVec = BM * kF32BK / 4 / C::kGroup;     // float4 loads of A per thread per stage
    constexpr int kBVec = kF32BK * BN / 4 / C::kGroup;
    extern __shared__ __align__(16) float smem[];

    const int tid = threadIdx.x;
    const int ks = tid / C::kGroup;          // K slice of this thread
    const int g = tid % C::kGroup;
    const int tx = g % (BN / TN), ty = g / (BN / TN);
    // 1-D grid, N tiles fastest
    const int tiles_n = (N + BN - 1) / BN;
    const int64_t m0 = (int64_t)(blockIdx.x / tiles_n) * BM;
    const int64_t n0 = (int64_t)(blockIdx.x % tiles_n) * BN;

    // Launched as a programmatic dependent: before the wait on the previous kernel nothing may be
    // read, but this CTA's rows of A and columns of B can be pulled into L2 (a prefetch cannot
    // make a later load stale), so that the dependent global-load round trips of the K loop below
    // are L2 hits instead of DRAM accesses.  Small problems are pure latency: this is most of it.
    if (KS > 1) {
        for (int r = tid; r < BM; r += C::kThreads) {                 // A: BM rows of K floats
            const int64_t m = m0 + r;
            if (m < M) {
                const float* row = A + m * K;
                for (int64_t k = 0; k < K; k += 4096) ptx::prefetch_l2_bulk(row + k, (uint32_t)((K - k < 4096 ? K - k : 4096) * 4));
            }
        }
        const uint32_t seg = (uint32_t)((N - n0 < BN ? N - n0 : BN) * 4);     // B: K rows of BN floats
        for (int k = tid; k < K; k += C::kThreads) ptx::prefetch_l2_bulk(B + (int64_t)k * N + n0, seg);
    }
    ptx::griddep_wait();
    ptx::griddep_launch_dependents();

    // K is cut into KS contiguous slices of whole BK steps.
    const int steps_total = (K + kF32BK - 1) / kF32BK;
    const int steps_per = (steps_total + KS - 1) / KS;
    const int step_begin = ks * steps_per;
    const int step_end = min(steps_total, step_begin + steps_per);

    float* stage0 = smem + (size_t)ks * 2 * C::kStage;
    auto As = [&](int buf) { return stage0 + buf * C::kStage; };
    auto Bs = [&](int buf) { return stage0 + buf * C::kStage + kF32BK * C::kLdA; };

    float4 ra[kAVec], rb[kBVec];
    // What does not change from step to step is computed once: the thread's first source pointers at
    // k = 0 (its further float4s lie a fixed number of rows below) and whether its rows of A / columns of
    // B lie inside the matrices (one bit each).
    constexpr int kARowStep = C::kGroup / (kF32BK / 4);     // rows of A between a thread's consecutive float4s
    constexpr int kBRowStep = C::kGroup / (BN / 4);         // rows of B between a thread's consecutive float4s
    static_assert(C::kGroup % (kF32BK / 4) == 0 && C::kGroup % (BN / 4) == 0, "a thread keeps its column within a stage");
    const int a_r0 = g / (kF32BK / 4), a_c = (g % (kF32BK / 4)) * 4;
    const int b_r0 = g / (BN / 4), b_c = (g % (BN / 4)) * 4;
    const float* a_src = A + (m0 + a_r0) * K + a_c;
    const float* b_src = B + (int64_t)b_r0 * N + n0 + b_c;
    const bool b_live = n0 + b_c < N;
    unsigned a_live = 0;
#pragma unroll
    for (int i = 0; i < kAVec; ++i) a_live |= (m0 + a_r0 + i * kARowStep < M ? 1u : 0u) << i;
    auto load_global = [&](int step) {
        const int k0 = step * kF32BK;
#pragma unroll
        for (int i = 0; i < kAVec; ++i)
            ra[i] = ((a_live >> i) & 1u) && k0 + a_c < K
                        ? *reinterpret_cast<const float4*>(a_src + (int64_t)(i * kARowStep) * K + k0) : make_float4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < kBVec; ++i)
            rb[i] = b_live && k0 + b_r0 + i * kBRowStep < K
                        ? *reinterpret_cast<const float4*>(b_src + (int64_t)(k0 + i * kBRowStep) * N) : make_float4(0, 0, 0, 0);
    };
    auto store_shared = [&](int buf) {
        float* a = As(buf);
        float* b = Bs(buf);
#pragma unroll
        for (int i = 0; i < kAVec; ++i) {
            const int e = g + i * C::kGroup;
            const int r = e / (kF32BK / 4), c4 = e % (kF32BK / 4);
            a[(c4 * 4 + 0) * C::kLdA + r] = ra[i].x;
            a[(c4 * 4 + 1) * C::kLdA + r] = ra[i].y;
            a[(c4 * 4 + 2) * C::kLdA + r] = ra[i].z;
            a[(c4 * 4 + 3) * C::kLdA + r] = ra[i].w;
        }
#pragma unroll
        for (int i = 0; i < kBVec; ++i) {
            const int e = g + i * C::kGroup;
            const int r = e / (BN / 4), c4 = e % (BN / 4);
            *reinterpret_cast<float4*>(b + r * BN + c4 * 4) = rb[i];
        }
    };

    // accumulators as pairs of neighbouring columns: the operand form of the packed FMA below
    float2 acc2[TM][TN / 2];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN / 2; ++j) acc2[i][j] = make_float2(0.0f, 0.0f);

    // Every K slice runs the same number of loop trips so the barriers line up; a slice
    // that has run out of steps loads zeros (its step index is past the end of K).
    int buf = 0;
    load_global(step_begin);
    store_shared(0);
    __syncthreads();
    for (int s = 0; s < steps_per; ++s) {
        const int step = step_begin + s;
        if (s + 1 < steps_per) load_global(step + 1 < step_end ? step + 1 : steps_total);
        if (step < step_end) {
            const float* a = As(buf);
            const float* b = Bs(buf);
#pragma unroll
            for (int kk = 0; kk < kF32BK; ++kk) {
                __align__(16) float av[TM];
                __align__(16) float bv[TN];
#pragma unroll
                for (int i = 0; i < TM; i += 4)
                    *reinterpret_cast<float4*>(&av[i]) =
                        *reinterpret_cast<const float4*>(a + kk * C::kLdA + C::row_of(ty, i));
#pragma unroll
                for (int j = 0; j < TN; j += 4)
                    *reinterpret_cast<float4*>(&bv[j]) = *reinterpret_cast<const float4*>(b + kk * BN + C::col_of(tx, j));
                // packed FMAs (two fp32 lanes per instruction, each an ordinary round-to-nearest fp32
                // FMA): half the issue slots of 64 scalar FMAs, which leaves room for the loads
#pragma unroll
                for (int i = 0; i < TM; ++i) {
                    const float2 aa = make_float2(av[i], av[i]);
#pragma unroll
                    for (int j = 0; j < TN / 2; ++j)
                        acc2[i][j] = ptx::ffma2(aa, make_float2(bv[2 * j], bv[2 * j + 1]), acc2[i][j]);
                }
            }
        }
        if (s + 1 < steps_per) {
            store_shared(buf ^ 1);
            __syncthreads();
            buf ^= 1;
        }
    }

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN / 2; ++j) {
            acc[i][2 * j] = acc2[i][j].x;
            acc[i][2 * j + 1] = acc2[i][j].y;
        }

    if (KS > 1) {
        // Sum the K slices in slice order: slices 1..KS-1 park their tiles in shared memory
        // (the staging buffers are free now), slice 0 adds them one after another.
        __syncthreads();
        float* red = smem;   // (KS-1) x kGroup x (TM*TN)
        if (ks > 0) {
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) red[((size_t)(ks - 1) * TM * TN + i * TN + j) * C::kGroup + g] = acc[i][j];
        }
        __syncthreads();
        if (ks > 0) return;
        for (int q = 0; q < KS - 1; ++q)
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] += red[((size_t)q * TM * TN + i * TN + j) * C::kGroup + g];
    }

#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t m = m0 + C::row_of(ty, i);
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < TN; j += 4) {
            const int64_t n = n0 + C::col_of(tx, j);
            if (n >= N) continue;      // N % 4 == 0: the float4 is wholly inside or outside
            float4 bv = bias ? *reinterpret_cast<const float4*>(bias + n) : make_float4(0, 0, 0, 0);
            float4 o;
            o.x = epilogue<ACT, false>(acc[i][j + 0], bv.x);
            o.y = epilogue<ACT, false>(acc[i][j + 1], bv.y);
            o.z = epilogue<ACT, false>(acc[i][j + 2], bv.z);
            o.w = epilogue<ACT, false>(acc[i][j + 3], bv.w);
            *reinterpret_cast<float4*>(Y + m * N + n) = o;
        }
    }
}

}  // namespace optiml
