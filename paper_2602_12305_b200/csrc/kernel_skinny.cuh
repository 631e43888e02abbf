// Skinny variant (bf16, M <= 128): the problem is a single pass over B, so it is laid
// out as a stream over HBM, but the multiply-accumulates go to the tensor cores: at
// M = 16 the FMA pipes cannot keep up with HBM (about 100 TFLOP/s would be needed).
//
// Operands are swapped: the MMA computes Y^T tiles, D[n, m] = sum_k B[k, n] A[m, k].
//   MMA "A" operand = a 128(n) x 64(k) tile of B, N contiguous (MN-major), two 64-column
//                     TMA boxes with 128-byte swizzle;
//   MMA "B" operand = the MP x 64 tile of A (rows >= M are zero-filled by TMA), K-major;
//   accumulator     = 128 TMEM lanes (n) x MP fp32 columns (m), double buffered.
//
// Work is cut stream-K style: the (column tile, K block) units, in column-tile-major
// order, are dealt in equal contiguous ranges to one CTA per SM, so every SM streams the
// same number of bytes whatever N and K are.  A CTA's range is a sequence of segments
// (one column tile, a range of K blocks).  A segment spanning all of K goes straight
// through the fused epilogue.  Otherwise the fp32 partial tile is written to the handle's
// scratch and an arrival counter per column tile is bumped; the CTA that arrives last
// (nobody waits) adds the partials in K order, applies bias + activation and stores Y.
// The order of the sum is fixed, so results are reproducible.
//
// Roles: warp 0 TMA producer, warp 1 TMEM allocation + MMA issue, warps 2-5 epilogue.
// All mbarrier waits are bounded; see kernel_umma.cuh for the tear-down protocol.
#pragma once

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

template <int MP>
struct SkinnyCfg {
    static_assert(MP == 16 || MP == 32 || MP == 64 || MP == 128, "padded M");
    static constexpr int BN = 128, BK = 64;
    static constexpr int kBChunkBytes = BK * 64 * 2;           // 64 k-rows x 64 columns: 8 KiB
    static constexpr int kBBytes = 2 * kBChunkBytes;           // 16 KiB
    static constexpr int kABytes = MP * BK * 2;
    static constexpr int kStageBytes = kBBytes + kABytes;      // multiple of 1024
    static constexpr int kMaxStages = 12;
    static constexpr int kFit = (216 * 1024) / kStageBytes;
    static constexpr int kStages = kFit < kMaxStages ? kFit : kMaxStages;
    static constexpr int kThreads = 192;
    static constexpr int kTmemCols = 2 * MP < 32 ? 32 : 2 * MP;
    static constexpr int kChunk = MP < 32 ? MP : 32;           // accumulator columns per tcgen05.ld
    static constexpr int kSmemBytes = kStages * kStageBytes + 512 + 1024;
    static constexpr int kSlotFloats = MP * BN;                // one partial tile in scratch
};

template <int MP>
struct SkinnyShared {
    uint64_t full[SkinnyCfg<MP>::kStages];
    uint64_t empty[SkinnyCfg<MP>::kStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
    int last_flag;
};

// Stream-K bookkeeping: U units over G CTAs; CTA c owns units [U*c/G, U*(c+1)/G).
__device__ __forceinline__ int64_t sk_begin(int64_t U, int G, int c) { return U * c / G; }
__device__ __forceinline__ int sk_owner(int64_t U, int G, int64_t u) { return (int)(((u + 1) * G + U - 1) / U - 1); }

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int MP>
__global__ void __launch_bounds__(SkinnyCfg<MP>::kThreads, 1)
gemm_skinny_umma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                        const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ Y, int M, int N, int K,
                        int act, float* __restrict__ partials, unsigned int* __restrict__ counters,
                        int* __restrict__ status) {
    using C = SkinnyCfg<MP>;
    using Sh = SkinnyShared<MP>;
    static_assert(sizeof(Sh) <= 512, "barrier block");
    extern __shared__ uint8_t smem_raw[];
    Sh* sh = reinterpret_cast<Sh*>(smem_raw);
    const uint32_t ring_base = (ptx::smem_u32(smem_raw) + 512 + 1023) & ~1023u;
    uint8_t* ring = smem_raw + (ring_base - ptx::smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, c = blockIdx.x;
    const int KB = (K + C::BK - 1) / C::BK;
    const int tiles_n = (N + C::BN - 1) / C::BN;
    const int64_t U = (int64_t)tiles_n * KB;
    const int64_t u0 = sk_begin(U, G, c), u1 = sk_begin(U, G, c + 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(&sh->full[s], 1);
            ptx::mbar_init(&sh->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&sh->tmem_full[a], 1);
            ptx::mbar_init(&sh->tmem_empty[a], 128);
        }
        ptx::mbar_init(&sh->drain, 1);
        sh->abort = 0;
        sh->last_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(&sh->tmem_base, C::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    ptx::tcgen05_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&map_a);
            ptx::prefetch_tensormap(&map_b);
            const uint64_t pol_stream = ptx::policy_evict_first();   // B is read exactly once
            const uint64_t pol_keep = ptx::policy_evict_last();      // A is re-read by every CTA
            uint32_t it = 0;
            bool ok = true;
            for (int64_t u = u0; u < u1; ++u, ++it) {
                const int tile = (int)(u / KB), kb = (int)(u % KB);
                const int s = it % C::kStages;
                const uint32_t ph = (it / C::kStages) & 1;
                if (sh->abort || !ptx::mbar_wait(&sh->empty[s], ph ^ 1)) { ok = false; break; }
                uint8_t* b_dst = ring + s * C::kStageBytes;
                uint8_t* a_dst = b_dst + C::kBBytes;
                ptx::mbar_arrive_expect_tx(&sh->full[s], C::kStageBytes);
                ptx::tma_load_2d_hint(b_dst, &map_b, &sh->full[s], tile * C::BN, kb * C::BK, pol_stream);
                ptx::tma_load_2d_hint(b_dst + C::kBChunkBytes, &map_b, &sh->full[s], tile * C::BN + 64, kb * C::BK,
                                      pol_stream);
                ptx::tma_load_2d_hint(a_dst, &map_a, &sh->full[s], kb * C::BK, 0, pol_keep);
            }
            if (!ok) {
                atomicExch(status, kDevTimeout);
                sh->abort = 1;
                const uint32_t n_back = it < (uint32_t)C::kStages ? it : (uint32_t)C::kStages;
                for (uint32_t b = 1; b <= n_back; ++b) {
                    const uint32_t j = it - b;
                    ptx::mbar_wait(&sh->full[j % C::kStages], (j / C::kStages) & 1);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(C::BN, MP, /*a_mn_major=*/true, /*b_mn_major=*/false);
            uint32_t it = 0, seg_it = 0;
            bool ok = true;
            for (int64_t u = u0; u < u1 && ok; ++seg_it) {
                const int kb0 = (int)(u % KB);
                const int64_t left = u1 - u;
                const int kb1 = (int)(left < KB - kb0 ? kb0 + left : KB);
                const int a = seg_it & 1;
                const uint32_t aph = (seg_it >> 1) & 1;
                if (sh->abort || !ptx::mbar_wait(&sh->tmem_empty[a], aph ^ 1)) { ok = false; break; }
                ptx::tcgen05_fence_after_sync();
                const uint32_t d_tmem = tmem_base + a * MP;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1;
                    if (sh->abort || !ptx::mbar_wait(&sh->full[s], ph)) { ok = false; break; }
                    ptx::tcgen05_fence_after_sync();
                    const uint32_t b_addr = ring_base + s * C::kStageBytes;   // tile of B
                    const uint32_t a_addr = b_addr + C::kBBytes;              // tile of A
#pragma unroll
                    for (int k4 = 0; k4 < C::BK / 16; ++k4) {
                        const uint64_t da = ptx::umma_smem_desc(b_addr + k4 * 2048, C::kBChunkBytes, 1024);
                        const uint64_t db = ptx::umma_smem_desc(a_addr + k4 * 32, 16, 1024);
                        ptx::umma_bf16(d_tmem, da, db, idesc, (kb != kb0) || (k4 != 0));
                    }
                    ptx::umma_commit(&sh->empty[s]);
                }
                if (ok) ptx::umma_commit(&sh->tmem_full[a]);
                u += kb1 - kb0;
            }
            if (!ok) {
                atomicExch(status, kDevTimeout);
                sh->abort = 1;
            }
            ptx::umma_commit(&sh->drain);
            ptx::mbar_wait(&sh->drain, 0);
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int q = warp & 3;
        const int r = q * 32 + lane;                      // n within the column tile = TMEM lane
        const int et = threadIdx.x - 64;                  // 0..127 among the epilogue threads
        const int m_valid = M < MP ? M : MP;
        uint32_t seg_it = 0;
        bool ok = true;
        for (int64_t u = u0; u < u1 && ok; ++seg_it) {
            const int tile = (int)(u / KB), kb0 = (int)(u % KB);
            const int64_t left = u1 - u;
            const int kb1 = (int)(left < KB - kb0 ? kb0 + left : KB);
            const bool whole = (kb0 == 0 && kb1 == KB);
            const int a = seg_it & 1;
            const uint32_t aph = (seg_it >> 1) & 1;
            bool got = !sh->abort && ptx::mbar_wait(&sh->tmem_full[a], aph);
            got = __all_sync(0xffffffffu, got);
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();

            const int64_t n = (int64_t)tile * C::BN + r;
            const float bv = (bias && n < N) ? __bfloat162float(bias[n]) : 0.0f;
            float* slot = partials + ((size_t)2 * c + (u == u0 ? 0 : 1)) * C::kSlotFloats;
#pragma unroll 1
            for (int m0 = 0; m0 < MP; m0 += C::kChunk) {
                uint32_t v[C::kChunk];
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * MP + m0;
                if constexpr (C::kChunk == 16) ptx::tmem_ld_32x16(taddr, v);
                else ptx::tmem_ld_32x32(taddr, v);
                ptx::tmem_ld_wait();
                if (whole) {
#pragma unroll
                    for (int j = 0; j < C::kChunk; ++j) {
                        const int m = m0 + j;
                        if (m < m_valid && n < N)
                            Y[(int64_t)m * N + n] = __float2bfloat16_rn(epilogue_rt<true>(__uint_as_float(v[j]), bv, act));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < C::kChunk; ++j)
                        if (m0 + j < m_valid) slot[(m0 + j) * C::BN + r] = __uint_as_float(v[j]);
                }
            }
            // accumulator read out: hand it back before the (slower) cross-CTA part
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive(&sh->tmem_empty[a]);

            if (!whole) {
                __threadfence();
                epi_bar_sync();
                const int64_t tile_first = (int64_t)tile * KB, tile_last = tile_first + KB - 1;
                const int c_first = sk_owner(U, G, tile_first), c_last = sk_owner(U, G, tile_last);
                if (et == 0) {
                    const unsigned int prev = atomicAdd(&counters[tile], 1u);
                    const int last = (prev == (unsigned int)(c_last - c_first));
                    if (last) counters[tile] = 0u;        // everyone has arrived: re-arm for the next call
                    sh->last_flag = last;
                }
                epi_bar_sync();
                if (sh->last_flag) {
                    __threadfence();
                    for (int m = 0; m < m_valid; ++m) {
                        float s = 0.0f;
                        for (int cc = c_first; cc <= c_last; ++cc) {
                            const int64_t b0 = sk_begin(U, G, cc);
                            const int which = (b0 >= tile_first) ? 0 : 1;   // segment starts at its CTA's range start?
                            const float* p = partials + ((size_t)2 * cc + which) * C::kSlotFloats;
                            s += __ldcg(p + m * C::BN + r);
                        }
                        if (n < N) Y[(int64_t)m * N + n] = __float2bfloat16_rn(epilogue_rt<true>(s, bv, act));
                    }
                }
            }
            u += kb1 - kb0;
        }
        if (!ok && lane == 0) {
            atomicExch(status, kDevTimeout);
            sh->abort = 1;
        }
    }

    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        ptx::tcgen05_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

}  // namespace optiml
