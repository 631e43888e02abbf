// Compute-bound variant (bf16): persistent, warp-specialised tcgen05 GEMM.
//
//   warp 0      TMA producer: A tile 128 x 64 (K-major) and B tile 64 x 256 (N contiguous,
//               i.e. MN-major for the MMA) into a kStages-deep ring of 128-byte swizzled
//               shared-memory buffers, one mbarrier pair (full/empty) per stage.
//   warp 1      allocates tensor memory, then one elected lane issues
//               tcgen05.mma.cta_group::1.kind::f16 (M=128, N=256, K=16), four per stage,
//               into one of two 128 x 256 fp32 accumulators in TMEM (2 x 256 = all 512
//               columns); tcgen05.commit frees the stage and, after the last K block,
//               publishes the accumulator.
//   warps 2-5   epilogue: tcgen05.ld the accumulator (each warp owns the TMEM lane quarter
//               32 * (warp % 4)), add bias, activate, round once to bf16 in registers and
//               store 64 contiguous bytes per thread; the other accumulator is being
//               filled meanwhile, so the epilogue hides under the next tile's MMAs.
//
// Tiles are walked in groups of 16 tile-rows so the CTAs running at the same time share
// A and B panels in L2.  Ragged M, N, K edges cost nothing special: TMA zero-fills
// out-of-range elements and the epilogue predicates its stores.  Needs N % 8 == 0 and
// K % 8 == 0 (16-byte global strides for TMA) and 16-byte aligned pointers.
//
// Every mbarrier wait is bounded.  A wait that gives up sets the status word, raises the
// CTA's abort flag and every role falls through to the common tear-down: the producer
// waits (bounded) for copies it still has in flight, the MMA lane waits (bounded) for its
// outstanding MMAs, then TMEM is freed.
#pragma once

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

struct UmmaCfg {
    static constexpr int BM = 128, BN = 256, BK = 64, kStages = 4;
    static constexpr int kABytes = BM * BK * 2;              // 16 KiB
    static constexpr int kBChunkBytes = BK * 64 * 2;         // one 64-column chunk: 8 KiB
    static constexpr int kBBytes = kBChunkBytes * (BN / 64); // 32 KiB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kThreads = 192;
    static constexpr int kTmemCols = 512;
    static constexpr int kGroupM = 16;
    // ring + barriers + slack for aligning the ring to 1024 B
    static constexpr int kSmemBytes = kStages * kStageBytes + 256 + 1024;
};

struct UmmaShared {
    uint64_t full[UmmaCfg::kStages];
    uint64_t empty[UmmaCfg::kStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ void umma_tile_coords(int t, int tiles_m, int tiles_n, int& tm, int& tn) {
    const int group_size = UmmaCfg::kGroupM * tiles_n;
    const int group = t / group_size;
    const int first_m = group * UmmaCfg::kGroupM;
    const int rows = min(UmmaCfg::kGroupM, tiles_m - first_m);
    const int in_group = t - group * group_size;
    tm = first_m + in_group % rows;
    tn = in_group / rows;
}

template <int ACT>
__global__ void __launch_bounds__(UmmaCfg::kThreads, 1)
gemm_umma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ Y, int M, int N, int K,
                 int* __restrict__ status) {
    using C = UmmaCfg;
    extern __shared__ uint8_t smem_raw[];
    // barriers first, then the ring at the next 1024-byte boundary (128-byte swizzle atoms)
    UmmaShared* sh = reinterpret_cast<UmmaShared*>(smem_raw);
    const uint32_t ring_base = (ptx::smem_u32(smem_raw) + 256 + 1023) & ~1023u;
    uint8_t* ring = smem_raw + (ring_base - ptx::smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (M + C::BM - 1) / C::BM, tiles_n = (N + C::BN - 1) / C::BN;
    const int num_tiles = tiles_m * tiles_n;
    const int num_kb = (K + C::BK - 1) / C::BK;

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
    // set-up above overlapped the previous kernel's tail; from here on global memory is touched
    ptx::griddep_wait();
    ptx::griddep_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&map_a);
            ptx::prefetch_tensormap(&map_b);
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                int tm, tn;
                umma_tile_coords(t, tiles_m, tiles_n, tm, tn);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1;
                    if (sh->abort || !ptx::mbar_wait(&sh->empty[s], ph ^ 1)) { ok = false; break; }
                    uint8_t* a_dst = ring + s * C::kStageBytes;
                    uint8_t* b_dst = a_dst + C::kABytes;
                    ptx::mbar_arrive_expect_tx(&sh->full[s], C::kStageBytes);
                    ptx::tma_load_2d(a_dst, &map_a, &sh->full[s], kb * C::BK, tm * C::BM);
#pragma unroll
                    for (int j = 0; j < C::BN / 64; ++j)
                        ptx::tma_load_2d(b_dst + j * C::kBChunkBytes, &map_b, &sh->full[s], tn * C::BN + j * 64,
                                         kb * C::BK);
                }
            }
            if (!ok) {
                atomicExch(status, kDevTimeout);
                sh->abort = 1;
                // copies already issued must land before the CTA may exit
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
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(C::BM, C::BN, /*a_mn_major=*/false, /*b_mn_major=*/true);
            uint32_t it = 0, tile_it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_it) {
                const int a = tile_it & 1;
                const uint32_t aph = (tile_it >> 1) & 1;
                if (sh->abort || !ptx::mbar_wait(&sh->tmem_empty[a], aph ^ 1)) { ok = false; break; }
                ptx::tcgen05_fence_after_sync();
                const uint32_t d_tmem = tmem_base + a * C::BN;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1;
                    if (sh->abort || !ptx::mbar_wait(&sh->full[s], ph)) { ok = false; break; }
                    ptx::tcgen05_fence_after_sync();
                    const uint32_t a_addr = ring_base + s * C::kStageBytes;
                    const uint32_t b_addr = a_addr + C::kABytes;
#pragma unroll
                    for (int k4 = 0; k4 < C::BK / 16; ++k4) {
                        // A: K-major, 16 k = 32 bytes along the 128-byte row.
                        // B: MN-major, 16 k = 16 rows of 128 bytes; 64-column chunks 8 KiB apart.
                        const uint64_t a_desc = ptx::umma_smem_desc(a_addr + k4 * 32, 16, 1024);
                        const uint64_t b_desc = ptx::umma_smem_desc(b_addr + k4 * 2048, C::kBChunkBytes, 1024);
                        ptx::umma_bf16(d_tmem, a_desc, b_desc, idesc, (kb | k4) != 0);
                    }
                    ptx::umma_commit(&sh->empty[s]);      // stage reusable once these MMAs have read it
                }
                if (ok) ptx::umma_commit(&sh->tmem_full[a]);
            }
            if (!ok) {
                atomicExch(status, kDevTimeout);
                sh->abort = 1;
            }
            // nothing may be in flight on the tensor pipe when TMEM is freed
            ptx::umma_commit(&sh->drain);
            ptx::mbar_wait(&sh->drain, 0);
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        uint32_t tile_it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_it) {
            int tm, tn;
            umma_tile_coords(t, tiles_m, tiles_n, tm, tn);
            const int a = tile_it & 1;
            const uint32_t aph = (tile_it >> 1) & 1;
            bool got = !sh->abort && ptx::mbar_wait(&sh->tmem_full[a], aph);
            got = __all_sync(0xffffffffu, got);       // keep the warp together for tcgen05.ld
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();
            const int64_t row = (int64_t)tm * C::BM + q * 32 + lane;
            const int64_t col0 = (int64_t)tn * C::BN;
            __nv_bfloat16* yrow = Y + row * N + col0;
#pragma unroll 1
            for (int c = 0; c < C::BN / 32; ++c) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + a * C::BN + c * 32, r);
                ptx::tmem_ld_wait();
                if (col0 + c * 32 >= N) continue;     // uniform across the warp
#pragma unroll
                for (int v = 0; v < 4; ++v) {         // 8 columns = one 16-byte store
                    const int64_t n = col0 + c * 32 + v * 8;
                    if (n >= N) break;                // N % 8 == 0
                    uint4 bw = make_uint4(0, 0, 0, 0);
                    if (bias) bw = *reinterpret_cast<const uint4*>(bias + n);
                    const uint32_t bwv[4] = {bw.x, bw.y, bw.z, bw.w};
                    uint32_t o[4];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        const float y0 = epilogue<ACT, true>(__uint_as_float(r[v * 8 + 2 * p]), bf16lo_to_f32(bwv[p]));
                        const float y1 = epilogue<ACT, true>(__uint_as_float(r[v * 8 + 2 * p + 1]), bf16hi_to_f32(bwv[p]));
                        o[p] = pack_bf16x2(y0, y1);
                    }
                    if (row < M) *reinterpret_cast<uint4*>(yrow + c * 32 + v * 8) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive(&sh->tmem_empty[a]);
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
