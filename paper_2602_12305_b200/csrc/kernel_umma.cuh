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
//               32 * (warp % 4)), add bias, activate, round once to bf16 in registers, stage
//               32 rows x 64 columns in swizzled shared memory and let TMA store the block
//               (whole 128-byte lines, clipped at the edges of Y); the other accumulator is
//               being filled meanwhile, so the epilogue hides under the next tile's MMAs.
//
// Tiles are walked in groups of 16 tile-rows so the CTAs running at the same time share
// A and B panels in L2.  Tiles are dealt round-robin to one CTA per SM; when the last
// round would leave most SMs idle (tiles = q * SMs + r with r <= SMs / 2), each of those r
// tiles is cut into s = SMs / r slices along K and every slice goes to its own CTA: the
// slices leave fp32 partial tiles in the handle's scratch and the CTA that arrives last on
// a tile (arrival counter, nobody waits) adds them in K order and runs the fused epilogue.
// 4096^3 is 512 tiles on 148 SMs: 3 full rounds plus 68 tiles, i.e. 3.5 rounds' time
// instead of 4.  Ragged M, N, K edges cost nothing special: TMA zero-fills
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
    static constexpr int kOutBytes = 32 * 128;               // epilogue staging: 32 rows x 64 bf16
    // ring + epilogue staging (4 warps x 2 buffers) + barriers + slack for aligning to 1024 B
    static constexpr int kSmemBytes = kStages * kStageBytes + 8 * kOutBytes + 256 + 1024;
};

// Host-made work split; see the header comment.
struct UmmaPlan {
    int tiles_m, tiles_n, num_kb;
    int grid;         // CTAs
    int full_tiles;   // tiles computed whole, dealt round-robin
    int rem_tiles;    // tiles of the last, partial round that are cut along K
    int split;        // K slices per such tile (1 = nothing is cut)
};

inline UmmaPlan make_umma_plan(int64_t M, int64_t N, int64_t K, int num_sms) {
    UmmaPlan p;
    p.tiles_m = (int)((M + UmmaCfg::BM - 1) / UmmaCfg::BM);
    p.tiles_n = (int)((N + UmmaCfg::BN - 1) / UmmaCfg::BN);
    p.num_kb = (int)((K + UmmaCfg::BK - 1) / UmmaCfg::BK);
    const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
    const int64_t q = tiles / num_sms, r = tiles - q * num_sms;
    int split = 1;
    if (r > 0) {
        split = (int)(num_sms / r);
        if (split > 8) split = 8;                        // bounds the partial-tile traffic
        if (split > p.num_kb / 4) split = p.num_kb / 4;  // at least 4 K blocks per slice
        if (split < 1) split = 1;
    }
    if (split == 1) {
        p.full_tiles = (int)tiles;
        p.rem_tiles = 0;
        p.grid = (int)(tiles < num_sms ? tiles : num_sms);
    } else {
        p.full_tiles = (int)(q * num_sms);
        p.rem_tiles = (int)r;
        p.grid = q > 0 ? num_sms : (int)(r * split);
    }
    p.split = split;
    return p;
}

struct UmmaWork {
    int tm, tn, kb0, kb1;
    int rem_idx;      // -1: whole tile; otherwise index of the cut tile
    int chunk;        // K slice of a cut tile
};

struct UmmaShared {
    uint64_t full[UmmaCfg::kStages];
    uint64_t empty[UmmaCfg::kStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
    int last_flag;
    int vote[4];
};

__device__ __forceinline__ void umma_epi_bar_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }

__device__ __forceinline__ void umma_tile_coords(int t, int tiles_m, int tiles_n, int& tm, int& tn) {
    const int group_size = UmmaCfg::kGroupM * tiles_n;
    const int group = t / group_size;
    const int first_m = group * UmmaCfg::kGroupM;
    const int rows = min(UmmaCfg::kGroupM, tiles_m - first_m);
    const int in_group = t - group * group_size;
    tm = first_m + in_group % rows;
    tn = in_group / rows;
}

// i-th work item of CTA `c` (i counts from 0); false when there is none.
__device__ __forceinline__ bool umma_work_item(const UmmaPlan& p, int c, int i, UmmaWork& w) {
    const int64_t t = (int64_t)c + (int64_t)i * p.grid;
    if (t < p.full_tiles) {
        umma_tile_coords((int)t, p.tiles_m, p.tiles_n, w.tm, w.tn);
        w.kb0 = 0;
        w.kb1 = p.num_kb;
        w.rem_idx = -1;
        w.chunk = 0;
        return true;
    }
    // the first index past the whole tiles is this CTA's slice of a cut tile, if it has one
    const int n_full = c < p.full_tiles ? (p.full_tiles - c + p.grid - 1) / p.grid : 0;
    if (i != n_full || c >= p.rem_tiles * p.split) return false;
    w.rem_idx = c / p.split;
    w.chunk = c % p.split;
    umma_tile_coords(p.full_tiles + w.rem_idx, p.tiles_m, p.tiles_n, w.tm, w.tn);
    w.kb0 = (int)((int64_t)p.num_kb * w.chunk / p.split);
    w.kb1 = (int)((int64_t)p.num_kb * (w.chunk + 1) / p.split);
    return true;
}

template <int ACT>
__global__ void __launch_bounds__(UmmaCfg::kThreads, 1)
gemm_umma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_y, const __nv_bfloat16* __restrict__ bias, int M, int N, int K,
                 const __grid_constant__ UmmaPlan plan, float* __restrict__ partials,
                 unsigned int* __restrict__ counters, int* __restrict__ status) {
    using C = UmmaCfg;
    extern __shared__ uint8_t smem_raw[];
    // barriers first, then the ring at the next 1024-byte boundary (128-byte swizzle atoms)
    UmmaShared* sh = reinterpret_cast<UmmaShared*>(smem_raw);
    const uint32_t ring_base = (ptx::smem_u32(smem_raw) + 256 + 1023) & ~1023u;
    uint8_t* ring = smem_raw + (ring_base - ptx::smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

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
            int site = 0;
            UmmaWork w;
            for (int wi = 0; ok && umma_work_item(plan, blockIdx.x, wi, w); ++wi) {
                const int tm = w.tm, tn = w.tn;
                for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1;
                    if (sh->abort || (site = 1, !ptx::mbar_wait(&sh->empty[s], ph ^ 1))) { ok = false; break; }
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
                report_timeout(status, site);
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
            int site = 0;
            UmmaWork w;
            for (int wi = 0; ok && umma_work_item(plan, blockIdx.x, wi, w); ++wi, ++tile_it) {
                const int a = tile_it & 1;
                const uint32_t aph = (tile_it >> 1) & 1;
                if (sh->abort || (site = 2, !ptx::mbar_wait(&sh->tmem_empty[a], aph ^ 1))) { ok = false; break; }
                ptx::tcgen05_fence_after_sync();
                const uint32_t d_tmem = tmem_base + a * C::BN;
                for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1;
                    if (sh->abort || (site = 4, !ptx::mbar_wait(&sh->full[s], ph))) { ok = false; break; }
                    ptx::tcgen05_fence_after_sync();
                    const uint32_t a_addr = ring_base + s * C::kStageBytes;
                    const uint32_t b_addr = a_addr + C::kABytes;
#pragma unroll
                    for (int k4 = 0; k4 < C::BK / 16; ++k4) {
                        // A: K-major, 16 k = 32 bytes along the 128-byte row.
                        // B: MN-major, 16 k = 16 rows of 128 bytes; 64-column chunks 8 KiB apart.
                        const uint64_t a_desc = ptx::umma_smem_desc(a_addr + k4 * 32, 16, 1024);
                        const uint64_t b_desc = ptx::umma_smem_desc(b_addr + k4 * 2048, C::kBChunkBytes, 1024);
                        ptx::umma_bf16(d_tmem, a_desc, b_desc, idesc, (kb != w.kb0) || (k4 != 0));
                    }
                    ptx::umma_commit(&sh->empty[s]);      // stage reusable once these MMAs have read it
                }
                if (ok) ptx::umma_commit(&sh->tmem_full[a]);
            }
            if (!ok) {
                report_timeout(status, site);
                sh->abort = 1;
            }
            // nothing may be in flight on the tensor pipe when TMEM is freed
            ptx::umma_commit(&sh->drain);
            ptx::mbar_wait(&sh->drain, 0);
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int et = threadIdx.x - 64;              // 0..127 among the epilogue threads
        // Two 32-row x 128-byte staging buffers per warp (128-byte swizzled, the layout the Y
        // tensor map expects): the warp converts 64 columns of its 32 rows, and one lane hands
        // the block to TMA, which writes whole 128-byte lines and clips at the edges of Y.
        uint8_t* stage_buf = ring + C::kStages * C::kStageBytes + (warp - 2) * 2 * C::kOutBytes;
        uint32_t n_stores = 0;

        // 32 fp32 values of this thread's row (columns c32*32 ..) -> bf16 -> staging row
        auto put32 = [&](uint8_t* buf, const float (&x)[32], int c32, int64_t col0) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int64_t n = col0 + c32 * 32 + v * 8;
                uint4 bw = make_uint4(0, 0, 0, 0);
                if (bias && n < N) bw = *reinterpret_cast<const uint4*>(bias + n);    // N % 8 == 0
                const uint32_t bwv[4] = {bw.x, bw.y, bw.z, bw.w};
                uint32_t o[4];
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const float y0 = epilogue<ACT, true>(x[v * 8 + 2 * p], bf16lo_to_f32(bwv[p]));
                    const float y1 = epilogue<ACT, true>(x[v * 8 + 2 * p + 1], bf16hi_to_f32(bwv[p]));
                    o[p] = pack_bf16x2(y0, y1);
                }
                const int chunk16 = (c32 & 1) * 4 + v;                  // 16-byte chunk within the 128-byte row
                *reinterpret_cast<uint4*>(buf + lane * 128 + ((chunk16 ^ (lane & 7)) << 4)) =
                    make_uint4(o[0], o[1], o[2], o[3]);
            }
        };
        auto begin_block = [&]() -> uint8_t* {
            // the buffer used two blocks ago must have been read out by its TMA store
            if (n_stores >= 2) {
                if (lane == 0) ptx::tma_store_wait_read<1>();
                __syncwarp();
            }
            return stage_buf + (n_stores & 1) * C::kOutBytes;
        };
        auto end_block = [&](uint8_t* buf, int64_t x, int64_t y) {
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                if (x < N && y < M) ptx::tma_store_2d(&map_y, buf, (int)x, (int)y);
                ptx::tma_store_commit();
            }
            ++n_stores;
        };

        uint32_t tile_it = 0;
        bool ok = true;
        UmmaWork w;
        for (int wi = 0; ok && umma_work_item(plan, blockIdx.x, wi, w); ++wi, ++tile_it) {
            const int a = tile_it & 1;
            const uint32_t aph = (tile_it >> 1) & 1;
            bool got = !sh->abort && ptx::mbar_wait(&sh->tmem_full[a], aph);
            got = __all_sync(0xffffffffu, got);       // keep the warp together for tcgen05.ld
            if (w.rem_idx >= 0) {
                // the four warps meet at named barriers below and must decide alike (every
                // warp reaches this vote: its wait is bounded)
                if (lane == 0) sh->vote[q] = got;
                umma_epi_bar_sync();
                got = sh->vote[0] && sh->vote[1] && sh->vote[2] && sh->vote[3];
                umma_epi_bar_sync();
            }
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();
            const int64_t row0 = (int64_t)w.tm * C::BM + q * 32;     // first row of this warp
            const int64_t col0 = (int64_t)w.tn * C::BN;
            const uint32_t t_acc = tmem_base + ((uint32_t)(q * 32) << 16) + a * C::BN;

            if (w.rem_idx < 0) {
                // ---- whole tile: fused epilogue straight from TMEM
#pragma unroll 1
                for (int cc = 0; cc < C::BN / 64; ++cc) {
                    uint8_t* buf = begin_block();
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        uint32_t r[32];
                        ptx::tmem_ld_32x32(t_acc + cc * 64 + hh * 32, r);
                        ptx::tmem_ld_wait();
                        float x[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(r[i]);
                        put32(buf, x, cc * 2 + hh, col0);
                    }
                    end_block(buf, col0 + cc * 64, row0);
                }
                ptx::tcgen05_fence_before_sync();
                ptx::mbar_arrive(&sh->tmem_empty[a]);
                continue;
            }

            // ---- K slice of a cut tile: park the fp32 partial, the last arriver finishes the tile.
            // Partial layout: float4 index ((c32 * 8 + v) * 128 + row): a warp's store covers 512
            // contiguous bytes.
            const size_t tile_floats = (size_t)C::BM * C::BN;
            float4* mine = reinterpret_cast<float4*>(partials + ((size_t)w.rem_idx * plan.split + w.chunk) * tile_floats) +
                           (q * 32 + lane);
#pragma unroll 1
            for (int c = 0; c < C::BN / 32; ++c) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(t_acc + c * 32, r);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    mine[(c * 8 + v) * C::BM] = make_float4(__uint_as_float(r[v * 4]), __uint_as_float(r[v * 4 + 1]),
                                                            __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
            }
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive(&sh->tmem_empty[a]);
            __threadfence();
            umma_epi_bar_sync();
            if (et == 0) {
                const unsigned int prev = atomicAdd(&counters[w.rem_idx], 1u);
                const int last = (prev == (unsigned int)(plan.split - 1));
                if (last) counters[w.rem_idx] = 0u;       // all slices are in: re-arm for the next call
                sh->last_flag = last;
            }
            umma_epi_bar_sync();
            if (sh->last_flag) {
                __threadfence();
                const float4* all = reinterpret_cast<const float4*>(partials + (size_t)w.rem_idx * plan.split * tile_floats) +
                                    (q * 32 + lane);
#pragma unroll 1
                for (int cc = 0; cc < C::BN / 64; ++cc) {
                    uint8_t* buf = begin_block();
#pragma unroll 1
                    for (int hh = 0; hh < 2; ++hh) {
                        const int c = cc * 2 + hh;
                        float x[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) x[i] = 0.0f;
                        for (int sl = 0; sl < plan.split; ++sl) {         // slices in ascending K
                            const float4* src = all + (size_t)sl * (tile_floats / 4);
                            float4 t[8];
#pragma unroll
                            for (int v = 0; v < 8; ++v) t[v] = __ldcg(src + (c * 8 + v) * C::BM);
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                x[v * 4 + 0] += t[v].x;
                                x[v * 4 + 1] += t[v].y;
                                x[v * 4 + 2] += t[v].z;
                                x[v * 4 + 3] += t[v].w;
                            }
                        }
                        put32(buf, x, c, col0);
                    }
                    end_block(buf, col0 + cc * 64, row0);
                }
            }
        }
        // every TMA store of this warp has finished before the CTA can go away
        if (lane == 0) ptx::tma_store_wait_all<0>();
        __syncwarp();
        if (!ok && lane == 0) {
            report_timeout(status, 5);
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
