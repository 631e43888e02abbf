// Compute-bound variant (bf16), two-SM form: a thread-block cluster of two CTAs computes one
// 256 x 256 tile of Y with tcgen05.mma.cta_group::2.
//
// Why: with one CTA per 128 x 256 tile every SM pulls 48 KiB per K block through L2 and
// shared memory; that traffic, not the tensor pipe, bounds the single-CTA kernel at about
// 60 % (4096^3) to 80 % (long K) tensor utilisation.  In the pair, CTA r stages rows
// [128 r, 128 r + 128) of the A tile and columns [128 r, 128 r + 128) of the B tile, 32 KiB
// per K block, and the MMA reads both halves: a third less traffic per flop.  Each CTA
// fetches its own halves with plain TMA loads (no load is shared between CTAs).
//
//   warp 0      TMA producer in BOTH CTAs: own A half (K-major) and own B half (N contiguous)
//               into a kStages ring; the bytes are counted on the LEADER's (rank 0) "full"
//               barrier, on which each producer also posts its expected byte count.
//   warp 1      allocates TMEM (cta_group::2, both CTAs); in the leader one lane issues
//               tcgen05.mma.cta_group::2.kind::f16 M=256 N=256 K=16, four per stage;
//               tcgen05.commit (cta_group::2) signals the "empty" barrier of the stage in both CTAs and,
//               after the last K block, the "accumulator full" barrier in both CTAs.
//   warps 2-5   epilogue in both CTAs: each CTA holds 128 rows x 256 columns of the tile in its
//               own TMEM (two accumulators), runs the fused epilogue and TMA-stores its rows;
//               all 256 epilogue threads of the pair release the accumulator on the leader's
//               "accumulator empty" barrier.
//
// Work split, split-K tail round, partial-tile layout and the bounded waits are those of
// kernel_umma.cuh, with CTA pairs in place of CTAs (a cut tile's halves are reduced by the
// CTAs of the same rank).  The pair synchronises (barrier.cluster) after barrier set-up and
// before exit, so neither CTA touches the other's shared memory outside its lifetime.
#pragma once

#include "common.cuh"
#include "kernel_umma.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

struct Umma2Cfg {
    // A stage holds one 64-k block.  (Every stage costs each issuing lane one barrier round trip,
    // but three 128-k stages measured no better than six 64-k stages: 4096^3 103.4 against
    // 101.6 us, 8192 x 8192 x 16384 1505 against 1491 us.)
    static constexpr int kSubK = 1;
    static constexpr int BM = 256, BN = 256, BK = 64 * kSubK, kStages = 6 / kSubK;   // tile of the CTA pair
    static constexpr int kASubBytes = 128 * 64 * 2;          // this CTA's 128 rows x 64 k of A: 16 KiB
    static constexpr int kABytes = kSubK * kASubBytes;
    static constexpr int kBChunkBytes = 64 * 64 * 2;         // 64 k x one 64-column chunk: 8 KiB
    static constexpr int kBSubBytes = 2 * kBChunkBytes;      // 64 k x this CTA's 128 columns of B: 16 KiB
    static constexpr int kBBytes = kSubK * kBSubBytes;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kThreads = 192;
    static constexpr int kTmemCols = 512;
    static constexpr int kGroupM = 8;                        // 8 x 256 rows, as in the single-CTA kernel
    static constexpr int kOutBytes = 32 * 128;               // epilogue staging: 32 rows x 64 bf16
    static constexpr int kSmemBytes = kStages * kStageBytes + 8 * kOutBytes + 256 + 1024;
};

// Same work split as make_umma_plan, over 256 x 256 tiles and CTA pairs.
inline UmmaPlan make_umma2_plan(int64_t M, int64_t N, int64_t K, int num_sms, int split_max = 8) {
    const int pairs = num_sms / 2;
    UmmaPlan p;
    p.tiles_m = (int)((M + Umma2Cfg::BM - 1) / Umma2Cfg::BM);
    p.tiles_n = (int)((N + Umma2Cfg::BN - 1) / Umma2Cfg::BN);
    p.num_kb = (int)((K + Umma2Cfg::BK - 1) / Umma2Cfg::BK);
    const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
    const int64_t q = tiles / pairs, r = tiles - q * pairs;
    int split = 1;
    if (r > 0) {
        split = (int)(pairs / r);
        if (split > split_max) split = split_max;
        if (split > p.num_kb * Umma2Cfg::kSubK / 4) split = p.num_kb * Umma2Cfg::kSubK / 4;   // at least 256 k per slice
        if (split > p.num_kb) split = p.num_kb;
        if (split < 1) split = 1;
    }
    if (split == 1) {
        p.full_tiles = (int)tiles;
        p.rem_tiles = 0;
        p.grid = (int)(tiles < pairs ? tiles : pairs);
    } else {
        p.full_tiles = (int)(q * pairs);
        p.rem_tiles = (int)r;
        p.grid = q > 0 ? pairs : (int)(r * split);
    }
    p.split = split;
    return p;
}

// i-th work item of CTA pair `c`; tile coordinates in units of 256 x 256.
__host__ __device__ __forceinline__ bool umma2_work_item(const UmmaPlan& p, int c, int i, UmmaWork& w) {
    auto coords = [&](int t, int& tm, int& tn) {
        const int group_size = Umma2Cfg::kGroupM * p.tiles_n;
        const int group = t / group_size;
        const int first_m = group * Umma2Cfg::kGroupM;
        const int left = p.tiles_m - first_m;
        const int rows = left < Umma2Cfg::kGroupM ? left : Umma2Cfg::kGroupM;
        const int in_group = t - group * group_size;
        tm = first_m + in_group % rows;
        tn = in_group / rows;
    };
    const int64_t t = (int64_t)c + (int64_t)i * p.grid;
    if (t < p.full_tiles) {
        coords((int)t, w.tm, w.tn);
        w.kb0 = 0;
        w.kb1 = p.num_kb;
        w.rem_idx = -1;
        w.chunk = 0;
        return true;
    }
    const int n_full = c < p.full_tiles ? (p.full_tiles - c + p.grid - 1) / p.grid : 0;
    if (i != n_full || c >= p.rem_tiles * p.split) return false;
    w.rem_idx = c / p.split;
    w.chunk = c % p.split;
    coords(p.full_tiles + w.rem_idx, w.tm, w.tn);
    w.kb0 = (int)((int64_t)p.num_kb * w.chunk / p.split);
    w.kb1 = (int)((int64_t)p.num_kb * (w.chunk + 1) / p.split);
    return true;
}

struct Umma2Shared {
    uint64_t full[Umma2Cfg::kStages];      // used in the leader: bytes of both CTAs land here
    uint64_t empty[Umma2Cfg::kStages];     // per CTA, signalled by the leader's commit
    uint64_t tmem_full[2];                 // per CTA, signalled by the leader's commit
    uint64_t tmem_empty[2];                // used in the leader: 256 epilogue threads arrive
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
    int last_flag;
    int vote[4];
};

__device__ __forceinline__ void umma2_epi_bar_sync() { asm volatile("bar.sync 3, 128;" ::: "memory"); }

template <int ACT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Umma2Cfg::kThreads, 1)
gemm_umma2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_y, const __nv_bfloat16* __restrict__ bias, int M, int N, int K,
                 const __grid_constant__ UmmaPlan plan, float* __restrict__ partials,
                 unsigned int* __restrict__ counters, int* __restrict__ status) {
    using C = Umma2Cfg;
    extern __shared__ uint8_t smem_raw[];
    // barriers first, then the ring at the next 1024-byte boundary (128-byte swizzle atoms)
    Umma2Shared* sh = reinterpret_cast<Umma2Shared*>(smem_raw);
    const uint32_t ring_base = (ptx::smem_u32(smem_raw) + 256 + 1023) & ~1023u;
    uint8_t* ring = smem_raw + (ring_base - ptx::smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();       // 0 = leader of the pair
    const int pair = blockIdx.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(&sh->full[s], 2);              // one arrive.expect_tx per producer of the pair
            ptx::mbar_init(&sh->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&sh->tmem_full[a], 1);
            ptx::mbar_init(&sh->tmem_empty[a], 256);      // the epilogue threads of both CTAs
        }
        ptx::mbar_init(&sh->drain, 1);
        sh->abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc_2cta(&sh->tmem_base, C::kTmemCols);
        ptx::tmem_relinquish_2cta();
    }
    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                                // the peer's barriers exist before anyone signals them
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
            uint32_t it = 0, s = 0, ph = 0;
            bool ok = true;
            int site = 0;
            UmmaWork w;
            // the leader's "full" barriers as seen from this CTA (consecutive 8-byte words)
            const uint32_t full_leader0 = ptx::mapa_shared(ptx::smem_u32(&sh->full[0]), 0);
            for (int wi = 0; ok && umma2_work_item(plan, pair, wi, w); ++wi) {
                const int tm = w.tm, tn = w.tn;
                if (sh->abort) { ok = false; break; }
                // whole tiles walk K forwards and backwards in turn: the end of the panels a wave has just
                // streamed is what L2 still holds when the next tiles start (same order in the MMA lane)
                const bool rev = w.rem_idx < 0 && (wi & 1);
                for (int kbi = w.kb0; kbi < w.kb1; ++kbi, ++it) {
                    const int kb = rev ? w.kb1 - 1 - (kbi - w.kb0) : kbi;
                    if ((site = 1, !ptx::mbar_wait(&sh->empty[s], ph ^ 1))) { ok = false; break; }
                    uint8_t* a_dst = ring + s * C::kStageBytes;
                    uint8_t* b_dst = a_dst + C::kABytes;
                    const uint32_t full_leader = full_leader0 + 8u * s;
                    ptx::mbar_arrive_expect_tx_cluster(full_leader, C::kStageBytes);
#pragma unroll
                    for (int u = 0; u < C::kSubK; ++u) {
                        ptx::tma_load_2d_2cta(a_dst + u * C::kASubBytes, &map_a, full_leader, kb * C::BK + u * 64,
                                              tm * C::BM + (int)rank * 128);
#pragma unroll
                        for (int j = 0; j < 2; ++j)
                            ptx::tma_load_2d_2cta(b_dst + u * C::kBSubBytes + j * C::kBChunkBytes, &map_b, full_leader,
                                                  tn * C::BN + (int)rank * 128 + j * 64, kb * C::BK + u * 64);
                    }
                    if (++s == C::kStages) { s = 0; ph ^= 1; }
                }
            }
            if (!ok) {
                report_timeout(status, site);
                sh->abort = 1;
                // copies already issued must land before the CTA may exit; their bytes are
                // counted on the leader's barriers, so only the leader can watch them land --
                // the peer is held by the cluster barrier at the end until the leader is done
                if (rank == 0) {
                    const uint32_t n_back = it < (uint32_t)C::kStages ? it : (uint32_t)C::kStages;
                    for (uint32_t b = 1; b <= n_back; ++b) {
                        const uint32_t j = it - b;
                        ptx::mbar_wait(&sh->full[j % C::kStages], (j / C::kStages) & 1);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(C::BM, C::BN, /*a_mn_major=*/false, /*b_mn_major=*/true);
            // The issuing lane is on the critical path (a K block costs it the barrier wait plus four
            // MMA issues, against 512 cycles on the tensor pipe), so its loop is kept lean: the low
            // words of the shared-memory descriptors advance by constants from stage to stage and
            // from K step to K step (start address in 16-byte units: A 2 per 16 k, B 128 per 16 k), the
            // high word never changes, and the stage index wraps by comparison instead of a division.
            constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);   // stride 1024 B, version 1, 128-B swizzle
            const uint32_t a_lo0 = ((ring_base & 0x3FFFFu) >> 4) | ((16u >> 4) << 16);
            const uint32_t b_lo0 = (((ring_base + C::kABytes) & 0x3FFFFu) >> 4) | ((uint32_t)(C::kBChunkBytes >> 4) << 16);
            auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
            uint32_t it = 0, tile_it = 0, s = 0, ph = 0;
            bool ok = true;
            int site = 0;
            UmmaWork w;
            for (int wi = 0; ok && umma2_work_item(plan, pair, wi, w); ++wi, ++tile_it) {
                const int a = tile_it & 1;
                const uint32_t aph = (tile_it >> 1) & 1;
                if (sh->abort || (site = 2, !ptx::mbar_wait(&sh->tmem_empty[a], aph ^ 1))) { ok = false; break; }
                ptx::tcgen05_fence_after_sync();
                const uint32_t d_tmem = tmem_base + a * C::BN;
                for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {     // kb counts the K blocks in the order the producer sends them
                    // (the abort flag is looked at once per tile, above: every wait is bounded anyway)
                    if ((site = 4, !ptx::mbar_wait(&sh->full[s], ph))) { ok = false; break; }
                    ptx::tcgen05_fence_after_sync();
                    const uint32_t a_lo = a_lo0 + s * (uint32_t)(C::kStageBytes >> 4);
                    const uint32_t b_lo = b_lo0 + s * (uint32_t)(C::kStageBytes >> 4);
                    // Each descriptor names this CTA's half; the peer's half sits at the same
                    // shared-memory offsets in the peer CTA.
                    // A: K-major, 16 k = 32 bytes along the 128-byte row.
                    // B: MN-major, 16 k = 16 rows of 128 bytes; 64-column chunks 8 KiB apart.
                    ptx::umma_bf16_2cta(d_tmem, desc(a_lo), desc(b_lo), idesc, kb != w.kb0);
#pragma unroll
                    for (int k4 = 1; k4 < C::BK / 16; ++k4)
                        ptx::umma_bf16_2cta_acc(d_tmem, desc(a_lo + (k4 / 4) * (C::kASubBytes >> 4) + 2 * (k4 % 4)),
                                                desc(b_lo + (k4 / 4) * (C::kBSubBytes >> 4) + 128 * (k4 % 4)), idesc);
                    ptx::umma_commit_2cta(&sh->empty[s]);    // both CTAs: stage reusable once these MMAs have read it
                    if (++s == C::kStages) { s = 0; ph ^= 1; }
                }
                if (ok) ptx::umma_commit_2cta(&sh->tmem_full[a]);
            }
            if (!ok) {
                report_timeout(status, site);
                sh->abort = 1;
            }
            // nothing may be in flight on the tensor pipe when TMEM is freed
            ptx::umma_commit_2cta_local(&sh->drain);
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
        for (int wi = 0; ok && umma2_work_item(plan, pair, wi, w); ++wi, ++tile_it) {
            const int a = tile_it & 1;
            const uint32_t aph = (tile_it >> 1) & 1;
            bool got = !sh->abort && ptx::mbar_wait(&sh->tmem_full[a], aph);
            got = __all_sync(0xffffffffu, got);       // keep the warp together for tcgen05.ld
            if (w.rem_idx >= 0) {
                // the four warps meet at named barriers below and must decide alike (every
                // warp reaches this vote: its wait is bounded)
                if (lane == 0) sh->vote[q] = got;
                umma2_epi_bar_sync();
                got = sh->vote[0] && sh->vote[1] && sh->vote[2] && sh->vote[3];
                umma2_epi_bar_sync();
            }
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();
            const int64_t row0 = (int64_t)w.tm * C::BM + (int64_t)rank * 128 + q * 32;     // first row of this warp
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
                ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&sh->tmem_empty[a]), 0));
                continue;
            }

            // ---- K slice of a cut tile: park the fp32 partial, the last arriver finishes the tile.
            // Partial layout: float4 index ((c32 * 8 + v) * 128 + row): a warp's store covers 512
            // contiguous bytes.
            const size_t tile_floats = (size_t)128 * C::BN;      // this CTA's half of the tile
            const size_t rem_half = (size_t)w.rem_idx * 2 + rank;
            float4* mine = reinterpret_cast<float4*>(partials + (rem_half * plan.split + w.chunk) * tile_floats) +
                           (q * 32 + lane);
#pragma unroll 1
            for (int c = 0; c < C::BN / 32; ++c) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(t_acc + c * 32, r);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    mine[(c * 8 + v) * 128] = make_float4(__uint_as_float(r[v * 4]), __uint_as_float(r[v * 4 + 1]),
                                                            __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
            }
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&sh->tmem_empty[a]), 0));
            __threadfence();
            umma2_epi_bar_sync();
            if (et == 0) {
                const unsigned int prev = atomicAdd(&counters[rem_half], 1u);
                const int last = (prev == (unsigned int)(plan.split - 1));
                if (last) counters[rem_half] = 0u;        // all slices are in: re-arm for the next call
                sh->last_flag = last;
            }
            umma2_epi_bar_sync();
            if (sh->last_flag) {
                __threadfence();
                const float4* all = reinterpret_cast<const float4*>(partials + rem_half * plan.split * tile_floats) +
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
                            for (int v = 0; v < 8; ++v) t[v] = __ldcg(src + (c * 8 + v) * 128);
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
    ptx::cluster_sync();        // no MMA, copy or remote arrive of the pair is outstanding past this point
    if (warp == 1) {
        __syncwarp();
        ptx::tcgen05_fence_after_sync();
        ptx::tmem_dealloc_2cta(tmem_base, C::kTmemCols);
    }
}

}  // namespace optiml
