// Skinny variant (bf16, M <= 128): the problem is a single pass over B, so it is laid
// out as a stream over HBM, but the multiply-accumulates go to the tensor cores: at
// M = 16 the FMA pipes cannot keep up with HBM (about 100 TFLOP/s would be needed).
//
// Operands are swapped: the MMA computes Y^T tiles, D[n, m] = sum_k B[k, n] A[m, k].
//   MMA "A" operand = a 128(n) x 64(k) tile of B, N contiguous (MN-major), two 64-column
//                     TMA boxes with 128-byte swizzle;
//   MMA "B" operand = the MP x 64 tile of A (rows >= M are zero-filled by TMA), K-major;
//   accumulator     = 128 TMEM lanes (n) x MP fp32 columns (m) per column tile.
//
// Schedule (SkinnyPlan, made on the host).  One CTA per SM.  The (column tile, K block)
// grid, T x KB units, is cut into one rectangle per CTA, all of about the same area, so
// every SM streams the same number of bytes.  The rectangles are arranged in horizontal
// BANDS: a band is a range of K blocks in which the T column tiles are dealt left to
// right to the band's CTAs.  A CTA sweeps its rectangle K-major (for each K block, all of
// its column tiles) with one TMEM accumulator per column tile.  All CTAs of a band
// therefore walk down the same rows of B at the same pace and between them read whole
// rows: DRAM sees long sequential bursts.  (CTAs streaming unrelated 256-byte wide strips
// reach only half the HBM throughput on B200.)
//   * S "full" bands: T CTAs each, one column tile per CTA;
//   * up to two "wide" bands for the CTAs left over (or for all CTAs when T > CTAs), where
//     a CTA takes several adjacent column tiles; the band heights are chosen so that all
//     rectangles have the same area.
//
// With a single band every column tile is finished by one CTA and goes straight through
// the fused epilogue.  Otherwise each band's CTA writes its fp32 partial tile to the
// handle's scratch and bumps the tile's arrival counter; the CTA that arrives last (nobody
// waits) adds the partials in band (= K) order, applies bias + activation and stores Y.
// The order of the sum is fixed, so results are reproducible.
//
// Roles: warp 0 TMA producer (a ring of B tiles, a small ring of A tiles: one A tile per
// K block serves all the column tiles of the sweep), warp 1 TMEM allocation + MMA issue,
// warps 2-5 epilogue.  TMEM holds two sets of accumulators so that, when a CTA's
// rectangle is wider than one set, the epilogue of one chunk overlaps the next sweep.
// All mbarrier waits are bounded; see kernel_umma.cuh for the tear-down protocol.
#pragma once

#include <math.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

// MP: padded M (accumulator columns).  SUB: 64-row sub-blocks of K per pipeline stage.
template <int MP, int SUB>
struct SkinnyCfg {
    static_assert(MP == 16 || MP == 32 || MP == 64 || MP == 128, "padded M");
    static_assert(SUB == 2 || SUB == 3, "sub-blocks per stage");
    // One pipeline stage carries kSub sub-blocks of 64 K rows: every stage costs one
    // tcgen05.commit / mbarrier round trip, and with the tiny MMAs of this kernel that round
    // trip, not HBM, limits a 64-row stage.
    // (measured, 16 x 14336 x 4096: 64-row stages 41 us, 128-row 25.7 us, 192-row 23.9 us;
    // larger stages leave too few of them in the ring)
    static constexpr int kSub = SUB;
    static constexpr int BN = 128, BK = 64 * kSub;
    static constexpr int kBChunkBytes = 64 * 64 * 2;           // 64 k-rows x 64 columns: 8 KiB
    static constexpr int kBSubBytes = 2 * kBChunkBytes;        // 64 k-rows x 128 columns
    static constexpr int kBBytes = kSub * kBSubBytes;          // one stage of the B ring
    static constexpr int kASubBytes = MP * 64 * 2;
    static constexpr int kABytes = kSub * kASubBytes;          // one slot of the A ring
    static constexpr int kBarrierBytes = 512;                  // SkinnyShared, after the rings
    static constexpr int kFit = (226 * 1024 - kBarrierBytes - kABytes) / (kBBytes + kABytes);
    static constexpr int kStages = kFit < 12 ? kFit : 12;      // deepest B ring a CTA can hold
    // The A ring needs no "empty" barrier: a slot is reused (stages + 1) K blocks later, and by
    // then the producer has waited for B stages whose release implies that every MMA of the
    // old K block is done (it can be at most `stages` stages ahead of the MMAs).
    static constexpr int kAStages = kStages + 1;
    // MMA-issuing lanes.  A tcgen05.mma with so small an N costs its issuer about 60 cycles, the
    // tensor pipe under 40, and the issuer also waits on the barriers of every stage: measured
    // on 16 x 14336 x 4096, one lane needed 0.9 us per 192-row stage, which capped a CTA at
    // 53 GB/s.  With two lanes each issues every other 16-row step of K into an accumulator of
    // its own (the epilogue adds the two, always in the same order).  The second set of
    // accumulators halves the column tiles a sweep can hold (kAcc).  At MP = 128 an MMA takes 64
    // cycles on the pipe, about what one lane needs to issue it; two lanes still gain 2-3 %
    // (128 x 14336 x 4096: 26.3 -> 25.6 us), so every configuration has two.
    static constexpr int kIssuers = 2;
    static constexpr int kThreads = 192 + 32 * (kIssuers - 1); // warp 6: the second issuing lane
    static constexpr int kAccFit = 256 / (MP * kIssuers);
    static constexpr int kAcc = kAccFit < 8 ? kAccFit : 8;     // column tiles per sweep
    static constexpr int kTmemCols = 2 * kAcc * MP * kIssuers; // 512 in every configuration
    static constexpr int kChunk = MP < 32 ? MP : 32;           // accumulator columns per tcgen05.ld
    // dynamic shared memory of a launch whose B ring is `stages` deep (A ring: one more)
    static constexpr int smem_bytes(int stages) { return stages * kBBytes + (stages + 1) * kABytes + kBarrierBytes; }
    static constexpr int kSmemBytes = smem_bytes(kStages);
    // Deepest ring that lets two CTAs share an SM (228 KiB, 1 KiB reserved per CTA), so that the
    // next call's CTAs could be resident and set up while this call's CTAs finish; 0 where not
    // even two stages fit.  (Measured on 16 x 14336 x 4096: such short rings of 128-row stages
    // lose more, 3-4 us, than the overlap wins; the launcher uses the deepest ring by default.)
    static constexpr int kFit2 = (113 * 1024 - kBarrierBytes - kABytes) / (kBBytes + kABytes);
    static constexpr int kStagesShared = kFit2 >= 2 ? kFit2 : 0;
    static constexpr int kSlotFloats = MP * BN;                // one partial tile in scratch
};

template <int MP, int SUB>
struct SkinnyShared {
    uint64_t full[SkinnyCfg<MP, SUB>::kStages];
    uint64_t empty[SkinnyCfg<MP, SUB>::kStages];
    uint64_t a_full[SkinnyCfg<MP, SUB>::kAStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
    int last_flag[8];
    int vote[4];
};

// Host-made schedule; see the header comment.
struct SkinnyPlan {
    int T;         // column tiles
    int KB;        // K blocks
    int G;         // CTAs = S*T + G1 + G2
    int S;         // full bands, covering K blocks [0, k_split)
    int k_split;
    int G1;        // CTAs of wide band 1, K blocks [k_split, k_mid)
    int k_mid;
    int G2;        // CTAs of wide band 2, K blocks [k_mid, KB)
    int nbands;    // S + (G1 > 0) + (G2 > 0): segments per column tile
};

struct SkinnyRect {
    int t0, t1, kb0, kb1, band;
};

// Run-time tuning of the streaming pipeline (set per handle; see optiml_set_option).
struct SkinnyTune {
    int stages;          // depth of the B ring, 2 .. SkinnyCfg::kStages
    int prefetch_early;  // units (one stage of B each) prefetched into L2 before the wait on the previous kernel
    int late_trigger;    // 1: let the next kernel's CTAs start when this CTA has issued its last load
};

// Walks the units of a CTA's rectangle in the order the pipeline consumes them: chunks of up to
// kAcc column tiles; within a chunk K-major, the chunk's tiles for every K block.
template <int kAcc>
struct SkinnySweep {
    int tc, kb, j, nt;
    bool done;
    __device__ __forceinline__ void start(const SkinnyRect& r) {
        tc = r.t0;
        kb = r.kb0;
        j = 0;
        nt = min(kAcc, r.t1 - r.t0);
        done = r.t0 >= r.t1 || r.kb0 >= r.kb1;
    }
    __device__ __forceinline__ void next(const SkinnyRect& r) {
        if (++j < nt) return;
        j = 0;
        if (++kb < r.kb1) return;
        kb = r.kb0;
        tc += kAcc;
        if (tc >= r.t1) {
            done = true;
            return;
        }
        nt = min(kAcc, r.t1 - tc);
    }
};

__host__ __device__ __forceinline__ SkinnyRect skinny_rect(const SkinnyPlan& p, int c) {
    SkinnyRect r;
    if (c < p.S * p.T) {
        const int s = c / p.T;
        r.t0 = c % p.T;
        r.t1 = r.t0 + 1;
        r.kb0 = (int)((int64_t)p.k_split * s / p.S);
        r.kb1 = (int)((int64_t)p.k_split * (s + 1) / p.S);
        r.band = s;
        return r;
    }
    int i = c - p.S * p.T;
    if (i < p.G1) {
        r.t0 = (int)((int64_t)p.T * i / p.G1);
        r.t1 = (int)((int64_t)p.T * (i + 1) / p.G1);
        r.kb0 = p.k_split;
        r.kb1 = p.k_mid;
        r.band = p.S;
    } else {
        i -= p.G1;
        r.t0 = (int)((int64_t)p.T * i / p.G2);
        r.t1 = (int)((int64_t)p.T * (i + 1) / p.G2);
        r.kb0 = p.k_mid;
        r.kb1 = p.KB;
        r.band = p.S + (p.G1 > 0 ? 1 : 0);
    }
    return r;
}

// Best banding for `num_sms` CTAs; `max_slots` bounds bands * T, the partial tiles the
// scratch can hold.  With unit_us <= 0 the cost of a plan is the largest rectangle area
// (K blocks x column tiles) any CTA has to stream, ties going to fewer bands.  With
// unit_us > 0 (the time one CTA needs to stream one unit at the per-SM rate) the cost is an
// estimated run time, fitted to measurements on B200: a CTA streams at most at its own rate
// (unit_us per unit), all of them together at most `dram_ctas` CTAs' worth of that (HBM), the
// two limits combine like a 4-norm, and any split along K costs about 2.5 us for the
// partial-tile round trip.  So 112 whole tiles on 112 SMs beat a perfectly balanced two-band
// plan, while 64 tiles are better off cut into three bands on all SMs.
inline SkinnyPlan make_skinny_plan(int64_t tiles, int64_t kblocks, int num_sms, int64_t max_slots,
                                   double unit_us = 0.0, double dram_ctas = 112.0) {
    const int64_t T = tiles, KB = kblocks;
    SkinnyPlan best;
    best.T = (int)T;
    best.KB = (int)KB;
    // fallback: one wide band over everything
    best.S = 0;
    best.k_split = 0;
    best.G1 = (int)(T < num_sms ? T : num_sms);
    best.k_mid = (int)KB;
    best.G2 = 0;
    best.nbands = 1;
    best.G = best.G1;
    auto estimate = [&](int64_t area, int nb) -> double {
        if (unit_us <= 0.0) return (double)area;
        const double t_sm = (double)area * unit_us;
        const double t_dram = (double)(T * KB) * unit_us / dram_ctas;
        const double t = sqrt(sqrt(t_sm * t_sm * t_sm * t_sm + t_dram * t_dram * t_dram * t_dram));
        return t + (nb > 1 ? 2.5 : 0.0);
    };
    double best_cost = estimate(((T + best.G1 - 1) / best.G1) * KB, 1);

    auto consider = [&](int S, int64_t k_split, int G1, int64_t k_mid, int G2) {
        const int nb = S + (G1 > 0) + (G2 > 0);
        if (nb < 1 || (nb > 1 && nb * T > max_slots)) return;
        if (S > 0 && k_split < S) return;
        if (G1 > 0 && k_mid <= k_split) return;
        if (G2 > 0 && KB <= k_mid) return;
        if (G2 == 0 && k_mid != KB) return;
        if (G1 == 0 && (k_split != KB || G2 != 0)) return;
        int64_t area = S > 0 ? (k_split + S - 1) / S : 0;
        if (G1 > 0) {
            const int64_t c1 = ((T + G1 - 1) / G1) * (k_mid - k_split);
            if (c1 > area) area = c1;
        }
        if (G2 > 0) {
            const int64_t c2 = ((T + G2 - 1) / G2) * (KB - k_mid);
            if (c2 > area) area = c2;
        }
        const double cost = estimate(area, nb);
        if (cost < best_cost || (cost == best_cost && nb < best.nbands)) {
            best_cost = cost;
            best.S = S;
            best.k_split = (int)k_split;
            best.G1 = G1;
            best.k_mid = (int)k_mid;
            best.G2 = G2;
            best.nbands = nb;
            best.G = (int)(S * T) + G1 + G2;
        }
    };

    const int s_max = (int)(num_sms / T);
    for (int S = s_max; S >= 1; --S) {
        const int left = (int)(num_sms - S * T);
        consider(S, KB, 0, KB, 0);                               // full bands only
        if (left > 0) {
            const int G1 = (int)(left < T ? left : T);
            const int64_t w1 = (T + G1 - 1) / G1;
            // S*a + h = KB with a ~ w1*h
            const int64_t h0 = KB / (S * w1 + 1);
            for (int64_t h = h0 - 1; h <= h0 + 2; ++h)
                if (h >= 1 && h < KB) consider(S, KB - h, G1, KB, 0);
        }
    }
    // no full band: two wide bands over all CTAs (covers T >= CTAs as well)
    for (int G1 = 1; G1 < num_sms; ++G1) {
        if (G1 > T) break;
        int G2 = num_sms - G1;
        if (G2 > T) G2 = (int)T;
        const int64_t w1 = (T + G1 - 1) / G1, w2 = (T + G2 - 1) / G2;
        const int64_t h0 = KB * w2 / (w1 + w2);
        for (int64_t h = h0 - 1; h <= h0 + 2; ++h)
            if (h >= 1 && h < KB) consider(0, 0, G1, h, G2);
    }
    return best;
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// First tensor-memory column of the accumulator of issuing lane w, accumulator set `half`
// (alternating between sweeps), column tile j of the sweep.
template <int MP, int SUB>
__device__ __forceinline__ uint32_t skinny_acc_col(int w, int half, int j) {
    using C = SkinnyCfg<MP, SUB>;
    return (uint32_t)(((w * 2 + half) * C::kAcc + j) * MP);
}

template <int MP, int SUB>
__global__ void __launch_bounds__(SkinnyCfg<MP, SUB>::kThreads, SkinnyCfg<MP, SUB>::kStagesShared ? 2 : 1)
gemm_skinny_umma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                        const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ Y, int M, int N, int K,
                        int act, const __grid_constant__ SkinnyPlan plan, const SkinnyTune tune,
                        float* __restrict__ partials, unsigned int* __restrict__ counters, int* __restrict__ status) {
    using C = SkinnyCfg<MP, SUB>;
    using Sh = SkinnyShared<MP, SUB>;
    static_assert(sizeof(Sh) <= C::kBarrierBytes, "barrier block");
    // B ring, A ring, barrier block.  The rings hold 128-byte-swizzled tiles and need a 1024-byte
    // aligned base; no slack is reserved for aligning by hand (it would cost the second CTA per
    // SM its place), so a base that is not aligned is reported instead of used.
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t ring_base = ptx::smem_u32(smem_raw);
    if (ring_base & 1023u) {
        if (threadIdx.x == 0) report_timeout(status, 6);
        return;
    }
    const int kStagesRt = tune.stages, kAStagesRt = tune.stages + 1;   // ring depths of this launch
    uint8_t* ring = smem_raw;
    const uint32_t aring_base = ring_base + kStagesRt * C::kBBytes;
    uint8_t* aring = ring + kStagesRt * C::kBBytes;
    Sh* sh = reinterpret_cast<Sh*>(aring + kAStagesRt * C::kABytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const SkinnyRect rect = skinny_rect(plan, blockIdx.x);

    // L2 prefetch of B: the first `prefetch_early` units of this CTA's sweep are requested by one
    // lane BEFORE the wait on the previous kernel.  A prefetch only moves DRAM
    // lines into L2, so it may overtake that kernel; HBM then stays busy while it drains.
    // (Prefetching further units ahead of the TMA loads during the sweep was measured too and
    // only slowed the stream down: the requests pass through the same TMA unit as the loads.)
    // It comes first of all, and from a warp that has no part in the set-up below, because the
    // tensor-memory allocation there may have to wait for the previous call's CTA on this SM.
    if (warp == 2 && lane == 0) {
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
        SkinnySweep<C::kAcc> pf;
        pf.start(rect);
        for (int i = 0; i < tune.prefetch_early && !pf.done; ++i, pf.next(rect)) {
#pragma unroll
            for (int u = 0; u < C::kSub; ++u) {
                ptx::prefetch_l2_tma_2d(&map_b, (pf.tc + pf.j) * C::BN, pf.kb * C::BK + u * 64);
                ptx::prefetch_l2_tma_2d(&map_b, (pf.tc + pf.j) * C::BN + 64, pf.kb * C::BK + u * 64);
            }
        }
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(&sh->full[s], 1);
            ptx::mbar_init(&sh->empty[s], C::kIssuers);       // one commit per issuing lane
        }
        for (int s = 0; s < C::kAStages; ++s) ptx::mbar_init(&sh->a_full[s], 1);
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&sh->tmem_full[a], C::kIssuers);
            ptx::mbar_init(&sh->tmem_empty[a], 128);
        }
        ptx::mbar_init(&sh->drain, C::kIssuers);
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
    if (!tune.late_trigger) ptx::griddep_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_stream = ptx::policy_evict_first();   // B is read exactly once
            const uint64_t pol_keep = ptx::policy_evict_last();      // A is re-read by every CTA
            // ring positions and phases are carried along and wrapped by comparison: the issuing
            // lanes are the critical path of this kernel, and a division per stage shows
            uint32_t it = 0, ait = 0;
            int s = 0, sa = 0;
            uint32_t ph = 0;
            bool ok = true;
            int site = 0;
            for (int tc = rect.t0; tc < rect.t1 && ok; tc += C::kAcc) {
                const int nt = min(C::kAcc, rect.t1 - tc);
                for (int kb = rect.kb0; kb < rect.kb1 && ok; ++kb, ++ait) {
                    ptx::mbar_arrive_expect_tx(&sh->a_full[sa], C::kABytes);
#pragma unroll
                    for (int u = 0; u < C::kSub; ++u)
                        ptx::tma_load_2d_hint(aring + sa * C::kABytes + u * C::kASubBytes, &map_a, &sh->a_full[sa],
                                              kb * C::BK + u * 64, 0, pol_keep);
                    if (++sa == kAStagesRt) sa = 0;
                    for (int j = 0; j < nt; ++j, ++it) {
                        if (sh->abort || (site = 1, !ptx::mbar_wait(&sh->empty[s], ph ^ 1))) { ok = false; break; }
                        uint8_t* b_dst = ring + s * C::kBBytes;
                        ptx::mbar_arrive_expect_tx(&sh->full[s], C::kBBytes);
#pragma unroll
                        for (int u = 0; u < C::kSub; ++u) {
                            ptx::tma_load_2d_hint(b_dst + u * C::kBSubBytes, &map_b, &sh->full[s], (tc + j) * C::BN,
                                                  kb * C::BK + u * 64, pol_stream);
                            ptx::tma_load_2d_hint(b_dst + u * C::kBSubBytes + C::kBChunkBytes, &map_b, &sh->full[s],
                                                  (tc + j) * C::BN + 64, kb * C::BK + u * 64, pol_stream);
                        }
                        if (++s == kStagesRt) { s = 0; ph ^= 1; }
                    }
                }
            }
            // every load of this CTA is on its way: the next kernel's CTAs may take the SMs that
            // free up and start their own prefetch while this one computes and stores
            if (tune.late_trigger) ptx::griddep_launch_dependents();
            if (!ok) {
                report_timeout(status, site);
                sh->abort = 1;
                // copies already issued must land before the CTA may exit
                const uint32_t n_back = it < (uint32_t)kStagesRt ? it : (uint32_t)kStagesRt;
                for (uint32_t b = 1; b <= n_back; ++b) {
                    const uint32_t j = it - b;
                    ptx::mbar_wait(&sh->full[j % kStagesRt], (j / kStagesRt) & 1);
                }
                const uint32_t a_back = ait < (uint32_t)kAStagesRt ? ait : (uint32_t)kAStagesRt;
                for (uint32_t b = 1; b <= a_back; ++b) {
                    const uint32_t j = ait - b;
                    ptx::mbar_wait(&sh->a_full[j % kAStagesRt], (j / kAStagesRt) & 1);
                }
            }
        }
    } else if (warp == 1 || warp == 6) {
        // ------------------------------------------------------------ MMA issuers
        // (warp 6 exists only where C::kIssuers == 2)
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(C::BN, MP, /*a_mn_major=*/true, /*b_mn_major=*/false);
            const int w = warp == 1 ? 0 : 1;                  // this lane takes the K steps w, w + kIssuers, ...
            // Lean loop: ring positions and phases wrap by comparison (no division per stage), the
            // abort flag is read once per K block, and the shared-memory descriptors are a constant
            // high word plus a low word (start address in 16-byte units | leading offset << 16) that
            // moves by constants from step to step.
            constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);   // stride 1024 B, version 1, 128-B swizzle
            auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
            const uint32_t b_lo0 = ((ring_base & 0x3FFFFu) >> 4) | ((uint32_t)(C::kBChunkBytes >> 4) << 16);   // tiles of B (MMA "A")
            const uint32_t a_lo0 = ((aring_base & 0x3FFFFu) >> 4) | ((16u >> 4) << 16);                          // tiles of A (MMA "B")
            uint32_t it = 0, ait = 0, chunk_it = 0;
            int s = 0, sa = 0;
            uint32_t ph = 0, pha = 0;
            bool ok = true;
            int site = 0;
            for (int tc = rect.t0; tc < rect.t1 && ok; tc += C::kAcc, ++chunk_it) {
                const int nt = min(C::kAcc, rect.t1 - tc);
                const int half = chunk_it & 1;
                if (sh->abort || (site = 2, !ptx::mbar_wait(&sh->tmem_empty[half], ((chunk_it >> 1) & 1) ^ 1))) { ok = false; break; }
                ptx::tcgen05_fence_after_sync();
                for (int kb = rect.kb0; kb < rect.kb1 && ok; ++kb, ++ait) {
                    if (sh->abort || (site = 3, !ptx::mbar_wait(&sh->a_full[sa], pha))) { ok = false; break; }
                    const uint32_t a_lo = a_lo0 + (uint32_t)sa * (uint32_t)(C::kABytes >> 4);
                    if (++sa == kAStagesRt) { sa = 0; pha ^= 1; }
                    for (int j = 0; j < nt; ++j, ++it) {
                        if ((site = 4, !ptx::mbar_wait(&sh->full[s], ph))) { ok = false; break; }
                        ptx::tcgen05_fence_after_sync();
                        const uint32_t b_lo = b_lo0 + (uint32_t)s * (uint32_t)(C::kBBytes >> 4);
                        const uint32_t d_tmem = tmem_base + skinny_acc_col<MP, SUB>(w, half, j);
#pragma unroll
                        for (int q = 0; q < C::BK / 16 / C::kIssuers; ++q) {
                            const int k4 = q * C::kIssuers + w;
                            const uint64_t da = desc(b_lo + (uint32_t)((k4 / 4) * (C::kBSubBytes >> 4) + (k4 % 4) * (2048 >> 4)));
                            const uint64_t db = desc(a_lo + (uint32_t)((k4 / 4) * (C::kASubBytes >> 4) + (k4 % 4) * (32 >> 4)));
                            ptx::umma_bf16(d_tmem, da, db, idesc, (kb != rect.kb0) || (q != 0));
                        }
                        ptx::umma_commit(&sh->empty[s]);
                        if (++s == kStagesRt) { s = 0; ph ^= 1; }
                    }
                }
                if (ok) ptx::umma_commit(&sh->tmem_full[half]);
            }
            if (!ok) {
                report_timeout(status, site);
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
        const bool whole = plan.nbands == 1;
        uint32_t chunk_it = 0;
        bool ok = true;
        for (int tc = rect.t0; tc < rect.t1 && ok; tc += C::kAcc, ++chunk_it) {
            const int nt = min(C::kAcc, rect.t1 - tc);
            const int half = chunk_it & 1;
            bool got = !sh->abort && ptx::mbar_wait(&sh->tmem_full[half], (chunk_it >> 1) & 1);
            got = __all_sync(0xffffffffu, got);
            // the four epilogue warps meet at named barriers below: they must take the same
            // decision, so they vote (every warp reaches this barrier: its wait is bounded)
            if (lane == 0) sh->vote[q] = got;
            epi_bar_sync();
            got = sh->vote[0] && sh->vote[1] && sh->vote[2] && sh->vote[3];
            epi_bar_sync();
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();

            for (int j = 0; j < nt; ++j) {
                const int tile = tc + j;
                const int64_t n = (int64_t)tile * C::BN + r;
                const float bv = (whole && bias && n < N) ? __bfloat162float(bias[n]) : 0.0f;
                float* slot = partials + ((size_t)rect.band * plan.T + tile) * C::kSlotFloats;
#pragma unroll 1
                for (int m0 = 0; m0 < MP; m0 += C::kChunk) {
                    uint32_t v[C::kChunk];
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + skinny_acc_col<MP, SUB>(0, half, j) + m0;
                    if constexpr (C::kChunk == 16) ptx::tmem_ld_32x16(taddr, v);
                    else ptx::tmem_ld_32x32(taddr, v);
                    if constexpr (C::kIssuers == 2) {
                        // the second lane's share of K: acc0 + acc1, always in this order
                        uint32_t v1[C::kChunk];
                        const uint32_t taddr1 = tmem_base + ((uint32_t)(q * 32) << 16) + skinny_acc_col<MP, SUB>(1, half, j) + m0;
                        if constexpr (C::kChunk == 16) ptx::tmem_ld_32x16(taddr1, v1);
                        else ptx::tmem_ld_32x32(taddr1, v1);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < C::kChunk; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + __uint_as_float(v1[i]));
                    } else {
                        ptx::tmem_ld_wait();
                    }
                    if (whole) {
#pragma unroll
                        for (int i = 0; i < C::kChunk; ++i) {
                            const int m = m0 + i;
                            if (m < m_valid && n < N)
                                Y[(int64_t)m * N + n] =
                                    __float2bfloat16_rn(epilogue_rt<true>(__uint_as_float(v[i]), bv, act));
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < C::kChunk; ++i)
                            if (m0 + i < m_valid) slot[(m0 + i) * C::BN + r] = __uint_as_float(v[i]);
                    }
                }
            }
            // accumulators read out: hand them back before the (slower) cross-CTA part
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive(&sh->tmem_empty[half]);

            if (!whole) {
                __threadfence();
                epi_bar_sync();
                if (et < nt) {
                    const int tile = tc + et;
                    const unsigned int prev = atomicAdd(&counters[tile], 1u);
                    const int last = (prev == (unsigned int)(plan.nbands - 1));
                    if (last) counters[tile] = 0u;        // every band has arrived: re-arm for the next call
                    sh->last_flag[et] = last;
                }
                epi_bar_sync();
                for (int j = 0; j < nt; ++j) {
                    if (!sh->last_flag[j]) continue;
                    __threadfence();
                    const int tile = tc + j;
                    const int64_t n = (int64_t)tile * C::BN + r;
                    const float bv = (bias && n < N) ? __bfloat162float(bias[n]) : 0.0f;
                    // 8 rows at a time: all loads of a batch are issued before the first add, so
                    // the L2 round trips overlap instead of forming one long dependent chain
                    const float* base = partials + (size_t)tile * C::kSlotFloats + r;
                    const size_t band_stride = (size_t)plan.T * C::kSlotFloats;
                    for (int m0 = 0; m0 < m_valid; m0 += 8) {
                        float s[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) s[i] = 0.0f;
                        for (int b = 0; b < plan.nbands; ++b) {         // bands in ascending K
                            float t[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                t[i] = (m0 + i < m_valid) ? __ldcg(base + b * band_stride + (m0 + i) * C::BN) : 0.0f;
#pragma unroll
                            for (int i = 0; i < 8; ++i) s[i] += t[i];
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (m0 + i < m_valid && n < N)
                                Y[(int64_t)(m0 + i) * N + n] = __float2bfloat16_rn(epilogue_rt<true>(s[i], bv, act));
                    }
                }
                epi_bar_sync();                           // last_flag is rewritten by the next chunk
            }
        }
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
