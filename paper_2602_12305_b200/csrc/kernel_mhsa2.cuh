// Multi-head self-attention at d_k = 128 as a CTA PAIR (paper: Prompts appendix, task 6; see
// kernel_mhsa.cuh for the operation and for the single-CTA kernel this one grew out of).
//
// Why a pair.  In the single-CTA kernel both operands of every tcgen05.mma come from shared
// memory, and at d_k = 128 the shared-memory data path, not the tensor pipe, sets the pace: per
// pair of key blocks 256 KiB of MMA operands, 64 KiB of probabilities written by the softmax
// threads and 64 KiB of K and V written by TMA, 384 KiB at 128 bytes per clock = 3072 cycles
// against 2048 cycles of MMA time.  With tcgen05.mma.cta_group::2 the two CTAs of a cluster run
// one M = 256 product over their two 128-row query tiles, and the B operand (the key block for
// S = Q K^T, the value block for O += P V) is SPLIT between them: CTA r stages keys
// [64 r, 64 r + 64) of every key block and columns [64 r, 64 r + 64) of every value block.  Per
// CTA that is 192 KiB of operand reads and 32 KiB of TMA writes per pair of key blocks instead
// of 256 + 64, and the smaller K / V slots leave room for three of each (the single-CTA kernel
// has one K slot).  Each CTA fetches its own halves with plain TMA loads; nothing is multicast.
//
// A CTA still owns two query tiles (so a pair covers 512 query rows) and everything per row --
// scores to registers, online softmax with the lazily raised maximum, probabilities to shared
// memory, rescaling of O in tensor memory, the final division -- is as in kernel_mhsa.cuh.
// What changes is who signals whom:
//   * the two MMA lanes (one per query tile) run in the LEADER (rank 0) only;
//   * "full" barriers of Q, K and V slots live in the leader and count the bytes of both CTAs;
//   * tcgen05.commit arrives on the barriers of BOTH CTAs ("slot empty", "scores ready",
//     "P V done");
//   * the softmax warps of both CTAs arrive (one lane per warp) on the leader's "scores read" and
//     "probabilities written" barriers.
// The pair meets at the hardware cluster barrier after set-up and before exit; every other wait
// is an mbarrier wait with a limit.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"
#include "kernel_mhsa.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

struct Mhsa2Cfg {
    static constexpr int DK = 128;
    static constexpr int BQ = 128;                       // query rows per tile (TMEM lanes)
    static constexpr int kQTiles = 2;                    // query tiles per CTA
    static constexpr int BKV = 128;                      // keys per block (64 staged by each CTA)
    static constexpr int kChunkBytes = 128 * 128;        // 128 rows x 128 bytes (one 64-column swizzle atom column)
    static constexpr int kQTileBytes = 2 * kChunkBytes;  // 128 rows x 128 columns
    static constexpr int kKChunkBytes = 64 * 128;        // this CTA's 64 keys x 64 columns
    static constexpr int kKHalfBytes = 2 * kKChunkBytes; // this CTA's 64 keys x 128 columns
    static constexpr int kVHalfBytes = kChunkBytes;      // 128 keys x this CTA's 64 columns
    static constexpr int kPBytes = 2 * kChunkBytes;      // 128 x 128 bf16 probabilities
    static constexpr int kKSlots = 3, kVSlots = 3;
    static constexpr int kThreads = 384;
    static constexpr int kLaunchRegs = 168, kControlRegs = 88, kSoftmaxRegs = 208;   // (56 / 224 spilled two values here)
    static_assert(128 * kControlRegs + 256 * kSoftmaxRegs <= kThreads * kLaunchRegs, "register shares exceed the launch's pool");
    static constexpr int kTmemCols = 512;                // S0, S1: 2 x 128; O0, O1: 2 x 128
    static constexpr int kColS = 0, kColO = 256;
    static constexpr int kOffP = kQTiles * kQTileBytes;
    static constexpr int kOffK = kOffP + kQTiles * kPBytes;
    static constexpr int kOffV = kOffK + kKSlots * kKHalfBytes;
    static constexpr int kSmemBytes = 256 + 1024 + kOffV + kVSlots * kVHalfBytes;
    static constexpr float kRescaleThreshold = 8.0f;     // log2 units
};

struct Mhsa2Shared {
    uint64_t k_full[3], k_empty[3], v_full[3], v_empty[3];
    uint64_t q_full;
    uint64_t s_full[2], s_free[2], p_full[2], pv_done[2];
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
};
static_assert(sizeof(Mhsa2Shared) <= 256, "barrier block");

// Wait sites reported on a time-out: as in kernel_mhsa.cuh (1 producer/free K slot, 2 producer/free
// V slot, 3 MMA/Q, 4 MMA/K block, 5 MMA/V block, 6 MMA/scores read, 7 MMA/probabilities,
// 8 softmax/scores, 9 softmax/previous P V, 10 softmax/final accumulator).
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Mhsa2Cfg::kThreads, 1)
mhsa_umma2_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, __nv_bfloat16* __restrict__ Y, int N, int d_model,
                  float scale_log2, int* __restrict__ status) {
    using C = Mhsa2Cfg;
    constexpr int DK = C::DK;
    extern __shared__ uint8_t smem_raw[];
    Mhsa2Shared* sh = reinterpret_cast<Mhsa2Shared*>(smem_raw);
    const uint32_t data_base = (ptx::smem_u32(smem_raw) + 256 + 1023) & ~1023u;
    uint8_t* data = smem_raw + (data_base - ptx::smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();        // 0 = leader of the pair
    const int head = blockIdx.y;
    const int q0 = (int)blockIdx.x * (C::kQTiles * C::BQ);    // consecutive CTAs of a pair: consecutive 256-row slabs
    const int nblk = (N + C::BKV - 1) / C::BKV;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 3; ++s) {
            ptx::mbar_init(&sh->k_full[s], 2);             // one arrive.expect_tx per producer of the pair
            ptx::mbar_init(&sh->k_empty[s], 2);            // released by both tiles' MMA lanes
            ptx::mbar_init(&sh->v_full[s], 2);
            ptx::mbar_init(&sh->v_empty[s], 2);
        }
        ptx::mbar_init(&sh->q_full, 2);
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(&sh->s_full[t], 1);
            ptx::mbar_init(&sh->s_free[t], 8);             // one lane of each softmax warp of the tile, both CTAs
            ptx::mbar_init(&sh->p_full[t], 8);
            ptx::mbar_init(&sh->pv_done[t], 1);
        }
        ptx::mbar_init(&sh->drain, 2);
        sh->abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        ptx::prefetch_tensormap(&map_q);
        ptx::prefetch_tensormap(&map_k);
        ptx::prefetch_tensormap(&map_v);
    }
    if (warp == 1) {
        ptx::tmem_alloc_2cta(&sh->tmem_base, C::kTmemCols);
        ptx::tmem_relinquish_2cta();
    }
    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                                 // the peer's barriers exist before anyone signals them
    ptx::tcgen05_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    ptx::griddep_wait();

    if (warp < 4) {
        // control warpgroup: keeps few registers, the rest goes back to the pool
        ptx::setmaxnreg_dec<C::kControlRegs>();
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer (both CTAs, own halves)
            if (lane == 0) {
                const uint32_t q_full_l = ptx::mapa_shared(ptx::smem_u32(&sh->q_full), 0);
                const uint32_t k_full_l = ptx::mapa_shared(ptx::smem_u32(&sh->k_full[0]), 0);
                const uint32_t v_full_l = ptx::mapa_shared(ptx::smem_u32(&sh->v_full[0]), 0);
                ptx::mbar_arrive_expect_tx_cluster(q_full_l, C::kQTiles * C::kQTileBytes);
                for (int t = 0; t < C::kQTiles; ++t)
                    for (int c = 0; c < 2; ++c)
                        ptx::tma_load_2d_2cta(data + t * C::kQTileBytes + c * C::kChunkBytes, &map_q, q_full_l,
                                              head * DK + c * 64, q0 + t * C::BQ);
                bool ok = true;
                int site = 0, j = 0;
                int ks = 0, vs = 0;
                uint32_t kph = 0, vph = 0;
                for (; ok && j < nblk; ++j) {
                    if (sh->abort || (site = 1, !ptx::mbar_wait(&sh->k_empty[ks], kph ^ 1))) { ok = false; break; }
                    ptx::mbar_arrive_expect_tx_cluster(k_full_l + 8u * ks, C::kKHalfBytes);
                    for (int c = 0; c < 2; ++c)
                        ptx::tma_load_2d_2cta(data + C::kOffK + ks * C::kKHalfBytes + c * C::kKChunkBytes, &map_k,
                                              k_full_l + 8u * ks, head * DK + c * 64, j * C::BKV + (int)rank * 64);
                    if (++ks == C::kKSlots) { ks = 0; kph ^= 1; }
                    if (sh->abort || (site = 2, !ptx::mbar_wait(&sh->v_empty[vs], vph ^ 1))) { ok = false; break; }
                    ptx::mbar_arrive_expect_tx_cluster(v_full_l + 8u * vs, C::kVHalfBytes);
                    ptx::tma_load_2d_2cta(data + C::kOffV + vs * C::kVHalfBytes, &map_v, v_full_l + 8u * vs,
                                          head * DK + (int)rank * 64, j * C::BKV);
                    if (++vs == C::kVSlots) { vs = 0; vph ^= 1; }
                }
                if (!ok) {
                    report_timeout(status, site);
                    sh->abort = 1;
                    // Copies already issued must land before the CTA may exit.  Their bytes are counted
                    // in the leader, so only the leader can watch them; its own MMA lanes stop at their
                    // next bounded wait, and the peer is held by the cluster barrier at the end.  The
                    // leader's lanes consume every slot in order, so waiting for the last phase of each
                    // slot that was armed is enough.
                    if (rank == 0) {
                        ptx::mbar_wait(&sh->q_full, 0);
                        for (int b = 1; b <= C::kKSlots && b <= j; ++b)
                            ptx::mbar_wait(&sh->k_full[(j - b) % C::kKSlots], ((j - b) / C::kKSlots) & 1);
                        for (int b = 1; b <= C::kVSlots && b <= j; ++b)
                            ptx::mbar_wait(&sh->v_full[(j - b) % C::kVSlots], ((j - b) / C::kVSlots) & 1);
                    }
                }
            }
        } else if ((warp == 1 || warp == 2) && rank == 0) {
            // ------------------------------------------------------------ MMA issuers (leader), one per query tile
            if (lane == 0) {
                const int t = warp - 1;
                constexpr uint32_t idesc_s = ptx::umma_idesc_bf16(2 * C::BQ, C::BKV, false, false);   // Q, K: both K-major
                constexpr uint32_t idesc_o = ptx::umma_idesc_bf16(2 * C::BQ, DK, false, true);        // P K-major, V MN-major
                bool ok = true;
                int site = 0;
                constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);   // stride 1024 B, version 1, 128-B swizzle
                auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
                auto lo_k = [&](uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | ((16u >> 4) << 16); };                          // K-major
                auto lo_mn = [&](uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | ((uint32_t)(C::kChunkBytes >> 4) << 16); };    // MN-major
                const uint32_t q_lo = lo_k(data_base + t * C::kQTileBytes);
                const uint32_t p_lo = lo_k(data_base + C::kOffP + t * C::kPBytes);
                const uint32_t k_lo0 = lo_k(data_base + C::kOffK), v_lo0 = lo_mn(data_base + C::kOffV);
                const uint32_t d_s = tmem_base + C::kColS + t * C::BKV, d_o = tmem_base + C::kColO + t * DK;
                // S_t = Q_t K^T over both CTAs' query tiles t; contraction over d_k in steps of 16 (32 bytes
                // inside a 128-byte row).  Q: 64-column chunks 16 KiB apart; this CTA's 64 keys: 8 KiB apart.
                auto issue_s = [&](uint32_t k_lo) {
#pragma unroll
                    for (int ks = 0; ks < DK / 16; ++ks) {
                        const uint32_t q_off = (uint32_t)(((ks >> 2) * C::kChunkBytes + (ks & 3) * 32) >> 4);
                        const uint32_t k_off = (uint32_t)(((ks >> 2) * C::kKChunkBytes + (ks & 3) * 32) >> 4);
                        ptx::umma_bf16_2cta(d_s, desc(q_lo + q_off), desc(k_lo + k_off), idesc_s, ks != 0);
                    }
                    ptx::umma_commit_2cta(&sh->s_full[t]);
                };
                // O_t (+)= P_t V, contraction over the 128 keys in steps of 16 (16 rows of this CTA's 64 columns of V)
                auto issue_pv = [&](uint32_t v_lo, bool first) {
#pragma unroll
                    for (int ks = 0; ks < C::BKV / 16; ++ks) {
                        const uint32_t p_off = (uint32_t)(((ks >> 2) * C::kChunkBytes + (ks & 3) * 32) >> 4);
                        ptx::umma_bf16_2cta(d_o, desc(p_lo + p_off), desc(v_lo + (uint32_t)(ks * (2048 >> 4))), idesc_o, !first || ks != 0);
                    }
                    ptx::umma_commit_2cta(&sh->pv_done[t]);
                };
                int ks_slot = 0, vs_slot = 0;                 // ring slots of K block j + 1 and of V block j
                uint32_t k_ph = 0, v_ph = 0;
                if (sh->abort || (site = 3, !ptx::mbar_wait(&sh->q_full, 0)) || (site = 4, !ptx::mbar_wait(&sh->k_full[0], 0))) ok = false;
                if (ok) {
                    ptx::tcgen05_fence_after_sync();
                    issue_s(k_lo0);
                    ptx::umma_commit_2cta(&sh->k_empty[0]);
                }
                if (++ks_slot == C::kKSlots) { ks_slot = 0; k_ph ^= 1; }
                for (int j = 0; ok && j < nblk; ++j) {
                    if (sh->abort) { ok = false; break; }
                    if (j + 1 < nblk) {
                        // the scores of block j + 1 as soon as the softmax threads hold block j in registers
                        if ((site = 4, !ptx::mbar_wait(&sh->k_full[ks_slot], k_ph))) { ok = false; break; }
                        if ((site = 6, !ptx::mbar_wait(&sh->s_free[t], j & 1))) { ok = false; break; }
                        ptx::tcgen05_fence_after_sync();
                        issue_s(k_lo0 + (uint32_t)ks_slot * (uint32_t)(C::kKHalfBytes >> 4));
                        ptx::umma_commit_2cta(&sh->k_empty[ks_slot]);
                        if (++ks_slot == C::kKSlots) { ks_slot = 0; k_ph ^= 1; }
                    }
                    if ((site = 5, !ptx::mbar_wait(&sh->v_full[vs_slot], v_ph))) { ok = false; break; }
                    if ((site = 7, !ptx::mbar_wait(&sh->p_full[t], j & 1))) { ok = false; break; }
                    ptx::tcgen05_fence_after_sync();
                    issue_pv(v_lo0 + (uint32_t)vs_slot * (uint32_t)(C::kVHalfBytes >> 4), j == 0);
                    ptx::umma_commit_2cta(&sh->v_empty[vs_slot]);
                    if (++vs_slot == C::kVSlots) { vs_slot = 0; v_ph ^= 1; }
                }
                if (!ok) {
                    report_timeout(status, site);
                    sh->abort = 1;
                }
                // nothing may be in flight on the tensor pipe when tensor memory is freed
                ptx::umma_commit_2cta_local(&sh->drain);
                ptx::mbar_wait(&sh->drain, 0);
            }
        }
    } else {
        // softmax warpgroups: wait for their larger share (handed back above)
        ptx::setmaxnreg_inc<C::kSoftmaxRegs>();
        // ------------------------------------------------------------ softmax + output, one thread per query row
        const int t = (warp - 4) >> 2;                   // query tile of this warpgroup
        const int quarter = warp & 3;                    // TMEM lane quarter this warp may touch
        const int r = quarter * 32 + lane;               // row within the tile
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t s_addr = lane_base + C::kColS + t * C::BKV;
        const uint32_t o_addr = lane_base + C::kColO + t * DK;
        uint8_t* p_row = data + C::kOffP + t * C::kPBytes + r * 128;
        // the leader's barriers this warp signals (one lane per warp)
        const uint32_t s_free_l = ptx::mapa_shared(ptx::smem_u32(&sh->s_free[t]), 0);
        const uint32_t p_full_l = ptx::mapa_shared(ptx::smem_u32(&sh->p_full[t]), 0);
        const float2 scale2 = make_float2(scale_log2, scale_log2);
        float m_used = 0.0f;
        float2 l2[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
        bool ok = true;
        int site = 8;
        for (int j = 0; j < nblk; ++j) {
            bool got = !sh->abort && ptx::mbar_wait(&sh->s_full[t], j & 1);
            got = __all_sync(0xffffffffu, got);
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();
            // the whole row of scores into registers, then the tensor-memory block is free again
            uint32_t v[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32(s_addr + c * 32, v[c]);
            ptx::tmem_ld_wait();
            ptx::tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(s_free_l);
            const int nvalid = N - j * C::BKV;
            if (nvalid < C::BKV) {
                // keys past the end of the sequence (zero-filled by TMA) take no part
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c * 32 + i >= nvalid) v[c][i] = __float_as_uint(-INFINITY);
            }
            float mx4[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float a = __uint_as_float(v[c][0]);
#pragma unroll
                for (int i = 1; i < 32; i += 2)
                    a = ptx::fmax3(a, __uint_as_float(v[c][i]), __uint_as_float(v[c][(i + 1) & 31]));
                mx4[c] = a;
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
            bool raise = false;
            if (j == 0) {
                m_used = mx;
            } else if (mx > m_used + C::kRescaleThreshold) {
                raise = true;
            }
            bool prev_done = j == 0;                     // has P V of block j - 1 been waited for?
            if (__any_sync(0xffffffffu, raise)) {
                // the accumulator is rescaled in place once the previous P V has finished
                got = __all_sync(0xffffffffu, ptx::mbar_wait(&sh->pv_done[t], (j - 1) & 1));
                if (!got) { ok = false; site = 9; break; }
                prev_done = true;
                ptx::tcgen05_fence_after_sync();
                const float alpha = raise ? ptx::ex2_approx(m_used - mx) : 1.0f;
                if (raise) {
                    l2[0].x *= alpha; l2[0].y *= alpha; l2[1].x *= alpha; l2[1].y *= alpha;
                    m_used = mx;
                }
#pragma unroll 1
                for (int c = 0; c < DK / 8; ++c) {          // 8 columns at a time: the whole row of scores is live here
                    uint32_t o[8];
                    ptx::tmem_ld_32x8(o_addr + c * 8, o);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    ptx::tmem_st_32x8(o_addr + c * 8, o);
                }
                ptx::tmem_st_wait();
            }
            // probabilities relative to m_used: 2^(s * scale - m), packed to bf16 in place
            const float2 negm2 = make_float2(-m_used, -m_used);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float2 x = ptx::ffma2(make_float2(__uint_as_float(v[c][i]), __uint_as_float(v[c][i + 1])), scale2, negm2);
                    const float2 e = make_float2(ptx::ex2_approx(x.x), ptx::ex2_approx(x.y));
                    l2[(i >> 1) & 1] = ptx::fadd2(l2[(i >> 1) & 1], e);
                    v[c][i >> 1] = pack_bf16x2(e.x, e.y);
                }
            }
            if (!prev_done) {
                // the previous P V still reads this tile's P buffer until it has finished
                got = __all_sync(0xffffffffu, ptx::mbar_wait(&sh->pv_done[t], (j - 1) & 1));
                if (!got) { ok = false; site = 9; break; }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint8_t* atom_row = p_row + (c >> 1) * C::kChunkBytes;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int chunk16 = (c & 1) * 4 + g;
                    *reinterpret_cast<uint4*>(atom_row + ((chunk16 ^ (lane & 7)) << 4)) =
                        make_uint4(v[c][4 * g], v[c][4 * g + 1], v[c][4 * g + 2], v[c][4 * g + 3]);
                }
            }
            ptx::fence_proxy_async_smem();
            ptx::tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(p_full_l);
        }
        if (ok) {
            bool got = !sh->abort && ptx::mbar_wait(&sh->pv_done[t], (nblk - 1) & 1);
            got = __all_sync(0xffffffffu, got);
            if (!got) { ok = false; site = 10; }
        }
        if (!ok) {
            if (lane == 0) report_timeout(status, site);
            sh->abort = 1;
        }
        ptx::griddep_launch_dependents();
        if (ok) {
            ptx::tcgen05_fence_after_sync();
            const float inv = 1.0f / ((l2[0].x + l2[0].y) + (l2[1].x + l2[1].y));
            const int row = q0 + t * C::BQ + r;
            __nv_bfloat16* y_row = Y + (size_t)row * d_model + head * DK;
#pragma unroll 1
            for (int c = 0; c < DK / 32; ++c) {
                uint32_t o[32];
                ptx::tmem_ld_32x32(o_addr + c * 32, o);
                ptx::tmem_ld_wait();
                if (row < N) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint32_t w[4];
#pragma unroll
                        for (int p = 0; p < 4; ++p)
                            w[p] = pack_bf16x2(__uint_as_float(o[g * 8 + 2 * p]) * inv, __uint_as_float(o[g * 8 + 2 * p + 1]) * inv);
                        *reinterpret_cast<uint4*>(y_row + c * 32 + g * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
    }

    __syncwarp();
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
