// Multi-head self-attention (paper: Prompts appendix, task 6):
//     head_i = softmax(Q_i K_i^T / sqrt(d_k)) V_i,   Y = Concat(head_1 .. head_h)
// Q, K, V, Y are N x d_model row-major; head i owns columns [i d_k, (i+1) d_k).  No mask.
//
// mhsa_umma_kernel<DK> (bf16, d_k = 64 or 128): one CTA per (256 query rows, head).  The scores
// never leave the SM: S = Q K^T is a tcgen05.mma into tensor memory, the softmax threads turn it
// into bf16 probabilities in shared memory, and O += P V is a second tcgen05.mma whose
// accumulator stays in tensor memory for the whole sweep over the keys (online softmax with a
// running maximum).  Warp roles:
//   warp 0      TMA producer: the two 128-row Q tiles once, then K_0, V_0, K_1, V_1, ... through a ring
//   warp 1      one lane issues the MMAs of query tile 0: S_0,j = Q_0 K_j^T and O_0 += P_0,j V_j
//   warp 2      one lane issues the MMAs of query tile 1
//   warp 3      spare (completes the control warpgroup, which gives most of its registers away)
//   warps 4-7   softmax + output for query tile 0 (one thread per query row = one TMEM lane)
//   warps 8-11  the same for query tile 1
// (One lane for both tiles was the bottleneck: a tcgen05.mma costs its issuer about 60 cycles and
// every block also costs it six barrier waits, about 3000 cycles per key block in all, more than
// the tensor pipe or the special-function unit need.)
// The two query tiles alternate on the tensor pipe: while one tile's threads exponentiate, the
// other tile's MMAs run.  The running maximum is only raised when a row's new maximum exceeds it
// by more than 2^8 (in the exp2 domain): the accumulator is then rescaled in tensor memory;
// otherwise probabilities are simply taken relative to the stale maximum, which changes
// nothing mathematically because numerator and denominator carry the same factor.
//
// mhsa_generic_kernel<T> (any d_k <= 256, fp32 or bf16, any alignment): one warp per (query row,
// head), keys in groups of 32 (one score per lane), FMA pipes only.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

template <int DK>
struct MhsaCfg {
    static_assert(DK == 64 || DK == 128, "d_k must be 64 or 128");
    static constexpr int BQ = 128;                       // query rows per tile (TMEM lanes)
    static constexpr int kQTiles = 2;                    // query tiles per CTA
    static constexpr int BKV = 128;                      // keys per block
    static constexpr int kChunks = DK / 64;              // 64-column (128-byte) swizzle atoms per row
    static constexpr int kChunkBytes = 128 * 128;        // 128 rows x 128 bytes
    static constexpr int kTileBytes = kChunks * kChunkBytes;      // one Q tile, K block or V block
    static constexpr int kPBytes = 2 * kChunkBytes;      // 128 x 128 bf16 probabilities
    // K blocks are released early in an iteration and V blocks late, so each has its own ring:
    // the next K block has almost a whole iteration to arrive even with a single slot, the V
    // ring is double-buffered
    static constexpr int kKSlots = DK == 64 ? 3 : 1;
    static constexpr int kVSlots = DK == 64 ? 3 : 2;
    // 12 warps = 3 warpgroups: control (producer, MMA lane of tile 0, MMA lane of tile 1, one spare
    // warp) and one softmax warpgroup per query tile.  Three warps share each SM sub-partition's
    // 16384 registers, so a launch gives every thread 168; the control warpgroup hands most of
    // its share back and the softmax warpgroups, which hold a whole row of scores, take it.
    // (With 48 registers the MMA lanes of the d_k = 128 instantiation spilled two values that they
    // re-read every key block; 56 is what the pool leaves beside 2 x 128 x 224.)
    static constexpr int kThreads = 384;
    static constexpr int kLaunchRegs = 168, kControlRegs = 56, kSoftmaxRegs = 224;
    static_assert(128 * kControlRegs + 256 * kSoftmaxRegs <= kThreads * kLaunchRegs, "register shares exceed the launch's pool");
    static constexpr int kTmemCols = 512;                // S0, S1: 2 x 128; O0, O1: 2 x DK; P0, P1: 2 x 64
    static constexpr int kColS = 0, kColO = 256;
    // d_k = 64 leaves 128 columns of tensor memory for the probabilities (two bf16 per column),
    // which the P V product then reads as its A operand; at d_k = 128 they go through shared memory
    static constexpr bool kPInTmem = DK == 64;
    static constexpr int kColP = 384;
    static constexpr int kOffP = kQTiles * kTileBytes;
    static constexpr int kOffK = kOffP + (kPInTmem ? 0 : kQTiles * kPBytes);
    static constexpr int kOffV = kOffK + kKSlots * kTileBytes;
    static constexpr int kSmemBytes = 256 + 1024 + kOffV + kVSlots * kTileBytes;
    static constexpr float kRescaleThreshold = 8.0f;     // log2 units
    // Softmax warps overlap the round trips of their barrier waits with arithmetic (the abort flag
    // is loaded beside the wait for the scores, the previous P V is polled once before the
    // exponentials).  Measured at N = 16384 with 16 heads: d_k = 64 1375 -> 1267 us, but
    // d_k = 128 1765 -> 2024 us: there the tensor pipe is the busy unit, K has a single slot, and
    // softmax warps that arrive sooner make the two tiles' MMAs queue up in a worse order.
    static constexpr bool kOverlapWaits = DK == 64;
};

struct MhsaShared {
    uint64_t k_full[3], k_empty[3], v_full[3], v_empty[3];
    uint64_t q_full;
    uint64_t s_full[2], s_free[2], p_full[2], pv_done[2];
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
};
static_assert(sizeof(MhsaShared) <= 256, "barrier block");

// Wait sites reported on a time-out: 1 producer/free K slot, 2 producer/free V slot, 3 MMA/Q,
// 4 MMA/K block, 5 MMA/V block, 6 MMA/scores read, 7 MMA/probabilities, 8 softmax/scores,
// 9 softmax/previous P V, 10 softmax/final accumulator.
template <int DK>
__global__ void __launch_bounds__(MhsaCfg<DK>::kThreads, 1)
mhsa_umma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, __nv_bfloat16* __restrict__ Y, int N, int d_model,
                 float scale_log2, int* __restrict__ status) {
    using C = MhsaCfg<DK>;
    extern __shared__ uint8_t smem_raw[];
    MhsaShared* sh = reinterpret_cast<MhsaShared*>(smem_raw);
    const uint32_t data_base = (ptx::smem_u32(smem_raw) + 256 + 1023) & ~1023u;
    uint8_t* data = smem_raw + (data_base - ptx::smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head = blockIdx.y;
    const int q0 = blockIdx.x * (C::kQTiles * C::BQ);
    const int nblk = (N + C::BKV - 1) / C::BKV;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 3; ++s) {
            ptx::mbar_init(&sh->k_full[s], 1);
            ptx::mbar_init(&sh->k_empty[s], 2);            // released by both tiles' MMA lanes
            ptx::mbar_init(&sh->v_full[s], 1);
            ptx::mbar_init(&sh->v_empty[s], 2);
        }
        ptx::mbar_init(&sh->q_full, 1);
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(&sh->s_full[t], 1);
            ptx::mbar_init(&sh->s_free[t], C::BQ);
            ptx::mbar_init(&sh->p_full[t], C::BQ);
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
        ptx::tmem_alloc(&sh->tmem_base, C::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    ptx::tcgen05_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    ptx::griddep_wait();

    if (warp < 4) {
        // control warpgroup: keeps few registers, the rest goes back to the pool
        ptx::setmaxnreg_dec<C::kControlRegs>();
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer
            if (lane == 0) {
                ptx::mbar_arrive_expect_tx(&sh->q_full, C::kQTiles * C::kTileBytes);
                for (int t = 0; t < C::kQTiles; ++t)
                    for (int c = 0; c < C::kChunks; ++c)
                        ptx::tma_load_2d(data + t * C::kTileBytes + c * C::kChunkBytes, &map_q, &sh->q_full,
                                         head * DK + c * 64, q0 + t * C::BQ);
                bool ok = true;
                int site = 0, j = 0, done_k = 0, done_v = 0;
                for (; ok && j < nblk; ++j) {
                    {
                        const int s = j % C::kKSlots;
                        const uint32_t ph = (j / C::kKSlots) & 1;
                        if (sh->abort || (site = 1, !ptx::mbar_wait(&sh->k_empty[s], ph ^ 1))) { ok = false; break; }
                        ptx::mbar_arrive_expect_tx(&sh->k_full[s], C::kTileBytes);
                        for (int c = 0; c < C::kChunks; ++c)
                            ptx::tma_load_2d(data + C::kOffK + s * C::kTileBytes + c * C::kChunkBytes, &map_k, &sh->k_full[s],
                                             head * DK + c * 64, j * C::BKV);
                        done_k = j + 1;
                    }
                    {
                        const int s = j % C::kVSlots;
                        const uint32_t ph = (j / C::kVSlots) & 1;
                        if (sh->abort || (site = 2, !ptx::mbar_wait(&sh->v_empty[s], ph ^ 1))) { ok = false; break; }
                        ptx::mbar_arrive_expect_tx(&sh->v_full[s], C::kTileBytes);
                        for (int c = 0; c < C::kChunks; ++c)
                            ptx::tma_load_2d(data + C::kOffV + s * C::kTileBytes + c * C::kChunkBytes, &map_v, &sh->v_full[s],
                                             head * DK + c * 64, j * C::BKV);
                        done_v = j + 1;
                    }
                }
                if (!ok) {
                    report_timeout(status, site);
                    sh->abort = 1;
                    // copies already issued must land before the CTA may exit
                    ptx::mbar_wait(&sh->q_full, 0);
                    for (int b = 1; b <= C::kKSlots && b <= done_k; ++b)
                        ptx::mbar_wait(&sh->k_full[(done_k - b) % C::kKSlots], ((done_k - b) / C::kKSlots) & 1);
                    for (int b = 1; b <= C::kVSlots && b <= done_v; ++b)
                        ptx::mbar_wait(&sh->v_full[(done_v - b) % C::kVSlots], ((done_v - b) / C::kVSlots) & 1);
                }
            }
        } else if (warp == 1 || warp == 2) {
            // ------------------------------------------------------------ MMA issuers, one per query tile
            if (lane == 0) {
                const int t = warp - 1;
                constexpr uint32_t idesc_s = ptx::umma_idesc_bf16(C::BQ, C::BKV, false, false);   // Q, K: both K-major
                constexpr uint32_t idesc_o = ptx::umma_idesc_bf16(C::BQ, DK, false, true);        // P K-major, V MN-major
                bool ok = true;
                int site = 0;
                // Lean issuing loop (this lane is on the critical path): shared-memory descriptors are a
                // constant high word plus a low word (start address in 16-byte units | leading offset
                // << 16) advanced by constants; ring slots and phases wrap by comparison; the abort flag
                // is read once per block.
                constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);   // stride 1024 B, version 1, 128-B swizzle
                auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
                auto lo_k = [&](uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | ((16u >> 4) << 16); };                          // K-major
                auto lo_mn = [&](uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | ((uint32_t)(C::kChunkBytes >> 4) << 16); };    // MN-major
                const uint32_t q_lo = lo_k(data_base + t * C::kTileBytes);
                const uint32_t p_lo = lo_k(data_base + C::kOffP + t * C::kPBytes);
                const uint32_t k_lo0 = lo_k(data_base + C::kOffK), v_lo0 = lo_mn(data_base + C::kOffV);
                const uint32_t d_s = tmem_base + C::kColS + t * C::BKV, d_o = tmem_base + C::kColO + t * DK;
                const uint32_t p_tmem = tmem_base + C::kColP + t * 64;
                // S_t = Q_t K^T, contraction over d_k in steps of 16 (32 bytes inside a 128-byte row)
                auto issue_s = [&](uint32_t k_lo) {
    #pragma unroll
                    for (int ks = 0; ks < DK / 16; ++ks) {
                        const uint32_t off = (uint32_t)(((ks >> 2) * C::kChunkBytes + (ks & 3) * 32) >> 4);
                        ptx::umma_bf16(d_s, desc(q_lo + off), desc(k_lo + off), idesc_s, ks != 0);
                    }
                    ptx::umma_commit(&sh->s_full[t]);
                };
                // O_t (+)= P_t V, contraction over the 128 keys in steps of 16 (16 rows of V)
                auto issue_pv = [&](uint32_t v_lo, bool first) {
    #pragma unroll
                    for (int ks = 0; ks < C::BKV / 16; ++ks) {
                        const uint32_t p_off = (uint32_t)(((ks >> 2) * C::kChunkBytes + (ks & 3) * 32) >> 4);
                        if (C::kPInTmem)
                            ptx::umma_bf16_tmem_a(d_o, p_tmem + ks * 8, desc(v_lo + (uint32_t)(ks * (2048 >> 4))), idesc_o, !first || ks != 0);
                        else
                            ptx::umma_bf16(d_o, desc(p_lo + p_off), desc(v_lo + (uint32_t)(ks * (2048 >> 4))), idesc_o, !first || ks != 0);
                    }
                    ptx::umma_commit(&sh->pv_done[t]);
                };
                int ks_slot = 0, vs_slot = 0;                 // ring slots of K block j + 1 and of V block j
                uint32_t k_ph = 0, v_ph = 0;
                if (sh->abort || (site = 3, !ptx::mbar_wait(&sh->q_full, 0)) || (site = 4, !ptx::mbar_wait(&sh->k_full[0], 0))) ok = false;
                if (ok) {
                    ptx::tcgen05_fence_after_sync();
                    issue_s(k_lo0);
                    ptx::umma_commit(&sh->k_empty[0]);
                }
                if (++ks_slot == C::kKSlots) { ks_slot = 0; k_ph ^= 1; }
                for (int j = 0; ok && j < nblk; ++j) {
                    if (sh->abort) { ok = false; break; }
                    if (j + 1 < nblk) {
                        // the scores of block j + 1 as soon as the softmax threads hold block j in registers
                        if ((site = 4, !ptx::mbar_wait(&sh->k_full[ks_slot], k_ph))) { ok = false; break; }
                        if ((site = 6, !ptx::mbar_wait(&sh->s_free[t], j & 1))) { ok = false; break; }
                        ptx::tcgen05_fence_after_sync();
                        issue_s(k_lo0 + (uint32_t)ks_slot * (uint32_t)(C::kTileBytes >> 4));
                        ptx::umma_commit(&sh->k_empty[ks_slot]);
                        if (++ks_slot == C::kKSlots) { ks_slot = 0; k_ph ^= 1; }
                    }
                    if ((site = 5, !ptx::mbar_wait(&sh->v_full[vs_slot], v_ph))) { ok = false; break; }
                    if ((site = 7, !ptx::mbar_wait(&sh->p_full[t], j & 1))) { ok = false; break; }
                    ptx::tcgen05_fence_after_sync();
                    issue_pv(v_lo0 + (uint32_t)vs_slot * (uint32_t)(C::kTileBytes >> 4), j == 0);
                    ptx::umma_commit(&sh->v_empty[vs_slot]);
                    if (++vs_slot == C::kVSlots) { vs_slot = 0; v_ph ^= 1; }
                }
                if (!ok) {
                    report_timeout(status, site);
                    sh->abort = 1;
                }
                // nothing may be in flight on the tensor pipe when tensor memory is freed
                ptx::umma_commit(&sh->drain);
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
        const float2 scale2 = make_float2(scale_log2, scale_log2);
        float m_used = 0.0f;
        float2 l2[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
        bool ok = true;
        int site = 8;
        // Every serial step of this loop is paid once per key block by a warp that has only one
        // other warp on its sub-partition to hide behind, so the abort flag is read once per block
        // (two more reads cost 5 % at d_k = 64); a wait whose partner has given up runs out by itself.
        for (int j = 0; j < nblk; ++j) {
            bool got;
            if (C::kOverlapWaits) {
                const int aborted = sh->abort;           // its latency overlaps the wait's
                got = ptx::mbar_wait(&sh->s_full[t], j & 1) && !aborted;
            } else {
                got = !sh->abort && ptx::mbar_wait(&sh->s_full[t], j & 1);
            }
            got = __all_sync(0xffffffffu, got);
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();
            // the whole row of scores into registers, then the tensor-memory block is free again
            uint32_t v[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32(s_addr + c * 32, v[c]);
            ptx::tmem_ld_wait();
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive(&sh->s_free[t]);
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
            // one early look at the previous P V (it has usually finished by now), so that the
            // barrier's round trip overlaps the exponentials instead of following them
            if (C::kOverlapWaits && !prev_done) prev_done = ptx::mbar_try_wait(&sh->pv_done[t], (j - 1) & 1);
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
            if (!(C::kOverlapWaits ? __all_sync(0xffffffffu, prev_done) : prev_done)) {
                // the previous P V still reads this tile's P buffer until it has finished
                got = __all_sync(0xffffffffu, ptx::mbar_wait(&sh->pv_done[t], (j - 1) & 1));
                if (!got) { ok = false; site = 9; break; }
            }
            if (C::kPInTmem) {
                // 128 probabilities = 64 packed columns of this thread's lane
                uint32_t w[32];
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) w[i] = v[2 * hh + (i >> 4)][i & 15];
                    ptx::tmem_st_32x32(lane_base + C::kColP + t * 64 + hh * 32, w);
                }
                ptx::tmem_st_wait();
            } else {
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
            }
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive(&sh->p_full[t]);
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

    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tcgen05_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ---------------------------------------------------------------- generic kernel (FMA pipes)

constexpr int kMhsaGenericMaxDk = 256;
constexpr int kMhsaGenericWarps = 4;

template <typename T> __device__ __forceinline__ float mhsa_to_f32(T x);
template <> __device__ __forceinline__ float mhsa_to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float mhsa_to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T mhsa_from_f32(float x);
template <> __device__ __forceinline__ float mhsa_from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 mhsa_from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// One warp per (query row, head): 32 keys at a time, one score per lane; running maximum and
// sum as in any online softmax; each lane accumulates output columns lane, lane + 32, ...
template <typename T>
__global__ void __launch_bounds__(kMhsaGenericWarps * 32)
mhsa_generic_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V, T* __restrict__ Y, int N,
                    int d_model, int heads, float scale) {
    __shared__ float q_sh[kMhsaGenericWarps][kMhsaGenericMaxDk];
    ptx::griddep_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t idx = (int64_t)blockIdx.x * kMhsaGenericWarps + warp;
    if (idx >= (int64_t)N * heads) return;
    const int row = (int)(idx / heads), head = (int)(idx % heads);
    const int dk = d_model / heads;
    const size_t col0 = (size_t)head * dk;
    for (int d = lane; d < dk; d += 32) q_sh[warp][d] = mhsa_to_f32(Q[(size_t)row * d_model + col0 + d]);
    __syncwarp();
    constexpr int kPerLane = kMhsaGenericMaxDk / 32;
    float acc[kPerLane];
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) acc[i] = 0.0f;
    float m = -INFINITY, l = 0.0f;
    for (int k0 = 0; k0 < N; k0 += 32) {
        const int k = k0 + lane;
        float s = -INFINITY;
        if (k < N) {
            const T* k_row = K + (size_t)k * d_model + col0;
            float dot = 0.0f;
            for (int d = 0; d < dk; ++d) dot = fmaf(q_sh[warp][d], mhsa_to_f32(k_row[d]), dot);
            s = dot * scale;
        }
        float cm = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
        const float m_new = fmaxf(m, cm);
        const float alpha = expf(m - m_new);             // 0 on the first group (m = -inf)
        const float p = k < N ? expf(s - m_new) : 0.0f;
        float ps = p;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
        l = l * alpha + ps;
#pragma unroll
        for (int i = 0; i < kPerLane; ++i) acc[i] *= alpha;
        const int kn = min(32, N - k0);
        for (int kk = 0; kk < kn; ++kk) {
            const float pk = __shfl_sync(0xffffffffu, p, kk);
            const T* v_row = V + (size_t)(k0 + kk) * d_model + col0;
#pragma unroll
            for (int i = 0; i < kPerLane; ++i) {
                const int d = lane + 32 * i;
                if (d < dk) acc[i] = fmaf(pk, mhsa_to_f32(v_row[d]), acc[i]);
            }
        }
        m = m_new;
    }
    const float inv = 1.0f / l;
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        const int d = lane + 32 * i;
        if (d < dk) Y[(size_t)row * d_model + col0 + d] = mhsa_from_f32<T>(acc[i] * inv);
    }
}

}  // namespace optiml
