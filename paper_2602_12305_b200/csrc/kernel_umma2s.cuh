// Streaming form of the CTA-pair tensor-core GEMM (bf16), for problems with FEWER 256 x 256
// tiles than CTA pairs (64 < M <= 512 or so with a long K): every element of B is then used by
// one tile row only, so the problem is a stream over B, and what decides the time is how many
// SMs pull on that stream and how short the fixed part around the main loop is.
//
// One thread-block cluster of 2 S CTAs (S = 1, 2 or 4) per tile.  The cluster holds S CTA pairs
// ("bands"); band b computes the tile over K blocks [KB b / S, KB (b + 1) / S) with
// tcgen05.mma.cta_group::2 exactly as the persistent CTA-pair kernel does (each CTA stages its
// own 128 rows of A and 128 columns of B with plain TMA loads; no load is shared between CTAs).
// With S = 2 the two partial tiles never leave the chip.  After its main loop a CTA (band b,
// half h of its pair) keeps columns [128 b, 128 b + 128) of its 128 rows and hands the other
// 128 columns to its partner, the CTA of the other band with the same h: it copies them from
// tensor memory into its own (now idle) operand ring and one bulk copy moves the 64 KiB into
// the partner's ring through distributed shared memory, counted on the partner's mbarrier.
// Each CTA then adds the two shares in band order (= ascending K, one fixed order), applies
// bias + activation and stores its 128 x 128 block of Y: a reduce-scatter, so the
// epilogue is halved as well, nothing goes through global scratch and nothing is counted with
// atomics.  (Writing the partner's ring with ordinary remote stores instead took 2.8 us for the
// 64 KiB.)  With S = 4 (shapes of at most 18 tiles or so, where two pairs per tile would leave
// half of the SMs idle) the same happens among four CTAs: each keeps a quarter of its columns,
// sends the other three quarters to the three CTAs with the same h and adds four shares in band
// order.
//
//   warp 0      TMA producer (one lane), as in kernel_umma2.cuh
//   warp 1      tensor-memory allocation (256 columns, cta_group::2); MMA-issuing lane in the
//               leader (even rank) of each pair
//   warps 2-9   eight epilogue warps: two per tensor-memory lane quarter, each taking half of
//               the columns (the epilogue is not hidden under a next tile here, so it is
//               spread over twice the warps of the persistent kernel)
//
// The cluster synchronises with the hardware cluster barrier after barrier set-up and before
// exit; every thread executes both whatever happens.  Every other wait is an mbarrier wait
// with a limit; a wait that gives up records the time-out, raises the CTA's abort flag and
// skips the data movement that depended on it.
#pragma once

#include "common.cuh"
#include "kernel_umma2.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

// HM ("half-height"): the pair's tile is 128 rows high, 64 per CTA (tcgen05.mma.cta_group::2 with
// M = 128), for M <= 128.  With 256-row tiles such a problem leaves the second CTA of every pair
// multiplying zero rows while the first pulls 128 rows of A and 128 columns of B through its SM's
// port; here each CTA pulls 64 rows and 128 columns, a quarter less per SM, and both do useful
// work.  The accumulator of a CTA then sits in tensor memory as lanes [0, 64) = its 64 rows x
// columns [0, 128) of the tile and lanes [64, 128) = the same rows x columns [128, 256):
// 128 tensor-memory columns in all.
// BN_ = 128 (the "narrow" form): tiles of 128 columns, 64 per CTA, for shapes whose 256-column
// tiles are too few to give every SM a CTA even with the K split (N = 4096: 16 tiles).
template <bool HM, int BN_ = 256>
struct Umma2sCfgT {
    static_assert(BN_ == 256 || BN_ == 128, "tile width");
    static constexpr int BM = HM ? 128 : 256, BN = BN_, BK = 64;
    static constexpr int kRowsPerCta = BM / 2;
    static constexpr int kABytes = kRowsPerCta * 64 * 2;     // this CTA's rows x 64 k of A
    static constexpr int kBChunkBytes = 64 * 64 * 2;         // 64 k x 64 columns
    static constexpr int kBChunks = BN / 128;                // 64-column chunks of B per CTA
    static constexpr int kBBytes = kBChunks * kBChunkBytes;  // 64 k x this CTA's half of the tile's columns
    static constexpr int kStageBytes = kABytes + kBBytes;    // 32, 24 or 16 KiB
    static constexpr int kStages = 196608 / kStageBytes;     // a 192 KiB ring: 6, 8 or 12 stages
    static constexpr int kEpiWarps = 8;
    static constexpr int kThreads = 64 + 32 * kEpiWarps;
    static constexpr int kTmemCols = HM ? BN / 2 : BN;       // accumulator columns per lane
    // After the main loop the ring is reused: with two pairs per tile one share (the half of this
    // CTA's accumulator that the partner finishes) is received, one is held on its way to the partner.
    static constexpr int kShareBytes = 128 * (kTmemCols / 2) * 4;
    static constexpr int kRecvOffset = 0, kSendOffset = kShareBytes;
    static constexpr int kRingBytes = kStages * kStageBytes;
    static_assert(kStageBytes % 1024 == 0, "swizzle atoms start on 1024-byte boundaries");
    // S pairs per tile: S - 1 received and S - 1 outgoing shares of 128 lanes x (kTmemCols / S) columns
    static_assert(2 * 3 * 128 * (kTmemCols / 4) * 4 <= kRingBytes && kSendOffset + kShareBytes <= kRingBytes, "ring reuse");
    static constexpr int kSmemBytes = kRingBytes + 256 + 1024;
    static constexpr int kMaxSplit = 4;                      // cluster of 8 CTAs
};
using Umma2sCfg = Umma2sCfgT<false>;
using Umma2sHalfCfg = Umma2sCfgT<true>;
static_assert(Umma2sCfg::kSmemBytes >= Umma2sHalfCfg::kSmemBytes && Umma2sCfg::kSmemBytes >= Umma2sCfgT<false, 128>::kSmemBytes &&
              Umma2sCfg::kSmemBytes >= Umma2sCfgT<true, 128>::kSmemBytes && Umma2sCfg::kThreads == Umma2sHalfCfg::kThreads,
              "the resident-cluster counts are queried once, for the form that needs most shared memory");
constexpr int kUmma2sMaxStages = 12;

struct Umma2sPlan {
    int tiles_m, tiles_n, num_kb;
    int split;          // S: CTA pairs per tile = K slices; the cluster has 2 S CTAs
};

struct Umma2sShared {
    uint64_t full[kUmma2sMaxStages];       // used in the pair's leader: bytes of both CTAs land here
    uint64_t empty[kUmma2sMaxStages];      // per CTA, signalled by the leader's commit
    uint64_t tmem_full;                    // per CTA, signalled by the leader's commit
    uint64_t drain;
    uint64_t partner_idle;                 // the partners' main loops are over (S - 1 arrivals): their rings may be written
    uint64_t recv_full;                    // the partners' shares have landed in this CTA's ring
    uint32_t tmem_base;
    volatile int abort;
};
static_assert(sizeof(Umma2sShared) <= 256, "barrier block");

__device__ __forceinline__ void umma2s_epi_bar_sync() { asm volatile("bar.sync 4, 256;" ::: "memory"); }

// tcgen05.commit of a CTA pair that sits at ranks (leader, leader + 1) of a larger cluster.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar, uint32_t leader_rank) {
    const uint16_t mask = (uint16_t)(3u << leader_rank);
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(ptx::smem_u32(bar)), "h"(mask)
        : "memory");
}

// Bulk copy from this CTA's shared memory into the shared memory of another CTA of the cluster;
// the bytes are counted on an mbarrier of the destination CTA.  Addresses and size are
// multiples of 16; dst and bar are cluster addresses (mapa).
__device__ __forceinline__ void bulk_copy_to_cluster(uint32_t dst_cluster, const void* src, uint32_t bytes,
                                                     uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(ptx::smem_u32(src)), "r"(bytes), "r"(bar_cluster)
                 : "memory");
}

template <int ACT, bool HM, int BN_>
__global__ void __launch_bounds__(Umma2sCfgT<HM, BN_>::kThreads, 1)
gemm_umma2s_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                   __nv_bfloat16* __restrict__ Y,
                   const __nv_bfloat16* __restrict__ bias, int M, int N, int K, const __grid_constant__ Umma2sPlan plan,
                   int* __restrict__ status) {
    using C = Umma2sCfgT<HM, BN_>;
    extern __shared__ uint8_t smem_raw[];
    Umma2sShared* sh = reinterpret_cast<Umma2sShared*>(smem_raw);
    const uint32_t ring_base = (ptx::smem_u32(smem_raw) + 256 + 1023) & ~1023u;
    uint8_t* ring = smem_raw + (ring_base - ptx::smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = plan.split;                           // 1 or 2
    const uint32_t rank = ptx::cluster_ctarank();       // 0 .. 2 S - 1
    const uint32_t leader = rank & ~1u;                 // even rank of this CTA's pair
    const uint32_t partner = rank ^ 2u;                 // S = 2: same half of the other band's pair
    const int band = (int)(rank >> 1), hc = (int)(rank & 1);
    const int tile = blockIdx.x / (2 * S);
    const int tm = tile % plan.tiles_m, tn = tile / plan.tiles_m;
    const int kb0 = (int)((int64_t)plan.num_kb * band / S), kb1 = (int)((int64_t)plan.num_kb * (band + 1) / S);

    if (threadIdx.x == 0) {
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(&sh->full[s], 2);              // one arrive.expect_tx per producer of the pair
            ptx::mbar_init(&sh->empty[s], 1);
        }
        ptx::mbar_init(&sh->tmem_full, 1);
        ptx::mbar_init(&sh->drain, 1);
        ptx::mbar_init(&sh->partner_idle, S > 1 ? S - 1 : 1);
        ptx::mbar_init(&sh->recv_full, 1);
        sh->abort = 0;
        ptx::fence_mbar_init();
        // the partner's copy may complete at any time after the cluster barrier below
        if (S > 1) ptx::mbar_arrive_expect_tx(&sh->recv_full, (uint32_t)((S - 1) * (128 * (C::kTmemCols / S) * 4)));
    }
    if (warp == 1) {
        ptx::tmem_alloc_2cta(&sh->tmem_base, C::kTmemCols);
        ptx::tmem_relinquish_2cta();
    }
    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                                // the peers' barriers exist before anyone signals them
    ptx::tcgen05_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    ptx::griddep_wait();
    ptx::griddep_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0, s = 0, ph = 0;
            bool ok = true;
            int site = 0;
            const uint32_t full_leader0 = ptx::mapa_shared(ptx::smem_u32(&sh->full[0]), leader);
            for (int kb = kb0; kb < kb1; ++kb, ++it) {
                if ((site = 1, !ptx::mbar_wait(&sh->empty[s], ph ^ 1))) { ok = false; break; }
                uint8_t* a_dst = ring + s * C::kStageBytes;
                uint8_t* b_dst = a_dst + C::kABytes;
                const uint32_t full_leader = full_leader0 + 8u * s;
                ptx::mbar_arrive_expect_tx_cluster(full_leader, C::kStageBytes);
                ptx::tma_load_2d_2cta(a_dst, &map_a, full_leader, kb * C::BK, tm * C::BM + hc * C::kRowsPerCta);
#pragma unroll
                for (int j = 0; j < C::kBChunks; ++j)
                    ptx::tma_load_2d_2cta(b_dst + j * C::kBChunkBytes, &map_b, full_leader, tn * C::BN + hc * (C::BN / 2) + j * 64,
                                          kb * C::BK);
                if (++s == C::kStages) { s = 0; ph ^= 1; }
            }
            if (!ok) {
                report_timeout(status, site);
                sh->abort = 1;
                // copies already issued must land before the ring is reused or the CTA exits; their
                // bytes are counted on the leader's barriers, which only the leader can watch (its
                // peer is held by the cluster barrier at the end until the leader is through)
                if (hc == 0) {
                    const uint32_t n_back = it < (uint32_t)C::kStages ? it : (uint32_t)C::kStages;
                    for (uint32_t b = 1; b <= n_back; ++b) {
                        const uint32_t j = it - b;
                        ptx::mbar_wait(&sh->full[j % C::kStages], (j / C::kStages) & 1);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (pair leader only)
        if (lane == 0 && hc == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(C::BM, C::BN, /*a_mn_major=*/false, /*b_mn_major=*/true);
            constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);   // stride 1024 B, version 1, 128-B swizzle
            const uint32_t a_lo0 = ((ring_base & 0x3FFFFu) >> 4) | ((16u >> 4) << 16);
            const uint32_t b_lo0 = (((ring_base + C::kABytes) & 0x3FFFFu) >> 4) | ((uint32_t)(C::kBChunkBytes >> 4) << 16);
            auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
            uint32_t s = 0, ph = 0;
            bool ok = true;
            int site = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                if ((site = 4, !ptx::mbar_wait(&sh->full[s], ph))) { ok = false; break; }
                ptx::tcgen05_fence_after_sync();
                const uint32_t a_lo = a_lo0 + s * (uint32_t)(C::kStageBytes >> 4);
                const uint32_t b_lo = b_lo0 + s * (uint32_t)(C::kStageBytes >> 4);
                // A: K-major, 16 k = 32 bytes along the 128-byte row; B: MN-major, 16 k = 16 rows of 128 bytes
                ptx::umma_bf16_2cta(tmem_base, desc(a_lo), desc(b_lo), idesc, kb != kb0);
#pragma unroll
                for (int k4 = 1; k4 < C::BK / 16; ++k4)
                    ptx::umma_bf16_2cta_acc(tmem_base, desc(a_lo + 2 * k4), desc(b_lo + 128 * k4), idesc);
                umma_commit_pair(&sh->empty[s], leader);
                if (++s == C::kStages) { s = 0; ph ^= 1; }
            }
            if (ok) umma_commit_pair(&sh->tmem_full, leader);
            else {
                report_timeout(status, site);
                sh->abort = 1;
            }
            // nothing may be in flight on the tensor pipe past this point
            ptx::umma_commit_2cta_local(&sh->drain);
            ptx::mbar_wait(&sh->drain, 0);
        }
    } else if (S > 2 || C::BN != 256) {
        // ------------------------------------------------------------ epilogue warps, any number of bands and either tile width
        // Tensor-memory lane L of this CTA holds one row of the tile in its kTmemCols columns (256-row
        // tiles: row L, all BN columns; 128-row tiles: row L % 64, columns [BN / 2 (L / 64), + BN / 2)).
        // Band b finishes columns [keep b, keep b + keep) of every lane, keep = kTmemCols / S, and sends
        // chunk d to the CTA of band d with the same h.  A share is 128 lanes x keep columns of fp32,
        // float4 index (column / 4) * 128 + lane; the ring holds S - 1 received shares, then S - 1
        // outgoing ones.  Of the two warps on a lane quarter each takes half of every chunk, 16 columns
        // at a time (keep / 2 is a multiple of 16: the host plans no other split).
        constexpr int CT = C::kTmemCols;
        const int ew = warp - 2, q = warp & 3, ch = ew >> 2;
        const int L = q * 32 + lane;
        const int keep = CT / S, W = keep / 2, ng = W / 16;        // ng = 1 .. 4
        const uint32_t share_bytes = (uint32_t)(128 * keep * 4);
        const uint32_t recv_off = 0, send_off = (uint32_t)(S - 1) * share_bytes;
        const bool rows_live = (int64_t)tm * C::BM + hc * C::kRowsPerCta < M;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        const int64_t m = (int64_t)tm * C::BM + hc * C::kRowsPerCta + (HM ? (L & 63) : L);
        const int64_t n0 = (int64_t)tn * C::BN + (HM ? (q >> 1) * (C::BN / 2) : 0) + band * keep + ch * W;   // first column of Y of this thread
        auto slot_of = [](int other, int self) { return other < self ? other : other - 1; };   // index among the S - 1 others

        uint4 bias_w[4][2];                                 // fetched while the main loop runs
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                const int64_t n = n0 + g * 16 + v * 8;
                bias_w[g][v] = (bias && g < ng && n < N) ? *reinterpret_cast<const uint4*>(bias + n)   // N % 8 == 0
                                                         : make_uint4(0, 0, 0, 0);
            }

        bool ok = (kb1 > kb0) && !sh->abort && ptx::mbar_wait(&sh->tmem_full, 0);
        ok = __all_sync(0xffffffffu, ok);
        int site = 5;
        ptx::tcgen05_fence_after_sync();

        if (S > 1) {
            if (ok && threadIdx.x == 64) {
                for (int d = 0; d < S; ++d)
                    if (d != band) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&sh->partner_idle), (uint32_t)(2 * d + hc)));
            }
            if (ok && rows_live) {
                for (int d = 0; d < S; ++d) {
                    if (d == band) continue;
                    float4* send = reinterpret_cast<float4*>(ring + send_off + (uint32_t)slot_of(d, band) * share_bytes) + L;
                    for (int g = 0; g < ng; ++g) {
                        uint32_t r[16];
                        ptx::tmem_ld_32x16(t_lane + d * keep + ch * W + g * 16, r);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            send[((ch * W + g * 16) / 4 + v) * 128] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                                                  __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                    }
                }
                ptx::fence_proxy_async_smem();
            }
            umma2s_epi_bar_sync();
            if (threadIdx.x == 64 && ok && rows_live) {
                if (ptx::mbar_wait(&sh->partner_idle, 0)) {
                    for (int d = 0; d < S; ++d) {
                        if (d == band) continue;
                        const uint32_t peer = (uint32_t)(2 * d + hc);
                        bulk_copy_to_cluster(ptx::mapa_shared(ring_base + recv_off + (uint32_t)slot_of(band, d) * share_bytes, peer),
                                             ring + send_off + (uint32_t)slot_of(d, band) * share_bytes, share_bytes,
                                             ptx::mapa_shared(ptx::smem_u32(&sh->recv_full), peer));
                    }
                } else {
                    site = 8;
                }
            }
        }

        // this warp's own first columns leave tensor memory while the partners' shares are on their way
        uint32_t racc[16];
        if (ok && rows_live) ptx::tmem_ld_32x16(t_lane + band * keep + ch * W, racc);
        if (S > 1) {
            if (ok && rows_live && !ptx::mbar_wait(&sh->recv_full, 0)) {
                ok = false;
                site = 9;
            }
            ok = __all_sync(0xffffffffu, ok);
        }

        if (ok && rows_live) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (g >= ng) continue;                  // (no break: the loop stays unrolled and bias_w in registers)
                if (g > 0) ptx::tmem_ld_32x16(t_lane + band * keep + ch * W + g * 16, racc);
                ptx::tmem_ld_wait();
                float x[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) x[i] = 0.0f;
                // shares in band order = ascending K, this CTA's own among them
                for (int sb = 0; sb < S; ++sb) {
                    if (sb == band) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) x[i] += __uint_as_float(racc[i]);
                    } else {
                        const float4* recv = reinterpret_cast<const float4*>(ring + recv_off + (uint32_t)slot_of(sb, band) * share_bytes) + L;
                        float4 t[4];
#pragma unroll
                        for (int v = 0; v < 4; ++v) t[v] = recv[((ch * W + g * 16) / 4 + v) * 128];
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            x[4 * v] += t[v].x;
                            x[4 * v + 1] += t[v].y;
                            x[4 * v + 2] += t[v].z;
                            x[4 * v + 3] += t[v].w;
                        }
                    }
                }
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    const int64_t n = n0 + g * 16 + v * 8;
                    const uint4 bw = bias_w[g][v];
                    const uint32_t bwv[4] = {bw.x, bw.y, bw.z, bw.w};
                    uint32_t o[4];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        const float y0 = epilogue<ACT, true>(x[v * 8 + 2 * p], bf16lo_to_f32(bwv[p]));
                        const float y1 = epilogue<ACT, true>(x[v * 8 + 2 * p + 1], bf16hi_to_f32(bwv[p]));
                        o[p] = pack_bf16x2(y0, y1);
                    }
                    if (m < M && n < N) *reinterpret_cast<uint4*>(Y + m * N + n) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
        if (!ok && lane == 0 && kb1 > kb0) {
            report_timeout(status, site);
            sh->abort = 1;
        }
        if (site == 8) report_timeout(status, 8);
    } else if constexpr (!HM) {
        // ------------------------------------------------------------ epilogue warps
        const int ew = warp - 2;                            // 0..7 among the epilogue warps
        const int q = warp & 3;                             // tensor-memory lane quarter this warp may read
        const int colhalf = ew >> 2;                        // which half of the columns this warp takes
        const int row = q * 32 + lane;                      // row within this CTA's 128
        const bool rows_live = (int64_t)tm * C::BM + hc * 128 < M;     // CTA-uniform: any row of this half inside Y?
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        const int chunk_cols = C::BN / S;                   // columns this CTA finishes: 256 or 128
        const float4* recv = reinterpret_cast<const float4*>(ring + C::kRecvOffset) + row;
        const int64_t row0 = (int64_t)tm * C::BM + hc * 128 + q * 32;       // first row of this warp
        const int64_t col0 = (int64_t)tn * C::BN + band * chunk_cols;       // first column of this CTA's chunk
        const int nblk = chunk_cols / 128;                                  // 64-column blocks per warp: 2 or 1

        // The bias of this warp's columns is fetched now, while the main loop runs: at the end nothing
        // but the accumulator stands between the last MMA and the stores.
        uint4 bias_w[2][2][4];                              // [block][32-column group][8 columns]
#pragma unroll
        for (int bi = 0; bi < 2; ++bi)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int64_t n = col0 + ((colhalf * nblk + bi) * 2 + hh) * 32 + v * 8;
                    bias_w[bi][hh][v] = (bias && bi < nblk && n < N) ? *reinterpret_cast<const uint4*>(bias + n)   // N % 8 == 0
                                                                     : make_uint4(0, 0, 0, 0);
                }

        bool ok = (kb1 > kb0) && !sh->abort && ptx::mbar_wait(&sh->tmem_full, 0);
        ok = __all_sync(0xffffffffu, ok);
        int site = 5;
        ptx::tcgen05_fence_after_sync();

        if (S > 1) {
            // this CTA's main loop is over (its ring is idle): tell the partner, which writes into it
            if (ok && threadIdx.x == 64) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&sh->partner_idle), partner));
            if (ok && rows_live) {
                // the partner's 128 columns: tensor memory -> send buffer, float4 index (column / 4) * 128 + row,
                // so that a warp writes (and later reads) 512 contiguous bytes
                float4* send = reinterpret_cast<float4*>(ring + C::kSendOffset) + row;
                const int other = (band ^ 1) * chunk_cols;
#pragma unroll
                for (int gg = 0; gg < 2; ++gg) {
                    const int g = colhalf * 2 + gg;     // 32-column group within the 128 columns
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(t_lane + other + g * 32, r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        send[(g * 8 + v) * 128] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                              __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                }
                ptx::fence_proxy_async_smem();          // these writes are read by the bulk copy
            }
            umma2s_epi_bar_sync();                      // all eight warps (the condition above is uniform over the CTA's warps
                                                        // except for `ok`, which a warp that gave up carries to the end)
            if (threadIdx.x == 64 && ok && rows_live) {
                if (ptx::mbar_wait(&sh->partner_idle, 0))
                    bulk_copy_to_cluster(ptx::mapa_shared(ring_base + C::kRecvOffset, partner), ring + C::kSendOffset,
                                         C::kShareBytes, ptx::mapa_shared(ptx::smem_u32(&sh->recv_full), partner));
                else
                    site = 8;                           // reported below; the partner's wait for the share runs out too
            }
        }

        // this warp's own share of its first 64-column block leaves tensor memory while the partner's
        // share is still on its way
        uint32_t racc[2][32];
        if (ok && rows_live) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) ptx::tmem_ld_32x32(t_lane + band * chunk_cols + (colhalf * nblk * 2 + hh) * 32, racc[hh]);
        }
        if (S > 1) {
            if (ok && rows_live && !ptx::mbar_wait(&sh->recv_full, 0)) {
                ok = false;
                site = 9;
            }
            ok = __all_sync(0xffffffffu, ok);
        }

        if (ok && rows_live) {
            // ---- sum in band order, bias + activation, one rounding, store
#pragma unroll
            for (int bi = 0; bi < 2; ++bi) {
                if (bi >= nblk) break;
                const int blk = colhalf * nblk + bi;                            // 64-column block within the chunk
                if (bi > 0) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) ptx::tmem_ld_32x32(t_lane + band * chunk_cols + (blk * 2 + hh) * 32, racc[hh]);
                }
                ptx::tmem_ld_wait();
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int g = blk * 2 + hh;             // 32-column group within the chunk
                    float x[32];
                    const uint32_t (&r)[32] = racc[hh];
                    if (S > 1) {
                        float4 t[8];
#pragma unroll
                        for (int v = 0; v < 8; ++v) t[v] = recv[(g * 8 + v) * 128];
                        // band 0 holds the first half of K: its share comes first in the sum
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            const float p[4] = {t[v].x, t[v].y, t[v].z, t[v].w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float mine = __uint_as_float(r[4 * v + i]);
                                x[4 * v + i] = band == 0 ? mine + p[i] : p[i] + mine;
                            }
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(r[i]);
                    }
                    // 32 fp32 values of this thread's row -> 32 bf16 = 64 contiguous bytes of Y, stored
                    // straight from registers: nothing to stage and nothing to wait for before the CTA
                    // can leave (the block is only 128 x 128 or 128 x 256 per CTA, and staging it for a TMA
                    // store cost more time than the half-used 128-byte lines of these stores)
                    const int64_t m = row0 + lane;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const int64_t n = col0 + g * 32 + v * 8;
                        const uint4 bw = bias_w[bi][hh][v];
                        const uint32_t bwv[4] = {bw.x, bw.y, bw.z, bw.w};
                        uint32_t o[4];
#pragma unroll
                        for (int p = 0; p < 4; ++p) {
                            const float y0 = epilogue<ACT, true>(x[v * 8 + 2 * p], bf16lo_to_f32(bwv[p]));
                            const float y1 = epilogue<ACT, true>(x[v * 8 + 2 * p + 1], bf16hi_to_f32(bwv[p]));
                            o[p] = pack_bf16x2(y0, y1);
                        }
                        if (m < M && n < N) *reinterpret_cast<uint4*>(Y + m * N + n) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
        if (!ok && lane == 0 && kb1 > kb0) {
            report_timeout(status, site);
            sh->abort = 1;
        }
        if (site == 8) report_timeout(status, 8);
    } else {
        // ------------------------------------------------------------ epilogue warps, 64 rows per CTA
        // Tensor-memory lane L holds row L % 64 of this CTA; its 128 columns are columns
        // [128 (L / 64), 128 (L / 64) + 128) of the tile.  With S = 2 band b finishes tensor-memory
        // columns [64 b, 64 b + 64) of every lane and hands the other 64 to its partner (a 32 KiB
        // share); with S = 1 a CTA finishes all 128.  Of the two warps on a lane quarter each takes
        // half of those columns.
        const int ew = warp - 2, q = warp & 3, ch = ew >> 2;
        const int L = q * 32 + lane;
        const bool rows_live = (int64_t)tm * C::BM + hc * C::kRowsPerCta < M;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        const int ngroups = S == 1 ? 2 : 1;                                  // 32-column groups this warp finishes
        const int keep0 = S == 1 ? 64 * ch : 64 * band + 32 * ch;            // its first tensor-memory column
        const int64_t m = (int64_t)tm * C::BM + hc * C::kRowsPerCta + (L & 63);
        const int64_t n0 = (int64_t)tn * C::BN + (q >> 1) * 128 + keep0;     // first column of Y of this thread
        const float4* recv = reinterpret_cast<const float4*>(ring + C::kRecvOffset) + L;

        uint4 bias_w[2][4];                                 // fetched while the main loop runs
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int64_t n = n0 + g * 32 + v * 8;
                bias_w[g][v] = (bias && g < ngroups && n < N) ? *reinterpret_cast<const uint4*>(bias + n)   // N % 8 == 0
                                                              : make_uint4(0, 0, 0, 0);
            }

        bool ok = (kb1 > kb0) && !sh->abort && ptx::mbar_wait(&sh->tmem_full, 0);
        ok = __all_sync(0xffffffffu, ok);
        int site = 5;
        ptx::tcgen05_fence_after_sync();

        if (S > 1) {
            if (ok && threadIdx.x == 64) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&sh->partner_idle), partner));
            if (ok && rows_live) {
                // float4 index (column / 4) * 128 + lane: a warp writes (and later reads) 512 contiguous bytes
                float4* send = reinterpret_cast<float4*>(ring + C::kSendOffset) + L;
                uint32_t r[32];
                ptx::tmem_ld_32x32(t_lane + 64 * (band ^ 1) + 32 * ch, r);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    send[(ch * 8 + v) * 128] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                           __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                ptx::fence_proxy_async_smem();
            }
            umma2s_epi_bar_sync();
            if (threadIdx.x == 64 && ok && rows_live) {
                if (ptx::mbar_wait(&sh->partner_idle, 0))
                    bulk_copy_to_cluster(ptx::mapa_shared(ring_base + C::kRecvOffset, partner), ring + C::kSendOffset,
                                         C::kShareBytes, ptx::mapa_shared(ptx::smem_u32(&sh->recv_full), partner));
                else
                    site = 8;
            }
        }

        uint32_t racc[2][32];
        if (ok && rows_live) {
#pragma unroll
            for (int g = 0; g < 2; ++g)
                if (g < ngroups) ptx::tmem_ld_32x32(t_lane + keep0 + g * 32, racc[g]);
        }
        if (S > 1) {
            if (ok && rows_live && !ptx::mbar_wait(&sh->recv_full, 0)) {
                ok = false;
                site = 9;
            }
            ok = __all_sync(0xffffffffu, ok);
        }

        if (ok && rows_live) {
            ptx::tmem_ld_wait();
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                if (g >= ngroups) break;
                float x[32];
                const uint32_t (&r)[32] = racc[g];
                if (S > 1) {
                    float4 t[8];
#pragma unroll
                    for (int v = 0; v < 8; ++v) t[v] = recv[(ch * 8 + v) * 128];
                    // band 0 holds the first half of K: its share comes first in the sum
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const float p[4] = {t[v].x, t[v].y, t[v].z, t[v].w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float mine = __uint_as_float(r[4 * v + i]);
                            x[4 * v + i] = band == 0 ? mine + p[i] : p[i] + mine;
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(r[i]);
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int64_t n = n0 + g * 32 + v * 8;
                    const uint4 bw = bias_w[g][v];
                    const uint32_t bwv[4] = {bw.x, bw.y, bw.z, bw.w};
                    uint32_t o[4];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        const float y0 = epilogue<ACT, true>(x[v * 8 + 2 * p], bf16lo_to_f32(bwv[p]));
                        const float y1 = epilogue<ACT, true>(x[v * 8 + 2 * p + 1], bf16hi_to_f32(bwv[p]));
                        o[p] = pack_bf16x2(y0, y1);
                    }
                    if (m < M && n < N) *reinterpret_cast<uint4*>(Y + m * N + n) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
        if (!ok && lane == 0 && kb1 > kb0) {
            report_timeout(status, site);
            sh->abort = 1;
        }
        if (site == 8) report_timeout(status, 8);
    }

    __syncwarp();                   // the role branches diverge inside warps 0 and 1
    ptx::tcgen05_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();            // no MMA, copy, remote arrive or remote read of the cluster is outstanding past this point
    if (warp == 1) {
        __syncwarp();
        ptx::tcgen05_fence_after_sync();
        ptx::tmem_dealloc_2cta(tmem_base, C::kTmemCols);
    }
}

}  // namespace optiml
