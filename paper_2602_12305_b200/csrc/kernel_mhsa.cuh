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
//   warp 1      one lane issues every MMA: S_t,j = Q_t K_j^T and O_t += P_t,j V_j for t = 0, 1
//   warps 2-5   softmax + output for query tile 0 (one thread per query row = one TMEM lane)
//   warps 6-9   the same for query tile 1
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
    static constexpr int kSlots = DK == 64 ? 6 : 3;      // ring slots, each one K or V block
    static constexpr int kThreads = 320;
    static constexpr int kTmemCols = 512;                // S0, S1: 2 x 128; O0, O1: 2 x DK
    static constexpr int kColS = 0, kColO = 256;
    static constexpr int kSmemBytes = 256 + 1024 + kQTiles * kTileBytes + kQTiles * kPBytes + kSlots * kTileBytes;
    static constexpr float kRescaleThreshold = 8.0f;     // log2 units
};

struct MhsaShared {
    uint64_t full[6], empty[6];       // ring slots
    uint64_t q_full;
    uint64_t s_full[2], p_full[2], o_final[2];
    uint64_t drain;
    uint32_t tmem_base;
    volatile int abort;
};
static_assert(sizeof(MhsaShared) <= 256, "barrier block");

// Wait sites reported on a time-out: 1 producer/free slot, 2 MMA/Q, 3 MMA/K block, 4 MMA/V block,
// 5 MMA/probabilities, 6 softmax/scores, 7 softmax/final accumulator.
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
    uint8_t* q_smem = data;                                        // [2][kTileBytes]
    uint8_t* p_smem = q_smem + C::kQTiles * C::kTileBytes;         // [2][kPBytes]
    uint8_t* ring = p_smem + C::kQTiles * C::kPBytes;              // [kSlots][kTileBytes]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head = blockIdx.y;
    const int q0 = blockIdx.x * (C::kQTiles * C::BQ);
    const int nblk = (N + C::BKV - 1) / C::BKV;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kSlots; ++s) {
            ptx::mbar_init(&sh->full[s], 1);
            ptx::mbar_init(&sh->empty[s], 1);
        }
        ptx::mbar_init(&sh->q_full, 1);
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(&sh->s_full[t], 1);
            ptx::mbar_init(&sh->p_full[t], C::BQ);
            ptx::mbar_init(&sh->o_final[t], 1);
        }
        ptx::mbar_init(&sh->drain, 1);
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

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::mbar_arrive_expect_tx(&sh->q_full, C::kQTiles * C::kTileBytes);
            for (int t = 0; t < C::kQTiles; ++t)
                for (int c = 0; c < C::kChunks; ++c)
                    ptx::tma_load_2d(q_smem + t * C::kTileBytes + c * C::kChunkBytes, &map_q, &sh->q_full,
                                     head * DK + c * 64, q0 + t * C::BQ);
            uint32_t it = 0;
            bool ok = true;
            for (int j = 0; ok && j < nblk; ++j) {
                for (int kv = 0; kv < 2; ++kv, ++it) {
                    const int s = it % C::kSlots;
                    const uint32_t ph = (it / C::kSlots) & 1;
                    if (sh->abort || !ptx::mbar_wait(&sh->empty[s], ph ^ 1)) { ok = false; break; }
                    ptx::mbar_arrive_expect_tx(&sh->full[s], C::kTileBytes);
                    for (int c = 0; c < C::kChunks; ++c)
                        ptx::tma_load_2d(ring + s * C::kTileBytes + c * C::kChunkBytes, kv ? &map_v : &map_k,
                                         &sh->full[s], head * DK + c * 64, j * C::BKV);
                }
            }
            if (!ok) {
                report_timeout(status, 1);
                sh->abort = 1;
                // copies already issued must land before the CTA may exit
                ptx::mbar_wait(&sh->q_full, 0);
                const uint32_t n_back = it < (uint32_t)C::kSlots ? it : (uint32_t)C::kSlots;
                for (uint32_t b = 1; b <= n_back; ++b) {
                    const uint32_t i = it - b;
                    ptx::mbar_wait(&sh->full[i % C::kSlots], (i / C::kSlots) & 1);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = ptx::umma_idesc_bf16(C::BQ, C::BKV, false, false);   // Q, K: both K-major
            constexpr uint32_t idesc_o = ptx::umma_idesc_bf16(C::BQ, DK, false, true);        // P K-major, V MN-major
            bool ok = true;
            int site = 0;
            auto slot_addr = [&](uint32_t i) { return data_base + (uint32_t)(C::kQTiles * (C::kTileBytes + C::kPBytes)) +
                                                      (i % C::kSlots) * C::kTileBytes; };
            auto wait_slot = [&](uint32_t i) { return ptx::mbar_wait(&sh->full[i % C::kSlots], (i / C::kSlots) & 1); };
            // S_t = Q_t K_j^T, contraction over d_k in steps of 16 (32 bytes inside a 128-byte row)
            auto issue_s = [&](int t, uint32_t k_slot) {
                const uint32_t q_addr = data_base + t * C::kTileBytes;
                const uint32_t k_addr = slot_addr(k_slot);
#pragma unroll
                for (int ks = 0; ks < DK / 16; ++ks) {
                    const uint32_t off = (ks >> 2) * C::kChunkBytes + (ks & 3) * 32;
                    ptx::umma_bf16(tmem_base + C::kColS + t * C::BKV, ptx::umma_smem_desc(q_addr + off, 16, 1024),
                                   ptx::umma_smem_desc(k_addr + off, 16, 1024), idesc_s, ks != 0);
                }
                ptx::umma_commit(&sh->s_full[t]);
            };
            // O_t (+)= P_t V_j, contraction over the 128 keys in steps of 16 (16 rows of V)
            auto issue_pv = [&](int t, uint32_t v_slot, bool accumulate) {
                const uint32_t p_addr = data_base + C::kQTiles * C::kTileBytes + t * C::kPBytes;
                const uint32_t v_addr = slot_addr(v_slot);
#pragma unroll
                for (int ks = 0; ks < C::BKV / 16; ++ks) {
                    const uint32_t p_off = (ks >> 2) * C::kChunkBytes + (ks & 3) * 32;
                    ptx::umma_bf16(tmem_base + C::kColO + t * DK, ptx::umma_smem_desc(p_addr + p_off, 16, 1024),
                                   ptx::umma_smem_desc(v_addr + ks * 2048, C::kChunkBytes, 1024), idesc_o,
                                   accumulate || ks != 0);
                }
            };
            if (sh->abort || (site = 2, !ptx::mbar_wait(&sh->q_full, 0)) || (site = 3, !wait_slot(0))) ok = false;
            if (ok) {
                ptx::tcgen05_fence_after_sync();
                issue_s(0, 0);
                issue_s(1, 0);
                ptx::umma_commit(&sh->empty[0]);
            }
            for (int j = 0; ok && j < nblk; ++j) {
                const uint32_t v_it = 2 * j + 1, k_next = 2 * j + 2;
                for (int t = 0; t < 2; ++t) {
                    if (sh->abort || (site = 5, !ptx::mbar_wait(&sh->p_full[t], j & 1))) { ok = false; break; }
                    if (t == 0 && (site = 4, !wait_slot(v_it))) { ok = false; break; }
                    ptx::tcgen05_fence_after_sync();
                    issue_pv(t, v_it, j != 0);
                    if (t == 1) ptx::umma_commit(&sh->empty[v_it % C::kSlots]);
                    if (j + 1 < nblk) {
                        if (t == 0 && (site = 3, !wait_slot(k_next))) { ok = false; break; }
                        ptx::tcgen05_fence_after_sync();
                        issue_s(t, k_next);
                        if (t == 1) ptx::umma_commit(&sh->empty[k_next % C::kSlots]);
                    } else {
                        ptx::umma_commit(&sh->o_final[t]);
                    }
                }
            }
            if (!ok) {
                report_timeout(status, site);
                sh->abort = 1;
            }
            // nothing may be in flight on the tensor pipe when tensor memory is freed
            ptx::umma_commit(&sh->drain);
            ptx::mbar_wait(&sh->drain, 0);
        }
    } else {
        // ------------------------------------------------------------ softmax + output, one thread per query row
        const int t = (warp - 2) >> 2;                   // query tile of this warp group
        const int quarter = warp & 3;                    // TMEM lane quarter this warp may touch
        const int r = quarter * 32 + lane;               // row within the tile
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t s_addr = lane_base + C::kColS + t * C::BKV;
        const uint32_t o_addr = lane_base + C::kColO + t * DK;
        uint8_t* p_row = p_smem + t * C::kPBytes + r * 128;
        float m_used = 0.0f, l = 0.0f;
        bool ok = true;
        for (int j = 0; j < nblk; ++j) {
            bool got = !sh->abort && ptx::mbar_wait(&sh->s_full[t], j & 1);
            got = __all_sync(0xffffffffu, got);
            if (!got) { ok = false; break; }
            ptx::tcgen05_fence_after_sync();
            const int nvalid = min(C::BKV, N - j * C::BKV);
            // pass 1: row maximum of the valid scores
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(s_addr + c * 32, v);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c * 32 + i < nvalid) mx = fmaxf(mx, __uint_as_float(v[i]));
            }
            mx *= scale_log2;
            bool raise = false;
            if (j == 0) {
                m_used = mx;
            } else if (mx > m_used + C::kRescaleThreshold) {
                raise = true;
            }
            if (__any_sync(0xffffffffu, raise)) {
                // every earlier P V of this tile has finished (the MMA that produced these scores
                // was issued after it), so the accumulator can be rescaled in place
                const float alpha = raise ? ptx::ex2_approx(m_used - mx) : 1.0f;
                if (raise) {
                    l *= alpha;
                    m_used = mx;
                }
#pragma unroll 1
                for (int c = 0; c < DK / 32; ++c) {
                    uint32_t v[32];
                    ptx::tmem_ld_32x32(o_addr + c * 32, v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                    ptx::tmem_st_32x32(o_addr + c * 32, v);
                }
                ptx::tmem_st_wait();
            }
            // pass 2: probabilities relative to m_used, bf16, into the swizzled K-major P tile
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(s_addr + c * 32, v);
                ptx::tmem_ld_wait();
                uint8_t* atom_row = p_row + (c >> 1) * C::kChunkBytes;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    uint32_t o[4];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        const int i0 = g * 8 + 2 * p;
                        float e0 = ptx::ex2_approx(fmaf(__uint_as_float(v[i0]), scale_log2, -m_used));
                        float e1 = ptx::ex2_approx(fmaf(__uint_as_float(v[i0 + 1]), scale_log2, -m_used));
                        if (c * 32 + i0 >= nvalid) e0 = 0.0f;
                        if (c * 32 + i0 + 1 >= nvalid) e1 = 0.0f;
                        l += e0 + e1;
                        o[p] = pack_bf16x2(e0, e1);
                    }
                    const int chunk16 = (c & 1) * 4 + g;
                    *reinterpret_cast<uint4*>(atom_row + ((chunk16 ^ (lane & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            ptx::fence_proxy_async_smem();
            ptx::tcgen05_fence_before_sync();
            ptx::mbar_arrive(&sh->p_full[t]);
        }
        if (ok) {
            bool got = !sh->abort && ptx::mbar_wait(&sh->o_final[t], 0);
            got = __all_sync(0xffffffffu, got);
            if (!got) {
                ok = false;
                if (lane == 0) report_timeout(status, 7);
            }
        } else if (lane == 0) {
            report_timeout(status, 6);
        }
        if (!ok) sh->abort = 1;
        ptx::griddep_launch_dependents();
        if (ok) {
            ptx::tcgen05_fence_after_sync();
            const float inv = 1.0f / l;
            const int row = q0 + t * C::BQ + r;
            __nv_bfloat16* y_row = Y + (size_t)row * d_model + head * DK;
#pragma unroll 1
            for (int c = 0; c < DK / 32; ++c) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(o_addr + c * 32, v);
                ptx::tmem_ld_wait();
                if (row < N) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint32_t o[4];
#pragma unroll
                        for (int p = 0; p < 4; ++p)
                            o[p] = pack_bf16x2(__uint_as_float(v[g * 8 + 2 * p]) * inv, __uint_as_float(v[g * 8 + 2 * p + 1]) * inv);
                        *reinterpret_cast<uint4*>(y_row + c * 32 + g * 8) = make_uint4(o[0], o[1], o[2], o[3]);
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
