// C ABI of the library (include/optiml.h): handle, argument checks, the shape-based
// dispatcher and the kernel launches.  Host code only touches scalars and pointers;
// every arithmetic step of Y = act(A.B + bias) runs in the kernels included below.
#include "../../include/optiml.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <utility>

#include "common.cuh"
#include "kernel_f32.cuh"
#include "kernel_gemv.cuh"
#include "kernel_generic.cuh"
#include "kernel_mhsa.cuh"
#include "kernel_mhsa2.cuh"
#include "kernel_reduce.cuh"
#include "kernel_repack.cuh"
#include "kernel_selftest.cuh"
#include "kernel_skinny.cuh"
#include "kernel_umma.cuh"
#include "kernel_umma2.cuh"
#include "kernel_umma2s.cuh"

using namespace optiml;

namespace {

constexpr int kVersion = 10000 * 0 + 100 * 1 + 0;
constexpr size_t kPartialBytes = (size_t)32 << 20;   // split-K / stream-K partial sums
constexpr int kNumCounters = 1 << 16;                 // one arrival counter per column block / tile
constexpr int kMapCache = 32;
// Defaults of the tuning options (optiml_option_t order), chosen from sweeps on B200.
constexpr int64_t kOptionDefaults[OPTIML_OPT_COUNT] = {
    // 1 x 8192 x 8192 bf16: 22.8 us without prefetch, 21.7-21.9 us with 48-96 rows, 23.9 us with 192
    /* GEMV_PREFETCH_ROWS    */ 96,
    // 16 x 14336 x 4096 (two MMA lanes): 128-row stages 22.0-22.4 us, 192-row stages 20.9 us;
    // four stages prefetched before the wait and the late trigger: 19.9 us
    /* SKINNY_STAGE_ROWS     */ 192,
    /* SKINNY_RING_STAGES    */ 0,
    /* SKINNY_PREFETCH_EARLY */ 4,
    /* SKINNY_LATE_TRIGGER   */ 1,
    /* PAIR_SPLIT_MAX        */ 8,
    /* PAIR_HALF_HEIGHT      */ 1,
    /* PAIR_TILE_WIDTH       */ 0,
};

// Streaming rates the skinny kernel's schedule is costed with (see launch_skinny_cfg).
constexpr double kSkinnyCtaGBs = 110.0, kSkinnyAllGBs = 7000.0;

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapEntry {
    const void* ptr = nullptr;
    uint64_t rows = 0, cols = 0;
    uint32_t box_rows = 0, box_cols = 0;
    CUtensorMap map;
    bool valid = false;
};

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    bool ok = false;            // `dev` is the current device while the guard lives
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        if (prev == dev) {
            ok = true;
            return;
        }
        ok = switched = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

// Every device allocation of the library goes through here, so that a test can make the
// n-th one fail (optiml_set_alloc_hook) without exhausting a GPU's memory.
optiml_alloc_hook_t g_alloc_hook = nullptr;
void* g_alloc_hook_user = nullptr;

template <typename T>
bool dev_alloc(T** p, size_t bytes) {
    *p = nullptr;
    if (g_alloc_hook && g_alloc_hook(bytes, g_alloc_hook_user) != 0) return false;
    if (cudaMalloc(reinterpret_cast<void**>(p), bytes) != cudaSuccess) {
        cudaGetLastError();
        *p = nullptr;
        return false;
    }
    return true;
}

}  // namespace

struct optiml_handle_s {
    int device = 0;
    int num_sms = 0;
    float* partials = nullptr;
    unsigned int* counters = nullptr;
    int* status = nullptr;
    int forced = OPTIML_VARIANT_AUTO;
    int64_t launches = 0;
    bool log = false;
    encode_tiled_fn encode = nullptr;
    MapEntry maps[kMapCache];
    int next_map = 0;
    void* stage[4] = {nullptr, nullptr, nullptr, nullptr};     // host entry point: A, B, bias, Y on the device
    size_t stage_bytes[4] = {0, 0, 0, 0};
    void* pad[4] = {nullptr, nullptr, nullptr, nullptr};       // re-pitched copies of A, B, bias, Y (unaligned bf16 shapes)
    size_t pad_bytes[4] = {0, 0, 0, 0};
    int64_t options[OPTIML_OPT_COUNT];
    int stream_clusters[3] = {0, 0, 0};   // clusters of 2, 4 and 8 CTAs of the streaming pair kernel the device can hold at once
};

namespace {

// ---------------------------------------------------------------- tensor maps

// Row-major bf16 matrix [rows][cols] -> 2-D tiled map with a {box_cols, box_rows} box and
// 128-byte swizzle (box_cols * 2 bytes == 128).  Cached by (pointer, shape, box).  The map is
// COPIED into `out`, which the caller owns: a launch looks up two or three maps, and a miss on
// a later lookup may recycle the very slot an earlier lookup of the same launch has hit.
bool get_map(optiml_handle_t h, CUtensorMap* out, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows,
             uint32_t box_cols) {
    for (int i = 0; i < kMapCache; ++i) {
        const MapEntry& e = h->maps[i];
        if (e.valid && e.ptr == ptr && e.rows == rows && e.cols == cols && e.box_rows == box_rows &&
            e.box_cols == box_cols) {
            *out = e.map;
            return true;
        }
    }
    MapEntry& e = h->maps[h->next_map];
    h->next_map = (h->next_map + 1) % kMapCache;
    e.valid = false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = h->encode(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    e.ptr = ptr;
    e.rows = rows;
    e.cols = cols;
    e.box_rows = box_rows;
    e.box_cols = box_cols;
    e.valid = true;
    *out = e.map;
    return true;
}

// ---------------------------------------------------------------- dispatcher

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

bool variant_supports(optiml_handle_t h, int v, int64_t M, int64_t N, int64_t K, int dtype, bool al16) {
    switch (v) {
    case OPTIML_VARIANT_GENERIC:
        return true;
    case OPTIML_VARIANT_F32_TILED:
        return dtype == OPTIML_F32 && N % 4 == 0 && K % 4 == 0 && al16;
    case OPTIML_VARIANT_GEMV_SPLITK:
        return M <= 4 && N % (dtype == OPTIML_F32 ? 4 : 8) == 0 && al16 &&
               ceil_div64(N, dtype == OPTIML_F32 ? GemvVec<float>::kCols : kGemvCols) <= kNumCounters;
    case OPTIML_VARIANT_SKINNY_UMMA:
        return dtype == OPTIML_BF16 && M <= 128 && N % 8 == 0 && K % 8 == 0 && al16 &&
               ceil_div64(N, 128) <= kNumCounters;
    case OPTIML_VARIANT_UMMA:
    case OPTIML_VARIANT_UMMA_2CTA:
        return dtype == OPTIML_BF16 && N % 8 == 0 && K % 8 == 0 && al16 &&
               ceil_div64(M, UmmaCfg::BM) * ceil_div64(N, UmmaCfg::BN) < (int64_t)1 << 31;
    case OPTIML_VARIANT_UMMA_2CTA_STREAM:
        // one cluster per 256 x 256 tile, all of them resident at once
        return dtype == OPTIML_BF16 && N % 8 == 0 && K % 8 == 0 && al16 &&
               ceil_div64(M, Umma2sCfg::BM) * ceil_div64(N, Umma2sCfg::BN) <= h->stream_clusters[0];
    default:
        return false;
    }
}

// K slices (CTA pairs per tile) of the streaming pair kernel: as many as the device can hold
// clusters for, with at least four K blocks per slice; a CTA must keep a multiple of 32
// accumulator columns (its two epilogue warps per lane quarter work in pieces of 16).
int stream_split(optiml_handle_t h, int64_t tiles, int64_t num_kb, int tmem_cols) {
    int split = 1;
    for (int i = 1; (1 << i) <= Umma2sCfg::kMaxSplit; ++i) {
        const int s = 1 << i;
        if (tiles <= h->stream_clusters[i] && num_kb >= 4 * s && (tmem_cols / s) % 32 == 0) split = s;
    }
    const int64_t cap = h->options[OPTIML_OPT_PAIR_SPLIT_MAX];
    while (split > 1 && split > cap) split >>= 1;
    return split;
}

// Tile width of the streaming pair kernel.  What decides its time is how many bytes each SM has
// to pull (its port takes about 90 GB/s) against the stream over B from HBM; 128-column tiles
// double the number of CTAs where 256-column tiles are too few for the clusters the device
// holds (N = 4096: 16 tiles, two pairs each = 64 CTAs; 32 narrow tiles = 128 CTAs) at the price
// of reading A once more per column of tiles.
int stream_tile_width(optiml_handle_t h, int64_t M, int64_t N, int64_t K, bool half_height) {
    const int64_t cap = h->options[OPTIML_OPT_PAIR_TILE_WIDTH];
    if (cap == 128 || cap == 256) return (int)cap;
    const int bm = half_height ? 128 : 256, rows = bm / 2;
    const int64_t tiles_m = ceil_div64(M, bm), num_kb = ceil_div64(K, 64);
    double best = 0.0;
    int width = 256;
    for (int bn = 256; bn >= 128; bn -= 128) {
        const int64_t tiles = tiles_m * ceil_div64(N, bn);
        if (tiles > h->stream_clusters[0]) continue;
        const int s = stream_split(h, tiles, num_kb, half_height ? bn / 2 : bn);
        const double per_cta = (double)(rows + bn / 2) * 128.0 * (double)ceil_div64(num_kb, s);       // bytes through one SM's port
        const double all = 2.0 * ((double)K * N + (double)M * K);
        const double us = std::max(per_cta / 90e3, all / 6.3e6) + 5.0 + 1.0 * (s - 1);
        if (best == 0.0 || us < best * 0.97) {       // the narrow form has to win by a margin
            best = us;
            width = bn;
        }
    }
    return width;
}

// Whether the skinny kernel's schedule for this shape finishes every column tile in one CTA
// (a single band: no partial tiles, no second pass).
template <int MP, int SUB>
bool skinny_single_band_cfg(optiml_handle_t h, int64_t N, int64_t K) {
    using C = SkinnyCfg<MP, SUB>;
    const int64_t max_slots = kPartialBytes / (C::kSlotFloats * sizeof(float));
    const double unit_us = (double)(C::kBBytes + C::kABytes) / (kSkinnyCtaGBs * 1e3);
    return make_skinny_plan(ceil_div64(N, C::BN), ceil_div64(K, C::BK), h->num_sms, max_slots, unit_us,
                            kSkinnyAllGBs / kSkinnyCtaGBs).nbands == 1;
}
bool skinny_single_band(optiml_handle_t h, int64_t M, int64_t N, int64_t K) {
    return M <= 64 ? skinny_single_band_cfg<64, 2>(h, N, K) : skinny_single_band_cfg<128, 2>(h, N, K);
}

// Shape-based choice.  fp32 goes to the FMA tiles.  bf16: M = 1 is a pure stream over B
// (CUDA-core split-K; measured 5.5 TB/s against 4.9 TB/s for the tensor-core stream; at
// M = 4 the FMA pipes already fall behind: 81 us against 28 us on 4 x 8192 x 8192),
// M <= 64 is still bandwidth-bound but needs tensor-core MACs
// (stream-K tcgen05 with N as the MMA M dimension), larger M is compute-bound.
int choose_variant(optiml_handle_t h, int64_t M, int64_t N, int64_t K, int dtype, bool al16) {
    if (h->forced != OPTIML_VARIANT_AUTO) return h->forced;
    if (dtype == OPTIML_F32) {
        // fp32 has no tensor-core path: up to 4 rows stream over B (measured 1 x 8192 x 8192: 163 us
        // on the tiles, a fifth of that on the streaming kernel), everything else goes to the FMA tiles
        if (M <= 4 && variant_supports(h, OPTIML_VARIANT_GEMV_SPLITK, M, N, K, dtype, al16)) return OPTIML_VARIANT_GEMV_SPLITK;
        return variant_supports(h, OPTIML_VARIANT_F32_TILED, M, N, K, dtype, al16) ? OPTIML_VARIANT_F32_TILED
                                                                                 : OPTIML_VARIANT_GENERIC;
    }
    if (M == 1 && variant_supports(h, OPTIML_VARIANT_GEMV_SPLITK, M, N, K, dtype, al16)) return OPTIML_VARIANT_GEMV_SPLITK;
    const bool skinny_ok = variant_supports(h, OPTIML_VARIANT_SKINNY_UMMA, M, N, K, dtype, al16);
    const bool stream_ok = variant_supports(h, OPTIML_VARIANT_UMMA_2CTA_STREAM, M, N, K, dtype, al16);
    // up to 32 rows the stream-K kernel spreads any shape over all SMs (4096 x 14336 with 16 column tiles of 256:
    // 32 rows 25.5 us against 33.1 us for the cluster kernel, which has 64 CTAs there; 8192 x 8192: 25.8 against 25.0 us)
    if (M <= 32 && skinny_ok) return OPTIML_VARIANT_SKINNY_UMMA;
    if (M <= 128 && skinny_ok) {
        // Between 33 and 128 rows the streaming kernel with N as the MMA M dimension wins up to 64 rows where
        // every column tile is finished by one CTA (measured 64 x 14336 x 4096: 21.4 us against 23.0 us for
        // the cluster kernel with 64 rows per CTA), and loses above (128 rows: 25.3 against 23.4 us) and
        // wherever its tiles are cut along K (48 x 8192 x 8192: 28.8 against 25.2 us; 64 rows: 31.2 against
        // 25.5 us; 128 rows: 41.5 against 25.5 us; 48 x 2048 x 8192: 38.3 against 20.8 us).
        if (!stream_ok || (M <= 64 && skinny_single_band(h, M, N, K))) return OPTIML_VARIANT_SKINNY_UMMA;
        return OPTIML_VARIANT_UMMA_2CTA_STREAM;
    }
    // fewer tiles than CTA pairs: the problem is a stream over B; one cluster per tile, K cut across its pairs
    if (stream_ok) return OPTIML_VARIANT_UMMA_2CTA_STREAM;
    // above 64 rows a CTA pair shares one 256 x 256 tile (a third less operand traffic per flop); measured
    // at least as fast as the single-CTA kernel from M = 96 up, which stays as a forced variant
    if (variant_supports(h, OPTIML_VARIANT_UMMA_2CTA, M, N, K, dtype, al16)) return OPTIML_VARIANT_UMMA_2CTA;
    if (variant_supports(h, OPTIML_VARIANT_UMMA, M, N, K, dtype, al16)) return OPTIML_VARIANT_UMMA;
    return OPTIML_VARIANT_GENERIC;
}

// ---------------------------------------------------------------- launches

// Launch as a programmatic dependent of the previous kernel in the stream: this kernel's
// CTAs may be scheduled, and run their set-up, while that kernel drains; the kernels call
// griddepcontrol.wait before they touch global memory, so stream order is preserved.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename T>
optiml_status_t launch_generic(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M,
                               int N, int K, int act, cudaStream_t st) {
    const int64_t tiles = ceil_div64(M, kGenBM) * ceil_div64(N, kGenBN);
    if (tiles >= (int64_t)1 << 31) return OPTIML_ERR_UNSUPPORTED;
    gemm_generic_kernel<T><<<(unsigned)tiles, kGenThreads, 0, st>>>((const T*)A, (const T*)B, (const T*)bias, (T*)Y, M,
                                                                     N, K, act);
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

template <int BM, int BN, int TM, int TN, int KS>
optiml_status_t launch_f32_cfg(optiml_handle_t h, const float* A, const float* B, const float* bias, float* Y, int M,
                               int N, int K, int act, cudaStream_t st) {
    using C = F32Cfg<BM, BN, TM, TN, KS>;
    const int64_t tiles = ceil_div64(M, BM) * ceil_div64(N, BN);
    if (tiles >= (int64_t)1 << 31) return OPTIML_ERR_UNSUPPORTED;
    const size_t smem = C::kSmemFloats * sizeof(float);
    switch (act) {
    case OPTIML_ACT_RELU:
        launch_pdl(gemm_f32_tiled_kernel<BM, BN, TM, TN, KS, kActRelu>, dim3((unsigned)tiles), dim3(C::kThreads), smem, st, A, B, bias, Y, M, N, K);
        break;
    case OPTIML_ACT_GELU_TANH:
        launch_pdl(gemm_f32_tiled_kernel<BM, BN, TM, TN, KS, kActGeluTanh>, dim3((unsigned)tiles), dim3(C::kThreads), smem, st, A, B, bias, Y, M, N, K);
        break;
    case OPTIML_ACT_SIGMOID:
        launch_pdl(gemm_f32_tiled_kernel<BM, BN, TM, TN, KS, kActSigmoid>, dim3((unsigned)tiles), dim3(C::kThreads), smem, st, A, B, bias, Y, M, N, K);
        break;
    default:
        launch_pdl(gemm_f32_tiled_kernel<BM, BN, TM, TN, KS, kActNone>, dim3((unsigned)tiles), dim3(C::kThreads), smem, st, A, B, bias, Y, M, N, K);
        break;
    }
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

// Largest tile that still gives every SM a CTA; small problems take 32x32 tiles with the
// K loop split four ways inside the CTA.
optiml_status_t launch_f32(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M, int N,
                           int K, int act, cudaStream_t st) {
    const float *a = (const float*)A, *b = (const float*)B, *bi = (const float*)bias;
    float* y = (float*)Y;
    if (ceil_div64(M, 128) * ceil_div64(N, 128) >= h->num_sms)
        return launch_f32_cfg<128, 128, 8, 8, 1>(h, a, b, bi, y, M, N, K, act, st);
    if (ceil_div64(M, 64) * ceil_div64(N, 64) >= h->num_sms)
        return launch_f32_cfg<64, 64, 4, 4, 1>(h, a, b, bi, y, M, N, K, act, st);
    // (8 or 16 slices of K per CTA instead of 4 were measured too: 5.6 and 6.2 us against 5.4 us on 256^3)
    return launch_f32_cfg<32, 32, 4, 4, 4>(h, a, b, bi, y, M, N, K, act, st);
}

template <int MR>
void launch_gemv_mr(const void* A, const void* B, const void* bias, void* Y, int M, int N, int K, int act, dim3 grid,
                    float* partials, unsigned int* counters, int prefetch_rows, cudaStream_t st) {
    launch_pdl(gemv_splitk_kernel<__nv_bfloat16, MR>, grid, dim3(kGemvThreads), 0, st, (const __nv_bfloat16*)A,
               (const __nv_bfloat16*)B, (const __nv_bfloat16*)bias, (__nv_bfloat16*)Y, M, N, K, act, partials, counters,
               prefetch_rows);
}

template <int MR>
void launch_gemv_f32_mr(const void* A, const void* B, const void* bias, void* Y, int M, int N, int K, int act, dim3 grid,
                        float* partials, unsigned int* counters, int prefetch_rows, cudaStream_t st) {
    launch_pdl(gemv_splitk_kernel<float, MR>, grid, dim3(kGemvThreads), 0, st, (const float*)A, (const float*)B,
               (const float*)bias, (float*)Y, M, N, K, act, partials, counters, prefetch_rows);
}

optiml_status_t launch_gemv(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M, int N,
                            int K, int dtype, int act, cudaStream_t st) {
    const int MR = M == 1 ? 1 : (M == 2 ? 2 : 4);
    const int cols = dtype == OPTIML_F32 ? GemvVec<float>::kCols : GemvVec<__nv_bfloat16>::kCols;
    const int64_t col_blocks = ceil_div64(N, cols);
    // K slices: fill every SM with its resident CTAs in one wave, keep at least 64 rows per slice,
    // stay inside the scratch and the 65535 limit of gridDim.y.
    int64_t S = (gemv_ctas_per_sm(MR) * (int64_t)h->num_sms) / col_blocks;
    if (S > K / 64) S = K / 64;
    const int64_t per_slice = (int64_t)MR * cols * sizeof(float);
    if (S * col_blocks * per_slice > (int64_t)kPartialBytes) S = kPartialBytes / (col_blocks * per_slice);
    if (S > 65535) S = 65535;
    if (S < 1) S = 1;
    dim3 grid((unsigned)col_blocks, (unsigned)S);
    const int pf = (int)h->options[OPTIML_OPT_GEMV_PREFETCH_ROWS];
    if (dtype == OPTIML_F32) {
        if (MR == 1) launch_gemv_f32_mr<1>(A, B, bias, Y, M, N, K, act, grid, h->partials, h->counters, pf, st);
        else if (MR == 2) launch_gemv_f32_mr<2>(A, B, bias, Y, M, N, K, act, grid, h->partials, h->counters, pf, st);
        else launch_gemv_f32_mr<4>(A, B, bias, Y, M, N, K, act, grid, h->partials, h->counters, pf, st);
    } else {
        if (MR == 1) launch_gemv_mr<1>(A, B, bias, Y, M, N, K, act, grid, h->partials, h->counters, pf, st);
        else if (MR == 2) launch_gemv_mr<2>(A, B, bias, Y, M, N, K, act, grid, h->partials, h->counters, pf, st);
        else launch_gemv_mr<4>(A, B, bias, Y, M, N, K, act, grid, h->partials, h->counters, pf, st);
    }
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

template <int MP, int SUB>
optiml_status_t launch_skinny_cfg(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M,
                                  int N, int K, int act, cudaStream_t st) {
    using C = SkinnyCfg<MP, SUB>;
    CUtensorMap ma, mb;
    if (!get_map(h, &ma, A, (uint64_t)M, (uint64_t)K, MP, 64) || !get_map(h, &mb, B, (uint64_t)K, (uint64_t)N, 64, 64))
        return OPTIML_ERR_CUDA;
    const int64_t max_slots = kPartialBytes / (C::kSlotFloats * sizeof(float));
    // one unit = one K block of one column tile; with two MMA lanes a CTA streams it at about 110 GB/s,
    // all CTAs together at about 7 TB/s (measured: 16 x 14336 x 16384 as 112 whole tiles 67 us = 7.0 TB/s,
    // as two balanced bands on 148 CTAs 76 us; 8 x 28672 x 4096 as one band on 148 CTAs 37.6 us, as two
    // bands 46.7 us; 16 x 8192 x 8192 as three bands 22.9 us, as 64 whole tiles 26.3 us)
    const double unit_us = (double)(C::kBBytes + C::kABytes) / (kSkinnyCtaGBs * 1e3);
    const SkinnyPlan plan = make_skinny_plan(ceil_div64(N, C::BN), ceil_div64(K, C::BK), h->num_sms, max_slots, unit_us,
                                             kSkinnyAllGBs / kSkinnyCtaGBs);
    if (h->log) fprintf(stderr, "[optiml] skinny plan: G=%d S=%d k_split=%d G1=%d k_mid=%d G2=%d bands=%d\n", plan.G, plan.S, plan.k_split, plan.G1, plan.k_mid, plan.G2, plan.nbands);
    SkinnyTune tune;
    const int64_t want = h->options[OPTIML_OPT_SKINNY_RING_STAGES];
    // default depth: all that fit, except three 192-row stages at M <= 16 (measured on 16 x 14336 x 4096
    // with two MMA lanes: 2 / 3 / 4 stages 21.6 / 19.9 / 20.2 us)
    const int dflt = (MP == 16 && SUB == 3 && C::kStages > 3) ? 3 : C::kStages;
    tune.stages = want < 2 ? dflt : (want > C::kStages ? C::kStages : (int)want);
    tune.prefetch_early = (int)h->options[OPTIML_OPT_SKINNY_PREFETCH_EARLY];
    tune.late_trigger = h->options[OPTIML_OPT_SKINNY_LATE_TRIGGER] != 0;
    launch_pdl(gemm_skinny_umma_kernel<MP, SUB>, dim3(plan.G), dim3(C::kThreads), C::smem_bytes(tune.stages), st, ma,
               mb, (const __nv_bfloat16*)bias, (__nv_bfloat16*)Y, M, N, K, act, plan, tune, h->partials, h->counters,
               h->status);
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

// Rows of K per pipeline stage: 128 or 192 (option SKINNY_STAGE_ROWS; 192 only up to 32 rows of A).
template <int MP>
optiml_status_t launch_skinny_mp(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M,
                                 int N, int K, int act, cudaStream_t st) {
    if constexpr (MP <= 32) {
        if (h->options[OPTIML_OPT_SKINNY_STAGE_ROWS] == 192)
            return launch_skinny_cfg<MP, 3>(h, A, B, bias, Y, M, N, K, act, st);
    }
    return launch_skinny_cfg<MP, 2>(h, A, B, bias, Y, M, N, K, act, st);
}

optiml_status_t launch_skinny(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M, int N,
                              int K, int act, cudaStream_t st) {
    if (M <= 16) return launch_skinny_mp<16>(h, A, B, bias, Y, M, N, K, act, st);
    if (M <= 32) return launch_skinny_mp<32>(h, A, B, bias, Y, M, N, K, act, st);
    if (M <= 64) return launch_skinny_mp<64>(h, A, B, bias, Y, M, N, K, act, st);
    return launch_skinny_mp<128>(h, A, B, bias, Y, M, N, K, act, st);
}

optiml_status_t launch_umma(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M, int N,
                            int K, int act, cudaStream_t st) {
    using C = UmmaCfg;
    CUtensorMap ma, mb, my;
    if (!get_map(h, &ma, A, (uint64_t)M, (uint64_t)K, C::BM, 64) || !get_map(h, &mb, B, (uint64_t)K, (uint64_t)N, 64, 64) ||
        !get_map(h, &my, Y, (uint64_t)M, (uint64_t)N, 32, 64))
        return OPTIML_ERR_CUDA;
    const UmmaPlan plan = make_umma_plan(M, N, K, h->num_sms);
    if ((size_t)plan.rem_tiles * plan.split * C::BM * C::BN * sizeof(float) > kPartialBytes) return OPTIML_ERR_UNSUPPORTED;
    const int grid = plan.grid;
    const __nv_bfloat16* bi = (const __nv_bfloat16*)bias;
    switch (act) {
    case OPTIML_ACT_RELU:
        launch_pdl(gemm_umma_kernel<kActRelu>, dim3(grid), dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N, K,
                   plan, h->partials, h->counters, h->status);
        break;
    case OPTIML_ACT_GELU_TANH:
        launch_pdl(gemm_umma_kernel<kActGeluTanh>, dim3(grid), dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N, K,
                   plan, h->partials, h->counters, h->status);
        break;
    case OPTIML_ACT_SIGMOID:
        launch_pdl(gemm_umma_kernel<kActSigmoid>, dim3(grid), dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N, K,
                   plan, h->partials, h->counters, h->status);
        break;
    default:
        launch_pdl(gemm_umma_kernel<kActNone>, dim3(grid), dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N, K,
                   plan, h->partials, h->counters, h->status);
        break;
    }
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

optiml_status_t launch_umma2(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M, int N,
                             int K, int act, cudaStream_t st) {
    using C = Umma2Cfg;
    CUtensorMap ma, mb, my;
    if (!get_map(h, &ma, A, (uint64_t)M, (uint64_t)K, 128, 64) || !get_map(h, &mb, B, (uint64_t)K, (uint64_t)N, 64, 64) ||
        !get_map(h, &my, Y, (uint64_t)M, (uint64_t)N, 32, 64))
        return OPTIML_ERR_CUDA;
    const UmmaPlan plan = make_umma2_plan(M, N, K, h->num_sms, (int)h->options[OPTIML_OPT_PAIR_SPLIT_MAX]);
    if ((size_t)plan.rem_tiles * plan.split * C::BM * C::BN * sizeof(float) > kPartialBytes) return OPTIML_ERR_UNSUPPORTED;
    if (2 * plan.rem_tiles > kNumCounters) return OPTIML_ERR_UNSUPPORTED;
    const dim3 grid(2 * plan.grid);          // CTA pairs: the kernel is compiled with cluster dimensions (2, 1, 1)
    const __nv_bfloat16* bi = (const __nv_bfloat16*)bias;
    switch (act) {
    case OPTIML_ACT_RELU:
        launch_pdl(gemm_umma2_kernel<kActRelu>, grid, dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N, K,
                   plan, h->partials, h->counters, h->status);
        break;
    case OPTIML_ACT_GELU_TANH:
        launch_pdl(gemm_umma2_kernel<kActGeluTanh>, grid, dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N,
                   K, plan, h->partials, h->counters, h->status);
        break;
    case OPTIML_ACT_SIGMOID:
        launch_pdl(gemm_umma2_kernel<kActSigmoid>, grid, dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N,
                   K, plan, h->partials, h->counters, h->status);
        break;
    default:
        launch_pdl(gemm_umma2_kernel<kActNone>, grid, dim3(C::kThreads), C::kSmemBytes, st, ma, mb, my, bi, M, N, K,
                   plan, h->partials, h->counters, h->status);
        break;
    }
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

// The streaming pair kernel: programmatic dependent launch plus a cluster of 2 * split CTAs.
template <int ACT, bool HM, int BN>
cudaError_t launch_umma2s_act(dim3 grid, int cluster, cudaStream_t st, const CUtensorMap& ma, const CUtensorMap& mb,
                              __nv_bfloat16* Y, const __nv_bfloat16* bias, int M, int N, int K,
                              const Umma2sPlan& plan, int* status) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(Umma2sCfgT<HM, BN>::kThreads);
    cfg.dynamicSmemBytes = Umma2sCfgT<HM, BN>::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_umma2s_kernel<ACT, HM, BN>, ma, mb, Y, bias, M, N, K, plan, status);
}

// Up to 128 rows a pair shares a 128-row tile (64 rows per CTA); above, a 256-row tile.
bool stream_half_height(optiml_handle_t h, int64_t M) { return M <= Umma2sHalfCfg::BM && h->options[OPTIML_OPT_PAIR_HALF_HEIGHT] != 0; }

template <bool HM, int BN>
optiml_status_t launch_umma2s_form(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M, int N,
                                   int K, int act, cudaStream_t st) {
    using C = Umma2sCfgT<HM, BN>;
    CUtensorMap ma, mb;
    if (!get_map(h, &ma, A, (uint64_t)M, (uint64_t)K, C::kRowsPerCta, 64) || !get_map(h, &mb, B, (uint64_t)K, (uint64_t)N, 64, 64))
        return OPTIML_ERR_CUDA;
    Umma2sPlan plan;
    plan.tiles_m = (int)ceil_div64(M, C::BM);
    plan.tiles_n = (int)ceil_div64(N, C::BN);
    plan.num_kb = (int)ceil_div64(K, C::BK);
    const int64_t tiles = (int64_t)plan.tiles_m * plan.tiles_n;
    if (tiles > h->stream_clusters[0]) return OPTIML_ERR_UNSUPPORTED;
    plan.split = stream_split(h, tiles, plan.num_kb, C::kTmemCols);
    if (h->log) fprintf(stderr, "[optiml] streaming pair plan: %d x %d tiles=%lld split=%d kb=%d\n", C::BM, C::BN, (long long)tiles, plan.split, plan.num_kb);
    const int cluster = 2 * plan.split;
    const dim3 grid((unsigned)(tiles * cluster));
    const __nv_bfloat16* bi = (const __nv_bfloat16*)bias;
    switch (act) {
    case OPTIML_ACT_RELU: launch_umma2s_act<kActRelu, HM, BN>(grid, cluster, st, ma, mb, (__nv_bfloat16*)Y, bi, M, N, K, plan, h->status); break;
    case OPTIML_ACT_GELU_TANH: launch_umma2s_act<kActGeluTanh, HM, BN>(grid, cluster, st, ma, mb, (__nv_bfloat16*)Y, bi, M, N, K, plan, h->status); break;
    case OPTIML_ACT_SIGMOID: launch_umma2s_act<kActSigmoid, HM, BN>(grid, cluster, st, ma, mb, (__nv_bfloat16*)Y, bi, M, N, K, plan, h->status); break;
    default: launch_umma2s_act<kActNone, HM, BN>(grid, cluster, st, ma, mb, (__nv_bfloat16*)Y, bi, M, N, K, plan, h->status); break;
    }
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

optiml_status_t launch_umma2s(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int M, int N,
                              int K, int act, cudaStream_t st) {
    const bool hm = stream_half_height(h, M);
    const bool narrow = stream_tile_width(h, M, N, K, hm) == 128;
    if (hm) return narrow ? launch_umma2s_form<true, 128>(h, A, B, bias, Y, M, N, K, act, st)
                          : launch_umma2s_form<true, 256>(h, A, B, bias, Y, M, N, K, act, st);
    return narrow ? launch_umma2s_form<false, 128>(h, A, B, bias, Y, M, N, K, act, st)
                  : launch_umma2s_form<false, 256>(h, A, B, bias, Y, M, N, K, act, st);
}

// Clusters of `cluster` CTAs of the streaming pair kernel that can be resident at the same time.
int query_stream_clusters(int cluster) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(cluster * 64));
    cfg.blockDim = dim3(Umma2sCfg::kThreads);
    cfg.dynamicSmemBytes = Umma2sCfg::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_umma2s_kernel<kActNone, false, 256>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

template <typename F>
bool set_smem(F* fn, int bytes) {
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// Streaming kernels: the whole shared-memory carve-out (with a short ring, option
// SKINNY_RING_STAGES, this call's and the next call's CTAs can then share an SM).
template <typename F>
bool set_skinny(F* fn, int bytes) {
    return set_smem(fn, bytes) &&
           cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) ==
               cudaSuccess;
}

bool configure_kernels() {
    bool ok = true;
    ok &= set_smem(gemm_umma_kernel<kActNone>, UmmaCfg::kSmemBytes);
    ok &= set_smem(gemm_umma_kernel<kActRelu>, UmmaCfg::kSmemBytes);
    ok &= set_smem(gemm_umma_kernel<kActGeluTanh>, UmmaCfg::kSmemBytes);
    ok &= set_smem(gemm_umma_kernel<kActSigmoid>, UmmaCfg::kSmemBytes);
    ok &= set_smem(gemm_umma2_kernel<kActNone>, Umma2Cfg::kSmemBytes);
    ok &= set_smem(gemm_umma2_kernel<kActRelu>, Umma2Cfg::kSmemBytes);
    ok &= set_smem(gemm_umma2_kernel<kActGeluTanh>, Umma2Cfg::kSmemBytes);
    ok &= set_smem(gemm_umma2_kernel<kActSigmoid>, Umma2Cfg::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActNone, false, 256>, Umma2sCfgT<false, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActRelu, false, 256>, Umma2sCfgT<false, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActGeluTanh, false, 256>, Umma2sCfgT<false, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActSigmoid, false, 256>, Umma2sCfgT<false, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActNone, false, 128>, Umma2sCfgT<false, 128>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActRelu, false, 128>, Umma2sCfgT<false, 128>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActGeluTanh, false, 128>, Umma2sCfgT<false, 128>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActSigmoid, false, 128>, Umma2sCfgT<false, 128>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActNone, true, 256>, Umma2sCfgT<true, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActRelu, true, 256>, Umma2sCfgT<true, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActGeluTanh, true, 256>, Umma2sCfgT<true, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActSigmoid, true, 256>, Umma2sCfgT<true, 256>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActNone, true, 128>, Umma2sCfgT<true, 128>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActRelu, true, 128>, Umma2sCfgT<true, 128>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActGeluTanh, true, 128>, Umma2sCfgT<true, 128>::kSmemBytes);
    ok &= set_smem(gemm_umma2s_kernel<kActSigmoid, true, 128>, Umma2sCfgT<true, 128>::kSmemBytes);
    ok &= set_skinny(gemm_skinny_umma_kernel<16, 2>, SkinnyCfg<16, 2>::kSmemBytes);
    ok &= set_skinny(gemm_skinny_umma_kernel<16, 3>, SkinnyCfg<16, 3>::kSmemBytes);
    ok &= set_skinny(gemm_skinny_umma_kernel<32, 2>, SkinnyCfg<32, 2>::kSmemBytes);
    ok &= set_skinny(gemm_skinny_umma_kernel<32, 3>, SkinnyCfg<32, 3>::kSmemBytes);
    ok &= set_skinny(gemm_skinny_umma_kernel<64, 2>, SkinnyCfg<64, 2>::kSmemBytes);
    ok &= set_skinny(gemm_skinny_umma_kernel<128, 2>, SkinnyCfg<128, 2>::kSmemBytes);
    ok &= set_smem(mhsa_umma_kernel<64>, MhsaCfg<64>::kSmemBytes);
    ok &= set_smem(mhsa_umma_kernel<128>, MhsaCfg<128>::kSmemBytes);
    // the attention kernel re-divides its registers between warpgroups and would wait forever
    // if the launch handed out fewer than its shares add up to
    cudaFuncAttributes fa;
    ok = ok && cudaFuncGetAttributes(&fa, mhsa_umma_kernel<64>) == cudaSuccess && fa.numRegs >= MhsaCfg<64>::kLaunchRegs;
    ok = ok && cudaFuncGetAttributes(&fa, mhsa_umma_kernel<128>) == cudaSuccess && fa.numRegs >= MhsaCfg<128>::kLaunchRegs;
    ok = ok && set_smem(mhsa_umma2_kernel, Mhsa2Cfg::kSmemBytes);
    ok = ok && cudaFuncGetAttributes(&fa, mhsa_umma2_kernel) == cudaSuccess && fa.numRegs >= Mhsa2Cfg::kLaunchRegs;
    return ok;
}

template <int DK>
optiml_status_t launch_mhsa_umma(optiml_handle_t h, const void* Q, const void* K, const void* V, void* Y, int N,
                                 int d_model, int heads, cudaStream_t st) {
    using C = MhsaCfg<DK>;
    CUtensorMap mq, mk, mv;
    if (!get_map(h, &mq, Q, (uint64_t)N, (uint64_t)d_model, 128, 64) || !get_map(h, &mk, K, (uint64_t)N, (uint64_t)d_model, 128, 64) ||
        !get_map(h, &mv, V, (uint64_t)N, (uint64_t)d_model, 128, 64))
        return OPTIML_ERR_CUDA;
    const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)DK));
    const dim3 grid((unsigned)ceil_div64(N, C::kQTiles * C::BQ), (unsigned)heads);
    launch_pdl(mhsa_umma_kernel<DK>, grid, dim3(C::kThreads), C::kSmemBytes, st, mq, mk, mv, (__nv_bfloat16*)Y, N,
               d_model, scale_log2, h->status);
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

// d_k = 128 as a CTA pair: 512 query rows per cluster of two CTAs, each staging half of every K and V block
optiml_status_t launch_mhsa_umma2(optiml_handle_t h, const void* Q, const void* K, const void* V, void* Y, int N,
                                  int d_model, int heads, cudaStream_t st) {
    using C = Mhsa2Cfg;
    CUtensorMap mq, mk, mv;
    if (!get_map(h, &mq, Q, (uint64_t)N, (uint64_t)d_model, 128, 64) || !get_map(h, &mk, K, (uint64_t)N, (uint64_t)d_model, 64, 64) ||
        !get_map(h, &mv, V, (uint64_t)N, (uint64_t)d_model, 128, 64))
        return OPTIML_ERR_CUDA;
    const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)C::DK));
    const dim3 grid((unsigned)(2 * ceil_div64(N, 2 * C::kQTiles * C::BQ)), (unsigned)heads);   // the kernel is compiled with cluster dimensions (2, 1, 1)
    launch_pdl(mhsa_umma2_kernel, grid, dim3(C::kThreads), C::kSmemBytes, st, mq, mk, mv, (__nv_bfloat16*)Y, N, d_model,
               scale_log2, h->status);
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

template <typename T>
optiml_status_t launch_mhsa_generic(optiml_handle_t h, const void* Q, const void* K, const void* V, void* Y, int N,
                                    int d_model, int heads, cudaStream_t st) {
    const int64_t warps = (int64_t)N * heads;
    const float scale = (float)(1.0 / sqrt((double)(d_model / heads)));
    launch_pdl(mhsa_generic_kernel<T>, dim3((unsigned)ceil_div64(warps, kMhsaGenericWarps)), dim3(kMhsaGenericWarps * 32), 0,
               st, (const T*)Q, (const T*)K, (const T*)V, (T*)Y, N, d_model, heads, scale);
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

// tcgen05 attention needs bf16, d_k of 64 or 128 and 16-byte aligned rows
bool mhsa_umma_supported(int64_t d_model, int64_t heads, int dtype, bool al16) {
    const int64_t dk = d_model / heads;
    return dtype == OPTIML_BF16 && (dk == 64 || dk == 128) && al16 && heads <= 65535;
}

// Grow one of the handle's on-demand device buffers to `need` bytes.  Earlier work on the
// stream may still use the old buffer, so the stream is synchronised before it is freed.
optiml_status_t grow_buffer(void** buf, size_t* have, size_t need, cudaStream_t st) {
    if (*have >= need) return OPTIML_OK;
    if (cudaStreamSynchronize(st) != cudaSuccess) return OPTIML_ERR_CUDA;
    cudaFree(*buf);
    *buf = nullptr;
    *have = 0;
    if (!dev_alloc(buf, need)) return OPTIML_ERR_ALLOC;   // the handle stays usable; this buffer is empty
    *have = need;
    return OPTIML_OK;
}

// Problems whose N or K is not a multiple of 16 bytes' worth of elements (8 bf16, 4 fp32) cannot be
// addressed by TMA, nor by the 128-bit loads of the fp32 tiles, in place.  Large ones are worth two or
// three extra streaming passes: A (if K is ragged) and B are copied into zero-padded buffers with
// 16-byte row pitches, the fast variant for the padded shape runs into a padded Y (if N is ragged),
// and the leading N columns are copied back.  (bf16 4096 x 4100 x 4096: 5.6 ms on the predicated FMA
// kernel, 0.14 ms this way.)
optiml_status_t gemm_repacked(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int64_t M,
                              int64_t N, int64_t K, optiml_dtype_t dtype, optiml_act_t act, void* stream);
bool worth_repacking(int64_t M, int64_t N, int64_t K) { return M >= 16 && (double)M * (double)N * (double)K >= 134217728.0; }

optiml_status_t check_args(optiml_handle_t h, const void* A, const void* B, const void* Y, int64_t M, int64_t N,
                           int64_t K, int dtype, int act) {
    if (!h || !A || !B || !Y) return OPTIML_ERR_INVALID_ARG;
    if (M < 1 || N < 1 || K < 1 || M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return OPTIML_ERR_INVALID_ARG;
    if (dtype != OPTIML_F32 && dtype != OPTIML_BF16) return OPTIML_ERR_INVALID_ARG;
    if (act != OPTIML_ACT_NONE && act != OPTIML_ACT_RELU && act != OPTIML_ACT_GELU_TANH && act != OPTIML_ACT_SIGMOID) return OPTIML_ERR_INVALID_ARG;
    return OPTIML_OK;
}

}  // namespace

// ---------------------------------------------------------------- exported entry points

extern "C" {

optiml_status_t optiml_create(optiml_handle_t* out, int device) {
    if (!out) return OPTIML_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) return OPTIML_ERR_CUDA;
    if (device < 0 || device >= count) return OPTIML_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return OPTIML_ERR_CUDA;
    if (prop.major != 10 || prop.minor != 0) return OPTIML_ERR_ARCH;

    optiml_handle_t h = new (std::nothrow) optiml_handle_s();
    if (!h) return OPTIML_ERR_ALLOC;
    h->device = device;
    h->num_sms = prop.multiProcessorCount;
    const char* lg = getenv("OPTIML_LOG");
    h->log = lg && lg[0] == '1';
    for (int i = 0; i < OPTIML_OPT_COUNT; ++i) h->options[i] = kOptionDefaults[i];

    DeviceGuard guard(device);
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        delete h;
        return OPTIML_ERR_CUDA;
    }
    h->encode = reinterpret_cast<encode_tiled_fn>(fn);

    bool ok = dev_alloc(&h->partials, kPartialBytes);
    ok = ok && dev_alloc(&h->counters, kNumCounters * sizeof(unsigned int));
    ok = ok && dev_alloc(&h->status, sizeof(int));
    if (!ok) {
        optiml_destroy(h);       // frees what was allocated before the failure
        return OPTIML_ERR_ALLOC;
    }
    ok = cudaMemset(h->counters, 0, kNumCounters * sizeof(unsigned int)) == cudaSuccess;
    ok = ok && cudaMemset(h->status, 0, sizeof(int)) == cudaSuccess;
    ok = ok && configure_kernels();
    if (ok)
        for (int i = 0; i < 3; ++i) h->stream_clusters[i] = query_stream_clusters(2 << i);
    if (h->log) fprintf(stderr, "[optiml] resident clusters of the streaming pair kernel: %d of 2 CTAs, %d of 4, %d of 8\n", h->stream_clusters[0], h->stream_clusters[1], h->stream_clusters[2]);
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        optiml_destroy(h);
        return OPTIML_ERR_CUDA;
    }
    *out = h;
    return OPTIML_OK;
}

optiml_status_t optiml_destroy(optiml_handle_t h) {
    if (!h) return OPTIML_OK;
    DeviceGuard guard(h->device);
    cudaDeviceSynchronize();
    cudaFree(h->partials);
    cudaFree(h->counters);
    cudaFree(h->status);
    for (int i = 0; i < 4; ++i) cudaFree(h->stage[i]);
    for (int i = 0; i < 4; ++i) cudaFree(h->pad[i]);
    cudaGetLastError();
    delete h;
    return OPTIML_OK;
}

optiml_status_t optiml_gemm_epilogue(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y,
                                     int64_t M, int64_t N, int64_t K, optiml_dtype_t dtype, optiml_act_t act,
                                     void* stream) {
    optiml_status_t s = check_args(h, A, B, Y, M, N, K, (int)dtype, (int)act);
    if (s != OPTIML_OK) return s;
    const uintptr_t es = dtype == OPTIML_F32 ? 4 : 2;
    const uintptr_t all = reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) |
                          reinterpret_cast<uintptr_t>(bias) | reinterpret_cast<uintptr_t>(Y);
    if (all & (es - 1)) return OPTIML_ERR_ALIGNMENT;
    const bool al16 = aligned16(A) && aligned16(B) && aligned16(bias) && aligned16(Y);
    const int64_t vec = dtype == OPTIML_F32 ? 4 : 8;       // elements per 16 bytes
    if ((N % vec != 0 || K % vec != 0) && al16 && h->forced == OPTIML_VARIANT_AUTO && worth_repacking(M, N, K))
        return gemm_repacked(h, A, B, bias, Y, M, N, K, dtype, act, stream);
    const int v = choose_variant(h, M, N, K, (int)dtype, al16);
    if (!variant_supports(h, v, M, N, K, (int)dtype, al16)) return OPTIML_ERR_UNSUPPORTED;
    if (h->log)
        fprintf(stderr, "[optiml] M=%lld N=%lld K=%lld dtype=%d act=%d -> %s\n", (long long)M, (long long)N,
                (long long)K, (int)dtype, (int)act, optiml_variant_name(v));

    DeviceGuard guard(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int m = (int)M, n = (int)N, k = (int)K;
    switch (v) {
    case OPTIML_VARIANT_F32_TILED:
        return launch_f32(h, A, B, bias, Y, m, n, k, (int)act, st);
    case OPTIML_VARIANT_GEMV_SPLITK:
        return launch_gemv(h, A, B, bias, Y, m, n, k, (int)dtype, (int)act, st);
    case OPTIML_VARIANT_SKINNY_UMMA:
        return launch_skinny(h, A, B, bias, Y, m, n, k, (int)act, st);
    case OPTIML_VARIANT_UMMA:
        return launch_umma(h, A, B, bias, Y, m, n, k, (int)act, st);
    case OPTIML_VARIANT_UMMA_2CTA:
        return launch_umma2(h, A, B, bias, Y, m, n, k, (int)act, st);
    case OPTIML_VARIANT_UMMA_2CTA_STREAM:
        return launch_umma2s(h, A, B, bias, Y, m, n, k, (int)act, st);
    default:
        return dtype == OPTIML_F32 ? launch_generic<float>(h, A, B, bias, Y, m, n, k, (int)act, st)
                                   : launch_generic<__nv_bfloat16>(h, A, B, bias, Y, m, n, k, (int)act, st);
    }
}

}  // extern "C"

namespace {

template <typename E>
optiml_status_t gemm_repacked_t(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int64_t M,
                                int64_t N, int64_t K, optiml_dtype_t dtype, optiml_act_t act, void* stream) {
    constexpr int64_t V = RepackVec<E>::V;
    DeviceGuard guard(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t Np = (N + V - 1) / V * V, Kp = (K + V - 1) / V * V;
    const bool pad_a = Kp != K, pad_n = Np != N;
    const size_t es = sizeof(E);
    const size_t need[4] = {pad_a ? (size_t)M * Kp * es : 0, (size_t)Kp * Np * es, pad_n && bias ? (size_t)Np * es : 0,
                            pad_n ? (size_t)M * Np * es : 0};
    for (int i = 0; i < 4; ++i) {
        const optiml_status_t s = grow_buffer(&h->pad[i], &h->pad_bytes[i], need[i], st);
        if (s != OPTIML_OK) return s;
    }
    auto blocks = [&](int64_t rows, int64_t cols_pad) {
        const int64_t want = ceil_div64(rows * (cols_pad / V), kRepackThreads);
        const int64_t cap = (int64_t)h->num_sms * 16;
        return dim3((unsigned)(want < cap ? (want < 1 ? 1 : want) : cap));
    };
    const void *a = A, *b = B, *bi = bias;
    void* y = Y;
    if (pad_a) {
        pad_rows_kernel<E><<<blocks(M, Kp), kRepackThreads, 0, st>>>((const E*)A, (E*)h->pad[0], M, M, K, Kp);
        a = h->pad[0];
        h->launches += 1;
    }
    // B always moves: its row pitch changes with N, and with a ragged K it gains zero rows up to Kp
    pad_rows_kernel<E><<<blocks(Kp, Np), kRepackThreads, 0, st>>>((const E*)B, (E*)h->pad[1], K, Kp, N, Np);
    b = h->pad[1];
    h->launches += 1;
    if (pad_n) {
        y = h->pad[3];
        if (bias) {
            pad_rows_kernel<E><<<blocks(1, Np), kRepackThreads, 0, st>>>((const E*)bias, (E*)h->pad[2], 1, 1, N, Np);
            bi = h->pad[2];
            h->launches += 1;
        }
    }
    if (cudaGetLastError() != cudaSuccess) return OPTIML_ERR_CUDA;
    const optiml_status_t s = optiml_gemm_epilogue(h, a, b, bi, y, M, Np, Kp, dtype, act, stream);
    if (s != OPTIML_OK) return s;
    if (pad_n) {
        unpad_rows_kernel<E><<<blocks(M, Np), kRepackThreads, 0, st>>>((const E*)h->pad[3], (E*)Y, M, N, Np);   // Y is 16-byte aligned here
        h->launches += 1;
    }
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

optiml_status_t gemm_repacked(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y, int64_t M,
                              int64_t N, int64_t K, optiml_dtype_t dtype, optiml_act_t act, void* stream) {
    return dtype == OPTIML_F32 ? gemm_repacked_t<uint32_t>(h, A, B, bias, Y, M, N, K, dtype, act, stream)
                               : gemm_repacked_t<uint16_t>(h, A, B, bias, Y, M, N, K, dtype, act, stream);
}

}  // namespace

extern "C" {

optiml_status_t optiml_gemm_epilogue_host(optiml_handle_t h, const void* A_host, const void* B_host,
                                          const void* bias_host, void* Y_host, int64_t M, int64_t N, int64_t K,
                                          optiml_dtype_t dtype, optiml_act_t act, void* stream) {
    optiml_status_t s = check_args(h, A_host, B_host, Y_host, M, N, K, (int)dtype, (int)act);
    if (s != OPTIML_OK) return s;
    DeviceGuard guard(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t es = dtype == OPTIML_F32 ? 4 : 2;
    const size_t need[4] = {(size_t)M * K * es, (size_t)K * N * es, (size_t)N * es, (size_t)M * N * es};
    for (int i = 0; i < 4; ++i) {
        const optiml_status_t g = grow_buffer(&h->stage[i], &h->stage_bytes[i], need[i], st);
        if (g != OPTIML_OK) return g;
    }
    bool ok = cudaMemcpyAsync(h->stage[0], A_host, need[0], cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h->stage[1], B_host, need[1], cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (bias_host) ok = ok && cudaMemcpyAsync(h->stage[2], bias_host, need[2], cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!ok) return OPTIML_ERR_CUDA;
    s = optiml_gemm_epilogue(h, h->stage[0], h->stage[1], bias_host ? h->stage[2] : nullptr, h->stage[3], M, N, K, dtype,
                             act, stream);
    if (s != OPTIML_OK) return s;
    ok = cudaMemcpyAsync(Y_host, h->stage[3], need[3], cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    return ok ? OPTIML_OK : OPTIML_ERR_CUDA;
}

optiml_status_t optiml_get_last_status(optiml_handle_t h) {
    if (!h) return OPTIML_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    int word = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return OPTIML_ERR_CUDA;
    if (cudaMemcpy(&word, h->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return OPTIML_ERR_CUDA;
    if (word != kDevOk) {
        if (h->log)
            fprintf(stderr, "[optiml] bounded wait gave up: wait site %d in CTA %d\n", (word >> 8) & 0xFF, (word >> 16) & 0x7FFF);
        // a kernel that gave up may have left arrival counters half way: re-arm everything
        cudaMemset(h->status, 0, sizeof(int));
        cudaMemset(h->counters, 0, kNumCounters * sizeof(unsigned int));
        cudaDeviceSynchronize();
        return OPTIML_ERR_TIMEOUT;
    }
    return OPTIML_OK;
}

optiml_status_t optiml_selftest_timeout(optiml_handle_t h, int64_t limit_cycles, void* stream) {
    if (!h || limit_cycles < 1 || limit_cycles > kSelftestMaxCycles) return OPTIML_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    launch_pdl(selftest_timeout_kernel, dim3(1), dim3(32), 0, static_cast<cudaStream_t>(stream), (long long)limit_cycles,
               h->status);
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

optiml_status_t optiml_set_alloc_hook(optiml_alloc_hook_t hook, void* user) {
    g_alloc_hook = hook;
    g_alloc_hook_user = user;
    return OPTIML_OK;
}

optiml_status_t optiml_reduce_f32(optiml_handle_t h, optiml_reduce_t kind, const float* x, const float* y, int64_t n,
                                  float* out, void* stream) {
    if (!h || !x || !out || n < 1) return OPTIML_ERR_INVALID_ARG;
    if (kind != OPTIML_REDUCE_SUM && kind != OPTIML_REDUCE_DOT && kind != OPTIML_REDUCE_MSE) return OPTIML_ERR_INVALID_ARG;
    if (kind != OPTIML_REDUCE_SUM && !y) return OPTIML_ERR_INVALID_ARG;
    if (!aligned16(x) || (kind != OPTIML_REDUCE_SUM && !aligned16(y)) || (reinterpret_cast<uintptr_t>(out) & 3))
        return OPTIML_ERR_ALIGNMENT;
    DeviceGuard guard(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // one wave of resident CTAs, fewer when the vector is short: one float4 per thread at least
    int64_t ctas = (int64_t)h->num_sms * kReduceCtasPerSm;
    const int64_t need = ceil_div64(ceil_div64(n, 4), kReduceThreads);
    if (ctas > need) ctas = need;
    if (ctas < 1) ctas = 1;
    double* partials = reinterpret_cast<double*>(h->partials);
    const dim3 grid((unsigned)ctas), block(kReduceThreads);
    switch (kind) {
    case OPTIML_REDUCE_DOT:
        launch_pdl(reduce_f32_kernel<kReduceDot>, grid, block, 0, st, x, y, n, out, partials, h->counters);
        break;
    case OPTIML_REDUCE_MSE:
        launch_pdl(reduce_f32_kernel<kReduceMse>, grid, block, 0, st, x, y, n, out, partials, h->counters);
        break;
    default:
        launch_pdl(reduce_f32_kernel<kReduceSum>, grid, block, 0, st, x, y, n, out, partials, h->counters);
        break;
    }
    h->launches += 1;
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

optiml_status_t optiml_mhsa(optiml_handle_t h, const void* Q, const void* K, const void* V, void* Y, int64_t N,
                            int64_t d_model, int64_t heads, optiml_dtype_t dtype, void* stream) {
    if (!h || !Q || !K || !V || !Y) return OPTIML_ERR_INVALID_ARG;
    if (N < 1 || d_model < 1 || heads < 1 || N > INT32_MAX || d_model > INT32_MAX || d_model % heads != 0)
        return OPTIML_ERR_INVALID_ARG;
    if (dtype != OPTIML_F32 && dtype != OPTIML_BF16) return OPTIML_ERR_INVALID_ARG;
    const uintptr_t es = dtype == OPTIML_F32 ? 4 : 2;
    const uintptr_t all = reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) |
                          reinterpret_cast<uintptr_t>(V) | reinterpret_cast<uintptr_t>(Y);
    if (all & (es - 1)) return OPTIML_ERR_ALIGNMENT;
    const bool al16 = (all & 15) == 0 && d_model % 8 == 0;
    const int64_t dk = d_model / heads;
    const bool fast = mhsa_umma_supported(d_model, heads, (int)dtype, al16);
    const bool want_fast = h->forced == OPTIML_VARIANT_AUTO ? fast : h->forced != OPTIML_VARIANT_GENERIC;
    if (want_fast && !fast) return OPTIML_ERR_UNSUPPORTED;
    if (!want_fast && (dk > kMhsaGenericMaxDk || (int64_t)N * heads > ((int64_t)1 << 32))) return OPTIML_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (h->log)
        fprintf(stderr, "[optiml] mhsa N=%lld d_model=%lld heads=%lld dtype=%d -> %s\n", (long long)N, (long long)d_model,
                (long long)heads, (int)dtype,
                !want_fast ? "mhsa_generic_fma" : (dk == 128 && h->forced == OPTIML_VARIANT_UMMA_2CTA ? "mhsa_tcgen05_cta_pair" : "mhsa_tcgen05"));
    if (want_fast) {
        if (dk == 64) return launch_mhsa_umma<64>(h, Q, K, V, Y, (int)N, (int)d_model, (int)heads, st);
        // d_k = 128: the single-CTA kernel; the CTA-pair kernel only as the forced variant OPTIML_VARIANT_UMMA_2CTA
        // (measured at N = 16384, 16 heads: 1776 us against 2029 us for the pair in short regions, 2061 against
        // 2056 us back to back under the power cap)
        if (h->forced != OPTIML_VARIANT_UMMA_2CTA) return launch_mhsa_umma<128>(h, Q, K, V, Y, (int)N, (int)d_model, (int)heads, st);
        return launch_mhsa_umma2(h, Q, K, V, Y, (int)N, (int)d_model, (int)heads, st);
    }
    return dtype == OPTIML_F32 ? launch_mhsa_generic<float>(h, Q, K, V, Y, (int)N, (int)d_model, (int)heads, st)
                               : launch_mhsa_generic<__nv_bfloat16>(h, Q, K, V, Y, (int)N, (int)d_model, (int)heads, st);
}

optiml_status_t optiml_force_variant(optiml_handle_t h, optiml_variant_t v) {
    if (!h || (int)v < OPTIML_VARIANT_AUTO || (int)v >= OPTIML_VARIANT_COUNT) return OPTIML_ERR_INVALID_ARG;
    h->forced = (int)v;
    return OPTIML_OK;
}

int optiml_select_variant(optiml_handle_t h, int64_t M, int64_t N, int64_t K, optiml_dtype_t dtype) {
    if (!h || M < 1 || N < 1 || K < 1 || (dtype != OPTIML_F32 && dtype != OPTIML_BF16)) return -1;
    return choose_variant(h, M, N, K, (int)dtype, true);
}

int64_t optiml_launch_count(optiml_handle_t h) { return h ? h->launches : -1; }

optiml_status_t optiml_set_option(optiml_handle_t h, optiml_option_t opt, int64_t value) {
    if (!h || (int)opt < 0 || (int)opt >= OPTIML_OPT_COUNT) return OPTIML_ERR_INVALID_ARG;
    if (value < 0 || value > (1 << 20)) return OPTIML_ERR_INVALID_ARG;
    h->options[opt] = value;
    return OPTIML_OK;
}

int64_t optiml_get_option(optiml_handle_t h, optiml_option_t opt) {
    if (!h || (int)opt < 0 || (int)opt >= OPTIML_OPT_COUNT) return -1;
    return h->options[opt];
}

const char* optiml_status_string(optiml_status_t s) {
    switch (s) {
    case OPTIML_OK: return "ok";
    case OPTIML_ERR_INVALID_ARG: return "invalid argument";
    case OPTIML_ERR_UNSUPPORTED: return "shape or dtype not supported by the forced variant";
    case OPTIML_ERR_ALIGNMENT: return "pointer not aligned to its element size";
    case OPTIML_ERR_ARCH: return "device is not compute capability 10.0 (B200)";
    case OPTIML_ERR_ALLOC: return "allocation failed";
    case OPTIML_ERR_CUDA: return "CUDA call failed";
    case OPTIML_ERR_TIMEOUT: return "a bounded on-device wait gave up";
    default: return "unknown status";
    }
}

const char* optiml_variant_name(int variant) {
    switch (variant) {
    case OPTIML_VARIANT_AUTO: return "auto";
    case OPTIML_VARIANT_GENERIC: return "generic_fma";
    case OPTIML_VARIANT_F32_TILED: return "f32_tiled_fma";
    case OPTIML_VARIANT_GEMV_SPLITK: return "gemv_splitk_stream";
    case OPTIML_VARIANT_SKINNY_UMMA: return "skinny_streamk_tcgen05";
    case OPTIML_VARIANT_UMMA: return "persistent_tcgen05";
    case OPTIML_VARIANT_UMMA_2CTA: return "persistent_tcgen05_cta_pair";
    case OPTIML_VARIANT_UMMA_2CTA_STREAM: return "cluster_splitk_tcgen05_cta_pair";
    default: return "unknown";
    }
}

int optiml_version(void) { return kVersion; }

// ---------------------------------------------------------------- entry point that allocates nothing

}  // extern "C"

namespace {

// Scratch of optiml_gemv_noalloc: arrival counters (one per 256-column block) followed by the
// split-K partial sums.  It lives in the library image, so every GPU that loads the library
// holds these bytes until the process exits, whether or not the entry point is ever called.
constexpr int kNoAllocMaxN = 65536;
constexpr size_t kNoAllocCounterBytes = (kNoAllocMaxN / kGemvCols) * sizeof(unsigned int);   // 1 KiB
constexpr size_t kNoAllocPartialBytes = (size_t)2 << 20;                                      // 2 MiB
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocCounterBytes + kNoAllocPartialBytes];

constexpr int kNoAllocMaxDevices = 64;
unsigned char* g_noalloc_ptr[kNoAllocMaxDevices] = {};   // device address of the array, per device
int g_noalloc_sms[kNoAllocMaxDevices] = {};

}  // namespace

extern "C" {

optiml_status_t optiml_gemv_noalloc(const void* A, const void* B, const void* bias, void* Y, int64_t M, int64_t N,
                                    int64_t K, optiml_act_t act, int device, void* stream) {
    if (!A || !B || !Y || M < 1 || N < 1 || K < 1 || K > INT32_MAX) return OPTIML_ERR_INVALID_ARG;
    if (act != OPTIML_ACT_NONE && act != OPTIML_ACT_RELU && act != OPTIML_ACT_GELU_TANH && act != OPTIML_ACT_SIGMOID) return OPTIML_ERR_INVALID_ARG;
    int device_count = 0;
    if (cudaGetDeviceCount(&device_count) != cudaSuccess) {
        cudaGetLastError();
        return OPTIML_ERR_CUDA;
    }
    if (device < 0 || device >= device_count || device >= kNoAllocMaxDevices) return OPTIML_ERR_INVALID_ARG;
    // limits of the fixed scratch and of the kernel: refuse, never truncate
    if (M > 4 || N > kNoAllocMaxN || N % 8 != 0) return OPTIML_ERR_UNSUPPORTED;
    if (!(aligned16(A) && aligned16(B) && aligned16(bias) && aligned16(Y))) return OPTIML_ERR_ALIGNMENT;

    DeviceGuard guard(device);
    if (!guard.ok) {
        cudaGetLastError();
        return OPTIML_ERR_CUDA;
    }
    if (!g_noalloc_ptr[device]) {
        // One-time set-up on this device (it must be the current one here).  In host code the
        // name of a __device__ array is only a stand-in; the address a kernel may use comes
        // from cudaGetSymbolAddress.
        int major = 0, minor = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            cudaGetLastError();
            return OPTIML_ERR_CUDA;
        }
        if (major != 10 || minor != 0) return OPTIML_ERR_ARCH;
        unsigned char* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return OPTIML_ERR_CUDA;
        }
        g_noalloc_sms[device] = sms;
        g_noalloc_ptr[device] = p;       // published last: a non-null pointer means the SM count is set
    }
    unsigned char* base = g_noalloc_ptr[device];
    unsigned int* counters = reinterpret_cast<unsigned int*>(base);
    float* partials = reinterpret_cast<float*>(base + kNoAllocCounterBytes);

    const int m = (int)M, n = (int)N, k = (int)K;
    const int MR = m == 1 ? 1 : (m == 2 ? 2 : 4);
    const int64_t col_blocks = ceil_div64(N, kGemvCols);
    int64_t S = (2 * (int64_t)g_noalloc_sms[device]) / col_blocks;
    if (S > K / 64) S = K / 64;
    const int64_t per_slice = (int64_t)MR * kGemvCols * sizeof(float);
    if (S * col_blocks * per_slice > (int64_t)kNoAllocPartialBytes) S = kNoAllocPartialBytes / (col_blocks * per_slice);
    if (S < 1) S = 1;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the last call left behind.  The counters must start at zero
    // (the partial sums need not: every slot that is read is written first).
    if (cudaMemsetAsync(counters, 0, kNoAllocCounterBytes, st) != cudaSuccess) return OPTIML_ERR_CUDA;
    dim3 grid((unsigned)col_blocks, (unsigned)S);
    if (MR == 1) launch_gemv_mr<1>(A, B, bias, Y, m, n, k, (int)act, grid, partials, counters, 0, st);
    else if (MR == 2) launch_gemv_mr<2>(A, B, bias, Y, m, n, k, (int)act, grid, partials, counters, 0, st);
    else launch_gemv_mr<4>(A, B, bias, Y, m, n, k, (int)act, grid, partials, counters, 0, st);
    return cudaGetLastError() == cudaSuccess ? OPTIML_OK : OPTIML_ERR_CUDA;
}

}  // extern "C"
