/*
 * optiml.h -- C ABI of the fused GEMM + bias + activation library for NVIDIA B200
 * (sm_100a):
 *
 *     Y = act(A . B + bias)
 *
 * The contraction is the matrix product of the paper's Prompts appendix, task 2
 * ("Matrix Multiplication": A is M x K, B is K x N, C = A x B is M x N), stored as
 * in its matmul case study, "Common setup": every matrix dense and row-major,
 * element (r, c) of an R x C matrix at index r*C + c, so A[m*K + k], B[k*N + n],
 * Y[m*N + n].  act = ReLU is max(0, x) as in the Prompts appendix, task 10.  The
 * length-N bias (added to every row) and the tanh form of GELU,
 *     GELU(x) = 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))),
 * have no counterpart in the paper; they are this library's problem statement.
 *
 * Arithmetic.  OPTIML_F32: fp32 inputs, fp32 products and sums on the plain FMA
 * pipes (no TF32, no split-precision tensor-core emulation), fp32 output.
 * OPTIML_BF16: bf16 inputs, exact products, fp32 accumulation, bias widened to
 * fp32, activation in fp32, one round-to-nearest-even to bf16 at the store.
 * The summation order over k is unspecified but fixed for a given shape, device
 * and variant: the same call gives the same bits every time.
 *
 * Threading / streams.  A handle is not thread-safe and serialises its own
 * scratch memory in stream order: use one handle per stream.  Calls enqueue
 * work on `stream` and return without synchronising unless stated otherwise.
 *
 * Errors are return codes; nothing aborts, traps or throws.
 */
#ifndef OPTIML_H_
#define OPTIML_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct optiml_handle_s* optiml_handle_t;

typedef enum {
    OPTIML_OK = 0,
    OPTIML_ERR_INVALID_ARG = 1, /* null pointer, non-positive dimension, bad enum         */
    OPTIML_ERR_UNSUPPORTED = 2, /* forced variant cannot run this shape / dtype           */
    OPTIML_ERR_ALIGNMENT = 3,   /* a device pointer is not aligned to its element size    */
    OPTIML_ERR_ARCH = 4,        /* device is not compute capability 10.0                  */
    OPTIML_ERR_ALLOC = 5,       /* device or host allocation failed                       */
    OPTIML_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed                    */
    OPTIML_ERR_TIMEOUT = 7      /* a bounded on-device wait gave up (see get_last_status) */
} optiml_status_t;

typedef enum { OPTIML_F32 = 0, OPTIML_BF16 = 1 } optiml_dtype_t;

typedef enum {
    OPTIML_ACT_NONE = 0,
    OPTIML_ACT_RELU = 1,      /* max(0, x): Prompts appendix, task 10 */
    OPTIML_ACT_GELU_TANH = 2, /* tanh form, see the top of this header */
    OPTIML_ACT_SIGMOID = 3    /* 1 / (1 + exp(-x)): Prompts appendix, task 1 */
} optiml_act_t;

/* Kernel variants the shape-based dispatcher chooses between. */
typedef enum {
    OPTIML_VARIANT_AUTO = -1,
    OPTIML_VARIANT_GENERIC = 0,     /* predicated FMA tiles: any shape, any alignment, both dtypes      */
    OPTIML_VARIANT_F32_TILED = 1,   /* fp32 FMA tiles, 128-bit loads: needs N % 4 == 0 and K % 4 == 0    */
    OPTIML_VARIANT_GEMV_SPLITK = 2, /* M <= 4: split-K streaming, 128-bit loads; N % 8 (bf16) / 4 (fp32) */
    OPTIML_VARIANT_SKINNY_UMMA = 3, /* bf16, M <= 128: stream-K over B with tcgen05 (N is the MMA M dim) */
    OPTIML_VARIANT_UMMA = 4,        /* bf16: persistent TMA + tcgen05 + TMEM tiles, N % 8 == K % 8 == 0  */
    OPTIML_VARIANT_UMMA_2CTA = 5,   /* bf16: the same with CTA pairs (tcgen05 cta_group::2, 256 x 256 tiles) */
    OPTIML_VARIANT_UMMA_2CTA_STREAM = 6, /* bf16, fewer tiles than CTA pairs: one cluster of 2, 4 or 8 CTAs per tile
                                            (256 x 256; 128 x 256 with 64 rows per CTA for M <= 128), K cut across
                                            its CTA pairs, partial sums exchanged through distributed shared memory */
    OPTIML_VARIANT_COUNT = 7
} optiml_variant_t;

/*
 * Create a handle on CUDA device `device` (host call).  Checks that the device is
 * compute capability 10.0 (else OPTIML_ERR_ARCH), and allocates the handle's
 * device scratch: split-K partial sums, arrival counters and a status word, about
 * 40 MiB.  The calling thread's current device is left unchanged.
 */
optiml_status_t optiml_create(optiml_handle_t* out, int device);

/* Free the handle and its scratch.  Synchronises the device first.  NULL is OK. */
optiml_status_t optiml_destroy(optiml_handle_t h);

/*
 * Y = act(A . B + bias), enqueued on `stream` (a cudaStream_t; NULL = default
 * stream).  Definition: header comment above (Prompts appendix task 2 and task 10;
 * matmul case study, "Common setup").
 *
 *   A     device, M*K elements of dtype, row-major          read only
 *   B     device, K*N elements of dtype, row-major          read only
 *   bias  device, N elements of dtype, or NULL for zeros    read only
 *   Y     device, M*N elements of dtype, row-major          written once; must not
 *         overlap A, B or bias
 *   M, N, K  >= 1, each <= 2^31 - 1
 *
 * All four buffers stay owned by the caller and must stay valid until the work
 * has run; the library keeps no reference after that.  Pointers must be aligned
 * to the element size; the fast variants also need 16-byte aligned pointers and
 * N, K multiples of 8 (bf16) or 4 (fp32) -- other shapes run on the generic
 * variant, never on the CPU.  One exception: a large problem (M >= 16, M N K >= 2^27)
 * with 16-byte aligned pointers whose N or K is not a multiple of 8 (bf16) or 4 (fp32) is copied into
 * zero-padded buffers with 16-byte row pitches (A if K is ragged, B always, Y on the way
 * back if N is ragged) and runs on the fast variants; those buffers belong to the handle
 * and grow on demand, which synchronises `stream` and allocates on the first such call and
 * whenever a larger problem arrives (OPTIML_ERR_ALLOC if that fails; the handle stays
 * usable).  Inputs must be finite.  Scratch use is serialised on `stream`; do not use one
 * handle on two streams at once.
 *
 * Returns OPTIML_OK once the work is enqueued; INVALID_ARG / ALIGNMENT before
 * anything is launched; CUDA if a launch failed.  A bounded on-device wait that
 * gave up is reported by optiml_get_last_status after synchronisation.
 */
optiml_status_t optiml_gemm_epilogue(optiml_handle_t h, const void* A, const void* B, const void* bias, void* Y,
                                     int64_t M, int64_t N, int64_t K, optiml_dtype_t dtype, optiml_act_t act,
                                     void* stream);

/*
 * Same operation with HOST buffers (same shapes and dtype as above): copies A, B
 * and bias to device staging memory owned by the handle (grown on demand, which
 * allocates), runs optiml_gemm_epilogue on `stream`, copies Y back and
 * synchronises `stream` before returning.  Pinned host memory makes the copies
 * asynchronous with respect to the host until that final synchronisation.
 */
optiml_status_t optiml_gemm_epilogue_host(optiml_handle_t h, const void* A_host, const void* B_host,
                                          const void* bias_host, void* Y_host, int64_t M, int64_t N, int64_t K,
                                          optiml_dtype_t dtype, optiml_act_t act, void* stream);

/*
 * Y = act(A . B + bias) for bf16 GEMV-like problems, for callers that must not allocate.
 * (The paper has no counterpart of this entry point; the operation is the one defined at
 * the top of this header.)
 *
 * Who needs it: code that runs where cudaMalloc is off the table -- a process whose
 * device memory has been handed in full to another allocator (an inference server's
 * arena, a framework's caching allocator) so that a fresh cudaMalloc fails, or a
 * latency-critical loop that cannot afford the device-wide synchronisation an allocation
 * may imply.  Such callers cannot create a handle either, because optiml_create
 * allocates the handle's scratch.  This call takes no handle and calls no cudaMalloc,
 * cudaFree or other allocating routine; the split-K scratch it needs (arrival counters
 * and partial sums, 2 MiB + 1 KiB) is a fixed array inside the library image, which every
 * GPU that loads the library holds until the process exits.
 *
 *   A, B, bias, Y   device pointers as for optiml_gemm_epilogue, dtype bf16, 16-byte
 *                   aligned; bias may be NULL; the caller owns all four
 *   M               1..4
 *   N               multiple of 8, at most 65536 (the fixed scratch covers no more)
 *   K               >= 1
 *   device          CUDA device that owns the pointers and `stream`
 *   stream          cudaStream_t (NULL = default stream); work is enqueued, not awaited
 *
 * Returns OPTIML_ERR_UNSUPPORTED for M > 4, N > 65536 or N % 8 != 0 (nothing is
 * launched), ALIGNMENT for pointers that are not 16-byte aligned, ARCH on a device that
 * is not compute capability 10.0, INVALID_ARG for a device index the process does not
 * have (and as elsewhere), CUDA if a runtime call failed.
 *
 * The first call on each device looks up the scratch array's device address and the SM
 * count (host-side queries only) and keeps them for later calls; that first call
 * should come before any stream capture.  Every call on a device shares the one array, which still
 * holds what the previous call left: each call re-zeroes the counters on `stream` before
 * its kernel.  Two calls whose work overlaps on the GPU (different streams, or different
 * host threads) therefore race on the scratch and give undefined results -- keep calls on
 * one device in a single stream order.  Not thread-safe on first use per device.
 */
optiml_status_t optiml_gemv_noalloc(const void* A, const void* B, const void* bias, void* Y, int64_t M, int64_t N,
                                    int64_t K, optiml_act_t act, int device, void* stream);

/*
 * Read the device-written status word (synchronises the device): OPTIML_OK, or
 * OPTIML_ERR_TIMEOUT if any kernel of this handle gave up a bounded wait since the
 * last call of this function; the word is cleared.  A call that reported a
 * time-out has left Y undefined.
 */
optiml_status_t optiml_get_last_status(optiml_handle_t h);

/*
 * Self-test of the failure path (host call, enqueues one tiny kernel on `stream`).  The paper
 * prunes a candidate kernel that fails to run (Section 3.2, "Execution gate"); the counterpart
 * here is that a kernel which gives up a bounded wait must REPORT it.  One CTA waits with the
 * library's bounded wait, limited to `limit_cycles` SM cycles (1 .. 2e9), on a barrier that
 * nobody signals, records the time-out in the handle's status word like every compute kernel
 * would, and returns normally: no trap, no fault, the context stays usable.  Afterwards
 * optiml_get_last_status returns OPTIML_ERR_TIMEOUT once (wait site 7 in the log), then OK.
 * Returns INVALID_ARG for a NULL handle or a limit outside the range.
 */
optiml_status_t optiml_selftest_timeout(optiml_handle_t h, int64_t limit_cycles, void* stream);

/*
 * Failure injection for the library's own device allocations (host call; process-wide, not
 * thread-safe; no counterpart in the paper).  While a hook is set, every allocation the library
 * is about to make (handle scratch in optiml_create, staging buffers of
 * optiml_gemm_epilogue_host) first calls hook(bytes, user); a non-zero return makes that
 * allocation fail as if the device were out of memory, so the caller sees OPTIML_ERR_ALLOC.
 * NULL removes the hook.  optiml_create frees whatever it had allocated before the failure;
 * optiml_gemm_epilogue_host leaves the handle usable (the buffer that failed to grow is empty
 * and is allocated again by the next call).
 */
typedef int (*optiml_alloc_hook_t)(size_t bytes, void* user);
optiml_status_t optiml_set_alloc_hook(optiml_alloc_hook_t hook, void* user);

/*
 * The K reduction on its own, over fp32 vectors of n elements (paper: Prompts appendix,
 * task 14 "Reduction": the sum of all elements; task 15 "Dot Product": sum_i x_i * y_i;
 * task 7 "Mean Square Error": (1/n) sum_i (x_i - y_i)^2 with x the predictions and y the
 * targets):
 *
 *   OPTIML_REDUCE_SUM   *out = sum_i x[i]                       (y is ignored, may be NULL)
 *   OPTIML_REDUCE_DOT   *out = sum_i x[i] * y[i]
 *   OPTIML_REDUCE_MSE   *out = (1/n) sum_i (x[i] - y[i])^2
 *
 * x, y: device, n fp32 elements, 16-byte aligned, read only, owned by the caller.  out:
 * device, one fp32, written once.  n >= 1.  One pass over the data; terms are accumulated
 * in fp32 in many short chains and combined in fp64, in a fixed order.  Enqueued on
 * `stream`; uses the handle's scratch like the other calls.  Returns INVALID_ARG /
 * ALIGNMENT before anything is launched, CUDA if the launch failed.
 */
typedef enum { OPTIML_REDUCE_SUM = 0, OPTIML_REDUCE_DOT = 1, OPTIML_REDUCE_MSE = 2 } optiml_reduce_t;
optiml_status_t optiml_reduce_f32(optiml_handle_t h, optiml_reduce_t kind, const float* x, const float* y, int64_t n,
                                  float* out, void* stream);

/*
 * Multi-head self-attention (paper: Prompts appendix, task 6).  Q, K, V and Y are N x d_model,
 * dense row-major; with d_k = d_model / heads, head i owns columns [i d_k, (i+1) d_k) of each:
 *
 *   head_i = softmax(Q_i K_i^T / sqrt(d_k)) V_i     softmax over the keys, row by row
 *   Y      = Concat(head_1, ..., head_h)             head i written back to its own columns
 *
 * No mask, no projection.  Q, K, V: device, N * d_model elements of dtype, read only.  Y: device,
 * N * d_model elements of dtype, written once, must not overlap the inputs.  N >= 1, d_model a
 * multiple of heads.  The caller owns all four buffers; they must stay valid until the work has
 * run.  Inputs must be finite.
 *
 * Arithmetic.  OPTIML_BF16 with d_k = 64 or 128, 16-byte aligned pointers and d_model % 8 == 0
 * runs on the tensor cores: exact bf16 products, fp32 accumulation, softmax in fp32 with
 * exp2 on the special-function unit, probabilities rounded to bf16 before they multiply V,
 * their sum kept unrounded in fp32, one rounding of the quotient to bf16 at the store.  Any other
 * d_k <= 256, unaligned pointers and OPTIML_F32 run on a plain FMA kernel (fp32 throughout; bf16
 * rounded once at the store).  d_k > 256 returns OPTIML_ERR_UNSUPPORTED.  A forced
 * OPTIML_VARIANT_GENERIC (optiml_force_variant) selects the FMA kernel; any other forced variant
 * demands the tensor-core kernel and returns UNSUPPORTED where it cannot run; a forced
 * OPTIML_VARIANT_UMMA_2CTA selects, at d_k = 128, the form in which a pair of CTAs shares every
 * K and V block (same arithmetic, same tolerance).
 *
 * Enqueued on `stream`; INVALID_ARG / ALIGNMENT / UNSUPPORTED before anything is launched, CUDA if
 * the launch failed; a device-side time-out is reported by optiml_get_last_status.
 */
optiml_status_t optiml_mhsa(optiml_handle_t h, const void* Q, const void* K, const void* V, void* Y, int64_t N,
                            int64_t d_model, int64_t heads, optiml_dtype_t dtype, void* stream);

/* Force one variant for later calls (tests, profiling), or OPTIML_VARIANT_AUTO to
 * give the choice back to the dispatcher.  A forced variant that cannot run a
 * shape makes optiml_gemm_epilogue return OPTIML_ERR_UNSUPPORTED. */
optiml_status_t optiml_force_variant(optiml_handle_t h, optiml_variant_t v);

/* Variant the dispatcher would run for this problem (honours a forced variant;
 * pointers are assumed 16-byte aligned), or -1 on bad arguments.  A large unaligned
 * shape that optiml_gemm_epilogue re-pitches is reported as OPTIML_VARIANT_GENERIC here;
 * ask with N and K rounded up to the vector width for the variant its padded copy runs on. */
int optiml_select_variant(optiml_handle_t h, int64_t M, int64_t N, int64_t K, optiml_dtype_t dtype);

/*
 * Tuning options of the streaming kernels (the GEMV-like and skinny shapes, which are bound
 * by HBM bandwidth, not by arithmetic).  They change how the stream over B is scheduled.  The
 * prefetch, ring and trigger options never change a result bit; SKINNY_STAGE_ROWS moves the
 * places where K is cut when a problem is split along K, so partial sums may then round
 * differently (still one fixed order per setting).  The defaults come from
 * sweeps on B200; optiml_set_option overrides one for later calls on this handle (values
 * 0 .. 2^20, else INVALID_ARG), optiml_get_option reads it back (-1 on bad arguments).
 *
 * Prefetching "ahead of the dependency wait": kernels are launched as programmatic
 * dependents, so a kernel's CTAs may start while the previous kernel in the stream still
 * drains.  They may not read or write anything before that kernel has finished, but they
 * may ask for lines of B to be brought from DRAM into L2: L2 is where this GPU's own writes
 * land, so a prefetch that overtakes a writer cannot make a later load see stale data.
 */
typedef enum {
    OPTIML_OPT_GEMV_PREFETCH_ROWS = 0,    /* GEMV: rows of its K slice each CTA prefetches into L2 before the wait */
    OPTIML_OPT_SKINNY_STAGE_ROWS = 1,     /* skinny: rows of K per pipeline stage, 128 or 192 (192: M <= 32 only)  */
    OPTIML_OPT_SKINNY_RING_STAGES = 2,    /* skinny: depth of the shared-memory ring of B tiles; 0 = the tuned depth */
    OPTIML_OPT_SKINNY_PREFETCH_EARLY = 3, /* skinny: ring stages of B prefetched into L2 before the wait            */
    OPTIML_OPT_SKINNY_LATE_TRIGGER = 4,   /* skinny: 1 = release the next kernel's CTAs after a CTA's last load,
                                             0 = as soon as the kernel starts                                       */
    OPTIML_OPT_PAIR_SPLIT_MAX = 5,        /* CTA-pair GEMMs: most K slices a tile is cut into (persistent form: tiles of
                                             the last, partial round, up to 8; streaming form: 1, 2 or 4)          */
    OPTIML_OPT_PAIR_HALF_HEIGHT = 6,      /* streaming CTA-pair form, M <= 128: 1 = 128-row tiles, 64 rows per CTA
                                             (default), 0 = 256-row tiles as for larger M                            */
    OPTIML_OPT_PAIR_TILE_WIDTH = 7,       /* streaming CTA-pair form: 0 = tile width chosen per shape (default),
                                             128 or 256 = that width                                                 */
    OPTIML_OPT_COUNT = 8
} optiml_option_t;
optiml_status_t optiml_set_option(optiml_handle_t h, optiml_option_t opt, int64_t value);
int64_t optiml_get_option(optiml_handle_t h, optiml_option_t opt);

/* Number of kernels launched by this handle since it was created. */
int64_t optiml_launch_count(optiml_handle_t h);

/* Static strings; never NULL. */
const char* optiml_status_string(optiml_status_t s);
const char* optiml_variant_name(int variant);

/* Library version, major*10000 + minor*100 + patch. */
int optiml_version(void);

#ifdef __cplusplus
}
#endif
#endif /* OPTIML_H_ */
