// Shared device helpers: the fused epilogue (bias add, activation, one rounding) and
// element load/convert routines used by every kernel variant.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace optiml {

enum : int { kActNone = 0, kActRelu = 1, kActGeluTanh = 2, kActSigmoid = 3 };

// Device status word values (written by kernels that give up a bounded wait).
enum : int { kDevOk = 0, kDevTimeout = 7 };

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// GELU, tanh form: 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))).
// kFast selects the hardware tanh approximation (relative error about 2^-11), used
// where the output is rounded to bf16 anyway; the fp32 path keeps tanhf.
template <bool kFast>
__device__ __forceinline__ float gelu_tanh(float x) {
    const float c = 0.7978845608028654f;
    float u = c * fmaf(0.044715f * x * x, x, x);
    float t;
    if (kFast) {
        asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
    } else {
        t = tanhf(u);
    }
    return 0.5f * x * (1.0f + t);
}

// sigmoid(x) = 1 / (1 + exp(-x)); kFast uses the hardware exponential and reciprocal.
template <bool kFast>
__device__ __forceinline__ float sigmoid(float x) {
    if (kFast) return __fdividef(1.0f, 1.0f + __expf(-x));
    return 1.0f / (1.0f + expf(-x));
}

// act(acc + bias) in fp32.  ReLU maps -0 and negatives to +0.
template <int kAct, bool kFast>
__device__ __forceinline__ float epilogue(float acc, float bias) {
    float x = acc + bias;
    if (kAct == kActRelu) return x > 0.0f ? x : 0.0f;
    if (kAct == kActGeluTanh) return gelu_tanh<kFast>(x);
    if (kAct == kActSigmoid) return sigmoid<kFast>(x);
    return x;
}

// Runtime-act version for kernels where the epilogue is a negligible share of the work.
template <bool kFast>
__device__ __forceinline__ float epilogue_rt(float acc, float bias, int act) {
    float x = acc + bias;
    if (act == kActRelu) return x > 0.0f ? x : 0.0f;
    if (act == kActGeluTanh) return gelu_tanh<kFast>(x);
    if (act == kActSigmoid) return sigmoid<kFast>(x);
    return x;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
    return *reinterpret_cast<uint32_t*>(&v);
}

// Exact widening of two packed bf16 values.
__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// 128-bit streaming load that does not allocate in L1 (data read exactly once).
__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Record a bounded wait that gave up: low byte = status, next byte = which wait (1 producer
// waiting for a free stage, 2 MMA waiting for a free accumulator, 3 MMA waiting for the A
// tile, 4 MMA waiting for a filled stage, 5 epilogue waiting for an accumulator; 6 is not a wait:
// the dynamic shared memory of a streaming kernel did not start on a 1024-byte boundary), upper
// half = CTA index.  The first report wins.
__device__ __forceinline__ void report_timeout(int* status, int site) {
    atomicCAS(status, kDevOk, kDevTimeout | (site << 8) | ((int)(blockIdx.x & 0x7FFF) << 16));
}

__host__ __device__ __forceinline__ int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

}  // namespace optiml
