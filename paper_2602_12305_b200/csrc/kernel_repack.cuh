// Row re-pitching for bf16 matrices whose row length is not a multiple of 8 elements (16
// bytes): TMA cannot address such rows, so the tensor-core kernels cannot read or write them
// in place.  pad_rows copies a [rows][cols] matrix into a [rows_pad][cols_pad] one (cols_pad a
// multiple of 8), zero-filling the tail of every row and the rows past `rows`; unpad_rows copies
// the leading `cols` elements of the first `rows` padded rows back.  Both are plain streaming copies: one 16-byte store per thread, element loads on
// the side whose rows are not 16-byte aligned.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace optiml {

constexpr int kRepackThreads = 256;

__global__ void __launch_bounds__(kRepackThreads)
pad_rows_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int64_t rows, int64_t rows_pad, int64_t cols,
                int64_t cols_pad) {
    const int64_t groups = cols_pad / 8;                 // 16-byte groups per padded row
    const int64_t total = rows_pad * groups;
    for (int64_t i = (int64_t)blockIdx.x * kRepackThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kRepackThreads) {
        const int64_t r = i / groups, c0 = (i - r * groups) * 8;
        const uint16_t* s = src + r * cols + c0;
        uint16_t v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (r < rows && c0 + j < cols) ? s[j] : (uint16_t)0;
        uint4 o;
        o.x = v[0] | ((uint32_t)v[1] << 16);
        o.y = v[2] | ((uint32_t)v[3] << 16);
        o.z = v[4] | ((uint32_t)v[5] << 16);
        o.w = v[6] | ((uint32_t)v[7] << 16);
        *reinterpret_cast<uint4*>(dst + r * cols_pad + c0) = o;
    }
}

// dst is dense ([rows][cols], 16-byte aligned base), so it is written as a flat array in 16-byte
// pieces of 8 consecutive elements; a piece may run over the end of a row, so every element finds
// its own place in the padded source (2-byte loads of neighbouring addresses, served by L1).
__global__ void __launch_bounds__(kRepackThreads)
unpad_rows_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int64_t rows, int64_t cols, int64_t cols_pad) {
    const int64_t total = rows * cols;
    const int64_t pieces = (total + 7) / 8;
    for (int64_t i = (int64_t)blockIdx.x * kRepackThreads + threadIdx.x; i < pieces; i += (int64_t)gridDim.x * kRepackThreads) {
        const int64_t e0 = i * 8;
        int64_t r = e0 / cols, c = e0 - r * cols;
        uint16_t v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            v[j] = (e0 + j < total) ? src[r * cols_pad + c] : (uint16_t)0;
            if (++c == cols) { c = 0; ++r; }
        }
        if (e0 + 8 <= total) {
            uint4 o;
            o.x = v[0] | ((uint32_t)v[1] << 16);
            o.y = v[2] | ((uint32_t)v[3] << 16);
            o.z = v[4] | ((uint32_t)v[5] << 16);
            o.w = v[6] | ((uint32_t)v[7] << 16);
            *reinterpret_cast<uint4*>(dst + e0) = o;
        } else {
            for (int j = 0; e0 + j < total; ++j) dst[e0 + j] = v[j];
        }
    }
}

}  // namespace optiml
