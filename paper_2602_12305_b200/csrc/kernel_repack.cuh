// Row re-pitching for matrices whose row length is not a multiple of 16 bytes (8 bf16 or 4 fp32
// elements): TMA cannot address such rows and the 128-bit loads of the FMA tiles cannot either, so
// the fast kernels cannot read or write them in place.  pad_rows copies a [rows][cols] matrix into
// a [rows_pad][cols_pad] one (cols_pad a multiple of the vector width), zero-filling the tail of
// every row and the rows past `rows`; unpad_rows copies the leading `cols` elements of the first
// `rows` padded rows back.  Both are plain streaming copies: one 16-byte store per thread, element
// loads on the side whose rows are not 16-byte aligned.  E is a 2- or 4-byte unsigned integer
// standing for the element's bits.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace optiml {

constexpr int kRepackThreads = 256;

template <typename E>
struct RepackVec {
    static constexpr int V = 16 / (int)sizeof(E);     // elements per 16-byte piece
    E e[V];
};

template <typename E>
__global__ void __launch_bounds__(kRepackThreads)
pad_rows_kernel(const E* __restrict__ src, E* __restrict__ dst, int64_t rows, int64_t rows_pad, int64_t cols, int64_t cols_pad) {
    constexpr int V = RepackVec<E>::V;
    const int64_t groups = cols_pad / V;                 // 16-byte pieces per padded row
    const int64_t total = rows_pad * groups;
    for (int64_t i = (int64_t)blockIdx.x * kRepackThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kRepackThreads) {
        const int64_t r = i / groups, c0 = (i - r * groups) * V;
        const E* s = src + r * cols + c0;
        __align__(16) RepackVec<E> v;
#pragma unroll
        for (int j = 0; j < V; ++j) v.e[j] = (r < rows && c0 + j < cols) ? s[j] : (E)0;
        *reinterpret_cast<uint4*>(dst + r * cols_pad + c0) = *reinterpret_cast<const uint4*>(&v);
    }
}

// dst is dense ([rows][cols], 16-byte aligned base), so it is written as a flat array in 16-byte
// pieces of consecutive elements; a piece may run over the end of a row, so every element finds
// its own place in the padded source (element loads of neighbouring addresses, served by L1).
template <typename E>
__global__ void __launch_bounds__(kRepackThreads)
unpad_rows_kernel(const E* __restrict__ src, E* __restrict__ dst, int64_t rows, int64_t cols, int64_t cols_pad) {
    constexpr int V = RepackVec<E>::V;
    const int64_t total = rows * cols;
    const int64_t pieces = (total + V - 1) / V;
    for (int64_t i = (int64_t)blockIdx.x * kRepackThreads + threadIdx.x; i < pieces; i += (int64_t)gridDim.x * kRepackThreads) {
        const int64_t e0 = i * V;
        int64_t r = e0 / cols, c = e0 - r * cols;
        __align__(16) RepackVec<E> v;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            v.e[j] = (e0 + j < total) ? src[r * cols_pad + c] : (E)0;
            if (++c == cols) { c = 0; ++r; }
        }
        if (e0 + V <= total) {
            *reinterpret_cast<uint4*>(dst + e0) = *reinterpret_cast<const uint4*>(&v);
        } else {
            for (int j = 0; e0 + j < total; ++j) dst[e0 + j] = v.e[j];
        }
    }
}

}  // namespace optiml
