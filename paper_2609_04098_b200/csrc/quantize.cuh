// Bandwidth-bound kernels: per-tensor amax (calibration) and bf16 -> NVFP4
// quantization (E2M1 codes + one E4M3 scale per 16 elements).
//
// Work decomposition: one warp owns 256 consecutive elements of one row (one
// 128-bit load per lane, fully coalesced 512 bytes per warp).  Two neighbouring
// lanes hold one 16-element block, so the block maximum is one shuffle; eight
// lanes hold the four blocks whose scale bytes form one 32-bit word of the
// tensor-core scale layout.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/nvfp4.h"

namespace nvfp4 {

struct SegTable {
    int32_t nseg;                          // 0: a single global scale g[0]
    int32_t row_end[NVFP4_MAX_SEGMENTS];   // exclusive end row of each segment (ascending)
};

__device__ __forceinline__ int seg_of(const SegTable& t, int32_t row) {
    int s = 0;
    while (s + 1 < t.nseg && row >= t.row_end[s]) ++s;
    return s;
}

// float -> E4M3 byte, round-to-nearest-even, saturating to 448.
__device__ __forceinline__ uint32_t f32_to_e4m3(float v) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(v));
    return static_cast<uint32_t>(r) & 0xFFu;
}
// E4M3 byte -> float (exact).
__device__ __forceinline__ float e4m3_to_f32(uint32_t b) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(static_cast<uint16_t>(b)));
    return __half2float(__ushort_as_half(static_cast<unsigned short>(h2 & 0xFFFFu)));
}
// 8 floats -> 8 E2M1 codes (RNE, saturating to +/-6), element i in nibble i.
__device__ __forceinline__ uint32_t f32x8_to_e2m1(const float (&y)[8]) {
    uint32_t out;
    asm("{\n\t"
        ".reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t"
        "}\n"
        : "=r"(out)
        : "f"(y[0]), "f"(y[1]), "f"(y[2]), "f"(y[3]), "f"(y[4]), "f"(y[5]), "f"(y[6]), "f"(y[7]));
    return out;
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float (&f)[8]) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}

// Byte offset of scale (row r, block b) in the tensor-core layout; katoms = ceil(K/64).
__device__ __forceinline__ int64_t sf_mma_offset(int32_t r, int32_t b, int32_t katoms) {
    const int32_t rr = r & 127;
    return (static_cast<int64_t>(r >> 7) * katoms + (b >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (b & 3);
}

// One 8-element slice of a block: returns the packed codes, and the block's scale
// byte through s8_out.  The operation order is the contract the bit-exact
// comparison relies on (binary32, RNE, no fused multiply-add).
__device__ __forceinline__ uint32_t quantize_slice(const float (&f)[8], float g, float c1, uint32_t& s8_out) {
    float m = fmaxf(fmaxf(fmaxf(fabsf(f[0]), fabsf(f[1])), fmaxf(fabsf(f[2]), fabsf(f[3]))),
                    fmaxf(fmaxf(fabsf(f[4]), fabsf(f[5])), fmaxf(fabsf(f[6]), fabsf(f[7]))));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));          // the other half of the block
    const uint32_t s8 = f32_to_e4m3(__fmul_rn(m, c1));
    s8_out = s8;
    if (s8 == 0u) return 0u;
    const float d = __fmul_rn(e4m3_to_f32(s8), g);
    const float q = __fdiv_rn(1.0f, d);
    float y[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = __fmul_rn(f[i], q);
    return f32x8_to_e2m1(y);
}

template <bool MMA_LAYOUT, int UNROLL>
__global__ void __launch_bounds__(256)
quantize_kernel(const uint16_t* __restrict__ x, int32_t M, int32_t K, int64_t ld,
                const float* __restrict__ g_ptr, SegTable segs,
                uint8_t* __restrict__ codes, uint8_t* __restrict__ sf,
                int32_t chunks_per_row, int32_t total_items) {
    const int lane = threadIdx.x & 31;
    const int32_t warp_global = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int32_t nwarps = gridDim.x * (blockDim.x >> 5);
    const int32_t KB = K >> 4;
    const int32_t katoms = (KB + 3) >> 2;
    const float g_single = (segs.nseg == 0) ? __ldg(g_ptr) : 0.0f;

    for (int32_t base = warp_global; base < total_items; base += nwarps * UNROLL) {
        uint4 v[UNROLL];
        int32_t row[UNROLL], col[UNROLL];
        bool live[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int32_t item = base + u * nwarps;
            live[u] = item < total_items;                       // warp-uniform
            row[u] = live[u] ? item / chunks_per_row : 0;
            col[u] = live[u] ? (item - row[u] * chunks_per_row) * 256 + lane * 8 : K;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (col[u] < K)
                v[u] = __ldcs(reinterpret_cast<const uint4*>(x + static_cast<int64_t>(row[u]) * ld + col[u]));
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            if (!live[u]) continue;                             // whole warp skips together
            const float g = (segs.nseg == 0) ? g_single : __ldg(g_ptr + seg_of(segs, row[u]));
            const float c1 = __fdiv_rn(1.0f, __fmul_rn(6.0f, g));
            float f[8];
            bf16x8_to_f32(v[u], f);
            uint32_t s8;
            const uint32_t word = quantize_slice(f, g, c1, s8);
            const bool in_range = col[u] < K;
            if (!in_range) s8 = 0u;
            if (in_range)
                *reinterpret_cast<uint32_t*>(codes + static_cast<int64_t>(row[u]) * (K >> 1) + (col[u] >> 1)) = word;
            // scale bytes: the even lane of each pair holds the block's byte
            const int l0 = lane & ~7;
            const uint32_t w = __shfl_sync(0xffffffffu, s8, l0) | (__shfl_sync(0xffffffffu, s8, l0 + 2) << 8) |
                               (__shfl_sync(0xffffffffu, s8, l0 + 4) << 16) |
                               (__shfl_sync(0xffffffffu, s8, l0 + 6) << 24);
            const int32_t kb = col[u] >> 4;
            if (MMA_LAYOUT) {
                if ((lane & 7) == 0 && kb < KB)                 // blocks past K inside the word are zero
                    *reinterpret_cast<uint32_t*>(sf + sf_mma_offset(row[u], kb, katoms)) = w;
            } else {
                if ((lane & 1) == 0 && in_range) sf[static_cast<int64_t>(row[u]) * KB + kb] = static_cast<uint8_t>(s8);
            }
        }
    }
}

// ------------------------------------------------------------------ calibration
// max |x| as the bit pattern of a non-negative float (ordering of such patterns as
// unsigned integers equals their ordering as floats), accumulated with atomicMax.
__global__ void __launch_bounds__(256)
amax_kernel(const uint16_t* __restrict__ x, int32_t rows, int32_t cols, int64_t ld,
            int32_t chunks_per_row, int32_t total_items, uint32_t* __restrict__ amax_bits) {
    const int lane = threadIdx.x & 31;
    const int32_t warp_global = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int32_t nwarps = gridDim.x * (blockDim.x >> 5);
    uint32_t best = 0u;                                          // packed 2 x 15-bit magnitudes
    for (int32_t item = warp_global; item < total_items; item += nwarps) {
        const int32_t r = item / chunks_per_row;
        const int32_t c = (item - r * chunks_per_row) * 256 + lane * 8;
        if (c + 8 <= cols) {
            const uint4 v = __ldcs(reinterpret_cast<const uint4*>(x + static_cast<int64_t>(r) * ld + c));
            best = __vmaxu2(best, v.x & 0x7FFF7FFFu);
            best = __vmaxu2(best, v.y & 0x7FFF7FFFu);
            best = __vmaxu2(best, v.z & 0x7FFF7FFFu);
            best = __vmaxu2(best, v.w & 0x7FFF7FFFu);
        } else {
            for (int32_t k = c; k < cols; ++k) {
                const uint32_t b = x[static_cast<int64_t>(r) * ld + k] & 0x7FFFu;
                best = __vmaxu2(best, b);
            }
        }
    }
    uint32_t m = max(best & 0xFFFFu, best >> 16);
    m = __reduce_max_sync(0xffffffffu, m);
    __shared__ uint32_t smax[8];
    if (lane == 0) smax[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (blockDim.x >> 5); ++w) m = max(m, smax[w]);
        if (m != 0u) atomicMax(amax_bits, m << 16);
    }
}

// generic fallback for unaligned pointers / leading dimensions
__global__ void __launch_bounds__(256)
amax_scalar_kernel(const uint16_t* __restrict__ x, int64_t rows, int64_t cols, int64_t ld,
                   uint32_t* __restrict__ amax_bits) {
    uint32_t m = 0u;
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / cols, c = i - r * cols;
        m = max(m, static_cast<uint32_t>(x[r * ld + c] & 0x7FFFu));
    }
    m = __reduce_max_sync(0xffffffffu, m);
    if ((threadIdx.x & 31) == 0 && m != 0u) atomicMax(amax_bits, m << 16);
}

// g = amax / 2688 (binary32 divide), 1 for an all-zero tensor; in place on the
// accumulator word.
__global__ void finalize_scale_kernel(float* __restrict__ g_inout, float* __restrict__ amax_out) {
    const float amax = *g_inout;
    if (amax_out != nullptr) *amax_out = amax;
    *g_inout = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, 2688.0f);
}

}  // namespace nvfp4
