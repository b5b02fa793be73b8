// Bandwidth-bound kernels: per-tensor amax (calibration) and bf16 -> NVFP4
// quantization (E2M1 codes + one E4M3 scale per 16 elements).
//
// Work decomposition: one lane owns one 16-element block (a 256-bit load; a warp reads
// 1024 contiguous bytes), so the block maximum needs no shuffle and there is one reciprocal
// per 16 elements; four neighbouring lanes hold the four scale bytes that form one 32-bit
// word of the tensor-core scale layout.  The kernel is issue-bound before it is
// bandwidth-bound, so the instruction count per element is what was optimised: packed
// bf16 maximum, no per-item division, per-row constants hoisted.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/nvfp4.h"
#include "ptx.cuh"

namespace nvfp4 {

struct SegTable {
    int32_t nseg;                          // 0: a single global scale g[0]
    int32_t row_end[NVFP4_MAX_SEGMENTS];   // exclusive end row of each segment (ascending)
    int32_t il_inner;                      // > 0: the tensor is [gate rows 0..inner) | up rows 0..inner)] and is written
                                           // with its rows interleaved 16 by 16 (see il_row)
};

// Output row of input row r when gate and up rows are interleaved in groups of 16: output rows
// 32 b .. 32 b + 15 are gate rows 16 b .. 16 b + 15, rows 32 b + 16 .. 32 b + 31 the matching up rows.
// A GEMM against weights in this order produces, per 32 output columns, the 16 gate and the 16 up
// values of one 16-element block of h = silu(gate) * up.
__device__ __forceinline__ int32_t il_row(int32_t r, int32_t inner) {
    const int32_t up = r >= inner ? 1 : 0;
    const int32_t q = r - up * inner;
    return (q >> 4) * 32 + up * 16 + (q & 15);
}

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

// Byte offset of scale (row r, block b) in the tensor-core layout; katoms = ceil(K/64).
__device__ __forceinline__ int64_t sf_mma_offset(int32_t r, int32_t b, int32_t katoms) {
    const int32_t rr = r & 127;
    return (static_cast<int64_t>(r >> 7) * katoms + (b >> 2)) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (b & 3);
}

// 256-bit streaming load: one 16-element block (32 bytes of bf16) per lane, never reused
__device__ __forceinline__ void ldg256_stream(const void* p, uint32_t (&v)[8]) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "l"(p));
}

// per 16-bit half: magnitude = max(|a|, |b|) (the sign bit of the result is sign(a) xor sign(b)
// and is masked off by the caller)
// 256-bit load that may stay in L1/L2 (data that is read again shortly)
__device__ __forceinline__ void ldg256_cached(const void* p, uint32_t (&v)[8]) {
    asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "l"(p));
}

__device__ __forceinline__ void stg256(void* p, const uint32_t (&v)[8]) {
    asm volatile("st.global.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                 ::"r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "l"(p)
                 : "memory");
}

// Two binary32 multiplies (or fused multiply-adds) in one instruction: each half is rounded to nearest
// even exactly like the scalar instruction, so results are bit-identical and the issue slots halve.
__device__ __forceinline__ void mul_f32x2(float& a0, float& a1, float b0, float b1) {
    asm("{\n\t"
        ".reg .b64 ra, rb;\n\t"
        "mov.b64 ra, {%0, %1};\n\t"
        "mov.b64 rb, {%2, %3};\n\t"
        "mul.rn.f32x2 ra, ra, rb;\n\t"
        "mov.b64 {%0, %1}, ra;\n\t"
        "}\n"
        : "+f"(a0), "+f"(a1)
        : "f"(b0), "f"(b1));
}
// (acc0, acc1) += (a0 * a0, a1 * a1), fused
__device__ __forceinline__ void fma_sq_f32x2(float& acc0, float& acc1, float a0, float a1) {
    asm("{\n\t"
        ".reg .b64 ra, rc;\n\t"
        "mov.b64 ra, {%2, %3};\n\t"
        "mov.b64 rc, {%0, %1};\n\t"
        "fma.rn.f32x2 rc, ra, ra, rc;\n\t"
        "mov.b64 {%0, %1}, rc;\n\t"
        "}\n"
        : "+f"(acc0), "+f"(acc1)
        : "f"(a0), "f"(a1));
}

__device__ __forceinline__ uint32_t bf16x2_absmax(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// One 16-element block held by one lane: returns the 16 packed codes (element i in nibble i)
// and the block's scale byte.  The operation order is the contract the bit-exact comparison
// relies on (binary32, round-to-nearest-even, no fused multiply-add):
//     s8 = e4m3(bmax * c1),  c1 = 1 / (6 g);   code = e2m1(x * (1 / (e4m3(s8) * g)))
__device__ __forceinline__ uint2 quantize_block(const uint32_t (&v)[8], float g, float c1, uint32_t& s8_out) {
    // block maximum on packed bf16 pairs (|x| is a bit mask; the maximum of bf16 values is exact)
    uint32_t m = bf16x2_absmax(bf16x2_absmax(v[0], v[1]), bf16x2_absmax(v[2], v[3]));
    const uint32_t m2 = bf16x2_absmax(bf16x2_absmax(v[4], v[5]), bf16x2_absmax(v[6], v[7]));
    m = bf16x2_absmax(m, m2) & 0x7FFF7FFFu;
    const float bmax = fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
    const uint32_t s8 = f32_to_e4m3(__fmul_rn(bmax, c1));
    s8_out = s8;
    const float d = __fmul_rn(e4m3_to_f32(s8), g);
    const float q = __frcp_rn(d);                             // the correctly rounded 1 / d (s8 == 0 gives inf; that block is zeroed below)
    uint2 out;
    {
        float y[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            y[2 * i] = __uint_as_float(v[i] << 16);
            y[2 * i + 1] = __uint_as_float(v[i] & 0xFFFF0000u);
            mul_f32x2(y[2 * i], y[2 * i + 1], q, q);
        }
        out.x = f32x8_to_e2m1(y);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            y[2 * i] = __uint_as_float(v[4 + i] << 16);
            y[2 * i + 1] = __uint_as_float(v[4 + i] & 0xFFFF0000u);
            mul_f32x2(y[2 * i], y[2 * i + 1], q, q);
        }
        out.y = f32x8_to_e2m1(y);
    }
    if (s8 == 0u) out = make_uint2(0u, 0u);                   // scale rounds to zero: codes 0, signs cleared
    return out;
}

// silu(g) * u = g / (1 + exp(-g)) * u in binary32 with the hardware's approximate exp2 and
// reciprocal (2 MUFU + 4 arithmetic instructions per element).  The relative error before the
// bf16 rounding is a few 2^-22 (the exponent's rounding adds |g| * 2^-24 * ln 2 for large |g|),
// so the rounded result equals the correctly rounded definition except in about one case in
// 10^4 and is never more than one bf16 ulp away -- down to magnitudes of about 2^-100: for
// g < -88 exp2 overflows to +inf and the result is a zero of the right sign where the definition
// gives |g| e^g |u| < 1e-36 |u| (no NVFP4 block can hold such a value next to anything else; the
// sign, which the codes keep, is right).  For g > 126 exp2 flushes to 0 and the result is g * u.
__device__ __forceinline__ float silu_mul(float g, float u) {
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(__fmul_rn(g, -1.44269504088896341f)));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(__fadd_rn(1.0f, e)));
    return __fmul_rn(__fmul_rn(g, r), u);
}

// The same for two elements at once: the three multiplies and the add are issued as two-wide binary32
// instructions (each half rounded exactly like the scalar form: the results are bit-identical).
__device__ __forceinline__ void add_f32x2(float& a0, float& a1, float b0, float b1) {
    asm("{\n\t"
        ".reg .b64 ra, rb;\n\t"
        "mov.b64 ra, {%0, %1};\n\t"
        "mov.b64 rb, {%2, %3};\n\t"
        "add.rn.f32x2 ra, ra, rb;\n\t"
        "mov.b64 {%0, %1}, ra;\n\t"
        "}\n"
        : "+f"(a0), "+f"(a1)
        : "f"(b0), "f"(b1));
}
__device__ __forceinline__ void silu_mul2(float g0, float g1, float u0, float u1, float& h0, float& h1) {
    float t0 = g0, t1 = g1, e0, e1, r0, r1;
    mul_f32x2(t0, t1, -1.44269504088896341f, -1.44269504088896341f);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(t0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(t1));
    add_f32x2(e0, e1, 1.0f, 1.0f);
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(e0));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(e1));
    h0 = g0;
    h1 = g1;
    mul_f32x2(h0, h1, r0, r1);
    mul_f32x2(h0, h1, u0, u1);
}

// 16 gate values and 16 up values (packed bf16) -> 16 values of bf16(silu(gate) * up), packed
__device__ __forceinline__ void swiglu_block(const uint32_t (&g)[8], const uint32_t (&u)[8], uint32_t (&h)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo, hi;
        silu_mul2(__uint_as_float(g[i] << 16), __uint_as_float(g[i] & 0xFFFF0000u), __uint_as_float(u[i] << 16),
                  __uint_as_float(u[i] & 0xFFFF0000u), lo, hi);
        __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
        h[i] = *reinterpret_cast<uint32_t*>(&b2);
    }
}

// 16 values x and 16 weights w (packed bf16) -> bf16((x * rstd) * w), packed
__device__ __forceinline__ void rmsnorm_block(const uint32_t (&x)[8], const uint32_t (&w)[8], float rstd, uint32_t (&y)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo = __uint_as_float(x[i] << 16), hi = __uint_as_float(x[i] & 0xFFFF0000u);
        mul_f32x2(lo, hi, rstd, rstd);
        mul_f32x2(lo, hi, __uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
        __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
        y[i] = *reinterpret_cast<uint32_t*>(&b2);
    }
}

constexpr int kQuantPlain = 0, kQuantSwiglu = 1, kQuantRmsnorm = 2;

// A warp owns `chunks_per_unit` consecutive 512-element chunks of one row (a "unit"); units are
// dealt round-robin to a persistent grid.
// MODE kQuantSwiglu: x is [M, 2K] (gate | up) and the tensor that is quantized is
// bf16(silu(gate) * up), [M, K].  MODE kQuantRmsnorm: the quantized tensor is
// bf16(x * rstd(row) * aux[k]) with rstd = 1 / sqrt(mean(x^2) + eps); a unit is then a whole row
// (units_per_row == 1): the warp first sums the squares of its row and reads the row a second
// time, from cache, to normalise and quantize it.  (Rows of up to 20480 elements take
// rmsnorm_quantize_kernel below, which keeps the row in registers; this is the general form.)
template <bool MMA_LAYOUT, int UNROLL, int MODE>
__global__ void __launch_bounds__(256, MODE == kQuantPlain ? 5 : 4)
quantize_kernel(const uint16_t* __restrict__ x, int32_t M, int32_t K, int64_t ld,
                const float* __restrict__ g_ptr, SegTable segs, const uint16_t* __restrict__ aux, float eps,
                uint8_t* __restrict__ codes, uint8_t* __restrict__ sf, uint16_t* __restrict__ h_out,
                int32_t chunks_per_row, int32_t chunks_per_unit, int32_t units_per_row, int32_t total_units) {
    // the kernel behind this one (the GEMM that consumes this tensor, or the next quantizer) may start
    // its prologue now; it waits for this kernel's completion before it reads anything
    ptx::pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int32_t warp_global = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int32_t nwarps = gridDim.x * (blockDim.x >> 5);
    const int32_t KB = K >> 4;
    const int32_t katoms = (KB + 3) >> 2;
    // this kernel itself may have been started early: everything it reads (the tensor, the global scale)
    // may come from the kernel in front of it
    ptx::pdl_wait();
    const float g_single = (segs.nseg == 0) ? __ldg(g_ptr) : 0.0f;
    const float c1_single = __fdiv_rn(1.0f, __fmul_rn(6.0f, g_single));

    // (row, part) of this warp's unit, advanced without a division per unit
    int32_t row = warp_global / units_per_row, part = warp_global - row * units_per_row;
    const int32_t d_row = nwarps / units_per_row, d_part = nwarps - d_row * units_per_row;
    for (int32_t unit = warp_global; unit < total_units; unit += nwarps, row += d_row, part += d_part) {
        if (part >= units_per_row) { part -= units_per_row; ++row; }
        const int32_t c_begin = part * chunks_per_unit;
        const int32_t c_end = min(chunks_per_row, c_begin + chunks_per_unit);
        if (row >= M) {
            // tensor-core layout only: rows that pad the last 128-row band get zero scales
            if (MMA_LAYOUT) {
                uint8_t* pad_row = sf + static_cast<int64_t>(row >> 7) * katoms * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4;
                for (int32_t c = c_begin; c < c_end; ++c) {
                    const int32_t kb = c * 32 + lane;
                    if ((lane & 3) == 0 && kb < KB) *reinterpret_cast<uint32_t*>(pad_row + static_cast<int64_t>(kb >> 2) * 512) = 0u;
                }
            }
            continue;
        }
        float g = g_single, c1 = c1_single;
        if (segs.nseg != 0) {
            g = __ldg(g_ptr + seg_of(segs, row));
            c1 = __fdiv_rn(1.0f, __fmul_rn(6.0f, g));
        }
        const uint16_t* xrow = x + static_cast<int64_t>(row) * ld;
        const int32_t orow = segs.il_inner > 0 ? il_row(row, segs.il_inner) : row;      // where this row is written
        uint8_t* crow = codes + static_cast<int64_t>(orow) * (K >> 1);
        // scale bytes of this row: byte offset of block kb is sf_row + (kb >> 2) * 512 + (kb & 3)
        // in the tensor-core layout, sf_row + kb in the linear one
        uint8_t* sf_row = MMA_LAYOUT
            ? sf + static_cast<int64_t>(orow >> 7) * katoms * 512 + (orow & 31) * 16 + ((orow & 127) >> 5) * 4
            : sf + static_cast<int64_t>(orow) * KB;
        float rstd = 0.0f;
        if (MODE == kQuantRmsnorm) {
            float ss = 0.0f;
            constexpr int PF = 4;                                   // loads in flight per lane
            for (int32_t c = 0; c < chunks_per_row; c += PF) {
                uint32_t v[PF][8];
#pragma unroll
                for (int u = 0; u < PF; ++u) {
                    const int32_t k0 = (c + u) * 512 + lane * 16;
                    if (k0 < K) {
                        ldg256_cached(xrow + k0, v[u]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[u][i] = 0u;   // adds +0: the sum is unchanged
                    }
                }
#pragma unroll
                for (int u = 0; u < PF; ++u) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float lo = __uint_as_float(v[u][i] << 16), hi = __uint_as_float(v[u][i] & 0xFFFF0000u);
                        ss = __fmaf_rn(lo, lo, ss);
                        ss = __fmaf_rn(hi, hi, ss);
                    }
                }
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, off));
            rstd = __frcp_rn(__fsqrt_rn(__fadd_rn(__fdiv_rn(ss, static_cast<float>(K)), eps)));
        }
        for (int32_t c0 = c_begin; c0 < c_end; c0 += UNROLL) {
            uint32_t v[UNROLL][8];
            int32_t col[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                col[u] = (c0 + u < c_end) ? (c0 + u) * 512 + lane * 16 : K;
                if (col[u] < K) {
                    ldg256_stream(xrow + col[u], v[u]);
                    if (MODE == kQuantSwiglu) {
                        uint32_t up[8], h[8];
                        ldg256_stream(xrow + K + col[u], up);
                        swiglu_block(v[u], up, h);
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[u][i] = h[i];
                    }
                    if (MODE == kQuantRmsnorm) {
                        uint32_t wv[8], y[8];
                        ldg256_cached(aux + col[u], wv);
                        rmsnorm_block(v[u], wv, rstd, y);
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[u][i] = y[i];
                    }
                    if (MODE != kQuantPlain && h_out != nullptr)        // testing aid: the tensor that is quantized
                        stg256(h_out + static_cast<int64_t>(row) * K + col[u], v[u]);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[u][i] = 0u;
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (c0 + u >= c_end) break;                         // warp-uniform
                uint32_t s8;
                const uint2 word = quantize_block(v[u], g, c1, s8);
                const bool in_range = col[u] < K;
                if (!in_range) s8 = 0u;
                if (in_range) *reinterpret_cast<uint2*>(crow + (col[u] >> 1)) = word;
                const int32_t kb = col[u] >> 4;                     // this lane's block index
                if (MMA_LAYOUT || ((KB & 3) == 0 && (reinterpret_cast<uintptr_t>(sf) & 3u) == 0)) {
                    // four neighbouring lanes hold the four scale bytes of one 32-bit word
                    uint32_t w = s8 | (__shfl_down_sync(0xffffffffu, s8, 1) << 8);
                    w |= __shfl_down_sync(0xffffffffu, w, 2) << 16;
                    if ((lane & 3) == 0 && kb < KB) {
                        if (MMA_LAYOUT) *reinterpret_cast<uint32_t*>(sf_row + static_cast<int64_t>(kb >> 2) * 512) = w;
                        else            *reinterpret_cast<uint32_t*>(sf_row + kb) = w;
                    }
                } else if (in_range) {
                    sf_row[kb] = static_cast<uint8_t>(s8);
                }
            }
        }
    }
}

// ------------------------------------------------------------------ RMSNorm -> quantize, row in registers
// A row is shared by W warps of one CTA (W = 1, 2, 4 or 8; each warp owns up to NCH consecutive
// 512-element chunks and each lane one 16-element block per chunk), so the row is read
// from HBM exactly once and stays in registers between the reduction and the quantization:
//   1. every lane loads its blocks (streaming loads, all in flight at once) and sums their squares;
//   2. warp butterfly, then the W partial sums meet in shared memory (one named barrier per row;
//      the two buffers alternate so that no second barrier is needed);
//   3. y = bf16((x * rstd) * w) per element, then the block is quantized as everywhere else.
// Rows are dealt round-robin to the row groups of a persistent grid.  Rows M .. M_pad-1 (tensor-core
// layout only) get zero scales.  (Three chunks per warp at three CTAs per SM measured no faster than
// five chunks at two: the kernel is bound by its instruction count -- square, normalise, scale and
// round on top of the quantizer's own work -- not by the loads it has in flight.)
constexpr int kRmsChunksMax = 5;

template <bool MMA_LAYOUT, int W, int NCH>
__global__ void __launch_bounds__(256, NCH <= 3 ? 3 : 2)
rmsnorm_quantize_kernel(const uint16_t* __restrict__ x, int32_t M, int32_t rows_total, int32_t K, int64_t ld,
                        const float* __restrict__ g_ptr, const uint16_t* __restrict__ gain, float eps,
                        uint8_t* __restrict__ codes, uint8_t* __restrict__ sf, uint16_t* __restrict__ y_out,
                        int32_t chunks_per_row, int32_t chunks_per_warp) {
    ptx::pdl_launch_dependents();
    __shared__ float red[2][8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = warp % W;                                  // this warp's part of the row
    const int group = warp / W;                                // row group inside the CTA
    constexpr int kGroups = 8 / W;
    const int32_t KB = K >> 4;
    const int32_t katoms = (KB + 3) >> 2;
    const float g = __ldg(g_ptr);
    const float c1 = __fdiv_rn(1.0f, __fmul_rn(6.0f, g));
    const int32_t c_begin = sub * chunks_per_warp;
    const int32_t c_end = min(chunks_per_row, c_begin + chunks_per_warp);
    uint32_t parity = 0;
    for (int32_t row = blockIdx.x * kGroups + group; row < rows_total; row += gridDim.x * kGroups) {
        uint8_t* sf_row = MMA_LAYOUT
            ? sf + static_cast<int64_t>(row >> 7) * katoms * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4
            : sf + static_cast<int64_t>(row) * KB;
        if (row >= M) {
            // only reached in the tensor-core layout: rows that pad the last 128-row band
            for (int32_t c = c_begin; c < c_end; ++c) {
                const int32_t kb = c * 32 + lane;
                if ((lane & 3) == 0 && kb < KB) *reinterpret_cast<uint32_t*>(sf_row + static_cast<int64_t>(kb >> 2) * 512) = 0u;
            }
            continue;                                           // a whole group skips together: no barrier is missed
        }
        const uint16_t* xrow = x + static_cast<int64_t>(row) * ld;
        uint32_t v[NCH][8];
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int32_t col = (c_begin + i) * 512 + lane * 16;
            if (c_begin + i < c_end && col < K) {
                ldg256_stream(xrow + col, v[i]);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) v[i][e] = 0u;
            }
        }
        // one pair of partial sums per chunk (independent chains, two squares per instruction), then added up
        float ss = 0.0f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
            for (int e = 0; e < 8; ++e)
                fma_sq_f32x2(s0, s1, __uint_as_float(v[i][e] << 16), __uint_as_float(v[i][e] & 0xFFFF0000u));
            ss = __fadd_rn(ss, __fadd_rn(s0, s1));
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, off));
        if (W > 1) {
            if (lane == 0) red[parity][warp] = ss;
            ptx::named_bar_sync(1 + group, W * 32);
            ss = 0.0f;
#pragma unroll
            for (int w = 0; w < W; ++w) ss = __fadd_rn(ss, red[parity][group * W + w]);
            parity ^= 1u;
        }
        const float rstd = __frcp_rn(__fsqrt_rn(__fadd_rn(__fdiv_rn(ss, static_cast<float>(K)), eps)));
        uint8_t* crow = codes + static_cast<int64_t>(row) * (K >> 1);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            if (c_begin + i >= c_end) break;                    // warp-uniform
            const int32_t col = (c_begin + i) * 512 + lane * 16;
            const bool in_range = col < K;
            uint32_t y[8];
            if (in_range) {
                uint32_t wv[8];
                ldg256_cached(gain + col, wv);
                rmsnorm_block(v[i], wv, rstd, y);
                if (y_out != nullptr) stg256(y_out + static_cast<int64_t>(row) * K + col, y);   // testing aid
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) y[e] = 0u;
            }
            uint32_t s8;
            const uint2 word = quantize_block(y, g, c1, s8);
            if (!in_range) s8 = 0u;
            if (in_range) *reinterpret_cast<uint2*>(crow + (col >> 1)) = word;
            const int32_t kb = col >> 4;
            if (MMA_LAYOUT || ((KB & 3) == 0 && (reinterpret_cast<uintptr_t>(sf) & 3u) == 0)) {
                uint32_t w4 = s8 | (__shfl_down_sync(0xffffffffu, s8, 1) << 8);
                w4 |= __shfl_down_sync(0xffffffffu, w4, 2) << 16;
                if ((lane & 3) == 0 && kb < KB) {
                    if (MMA_LAYOUT) *reinterpret_cast<uint32_t*>(sf_row + static_cast<int64_t>(kb >> 2) * 512) = w4;
                    else            *reinterpret_cast<uint32_t*>(sf_row + kb) = w4;
                }
            } else if (in_range) {
                sf_row[kb] = static_cast<uint8_t>(s8);
            }
        }
    }
}

// ------------------------------------------------------------------ statistics
// Columns of the paper's activation/weight statistics table at NVFP4 granularity.  One lane per
// 16-element block; per block in binary32 (fused multiply-adds, fixed order), block results are
// added in double: out = {sum x^2, sum x^4, sum err^2, amax (float bits in out_amax), blocks, 1-hot}.
__global__ void __launch_bounds__(256)
stats_kernel(const uint16_t* __restrict__ x, int32_t rows, int32_t cols, int64_t ld, const float* __restrict__ g_ptr,
             double* __restrict__ out, uint32_t* __restrict__ out_amax) {
    const int32_t KB = cols >> 4;
    const int64_t total = static_cast<int64_t>(rows) * KB;
    const float g = __ldg(g_ptr);
    const float c1 = __fdiv_rn(1.0f, __fmul_rn(6.0f, g));
    double t2 = 0.0, t4 = 0.0, te = 0.0, hot = 0.0;
    float amax = 0.0f;
    for (int64_t b = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; b < total;
         b += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = b / KB;
        const int32_t kb = static_cast<int32_t>(b - r * KB);
        uint32_t v[8];
        ldg256_stream(x + r * ld + kb * 16, v);
        float f[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) { f[2 * i] = __uint_as_float(v[i] << 16); f[2 * i + 1] = __uint_as_float(v[i] & 0xFFFF0000u); }
        float s2 = 0.0f, s4 = 0.0f, bmax = 0.0f;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float q = __fmul_rn(f[i], f[i]);
            s2 = __fmaf_rn(f[i], f[i], s2);
            s4 = __fmaf_rn(q, q, s4);
            bmax = fmaxf(bmax, fabsf(f[i]));
        }
        amax = fmaxf(amax, bmax);
        if (__fmul_rn(__fmul_rn(bmax, bmax), 16.0f) > __fmul_rn(9.0f, s2)) hot += 1.0;
        const uint32_t s8 = f32_to_e4m3(__fmul_rn(bmax, c1));
        const float d = __fmul_rn(e4m3_to_f32(s8), g);
        const float qinv = __fdiv_rn(1.0f, d);
        float y[8];
        float se = 0.0f;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int i = 0; i < 8; ++i) y[i] = __fmul_rn(f[8 * h + i], qinv);
            const uint32_t codes = (s8 == 0u) ? 0u : f32x8_to_e2m1(y);
            // decode the codes again (E2M1 -> fp16 is exact)
            uint32_t h0, h1, h2, h3;
            asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\tmov.b32 {b0, b1, b2, b3}, %4;\n\t"
                "cvt.rn.f16x2.e2m1x2 %0, b0;\n\tcvt.rn.f16x2.e2m1x2 %1, b1;\n\t"
                "cvt.rn.f16x2.e2m1x2 %2, b2;\n\tcvt.rn.f16x2.e2m1x2 %3, b3;\n\t}\n"
                : "=r"(h0), "=r"(h1), "=r"(h2), "=r"(h3) : "r"(codes));
            const uint32_t hh[4] = {h0, h1, h2, h3};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 dq = __half22float2(*reinterpret_cast<const __half2*>(&hh[i]));
                const float e0 = __fsub_rn(f[8 * h + 2 * i], (s8 == 0u) ? 0.0f : __fmul_rn(dq.x, d));
                const float e1 = __fsub_rn(f[8 * h + 2 * i + 1], (s8 == 0u) ? 0.0f : __fmul_rn(dq.y, d));
                se = __fmaf_rn(e0, e0, se);
                se = __fmaf_rn(e1, e1, se);
            }
        }
        t2 += static_cast<double>(s2); t4 += static_cast<double>(s4); te += static_cast<double>(se);
    }
    // warp, then device reduction
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        t2 += __shfl_xor_sync(0xffffffffu, t2, off);
        t4 += __shfl_xor_sync(0xffffffffu, t4, off);
        te += __shfl_xor_sync(0xffffffffu, te, off);
        hot += __shfl_xor_sync(0xffffffffu, hot, off);
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(out + 0, t2); atomicAdd(out + 1, t4); atomicAdd(out + 2, te); atomicAdd(out + 5, hot);
        atomicMax(out_amax, __float_as_uint(amax));
    }
}

// out[3] = amax, out[4] = number of blocks
__global__ void stats_finalize_kernel(double* __restrict__ out, const uint32_t* __restrict__ amax_bits, double blocks) {
    out[3] = static_cast<double>(__uint_as_float(*amax_bits));
    out[4] = blocks;
}

// ------------------------------------------------------------------ scale harmonisation
// Shared global scale for a fused group: g* = max_j g_j; every scale byte of module j becomes
// e4m3(e4m3(s) * (g_j / g*)).  One thread handles the four scale bytes of one row and one
// 64-element group (one 32-bit word in either layout).
__global__ void __launch_bounds__(256)
harmonize_kernel(const uint8_t* __restrict__ sf_in, uint8_t* __restrict__ sf_out, int32_t rows, int32_t KB,
                 int32_t mma_layout, const float* __restrict__ g_seg, SegTable segs, float* __restrict__ g_shared) {
    float gstar = 0.0f;
    for (int j = 0; j < segs.nseg; ++j) gstar = fmaxf(gstar, __ldg(g_seg + j));
    if (blockIdx.x == 0 && threadIdx.x == 0) *g_shared = gstar;
    const int32_t words_per_row = (KB + 3) >> 2;
    const int64_t total = static_cast<int64_t>(rows) * words_per_row;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int32_t r = static_cast<int32_t>(i / words_per_row);
        const int32_t wq = static_cast<int32_t>(i - static_cast<int64_t>(r) * words_per_row);
        const float ratio = __fdiv_rn(__ldg(g_seg + seg_of(segs, r)), gstar);
        if (mma_layout) {
            const int64_t off = sf_mma_offset(r, wq * 4, words_per_row);
            const uint32_t w = *reinterpret_cast<const uint32_t*>(sf_in + off);
            uint32_t o = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b)
                o |= f32_to_e4m3(__fmul_rn(e4m3_to_f32((w >> (8 * b)) & 0xFFu), ratio)) << (8 * b);
            *reinterpret_cast<uint32_t*>(sf_out + off) = o;
        } else {
            for (int b = 0; b < 4 && wq * 4 + b < KB; ++b) {
                const int64_t off = static_cast<int64_t>(r) * KB + wq * 4 + b;
                sf_out[off] = static_cast<uint8_t>(f32_to_e4m3(__fmul_rn(e4m3_to_f32(sf_in[off]), ratio)));
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
