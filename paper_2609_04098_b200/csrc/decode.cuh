// Decode-sized batches (1 or 2 tokens): the linear layer is a weight-streaming problem, bound by
// HBM/L2 bandwidth and launch latency, not by the tensor cores -- a tile of 128 token rows would
// be almost all padding.  One kernel, no tensor memory, no TMA pipeline:
//   1. every CTA quantizes the few activation rows itself (same block arithmetic as
//      quantize_kernel, so the codes are the ones the oracle produces) and keeps them in shared
//      memory as exact fp16 values (E2M1 values need 3 bits) plus one float scale per block;
//   2. each warp streams whole weight rows: a lane takes 32 consecutive codes (two blocks) per
//      1024-element slice, decodes them to fp16, multiplies with the activation values
//      (products and 8-term partial sums are exact in fp16), adds the two halves in fp32, scales
//      the block sum by e4m3(s_a) * e4m3(s_w) (exact in fp32) and accumulates in fp32;
//   3. a warp shuffle adds the 32 lane sums; lane 0 applies g_a * g_seg[segment] and stores.
// The result differs from the exact product only by fp32 accumulation rounding.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <type_traits>

#include "../../include/nvfp4.h"
#include "ptx.cuh"
#include "quantize.cuh"

namespace nvfp4 {

struct DecodeParams {
    const uint16_t* x;       // bf16 [M, K], row stride ldx
    int64_t ldx;
    const float* g_a;
    const uint8_t* w_codes;  // [N, K/2]
    const uint8_t* w_sf;     // tensor-core scale layout
    const float* g_seg;
    void* y;
    int64_t ldy;
    uint32_t* status;        // first word of the workspace (a bad global scale is reported there)
    int32_t M, N, K;
    uint32_t flags;
    int32_t nseg;
    int32_t seg_end[NVFP4_MAX_SEGMENTS];
};

constexpr int kDecodeThreads = 512;
constexpr int kDecodeSlices = 5;              // 1024-element slices of a weight row in flight per lane

// eight packed E2M1 codes (one 32-bit word, element i in nibble i) -> four half2 (element 2j in .x)
__device__ __forceinline__ void e2m1x8_to_half2x4(uint32_t w, __half2 (&out)[4]) {
    uint32_t h0, h1, h2, h3;
    asm("{\n\t"
        ".reg .b8 b0, b1, b2, b3;\n\t"
        "mov.b32 {b0, b1, b2, b3}, %4;\n\t"
        "cvt.rn.f16x2.e2m1x2 %0, b0;\n\t"
        "cvt.rn.f16x2.e2m1x2 %1, b1;\n\t"
        "cvt.rn.f16x2.e2m1x2 %2, b2;\n\t"
        "cvt.rn.f16x2.e2m1x2 %3, b3;\n\t"
        "}\n"
        : "=r"(h0), "=r"(h1), "=r"(h2), "=r"(h3)
        : "r"(w));
    out[0] = *reinterpret_cast<__half2*>(&h0);
    out[1] = *reinterpret_cast<__half2*>(&h1);
    out[2] = *reinterpret_cast<__half2*>(&h2);
    out[3] = *reinterpret_cast<__half2*>(&h3);
}

// activation values per token: whole 1024-element slices, stored so that the 16-byte piece a lane
// reads next to its neighbours' is contiguous with theirs: element k = 1024 s + 32 lane + 8 q + e
// lives at half index ((4 s + q) * 32 + lane) * 8 + e   (bank-conflict-free 128-bit reads)
inline size_t decode_kpad(int64_t K) { return static_cast<size_t>((K + 1023) / 1024 * 1024); }
inline size_t decode_smem_bytes(int64_t M, int64_t K) {
    return static_cast<size_t>(M) * decode_kpad(K) * 2 + static_cast<size_t>(M) * static_cast<size_t>(K / 16) * 4;
}

template <int MT>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_gemv_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(16) uint8_t dsm[];
    const int K = p.K, KB = K >> 4;
    const int KP = ((K + 1023) >> 10) << 10;
    __half* a_val = reinterpret_cast<__half*>(dsm);                                   // [MT][KP], permuted
    float* a_scale = reinterpret_cast<float*>(dsm + static_cast<size_t>(MT) * KP * 2);    // [MT][K/16]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // ---- weight streaming set-up; the first item's loads are issued before the activations are
    // quantized so that their latency overlaps that work
    const int katoms = (KB + 3) >> 2;
    const int n_slices = (K + 1023) >> 10;
    const int warps_total = gridDim.x * (kDecodeThreads >> 5);
    const bool out_f32 = (p.flags & NVFP4_OUT_F32) != 0u;
    // a warp's work is a flat list of (row, group of kDecodeSlices slices); the loads of the next two
    // items are in flight while the current one is consumed (three register buffers), so a warp with
    // up to three items -- every warp of a 6144-row layer -- pays the memory latency once
    const int groups = (n_slices + kDecodeSlices - 1) / kDecodeSlices;
    const int first_row = blockIdx.x * (kDecodeThreads >> 5) + warp;
    const int my_rows = first_row < p.N ? (p.N - first_row + warps_total - 1) / warps_total : 0;
    const int items = my_rows * groups;
    constexpr int kBufs = 3;
    uint4 wv[kBufs][kDecodeSlices];
    uint32_t sfw[kBufs][kDecodeSlices];
    auto load_item = [&](int item, auto buf_c) {
        constexpr int buf = decltype(buf_c)::value;
        const int r = item / groups, s0 = (item - r * groups) * kDecodeSlices;
        const int n = first_row + r * warps_total;
        const uint8_t* wrow = p.w_codes + static_cast<int64_t>(n) * (K >> 1);
        const uint8_t* sfrow = p.w_sf + static_cast<int64_t>(n >> 7) * katoms * 512 + (n & 31) * 16 + ((n & 127) >> 5) * 4;
#pragma unroll
        for (int u = 0; u < kDecodeSlices; ++u) {
            const int k0 = (s0 + u) * 1024 + lane * 32;                     // this lane's 32 codes
            wv[buf][u] = make_uint4(0u, 0u, 0u, 0u);
            sfw[buf][u] = 0u;
            if (s0 + u < n_slices && k0 < K) {
                wv[buf][u] = __ldcs(reinterpret_cast<const uint4*>(wrow + (k0 >> 1)));
                const int kb = k0 >> 4;                                      // even: both scale bytes sit in one word
                sfw[buf][u] = *reinterpret_cast<const uint16_t*>(sfrow + static_cast<int64_t>(kb >> 2) * 512 + (kb & 3));
            }
        }
    };
    // This kernel releases the kernel behind it at once and may itself have been started under its
    // predecessor: the weights (if the caller flagged them resident) are requested right away, everything
    // else -- the activations, the global scales, the output -- waits for the predecessor to finish.
    ptx::pdl_launch_dependents();
    const bool w_early = (p.flags & NVFP4_W_RESIDENT) != 0u;
    if (!w_early) ptx::pdl_wait();
    if (items > 0) load_item(0, std::integral_constant<int, 0>{});
    if (items > 1) load_item(1, std::integral_constant<int, 1>{});
    // a warp whose whole share fits the three buffers (every warp of a layer with up to 3 x 16 x 148 rows of
    // up to 5120 elements) takes all its rows at once and reads each activation value once for all of them
    const bool joint = groups == 1 && items <= kBufs;
    if (joint && items > 2) load_item(2, std::integral_constant<int, 2>{});
    if (w_early) ptx::pdl_wait();
    if (blockIdx.x == 0 && warp == 0) {
        // global scales must be finite and positive; anything else is reported, not repaired
        const float ga = __ldg(p.g_a);
        bool bad = !(ga > 0.0f && ga <= 3.402823466e38f);
        for (int i = lane; i < p.nseg; i += 32) {
            const float gs = __ldg(p.g_seg + i);
            bad = bad || !(gs > 0.0f && gs <= 3.402823466e38f);
        }
        if (__any_sync(0xffffffffu, bad) && lane == 0) atomicExch(p.status, static_cast<uint32_t>(NVFP4_ERR_SCALE));
    }

    // ---- 1. quantize the activation rows (every CTA its own copy)
    {
        const float g = __ldg(p.g_a);
        const float c1 = __fdiv_rn(1.0f, __fmul_rn(6.0f, g));
        for (int b = threadIdx.x; b < MT * KB; b += kDecodeThreads) {
            const int m = b / KB, kb = b - m * KB;
            uint32_t v[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
            if (m < p.M) ldg256_cached(p.x + static_cast<int64_t>(m) * p.ldx + kb * 16, v);
            uint32_t s8;
            const uint2 codes = quantize_block(v, g, c1, s8);
            a_scale[m * KB + kb] = e4m3_to_f32(s8);
            const int k0 = kb * 16, sl = k0 >> 10, ln = (k0 & 1023) >> 5, q0 = (k0 & 31) >> 3;
            __half* base = a_val + static_cast<size_t>(m) * KP;
            __half2 lo[4], hi[4];
            e2m1x8_to_half2x4(codes.x, lo);
            e2m1x8_to_half2x4(codes.y, hi);
            *reinterpret_cast<uint4*>(base + ((sl * 4 + q0) * 32 + ln) * 8) = *reinterpret_cast<uint4*>(lo);
            *reinterpret_cast<uint4*>(base + ((sl * 4 + q0 + 1) * 32 + ln) * 8) = *reinterpret_cast<uint4*>(hi);
        }
    }
    __syncthreads();

    // ---- 2. stream weight rows
    // lane sums of one row -> output values (warp shuffle, global scales, store)
    auto finish_row = [&](int n, float (&sum)[MT]) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) sum[m] += __shfl_xor_sync(0xffffffffu, sum[m], off);
        if (lane == 0) {
            int sgi = 0;
            while (sgi + 1 < p.nseg && n >= p.seg_end[sgi]) ++sgi;
            const float alpha = __fmul_rn(__ldg(p.g_a), __ldg(p.g_seg + sgi));
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (m >= p.M) break;
                const float v = __fmul_rn(sum[m], alpha);
                if (out_f32) reinterpret_cast<float*>(p.y)[static_cast<int64_t>(m) * p.ldy + n] = v;
                else reinterpret_cast<__nv_bfloat16*>(p.y)[static_cast<int64_t>(m) * p.ldy + n] = __float2bfloat16_rn(v);
            }
        }
    };
    if (joint) {
        // Shared memory is what bounds the row-by-row form: every weight row re-reads the token's values
        // (10 KB for K = 5120).  Here a 16-byte piece of activations is read once and meets the matching
        // eight weights of each of the warp's rows, decoded on the spot; same arithmetic per row, same order.
        float accj[kBufs][MT];
#pragma unroll
        for (int b = 0; b < kBufs; ++b)
#pragma unroll
            for (int m = 0; m < MT; ++m) accj[b][m] = 0.0f;
#pragma unroll
        for (int u = 0; u < kDecodeSlices; ++u) {
            const int k0 = u * 1024 + lane * 32;
            if (!(u < n_slices && k0 < K)) continue;
            const int kb = k0 >> 4;
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const uint4* ap = reinterpret_cast<const uint4*>(a_val + static_cast<size_t>(m) * KP) +
                                  (static_cast<size_t>(u) * 4) * 32 + lane;
                __half2 sum0[kBufs], sum1[kBufs];
#pragma unroll
                for (int b = 0; b < kBufs; ++b) { sum0[b] = __float2half2_rn(0.0f); sum1[b] = sum0[b]; }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint4 av = ap[q * 32];
                    const __half2* a2 = reinterpret_cast<const __half2*>(&av);
#pragma unroll
                    for (int b = 0; b < kBufs; ++b) {
                        if (b >= items) break;                                   // warp-uniform
                        const uint32_t word = q == 0 ? wv[b][u].x : (q == 1 ? wv[b][u].y : (q == 2 ? wv[b][u].z : wv[b][u].w));
                        __half2 t[4];
                        e2m1x8_to_half2x4(word, t);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (q < 2) sum0[b] = __hfma2(a2[e], t[e], sum0[b]);
                            else       sum1[b] = __hfma2(a2[e], t[e], sum1[b]);
                        }
                    }
                }
                const float2 sa = *reinterpret_cast<const float2*>(a_scale + m * KB + kb);     // kb is even
#pragma unroll
                for (int b = 0; b < kBufs; ++b) {
                    if (b >= items) break;
                    uint32_t sh2;
                    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sh2) : "h"(static_cast<uint16_t>(sfw[b][u])));
                    const float2 sw = __half22float2(*reinterpret_cast<__half2*>(&sh2));
                    const float2 b0 = __half22float2(sum0[b]), b1 = __half22float2(sum1[b]);
                    accj[b][m] = __fmaf_rn(__fadd_rn(b0.x, b0.y), __fmul_rn(sa.x, sw.x), accj[b][m]);
                    accj[b][m] = __fmaf_rn(__fadd_rn(b1.x, b1.y), __fmul_rn(sa.y, sw.y), accj[b][m]);
                }
            }
        }
#pragma unroll
        for (int b = 0; b < kBufs; ++b) {
            if (b >= items) break;
            finish_row(first_row + b * warps_total, accj[b]);
        }
        return;
    }
    float acc[MT];
    auto do_item = [&](int item, auto buf_c) {
        constexpr int buf = decltype(buf_c)::value;
        const int r = item / groups, g0 = item - r * groups, s0 = g0 * kDecodeSlices;
        const int n = first_row + r * warps_total;
        if (item + 2 < items) load_item(item + 2, std::integral_constant<int, (buf + 2) % kBufs>{});
        if (g0 == 0) {
#pragma unroll
            for (int m = 0; m < MT; ++m) acc[m] = 0.0f;
        }
        {
#pragma unroll
            for (int u = 0; u < kDecodeSlices; ++u) {
                const int k0 = (s0 + u) * 1024 + lane * 32;
                if (!(s0 + u < n_slices && k0 < K)) continue;
                const uint4 wcur = wv[buf][u];
                const uint32_t scur = sfw[buf][u];
                // weight scales of the two blocks, weight values as half2
                uint32_t sh2;
                asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sh2) : "h"(static_cast<uint16_t>(scur)));
                const float2 sw = __half22float2(*reinterpret_cast<__half2*>(&sh2));
                __half2 wq[16];
                {
                    __half2 t[4];
                    e2m1x8_to_half2x4(wcur.x, t);
#pragma unroll
                    for (int j = 0; j < 4; ++j) wq[j] = t[j];
                    e2m1x8_to_half2x4(wcur.y, t);
#pragma unroll
                    for (int j = 0; j < 4; ++j) wq[4 + j] = t[j];
                    e2m1x8_to_half2x4(wcur.z, t);
#pragma unroll
                    for (int j = 0; j < 4; ++j) wq[8 + j] = t[j];
                    e2m1x8_to_half2x4(wcur.w, t);
#pragma unroll
                    for (int j = 0; j < 4; ++j) wq[12 + j] = t[j];
                }
                const int kb = k0 >> 4;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    // piece q of this lane: 32 lanes x 16 bytes apart from piece q + 1
                    const uint4* ap = reinterpret_cast<const uint4*>(a_val + static_cast<size_t>(m) * KP) +
                                      (static_cast<size_t>(s0 + u) * 4) * 32 + lane;
                    __half2 s0h = __float2half2_rn(0.0f), s1h = __float2half2_rn(0.0f);
#pragma unroll
                    for (int q = 0; q < 2; ++q) {                            // block 0: 8 half2
                        const uint4 av = ap[q * 32];
                        const __half2* a2 = reinterpret_cast<const __half2*>(&av);
#pragma unroll
                        for (int e = 0; e < 4; ++e) s0h = __hfma2(a2[e], wq[4 * q + e], s0h);
                    }
#pragma unroll
                    for (int q = 2; q < 4; ++q) {                            // block 1
                        const uint4 av = ap[q * 32];
                        const __half2* a2 = reinterpret_cast<const __half2*>(&av);
#pragma unroll
                        for (int e = 0; e < 4; ++e) s1h = __hfma2(a2[e], wq[4 * q + e], s1h);
                    }
                    const float2 b0 = __half22float2(s0h), b1 = __half22float2(s1h);
                    const float2 sa = *reinterpret_cast<const float2*>(a_scale + m * KB + kb);     // kb is even
                    acc[m] = __fmaf_rn(__fadd_rn(b0.x, b0.y), __fmul_rn(sa.x, sw.x), acc[m]);
                    acc[m] = __fmaf_rn(__fadd_rn(b1.x, b1.y), __fmul_rn(sa.y, sw.y), acc[m]);
                }
            }
        }
        if (g0 + 1 < groups) return;                       // more slices of this row to come
        // ---- 3. reduce over lanes, scale, store
        finish_row(n, acc);
    };
#pragma unroll 1
    for (int item = 0; item < items; item += kBufs) {
        do_item(item, std::integral_constant<int, 0>{});
        if (item + 1 < items) do_item(item + 1, std::integral_constant<int, 1>{});
        if (item + 2 < items) do_item(item + 2, std::integral_constant<int, 2>{});
    }
}

}  // namespace nvfp4
