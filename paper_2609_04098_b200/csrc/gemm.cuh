// Block-scaled FP4 GEMM for sm_100a with a per-segment global-scale epilogue.
//
//   Y[m, n] = (sum_k a_hat[m,k] w_hat[n,k]) * g_a * g_seg[seg(n)]
//
// One persistent CTA per SM, 320 threads, four roles:
//   warp 0      TMA producer: codes of A (128 x 256 elements) and W (BN x 256) per
//               stage as 128-byte-swizzled tiles, plus their scale bytes, which are
//               contiguous 512-byte atoms in the tensor-core scale layout and so
//               travel as plain bulk copies;
//   warps 6-9   scale loaders, one per 32-lane TMEM quarter: when a stage has landed
//               they read its scale atoms from shared memory and write them into that
//               stage's TMEM scale columns with tcgen05.st (a 512-byte atom is exactly
//               32 lanes x 4 columns, identical in all four quarters).  tcgen05.cp could
//               do this copy too, but it runs in the tensor pipe in series with the MMAs
//               (measured: ~70 cycles each, three per 128-cycle MMA);
//   warp 1      one thread walks the CTA's (tile, k) stream and issues tcgen05.mma
//               kind::mxf4nvf4 (M=128, N=BN, K=64) into the TMEM accumulator as soon as
//               a stage's scales are in TMEM;
//   warps 2-5   epilogue: tcgen05.ld a 32-lane quarter each, multiply every column by
//               its segment's global scale, round once to bf16, stage 32x64 pieces in
//               swizzled shared memory and hand them to TMA stores; the accumulator
//               is released as soon as its last column is in registers.
// Stages hand over through mbarriers; every wait is bounded (see ptx.cuh) and a CTA
// that gives up raises a status word instead of hanging.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/nvfp4.h"
#include "ptx.cuh"

namespace nvfp4 {

struct GemmParams {
    const uint8_t* sfa;      // A scales, tensor-core layout
    const uint8_t* sfb;      // W scales, tensor-core layout
    const float* g_a;        // device scalar
    const float* g_seg;      // device [nseg]
    void* y;
    int64_t ldy;
    uint32_t* status;        // first word of the workspace
    int32_t M, N, K;
    int32_t m_tiles, n_tiles, k_tiles;
    int32_t katoms;          // K / 64: 512-byte scale atoms per 128-row band
    int32_t sfa_bands;       // ceil(M / 128)
    int32_t sfb_bands;       // ceil(N / 128)
    uint32_t flags;
    uint32_t tma_store;      // 1: bf16 output through the TMA-store path (tmY valid)
    int32_t nseg;
    int32_t seg_end[NVFP4_MAX_SEGMENTS];
    uint64_t wait_limit_ns;
#ifdef NVFP4_PROBE
    uint32_t probe;          // timing experiments only (results are wrong): see the bits below
#endif
};
#ifdef NVFP4_PROBE
#define NVFP4_PROBE_BIT(p, b) (((p).probe >> (b)) & 1u)
#else
#define NVFP4_PROBE_BIT(p, b) 0u
#endif
// probe bits: 0 no MMA, 1 no operand TMA, 2 no scale bulk copies, 3 no scale TMEM writes, 4 no epilogue
// stores

constexpr int kGemmThreads = 320;
constexpr int kBM = 128;
constexpr int kBKBytes = 128;                 // 256 FP4 elements = one 128-byte swizzle row
constexpr int kStepsPerStage = 4;             // four K=64 MMAs per stage
constexpr int kTmemCols = 512;
constexpr int kOutPieceCols = 64;             // epilogue piece: 32 rows x 64 bf16 = 4 KB
constexpr int kOutPieceBytes = 32 * kOutPieceCols * 2;

template <int BN, int ACC, int STAGES>
struct GemmCfg {
    static constexpr int A_BYTES = kBM * kBKBytes;
    static constexpr int B_BYTES = BN * kBKBytes;
    static constexpr int NB_BANDS = BN / 128;
    static constexpr int SFA_BYTES = kStepsPerStage * 512;
    static constexpr int SFB_BYTES = NB_BANDS * kStepsPerStage * 512;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;
    static constexpr int OUT_BYTES = 4 * 2 * kOutPieceBytes;          // per epilogue warp: two pieces
    static constexpr int ALPHA_BYTES = 4 * BN * 4;                    // one private copy per epilogue warp
    static constexpr int BAR_BYTES = (3 * STAGES + 2 * ACC + 1) * 8 + 16;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + OUT_BYTES + ALPHA_BYTES + BAR_BYTES;
    // TMEM columns: accumulators first, then one set of scale columns per smem stage
    static constexpr int SFA_SET_COLS = kStepsPerStage * 4;
    static constexpr int SFB_SET_COLS = kStepsPerStage * (BN / 32);
    static constexpr int SFA_COL0 = ACC * BN;
    static constexpr int SFA_COLS = STAGES * SFA_SET_COLS;
    static constexpr int SFB_COL0 = SFA_COL0 + SFA_COLS;
    static constexpr int SFB_COLS = STAGES * SFB_SET_COLS;
    static_assert(BN % 128 == 0 && BN <= 256, "BN must be 128 or 256");
    static_assert(SFB_COL0 + SFB_COLS <= kTmemCols, "TMEM budget");
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
    static_assert(STAGE_BYTES % 1024 == 0, "stage alignment");
};

// instruction descriptor: E2M1 x E2M1, E4M3 scales, K-major A and B, M=128, N=BN
template <int BN>
__device__ __forceinline__ constexpr uint32_t nvf4_idesc() {
    return (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) | (0u << 23) |
           (static_cast<uint32_t>(kBM >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&b2);
}

template <int BN, int ACC, int STAGES>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmY, const __grid_constant__ GemmParams p) {
    using C = GemmCfg<BN, ACC, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* out_s = smem + STAGES * C::STAGE_BYTES;                   // 1024-byte aligned
    float* alpha_s = reinterpret_cast<float*>(out_s + C::OUT_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(out_s + C::OUT_BYTES + C::ALPHA_BYTES);
    uint64_t* full = bars;
    uint64_t* empty = bars + STAGES;
    uint64_t* sfready = bars + 2 * STAGES;
    uint64_t* tfull = bars + 3 * STAGES;
    uint64_t* tempty = bars + 3 * STAGES + ACC;
    uint64_t* drain = bars + 3 * STAGES + 2 * ACC;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int32_t total_tiles = p.m_tiles * p.n_tiles;
    const uint32_t my_tiles = (static_cast<uint32_t>(total_tiles) > blockIdx.x)
                                  ? (static_cast<uint32_t>(total_tiles) - blockIdx.x + gridDim.x - 1) / gridDim.x
                                  : 0u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], 1);
            ptx::mbar_init(&sfready[s], 4);
        }
        for (int a = 0; a < ACC; ++a) { ptx::mbar_init(&tfull[a], 1); ptx::mbar_init(&tempty[a], 4); }
        ptx::mbar_init(drain, 1);
        *abort_flag = 0u;
        ptx::fence_barrier_init();
    }
    // scale staging starts as zeros so that bands a tile never loads read as 0.0, not NaN
    for (int s = 0; s < STAGES; ++s) {
        uint4* z = reinterpret_cast<uint4*>(smem + s * C::STAGE_BYTES + C::A_BYTES + C::B_BYTES);
        for (int i = threadIdx.x; i < (C::SFA_BYTES + C::SFB_BYTES) / 16; i += kGemmThreads)
            z[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    ptx::fence_proxy_async_smem();
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&tmA);
            ptx::prefetch_tensormap(&tmB);
            uint32_t it = 0;
            bool ok = true;
            for (int32_t tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
                const int32_t m_t = tile % p.m_tiles, n_t = tile / p.m_tiles;
                for (int32_t kt = 0; kt < p.k_tiles; ++kt, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!ptx::mbar_wait_bounded(&empty[s], ph ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                    uint8_t* st = smem + s * C::STAGE_BYTES;
                    const int32_t steps = min(kStepsPerStage, p.katoms - kt * kStepsPerStage);
                    const uint32_t sf_bytes = static_cast<uint32_t>(steps) * 512u;
                    uint32_t tx = C::A_BYTES + C::B_BYTES + sf_bytes;
                    int nb_live = 0;
#pragma unroll
                    for (int c = 0; c < C::NB_BANDS; ++c)
                        if (n_t * C::NB_BANDS + c < p.sfb_bands) ++nb_live;
                    tx += nb_live * sf_bytes;
#ifdef NVFP4_PROBE
                    if (NVFP4_PROBE_BIT(p, 1)) tx -= C::A_BYTES + C::B_BYTES;
                    if (NVFP4_PROBE_BIT(p, 2)) tx -= (1 + nb_live) * sf_bytes;
#endif
                    ptx::mbar_arrive_expect_tx(&full[s], tx);
                    if (!NVFP4_PROBE_BIT(p, 1)) {
                        ptx::tma_load_2d(st, &tmA, kt * kBKBytes, m_t * kBM, &full[s]);
                        ptx::tma_load_2d(st + C::A_BYTES, &tmB, kt * kBKBytes, n_t * BN, &full[s]);
                    }
                    if (NVFP4_PROBE_BIT(p, 2)) continue;
                    ptx::bulk_load(st + C::A_BYTES + C::B_BYTES,
                                   p.sfa + (static_cast<int64_t>(m_t) * p.katoms + kt * kStepsPerStage) * 512,
                                   sf_bytes, &full[s]);
#pragma unroll
                    for (int c = 0; c < C::NB_BANDS; ++c) {
                        const int32_t band = n_t * C::NB_BANDS + c;
                        if (band < p.sfb_bands)
                            ptx::bulk_load(st + C::A_BYTES + C::B_BYTES + C::SFA_BYTES + c * (kStepsPerStage * 512),
                                           p.sfb + (static_cast<int64_t>(band) * p.katoms + kt * kStepsPerStage) * 512,
                                           sf_bytes, &full[s]);
                    }
                }
            }
            if (!ok) {
                // give copies already in flight a bounded chance to land before the CTA exits
                const uint32_t first = it > static_cast<uint32_t>(STAGES) ? it - STAGES : 0u;
                for (uint32_t i = first; i < it; ++i)
                    for (int spin = 0; spin < 4096 && !ptx::mbar_try_wait(&full[i % STAGES], (i / STAGES) & 1u); ++spin) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = nvf4_idesc<BN>();
            const uint32_t k_tiles = static_cast<uint32_t>(p.k_tiles);
            const uint32_t total_it = my_tiles * k_tiles;
            bool ok = true;
            for (uint32_t it = 0; ok && it < total_it; ++it) {
                const uint32_t kt = it % k_tiles, tl = it / k_tiles;
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                const uint32_t acc = tl % ACC, aph = (tl / ACC) & 1u;
                if (NVFP4_PROBE_BIT(p, 0)) {
                    if (!ptx::mbar_wait_bounded(&sfready[s], ph, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                    ptx::mbar_arrive(&empty[s]);
                    if (kt == k_tiles - 1) {
                        if (!ptx::mbar_wait_bounded(&tempty[acc], aph ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                        ptx::mbar_arrive(&tfull[acc]);
                    }
                    continue;
                }
                if (kt == 0) {
                    if (!ptx::mbar_wait_bounded(&tempty[acc], aph ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                }
                // scales in TMEM implies codes in shared memory (the loaders waited for the stage)
                if (!ptx::mbar_wait_bounded(&sfready[s], ph, abort_flag, p.wait_limit_ns)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t st = ptx::smem_u32(smem + s * C::STAGE_BYTES);
                const int32_t steps = min(kStepsPerStage, p.katoms - static_cast<int32_t>(kt) * kStepsPerStage);
                const uint32_t sfa_t = tmem_base + C::SFA_COL0 + s * C::SFA_SET_COLS;
                const uint32_t sfb_t = tmem_base + C::SFB_COL0 + s * C::SFB_SET_COLS;
                const uint32_t d_tmem = tmem_base + acc * BN;
                const uint64_t a_desc = ptx::smem_desc(st, 16, 1024, 2);
                const uint64_t b_desc = ptx::smem_desc(st + C::A_BYTES, 16, 1024, 2);
                for (int32_t j = 0; j < steps; ++j) {
                    // advancing K by 64 elements = 32 bytes inside the 128-byte swizzle row
                    ptx::tc_mma_nvf4(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, sfa_t + j * 4,
                                     sfb_t + j * (BN / 32), (kt | static_cast<uint32_t>(j)) != 0u ? 1u : 0u);
                }
                ptx::tc_commit(&empty[s]);                          // stage reusable once these MMAs have read it
                if (kt == k_tiles - 1) ptx::tc_commit(&tfull[acc]); // accumulator complete
            }
            if (!ok) {
                ptx::tc_commit(drain);                  // let issued MMAs finish before TMEM is freed
                for (int spin = 0; spin < (1 << 16) && !ptx::mbar_try_wait(drain, 0u); ++spin) {}
            }
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------ scale loaders
        // A stage's TMEM scale columns are free when its shared-memory buffers are: the
        // producer refilled the stage only after the MMAs that read both had completed.
        const uint32_t quarter = static_cast<uint32_t>(warp & 3);
        const uint32_t k_tiles = static_cast<uint32_t>(p.k_tiles);
        const uint32_t total_it = my_tiles * k_tiles;
        const uint32_t lane_field = (quarter * 32u) << 16;
        for (uint32_t it = 0; it < total_it; ++it) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            bool ok = ptx::mbar_wait_bounded(&full[s], ph, abort_flag, p.wait_limit_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (!NVFP4_PROBE_BIT(p, 3)) {
                const uint32_t sf_s = ptx::smem_u32(smem + s * C::STAGE_BYTES) + C::A_BYTES + C::B_BYTES + lane * 16;
                // A: atom j -> columns 4j..4j+3
                {
                    uint32_t r[16];
#pragma unroll
                    for (int j = 0; j < kStepsPerStage; ++j) {
                        const uint4 v = ptx::ld_shared_v4(sf_s + j * 512);
                        r[4 * j + 0] = v.x; r[4 * j + 1] = v.y; r[4 * j + 2] = v.z; r[4 * j + 3] = v.w;
                    }
                    ptx::tmem_st_32x16(tmem_base + lane_field + C::SFA_COL0 + s * C::SFA_SET_COLS, r);
                }
                // W: K-step j, 128-row band c -> columns j*(BN/32) + 4c ..
#pragma unroll
                for (int c = 0; c < C::NB_BANDS; ++c) {
                    uint32_t r[16];
#pragma unroll
                    for (int j = 0; j < kStepsPerStage; ++j) {
                        const uint4 v = ptx::ld_shared_v4(sf_s + C::SFA_BYTES + c * (kStepsPerStage * 512) + j * 512);
                        r[4 * j + 0] = v.x; r[4 * j + 1] = v.y; r[4 * j + 2] = v.z; r[4 * j + 3] = v.w;
                    }
                    if (C::NB_BANDS == 1) {
                        ptx::tmem_st_32x16(tmem_base + lane_field + C::SFB_COL0 + s * C::SFB_SET_COLS, r);
                    } else {
                        // bands interleave per K-step: four columns at a time
#pragma unroll
                        for (int j = 0; j < kStepsPerStage; ++j) {
                            const uint32_t q[4] = {r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]};
                            ptx::tmem_st_32x4(tmem_base + lane_field + C::SFB_COL0 + s * C::SFB_SET_COLS +
                                              j * (BN / 32) + c * 4, q);
                        }
                    }
                }
                ptx::tmem_st_wait();
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sfready[s]);
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                   // TMEM lanes this warp may read
        float* alpha_w = alpha_s + quarter * BN;
        uint8_t* out_w = out_s + quarter * (2 * kOutPieceBytes);
        const float g_a = __ldg(p.g_a);
        const bool out_f32 = (p.flags & NVFP4_OUT_F32) != 0u;
        const bool use_tma = p.tma_store != 0u;
        const bool vec_ok = out_f32 ? ((p.ldy & 3) == 0 && (reinterpret_cast<uintptr_t>(p.y) & 15) == 0)
                                    : ((p.ldy & 7) == 0 && (reinterpret_cast<uintptr_t>(p.y) & 15) == 0);
        if (use_tma && lane == 0) ptx::prefetch_tensormap(&tmY);
        uint32_t tl = 0, pieces_stored = 0;
        for (int32_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tl) {
            const int32_t m_t = tile % p.m_tiles, n_t = tile / p.m_tiles;
            const int32_t n0 = n_t * BN;
            const uint32_t acc = tl % ACC, aph = (tl / ACC) & 1u;
            // per-column global scale of this tile (each warp keeps a private copy)
            __syncwarp();
            for (int c = lane; c < BN; c += 32) {
                const int32_t n = n0 + c;
                float a = 0.0f;
                if (n < p.N) {
                    int sgi = 0;
                    while (sgi + 1 < p.nseg && n >= p.seg_end[sgi]) ++sgi;
                    a = __fmul_rn(g_a, __ldg(p.g_seg + sgi));
                }
                alpha_w[c] = a;
            }
            __syncwarp();
            bool ok = ptx::mbar_wait_bounded(&tfull[acc], aph, abort_flag, p.wait_limit_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            ptx::tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * BN;
            const int32_t row0 = m_t * kBM + quarter * 32;

            if (use_tma) {
                constexpr int NP = BN / kOutPieceCols;
                uint32_t ra[64], rb[64];
                ptx::tmem_ld_32x64(t_row, ra);
#pragma unroll
                for (int pc = 0; pc < NP; ++pc) {
                    uint32_t (&cur)[64] = (pc & 1) ? rb : ra;
                    uint32_t (&nxt)[64] = (pc & 1) ? ra : rb;
                    ptx::tmem_ld_wait();
                    if (pc + 1 < NP) {
                        ptx::tmem_ld_32x64(t_row + (pc + 1) * kOutPieceCols, nxt);
                    } else {
                        // last column is in registers: hand the accumulator back to the MMA warp
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&tempty[acc]);
                    }
                    const int32_t col0 = n0 + pc * kOutPieceCols;
                    if (col0 >= p.N || row0 >= p.M || NVFP4_PROBE_BIT(p, 4)) continue;   // warp-uniform
                    uint8_t* buf = out_w + (pieces_stored & 1u) * kOutPieceBytes;
                    if (pieces_stored >= 2u) {
                        if (lane == 0) ptx::bulk_wait_group_read<1>();   // the store that last used `buf` has read it
                        __syncwarp();
                    }
                    const float* al = alpha_w + pc * kOutPieceCols;
                    const uint32_t row_s = ptx::smem_u32(buf) + lane * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t w0 = pack_bf16x2(__fmul_rn(__uint_as_float(cur[8 * c + 0]), al[8 * c + 0]),
                                                        __fmul_rn(__uint_as_float(cur[8 * c + 1]), al[8 * c + 1]));
                        const uint32_t w1 = pack_bf16x2(__fmul_rn(__uint_as_float(cur[8 * c + 2]), al[8 * c + 2]),
                                                        __fmul_rn(__uint_as_float(cur[8 * c + 3]), al[8 * c + 3]));
                        const uint32_t w2 = pack_bf16x2(__fmul_rn(__uint_as_float(cur[8 * c + 4]), al[8 * c + 4]),
                                                        __fmul_rn(__uint_as_float(cur[8 * c + 5]), al[8 * c + 5]));
                        const uint32_t w3 = pack_bf16x2(__fmul_rn(__uint_as_float(cur[8 * c + 6]), al[8 * c + 6]),
                                                        __fmul_rn(__uint_as_float(cur[8 * c + 7]), al[8 * c + 7]));
                        // 128-byte swizzle: 16-byte chunk index XOR (row mod 8)
                        ptx::st_shared_v4(row_s + ((c ^ (lane & 7)) << 4), w0, w1, w2, w3);
                    }
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_2d(&tmY, buf, col0, row0);
                        ptx::bulk_commit_group();
                    }
                    ++pieces_stored;
                }
            } else {
                const int32_t row = row0 + lane;
                const bool row_ok = row < p.M;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    __syncwarp();
                    ptx::tmem_ld_32x32(t_row + c * 32, r);
                    ptx::tmem_ld_wait();
                    const int32_t col0 = n0 + c * 32;
                    if (!row_ok || col0 >= p.N || NVFP4_PROBE_BIT(p, 4)) continue;
                    const float* al = alpha_w + c * 32;
                    if (out_f32) {
                        float* yr = reinterpret_cast<float*>(p.y) + static_cast<int64_t>(row) * p.ldy + col0;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float4 o;
                            o.x = __fmul_rn(__uint_as_float(r[4 * j + 0]), al[4 * j + 0]);
                            o.y = __fmul_rn(__uint_as_float(r[4 * j + 1]), al[4 * j + 1]);
                            o.z = __fmul_rn(__uint_as_float(r[4 * j + 2]), al[4 * j + 2]);
                            o.w = __fmul_rn(__uint_as_float(r[4 * j + 3]), al[4 * j + 3]);
                            if (vec_ok && col0 + 4 * j + 4 <= p.N) {
                                *reinterpret_cast<float4*>(yr + 4 * j) = o;
                            } else {
                                const float e[4] = {o.x, o.y, o.z, o.w};
                                for (int t = 0; t < 4; ++t)
                                    if (col0 + 4 * j + t < p.N) yr[4 * j + t] = e[t];
                            }
                        }
                    } else {
                        __nv_bfloat16* yr =
                            reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<int64_t>(row) * p.ldy + col0;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t w[4];
#pragma unroll
                            for (int t = 0; t < 4; ++t)
                                w[t] = pack_bf16x2(__fmul_rn(__uint_as_float(r[8 * j + 2 * t]), al[8 * j + 2 * t]),
                                                   __fmul_rn(__uint_as_float(r[8 * j + 2 * t + 1]), al[8 * j + 2 * t + 1]));
                            if (vec_ok && col0 + 8 * j + 8 <= p.N) {
                                *reinterpret_cast<uint4*>(yr + 8 * j) = make_uint4(w[0], w[1], w[2], w[3]);
                            } else {
                                for (int t = 0; t < 8; ++t)
                                    if (col0 + 8 * j + t < p.N)
                                        reinterpret_cast<uint16_t*>(yr)[8 * j + t] =
                                            static_cast<uint16_t>((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xFFFFu));
                            }
                        }
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&tempty[acc]);
            }
        }
        if (use_tma && lane == 0) ptx::bulk_wait_group<0>();   // all output stores complete before exit
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag != 0u) atomicExch(p.status, static_cast<uint32_t>(NVFP4_ERR_TIMEOUT));
}

}  // namespace nvfp4
