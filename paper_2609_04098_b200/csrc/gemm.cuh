// Block-scaled FP4 GEMM for sm_100a with a per-segment global-scale epilogue.
//
//   Y[m, n] = (sum_k a_hat[m,k] w_hat[n,k]) * g_a * g_seg[seg(n)]
//
// One persistent CTA per SM (224 threads).  Two shapes of the same kernel:
//   single  one CTA computes a 128 x BN tile (BN = 128 or 256);
//   pair    two CTAs of a cluster compute a 256 x 256 tile with tcgen05 cta_group::2:
//           each CTA loads 128 rows of A and only HALF of the W tile, so a stage is
//           38 KB instead of 54 KB for the same tensor-core time and five stages fit.
//           No load is multicast.  The partner's TMA copies count their bytes on the
//           leader's "stage full" barrier; the leader's commits arrive on both CTAs'
//           "stage empty" / "accumulator full" barriers; both CTAs' epilogue warps arrive
//           on the leader's "accumulator empty" barrier.
// Warp roles:
//   warps 0-3   epilogue, one per 32-lane TMEM quarter: tcgen05.ld, multiply every column
//               by its segment's global scale, round once to bf16, stage 32x64 pieces in
//               swizzled shared memory, TMA store; the accumulator is handed back as soon
//               as its last column is in registers;
//   warp 4      TMA producer for A: codes (128 x 256 elements, 128-byte swizzle) and the
//               matching scale atoms (a 3-D box over [band][k-atom][512 bytes]);
//   warp 5      TMA producer for W, same;
//   warp 6      one thread (leader CTA only, in a pair) issues, per K=64 step, the three
//               tcgen05.cp that bring that step's scale atoms from shared memory to TMEM
//               and then the tcgen05.mma kind::mxf4nvf4.  Measured on B200 (one SM, operands in
//               shared memory): an MMA of N=256 occupies the tensor pipe for 128 cycles and the
//               three copies add ~4 cycles when the issuing thread keeps up; what decides
//               whether it keeps up is the SHAPE of the issuing code (see the loop).
// Every mbarrier wait is bounded (ptx.cuh); a CTA that gives up raises a status word and
// tells its partner instead of hanging.
#pragma once
#include <cstdint>
#include <type_traits>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/nvfp4.h"
#include "ptx.cuh"
#include "quantize.cuh"

namespace nvfp4 {

struct GemmParams {
    const float* g_a;        // device scalar
    const float* g_seg;      // device [nseg]
    void* y;
    int64_t ldy;
    uint32_t* status;        // first word of the workspace
    int32_t M, N, K;
    int32_t m_tiles;         // ceil(M / 128)
    int32_t n_tiles;         // ceil(N / BN)
    int32_t k_tiles;         // ceil(K / 256)
    int32_t katoms;          // K / 64: 512-byte scale atoms per 128-row band
    int32_t group_m;         // row units per raster group (see tile_of)
    int32_t a_box_bytes;     // bytes of one A code box: 128 rows x 128 bytes, fewer rows for decode-sized M
                             // (the tensor core still multiplies 128 rows; what the rows past the box hold in
                             // shared memory only reaches accumulator rows that are never stored)
    // split-K (small M): an output tile is computed by split_k CTAs, each over k_per_split
    // consecutive K tiles; partial sums meet in `partial` (fp32 [rows padded to 128][ldp], zero
    // between calls), `counters` (one per tile and lane quarter, zero between calls) tell the
    // last arrival, which applies the scales, writes Y and re-zeroes what it read
    int32_t split_k, k_per_split, ldp;
    float* partial;
    uint32_t* counters;
    uint32_t flags;
    uint32_t tma_store;      // 1: bf16 output through the TMA-store path (tmY valid)
    int32_t nseg;
    int32_t seg_end[NVFP4_MAX_SEGMENTS];
    uint64_t wait_limit_ns;
    // fused SwiGLU + quantize epilogue (EPI == kEpiSwiglu): the W rows are gate/up interleaved 16 by 16,
    // N = 2 * inner; the epilogue writes NVFP4 codes and scales of h = silu(gate) * up instead of Y
    const float* g_h;        // device scalar: global scale of h
    uint8_t* h_codes;        // [M, inner / 2]
    uint8_t* h_sf;           // tensor-core scale layout of an [M, inner] tensor
    int32_t h_katoms;        // inner / 64
    int32_t inner;
    void* dbg_y;             // optional testing outputs: bf16 [M, 2 * inner] (interleaved columns) ...
    void* dbg_h;             // ... and bf16 [M, inner]
    // activations quantized inside the kernel (cluster-split builds only, a handful of rows): bf16
    // [M, K] with row stride ldx; then no quantized copy of A exists in global memory at all
    const uint16_t* x;
    int64_t ldx;
};
constexpr int kEpiPlain = 0, kEpiSwiglu = 1, kEpiClusterSplit = 2, kEpiClusterSplitFew = 3;

constexpr int kGemmThreads = 224;
constexpr int kBM = 128;
constexpr int kBKBytes = 128;                 // 256 FP4 elements = one 128-byte swizzle row
constexpr int kStepsPerStage = 4;             // four K=64 MMAs per stage
constexpr int kTmemCols = 512;
constexpr int kOutPieceCols = 64;             // epilogue piece: 32 rows x 64 bf16 = 4 KB
constexpr int kOutPieceBytes = 32 * kOutPieceCols * 2;

constexpr int kClusterSplitSlotBytes = 32 * 128 * 4;      // fp32 partial sums of one 32-row quarter of a 128-wide tile
// landing slots in the cluster's first CTA: five beside four stages, or two beside five stages
__host__ __device__ constexpr int cluster_split_slots(int epi) { return epi == 2 ? 5 : (epi == 3 ? 2 : 0); }
constexpr int kScaleTabBytes = 4 * kOutPieceCols * 4;     // per epilogue warp: the global scales of one piece's columns
constexpr int kDefaultOutBytes = 4 * 2 * kOutPieceBytes + kScaleTabBytes;  // per epilogue warp: two pieces, and the scale table

template <int BN, int STAGES, bool PAIR, int OUT_BYTES_ = kDefaultOutBytes>
struct GemmCfg {
    // Two TMEM accumulators.  BN = 128: disjoint (0..127, 128..255).  BN = 256: they do not both
    // fit beside the scale columns, so they OVERLAP by one epilogue piece: columns 0..255 and
    // 192..447.  The epilogue drains the shared 64 columns of a tile first and only then lets
    // the next tile's MMAs start; the rest of its drain runs under those MMAs.
    static constexpr int ACC = 2;
    static constexpr bool OVERLAP = (BN == 256);
    static constexpr int ACC_STRIDE = OVERLAP ? BN - kOutPieceCols : BN;
    static constexpr int SF_SETS = OVERLAP ? 1 : STAGES;               // sets of scale columns
    static constexpr int B_ROWS = PAIR ? BN / 2 : BN;                  // W rows this CTA loads
    static constexpr int NB_BANDS = BN / 128;                          // 128-row scale bands of the W tile
    static constexpr int CTAS = PAIR ? 2 : 1;
    static constexpr int A_BYTES = kBM * kBKBytes;
    static constexpr int B_BYTES = B_ROWS * kBKBytes;
    static constexpr int SFA_BYTES = kStepsPerStage * 512;
    static constexpr int SFB_BYTES = NB_BANDS * kStepsPerStage * 512;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;
    static constexpr int OUT_BYTES = OUT_BYTES_;                       // output staging (or the cluster split's landing slots)
    static constexpr int BAR_BYTES = (2 * STAGES + 2 * ACC + 1) * 8 + 16;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + OUT_BYTES + BAR_BYTES;
    // TMEM columns: accumulators first, then the scale columns (one set per smem stage, or a
    // single set that every stage reuses: the copies into it are ordered behind the MMAs that
    // read it because both are issued by one thread into the same pipe)
    static constexpr int SFA_SET_COLS = kStepsPerStage * 4;
    static constexpr int SFB_SET_COLS = kStepsPerStage * (BN / 32);
    static constexpr int SFA_COL0 = ACC_STRIDE + BN;
    static constexpr int SFB_COL0 = SFA_COL0 + SF_SETS * SFA_SET_COLS;
    static_assert(BN == 128 || BN == 256, "BN must be 128 or 256");
    static_assert(!PAIR || BN == 256, "the pair kernel uses 256 x 256 tiles");
    static_assert(SFB_COL0 + SF_SETS * SFB_SET_COLS <= kTmemCols, "TMEM budget");
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
    static_assert(STAGE_BYTES % 1024 == 0, "stage alignment");
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&b2);
}

// FULLK: K is a multiple of 256, so every stage holds four K-steps and the issue loop has no
// per-step condition (a run-time branch around each step costs the loop ~20 %, measured).
// EPI: kEpiPlain writes Y; kEpiSwiglu (BN = 256 only) turns every 32 accumulator columns -- 16 gate
// and 16 up values of one row -- into one 16-element block of h = bf16(silu(bf16(gate)) * bf16(up))
// and writes its NVFP4 codes and scale byte: the 4 bytes per element that Y would cost become 0.5625.
// kEpiClusterSplit / kEpiClusterSplitFew (decode-sized M, BN = 128, K a multiple of 256; they differ only in how
// shared memory is divided between stages and landing slots): the `split_k` CTAs of a cluster share
// ONE output tile along K -- CTA r runs K tiles [r, r + 1) * k_per_split -- so that a layer with fewer
// tiles than SMs still pulls its weights through every SM's load path and spreads the MMA issue work.
// CTAs 1.. push their fp32 partial sums into landing slots in CTA 0's shared memory with bulk copies
// that count their bytes on a barrier of CTA 0; CTA 0 waits for that barrier, adds the
// slots to its own accumulator in a fixed order, applies the scales and writes Y.  One tile per
// cluster; nothing goes through global memory, nothing has to be zeroed, and no fence is needed.
// For a handful of rows the same variant also takes A as bf16 (GemmParams::x): the four epilogue warps
// quantize each K tile of A straight into the stage buffer (codes in the 128-byte swizzle, scale bytes in
// the atom layout, bit for bit what the quantize kernel would have written), which removes that kernel
// and its launch from the chain; every CTA quantizes the K range it multiplies.
template <int BN, int STAGES, bool PAIR, bool FULLK, int EPI = kEpiPlain>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmSFA, const __grid_constant__ CUtensorMap tmSFB,
            const __grid_constant__ CUtensorMap tmY, const __grid_constant__ GemmParams p) {
    using C = GemmCfg<BN, STAGES, PAIR, cluster_split_slots(EPI) != 0 ? cluster_split_slots(EPI) * kClusterSplitSlotBytes : kDefaultOutBytes>;
    constexpr int ACC = C::ACC;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* out_s = smem + STAGES * C::STAGE_BYTES;                   // 1024-byte aligned
    uint64_t* bars = reinterpret_cast<uint64_t*>(out_s + C::OUT_BYTES);
    uint64_t* full = bars;                    // (leader's copy) every CTA's loads of a stage have landed
    uint64_t* empty = bars + STAGES;          // the MMAs have finished reading a stage
    uint64_t* tfull = bars + 2 * STAGES;      // accumulator complete
    uint64_t* tempty = tfull + ACC;           // (leader's copy) every CTA has drained the accumulator
    uint64_t* drain = tempty + ACC;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint64_t* cs_ready = reinterpret_cast<uint64_t*>(tmem_slot + 2);   // cluster split: the other CTAs' partial sums are in place

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;          // 0 = leader
    constexpr bool CSPLIT = EPI == kEpiClusterSplit || EPI == kEpiClusterSplitFew;
    static_assert(!CSPLIT || (BN == 128 && !PAIR && FULLK), "cluster split-K: 128 x 128 tiles, whole K tiles");
    const uint32_t csize = CSPLIT ? static_cast<uint32_t>(p.split_k) : 1u;    // CTAs that share a tile along K
    const uint32_t crank = CSPLIT ? ptx::cluster_ctarank() : 0u;              // which part of K is this CTA's
    const uint32_t unit_id = PAIR ? (blockIdx.x >> 1) : (CSPLIT ? blockIdx.x / csize : blockIdx.x);    // CTA or cluster index
    const uint32_t n_units = PAIR ? (gridDim.x >> 1) : (CSPLIT ? gridDim.x / csize : gridDim.x);
    const uint32_t m_units = PAIR ? (static_cast<uint32_t>(p.m_tiles) + 1u) >> 1 : static_cast<uint32_t>(p.m_tiles);
    const uint32_t split_k = CSPLIT ? 1u : static_cast<uint32_t>(p.split_k);
    const uint32_t total_tiles = m_units * static_cast<uint32_t>(p.n_tiles) * split_k;    // work items
    const uint32_t my_tiles = total_tiles > unit_id ? (total_tiles - unit_id + n_units - 1) / n_units : 0u;
    const int32_t cs_kt0 = static_cast<int32_t>(crank) * p.k_per_split;       // cluster split: this CTA's K tiles
    const int32_t cs_kt1 = min(cs_kt0 + p.k_per_split, p.k_tiles);
    const uint32_t k_tiles = CSPLIT ? static_cast<uint32_t>(cs_kt1 - cs_kt0)
                                    : static_cast<uint32_t>(p.k_per_split);              // K tiles per item
    const uint32_t total_it = my_tiles * k_tiles;
    const uint32_t peer_abort =
        PAIR ? ptx::mapa_shared(ptx::smem_u32(const_cast<uint32_t*>(abort_flag)), rank ^ 1u) : 0u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // the two producer threads of every CTA of the tile; with A quantized in the kernel, the W
            // producer and the four quantizing warps
            ptx::mbar_init(&full[s], (CSPLIT && p.x != nullptr) ? 5 : 2 * C::CTAS);
            ptx::mbar_init(&empty[s], 1);
        }
        for (int a = 0; a < ACC; ++a) {
            ptx::mbar_init(&tfull[a], 1);
            ptx::mbar_init(&tempty[a], 4 * C::CTAS);     // epilogue warps of every CTA of the tile
        }
        ptx::mbar_init(drain, 1);
        if (CSPLIT) {
            // completes when every other CTA's partial sums (its live 32-row quarters, all 128 columns) have landed
            const uint32_t live_q = static_cast<uint32_t>(min(p.M, kBM) + 31) >> 5;
            ptx::mbar_init(cs_ready, 1);
            if (crank == 0u) ptx::mbar_arrive_expect_tx(cs_ready, (csize - 1u) * live_q * kClusterSplitSlotBytes);
        }
        *abort_flag = 0u;
        ptx::fence_barrier_init();
    }
    if (warp == 6) {
        if (PAIR) { ptx::tmem_alloc_pair(tmem_slot, kTmemCols); ptx::tmem_relinquish_pair(); }
        else      { ptx::tmem_alloc(tmem_slot, kTmemCols);      ptx::tmem_relinquish(); }
    }
    ptx::tc_fence_before();
    // barriers and TMEM exist from here on (cluster split: the barrier-init fence above is what makes
    // CTA 0's barrier visible to the other CTAs' remote copies; the cluster barrier only has to order execution)
    if (PAIR) ptx::cluster_sync_all(); else if (CSPLIT) ptx::cluster_sync_relaxed(); else __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // CTA 0 leaves its own clock readings in the status block (words 2..9: cycle counter and wall clock
    // at start and end), so that the host can tell at which SM clock the kernel really ran -- under a
    // power cap the clock drops within microseconds, long before a management-library sample shows it
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        reinterpret_cast<unsigned long long*>(p.status)[1] = static_cast<unsigned long long>(clock64());
        reinterpret_cast<unsigned long long*>(p.status)[2] = ptx::globaltimer_ns();
    }
    // This kernel may have been started while the kernel in front of it (the activation quantizer or
    // another GEMM, which release their dependents early) was still working, and it releases its own
    // dependents right away: they all wait (pdl_wait) before they touch anything a predecessor may
    // still read or write.  Here every role waits at its first access to such memory: the A producer
    // before its first load, the epilogue before it reads the global scales or writes Y, the W producer
    // too -- unless the caller has said that the weights were complete long before (NVFP4_W_RESIDENT):
    // then the weight stream of this layer starts under the tail of the previous one.
    ptx::pdl_launch_dependents();

    // tile index -> (row unit, column tile).  Tiles are visited in groups of `group_m` row
    // units; inside a group the row unit varies fastest, then the column tile.  The CTAs that
    // run at the same time then share W tiles through L2, and the A rows of one group (sized
    // by the host to a fraction of L2) stay resident while the group sweeps all of W.
    const uint32_t group_m = static_cast<uint32_t>(p.group_m);
    const uint32_t tiles_per_group = group_m * static_cast<uint32_t>(p.n_tiles);
    auto tile_of = [&](uint32_t t, int32_t& um, int32_t& un, int32_t& ks) {
        const uint32_t item = unit_id + t * n_units;
        const uint32_t tile = item / split_k;
        ks = static_cast<int32_t>(item - tile * split_k);
        const uint32_t group = tile / tiles_per_group, r = tile - group * tiles_per_group;
        const uint32_t first = group * group_m;
        const uint32_t gsize = min(group_m, m_units - first);
        un = static_cast<int32_t>(r / gsize);
        um = static_cast<int32_t>(first + (r - static_cast<uint32_t>(un) * gsize));
    };

    if (warp == 4 || warp == 5) {
        // ------------------------------------------------------------ TMA producers
        if (lane == 0 && !(CSPLIT && warp == 4 && p.x != nullptr)) {
            const bool is_a = warp == 4;
            const uint32_t leader_full = PAIR ? ptx::mapa_shared(ptx::smem_u32(full), 0u) : 0u;
            const CUtensorMap* tm_codes = is_a ? &tmA : &tmB;
            const CUtensorMap* tm_sf = is_a ? &tmSFA : &tmSFB;
            ptx::prefetch_tensormap(tm_codes);
            ptx::prefetch_tensormap(tm_sf);
            const uint32_t code_off = is_a ? 0u : C::A_BYTES;
            const uint32_t sf_off = C::A_BYTES + C::B_BYTES + (is_a ? 0u : C::SFA_BYTES);
            const uint32_t tx = is_a ? (static_cast<uint32_t>(p.a_box_bytes) + C::SFA_BYTES) : (C::B_BYTES + C::SFB_BYTES);
            if (is_a || (p.flags & NVFP4_W_RESIDENT) == 0u) ptx::pdl_wait();
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t t = 0; ok && t < my_tiles; ++t) {
                int32_t um, un, ks;
                tile_of(t, um, un, ks);
                const int32_t a_band = PAIR ? 2 * um + static_cast<int32_t>(rank) : um;
                const int32_t code_row = is_a ? a_band * kBM : un * BN + static_cast<int32_t>(rank) * C::B_ROWS;
                const int32_t sf_band = is_a ? a_band : un * C::NB_BANDS;
                const int32_t kt_end = CSPLIT ? cs_kt1 : (ks + 1) * p.k_per_split;    // K tiles past the tensor load zeros
                for (int32_t kt = CSPLIT ? cs_kt0 : ks * p.k_per_split; kt < kt_end; ++kt, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!ptx::mbar_wait_bounded(&empty[s], ph ^ 1u, abort_flag, p.wait_limit_ns, peer_abort)) { ok = false; break; }
                    uint8_t* st = smem + s * C::STAGE_BYTES;
                    // rows / bands / k-atoms past the tensor are zero-filled by TMA
                    if (PAIR) {
                        const uint32_t bar = leader_full + s * 8u;
                        ptx::mbar_arrive_expect_tx_cluster(bar, tx);
                        ptx::tma_load_2d_pair(st + code_off, tm_codes, kt * kBKBytes, code_row, bar);
                        ptx::tma_load_3d_pair(st + sf_off, tm_sf, 0, kt * kStepsPerStage, sf_band, bar);
                    } else {
                        ptx::mbar_arrive_expect_tx(&full[s], tx);
                        ptx::tma_load_2d(st + code_off, tm_codes, kt * kBKBytes, code_row, &full[s]);
                        ptx::tma_load_3d(st + sf_off, tm_sf, 0, kt * kStepsPerStage, sf_band, &full[s]);
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
    } else if (warp == 6) {
        // ------------------------------------------------------------ MMA issuer
        // Issue-side rules (all measured on B200): the thread that issues tcgen05 work has to stay in
        // warp-convergent code -- inside a single-lane branch every operand pays a vector-to-uniform
        // move and [3 copies + 1 MMA] cost ~200 cycles to issue, in convergent code with only the
        // instruction predicated they cost ~135 and the tensor pipe (128 cycles per MMA) stays busy.
        // So the whole warp walks the loop; `lp` is non-zero in one elected lane, the same throughout.
        // The ring of stages is unrolled (every shared-memory and TMEM address is base + compile-time
        // constant; a rolled loop with run-time stage addresses measured 8 % slower), descriptors are a
        // fixed high word and an incremented low word, there are no divisions, and the next stage's
        // barrier is polled right after the first MMA of the current stage has been queued, when the
        // pipe has most work ahead of it.
        if (rank == 0) {
            const uint32_t lp = ptx::elect_one() ? 1u : 0u;
            // E2M1 x E2M1, E4M3 scales, K-major A and B; M = 128 (single) or 256 (pair), N = BN
            constexpr uint32_t idesc = (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                                       (static_cast<uint32_t>((PAIR ? 256 : 128) >> 4) << 24);
            // descriptor words (see ptx::smem_desc): codes use the 128-byte swizzle with 1024 bytes
            // between 8-row groups; scale atoms are unswizzled with 128 bytes between 8-row groups
            constexpr uint32_t kCodeHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            constexpr uint32_t kCodeLoFlags = (16u >> 4) << 16;
            constexpr uint32_t kScaleHi = (128u >> 4) | (1u << 14);
            const uint32_t smem_enc = (ptx::smem_u32(smem) & 0x3FFFFu) >> 4;      // stage 0, in 16-byte units
            auto desc = [](uint32_t lo, uint32_t hi) { return (static_cast<uint64_t>(hi) << 32) | lo; };
            const int32_t tail_steps = p.katoms - (p.k_tiles - 1) * kStepsPerStage;   // K-steps of a tile's last stage
            bool ok = true;
            uint32_t it = 0, kt = 0, tl = 0, ph = 0;
            bool have_full = false;          // the coming iteration's "stage full" was already observed
            while (ok && it < total_it) {
#pragma unroll
                for (int s = 0; s < STAGES; ++s) {
                    if (it >= total_it) break;
                    const uint32_t acc = tl & 1u;
                    if (kt == 0) {
                        // disjoint accumulators: wait until tile tl-2 (same accumulator) is drained;
                        // overlapping ones: until tile tl-1 has given up the shared columns
                        const uint32_t dep = C::OVERLAP ? tl - 1u : tl - 2u;
                        if (tl >= (C::OVERLAP ? 1u : 2u)) {
                            if (!ptx::mbar_wait_bounded(&tempty[dep & 1u], (dep >> 1) & 1u, abort_flag, p.wait_limit_ns, peer_abort)) { ok = false; break; }
                            ptx::tc_fence_after();
                        }
                    }
                    if (!have_full) {
                        if (!ptx::mbar_wait_bounded(&full[s], ph, abort_flag, p.wait_limit_ns, peer_abort)) { ok = false; break; }
                        ptx::tc_fence_after();
                    }
                    have_full = false;
                    const uint32_t st_enc = smem_enc + s * (C::STAGE_BYTES >> 4);
                    const uint32_t sfa_t = tmem_base + C::SFA_COL0 + (C::SF_SETS == 1 ? 0 : s) * C::SFA_SET_COLS;
                    const uint32_t sfb_t = tmem_base + C::SFB_COL0 + (C::SF_SETS == 1 ? 0 : s) * C::SFB_SET_COLS;
                    const uint32_t d_tmem = tmem_base + acc * C::ACC_STRIDE;
                    const bool last_kt = kt + 1 == k_tiles;
                    const int32_t steps = last_kt ? tail_steps : kStepsPerStage;
#pragma unroll
                    for (int j = 0; j < kStepsPerStage; ++j) {
                        if (FULLK || j < steps) {
                            // this step's scale atoms: shared -> TMEM (32 rows x 16 bytes each, replicated into
                            // the four lane quarters), then the MMA that reads them
                            const uint32_t sf_enc = st_enc + ((C::A_BYTES + C::B_BYTES + j * 512) >> 4);
                            // advancing K by 64 elements = 32 bytes inside the 128-byte swizzle row
                            const uint64_t a_desc = desc((st_enc + j * 2) | kCodeLoFlags, kCodeHi);
                            const uint64_t b_desc = desc((st_enc + (C::A_BYTES >> 4) + j * 2) | kCodeLoFlags, kCodeHi);
                            const uint32_t accum = (j == 0) ? (kt != 0u ? 1u : 0u) : 1u;
                            if (PAIR) {
                                ptx::tc_cp_32x128b_warpx4_pair_if(sfa_t + j * 4, desc(sf_enc, kScaleHi), lp);
                                ptx::tc_cp_32x128b_warpx4_pair_if(sfb_t + j * (BN / 32), desc(sf_enc + (C::SFA_BYTES >> 4), kScaleHi), lp);
                                if (C::NB_BANDS == 2)
                                    ptx::tc_cp_32x128b_warpx4_pair_if(sfb_t + j * (BN / 32) + 4,
                                                                      desc(sf_enc + ((C::SFA_BYTES + kStepsPerStage * 512) >> 4), kScaleHi), lp);
                                ptx::tc_mma_nvf4_pair_if(d_tmem, a_desc, b_desc, idesc, sfa_t + j * 4, sfb_t + j * (BN / 32), accum, lp);
                            } else {
                                ptx::tc_cp_32x128b_warpx4_if(sfa_t + j * 4, desc(sf_enc, kScaleHi), lp);
                                ptx::tc_cp_32x128b_warpx4_if(sfb_t + j * (BN / 32), desc(sf_enc + (C::SFA_BYTES >> 4), kScaleHi), lp);
                                if (C::NB_BANDS == 2)
                                    ptx::tc_cp_32x128b_warpx4_if(sfb_t + j * (BN / 32) + 4,
                                                                 desc(sf_enc + ((C::SFA_BYTES + kStepsPerStage * 512) >> 4), kScaleHi), lp);
                                ptx::tc_mma_nvf4_if(d_tmem, a_desc, b_desc, idesc, sfa_t + j * 4, sfb_t + j * (BN / 32), accum, lp);
                            }
                            if (j == 0 && it + 1 < total_it) {
                                // with this stage's first MMA queued: has the next stage landed?
                                const int ns = (s + 1 == STAGES) ? 0 : s + 1;
                                if (ptx::mbar_try_wait(&full[ns], ns == 0 ? ph ^ 1u : ph)) { ptx::tc_fence_after(); have_full = true; }
                            }
                        }
                    }
                    // stage reusable once these MMAs have read it; after the last K tile the accumulator is complete
                    if (PAIR) {
                        ptx::tc_commit_pair_if(&empty[s], 3, lp);
                        if (last_kt) ptx::tc_commit_pair_if(&tfull[acc], 3, lp);
                    } else {
                        ptx::tc_commit_if(&empty[s], lp);
                        if (last_kt) ptx::tc_commit_if(&tfull[acc], lp);
                    }
                    ++it;
                    if (last_kt) { kt = 0; ++tl; } else { ++kt; }
                }
                ph ^= 1u;
            }
            if (!ok) {
                // let issued MMAs finish before TMEM is freed
                if (PAIR) ptx::tc_commit_pair_if(drain, 1, lp); else ptx::tc_commit_if(drain, lp);
                for (int spin = 0; spin < (1 << 16) && !ptx::mbar_try_wait(drain, 0u); ++spin) {}
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp;                       // TMEM lanes this warp may read
        uint8_t* out_w = out_s + quarter * (2 * kOutPieceBytes);
        ptx::pdl_wait();                                // the scales may come from, and Y may still be read by, a predecessor
        const float g_a = __ldg(p.g_a);
        const bool out_f32 = (p.flags & NVFP4_OUT_F32) != 0u;
        const bool use_tma = p.tma_store != 0u;
        const uint32_t leader_tempty = PAIR ? ptx::mapa_shared(ptx::smem_u32(tempty), 0u) : ptx::smem_u32(tempty);
        if (use_tma && lane == 0) ptx::prefetch_tensormap(&tmY);
        if (blockIdx.x == 0 && warp == 0) {
            // global scales must be finite and positive; anything else is reported, not repaired
            bool bad = !(g_a > 0.0f && g_a <= 3.402823466e38f);
            for (int i = lane; i < p.nseg; i += 32) {
                const float gs = __ldg(p.g_seg + i);
                bad = bad || !(gs > 0.0f && gs <= 3.402823466e38f);
            }
            if (__any_sync(0xffffffffu, bad) && lane == 0) atomicExch(p.status, static_cast<uint32_t>(NVFP4_ERR_SCALE));
        }
        if (CSPLIT && p.x != nullptr && my_tiles != 0u) {
            // ---- A from bf16.  Block b of a K tile = (row, 16-element block) with b = row * 16 + block; thread t
            // takes blocks t, t + 128, ... (16 neighbouring threads read the 512 contiguous bytes of one row).
            // The tile after the current one is loaded and quantized into registers while the stage it goes
            // to is still being read by the tensor core; only the shared-memory stores wait for the stage.
            constexpr int NB = 2;                                     // blocks per thread: up to 16 rows
            const int nb = (p.a_box_bytes / kBKBytes) >> 3;           // ... of which this call uses rows / 8
            const float c1 = __fdiv_rn(1.0f, __fmul_rn(6.0f, g_a));
            const int32_t r0 = static_cast<int32_t>(threadIdx.x) >> 4, kb = static_cast<int32_t>(threadIdx.x) & 15;
            uint4 lo[NB], hi[NB];
            auto load_tile = [&](int32_t kt) {
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (b >= nb) break;
                    const int32_t r = r0 + 8 * b;
                    lo[b] = make_uint4(0u, 0u, 0u, 0u);
                    hi[b] = lo[b];
                    if (r < p.M) {
                        const uint4* src = reinterpret_cast<const uint4*>(p.x + static_cast<int64_t>(r) * p.ldx +
                                                                          static_cast<int64_t>(kt) * 256 + kb * 16);
                        lo[b] = __ldg(src);
                        hi[b] = __ldg(src + 1);
                    }
                }
            };
            load_tile(cs_kt0);
            bool ok = true;
            uint32_t itq = 0;
            for (int32_t kt = cs_kt0; ok && kt < cs_kt1; ++kt, ++itq) {
                uint2 w[NB];
                uint32_t s8[NB];
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (b >= nb) break;
                    const uint32_t hw[8] = {lo[b].x, lo[b].y, lo[b].z, lo[b].w, hi[b].x, hi[b].y, hi[b].z, hi[b].w};
                    // rows past M: zero codes, zero scale (without the quantizer: its division takes the slow path on 1 / 0)
                    w[b] = make_uint2(0u, 0u);
                    s8[b] = 0u;
                    if (r0 + 8 * b < p.M) w[b] = quantize_block(hw, g_a, c1, s8[b]);
                }
                if (kt + 1 < cs_kt1) load_tile(kt + 1);
                const uint32_t s = itq % STAGES, ph = (itq / STAGES) & 1u;
                if (lane == 0) ok = ptx::mbar_wait_bounded(&empty[s], ph ^ 1u, abort_flag, p.wait_limit_ns, 0u);
                ok = __shfl_sync(0xffffffffu, static_cast<int>(ok), 0) != 0;
                if (!ok) break;
                const uint32_t st = ptx::smem_u32(smem) + s * C::STAGE_BYTES;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int32_t r = r0 + 8 * b;
                    if (b < nb) {
                        // 8 code bytes: 16-byte chunk (kb / 2) XOR (row mod 8) of the row's 128-byte swizzle line
                        ptx::st_shared_v2(st + static_cast<uint32_t>(r * 128 + (((kb >> 1) ^ (r & 7)) << 4) + (kb & 1) * 8), w[b].x, w[b].y);
                        // scale byte: atom kb / 4 of the stage, (row mod 32) * 16 + (row / 32) * 4 + kb mod 4
                        ptx::st_shared_u8(st + static_cast<uint32_t>(C::A_BYTES + C::B_BYTES + (kb >> 2) * 512 + (r & 31) * 16 +
                                                                     (r >> 5) * 4 + (kb & 3)), s8[b]);
                    }
                }
                ptx::fence_proxy_async_smem();                        // the tensor core reads these bytes through the async proxy
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&full[s]);
            }
        }
        uint32_t pieces_stored = 0;
        for (uint32_t t = 0; t < my_tiles; ++t) {
            int32_t um, un, ks;
            tile_of(t, um, un, ks);
            const int32_t n0 = un * BN;
            const uint32_t acc = t & 1u, aph = (t >> 1) & 1u;
            // global scale of columns n0 + 32 i + lane, i = 0 .. BN/32-1, in registers
            float areg[BN / 32];
#pragma unroll
            for (int i = 0; i < BN / 32; ++i) {
                const int32_t n = n0 + i * 32 + lane;
                float a = 0.0f;
                if (n < p.N) {
                    int sgi = 0;
                    while (sgi + 1 < p.nseg && n >= p.seg_end[sgi]) ++sgi;
                    a = __fmul_rn(g_a, __ldg(p.g_seg + sgi));
                }
                areg[i] = a;
            }
            // the scales are in registers BEFORE the wait below (otherwise the compiler sinks their loads to
            // the first use, and a global-memory latency lands between "accumulator full" and the first store)
#pragma unroll
            for (int i = 0; i < BN / 32; ++i) asm volatile("" : "+f"(areg[i]));
            // one lane polls (try_wait suspends the thread in hardware between looks): 128 threads
            // spinning on the barrier would take shared-memory cycles away from the MMAs
            bool ok = true;
            if (lane == 0) ok = ptx::mbar_wait_bounded(&tfull[acc], aph, abort_flag, p.wait_limit_ns, peer_abort);
            ok = __shfl_sync(0xffffffffu, static_cast<int>(ok), 0) != 0;
            if (!ok) break;
            ptx::tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * C::ACC_STRIDE;
            const int32_t row0 = (PAIR ? 2 * um + static_cast<int32_t>(rank) : um) * kBM + quarter * 32;
            constexpr int NP = BN / kOutPieceCols;
            if (EPI == kEpiSwiglu) {
                // ---- fused SwiGLU + quantize.  Piece order as in the plain epilogue (the columns shared by
                // the two accumulators go first); each piece of 64 columns holds two blocks of h.
                const float a_gate = __fmul_rn(g_a, __ldg(p.g_seg)), a_up = __fmul_rn(g_a, __ldg(p.g_seg + 1));
                const float g_h = __ldg(p.g_h);
                const float c1_h = __fdiv_rn(1.0f, __fmul_rn(6.0f, g_h));
                const int32_t row = row0 + lane;
                const int32_t m_pad = (p.M + 127) & ~127;
                const int first_piece = (C::OVERLAP && acc == 0u) ? NP - 1 : 0;
                uint32_t ra[64], rb[64];
                ptx::tmem_ld_32x64(t_row + first_piece * kOutPieceCols, ra);
#pragma unroll
                for (int k = 0; k < NP; ++k) {
                    uint32_t (&cur)[64] = (k & 1) ? rb : ra;
                    uint32_t (&nxt)[64] = (k & 1) ? ra : rb;
                    const int pc = (first_piece + k) % NP;
                    ptx::tmem_ld_wait();
                    if (k + 1 < NP) ptx::tmem_ld_32x64(t_row + ((pc + 1) % NP) * kOutPieceCols, nxt);
                    if (C::OVERLAP ? (k == 0) : (k + 1 == NP)) {
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (PAIR) ptx::mbar_arrive_cluster(leader_tempty + acc * 8u);
                            else      ptx::mbar_arrive(&tempty[acc]);
                        }
                    }
                    const int32_t col0 = n0 + pc * kOutPieceCols;             // interleaved column of this piece
                    if (col0 < p.N && row < m_pad) {
                    const int32_t hc0 = col0 >> 1;                            // first h column of this piece (32 of them)
                    uint2 words[2];
                    uint32_t s8[2];
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        uint32_t hw[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            // gate / up rounded to bf16 exactly as the plain epilogue would store them (two values per
                            // multiply and per rounding instruction; the rounded pair is unpacked again by shift and mask)
                            float g0 = __uint_as_float(cur[b * 32 + 2 * i]), g1 = __uint_as_float(cur[b * 32 + 2 * i + 1]);
                            float u0 = __uint_as_float(cur[b * 32 + 16 + 2 * i]), u1 = __uint_as_float(cur[b * 32 + 16 + 2 * i + 1]);
                            mul_f32x2(g0, g1, a_gate, a_gate);
                            mul_f32x2(u0, u1, a_up, a_up);
                            const uint32_t gb = pack_bf16x2(g0, g1), ub = pack_bf16x2(u0, u1);
                            float h0, h1;
                            silu_mul2(__uint_as_float(gb << 16), __uint_as_float(gb & 0xFFFF0000u), __uint_as_float(ub << 16),
                                      __uint_as_float(ub & 0xFFFF0000u), h0, h1);
                            hw[i] = pack_bf16x2(h0, h1);
                        }
                        words[b] = quantize_block(hw, g_h, c1_h, s8[b]);
                        if (p.dbg_h != nullptr && row < p.M)
                            stg256(reinterpret_cast<uint16_t*>(p.dbg_h) + static_cast<int64_t>(row) * p.inner + hc0 + b * 16, hw);
                    }
                    const int32_t kb0 = hc0 >> 4;                             // even: both scale bytes sit in one 16-bit word
                    uint8_t* sfp = p.h_sf + (static_cast<int64_t>(row >> 7) * p.h_katoms + (kb0 >> 2)) * 512 + (row & 31) * 16 +
                                   ((row & 127) >> 5) * 4 + (kb0 & 3);
                    if (row < p.M) {
                        *reinterpret_cast<uint4*>(p.h_codes + static_cast<int64_t>(row) * (p.inner >> 1) + (hc0 >> 1)) =
                            make_uint4(words[0].x, words[0].y, words[1].x, words[1].y);
                        *reinterpret_cast<uint16_t*>(sfp) = static_cast<uint16_t>(s8[0] | (s8[1] << 8));
                        if (p.dbg_y != nullptr) {
                            __nv_bfloat16* yr = reinterpret_cast<__nv_bfloat16*>(p.dbg_y) + static_cast<int64_t>(row) * p.N + col0;
#pragma unroll
                            for (int j = 0; j < 64; ++j)
                                yr[j] = __float2bfloat16_rn(__fmul_rn(__uint_as_float(cur[j]), (j & 16) ? a_up : a_gate));
                        }
                    } else {
                        *reinterpret_cast<uint16_t*>(sfp) = 0;                 // rows that pad the last 128-row band: zero scales
                    }
                    }
                }
                continue;
            }
            // one lane writes 64 finished values of its row (16-byte stores where the row allows them)
            auto store_row_piece = [&](const float (&v)[64], int32_t row, int32_t col0) {
                const bool vec_ok = (reinterpret_cast<uintptr_t>(p.y) & 15u) == 0 && (p.ldy & (out_f32 ? 3 : 7)) == 0 &&
                                    col0 + kOutPieceCols <= p.N;
                if (out_f32) {
                    float* yr = reinterpret_cast<float*>(p.y) + static_cast<int64_t>(row) * p.ldy + col0;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (vec_ok) {
                            *reinterpret_cast<float4*>(yr + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (col0 + 4 * j + e < p.N) yr[4 * j + e] = v[4 * j + e];
                        }
                    }
                } else {
                    __nv_bfloat16* yr = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<int64_t>(row) * p.ldy + col0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (vec_ok) {
                            *reinterpret_cast<uint4*>(yr + 8 * j) =
                                make_uint4(pack_bf16x2(v[8 * j], v[8 * j + 1]), pack_bf16x2(v[8 * j + 2], v[8 * j + 3]),
                                           pack_bf16x2(v[8 * j + 4], v[8 * j + 5]), pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
                        } else {
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (col0 + 8 * j + e < p.N) yr[8 * j + e] = __float2bfloat16_rn(v[8 * j + e]);
                        }
                    }
                }
            };
            if (CSPLIT) {
                // ---- cluster split-K.  Slot (c - 1) * live_q + quarter of CTA 0 holds CTA c's partial sums of
                // that quarter as float4 cells [column / 4][lane]: written and read 16 bytes per lane, no bank conflicts.
                const int32_t row = row0 + lane;
                const bool quarter_live = row0 < p.M;              // warp-uniform: rows past M are never sent or stored
                const uint32_t live_q = static_cast<uint32_t>(min(p.M, kBM) + 31) >> 5;
                const uint32_t cell0 = ptx::smem_u32(out_s) + static_cast<uint32_t>(lane * 16);
                if (crank != 0u) {
                    if (quarter_live) {
                        // registers -> this CTA's own stage buffers (idle: its K loop is over) -> one bulk copy
                        // per quarter into the slot, which counts its bytes on CTA 0's barrier
                        const uint32_t slot = (crank - 1u) * live_q + static_cast<uint32_t>(quarter);
                        const uint32_t local = ptx::smem_u32(smem) + static_cast<uint32_t>(quarter) * kClusterSplitSlotBytes;
#pragma unroll 1
                        for (int pc = 0; pc < NP; ++pc) {
                            uint32_t r[64];
                            __syncwarp();
                            ptx::tmem_ld_32x64(t_row + pc * kOutPieceCols, r);
                            ptx::tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                ptx::st_shared_v4(local + static_cast<uint32_t>((pc * 16 + j) * 512 + lane * 16), r[4 * j],
                                                  r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                        }
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0)
                            ptx::bulk_copy_to_cluster(ptx::mapa_shared(ptx::smem_u32(out_s) + slot * kClusterSplitSlotBytes, 0u), local,
                                                      kClusterSplitSlotBytes, ptx::mapa_shared(ptx::smem_u32(cs_ready), 0u));
                    }
                    continue;
                }
                // CTA 0.  While the other CTAs' copies are on their way (about 1 000 cycles for 16 KB) the
                // per-column global scales go into a small table in the stage area (idle by now), from where
                // they come back as broadcast reads (a shuffle per column costs more than the whole sum).
                const uint32_t scale_tab = ptx::smem_u32(smem) + static_cast<uint32_t>(quarter) * (BN * 4);
                if (quarter_live) {
#pragma unroll
                    for (int i = 0; i < BN / 32; ++i) ptx::st_shared_f32(scale_tab + static_cast<uint32_t>((i * 32 + lane) * 4), areg[i]);
                    __syncwarp();                                  // the table is complete before any lane reads it
                }
                if (lane == 0) ok = ptx::mbar_wait_bounded(cs_ready, 0u, abort_flag, p.wait_limit_ns, 0u);
                ok = __shfl_sync(0xffffffffu, static_cast<int>(ok), 0) != 0;
                if (!ok) break;
                if (!quarter_live) continue;
#pragma unroll 1
                for (int pc = 0; pc < NP; ++pc) {
                    const int32_t col0 = n0 + pc * kOutPieceCols;
                    if (col0 >= p.N) break;
                    uint32_t r[64];
                    float v[64];
                    __syncwarp();
                    ptx::tmem_ld_32x64(t_row + pc * kOutPieceCols, r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 64; ++j) v[j] = __uint_as_float(r[j]);
                    for (uint32_t c = 1; c < csize; ++c) {         // fixed order: the sum does not depend on timing
                        const uint32_t cell = cell0 + ((c - 1u) * live_q + static_cast<uint32_t>(quarter)) * kClusterSplitSlotBytes +
                                              static_cast<uint32_t>(pc * 16 * 512);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const uint4 q = ptx::ld_shared_v4(cell + static_cast<uint32_t>(j * 512));
                            v[4 * j] = __fadd_rn(v[4 * j], __uint_as_float(q.x));
                            v[4 * j + 1] = __fadd_rn(v[4 * j + 1], __uint_as_float(q.y));
                            v[4 * j + 2] = __fadd_rn(v[4 * j + 2], __uint_as_float(q.z));
                            v[4 * j + 3] = __fadd_rn(v[4 * j + 3], __uint_as_float(q.w));
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const uint4 sc = ptx::ld_shared_v4(scale_tab + static_cast<uint32_t>((pc * kOutPieceCols + 4 * j) * 4));
                        v[4 * j] = __fmul_rn(v[4 * j], __uint_as_float(sc.x));
                        v[4 * j + 1] = __fmul_rn(v[4 * j + 1], __uint_as_float(sc.y));
                        v[4 * j + 2] = __fmul_rn(v[4 * j + 2], __uint_as_float(sc.z));
                        v[4 * j + 3] = __fmul_rn(v[4 * j + 3], __uint_as_float(sc.w));
                    }
                    if (use_tma) {
                        // this piece's part of the first landing slot of this quarter is in registers by now:
                        // it serves as the staging buffer of the TMA store (rows past M are clipped there)
                        uint8_t* buf = out_s + quarter * kClusterSplitSlotBytes + pc * (kClusterSplitSlotBytes / NP);
                        __syncwarp();
                        const uint32_t row_s = ptx::smem_u32(buf) + lane * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c)     // 128-byte swizzle: 16-byte chunk index XOR (row mod 8)
                            ptx::st_shared_v4(row_s + ((c ^ (lane & 7)) << 4), pack_bf16x2(v[8 * c + 0], v[8 * c + 1]),
                                              pack_bf16x2(v[8 * c + 2], v[8 * c + 3]), pack_bf16x2(v[8 * c + 4], v[8 * c + 5]),
                                              pack_bf16x2(v[8 * c + 6], v[8 * c + 7]));
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            ptx::tma_store_2d(&tmY, buf, col0, row0);
                            ptx::bulk_commit_group();
                        }
                    } else if (row < p.M) {
                        store_row_piece(v, row, col0);
                    }
                }
                continue;
            }
            if (split_k > 1u) {
                // ---- split-K: add this item's partial sums to the tile's fp32 buffer; the last of
                // the split_k arrivals (per lane quarter) finishes the tile
                const int32_t row = row0 + lane;
                const bool row_ok = row < p.M;
                float* prow = p.partial + static_cast<int64_t>(row) * p.ldp + n0;
#pragma unroll 1
                for (int pc = 0; pc < NP; ++pc) {
                    uint32_t r[64];
                    __syncwarp();
                    ptx::tmem_ld_32x64(t_row + pc * kOutPieceCols, r);
                    ptx::tmem_ld_wait();
                    if (row_ok && n0 + pc * kOutPieceCols < p.N) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            ptx::red_add_v4_f32(prow + pc * kOutPieceCols + 4 * j, __uint_as_float(r[4 * j]),
                                                __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                                                __uint_as_float(r[4 * j + 3]));
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) ptx::mbar_arrive_cluster(leader_tempty + acc * 8u);
                    else      ptx::mbar_arrive(&tempty[acc]);
                }
                __threadfence();                                   // my adds are visible before my ticket
                uint32_t ticket = 0;
                uint32_t* counter = p.counters + (static_cast<uint32_t>(um) * p.n_tiles + un) * 4u + quarter;
                if (lane == 0) ticket = atomicAdd(counter, 1u);
                ticket = __shfl_sync(0xffffffffu, ticket, 0);
                if (ticket != split_k - 1u) continue;              // somebody else finishes this quarter
                __threadfence();                                   // their adds are visible before my reads
#pragma unroll 1
                for (int pc = 0; pc < NP; ++pc) {
                    const int32_t col0 = n0 + pc * kOutPieceCols;
                    if (col0 >= p.N) break;
                    float v[64];
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            float4* q4 = reinterpret_cast<float4*>(prow + pc * kOutPieceCols + 4 * j);
                            const float4 q = __ldcg(q4);
                            __stcg(q4, make_float4(0.0f, 0.0f, 0.0f, 0.0f));       // leave the buffer zero for the next call
                            v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 64; ++j) v[j] = 0.0f;
                    }
#pragma unroll
                    for (int j = 0; j < 64; ++j)
                        v[j] = __fmul_rn(v[j], __shfl_sync(0xffffffffu, areg[pc * 2 + (j >> 5)], j & 31));
                    if (!row_ok) continue;
                    store_row_piece(v, row, col0);
                }
                __syncwarp();
                if (lane == 0) *counter = 0u;                      // ready for the next call
                continue;
            }
            // piece order: with overlapping accumulators the shared columns go first (the last piece
            // of the lower accumulator, the first piece of the upper one)
            const uint32_t scale_tab = ptx::smem_u32(out_s) + 4 * 2 * kOutPieceBytes + static_cast<uint32_t>(quarter) * (kOutPieceCols * 4);
            auto drain = [&](auto first_c) {
            constexpr int first_piece = decltype(first_c)::value;
            uint32_t ra[64], rb[64];
            ptx::tmem_ld_32x64(t_row + first_piece * kOutPieceCols, ra);
#pragma unroll
            for (int k = 0; k < NP; ++k) {
                uint32_t (&cur)[64] = (k & 1) ? rb : ra;
                uint32_t (&nxt)[64] = (k & 1) ? ra : rb;
                const int pc = (first_piece + k) % NP;               // this piece; next is (pc + 1) % NP
                ptx::tmem_ld_wait();
                if (k + 1 < NP) ptx::tmem_ld_32x64(t_row + ((pc + 1) % NP) * kOutPieceCols, nxt);
                if (C::OVERLAP ? (k == 0) : (k + 1 == NP)) {
                    // overlapping: the shared columns are in registers, the next tile's MMAs may start;
                    // disjoint: the whole accumulator is in registers
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (PAIR) ptx::mbar_arrive_cluster(leader_tempty + acc * 8u);
                        else      ptx::mbar_arrive(&tempty[acc]);
                    }
                }
                const int32_t col0 = n0 + pc * kOutPieceCols;
                if (col0 >= p.N || row0 >= p.M) continue;        // warp-uniform
                // the 64 column scales of this piece go through a 256-byte table in shared memory and come
                // back as broadcast reads: 2 stores + 16 loads per lane instead of 64 shuffles (this warp
                // shares its scheduler with a producer or with the warp that issues the MMAs)
                float v[64];
                __syncwarp();
                ptx::st_shared_f32(scale_tab + static_cast<uint32_t>(lane * 4), areg[pc * 2]);
                ptx::st_shared_f32(scale_tab + static_cast<uint32_t>(128 + lane * 4), areg[pc * 2 + 1]);
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const uint4 sc = ptx::ld_shared_v4(scale_tab + static_cast<uint32_t>(j * 16));
                    v[4 * j] = __uint_as_float(cur[4 * j]);
                    v[4 * j + 1] = __uint_as_float(cur[4 * j + 1]);
                    v[4 * j + 2] = __uint_as_float(cur[4 * j + 2]);
                    v[4 * j + 3] = __uint_as_float(cur[4 * j + 3]);
                    mul_f32x2(v[4 * j], v[4 * j + 1], __uint_as_float(sc.x), __uint_as_float(sc.y));       // two products per instruction
                    mul_f32x2(v[4 * j + 2], v[4 * j + 3], __uint_as_float(sc.z), __uint_as_float(sc.w));
                }
                if (use_tma) {
                    uint8_t* buf = out_w + (pieces_stored & 1u) * kOutPieceBytes;
                    if (pieces_stored >= 2u) {
                        if (lane == 0) ptx::bulk_wait_group_read<1>();   // the store that last used `buf` has read it
                        __syncwarp();
                    }
                    const uint32_t row_s = ptx::smem_u32(buf) + lane * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c)     // 128-byte swizzle: 16-byte chunk index XOR (row mod 8)
                        ptx::st_shared_v4(row_s + ((c ^ (lane & 7)) << 4), pack_bf16x2(v[8 * c + 0], v[8 * c + 1]),
                                          pack_bf16x2(v[8 * c + 2], v[8 * c + 3]), pack_bf16x2(v[8 * c + 4], v[8 * c + 5]),
                                          pack_bf16x2(v[8 * c + 6], v[8 * c + 7]));
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_2d(&tmY, buf, col0, row0);
                        ptx::bulk_commit_group();
                    }
                    ++pieces_stored;
                } else {
                    // plain stores: float32 output, or bf16 rows that TMA cannot address
                    const int32_t row = row0 + lane;
                    if (row < p.M) {
#pragma unroll
                        for (int j = 0; j < 64; ++j) {
                            if (col0 + j < p.N) {
                                if (out_f32)
                                    reinterpret_cast<float*>(p.y)[static_cast<int64_t>(row) * p.ldy + col0 + j] = v[j];
                                else
                                    reinterpret_cast<__nv_bfloat16*>(p.y)[static_cast<int64_t>(row) * p.ldy + col0 + j] =
                                        __float2bfloat16_rn(v[j]);
                            }
                        }
                    }
                }
            }
            };
            if (C::OVERLAP && acc == 0u) drain(std::integral_constant<int, NP - 1>{});
            else                         drain(std::integral_constant<int, 0>{});
        }
        // every output store has read its shared-memory source before the CTA goes away (the writes
        // themselves are complete, like any other global write, when the kernel is)
        if (use_tma && lane == 0) ptx::bulk_wait_group_read<0>();
    }

    // ---------------------------------------------------------------- teardown
    // a CTA that gave up may still have copies and MMAs in flight (its own or its partner's,
    // which signal this CTA's barriers): give them time to land before anything is torn down
    if (*abort_flag != 0u) __nanosleep(50000);
    ptx::tc_fence_before();
    // (cluster split: CTA 0 arrives here only after the copies into its shared memory have landed -- or,
    // having given up, after the sleep above -- so the CTAs they read from are still alive while they run;
    // no data passes through this barrier, so it carries no memory ordering)
    if (PAIR) ptx::cluster_sync_all(); else if (CSPLIT) ptx::cluster_sync_relaxed(); else __syncthreads();   // nobody touches TMEM or a partner's barriers after this
    if (warp == 6) {
        ptx::tc_fence_after();
        if (PAIR) ptx::tmem_dealloc_pair(tmem_base, kTmemCols); else ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag != 0u) atomicExch(p.status, static_cast<uint32_t>(NVFP4_ERR_TIMEOUT));
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        reinterpret_cast<unsigned long long*>(p.status)[3] = static_cast<unsigned long long>(clock64());
        reinterpret_cast<unsigned long long*>(p.status)[4] = ptx::globaltimer_ns();
    }
}

}  // namespace nvfp4
