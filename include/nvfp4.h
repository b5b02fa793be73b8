/*
 * nvfp4.h -- C ABI of the B200 (sm_100a) NVFP4 W4A4 linear-layer library.
 *
 * The path (paper: Background, "NVFP4"; Section 6, "Per-module calibration vs.
 * fused-GEMM scaling"):
 *
 *   bf16 activations --nvfp4_quantize_act--> E2M1 codes + one E4M3 scale per
 *   16-element block (+ an FP32 per-tensor global scale)
 *   --nvfp4_linear--> block-scaled FP4 GEMM against weights quantized once by
 *   nvfp4_quantize_weight, with ONE GLOBAL SCALE PER FUSED MODULE applied to that
 *   module's slice of output columns in the epilogue.
 *
 * Conventions for every entry point
 *   - Pointers named d_* are DEVICE pointers; everything else is host memory.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream).  No call synchronises the device except
 *     nvfp4_device_status.  No call allocates or frees device memory.
 *   - The caller owns every buffer; the library keeps no pointer after the call
 *     returns other than cached TMA descriptors keyed by (address, shape), which
 *     hold no reference.
 *   - Host-detectable misuse returns a status before anything is launched.
 *     Nothing throws across this boundary.
 *   - Quantized tensor layout:  codes are row-major [rows, K/2] bytes, element k
 *     of a row in byte k/2, low nibble for even k.  Scale bytes (E4M3, one per
 *     16 consecutive k) are stored either
 *       NVFP4_SF_LINEAR: row-major [rows, K/16], or
 *       NVFP4_SF_MMA:    the order the block-scaled tensor-core instruction reads:
 *                        512-byte atoms of 128 rows x 4 blocks, byte offset of
 *                        (r, b) inside its atom = (r%32)*16 + ((r%128)/32)*4 + b%4,
 *                        atoms of one 128-row band contiguous along K; rows are
 *                        padded to a multiple of 128 and blocks to a multiple of
 *                        4, padding bytes are 0x00.
 *     nvfp4_sf_bytes gives the buffer size for either.
 *   - Global scales are "decode direction": x ~= e2m1 * e4m3 * g.  They must be
 *     finite and > 0.
 */
#ifndef NVFP4_H_
#define NVFP4_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NVFP4_OK = 0,
    NVFP4_ERR_NULL = 1,        /* a required pointer is NULL */
    NVFP4_ERR_SHAPE = 2,       /* a size is negative, or K is not a multiple of 16 (GEMM: 64) */
    NVFP4_ERR_ALIGN = 3,       /* a pointer or leading dimension breaks the stated alignment */
    NVFP4_ERR_SEGMENTS = 4,    /* segment table is not a sorted, gap-free cover of [0, N) */
    NVFP4_ERR_WORKSPACE = 5,   /* workspace missing or too small */
    NVFP4_ERR_ARCH = 6,        /* current device is not compute capability 10.x */
    NVFP4_ERR_CUDA = 7,        /* a CUDA runtime/driver call or a launch failed */
    NVFP4_ERR_TIMEOUT = 8,     /* a bounded wait inside a kernel ran out (see nvfp4_device_status) */
    NVFP4_ERR_LAYOUT = 9,      /* unknown scale layout / the GEMM needs NVFP4_SF_MMA */
    NVFP4_ERR_SCALE = 10       /* a global scale read on the device was not finite and > 0 (see nvfp4_device_status) */
} nvfp4_status;

/* One fused module's slice of the output columns (= rows of the weight matrix). */
typedef struct {
    int64_t col_begin;
    int64_t col_count;
} nvfp4_segment;

#define NVFP4_MAX_SEGMENTS 32

typedef enum { NVFP4_SF_LINEAR = 0, NVFP4_SF_MMA = 1 } nvfp4_sf_layout;

/* flags for nvfp4_linear* */
#define NVFP4_OUT_BF16 0u     /* Y is bf16 (default)                                  */
#define NVFP4_OUT_F32  1u     /* Y is float32 (testing aid: no output rounding)       */
#define NVFP4_WS_ZEROED 2u    /* caller's promise: the workspace was zero-filled once (e.g. cudaMemset) and has
                                 since been written by this library only.  Lets decode-sized calls (M <= 256)
                                 split K over several CTAs, which meet in the workspace and leave it zero again.
                                 After NVFP4_ERR_TIMEOUT zero the workspace before the next call with this flag. */
#define NVFP4_W_RESIDENT 4u   /* caller's promise: the weight operand (codes, scales, global scales) was complete before
                                 the work in front of this call in the stream was submitted -- true of model weights,
                                 false of a tensor quantized by the preceding call.  Lets the kernel start fetching
                                 weights while the kernel in front of it still runs (programmatic dependent launch);
                                 activations, global scales of activations and outputs are still ordered as usual. */

/*
 * Workspace layout (the same for every entry point and every problem size, so one zero-filled
 * workspace can serve calls of different shapes, e.g. the K = 5120 and K = 17408 layers of one model):
 *   [0, 256)                                    status block; its first word is the status flag
 *   [256, 256 + NVFP4_SPLIT_RESERVE_BYTES)      split-K counters and fp32 partial sums.  Used only with
 *                                               NVFP4_WS_ZEROED, and only as far as the workspace reaches;
 *                                               a call whose split-K area would not fit does not split K
 *   [256 + NVFP4_SPLIT_RESERVE_BYTES, ...)      nvfp4_linear_bf16 only: the quantized activations
 * Nothing the library writes outside the split-K part can land on it, and every call that uses that
 * part leaves it zero again: the NVFP4_WS_ZEROED promise, once true, stays true.
 */
#define NVFP4_SPLIT_RESERVE_BYTES (5u * 1024u * 1024u)

/* Size in bytes of the scale buffer for a [rows, K] tensor in `layout` (K % 16 == 0). */
size_t nvfp4_sf_bytes(int64_t rows, int64_t K, nvfp4_sf_layout layout);

/*
 * Global-scale calibration (paper: one FP32 scale per tensor / per linear module;
 * the value amax/(6*448) makes the block that holds the tensor maximum use the
 * largest E4M3 scale).
 *   d_x     bf16 [rows, cols], row stride ld elements (ld >= cols)
 *   d_g     out: *d_g = amax / 2688 in binary32, or 1.0f if the tensor is all zero
 *   d_amax  out, optional (may be NULL): max |x|
 * Errors: NULL d_x/d_g, negative sizes, ld < cols.  rows*cols == 0 gives g = 1.
 */
nvfp4_status nvfp4_calibrate(const void* d_x, int64_t rows, int64_t cols, int64_t ld,
                             float* d_g, float* d_amax, void* stream);

/*
 * On-the-fly activation quantization (paper: Background, "NVFP4": E2M1 values, one
 * E4M3 scale per 16-element block set to blockmax/6, one FP32 scale per tensor).
 * Per block of 16 consecutive k, in binary32 with round-to-nearest-even and no
 * fused multiply-add:
 *     s8   = e4m3_rne_sat( bmax * (1 / (6 * g)) )
 *     code = e2m1_rne_sat( x * (1 / (e4m3(s8) * g)) )     (all codes 0 if s8 == 0)
 *   d_x      bf16 [M, K], row stride ld elements; 32-byte aligned, ld % 16 == 0 (256-bit loads)
 *   d_g      in: the tensor's global scale (device scalar)
 *   d_codes  out: [M, K/2] bytes, 16-byte aligned
 *   d_sf     out: nvfp4_sf_bytes(M, K, layout) bytes (padding is written as zero)
 * Errors: NULL pointers, K % 16 != 0, misalignment, unknown layout.  M == 0 is a no-op.
 */
nvfp4_status nvfp4_quantize_act(const void* d_x, int64_t M, int64_t K, int64_t ld,
                                const float* d_g, uint8_t* d_codes, uint8_t* d_sf,
                                nvfp4_sf_layout layout, void* stream);

/*
 * Activation quantization fused into its producer (paper: Background -- the MLP is among the
 * 496 quantized linears, so the down projection's input silu(gate)*up is quantized on every
 * call; Section 9 names activation quantization as the overhead to remove).  Reads the fused
 * gate/up GEMM output once and writes only codes and scales: h is never stored in bf16.
 *     h = bf16_rne( silu(gate) * up ),  silu(g) = g / (1 + exp(-g)),  then exactly nvfp4_quantize_act(h)
 * The paper fixes no arithmetic for the activation (it is upstream of the quantized linears, in
 * bf16).  The kernel evaluates it in binary32 with the hardware's approximate exp2 and
 * reciprocal; the bf16 result equals the correctly rounded definition for all but a small
 * fraction of elements and is never more than one bf16 ulp away (results below about 2^-100 in
 * magnitude, from gates below -88, come out as zeros of the right sign).  Codes and scales are the
 * exact quantization of the h the kernel formed.
 *   d_gate_up  bf16 [M, 2*inner], gate in columns [0, inner), up in [inner, 2*inner); row
 *              stride ld >= 2*inner; 32-byte aligned, ld % 16 == 0, inner % 16 == 0
 *   d_g        in: global scale of h (calibrated offline, as for any activation)
 *   d_codes    out [M, inner/2]; d_sf out nvfp4_sf_bytes(M, inner, layout)
 *   d_h        optional (may be NULL), testing aid: out bf16 [M, inner] row-major, 32-byte aligned --
 *              the tensor h that was quantized
 * Errors: as nvfp4_quantize_act.
 */
nvfp4_status nvfp4_swiglu_quantize(const void* d_gate_up, int64_t M, int64_t inner, int64_t ld,
                                   const float* d_g, uint8_t* d_codes, uint8_t* d_sf,
                                   nvfp4_sf_layout layout, void* d_h, void* stream);

/*
 * Activation quantization fused into RMSNorm (paper: Background / Setup -- norms are excluded from
 * quantization and stay bf16 upstream of every quantized linear, so the in-projections quantize
 * a normalised residual stream on every call).  One pass over x from HBM:
 *     y = bf16_rne( x * rstd * w ),  rstd = 1 / sqrt(mean_k(x^2) + eps),  then nvfp4_quantize_act(y)
 * The paper fixes no arithmetic for the norm; the kernel sums the squares in binary32 (per lane,
 * then across the warp) and multiplies in binary32: y equals the correctly rounded definition for
 * all but a small fraction of elements, never more than one bf16 ulp away.  Codes and scales are the
 * exact quantization of the y the kernel formed.
 *   d_x       bf16 [M, K], row stride ld; 32-byte aligned, ld % 16 == 0
 *   d_weight  bf16 [K] (the norm's gain), 32-byte aligned;  eps >= 0
 *   d_g       in: global scale of y (calibrated offline);  outputs as nvfp4_quantize_act
 *   d_y       optional (may be NULL), testing aid: out bf16 [M, K] row-major, 32-byte aligned -- the
 *             tensor y that was quantized
 * Errors: as nvfp4_quantize_act, plus NULL / misaligned weight, negative or NaN eps.
 */
nvfp4_status nvfp4_rmsnorm_quantize(const void* d_x, int64_t M, int64_t K, int64_t ld, const void* d_weight,
                                    float eps, const float* d_g, uint8_t* d_codes, uint8_t* d_sf,
                                    nvfp4_sf_layout layout, void* d_y, void* stream);

/*
 * Offline weight quantization, same format, blocks along K, with one global scale
 * per fused module (paper: Section 6 -- the calibration tool keeps one FP32 global
 * scale per linear module; the modules are later served as one fused GEMM).
 *   d_w      bf16 [N, K], row stride ld; rows are the output features
 *   segs     host array of nseg segments covering rows [0, N) in order, no gaps
 *   d_g_seg  device float[nseg]: INPUT when calibrate_segments == 0; OUTPUT
 *            (per-segment amax/2688) when calibrate_segments != 0
 * Errors: as nvfp4_quantize_act, plus NVFP4_ERR_SEGMENTS, nseg < 1 or > NVFP4_MAX_SEGMENTS.
 */
nvfp4_status nvfp4_quantize_weight(const void* d_w, int64_t N, int64_t K, int64_t ld,
                                   const nvfp4_segment* segs, int nseg, float* d_g_seg,
                                   int calibrate_segments, uint8_t* d_codes, uint8_t* d_sf,
                                   nvfp4_sf_layout layout, void* stream);

/*
 * Weight quantization for the MLP's fused gate/up projection with the output rows INTERLEAVED
 * 16 by 16: output rows 32 b .. 32 b + 15 are gate rows 16 b .. 16 b + 15 and rows 32 b + 16 ..
 * 32 b + 31 the matching up rows.  Each module keeps its own global scale (paper: Section 6, one
 * FP32 global scale per linear module).  Quantization is per row, so codes and scale bytes are
 * those nvfp4_quantize_weight gives for the same rows; only the row order differs.  A GEMM
 * against weights in this order (nvfp4_linear_swiglu) produces, per 32 output columns, the 16
 * gate and 16 up values of one 16-element block of silu(gate) * up.
 *   d_w           bf16 [2 * inner, K]: gate rows [0, inner), then up rows [inner, 2 * inner); row stride ld
 *   d_g_gate_up   device float[2]: INPUT when calibrate_segments == 0, else OUTPUT (amax / 2688 of each module)
 *   d_codes       out [2 * inner, K / 2];  d_sf out nvfp4_sf_bytes(2 * inner, K, NVFP4_SF_MMA)
 * Errors: as nvfp4_quantize_weight; inner % 16 != 0 is NVFP4_ERR_SHAPE.
 */
nvfp4_status nvfp4_quantize_weight_gate_up(const void* d_w, int64_t inner, int64_t K, int64_t ld,
                                           float* d_g_gate_up, int calibrate_segments,
                                           uint8_t* d_codes, uint8_t* d_sf, void* stream);

/*
 * The MLP's gate/up projection with SwiGLU and the activation quantization of the down
 * projection's input inside the GEMM epilogue (paper: Background -- the MLP is among the 496
 * quantized linears; Section 9 names activation quantization as the overhead to remove): the
 * gate/up output is never written in bf16, only the NVFP4 codes and scale bytes of
 *     h = bf16_rne( silu(gate) * up ),  gate = bf16_rne(acc * g_a * g_gate),  up = bf16_rne(acc * g_a * g_up)
 * exactly as nvfp4_linear followed by nvfp4_swiglu_quantize would produce them (same roundings).
 *   d_a_codes/d_a_sf   activations [M, K] (NVFP4_SF_MMA);  d_g_a their global scale
 *   d_w_codes/d_w_sf   from nvfp4_quantize_weight_gate_up;  d_g_gate_up device float[2]
 *   d_g_h              in: global scale of h (calibrated offline, as for any activation)
 *   d_h_codes          out [M, inner / 2], 16-byte aligned
 *   d_h_sf             out nvfp4_sf_bytes(M, inner, NVFP4_SF_MMA) bytes (every byte is written)
 *   d_dbg_y, d_dbg_h   optional (may be NULL), testing aids, 32-byte aligned: bf16 [M, 2 * inner] gate/up in the
 *                      interleaved column order, and bf16 [M, inner] the tensor h that was quantized
 *   d_workspace        as for nvfp4_linear (256 bytes suffice)
 * Requirements: K % 64 == 0, inner % 64 == 0.  Errors and the status word as for nvfp4_linear.
 */
nvfp4_status nvfp4_linear_swiglu(const uint8_t* d_a_codes, const uint8_t* d_a_sf, const float* d_g_a,
                                 int64_t M, int64_t K,
                                 const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t inner,
                                 const float* d_g_gate_up, const float* d_g_h,
                                 uint8_t* d_h_codes, uint8_t* d_h_sf, void* d_dbg_y, void* d_dbg_h,
                                 void* d_workspace, size_t workspace_bytes, void* stream);

/*
 * Checkpoint-side repair (paper: Section 6, the fix applied to the released checkpoint: every
 * fused group gets one shared global scale and each module's ratio to it is multiplied into that
 * module's E4M3 block scales, which are rounded again; the paper bounds that re-rounding at 6.2 %):
 * lets a GEMM with ONE global scale serve a fused group whose modules were calibrated separately.
 *     g* = max_j g_seg[j];   s'_b = e4m3_rne_sat( e4m3(s_b) * (g_seg[j] / g*) )   (binary32)
 * Codes are unchanged.  Afterwards nvfp4_linear with the single segment [0, N) and g* reproduces
 * the per-module result up to the re-rounding of the scales; the per-segment epilogue of
 * nvfp4_linear remains the exact form of the repair.
 *   d_sf_in / d_sf_out  scale bytes of the [N, K] weight in `layout` (may be the same buffer)
 *   segs, d_g_seg       the modules and their calibrated scales (segs: host array)
 *   d_g_shared          out: g* (device scalar)
 * Errors: NULL, shape, layout, NVFP4_ERR_SEGMENTS, misaligned scale pointers.
 */
nvfp4_status nvfp4_harmonize_scales(const uint8_t* d_sf_in, int64_t N, int64_t K, nvfp4_sf_layout layout,
                                    const nvfp4_segment* segs, const float* d_g_seg, int nseg,
                                    uint8_t* d_sf_out, float* d_g_shared, void* stream);

/*
 * Statistics of a bf16 tensor at NVFP4 granularity (paper: Table "stats" -- max/RMS, kurtosis,
 * share of "1-hot" 16-element blocks with max/RMS > 3, relative error of quantizing the tensor
 * alone).  Writes seven doubles to d_out (8-byte aligned device memory):
 *   [0] sum x^2   [1] sum x^4   [2] sum (x - dequant(quant(x)))^2   [3] max |x|
 *   [4] number of blocks   [5] number of 1-hot blocks   [6] scratch
 * from which  max/RMS = [3] / sqrt([0]/n),  kurtosis = n [1] / [0]^2,  1-hot share = [5]/[4],
 * error = sqrt([2]/[0]).  Per-block sums are binary32 in a fixed order, blocks are added in double
 * by atomics (the last bits depend on arrival order).
 *   d_x  bf16 [rows, cols], row stride ld; 32-byte aligned, ld % 16 == 0, cols % 16 == 0;  d_g as usual
 */
nvfp4_status nvfp4_tensor_stats(const void* d_x, int64_t rows, int64_t cols, int64_t ld, const float* d_g,
                                double* d_out, void* stream);

/*
 * The W4A4 linear layer (paper: Background, "NVFP4": the GEMM runs on 4-bit tensor
 * cores; Section 6: per-module global scales meeting in one fused GEMM -- here each
 * segment of output columns gets its own global scale in the epilogue, which is
 * exact, instead of one scale for the whole fused GEMM):
 *     Y[m, n] = round_out( (sum_k a_hat[m,k] * w_hat[n,k]) * g_a * g_seg[seg(n)] )
 * where a_hat/w_hat are code*block-scale products, accumulated in FP32 on the tensor
 * cores.
 *   d_a_codes/d_a_sf   activations [M, K] as written by nvfp4_quantize_act with NVFP4_SF_MMA
 *   d_w_codes/d_w_sf   weights [N, K] as written by nvfp4_quantize_weight with NVFP4_SF_MMA
 *   d_g_a              device scalar; d_g_seg device float[nseg]
 *   segs               host array (copied into the launch; need not outlive the call)
 *   d_y                out [M, N], row stride ldy elements, bf16 or float per `flags`
 *   d_workspace        at least 256 bytes, 16-byte aligned; its first word is a status flag read
 *                      by nvfp4_device_status.  nvfp4_linear_workspace_bytes(...) is the size that
 *                      also holds the split-K area used with NVFP4_WS_ZEROED (more than 256 bytes
 *                      only for M <= 256; never more than 256 + NVFP4_SPLIT_RESERVE_BYTES)
 * Requirements: K % 64 == 0; code pointers 16-byte aligned; scale pointers 16-byte aligned.
 * Errors: see nvfp4_status; M == 0 or N == 0 is a no-op.  The kernel checks on the device that g_a and
 * every g_seg[j] is finite and > 0; if not, the status word becomes NVFP4_ERR_SCALE and Y is unspecified.
 */
nvfp4_status nvfp4_linear(const uint8_t* d_a_codes, const uint8_t* d_a_sf, const float* d_g_a,
                          int64_t M, int64_t K,
                          const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                          const nvfp4_segment* segs, const float* d_g_seg, int nseg,
                          void* d_y, int64_t ldy, uint32_t flags,
                          void* d_workspace, size_t workspace_bytes, void* stream);

size_t nvfp4_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int nseg);

/*
 * The same layer fed with bf16 activations: quantization runs inside the call
 * (paper: Section 9, "Decode overhead" -- activation quantization is the overhead
 * that matters at small batch), codes and scales live in the workspace.
 *   d_x   bf16 [M, K], row stride ldx, 32-byte aligned, ldx % 16 == 0
 * For M = 1 (and M = 2 where K is not a multiple of 256) the call is one weight-streaming kernel on
 * the CUDA cores that quantizes the activations itself (same codes); for up to 8 rows with K a
 * multiple of 256 it is one tensor-core kernel whose CTAs quantize the K tiles of A they multiply
 * (same codes again); both use only the status word of the workspace.  Above that it is the quantize
 * kernel followed by the tensor-core GEMM, which starts its prologue while the quantizer still runs.
 * With NVFP4_W_RESIDENT the GEMM also fetches weights before the work in front of the call is done.
 *   d_workspace  nvfp4_linear_bf16_workspace_bytes(M, N, K, nseg) bytes (status block, split-K
 *                reserve, codes and scales of the activations), 16-byte aligned
 * Every argument is checked before anything is enqueued.
 */
nvfp4_status nvfp4_linear_bf16(const void* d_x, int64_t ldx, const float* d_g_a,
                               int64_t M, int64_t K,
                               const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                               const nvfp4_segment* segs, const float* d_g_seg, int nseg,
                               void* d_y, int64_t ldy, uint32_t flags,
                               void* d_workspace, size_t workspace_bytes, void* stream);

size_t nvfp4_linear_bf16_workspace_bytes(int64_t M, int64_t N, int64_t K, int nseg);

/*
 * nvfp4_linear_bf16 for callers that cannot provide a workspace.  (The paper has no
 * counterpart for this call; it exists for integration only.)
 *
 * Some hosts of this library may not allocate device memory at the point where they
 * run a layer: an inference server that has handed all device memory to its own pool,
 * a plug-in running inside another framework's execution callback, code between
 * allocator-frozen phases of a serving loop.  They have nowhere to get the scratch
 * buffer that nvfp4_linear_bf16 needs for the quantized activations.  This variant
 * takes the same inputs and outputs and keeps that scratch in a fixed array inside
 * the library's own device image, NVFP4_STATIC_SCRATCH_BYTES large; every GPU that
 * loads the library holds the array until the process exits.
 *
 *   - It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The array is laid out like any workspace (status block, split-K reserve, quantized
 *     activations).  Sizes whose quantized activations (rows padded to 128, K/2 bytes of codes per
 *     row, plus their scales) do not fit behind the reserve are rejected with NVFP4_ERR_WORKSPACE
 *     before anything is launched; the limit fits decode-sized batches, e.g. M = 640 rows at
 *     K = 17408.
 *   - The first call on each device looks up the array's device address (once, with that
 *     device current).  Make that first call outside of any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents.  What must start
 *     at zero is kept at zero by the library itself: the split-K part is left zero by every call
 *     that uses it, whatever shapes earlier calls had.  Two calls that overlap on the
 *     GPU (different streams, no dependency) race on the array: serialise them.
 *   - nvfp4_static_status(stream) is nvfp4_device_status for this array.  If it reports a failure
 *     (a timeout, a bad global scale) it also clears the status word and re-zeroes the split-K
 *     part, so the next call starts clean; a caller has no other handle on the array.
 * Everything else (arguments, layouts, errors) is as for nvfp4_linear_bf16.
 */
#define NVFP4_STATIC_SCRATCH_BYTES (12u * 1024u * 1024u)
nvfp4_status nvfp4_linear_bf16_static(const void* d_x, int64_t ldx, const float* d_g_a,
                                      int64_t M, int64_t K,
                                      const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                                      const nvfp4_segment* segs, const float* d_g_seg, int nseg,
                                      void* d_y, int64_t ldy, uint32_t flags, void* stream);
nvfp4_status nvfp4_static_status(void* stream);

/*
 * Clears the status word of a workspace (enqueue before the first nvfp4_linear* that
 * uses it; the kernels only ever set it).
 */
nvfp4_status nvfp4_workspace_reset(void* d_workspace, size_t workspace_bytes, void* stream);

/*
 * Synchronises `stream` and returns the status word of the workspace: NVFP4_OK,
 * NVFP4_ERR_TIMEOUT if a kernel gave up on one of its bounded waits, or NVFP4_ERR_SCALE if a kernel
 * read a global scale that is not finite and > 0 (the output is then unspecified; the CUDA context
 * stays usable).
 */
nvfp4_status nvfp4_device_status(const void* d_workspace, void* stream);

/*
 * Gated delta-rule recurrence, clean and perturbed trajectory in lockstep (paper: Background, Eq. 1-2;
 * Section 5.3 and Appendix "Error propagation": one clean FP32 trajectory and perturbed ones on
 * identical inputs, state error over time).  Per value head h, with K = V = 128, in binary32:
 *     g_t = -exp(A_log[h]) * softplus(a_t + dt_bias[h]);  alpha_t = exp(g_t);  beta_t = sigmoid(b_t)
 *     S_t = alpha_t S_{t-1} + beta_t k_t (v_t - S_{t-1}^T k_t)^T;   o_t = S_t^T (q_t / sqrt(128));   S_0 = 0
 * run once on (q, k, v, a, b) and once on (q2, k2, v2, a2, b2) -- the same projections computed another
 * way, e.g. through the NVFP4 layer -- and compared every `sample_every` tokens:
 *     rel_state[s, h] = ||S2 - S||_F / ||S||_F,   rel_out[s, h] = ||o2 - o|| / ||o||   at token (s+1)*sample_every - 1
 *   d_q, d_k    float [T, Hk, 128], l2-normalised per head (the caller's job);  d_v float [T, Hv, 128]
 *   d_a, d_b    float [T, Hv] gate pre-activations;  d_A_log, d_dt_bias float [Hv]
 *   Hv % Hk == 0: value head h reads query/key head h / (Hv / Hk)
 *   impulse_step >= 0: after that token the second trajectory's state is scaled by (1 + impulse_rel), once
 *                      (the paper's one-off state perturbation); < 0: none
 *   d_rel_state, d_rel_out   out float [T / sample_every, Hv]
 *   d_final_state            optional (may be NULL) out float [2, Hv, 128 (k), 128 (v)]
 * Any second-trajectory pointer may equal its clean counterpart.  Errors: NULL, T < 0, Hv % Hk != 0,
 * sample_every < 1, impulse_rel <= -1.
 */
nvfp4_status nvfp4_gdn_lockstep(const float* d_q, const float* d_k, const float* d_v, const float* d_a, const float* d_b,
                                const float* d_q2, const float* d_k2, const float* d_v2, const float* d_a2, const float* d_b2,
                                const float* d_A_log, const float* d_dt_bias, int64_t T, int Hk, int Hv,
                                int64_t impulse_step, float impulse_rel, int64_t sample_every,
                                float* d_rel_state, float* d_rel_out, float* d_final_state, void* stream);

/*
 * Measurement aid: the SM clock the last tensor-core GEMM launched on this workspace really ran at
 * (its first CTA's cycle counter over the wall clock, both read inside the kernel and left in the
 * status block), and that CTA's lifetime in microseconds -- from its start, which may lie under the
 * tail of the kernel in front of it, to its end.  Under a power cap the clock drops within
 * microseconds, long before a management-library sample shows it.  Synchronises `stream`.
 */
nvfp4_status nvfp4_last_gemm_clock(const void* d_workspace, double* sm_mhz, double* kernel_us, void* stream);

/*
 * Time limit of every wait inside the GEMM kernel, in nanoseconds (0 restores the default of
 * 2 s).  A CTA whose wait runs out stops issuing work, lets what it has in flight finish, frees
 * its tensor memory and raises NVFP4_ERR_TIMEOUT in the workspace status word; the kernel
 * returns and the CUDA context stays usable.  Process-wide.  A limit shorter than a memory
 * round trip makes a correct launch give up, which is how the failure path is tested.
 */
nvfp4_status nvfp4_set_wait_limit_ns(uint64_t limit_ns);

/*
 * Failure-path self-test: one CTA waits, with the same bounded wait the GEMM uses, on a barrier
 * that nothing ever completes, for at most limit_ns (1 .. 1e9), then writes NVFP4_ERR_TIMEOUT to
 * the workspace status word and returns normally.  Read the result with nvfp4_device_status.
 */
nvfp4_status nvfp4_selftest_bounded_wait(void* d_workspace, size_t workspace_bytes, uint64_t limit_ns,
                                         void* stream);

/* Number of this library's kernel launches enqueued so far by this process. */
uint64_t nvfp4_launch_count(void);

/*
 * Tile shape of the GEMM kernel: 0 = choose from the problem size (default), otherwise
 * one of the values that nvfp4_gemm_variants() lists ("value=description,...").
 * Process-wide; meant for benchmarking and tests.  Errors: NVFP4_ERR_SHAPE.
 */
nvfp4_status nvfp4_set_gemm_variant(int variant);
const char* nvfp4_gemm_variants(void);

const char* nvfp4_status_string(nvfp4_status s);

#ifdef __cplusplus
}
#endif
#endif /* NVFP4_H_ */
