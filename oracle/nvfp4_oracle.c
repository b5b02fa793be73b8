/*
 * CPU oracle for the NVFP4 W4A4 linear layer.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, step-by-step restatement of what the path computes, written
 * from the paper's definition of the format (Background, "NVFP4" paragraph:
 * E2M1 values, one E4M3 scale per 16-element block set to blockmax/6, one FP32
 * scale per tensor) and of the fused-GEMM global-scale problem (Section 6,
 * "Per-module calibration vs. fused-GEMM scaling").  It shares no code, table
 * or constant generator with the CUDA library and must never be called from the
 * product path: only the tests, the smoke check and the benchmark's CPU-baseline
 * leg use it.
 *
 * Floating point: every '*' and '/' marked "f32" below is one IEEE-754 binary32
 * operation, round-to-nearest-even, no fused multiply-add (compile with
 * -ffp-contract=off and without -ffast-math), subnormals kept.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py except
 * the paper's own probe figures 0.35/0.57 (they need its checkpoint): for
 * those, "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* bf16 <-> f32 (bf16 is the top half of a binary32)                          */
/* ------------------------------------------------------------------------- */
static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* double -> bf16, round-to-nearest-even, done directly on the double so that
 * there is a single rounding (no trip through binary32). */
uint16_t orc_f64_to_bf16(double v) {
    if (v != v) return 0x7FC0;
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7F80;
    int e;
    (void)frexp(a, &e);          /* a = m * 2^e, m in [0.5,1)  -> floor(log2 a) = e-1 */
    int E = e - 1;
    if (E < -126) E = -126;      /* subnormal bf16: fixed quantum 2^-133 */
    double q = nearbyint(ldexp(a, 7 - E));   /* RNE; integer in [0, 256] */
    if (q >= 256.0) { q = 128.0; E += 1; }
    if (E > 127) return sign | 0x7F80;
    uint32_t qi = (uint32_t)q;
    if (qi < 128) return sign | (uint16_t)qi;                     /* subnormal or zero */
    return sign | (uint16_t)(((uint32_t)(E + 127) << 7) | (qi - 128));
}

void orc_f64_to_bf16_n(const double* v, int64_t n, uint16_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f64_to_bf16(v[i]);
}

/* ------------------------------------------------------------------------- */
/* E2M1: 1 sign, 2 exponent, 1 mantissa bit.  Background, "NVFP4".            */
/* ------------------------------------------------------------------------- */
float orc_e2m1_decode(uint8_t c) {
    int s = (c >> 3) & 1, e = (c >> 1) & 3, m = c & 1;
    float mag = (e == 0) ? 0.5f * (float)m : ldexpf(1.0f + 0.5f * (float)m, e - 1);
    return s ? -mag : mag;
}

/* nearest representable magnitude; a tie goes to the code whose mantissa bit is
 * 0 (round-to-nearest-even); anything above 6, infinities included, saturates
 * to 6; the sign bit of the input is kept (so -tiny -> 0x8). */
uint8_t orc_e2m1_encode(float y) {
    uint8_t sign = signbit(y) ? 8 : 0;
    double a = fabs((double)y);
    if (a != a) return 0x7;                     /* NaN: unspecified by the method */
    if (a >= 6.0) return sign | 0x7;            /* saturate (also keeps the distances below exact) */
    int best = 0;
    double bestd = INFINITY;
    for (int c = 0; c < 8; ++c) {
        double d = fabs(a - (double)orc_e2m1_decode((uint8_t)c));
        if (d < bestd || (d == bestd && (c & 1) == 0)) { best = c; bestd = d; }
    }
    return sign | (uint8_t)best;
}

/* ------------------------------------------------------------------------- */
/* E4M3 ("fn" flavour: bias 7, no infinity, 0x7F = NaN, max finite 448).      */
/* ------------------------------------------------------------------------- */
float orc_e4m3_decode(uint8_t b) {
    int s = b >> 7, e = (b >> 3) & 15, m = b & 7;
    float mag;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) mag = ldexpf((float)m, -9);              /* m/8 * 2^-6 */
    else        mag = ldexpf(8.0f + (float)m, e - 10);   /* (1+m/8) * 2^(e-7) */
    return s ? -mag : mag;
}

/* non-negative input (block scales are never negative); RNE, saturating. */
uint8_t orc_e4m3_encode(float v) {
    if (v != v) return 0x7F;
    double a = (double)v;
    if (a <= 0.0) return 0x00;
    if (a >= 464.0) return 0x7E;     /* 464 is the midpoint above 448; the tie goes to the even 448 */
    int e;
    (void)frexp(a, &e);
    int E = e - 1;                   /* floor(log2 a) */
    if (E < -6) {                    /* subnormal range: quantum 2^-9 */
        int q = (int)nearbyint(ldexp(a, 9));          /* RNE, 0..8 */
        return (uint8_t)q;           /* q == 8 is 0x08 = 2^-6, the smallest normal */
    }
    int q = (int)nearbyint(ldexp(a, 3 - E));          /* RNE, 8..16 */
    if (q == 16) { q = 8; E += 1; }
    return (uint8_t)(((E + 7) << 3) | (q - 8));
}

/* ------------------------------------------------------------------------- */
/* Global-scale calibration: g = amax / (6 * 448); an all-zero tensor gets 1. */
/* ------------------------------------------------------------------------- */
void orc_calibrate(const uint16_t* x, int64_t rows, int64_t cols, int64_t ld,
                   float* amax_out, float* g_out) {
    float amax = 0.0f;
    #pragma omp parallel for reduction(max : amax) schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float a = fabsf(bf16_to_f32(x[r * ld + c]));
            if (a > amax) amax = a;
        }
    *amax_out = amax;
    *g_out = (amax == 0.0f) ? 1.0f : amax / 2688.0f;          /* f32 divide */
}

/* ------------------------------------------------------------------------- */
/* Quantize rows [0,rows) of a bf16 matrix, blocks of 16 along the columns.   */
/* g_row[r] is the global scale that row r uses (activations: all equal;      */
/* weights: the scale of the fused segment the row belongs to).               */
/* Outputs: codes [rows, cols/2] (low nibble = even column), scale bytes      */
/* [rows, cols/16] row-major.                                                 */
/* ------------------------------------------------------------------------- */
int orc_quantize(const uint16_t* x, int64_t rows, int64_t cols, int64_t ld,
                 const float* g_row, uint8_t* codes, uint8_t* sf) {
    if (cols % 16 != 0) return 1;
    const int64_t nb = cols / 16;
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const float g = g_row[r];
        const float c1 = 1.0f / (6.0f * g);                    /* f32 mul, f32 divide */
        for (int64_t b = 0; b < nb; ++b) {
            const uint16_t* xb = x + r * ld + b * 16;
            float bmax = 0.0f;
            for (int i = 0; i < 16; ++i) {
                float a = fabsf(bf16_to_f32(xb[i]));
                if (a > bmax) bmax = a;
            }
            const float sfv = bmax * c1;                        /* f32 mul */
            const uint8_t s8 = orc_e4m3_encode(sfv);
            sf[r * nb + b] = s8;
            uint8_t c[16];
            if (s8 == 0) {
                for (int i = 0; i < 16; ++i) c[i] = 0;
            } else {
                const float sdec = orc_e4m3_decode(s8);
                const float d = sdec * g;                       /* f32 mul */
                const float q = 1.0f / d;                       /* f32 divide */
                for (int i = 0; i < 16; ++i) {
                    const float y = bf16_to_f32(xb[i]) * q;     /* f32 mul */
                    c[i] = orc_e2m1_encode(y);
                }
            }
            for (int j = 0; j < 8; ++j)
                codes[r * (cols / 2) + b * 8 + j] = (uint8_t)(c[2 * j] | (c[2 * j + 1] << 4));
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Producer fusion for the MLP: h = silu(gate) * up, rounded to bf16, is what  */
/* the down projection quantizes.  The activation sits upstream of the         */
/* quantized linears, in bf16, and the paper fixes no arithmetic for it: the   */
/* oracle is the definition, evaluated in double and rounded ONCE to bf16:     */
/*     silu(g) = g / (1 + exp(-g));   h = bf16_rne( silu(g) * u )              */
/* A kernel that evaluates it in binary32 may differ from this by one bf16 ulp */
/* on a small fraction of elements; the comparison allows exactly that.        */
/* ------------------------------------------------------------------------- */
double orc_silu_mul(double g, double u) {
    return g / (1.0 + exp(-g)) * u;
}

/* gate_up: bf16 [rows, 2*inner] (gate in columns [0, inner), up in [inner, 2*inner)), row */
/* stride ld; h: bf16 [rows, inner].                                                        */
void orc_swiglu_bf16(const uint16_t* gate_up, int64_t rows, int64_t inner, int64_t ld, uint16_t* h) {
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < inner; ++c)
            h[r * inner + c] = orc_f64_to_bf16(orc_silu_mul((double)bf16_to_f32(gate_up[r * ld + c]),
                                                            (double)bf16_to_f32(gate_up[r * ld + inner + c])));
}

/* ------------------------------------------------------------------------- */
/* Producer fusion for the in-projections: their input is RMSNorm(x) * w (the  */
/* norms stay bf16 upstream of every quantized linear).  The paper fixes no    */
/* arithmetic for it; the oracle is the definition in double, rounded once:    */
/*     y[k] = bf16_rne( x[k] / sqrt( mean_k(x^2) + eps ) * w[k] )              */
/* ------------------------------------------------------------------------- */
void orc_rmsnorm_bf16(const uint16_t* x, int64_t rows, int64_t cols, int64_t ld, const uint16_t* w, double eps,
                      uint16_t* y) {
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double ss = 0.0;
        for (int64_t k = 0; k < cols; ++k) {
            const double v = (double)bf16_to_f32(x[r * ld + k]);
            ss += v * v;
        }
        const double rstd = 1.0 / sqrt(ss / (double)cols + eps);
        for (int64_t k = 0; k < cols; ++k)
            y[r * cols + k] = orc_f64_to_bf16((double)bf16_to_f32(x[r * ld + k]) * rstd * (double)bf16_to_f32(w[k]));
    }
}

/* x_hat = e2m1(code) * e4m3(scale) * g, evaluated in double (every factor is a
 * binary32 with few significant bits, so the double product is exact). */
void orc_dequantize(const uint8_t* codes, const uint8_t* sf, const float* g_row,
                    int64_t rows, int64_t cols, double* out) {
    const int64_t nb = cols / 16;
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < cols; ++k) {
            uint8_t byte = codes[r * (cols / 2) + k / 2];
            uint8_t c = (k & 1) ? (byte >> 4) : (byte & 15);
            out[r * cols + k] = (double)orc_e2m1_decode(c) *
                                (double)orc_e4m3_decode(sf[r * nb + k / 16]) * (double)g_row[r];
        }
}

/* ------------------------------------------------------------------------- */
/* Statistics at NVFP4 granularity (the columns of the paper's Table "stats"): */
/* max/RMS, kurtosis, share of "1-hot" blocks (block max/RMS > 3, i.e. one     */
/* value holds more than 9/16 of the block's energy) and the relative error of */
/* quantizing the tensor alone.  Everything is the definition in double:       */
/*   sum x^2, sum x^4, sum (x - x_hat)^2 with x_hat from orc_quantize /        */
/*   orc_dequantize's formula, the maximum, and per block: bmax^2 * 16 > 9 * (block's sum x^2). */
/* (All of x^2, bmax^2 * 16 and 9 * sum are exact in double for bf16 inputs,   */
/* so the 1-hot count has no rounding in it.)                                  */
/* out: {sum x^2, sum x^4, sum err^2, amax, blocks, 1-hot blocks}.             */
/* ------------------------------------------------------------------------- */
int orc_stats(const uint16_t* x, int64_t rows, int64_t cols, int64_t ld, float g, double* out) {
    if (cols % 16 != 0) return 1;
    double t2 = 0.0, t4 = 0.0, te = 0.0, hot = 0.0, amax = 0.0;
    const float c1 = 1.0f / (6.0f * g);                         /* as in orc_quantize */
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < cols / 16; ++b) {
            const uint16_t* xb = x + r * ld + b * 16;
            double s2 = 0.0, bmax = 0.0;
            float bmaxf = 0.0f;
            for (int i = 0; i < 16; ++i) {
                const double v = (double)bf16_to_f32(xb[i]);
                s2 += v * v;
                t4 += (v * v) * (v * v);
                if (fabs(v) > bmax) { bmax = fabs(v); bmaxf = fabsf(bf16_to_f32(xb[i])); }
            }
            t2 += s2;
            if (bmax > amax) amax = bmax;
            if (bmax * bmax * 16.0 > 9.0 * s2) hot += 1.0;
            /* quantize this block exactly as orc_quantize does, dequantize as orc_dequantize does */
            const uint8_t s8 = orc_e4m3_encode(bmaxf * c1);
            const float sdec = orc_e4m3_decode(s8);
            const float q = 1.0f / (sdec * g);
            for (int i = 0; i < 16; ++i) {
                const float xv = bf16_to_f32(xb[i]);
                const double xh = (s8 == 0) ? 0.0
                    : (double)orc_e2m1_decode(orc_e2m1_encode(xv * q)) * (double)sdec * (double)g;
                const double e = (double)xv - xh;
                te += e * e;
            }
        }
    out[0] = t2; out[1] = t4; out[2] = te; out[3] = amax;
    out[4] = (double)(rows * (cols / 16)); out[5] = hot;
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Checkpoint-side repair of Section 6: give a fused group ONE global scale    */
/* (the maximum of its modules' scales) and fold each module's ratio into its  */
/* E4M3 block scales, re-rounding them:                                        */
/*     g* = max_j g_j ;  r_j = g_j / g*  (f32 divide) ;                        */
/*     s'_b = e4m3_rne_sat( e4m3(s_b) * r_j )   (f32 multiply)                 */
/* Codes are untouched.  sf / sf_out: [rows, nb] row-major; g_row[r] is the    */
/* scale of the module that row r belongs to.                                  */
/* ------------------------------------------------------------------------- */
float orc_harmonize_scales(const uint8_t* sf, int64_t rows, int64_t nb, const float* g_row, uint8_t* sf_out) {
    float gstar = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        if (g_row[r] > gstar) gstar = g_row[r];
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const float ratio = g_row[r] / gstar;                              /* f32 divide */
        for (int64_t b = 0; b < nb; ++b)
            sf_out[r * nb + b] = orc_e4m3_encode(orc_e4m3_decode(sf[r * nb + b]) * ratio);   /* f32 multiply */
    }
    return gstar;
}

/* ------------------------------------------------------------------------- */
/* Scale-byte storage order the block-scaled tensor-core instruction reads:   */
/* 128 rows x 4 blocks form one 512-byte atom; atoms of one 128-row band are  */
/* contiguous along K; rows padded to 128, blocks to 4, padding bytes zero.   */
/* ------------------------------------------------------------------------- */
int64_t orc_sf_mma_bytes(int64_t rows, int64_t cols) {
    int64_t nb = cols / 16;
    return ((rows + 127) / 128) * ((nb + 3) / 4) * 512;
}

int64_t orc_sf_mma_index(int64_t r, int64_t b, int64_t cols) {
    int64_t nb = cols / 16, katoms = (nb + 3) / 4;
    int64_t atom = (r / 128) * katoms + b / 4;
    int64_t rr = r % 128;
    return atom * 512 + (rr % 32) * 16 + (rr / 32) * 4 + (b % 4);
}

void orc_sf_to_mma(const uint8_t* sf_linear, int64_t rows, int64_t cols, uint8_t* sf_mma) {
    int64_t nb = cols / 16;
    memset(sf_mma, 0, (size_t)orc_sf_mma_bytes(rows, cols));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < nb; ++b)
            sf_mma[orc_sf_mma_index(r, b, cols)] = sf_linear[r * nb + b];
}

/* ------------------------------------------------------------------------- */
/* Exact GEMM on the decoded operands, with one global scale per fused        */
/* segment of output columns applied at the end (the repair of Section 6).    */
/*   Y[m,n] = ( sum_b  Sa[m,b]*Sw[n,b] * sum_{i<16} ua[m,16b+i]*uw[n,16b+i] )  */
/*            * 2^-20 * g_a * g_col[n]                                         */
/* with u = 2*e2m1 value (an integer) and S = 2^9 * e4m3 value (an integer):   */
/* the double sum is an exact int64; the roundings are its conversion to      */
/* double (only above 2^53) and the two final double multiplies.  row_idx / col_idx select which outputs to compute      */
/* (NULL = all).  out is [n_rows_sel, n_cols_sel] row-major.                  */
/* ------------------------------------------------------------------------- */
static inline int orc_u2(uint8_t c) {       /* 2 * e2m1 value, as an integer */
    return (int)lrintf(2.0f * orc_e2m1_decode(c));
}
static inline int64_t orc_s512(uint8_t b) { /* 512 * e4m3 value, as an integer */
    return (int64_t)lrintf(512.0f * orc_e4m3_decode(b));
}

int orc_gemm(const uint8_t* a_codes, const uint8_t* a_sf, float g_a, int64_t M, int64_t K,
             const uint8_t* w_codes, const uint8_t* w_sf, const float* g_col, int64_t N,
             const int64_t* row_idx, int64_t n_rows_sel,
             const int64_t* col_idx, int64_t n_cols_sel, double* out) {
    if (K % 16 != 0) return 1;
    const int64_t nb = K / 16;
    const int64_t R = row_idx ? n_rows_sel : M, C = col_idx ? n_cols_sel : N;
    /* decode once into small integers (a change of representation, not of the sum) */
    int8_t* ua = (int8_t*)malloc((size_t)(R * K));
    int8_t* uw = (int8_t*)malloc((size_t)(C * K));
    int32_t* sa = (int32_t*)malloc(sizeof(int32_t) * (size_t)(R * nb));
    int32_t* sw = (int32_t*)malloc(sizeof(int32_t) * (size_t)(C * nb));
    if (!ua || !uw || !sa || !sw) { free(ua); free(uw); free(sa); free(sw); return 2; }
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < R; ++i) {
        int64_t m = row_idx ? row_idx[i] : i;
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = a_codes[m * (K / 2) + k / 2];
            ua[i * K + k] = (int8_t)orc_u2((k & 1) ? (byte >> 4) : (byte & 15));
        }
        for (int64_t b = 0; b < nb; ++b) sa[i * nb + b] = (int32_t)orc_s512(a_sf[m * nb + b]);
    }
    #pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < C; ++j) {
        int64_t n = col_idx ? col_idx[j] : j;
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = w_codes[n * (K / 2) + k / 2];
            uw[j * K + k] = (int8_t)orc_u2((k & 1) ? (byte >> 4) : (byte & 15));
        }
        for (int64_t b = 0; b < nb; ++b) sw[j * nb + b] = (int32_t)orc_s512(w_sf[n * nb + b]);
    }
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < R; ++i) {
        for (int64_t j = 0; j < C; ++j) {
            int64_t n = col_idx ? col_idx[j] : j;
            int64_t total = 0;
            for (int64_t b = 0; b < nb; ++b) {
                int32_t dot = 0;
                for (int t = 0; t < 16; ++t)
                    dot += (int32_t)ua[i * K + b * 16 + t] * (int32_t)uw[j * K + b * 16 + t];
                total += (int64_t)dot * (int64_t)sa[i * nb + b] * (int64_t)sw[j * nb + b];
            }
            out[i * C + j] = ldexp((double)total, -20) * (double)g_a * (double)g_col[n];
        }
    }
    free(ua); free(uw); free(sa); free(sw);
    return 0;
}

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
