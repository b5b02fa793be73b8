// Gated delta-rule recurrence in lockstep (paper: Background, Eq. 1-2; Section 5.3 runs one clean
// and several perturbed trajectories on identical inputs and watches the state error over time).
//
//   g_t = -exp(A_log) * softplus(a_t + dt_bias),  alpha_t = exp(g_t),  beta_t = sigmoid(b_t)
//   S_t = alpha_t S_{t-1} + beta_t k_t (v_t - S_{t-1}^T k_t)^T,        o_t = S_t^T (q_t / sqrt(K))
//
// with K = V = 128 and the state S in R^{K x V} per value head.  Everything is binary32, as in the
// paper's lockstep study.  One CTA per value head runs BOTH trajectories: threads 0..127 hold the
// clean state (thread j owns column j of S: 128 registers), threads 128..255 the perturbed one,
// fed from a second set of inputs (the same projections computed through the quantized layer).  Every
// `sample_every` tokens the CTA reports  ||S' - S||_F / ||S||_F  and  ||o' - o|| / ||o||.
// Query/key heads may be shared by several value heads (value head h reads q/k head h / (Hv / Hk)).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace nvfp4 {

constexpr int kGdnDim = 128;      // K = V = 128

struct LockstepParams {
    const float* q[2];            // [T, Hk, 128], l2-normalised; [0] clean, [1] perturbed
    const float* k[2];            // [T, Hk, 128], l2-normalised
    const float* v[2];            // [T, Hv, 128]
    const float* a[2];            // [T, Hv] gate pre-activations
    const float* b[2];            // [T, Hv]
    const float* A_log;           // [Hv]
    const float* dt_bias;         // [Hv]
    int64_t T;
    int32_t Hk, Hv;
    int64_t impulse_step;         // < 0: none; else the perturbed state is scaled by (1 + impulse_rel) after this token
    float impulse_rel;
    int64_t sample_every;
    float* rel_state;             // [T / sample_every, Hv]
    float* rel_out;               // [T / sample_every, Hv]
    float* final_state;           // optional [2, Hv, 128 (k), 128 (v)]
};

__device__ __forceinline__ float softplus_f(float x) {
    return x > 20.0f ? x : log1pf(expf(x));
}

__global__ void __launch_bounds__(256, 1)
gdn_lockstep_kernel(const LockstepParams p) {
    __shared__ __align__(16) float k_s[2][2][kGdnDim];      // [buffer][trajectory][k]
    __shared__ __align__(16) float q_s[2][2][kGdnDim];
    __shared__ float red[3][8];
    extern __shared__ __align__(16) float col_s[];           // [128 (v)][129]: the clean state at a sample step
    const int h = blockIdx.x;
    const int traj = threadIdx.x >> 7;                       // 0 clean, 1 perturbed
    const int j = threadIdx.x & 127;                         // this thread's column of S (value index)
    const int hk = h / (p.Hv / p.Hk);
    const float neg_decay = -expf(p.A_log[h]);
    const float dtb = p.dt_bias[h];
    const float q_scale = 0.08838834764831845f;              // 1 / sqrt(128)
    float S[kGdnDim];
#pragma unroll
    for (int i = 0; i < kGdnDim; ++i) S[i] = 0.0f;

    const float* qp = p.q[traj] + static_cast<int64_t>(hk) * kGdnDim + j;
    const float* kp = p.k[traj] + static_cast<int64_t>(hk) * kGdnDim + j;
    const float* vp = p.v[traj] + static_cast<int64_t>(h) * kGdnDim + j;
    const float* ap = p.a[traj] + h;
    const float* bp = p.b[traj] + h;
    const int64_t qk_stride = static_cast<int64_t>(p.Hk) * kGdnDim, v_stride = static_cast<int64_t>(p.Hv) * kGdnDim;

    // token 0's inputs
    float kq = p.T > 0 ? kp[0] : 0.0f, qq = p.T > 0 ? qp[0] : 0.0f, vv = p.T > 0 ? vp[0] : 0.0f;
    float aa = p.T > 0 ? ap[0] : 0.0f, bb = p.T > 0 ? bp[0] : 0.0f;
    int64_t next_sample = p.sample_every > 0 ? p.sample_every - 1 : -1, sample_idx = 0;
    for (int64_t t = 0; t < p.T; ++t) {
        const int buf = static_cast<int>(t & 1);
        k_s[buf][traj][j] = kq;
        q_s[buf][traj][j] = qq * q_scale;
        const float v_t = vv;
        const float alpha = expf(neg_decay * softplus_f(aa + dtb));
        const float beta = 1.0f / (1.0f + expf(-bb));
        __syncthreads();                                      // one barrier per token (the buffers alternate)
        if (t + 1 < p.T) {                                    // next token's inputs, in flight during the arithmetic
            kq = kp[(t + 1) * qk_stride];
            qq = qp[(t + 1) * qk_stride];
            vv = vp[(t + 1) * v_stride];
            aa = ap[(t + 1) * p.Hv];
            bb = bp[(t + 1) * p.Hv];
        }
        const float4* k4 = reinterpret_cast<const float4*>(k_s[buf][traj]);
        const float4* q4 = reinterpret_cast<const float4*>(q_s[buf][traj]);
        // what the state predicts for this key: (S^T k)_j
        float pred = 0.0f;
#pragma unroll
        for (int i = 0; i < kGdnDim / 4; ++i) {
            const float4 kk = k4[i];
            pred = fmaf(S[4 * i], kk.x, pred);
            pred = fmaf(S[4 * i + 1], kk.y, pred);
            pred = fmaf(S[4 * i + 2], kk.z, pred);
            pred = fmaf(S[4 * i + 3], kk.w, pred);
        }
        const float corr = beta * (v_t - pred);
        float o = 0.0f;
#pragma unroll
        for (int i = 0; i < kGdnDim / 4; ++i) {
            const float4 kk = k4[i];
            const float4 qv = q4[i];
            S[4 * i] = fmaf(alpha, S[4 * i], kk.x * corr);
            S[4 * i + 1] = fmaf(alpha, S[4 * i + 1], kk.y * corr);
            S[4 * i + 2] = fmaf(alpha, S[4 * i + 2], kk.z * corr);
            S[4 * i + 3] = fmaf(alpha, S[4 * i + 3], kk.w * corr);
            o = fmaf(S[4 * i], qv.x, o);
            o = fmaf(S[4 * i + 1], qv.y, o);
            o = fmaf(S[4 * i + 2], qv.z, o);
            o = fmaf(S[4 * i + 3], qv.w, o);
        }
        if (traj == 1 && t == p.impulse_step) {
#pragma unroll
            for (int i = 0; i < kGdnDim; ++i) S[i] *= 1.0f + p.impulse_rel;
        }
        if (t == next_sample) {
            // clean threads publish their column, perturbed threads compare (all threads take this branch)
            if (traj == 0) {
#pragma unroll
                for (int i = 0; i < kGdnDim; ++i) col_s[j * (kGdnDim + 1) + i] = S[i];
                col_s[kGdnDim * (kGdnDim + 1) + j] = o;
            }
            __syncthreads();
            float d2 = 0.0f, r2 = 0.0f, od2 = 0.0f, or2 = 0.0f;
            if (traj == 1) {
#pragma unroll
                for (int i = 0; i < kGdnDim; ++i) {
                    const float c = col_s[j * (kGdnDim + 1) + i];
                    const float d = S[i] - c;
                    d2 = fmaf(d, d, d2);
                    r2 = fmaf(c, c, r2);
                }
                const float oc = col_s[kGdnDim * (kGdnDim + 1) + j];
                od2 = (o - oc) * (o - oc);
                or2 = oc * oc;
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                d2 += __shfl_xor_sync(0xffffffffu, d2, off);
                r2 += __shfl_xor_sync(0xffffffffu, r2, off);
                od2 += __shfl_xor_sync(0xffffffffu, od2, off);
                or2 += __shfl_xor_sync(0xffffffffu, or2, off);
            }
            if ((threadIdx.x & 31) == 0) {
                red[0][threadIdx.x >> 5] = d2;
                red[1][threadIdx.x >> 5] = r2;
                red[2][threadIdx.x >> 5] = od2;
            }
            __shared__ float red_o[8];
            if ((threadIdx.x & 31) == 0) red_o[threadIdx.x >> 5] = or2;
            __syncthreads();
            if (threadIdx.x == 0) {
                float sd = 0.0f, sr = 0.0f, so = 0.0f, sor = 0.0f;
                for (int w = 4; w < 8; ++w) { sd += red[0][w]; sr += red[1][w]; so += red[2][w]; sor += red_o[w]; }
                p.rel_state[sample_idx * p.Hv + h] = sr > 0.0f ? sqrtf(sd / sr) : 0.0f;
                p.rel_out[sample_idx * p.Hv + h] = sor > 0.0f ? sqrtf(so / sor) : 0.0f;
            }
            ++sample_idx;
            next_sample += p.sample_every;
        }
    }
    if (p.final_state != nullptr) {
        float* dst = p.final_state + (static_cast<int64_t>(traj) * p.Hv + h) * kGdnDim * kGdnDim;
#pragma unroll
        for (int i = 0; i < kGdnDim; ++i) dst[i * kGdnDim + j] = S[i];
    }
}

}  // namespace nvfp4
