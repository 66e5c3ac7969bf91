// The small kernels around the scan: fixed-order reductions of the backward's per-tile partial
// sums, and the combine of two segment summaries.  Included by one translation unit only.
#pragma once
#include "cawn_device.cuh"

namespace cawn {

// grad_gamma_j = Re(e^{i theta} Q_j), grad_theta_j = -Im(a_j Q_j), Q_j = sum of the per-tile
// partials in a fixed order, in double.  One warp per channel.
__global__ void cawn_bwd_finalize_kernel(const float2 *qpart, int nparts, int C,
                                         const float *gamma, const float *theta,
                                         float *grad_gamma, float *grad_theta, float clampv)
{
    const int lane = threadIdx.x & 31;
    const int ch = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (ch >= C) return;
    double sr = 0.0, si = 0.0;
    for (int p = lane; p < nparts; p += 32) {
        const float2 q = qpart[(long long)p * C + ch];
        sr += (double)q.x;
        si += (double)q.y;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        sr += __shfl_down_sync(0xffffffffu, sr, off);
        si += __shfl_down_sync(0xffffffffu, si, off);
    }
    if (lane == 0) {
        const double gm = gamma != nullptr ? (double)gamma[ch] : 1.0;   // time-varying: already in Q
        double sn, cs;
        sincos((double)theta[ch], &sn, &cs);
        double dg = cs * sr - sn * si;
        const double dth = -gm * (cs * si + sn * sr);
        if (clampv > 0.f) dg = fmin(fmax(dg, -(double)clampv), (double)clampv);
        if (grad_gamma != nullptr) grad_gamma[ch] = (float)dg;
        if (grad_theta != nullptr) grad_theta[ch] = (float)dth;
    }
}

// Time-varying retention: grad_freq_bias[k] = sum over tiles and heads of the per-channel
// partial sums of the logit gradient, in a fixed order, in double.  One warp per harmonic.
__global__ void cawn_bwd_freq_bias_kernel(const float *spart, int nparts, int H, int F, float *grad_freq_bias)
{
    const int lane = threadIdx.x & 31;
    const int kf = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (kf >= F) return;
    const long long C = (long long)H * F;
    double acc = 0.0;
    for (long long i = lane; i < (long long)nparts * H; i += 32) {
        const long long part = i / H, h = i % H;
        acc += (double)spart[part * C + h * F + kf];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, off);
    if (lane == 0) grad_freq_bias[kf] = (float)acc;
}

// state_out = a^n * state_prev + state_local with a^n = gamma^n (cos n theta, sin n theta)
// evaluated in double.
__global__ void cawn_state_carry_kernel(const float2 *prev, const float2 *local, float2 *out,
                                        const float *gamma, const float *theta,
                                        long long n_steps, int B, int C)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)B * C) return;
    const int ch = (int)(idx % C);
    const double gm = (double)gamma[ch], th = (double)theta[ch];
    const double mag = pow(gm, (double)n_steps);
    double sn, cs;
    sincos(th * (double)n_steps, &sn, &cs);
    const float2 p = prev[idx], l = local[idx];
    const double pr = (double)p.x, pi = (double)p.y;
    float2 o;
    o.x = (float)((double)l.x + mag * (pr * cs - pi * sn));
    o.y = (float)((double)l.y + mag * (pr * sn + pi * cs));
    out[idx] = o;
}

}  // namespace cawn
