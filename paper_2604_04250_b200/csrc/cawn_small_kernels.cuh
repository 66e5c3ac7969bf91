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

// Backward of the fused path, rows at tile seams.  The scan kernel (KIND_MIXBWD) leaves out
// grad_h of the three last rows in time of every tile, whose conv transpose reaches into the
// tile after them, and stores every tile's du at both ends instead (edge_du [B*K][6][C]: rows
// t_hi, t_hi-1, t_hi-2, then t_lo, t_lo+1, t_lo+2; tiles are counted from the END of the call:
// tile k covers t_hi = L-1-k*tile down to t_lo = max(L-(k+1)*tile, 0)).  Here:
//   grad_h(s) = sum_j w[j] du(s + 3 - j) (+ the incoming gradient of the conv history on the
//   call's last conv_k-1 rows)          for those rows (blockIdx.y = k < K), and
//   grad of the carried history rows s = -Kh .. -1 (blockIdx.y = K), which collect from du(0..2)
//   and, when the call is shorter than the history, pass part of the incoming gradient through.
// One thread per channel; taps right-aligned as in the scan kernel.
__global__ void cawn_mix_bwd_edges_kernel(const float *edge_du, const float *conv_w, const float *dtail_out,
                                          float *grad_h, float *dtail_in, long long L, int B, int C, int K,
                                          int tile, int Kc)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    const int kb = blockIdx.y, b = blockIdx.z;
    if (c >= C) return;
    const int Kh = Kc - 1;
    float wt[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) wt[j] = j >= 4 - Kc ? conv_w[(long long)c * Kc + (j - (4 - Kc))] : 0.f;
    // du at physical row r, from whichever tile end holds it
    auto DU = [&](long long r) -> float {
        if (r < 0 || r >= L) return 0.f;
        const long long kk = (L - 1 - r) / tile;
        const long long t_hi = L - 1 - kk * tile;
        long long t_lo = L - (kk + 1) * tile;
        if (t_lo < 0) t_lo = 0;
        const float *e = edge_du + (((long long)b * K + kk) * 6) * C + c;
        if (t_hi - r < 3) return e[(t_hi - r) * C];
        if (r - t_lo < 3) return e[(3 + (r - t_lo)) * C];
        return 0.f;                                  // not an edge row: never asked for
    };
    if (kb < K) {
        const long long t_hi = L - 1 - (long long)kb * tile;
        long long t_lo = L - (long long)(kb + 1) * tile;
        if (t_lo < 0) t_lo = 0;
        for (long long s = t_hi; s >= t_lo && s > t_hi - 3; --s) {
            float acc = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) acc = fmaf(wt[j], DU(s + 3 - j), acc);
            if (dtail_out != nullptr && s >= L - Kh) acc += dtail_out[((long long)b * Kh + (s - (L - Kh))) * C + c];
            grad_h[((long long)b * L + s) * C + c] = acc;
        }
    } else if (dtail_in != nullptr) {
        for (int r = 0; r < Kh; ++r) {
            const long long s = r - Kh;
            float acc = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) acc = fmaf(wt[j], DU(s + 3 - j), acc);
            if (dtail_out != nullptr && r >= L) acc += dtail_out[((long long)b * Kh + (r - L)) * C + c];
            dtail_in[((long long)b * Kh + r) * C + c] = acc;
        }
    }
}

// grad_conv_w[c][k] and grad_conv_bias[c] from the per-tile partials [nparts][C][5] (four
// right-aligned taps, then the bias), in double, fixed order.  One warp per channel.
__global__ void cawn_conv_grad_finalize_kernel(const float *part, int nparts, int C, int Kc,
                                               float *grad_w, float *grad_bias)
{
    const int lane = threadIdx.x & 31;
    const int ch = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (ch >= C) return;
    double acc[5] = {0.0, 0.0, 0.0, 0.0, 0.0};
    for (int p = lane; p < nparts; p += 32) {
        const float *q = part + ((long long)p * C + ch) * 5;
#pragma unroll
        for (int j = 0; j < 5; ++j) acc[j] += (double)q[j];
    }
#pragma unroll
    for (int j = 0; j < 5; ++j)
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc[j] += __shfl_down_sync(0xffffffffu, acc[j], off);
    if (lane == 0) {
        if (grad_w != nullptr)
            for (int k = 0; k < Kc; ++k) grad_w[(long long)ch * Kc + k] = (float)acc[k + (4 - Kc)];
        if (grad_bias != nullptr) grad_bias[ch] = (float)acc[4];
    }
}

// One 32-bit word, stream-ordered (the wait hook of a workspace header).
__global__ void cawn_set_word_kernel(unsigned *word, unsigned value) { *word = value; }

}  // namespace cawn
