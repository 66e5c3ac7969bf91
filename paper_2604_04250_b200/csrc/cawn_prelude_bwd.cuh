// Backward of the fused path's prelude: from the push gradient lam = dLoss/dz (what the reverse
// scan returns) to the gradients of the hidden states, the conv weights and bias, and the
// carried conv history.  No scan is involved any more: every output row depends on a window of
// conv_k rows only, so a CTA owns 8 x R rows of one (batch, 64-channel group) and each thread
// walks its R rows (plus conv_k-1 rows of look-ahead, recomputed redundantly) for two adjacent
// channels with a rolling window in registers.
//
// Per (b, t, c), with u, x, m, phase and the gate decision recomputed as the forward does
// (u as the fp32 fmaf chain in tap order, so the gate decision is the forward's bit for bit):
//   dm  = lam_r cos ph + lam_i sin ph                 straight-through: unmasked
//   dph = m_used (-lam_r sin ph + lam_i cos ph)       m_used = m if the gate is open else 0
//   dx  = dm m (1 - m) + dph pi (1 - tanh(x)^2)
//   du  = dx * d(silu(clamp(u)))/du  (flag) or dx
//   dh[s] = sum_k w[c,k] du[s + (Kc-1) - k],  dw[c,k] = sum du[t] hrow[t-(Kc-1)+k],  dbias = sum du
#pragma once
#include "cawn_device.cuh"

namespace cawn {

struct PreludeBwdParams {
    const float *h;              // [B,L,C]
    const float2 *lam;           // [B,L,C] complex64: gradient of the pushes
    const float *conv_w;         // [C][Kc]
    const float *conv_bias;      // [C] or NULL
    const float *tail_in;        // [B][Kc-1][C] or NULL
    const float *dtail_out;      // [B][Kc-1][C] or NULL: gradient arriving on the call's last rows
    float *dh;                   // [B,L,C]
    float *dtail_in;             // [B][Kc-1][C] or NULL
    float *part;                 // [B*RT][C][5]: per-CTA sums of du*hrow (4 taps, right-aligned) and du
    long long L;
    int B, C, G, RT, Kc;
    int clamp_silu;
    float gate_tau;
};

constexpr int kPbRows = 16;      // rows per thread
constexpr int kPbWarps = 8;

template <bool VEC>
__global__ void __launch_bounds__(kPbWarps * 32, 2) cawn_prelude_bwd_kernel(const PreludeBwdParams prm)
{
    constexpr int R = kPbRows;
    __shared__ float sPart[kPbWarps][32][10];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int g = blockIdx.x, b = blockIdx.y, rt = blockIdx.z;
    const int C = prm.C, Kc = prm.Kc, Kh = Kc - 1;
    const long long L = prm.L;
    const int c0 = g * 64 + 2 * lane;
    const bool vA = c0 < C, vB = c0 + 1 < C;
    const long long r0 = ((long long)rt * kPbWarps + w) * R;       // first owned row
    const bool act = prm.clamp_silu != 0;
    const float tau = prm.gate_tau;

    // right-aligned taps: wt[j] multiplies hrow(t - 3 + j); taps the conv does not have are zero
    float wA[4], wB[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int kk = j - (4 - Kc);
        wA[j] = (kk >= 0 && vA) ? prm.conv_w[(long long)c0 * Kc + kk] : 0.f;
        wB[j] = (kk >= 0 && vB) ? prm.conv_w[(long long)(c0 + 1) * Kc + kk] : 0.f;
    }
    const float bA = (prm.conv_bias != nullptr && vA) ? prm.conv_bias[c0] : 0.f;
    const float bB = (prm.conv_bias != nullptr && vB) ? prm.conv_bias[c0 + 1] : 0.f;

    // hidden row s of this lane's two channels: h for 0 <= s < L, the carried tail for -Kh <= s < 0
    auto hrow = [&](long long s) -> float2 {
        float2 v = make_float2(0.f, 0.f);
        if (s >= 0 && s < L) {
            const float *p = prm.h + ((long long)b * L + s) * C + c0;
            if (VEC) { if (vA) v = __ldcs(reinterpret_cast<const float2 *>(p)); }
            else { if (vA) v.x = p[0]; if (vB) v.y = p[1]; }
        } else if (s < 0 && s >= -Kh && prm.tail_in != nullptr) {
            const float *p = prm.tail_in + ((long long)b * Kh + (Kh + s)) * C + c0;
            if (vA) v.x = p[0];
            if (vB) v.y = p[1];
        }
        return v;
    };
    // du of one channel at one row
    auto du_of = [&](float u, float lr, float li) -> float {
        float x = u, dxdu = 1.f;
        if (act) {
            const float v = fminf(fmaxf(u, -50.f), 50.f);
            const float sg = __fdividef(1.f, 1.f + __expf(-v));
            x = v * sg;
            dxdu = (u >= -50.f && u <= 50.f) ? sg * fmaf(v, 1.f - sg, 1.f) : 0.f;
        }
        const float xc = fminf(fmaxf(x, -25.f), 25.f);
        const float q = __expf(-xc), q2 = q * q;
        const float rcp = __fdividef(1.f, (1.f + q) * (1.f + q2));
        const float m = (1.f + q2) * rcp;
        const float th = (1.f - q2) * (1.f + q) * rcp;
        float sn, cs;
        __sincosf(3.14159265358979f * th, &sn, &cs);
        const bool open = act || u >= tau;       // with clamp + SiLU every gate is open (see the forward)
        const float dm = fmaf(lr, cs, li * sn);
        const float dph = (open ? m : 0.f) * fmaf(li, cs, -lr * sn);
        const float dx = fmaf(dm * m, 1.f - m, dph * 3.14159265358979f * fmaf(-th, th, 1.f));
        return dx * dxdu;
    };

    float2 hw[4];                        // hrow(t-3), hrow(t-2), hrow(t-1), hrow(t)
    hw[1] = hrow(r0 - 3); hw[2] = hrow(r0 - 2); hw[3] = hrow(r0 - 1);
    float2 dq[4] = {};                   // du(t-3), du(t-2), du(t-1), du(t)
    float accA[5] = {0.f, 0.f, 0.f, 0.f, 0.f}, accB[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < R + 3; ++i) {
        const long long t = r0 + i;
        hw[0] = hw[1]; hw[1] = hw[2]; hw[2] = hw[3];
        dq[0] = dq[1]; dq[1] = dq[2]; dq[2] = dq[3];
        float2 du = make_float2(0.f, 0.f);
        if (t < L && i < R + Kh) {
            hw[3] = hrow(t);
            float uA = bA, uB = bB;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (j >= 4 - Kc) { uA = fmaf(wA[j], hw[j].x, uA); uB = fmaf(wB[j], hw[j].y, uB); }
            }
            const float2 *lp = prm.lam + ((long long)b * L + t) * C + c0;
            if (VEC) {
                if (vA) {
                    const float4 l = __ldcs(reinterpret_cast<const float4 *>(lp));
                    du.x = du_of(uA, l.x, l.y); du.y = du_of(uB, l.z, l.w);
                }
            } else {
                if (vA) { const float2 l = lp[0]; du.x = du_of(uA, l.x, l.y); }
                if (vB) { const float2 l = lp[1]; du.y = du_of(uB, l.x, l.y); }
            }
            if (i < R) {                 // owned row: parameter sums
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    accA[j] = fmaf(du.x, hw[j].x, accA[j]);
                    accB[j] = fmaf(du.y, hw[j].y, accB[j]);
                }
                accA[4] += du.x; accB[4] += du.y;
            }
        } else {
            hw[3] = make_float2(0.f, 0.f);
        }
        dq[3] = du;
        // row s = t - 3 is complete: dh[s] = sum_j wt[j] du(s + 3 - j)
        const long long s = t - 3;
        if (i >= 3 && s < L) {
            float dA = 0.f, dB = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) { dA = fmaf(wA[j], dq[3 - j].x, dA); dB = fmaf(wB[j], dq[3 - j].y, dB); }
            if (prm.dtail_out != nullptr && s >= L - Kh) {
                const float *p = prm.dtail_out + ((long long)b * Kh + (s - (L - Kh))) * C + c0;
                if (vA) dA += p[0];
                if (vB) dB += p[1];
            }
            float *o = prm.dh + ((long long)b * L + s) * C + c0;
            if (VEC) { if (vA) __stcs(reinterpret_cast<float2 *>(o), make_float2(dA, dB)); }
            else { if (vA) o[0] = dA; if (vB) o[1] = dB; }
        }
    }
    // gradient of the carried history: rows s = -Kh .. -1 collect from du(0 .. Kh-1), which the
    // thread that owns row 0 has just computed (they sit in dq when its loop passes them); redo
    // the few products here from a second, tiny walk
    if (prm.dtail_in != nullptr && r0 == 0) {
        float2 hv[4], dv[3];
        hv[1] = hrow(-3); hv[2] = hrow(-2); hv[3] = hrow(-1);
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            hv[0] = hv[1]; hv[1] = hv[2]; hv[2] = hv[3];
            dv[i] = make_float2(0.f, 0.f);
            if (i < L && i < Kh) {
                hv[3] = hrow(i);
                float uA = bA, uB = bB;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (j >= 4 - Kc) { uA = fmaf(wA[j], hv[j].x, uA); uB = fmaf(wB[j], hv[j].y, uB); }
                }
                const float2 *lp = prm.lam + ((long long)b * L + i) * C + c0;
                if (vA) { const float2 l = lp[0]; dv[i].x = du_of(uA, l.x, l.y); }
                if (vB) { const float2 l = lp[1]; dv[i].y = du_of(uB, l.x, l.y); }
            } else {
                hv[3] = make_float2(0.f, 0.f);
            }
        }
        for (int r = 0; r < Kh; ++r) {
            const int s = r - Kh;                        // -Kh .. -1
            float dA = 0.f, dB = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int t = s + 3 - j;                 // du row this tap reaches
                if (t >= 0 && t < 3) { dA = fmaf(wA[j], dv[t].x, dA); dB = fmaf(wB[j], dv[t].y, dB); }
            }
            // a call shorter than the history passes part of the incoming tail gradient through
            if (prm.dtail_out != nullptr && r >= L) {
                const float *p = prm.dtail_out + ((long long)b * Kh + (r - L)) * C + c0;
                if (vA) dA += p[0];
                if (vB) dB += p[1];
            }
            float *o = prm.dtail_in + ((long long)b * Kh + r) * C + c0;
            if (vA) o[0] = dA;
            if (vB) o[1] = dB;
        }
    }
    // per-CTA parameter sums, in a fixed order
#pragma unroll
    for (int j = 0; j < 5; ++j) { sPart[w][lane][j] = accA[j]; sPart[w][lane][5 + j] = accB[j]; }
    __syncthreads();
    if (w == 0) {
        float *o = prm.part + (((long long)b * prm.RT + rt) * C + c0) * 5;
#pragma unroll
        for (int j = 0; j < 10; ++j) {
            float a = 0.f;
#pragma unroll
            for (int i = 0; i < kPbWarps; ++i) a += sPart[i][lane][j];
            if (j < 5 ? vA : vB) o[j] = a;
        }
    }
}

// grad_conv_w[c][k] and grad_conv_bias[c] from the per-CTA partials, in double, fixed order.
// One warp per channel.
__global__ void cawn_prelude_bwd_finalize_kernel(const float *part, int nparts, int C, int Kc,
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

}  // namespace cawn
