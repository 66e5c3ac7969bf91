// The small kernels around the scan: fixed-order reductions of the backward's per-tile partial
// sums, and the combine of two segment summaries.  Included by one translation unit only.
#pragma once
#include "cawn_device.cuh"

namespace cawn {

// ---------------------------------------------------------------------------------------
// The backward's epilogue launch: everything that has to wait for the whole reverse scan, in one
// kernel.  A block does one of four jobs, chosen by its index:
//   [0, nb_q)            grad_gamma_j = Re(e^{i theta} Q_j), grad_theta_j = -Im(a_j Q_j), Q_j = sum of the
//                        per-tile partials qpart [nparts][C]; 8 channels per block
//   [nb_q, +nb_s)        time-varying retention: grad_freq_bias[k] = sum over tiles and heads of spart
//                        [nparts][C]; 2 harmonics per block
//   [.., +nb_c)          fused path: grad_conv_w[c][k], grad_conv_bias[c] from cpart [nparts][C][5];
//                        8 channels per block
//   the rest             fused path: grad_h of the rows at tile seams and the gradient of the carried conv
//                        history, from edge_du (see seam_rows below); one thread per channel
// Sums run in double in a fixed order.  A block owns CW adjacent channels; a lane is (sub, channel) =
// (lane / CW, lane % CW), so a warp load covers 32 / CW parts with CW contiguous channels each, and
// thread (warp w, sub) takes parts (w * 32 / CW + sub) + i * kEpiWarps * 32 / CW.  The warps' sums are added in
// warp order, then the subs' by a butterfly (both partners of an exchange form the same sum).
// Bitwise repeatable.
constexpr int kEpiWarps = 32;
constexpr int kEpiCW = 8;            // channels per block of the q and c jobs
constexpr int kEpiFW = 2;            // harmonics per block of the s job
constexpr int kEpiSeams = 4;         // seams per thread of the seam job: their loads are issued together
struct EpilogueParams {
    int nb_q, nb_s, nb_c, nb_ex;     // blocks per job; nb_ex: blocks along the channels of one seam
    int nparts, C, H, F, Kc;
    const float2 *qpart;
    const float *gamma, *theta;      // gamma NULL: time-varying retention (the factor is already in Q)
    float *grad_gamma, *grad_theta;
    float clampv;
    const float *spart;
    float *grad_fbias;
    const float *cpart;
    float *grad_w, *grad_bias;
    const float *edge_du, *conv_w, *dtail_out;
    float *grad_h, *dtail_in;
    long long L;
    int B, K, tile;
};

// Sum of NV doubles per thread over the block: first over the warps, lane by lane, in warp order,
// then over the lanes that hold the same channel (lanes CW apart).  Result valid in warp 0.
template <int NV, int CW>
__device__ __forceinline__ void block_sum_fixed_order(double (&v)[NV], double *sh)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < NV; ++j) sh[(w * NV + j) * 32 + lane] = v[j];
    __syncthreads();
    if (w == 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            double acc = sh[j * 32 + lane];
            for (int i = 1; i < kEpiWarps; ++i) acc += sh[(i * NV + j) * 32 + lane];
#pragma unroll
            for (int off = CW; off < 32; off <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            v[j] = acc;
        }
    }
}

// Backward of the fused path, rows at tile seams.  The scan kernel (KIND_MIXBWD) leaves out
// grad_h of the three last rows in time of every tile, whose conv transpose reaches into the
// tile after them, and stores every tile's du at both ends instead (edge_du [B*K][6][C]: rows
// t_hi, t_hi-1, t_hi-2, then t_lo, t_lo+1, t_lo+2; tiles are counted from the END of the call:
// tile k covers t_hi = L-1-k*tile down to t_lo = max(L-(k+1)*tile, 0)).  Here:
//   grad_h(s) = sum_j w[j] du(s + 3 - j) (+ the incoming gradient of the conv history on the
//   call's last conv_k-1 rows)          for those rows (kb < K), and
//   grad of the carried history rows s = -Kh .. -1 (kb = K), which collect from du(0..2)
//   and, when the call is shorter than the history, pass part of the incoming gradient through.
// One thread per channel and kEpiSeams adjacent seams (kb0 .. kb0 + kEpiSeams - 1, those <= K): the
// du values of all of them are requested before the first is used.  Taps right-aligned as in the
// scan kernel.
__device__ __forceinline__ void seam_rows(const EpilogueParams &ep, int c, int kb0, int b)
{
    const int C = ep.C, K = ep.K, tile = ep.tile, Kc = ep.Kc, Kh = Kc - 1;
    const long long L = ep.L;
    float wt[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) wt[j] = j >= 4 - Kc ? ep.conv_w[(long long)c * Kc + (j - (4 - Kc))] : 0.f;
    // du at physical row r, from whichever tile end holds it.  r lies within three rows of tile
    // `base` (the tile whose seam is being finished; for the history rows the last tile), so it
    // belongs to that tile or to one of its neighbours: no division is needed to find it.
    auto DU = [&](long long r, int base) -> float {
        if (r < 0 || r >= L) return 0.f;
        long long t_hi = L - 1 - (long long)base * tile;
        long long t_lo = L - (long long)(base + 1) * tile;
        if (t_lo < 0) t_lo = 0;
        int kk = base;
        if (r > t_hi) kk = base - 1; else if (r < t_lo) kk = base + 1;
        if (kk != base) {
            t_hi = L - 1 - (long long)kk * tile;
            t_lo = L - (long long)(kk + 1) * tile;
            if (t_lo < 0) t_lo = 0;
        }
        if (kk < 0 || kk >= K || r > t_hi || r < t_lo) return 0.f;      // never: three rows reach no further
        const float *e = ep.edge_du + (((long long)b * K + kk) * 6) * C + c;
        if (t_hi - r < 3) return e[(t_hi - r) * C];
        if (r - t_lo < 3) return e[(3 + (r - t_lo)) * C];
        return 0.f;                                  // not an edge row: never asked for
    };
    // The three latest rows of tile kb, t_hi - i (i = 0, 1, 2), reach du of rows t_hi + 3 .. t_hi - 2:
    // the three earliest rows of the tile after it in time (tile kb - 1, its second edge triple)
    // and this tile's own three latest (its first edge triple; rows it does not have hold 0).
    float d[kEpiSeams][6];                           // d[s][m + 2] = du(t_hi + m) of seam kb0 + s, m = -2 .. 3
#pragma unroll
    for (int s = 0; s < kEpiSeams; ++s) {
        const int kb = kb0 + s;
#pragma unroll
        for (int i = 0; i < 6; ++i) d[s][i] = 0.f;
        if (kb < K) {
            const float *own = ep.edge_du + (((long long)b * K + kb) * 6) * C + c;
#pragma unroll
            for (int i = 0; i < 3; ++i) d[s][2 - i] = __ldg(own + (long long)i * C);
            if (kb > 0) {
                const float *nxt = own - 3ll * C;     // the second edge triple of tile kb - 1
#pragma unroll
                for (int i = 0; i < 3; ++i) d[s][3 + i] = __ldg(nxt + (long long)i * C);
            }
        }
    }
#pragma unroll
    for (int s = 0; s < kEpiSeams; ++s) {
        const int kb = kb0 + s;
        if (kb >= K) continue;
        const long long t_hi = L - 1 - (long long)kb * tile;
        long long t_lo = L - (long long)(kb + 1) * tile;
        if (t_lo < 0) t_lo = 0;
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const long long srow = t_hi - i;
            if (srow >= t_lo) {
                float acc = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) acc = fmaf(wt[j], d[s][(3 - i - j) + 2], acc);
                if (ep.dtail_out != nullptr && srow >= L - Kh) acc += ep.dtail_out[((long long)b * Kh + (srow - (L - Kh))) * C + c];
                ep.grad_h[((long long)b * L + srow) * C + c] = acc;
            }
        }
    }
    if (kb0 + kEpiSeams <= K) return;                // seam K (the carried history) is not in this group
    if (ep.dtail_in != nullptr) {
        for (int r = 0; r < Kh; ++r) {
            const long long s = r - Kh;
            float acc = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) acc = fmaf(wt[j], DU(s + 3 - j, K - 1), acc);
            if (ep.dtail_out != nullptr && r >= L) acc += ep.dtail_out[((long long)b * Kh + (r - L)) * C + c];
            ep.dtail_in[((long long)b * Kh + r) * C + c] = acc;
        }
    }
}

__global__ void __launch_bounds__(kEpiWarps * 32) cawn_bwd_epilogue_kernel(const EpilogueParams ep)
{
    __shared__ double sh[kEpiWarps * 5 * 32];
    // launched with programmatic stream serialisation behind the reverse scan: let the launch after
    // this one start filling SMs, and touch nothing before the scan is complete
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int blk = blockIdx.x;
    const int C = ep.C, nparts = ep.nparts;
    constexpr int PW = 32 / kEpiCW;                   // parts per warp load (q and c jobs)
    if (blk < ep.nb_q) {
        const int ch = blk * kEpiCW + lane % kEpiCW;
        double v[2] = {0.0, 0.0};
        if (ch < C) {
#pragma unroll 8
            for (int p = w * PW + lane / kEpiCW; p < nparts; p += kEpiWarps * PW) {
                const float2 q = ep.qpart[(long long)p * C + ch];
                v[0] += (double)q.x;
                v[1] += (double)q.y;
            }
        }
        block_sum_fixed_order<2, kEpiCW>(v, sh);
        if (w == 0 && lane < kEpiCW && ch < C) {
            const double gm = ep.gamma != nullptr ? (double)ep.gamma[ch] : 1.0;   // time-varying: already in Q
            double sn, cs;
            sincos((double)ep.theta[ch], &sn, &cs);
            double dg = cs * v[0] - sn * v[1];
            const double dth = -gm * (cs * v[1] + sn * v[0]);
            if (ep.clampv > 0.f) dg = fmin(fmax(dg, -(double)ep.clampv), (double)ep.clampv);
            if (ep.grad_gamma != nullptr) ep.grad_gamma[ch] = (float)dg;
            if (ep.grad_theta != nullptr) ep.grad_theta[ch] = (float)dth;
        }
        return;
    }
    blk -= ep.nb_q;
    if (blk < ep.nb_s) {
        // the (part, head) pairs are the terms: pair q = p * H + h holds harmonic kf at spart[p * C + h * F + kf]
        constexpr int QW = 32 / kEpiFW;
        const int kf = blk * kEpiFW + lane % kEpiFW;
        const long long npairs = (long long)nparts * ep.H;
        double v[1] = {0.0};
        if (kf < ep.F) {
#pragma unroll 8
            for (long long q = w * QW + lane / kEpiFW; q < npairs; q += kEpiWarps * QW) {
                const long long p = q / ep.H, h = q - p * ep.H;
                v[0] += (double)ep.spart[p * C + h * ep.F + kf];
            }
        }
        block_sum_fixed_order<1, kEpiFW>(v, sh);
        if (w == 0 && lane < kEpiFW && kf < ep.F) ep.grad_fbias[kf] = (float)v[0];
        return;
    }
    blk -= ep.nb_s;
    if (blk < ep.nb_c) {
        // per-tile partials [nparts][C][5]: four right-aligned taps, then the bias
        const int ch = blk * kEpiCW + lane % kEpiCW;
        double v[5] = {0.0, 0.0, 0.0, 0.0, 0.0};
        if (ch < C) {
#pragma unroll 4
            for (int p = w * PW + lane / kEpiCW; p < nparts; p += kEpiWarps * PW) {
                const float *q = ep.cpart + ((long long)p * C + ch) * 5;
#pragma unroll
                for (int j = 0; j < 5; ++j) v[j] += (double)q[j];
            }
        }
        block_sum_fixed_order<5, kEpiCW>(v, sh);
        if (w == 0 && lane < kEpiCW && ch < C) {
            if (ep.grad_w != nullptr)
                for (int k = 0; k < ep.Kc; ++k) ep.grad_w[(long long)ch * ep.Kc + k] = (float)v[k + (4 - ep.Kc)];
            if (ep.grad_bias != nullptr) ep.grad_bias[ch] = (float)v[4];
        }
        return;
    }
    blk -= ep.nb_c;
    {
        const int groups = (ep.K + kEpiSeams) / kEpiSeams;       // seams 0 .. K in groups of kEpiSeams
        const int cb = blk % ep.nb_ex, rest = blk / ep.nb_ex;
        const int kg = rest % groups, b = rest / groups;
        const int c = cb * (kEpiWarps * 32) + threadIdx.x;
        if (c < C && b < ep.B) seam_rows(ep, c, kg * kEpiSeams, b);
    }
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

// One 32-bit word, stream-ordered (the wait hook of a workspace header).
__global__ void cawn_set_word_kernel(unsigned *word, unsigned value) { *word = value; }

}  // namespace cawn
