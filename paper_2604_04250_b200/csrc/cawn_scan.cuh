// The chunk-parallel phase-accumulation kernel.
//
// One CTA owns a tile of TILE = W*T consecutive time steps of one (batch, 64-channel group).
// Warp w owns T consecutive steps; lane l owns the adjacent channels 64g + 2l and 64g + 2l + 1,
// so a warp-wide access is one 512-byte row segment read or written as 32 float4.
// The tile lives in registers between its single read and its single write:
//
//   0. every thread issues all of its loads (T rows, independent); meanwhile 64 threads
//      prepare the per-channel coefficients a, a^T, a^TILE in double            [barrier 1]
//   1. gate (Cartesian forward), then each thread reduces its T steps from a zero start and
//      leaves the end state in shared memory                                     [barrier 2]
//   2. warp 0 folds the W ends into the tile aggregate and publishes it; then every warp
//      fetches one record of the carry window (below) into shared memory         [barrier 3]
//   3. every warp folds the window into the tile's carry-in, folds the earlier warps' ends on
//      top, re-runs its T steps as the plain recurrence from that state and stores them
//
// Carry window.  With M = W-1, the tiles k = M, 2M, ... of a chain are checkpoints: they also
// publish their carry-in X_k (the state before the tile).  Tile k reads the carry-in of the
// last checkpoint c < k (c = 0: the call's initial state) and the aggregates E_c .. E_{k-1},
// and evaluates X_k = A^(k-c) X_c + sum A^(k-1-i) E_i by Horner's rule, oldest first, A = a^TILE.
// What is read and the order it is combined in depend on k alone, never on timing, so results
// are bit-for-bit repeatable; aggregates are published before anything is waited for, so the
// only serial dependency runs from checkpoint to checkpoint.  A tile only ever waits for tiles
// with a smaller block index, which the hardware has dispatched before it.
//
// Each run of the fp32 recurrence is at most T steps long and everything that crosses a thread
// boundary is multiplied by a power of a_j rounded once from double: the rounding error of
// a_j does not build up with sequence length.
//
// The backward is the same operator run right-to-left with conj(a_j); it additionally
// accumulates sum conj(lam_t) P_{t-1} per channel for the retention and rotation gradients.
#pragma once
#include "cawn_device.cuh"

namespace cawn {

enum : int { KIND_FWD = 0, KIND_BWD = 2 };

struct ScanParams {
    const void *in;              // FWD: pushes p;  BWD: grad_y              [B,L,C] complex64
    void *out;                   // FWD: y;         BWD: grad_p
    const void *aux;             // BWD: saved unclamped states P (NULL: no parameter sums)
    const float *gamma, *theta;  // [C]
    const float2 *state_in;      // FWD: carried state or NULL;  BWD: forward's state_in or NULL
    const float2 *edge_in;       // BWD: grad_state_out or NULL (added to the first step)
    float2 *state_out;           // FWD: state_out;  BWD: grad_state_in
    uint32_t *mask;              // FWD: bit-packed gate mask or NULL
    WsHeader *ws;
    uint4 *agg;                  // aggregate records [B][G][K][64]
    uint4 *pre;                  // checkpoint carry-in records [B][G][KP][64]
    float2 *qpart;               // BWD: per-tile partial sums [B*K][C]
    long long L;
    int B, C, G, K, KP, MW;      // MW = mask words per row
    double eps2;                 // gate threshold squared
    float gate_lo, gate_hi;      // fp32 screen: below lo surely closed, at or above hi surely open
    float clampv;                // output (FWD) or gradient (BWD) clamp; <= 0 off
    unsigned poll_limit;
};

// |p| >= eps decided as re^2 + im^2 >= eps^2 in double: both squares are exact there and the
// sum rounds once, so the decision is reproducible bit for bit.  The fp32 sum of squares is
// within 2^-22 of the exact one, so it settles every case outside a 2^-21 band around the
// threshold; only the band takes the double path.
__device__ __forceinline__ bool gate_open(float re, float im, const ScanParams &prm)
{
    const float s = fmaf(re, re, im * im);
    bool open = s >= prm.gate_hi;
    if (!open && s >= prm.gate_lo)
        open = ((double)re * (double)re + (double)im * (double)im >= prm.eps2);
    return open;
}

template <int T, int W, int KIND, bool VEC, bool FULL>
__device__ __forceinline__ void scan_tile(const ScanParams &prm, float4 (*sE)[32], float4 (*sR)[32],
                                          float (*sCoef)[6], unsigned long long *sEpoch, int *sErr,
                                          const int g, const int b, const int k)
{
    constexpr bool REV = (KIND == KIND_BWD);
    constexpr int TILE = T * W;
    constexpr int M = W - 1;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int G = prm.G, C = prm.C, K = prm.K;
    const long long L = prm.L;
    const int c0 = g * 64 + 2 * lane;
    const bool vA = FULL || c0 < C, vB = FULL || c0 + 1 < C;
    const long long s0 = (long long)k * TILE + (long long)w * T;   // first logical step
    int nvalid = T;
    if (!FULL) {
        const long long rem = L - s0;
        nvalid = rem <= 0 ? 0 : (rem >= T ? T : (int)rem);
    }
    // logical step s <-> physical row t: forward t = s, reverse t = L-1-s
    const long long t_first = REV ? (L - 1 - s0) : s0;
    const long long rowstep = REV ? -(long long)C : (long long)C;
    const long long e0 = ((long long)b * L + t_first) * C + c0;    // only used when nvalid > 0

    // ---- 0. loads -------------------------------------------------------------------------
    float4 x[T];
    {
        const float2 *in = reinterpret_cast<const float2 *>(prm.in) + e0;
#pragma unroll
        for (int i = 0; i < T; ++i) {
            x[i] = zero4();
            if (FULL || i < nvalid) {
                const float2 *r = in + (long long)i * rowstep;
                if (VEC) {
                    if (vA) x[i] = __ldcs(reinterpret_cast<const float4 *>(r));
                } else {
                    if (vA) { const float2 v = __ldcs(r); x[i].x = v.x; x[i].y = v.y; }
                    if (vB) { const float2 v = __ldcs(r + 1); x[i].z = v.x; x[i].w = v.y; }
                }
            }
        }
    }
    float4 q[KIND == KIND_BWD ? T : 1];                            // P_{t-1}
    if constexpr (KIND == KIND_BWD) {
#pragma unroll
        for (int i = 0; i < T; ++i) {
            q[i] = zero4();
            if (prm.aux != nullptr && (FULL || i < nvalid)) {
                const long long t = t_first - i;
                if (t >= 1) {
                    const float2 *r = reinterpret_cast<const float2 *>(prm.aux) + e0 - C + (long long)i * rowstep;
                    if (VEC) {
                        if (vA) q[i] = __ldcs(reinterpret_cast<const float4 *>(r));
                    } else {
                        if (vA) { const float2 v = __ldcs(r); q[i].x = v.x; q[i].y = v.y; }
                        if (vB) { const float2 v = __ldcs(r + 1); q[i].z = v.x; q[i].w = v.y; }
                    }
                } else if (prm.state_in != nullptr) {
                    const float2 *r = prm.state_in + (long long)b * C + c0;
                    if (vA) { const float2 v = r[0]; q[i].x = v.x; q[i].y = v.y; }
                    if (vB) { const float2 v = r[1]; q[i].z = v.x; q[i].w = v.y; }
                }
            }
        }
        // lam_{L-1} = G_{L-1} + grad_state_out: fold it into the first logical step
        if (prm.edge_in != nullptr && s0 == 0 && nvalid > 0) {
            const float2 *r = prm.edge_in + (long long)b * C + c0;
            if (vA) { const float2 v = r[0]; x[0].x += v.x; x[0].y += v.y; }
            if (vB) { const float2 v = r[1]; x[0].z += v.x; x[0].w += v.y; }
        }
    }

    // ---- per-channel coefficients, in double, rounded once --------------------------------
    if (tid < 64) {
        const int ch = g * 64 + tid;
        float cf[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (ch < C) {
            const double gm = (double)prm.gamma[ch], th = (double)prm.theta[ch];
            double sn, cs;
            sincos(th, &sn, &cs);
            const double ar = gm * cs, ai = REV ? -(gm * sn) : gm * sn;
            double tr, ti, wr, wi;
            cpow_int<T>(ar, ai, tr, ti);
            cpow_int<W>(tr, ti, wr, wi);
            cf[0] = (float)ar; cf[1] = (float)ai;
            cf[2] = (float)tr; cf[3] = (float)ti;
            cf[4] = (float)wr; cf[5] = (float)wi;
        }
#pragma unroll
        for (int i = 0; i < 6; ++i) sCoef[tid][i] = cf[i];
    }
    unsigned long long epoch0 = 0;
    unsigned arrived = 0;
    if (tid == 0) {
        epoch0 = ld_volatile_u64(&prm.ws->epoch);
        *sEpoch = epoch0;
        *sErr = 0;
        // counted only once the epoch has been read (the increment depends on its value)
        arrived = atomicAdd(&prm.ws->done, 1u + (unsigned)(epoch0 >> 63));
    }
    __syncthreads();                                                           // barrier 1
    float4 a, aT;
    {
        // channel 2l: a, a^T, A at sCoef[2l][0..5]; channel 2l+1 follows: 12 contiguous floats
        const float4 *cp = reinterpret_cast<const float4 *>(&sCoef[2 * lane][0]);
        const float4 u0 = cp[0], u1 = cp[1], u2 = cp[2];
        a = make_float4(u0.x, u0.y, u1.z, u1.w);
        aT = make_float4(u0.z, u0.w, u2.x, u2.y);
    }
    const unsigned long long epoch = *sEpoch;

    // ---- 1. gate + local reduction from a zero start ---------------------------------------
    float4 e = zero4();
#pragma unroll
    for (int i = 0; i < T; ++i) {
        if constexpr (KIND == KIND_FWD) {
            const bool oA = vA && gate_open(x[i].x, x[i].y, prm);
            const bool oB = vB && gate_open(x[i].z, x[i].w, prm);
            if (!oA) { x[i].x = 0.f; x[i].y = 0.f; }
            if (!oB) { x[i].z = 0.f; x[i].w = 0.f; }
            if (prm.mask != nullptr) {
                // lanes 0..15 hold channels 0..31 of the group (word 0), lanes 16..31 word 1
                const unsigned bits = ((oA ? 1u : 0u) | (oB ? 2u : 0u)) << (2 * (lane & 15));
                const unsigned w0 = __reduce_or_sync(0xffffffffu, lane < 16 ? bits : 0u);
                const unsigned w1 = __reduce_or_sync(0xffffffffu, lane < 16 ? 0u : bits);
                if (FULL || i < nvalid) {
                    uint32_t *mrow = prm.mask + ((long long)b * L + (s0 + i)) * prm.MW + g * 2;
                    if (lane == 0) mrow[0] = w0;
                    if (lane == 16 && g * 2 + 1 < prm.MW) mrow[1] = w1;
                }
            }
        }
        if (FULL || i < nvalid) e = cfma2(a, e, x[i]);
    }
    sE[w][lane] = e;
    if (tid == 0 && arrived == gridDim.x - 1) {
        // every CTA of this launch has read the epoch: open the next one
        st_volatile_u32(&prm.ws->done, 0u);
        st_volatile_u64(&prm.ws->epoch, epoch0 + 1ull);
    }
    __syncthreads();                                                           // barrier 2

    // ---- 2. publish the aggregate, fetch the carry window ----------------------------------
    const long long chain = (long long)b * G + g;
    const int cpt = k > 0 ? M * ((k - 1) / M) : 0;       // last checkpoint before this tile
    const int nrec = k - cpt;                            // aggregates in the window, 0..M
    if (w == 0 && k + 1 < K) {
        float4 E = sE[0][lane];
#pragma unroll
        for (int i = 1; i < W; ++i) E = cfma2(aT, E, sE[i][lane]);
        publish_pair(prm.agg + (chain * K + k) * 64, lane, E, epoch, REC_AGGREGATE);
    }
    {
        float4 r = zero4();
        bool ok = true;
        if (w < nrec) {
            ok = poll_pair(prm.agg + (chain * K + (k - 1 - w)) * 64, lane, epoch, prm.poll_limit, r);
        } else if (w == W - 1) {
            if (cpt > 0) {
                ok = poll_pair(prm.pre + (chain * prm.KP + cpt / M) * 64, lane, epoch, prm.poll_limit, r);
            } else if (!REV && prm.state_in != nullptr) {
                const float2 *s = prm.state_in + (long long)b * C + c0;
                if (vA) { const float2 v = s[0]; r.x = v.x; r.y = v.y; }
                if (vB) { const float2 v = s[1]; r.z = v.x; r.w = v.y; }
            }
        }
        sR[w][lane] = r;
        if (!ok) {
            *sErr = 1;
            atomicMax(&prm.ws->status, 1u);              // CAWN_ERR_CARRY_TIMEOUT
        }
    }
    __syncthreads();                                                           // barrier 3

    // ---- 3. carry-in, the recurrence itself, stores -----------------------------------------
    const bool failed = (*sErr != 0);
    const bool checkpoint = (k > 0 && k % M == 0 && k + 1 < K);
    float4 qa = zero4();
    if (!failed) {
        float4 P = sR[W - 1][lane];
        {
            const float4 *cp = reinterpret_cast<const float4 *>(&sCoef[2 * lane][0]);
            const float4 u1 = cp[1], u2 = cp[2];
            const float4 AA = make_float4(u1.x, u1.y, u2.z, u2.w);
#pragma unroll
            for (int i = M - 1; i >= 0; --i)
                if (i < nrec) P = cfma2(AA, P, sR[i][lane]);
        }
        if (checkpoint && w == 0)
            publish_pair(prm.pre + (chain * prm.KP + k / M) * 64, lane, P, epoch, REC_PREFIX);
#pragma unroll
        for (int i = 0; i < W - 1; ++i)
            if (i < w) P = cfma2(aT, P, sE[i][lane]);

        float2 *out = reinterpret_cast<float2 *>(prm.out) + e0;
        const float cl = prm.clampv;
#pragma unroll
        for (int i = 0; i < T; ++i) {
            if (FULL || i < nvalid) {
                P = cfma2(a, P, x[i]);
                const float4 o = cl > 0.f ? clamp4(P, cl) : P;
                float2 *r = out + (long long)i * rowstep;
                if (VEC) {
                    if (vA) __stcs(reinterpret_cast<float4 *>(r), o);
                } else {
                    if (vA) __stcs(r, make_float2(o.x, o.y));
                    if (vB) __stcs(r + 1, make_float2(o.z, o.w));
                }
                if constexpr (KIND == KIND_BWD) {
                    // conj(lam) * P_{t-1}
                    qa.x = fmaf(P.x, q[i].x, fmaf(P.y, q[i].y, qa.x));
                    qa.y = fmaf(P.x, q[i].y, fmaf(-P.y, q[i].x, qa.y));
                    qa.z = fmaf(P.z, q[i].z, fmaf(P.w, q[i].w, qa.z));
                    qa.w = fmaf(P.z, q[i].w, fmaf(-P.w, q[i].z, qa.w));
                }
            }
        }
        // the thread that owns the last step writes the carried state (never clamped)
        if (prm.state_out != nullptr && nvalid > 0 && s0 + nvalid == L) {
            if (REV) P = cmul2(a, P);                    // grad_state_in = conj(a) lam_0
            float2 *s = prm.state_out + (long long)b * C + c0;
            if (vA) s[0] = make_float2(P.x, P.y);
            if (vB) s[1] = make_float2(P.z, P.w);
        }
    } else if (checkpoint && w == 0) {
        publish_pair(prm.pre + (chain * prm.KP + k / M) * 64, lane, zero4(), epoch, REC_POISON);
    }
    if constexpr (KIND == KIND_BWD) {
        if (prm.qpart != nullptr) {
            __syncthreads();
            sE[w][lane] = qa;
            __syncthreads();
            if (w == 0) {
                float4 acc = sE[0][lane];
#pragma unroll
                for (int i = 1; i < W; ++i) {
                    const float4 v = sE[i][lane];
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                float2 *qp = prm.qpart + ((long long)b * K + k) * C + c0;
                if (vA) qp[0] = make_float2(acc.x, acc.y);
                if (vB) qp[1] = make_float2(acc.z, acc.w);
            }
        }
    }
}

template <int T, int W, int KIND, bool VEC>
__global__ void __launch_bounds__(W * 32) cawn_scan_kernel(const ScanParams prm)
{
    constexpr int TILE = T * W;
    __shared__ float4 sE[W][32];
    __shared__ float4 sR[W][32];
    __shared__ __align__(16) float sCoef[64][6];
    __shared__ unsigned long long sEpoch;
    __shared__ int sErr;

    const int g = blockIdx.x % prm.G;
    const int bk = blockIdx.x / prm.G;
    const int b = bk % prm.B;
    const int k = bk / prm.B;                         // tile index along (logical) time
    const bool full = ((long long)(k + 1) * TILE <= prm.L) && (g * 64 + 64 <= prm.C);
    if (full) scan_tile<T, W, KIND, VEC, true>(prm, sE, sR, sCoef, &sEpoch, &sErr, g, b, k);
    else      scan_tile<T, W, KIND, VEC, false>(prm, sE, sR, sCoef, &sEpoch, &sErr, g, b, k);
}

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
        const double gm = (double)gamma[ch];
        double sn, cs;
        sincos((double)theta[ch], &sn, &cs);
        double dg = cs * sr - sn * si;
        const double dth = -gm * (cs * si + sn * sr);
        if (clampv > 0.f) dg = fmin(fmax(dg, -(double)clampv), (double)clampv);
        if (grad_gamma != nullptr) grad_gamma[ch] = (float)dg;
        if (grad_theta != nullptr) grad_theta[ch] = (float)dth;
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

}  // namespace cawn
