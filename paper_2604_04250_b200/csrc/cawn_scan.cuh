// The chunk-parallel phase-accumulation kernel.
//
// One CTA owns a tile of TILE = W*T consecutive time steps of one (batch, 64-channel group).
// Warp w owns T consecutive steps, lane l owns channels (64g + l) and (64g + 32 + l), so every
// warp-wide access is a run of 256 contiguous bytes and a tile row is 512 contiguous bytes.
// The tile lives in registers between its single read and its single write:
//
//   0. every thread issues all of its loads (T rows x 2 channels, independent);
//      meanwhile 64 threads prepare the per-channel coefficients a, a^T, a^TILE in double
//   1. gate (Cartesian forward), then the thread reduces its T steps from a zero start
//   2. warp 0 folds the W partial ends into the tile aggregate, publishes it, looks back
//      along time for the tile's carry-in (decoupled look-back over 16-byte tagged records),
//      publishes the inclusive prefix
//   3. every thread folds the earlier warps' ends onto the carry-in, re-runs its T steps as
//      the plain recurrence from that state and stores the results
//
// So each run of the fp32 recurrence is at most T steps long and everything that crosses a
// thread boundary is multiplied by a power of a_j rounded once from double: the systematic
// rounding error of a_j does not build up with sequence length.
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
    uint4 *rec;                  // carry records [B][G][K][64]
    float2 *qpart;               // BWD: per-tile partial sums [B*K][C]
    long long L;
    int B, C, G, K, MW;          // MW = mask words per row
    double eps2;                 // gate threshold squared
    float clampv;                // output (FWD) or gradient (BWD) clamp; <= 0 off
    unsigned poll_limit;
};

template <int T, int W, int KIND>
__global__ void __launch_bounds__(W * 32) cawn_scan_kernel(const ScanParams prm)
{
    constexpr bool REV = (KIND == KIND_BWD);
    constexpr int TILE = T * W;
    __shared__ float4 sE[W][32];
    __shared__ float sCoef[64][6];
    __shared__ float4 sS[32];
    __shared__ int sErr;

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int G = prm.G, B = prm.B, C = prm.C, K = prm.K;
    const long long L = prm.L;
    const int g = blockIdx.x % G;
    const int bk = blockIdx.x / G;
    const int b = bk % B;
    const int k = bk / B;                         // tile index along (logical) time
    const int c0 = g * 64 + lane, c1 = c0 + 32;
    const bool v0 = c0 < C, v1 = c1 < C;
    const long long s0 = (long long)k * TILE + (long long)w * T;   // first logical step
    const long long rem = L - s0;
    const int nvalid = rem <= 0 ? 0 : (rem >= T ? T : (int)rem);
    // logical step s <-> physical row t: forward t = s, reverse t = L-1-s
    const long long t_first = REV ? (L - 1 - s0) : s0;
    const long long rowstep = REV ? -(long long)C : (long long)C;
    const long long row0 = ((long long)b * L + t_first) * C;       // only used when nvalid > 0

    unsigned long long epoch = 0;
    if (w == 0) epoch = ld_volatile_u64(&prm.ws->epoch);
    if (tid == 0) sErr = 0;

    // ---- 0. loads -------------------------------------------------------------------------
    float2 x0[T], x1[T];
    {
        const float2 *in = reinterpret_cast<const float2 *>(prm.in);
#pragma unroll
        for (int i = 0; i < T; ++i) {
            x0[i] = make_float2(0.f, 0.f);
            x1[i] = make_float2(0.f, 0.f);
            if (i < nvalid) {
                const float2 *r = in + row0 + (long long)i * rowstep;
                if (v0) x0[i] = __ldcs(r + c0);
                if (v1) x1[i] = __ldcs(r + c1);
            }
        }
    }
    float2 q0[KIND == KIND_BWD ? T : 1], q1[KIND == KIND_BWD ? T : 1];   // P_{t-1}
    if constexpr (KIND == KIND_BWD) {
        const float2 *aux = reinterpret_cast<const float2 *>(prm.aux);
#pragma unroll
        for (int i = 0; i < T; ++i) {
            q0[i] = make_float2(0.f, 0.f);
            q1[i] = make_float2(0.f, 0.f);
            if (aux != nullptr && i < nvalid) {
                const long long t = t_first - i;
                if (t >= 1) {
                    const float2 *r = aux + ((long long)b * L + t - 1) * C;
                    if (v0) q0[i] = __ldcs(r + c0);
                    if (v1) q1[i] = __ldcs(r + c1);
                } else if (prm.state_in != nullptr) {
                    if (v0) q0[i] = prm.state_in[(long long)b * C + c0];
                    if (v1) q1[i] = prm.state_in[(long long)b * C + c1];
                }
            }
        }
        // lam_{L-1} = G_{L-1} + grad_state_out: fold it into the first logical step
        if (prm.edge_in != nullptr && s0 == 0 && nvalid > 0) {
            if (v0) { const float2 e = prm.edge_in[(long long)b * C + c0]; x0[0].x += e.x; x0[0].y += e.y; }
            if (v1) { const float2 e = prm.edge_in[(long long)b * C + c1]; x1[0].x += e.x; x1[0].y += e.y; }
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
    __syncthreads();
    const float2 a0 = make_float2(sCoef[lane][0], sCoef[lane][1]);
    const float2 a1 = make_float2(sCoef[lane + 32][0], sCoef[lane + 32][1]);
    const float2 aT0 = make_float2(sCoef[lane][2], sCoef[lane][3]);
    const float2 aT1 = make_float2(sCoef[lane + 32][2], sCoef[lane + 32][3]);

    // ---- 1. gate + local reduction from a zero start ---------------------------------------
    float2 e0 = make_float2(0.f, 0.f), e1 = e0;
#pragma unroll
    for (int i = 0; i < T; ++i) {
        if constexpr (KIND == KIND_FWD) {
            // |p| >= eps decided as re^2 + im^2 >= eps^2 in double: both squares are exact
            // there and the sum rounds once, so the mask is reproducible bit for bit.
            const bool o0 = v0 && ((double)x0[i].x * (double)x0[i].x +
                                   (double)x0[i].y * (double)x0[i].y >= prm.eps2);
            const bool o1 = v1 && ((double)x1[i].x * (double)x1[i].x +
                                   (double)x1[i].y * (double)x1[i].y >= prm.eps2);
            if (!o0) x0[i] = make_float2(0.f, 0.f);
            if (!o1) x1[i] = make_float2(0.f, 0.f);
            if (prm.mask != nullptr) {
                const unsigned m0 = __ballot_sync(0xffffffffu, o0);
                const unsigned m1 = __ballot_sync(0xffffffffu, o1);
                if (lane == 0 && i < nvalid) {
                    uint32_t *mrow = prm.mask + ((long long)b * L + (s0 + i)) * prm.MW + g * 2;
                    mrow[0] = m0;
                    if (g * 2 + 1 < prm.MW) mrow[1] = m1;
                }
            }
        }
        if (i < nvalid) {
            e0 = cfma(a0, e0, x0[i]);
            e1 = cfma(a1, e1, x1[i]);
        }
    }
    sE[w][lane] = make_float4(e0.x, e0.y, e1.x, e1.y);
    __syncthreads();

    // ---- 2. tile aggregate, look-back, inclusive prefix (warp 0) ----------------------------
    if (w == 0) {
        const float2 aW0 = make_float2(sCoef[lane][4], sCoef[lane][5]);
        const float2 aW1 = make_float2(sCoef[lane + 32][4], sCoef[lane + 32][5]);
        float4 v = sE[0][lane];
        float2 E0 = make_float2(v.x, v.y), E1 = make_float2(v.z, v.w);
#pragma unroll
        for (int i = 1; i < W; ++i) {
            v = sE[i][lane];
            E0 = cfma(aT0, E0, make_float2(v.x, v.y));
            E1 = cfma(aT1, E1, make_float2(v.z, v.w));
        }
        float2 S0 = make_float2(0.f, 0.f), S1 = S0;
        bool ok = true;
        uint4 *chain = prm.rec + ((long long)(b * G + g) * K) * 64;
        uint4 *mine = chain + (long long)k * 64;
        const bool publish = (k + 1 < K);
        if (k == 0) {
            if (!REV && prm.state_in != nullptr) {
                if (v0) S0 = prm.state_in[(long long)b * C + c0];
                if (v1) S1 = prm.state_in[(long long)b * C + c1];
            }
        } else {
            if (publish) {
                st_record(mine + lane, E0, epoch * 4ull + REC_AGGREGATE);
                st_record(mine + lane + 32, E1, epoch * 4ull + REC_AGGREGATE);
            }
            ok = carry_lookback(chain, k, lane, v0, v1, epoch, aW0, aW1, prm.poll_limit, S0, S1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (publish) {
            const unsigned kind = ok ? REC_PREFIX : REC_POISON;
            st_record(mine + lane, cfma(aW0, S0, E0), epoch * 4ull + kind);
            st_record(mine + lane + 32, cfma(aW1, S1, E1), epoch * 4ull + kind);
        }
        if (!ok && lane == 0) {
            sErr = 1;
            atomicMax(&prm.ws->status, 1u);          // CAWN_ERR_CARRY_TIMEOUT
        }
        sS[lane] = make_float4(S0.x, S0.y, S1.x, S1.y);
    }
    __syncthreads();

    // ---- 3. carry-in of this thread, the recurrence itself, stores --------------------------
    float2 qa0 = make_float2(0.f, 0.f), qa1 = qa0;
    if (sErr == 0) {
        const float4 sv = sS[lane];
        float2 P0 = make_float2(sv.x, sv.y), P1 = make_float2(sv.z, sv.w);
#pragma unroll
        for (int i = 0; i < W - 1; ++i) {
            if (i < w) {
                const float4 v = sE[i][lane];
                P0 = cfma(aT0, P0, make_float2(v.x, v.y));
                P1 = cfma(aT1, P1, make_float2(v.z, v.w));
            }
        }
        float2 *out = reinterpret_cast<float2 *>(prm.out);
        const float cl = prm.clampv;
#pragma unroll
        for (int i = 0; i < T; ++i) {
            if (i < nvalid) {
                P0 = cfma(a0, P0, x0[i]);
                P1 = cfma(a1, P1, x1[i]);
                float2 o0 = P0, o1 = P1;
                if (cl > 0.f) {
                    o0.x = clampf(o0.x, cl); o0.y = clampf(o0.y, cl);
                    o1.x = clampf(o1.x, cl); o1.y = clampf(o1.y, cl);
                }
                float2 *r = out + row0 + (long long)i * rowstep;
                if (v0) __stcs(r + c0, o0);
                if (v1) __stcs(r + c1, o1);
                if constexpr (KIND == KIND_BWD) {
                    // conj(lam) * P_{t-1}
                    qa0.x = fmaf(P0.x, q0[i].x, fmaf(P0.y, q0[i].y, qa0.x));
                    qa0.y = fmaf(P0.x, q0[i].y, fmaf(-P0.y, q0[i].x, qa0.y));
                    qa1.x = fmaf(P1.x, q1[i].x, fmaf(P1.y, q1[i].y, qa1.x));
                    qa1.y = fmaf(P1.x, q1[i].y, fmaf(-P1.y, q1[i].x, qa1.y));
                }
            }
        }
        // the thread that owns the last step writes the carried state (never clamped)
        if (prm.state_out != nullptr && nvalid > 0 && s0 + nvalid == L) {
            if (REV) { P0 = cmul(a0, P0); P1 = cmul(a1, P1); }   // grad_state_in = conj(a) lam_0
            if (v0) prm.state_out[(long long)b * C + c0] = P0;
            if (v1) prm.state_out[(long long)b * C + c1] = P1;
        }
    }
    if constexpr (KIND == KIND_BWD) {
        if (prm.qpart != nullptr) {
            __syncthreads();
            sE[w][lane] = make_float4(qa0.x, qa0.y, qa1.x, qa1.y);
            __syncthreads();
            if (w == 0) {
                float4 acc = sE[0][lane];
#pragma unroll
                for (int i = 1; i < W; ++i) {
                    const float4 v = sE[i][lane];
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                float2 *qp = prm.qpart + ((long long)b * K + k) * C;
                if (v0) qp[c0] = make_float2(acc.x, acc.y);
                if (v1) qp[c1] = make_float2(acc.z, acc.w);
            }
        }
    }

    // ---- launch bookkeeping: the last CTA opens the next epoch ------------------------------
    if (tid == 0) {
        const unsigned prev = atomicAdd(&prm.ws->done, 1u);
        if (prev == gridDim.x - 1) {
            prm.ws->done = 0;
            st_volatile_u64(&prm.ws->epoch, epoch + 1ull);
        }
    }
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
