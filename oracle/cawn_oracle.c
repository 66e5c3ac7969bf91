/*
 * CAWN phase-accumulation oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, sequential, fp64 CPU statement of what the Resonance Layer's causal
 * phase accumulation computes.  It exists so that the CUDA library can be
 * checked against something that can be compared with the paper by eye.  It
 * shares no code, header, table or constant with the CUDA path and nothing in
 * the product may call it: only the tests, the smoke check and the benchmark's
 * CPU-baseline leg do.  Nothing here is blocked, fused, vectorised or
 * re-associated: every function walks time once, in order.
 *
 * Array conventions (row-major, "complex" = two consecutive reals re, im):
 *   pushes / outputs   [B, L, C] complex
 *   states             [B, C]    complex
 *   gamma, theta       [C]       (static retention and rotation per channel)
 *   gamma_logit        [B, L, H] and freq_bias [F], C = H*F, j = h*F + k
 *   hidden input h     [B, L, C] real;  conv weights [C, Kc];  tail [B, Kc-1, C]
 * fp32 inputs are promoted element by element; all arithmetic is double.
 *
 * Pins (see tests/test_oracle_*.py): complex geometric series, prefix sum,
 * impulse response, brute-force O(L^2) weighted sums, scipy.signal.lfilter,
 * linearity, chunked == unchunked, gate ties, causal FIR, adjoint identity,
 * brute-force adjoint and central finite differences (also of the fused path's
 * backward, whose straight-through rule is pinned as a projection identity and
 * whose chunked form is pinned against the unchunked one).  No function in
 * this file is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_API __attribute__((visibility("default")))

/* ------------------------------------------------------------------------ */
/* Hard-threshold gate on Cartesian pushes (Section "Multi-Head Dynamic
 * Parameter Projection", item Hard-Threshold Gating: a valve below epsilon is
 * forced to exactly zero, a valve >= epsilon passes unchanged).  Read per
 * complex channel on the phasor magnitude: open <=> |p| >= eps, decided as
 * re^2 + im^2 >= eps^2 in double.  Both squares of fp32 values are exact in
 * double, so the sum is rounded once whatever the compiler contracts.        */
ORACLE_API
void cawn_oracle_gate(int64_t n, const float *p, float gate_eps,
                      double *z, uint8_t *mask)
{
    const double e2 = (double)gate_eps * (double)gate_eps;
    for (int64_t i = 0; i < n; ++i) {
        const double re = (double)p[2 * i], im = (double)p[2 * i + 1];
        const int open = (re * re + im * im >= e2);
        z[2 * i]     = open ? re : 0.0;
        z[2 * i + 1] = open ? im : 0.0;
        if (mask) mask[i] = (uint8_t)open;
    }
}

/* ------------------------------------------------------------------------ */
/* Retention of channel j = h*F + k at (b, t).
 * Static mode: gamma[j].  Dynamic mode (Section "Multi-Head Dynamic Parameter
 * Projection", item 4 and Frequency-Dependent Retention): a per-head logit
 * plus a static per-harmonic bias through a sigmoid.                         */
static double retention(const float *gamma, const float *gamma_logit,
                        const float *freq_bias, int H, int F,
                        int64_t bt, int j)
{
    if (gamma) return (double)gamma[j];
    const int h = j / F, k = j % F;
    const double s = (double)gamma_logit[bt * H + h] + (double)freq_bias[k];
    return 1.0 / (1.0 + exp(-s));
}

/* ------------------------------------------------------------------------ */
/* Causal phase accumulation, Eq. (phase_accum_r), Eq. (phase_accum_i):
 *   P_t = z_t + gamma_t * R(theta_j) * P_{t-1},   P_{-1} = state_in (or 0)
 * written out on real and imaginary parts exactly as the equations do.  The
 * new push is neither decayed nor rotated; the previous state is.
 * P_all (optional) receives the unclamped trajectory, y (optional) the output
 * after Eq. (phase_clamp) (component-wise clamp, applied to the OUTPUT only:
 * the recurrence and state_out carry the unclamped value).
 * clamp_abs <= 0 disables the clamp.                                         */
ORACLE_API
void cawn_oracle_scan(int B, int64_t L, int H, int F,
                      const double *z,
                      const float *gamma, const float *theta,
                      const float *gamma_logit, const float *freq_bias,
                      const double *state_in, double clamp_abs,
                      double *P_all, double *y, double *state_out)
{
    const int C = H * F;
    double *Pr = (double *)malloc(sizeof(double) * (size_t)C);
    double *Pi = (double *)malloc(sizeof(double) * (size_t)C);
    double *cs_j = (double *)malloc(sizeof(double) * (size_t)C);   /* cos theta_j, sin theta_j */
    double *sn_j = (double *)malloc(sizeof(double) * (size_t)C);
    for (int j = 0; j < C; ++j) { cs_j[j] = cos((double)theta[j]); sn_j[j] = sin((double)theta[j]); }
    for (int b = 0; b < B; ++b) {
        for (int j = 0; j < C; ++j) {
            Pr[j] = state_in ? state_in[2 * ((int64_t)b * C + j)] : 0.0;
            Pi[j] = state_in ? state_in[2 * ((int64_t)b * C + j) + 1] : 0.0;
        }
        for (int64_t t = 0; t < L; ++t) {
            const int64_t bt = (int64_t)b * L + t;
            for (int j = 0; j < C; ++j) {
                const double g  = retention(gamma, gamma_logit, freq_bias, H, F, bt, j);
                const double cs = cs_j[j], sn = sn_j[j];
                const int64_t e = 2 * (bt * C + j);
                const double nr = z[e]     + g * (Pr[j] * cs - Pi[j] * sn);
                const double ni = z[e + 1] + g * (Pr[j] * sn + Pi[j] * cs);
                Pr[j] = nr;
                Pi[j] = ni;
                if (P_all) { P_all[e] = nr; P_all[e + 1] = ni; }
                if (y) {
                    double yr = nr, yi = ni;
                    if (clamp_abs > 0.0) {
                        yr = yr > clamp_abs ? clamp_abs : (yr < -clamp_abs ? -clamp_abs : yr);
                        yi = yi > clamp_abs ? clamp_abs : (yi < -clamp_abs ? -clamp_abs : yi);
                    }
                    y[e] = yr; y[e + 1] = yi;
                }
            }
        }
        if (state_out)
            for (int j = 0; j < C; ++j) {
                state_out[2 * ((int64_t)b * C + j)]     = Pr[j];
                state_out[2 * ((int64_t)b * C + j) + 1] = Pi[j];
            }
    }
    free(Pr); free(Pi); free(cs_j); free(sn_j);
}

/* ------------------------------------------------------------------------ */
/* Temporal Syntax Cache prelude + phasor map + gate + push.
 *  (1) causal depthwise conv over time, left padding Kc-1 (Section "Temporal
 *      Syntax Cache"): u_t = bias + sum_k w[c,k] * h[t-(Kc-1)+k], rows left of
 *      t=0 come from tail_in (the carried last Kc-1 hidden rows, Section
 *      "Throughput and Autoregressive Efficiency": the small history buffer
 *      of the temporal conv) or are zero.  The last tap multiplies the current
 *      token (cross-correlation, as a framework Conv1d does).
 *  (2) optionally clamp to [-50,50] then SiLU (same section).
 *  (3) per-channel phasor map: magnitude m = sigmoid(x), phase = pi*tanh(x)
 *      (the benchmark's stand-in for the dense amplitude/phase projections).
 *  (4) hard gate on the magnitude, then Eq. (gated_push_r), Eq. (gated_push_i):
 *      z = m * (cos phase, sin phase) when open, exactly 0 when closed.
 * VALUES are computed in double.  The gate DECISION is an integer taken from
 * floating point, so it is taken in the arithmetic the fp32 method uses:
 * u32 = fmaf chain in tap order k=0..Kc-1 starting from bias (or +0.0f), all
 * in fp32 (fmaf is correctly rounded, so this is bit-reproducible anywhere);
 * without clamp+SiLU:  open <=> u32 >= tau, tau = logit(eps) rounded to fp32
 *                      by the caller (sigmoid is monotone, so this is
 *                      m >= eps without evaluating the sigmoid);
 * with clamp+SiLU:     open <=> sigmoid(x) >= eps in double.  SiLU >= -0.2785
 *                      so m >= 0.43 always: for eps < 0.43 every gate is open.
 * tail_out receives the last Kc-1 hidden rows seen (tail_in rows when L is
 * shorter than Kc-1).                                                        */
ORACLE_API
void cawn_oracle_prelude(int B, int64_t L, int C,
                         const float *h, const float *w, const float *bias,
                         int Kc, int clamp_silu,
                         const float *tail_in, float gate_eps, float gate_tau,
                         double *z, uint8_t *mask, float *tail_out)
{
    const double PI = 3.14159265358979323846;
    const int Kh = Kc - 1;
    for (int b = 0; b < B; ++b) {
        for (int64_t t = 0; t < L; ++t) {
            for (int c = 0; c < C; ++c) {
                double u = bias ? (double)bias[c] : 0.0;
                float u32 = bias ? bias[c] : 0.0f;
                for (int k = 0; k < Kc; ++k) {
                    const int64_t s = t - Kh + k;      /* source time step */
                    float hv;
                    if (s >= 0)       hv = h[((int64_t)b * L + s) * C + c];
                    else if (tail_in) hv = tail_in[((int64_t)b * Kh + (Kh + s)) * C + c];
                    else              hv = 0.0f;
                    u  += (double)w[(int64_t)c * Kc + k] * (double)hv;
                    u32 = fmaf(w[(int64_t)c * Kc + k], hv, u32);
                }
                double x = u;
                int open;
                if (clamp_silu) {
                    x = x > 50.0 ? 50.0 : (x < -50.0 ? -50.0 : x);
                    x = x / (1.0 + exp(-x));
                }
                const double m  = 1.0 / (1.0 + exp(-x));
                const double ph = PI * tanh(x);
                if (clamp_silu) open = (m >= (double)gate_eps);
                else            open = (u32 >= gate_tau);
                const int64_t e = ((int64_t)b * L + t) * C + c;
                z[2 * e]     = open ? m * cos(ph) : 0.0;
                z[2 * e + 1] = open ? m * sin(ph) : 0.0;
                if (mask) mask[e] = (uint8_t)open;
            }
        }
        if (tail_out)
            for (int r = 0; r < Kh; ++r) {
                const int64_t s = L - Kh + r;          /* source time step */
                for (int c = 0; c < C; ++c) {
                    float hv;
                    if (s >= 0)       hv = h[((int64_t)b * L + s) * C + c];
                    else if (tail_in) hv = tail_in[((int64_t)b * Kh + (Kh + s)) * C + c];
                    else              hv = 0.0f;
                    tail_out[((int64_t)b * Kh + r) * C + c] = hv;
                }
            }
    }
}

/* ------------------------------------------------------------------------ */
/* Reverse-time adjoint of the accumulation (the custom backward the paper
 * describes in Section "Complex Domain Synthesis and Hardware Compilation":
 * gradients for the pushes and the retention; the rotation and initial-state
 * gradients are the benchmark's additions).
 *
 * With the real loss  Loss = sum Re(conj(G_t) y_t) + Re(conj(dS_out) P_{L-1})
 * and the clamp treated as pass-through (the paper: hitting the bound does not
 * stop the gradient), the adjoint state is
 *   lam_t = G_t + conj(a_{t+1}) lam_{t+1},  lam_{L-1} = G_{L-1} + dS_out,
 *   a_t = gamma_t e^{i theta}.
 * The hard gate is a straight-through estimator: d z / d p = identity, so the
 * push gradient is lam_t at every position, open or closed.
 *   d gamma_t(b,t,j)  = Re(conj(lam_t) e^{i theta_j} P_{t-1})
 *   d theta_j        += Re(conj(lam_t) i a_t P_{t-1})
 *   d state_in        = conj(a_0) lam_0
 * Static mode sums d gamma_t over (b,t) into dgamma[C].  Dynamic mode chains
 * through the sigmoid: s = gamma(1-gamma) d gamma_t, added to
 * dgamma_logit[b,t,h] (sum over k) and dfreq_bias[k] (sum over b,t,h).
 * z is the gated push trajectory (double) that the forward consumed; the
 * forward trajectory is recomputed here, sequentially, and kept.
 * grad_clamp_abs > 0 clamps the returned dp and dgamma component-wise (same
 * section); <= 0 disables.                                                   */
ORACLE_API
void cawn_oracle_scan_bwd(int B, int64_t L, int H, int F,
                          const double *z,
                          const float *gamma, const float *theta,
                          const float *gamma_logit, const float *freq_bias,
                          const double *state_in,
                          const float *G, const double *dstate_out,
                          double grad_clamp_abs,
                          double *dp, double *dgamma, double *dtheta,
                          double *dstate_in,
                          double *dgamma_logit, double *dfreq_bias)
{
    const int C = H * F;
    const size_t n = (size_t)B * (size_t)L * (size_t)C;
    double *P = (double *)malloc(sizeof(double) * 2 * (n ? n : 1));
    cawn_oracle_scan(B, L, H, F, z, gamma, theta, gamma_logit, freq_bias,
                     state_in, 0.0, P, NULL, NULL);

    if (dgamma) memset(dgamma, 0, sizeof(double) * (size_t)C);
    if (dtheta) memset(dtheta, 0, sizeof(double) * (size_t)C);
    if (dgamma_logit) memset(dgamma_logit, 0, sizeof(double) * (size_t)B * (size_t)L * (size_t)H);
    if (dfreq_bias) memset(dfreq_bias, 0, sizeof(double) * (size_t)F);

    for (int b = 0; b < B; ++b) {
        for (int j = 0; j < C; ++j) {
            const double cs = cos((double)theta[j]), sn = sin((double)theta[j]);
            /* carry = conj(a_{t+1}) lam_{t+1}; at t = L-1 it is dS_out */
            double cr = dstate_out ? dstate_out[2 * ((int64_t)b * C + j)] : 0.0;
            double ci = dstate_out ? dstate_out[2 * ((int64_t)b * C + j) + 1] : 0.0;
            for (int64_t t = L - 1; t >= 0; --t) {
                const int64_t bt = (int64_t)b * L + t;
                const int64_t e = 2 * (bt * C + j);
                const double lr = (double)G[e] + cr;
                const double li = (double)G[e + 1] + ci;
                if (dp) { dp[e] = lr; dp[e + 1] = li; }
                /* previous state P_{t-1} */
                double qr, qi;
                if (t > 0) { qr = P[e - 2 * C]; qi = P[e - 2 * C + 1]; }
                else if (state_in) { qr = state_in[2 * ((int64_t)b * C + j)];
                                     qi = state_in[2 * ((int64_t)b * C + j) + 1]; }
                else { qr = 0.0; qi = 0.0; }
                const double g = retention(gamma, gamma_logit, freq_bias, H, F, bt, j);
                /* rotated previous state  R = e^{i theta} P_{t-1} */
                const double rr = qr * cs - qi * sn;
                const double ri = qr * sn + qi * cs;
                /* Re(conj(lam) R) and Re(conj(lam) i g R) = g (-lr*ri + li*rr) */
                const double dg = lr * rr + li * ri;
                const double dth = g * (li * rr - lr * ri);
                if (dtheta) dtheta[j] += dth;
                if (gamma) {
                    if (dgamma) dgamma[j] += dg;
                } else {
                    const double s = g * (1.0 - g) * dg;
                    if (dgamma_logit) dgamma_logit[bt * H + j / F] += s;
                    if (dfreq_bias) dfreq_bias[j % F] += s;
                }
                /* conj(a_t) lam_t : conj(a) = g (cs - i sn) */
                cr = g * (lr * cs + li * sn);
                ci = g * (li * cs - lr * sn);
            }
            if (dstate_in) {
                dstate_in[2 * ((int64_t)b * C + j)]     = cr;
                dstate_in[2 * ((int64_t)b * C + j) + 1] = ci;
            }
        }
    }
    if (grad_clamp_abs > 0.0) {
        const double c = grad_clamp_abs;
        if (dp) for (size_t i = 0; i < 2 * n; ++i)
            dp[i] = dp[i] > c ? c : (dp[i] < -c ? -c : dp[i]);
        if (dgamma) for (int j = 0; j < C; ++j)
            dgamma[j] = dgamma[j] > c ? c : (dgamma[j] < -c ? -c : dgamma[j]);
    }
    free(P);
}

/* ------------------------------------------------------------------------ */
/* Backward of the prelude (cawn_oracle_prelude) for a given push gradient
 * dz = dLoss/dz (complex, as cawn_oracle_scan_bwd returns it in dp).
 *
 * Chain, per (b, t, c), with u, x, m, phase and the gate decision recomputed
 * exactly as the forward does:
 *   z = m_used (cos ph, sin ph),  m_used = m if open else 0
 *   Straight-through gate (Section "Multi-Head Dynamic Parameter Projection",
 *   Hard-Threshold Gating: beta = beta_hard - sg(beta) + beta): the forward
 *   value of the magnitude is the gated one, its derivative with respect to
 *   the ungated magnitude is 1 whether the gate is open or not.  Hence
 *     dm  = Re(conj(dz) e^{i ph})        = dz_r cos ph + dz_i sin ph   (unmasked)
 *     dph = Re(conj(dz) i z)             = m_used (-dz_r sin ph + dz_i cos ph)
 *   m = sigmoid(x), ph = pi tanh(x):
 *     dx = dm m (1 - m) + dph pi (1 - tanh(x)^2)
 *   optional clamp to [-50,50] then SiLU (x = silu(clamp(u))): the clamp passes
 *   the gradient inside the closed interval, silu'(v) = s (1 + v (1 - s)),
 *   s = sigmoid(v); otherwise du = dx.
 *   conv: u_t = bias + sum_k w[c,k] hrow(t-(Kc-1)+k), hrow(s) = h[s] for s >= 0,
 *   the carried tail for s < 0:
 *     dbias[c] += du,  dw[c,k] += du hrow(s),  dh[s] += w[c,k] du  (s >= 0),
 *     dtail_in[Kh+s] += w[c,k] du (s < 0).
 * dtail_out (optional, [B,Kc-1,C]) is the gradient arriving on this call's
 * tail_out, i.e. on its last Kc-1 hidden rows as seen by the NEXT call: it is
 * added to dh of those rows (and, when the call is shorter than Kc-1, to
 * dtail_in of the rows it passed through).
 * Outputs dh [B,L,C], dw [C,Kc], dbias [C] (may be NULL), dtail_in (may be
 * NULL), all double, all overwritten.                                        */
ORACLE_API
void cawn_oracle_prelude_bwd(int B, int64_t L, int C,
                             const float *h, const float *w, const float *bias,
                             int Kc, int clamp_silu,
                             const float *tail_in, float gate_eps, float gate_tau,
                             const double *dz, const double *dtail_out,
                             double *dh, double *dw, double *dbias, double *dtail_in)
{
    const double PI = 3.14159265358979323846;
    const int Kh = Kc - 1;
    memset(dh, 0, sizeof(double) * (size_t)B * (size_t)L * (size_t)C);
    memset(dw, 0, sizeof(double) * (size_t)C * (size_t)Kc);
    if (dbias) memset(dbias, 0, sizeof(double) * (size_t)C);
    if (dtail_in) memset(dtail_in, 0, sizeof(double) * (size_t)B * (size_t)Kh * (size_t)C);
    for (int b = 0; b < B; ++b) {
        for (int64_t t = 0; t < L; ++t) {
            for (int c = 0; c < C; ++c) {
                double u = bias ? (double)bias[c] : 0.0;
                float u32 = bias ? bias[c] : 0.0f;
                for (int k = 0; k < Kc; ++k) {
                    const int64_t s = t - Kh + k;
                    float hv;
                    if (s >= 0)       hv = h[((int64_t)b * L + s) * C + c];
                    else if (tail_in) hv = tail_in[((int64_t)b * Kh + (Kh + s)) * C + c];
                    else              hv = 0.0f;
                    u  += (double)w[(int64_t)c * Kc + k] * (double)hv;
                    u32 = fmaf(w[(int64_t)c * Kc + k], hv, u32);
                }
                double x = u, dxdu = 1.0;
                if (clamp_silu) {
                    const double v = u > 50.0 ? 50.0 : (u < -50.0 ? -50.0 : u);
                    const double sg = 1.0 / (1.0 + exp(-v));
                    x = v * sg;
                    dxdu = (u >= -50.0 && u <= 50.0) ? sg * (1.0 + v * (1.0 - sg)) : 0.0;
                }
                const double m  = 1.0 / (1.0 + exp(-x));
                const double th = tanh(x);
                const double ph = PI * th;
                const int open = clamp_silu ? (m >= (double)gate_eps) : (u32 >= gate_tau);
                const int64_t e = ((int64_t)b * L + t) * C + c;
                const double dzr = dz[2 * e], dzi = dz[2 * e + 1];
                const double cs = cos(ph), sn = sin(ph);
                const double dm  = dzr * cs + dzi * sn;
                const double dph = (open ? m : 0.0) * (-dzr * sn + dzi * cs);
                const double dx  = dm * m * (1.0 - m) + dph * PI * (1.0 - th * th);
                const double du  = dx * dxdu;
                if (dbias) dbias[c] += du;
                for (int k = 0; k < Kc; ++k) {
                    const int64_t s = t - Kh + k;
                    const double wk = (double)w[(int64_t)c * Kc + k];
                    if (s >= 0) {
                        dw[(int64_t)c * Kc + k] += du * (double)h[((int64_t)b * L + s) * C + c];
                        dh[((int64_t)b * L + s) * C + c] += wk * du;
                    } else {
                        if (tail_in)
                            dw[(int64_t)c * Kc + k] += du * (double)tail_in[((int64_t)b * Kh + (Kh + s)) * C + c];
                        if (dtail_in) dtail_in[((int64_t)b * Kh + (Kh + s)) * C + c] += wk * du;
                    }
                }
            }
        }
        if (dtail_out)
            for (int r = 0; r < Kh; ++r) {
                const int64_t s = L - Kh + r;          /* the hidden row tail_out[r] holds */
                for (int c = 0; c < C; ++c) {
                    const double g = dtail_out[((int64_t)b * Kh + r) * C + c];
                    if (s >= 0) dh[((int64_t)b * L + s) * C + c] += g;
                    else if (dtail_in) dtail_in[((int64_t)b * Kh + (Kh + s)) * C + c] += g;
                }
            }
    }
}
