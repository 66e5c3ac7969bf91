/*
 * libcawn -- causal phase accumulation of the CAWN Resonance Layer on NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every pointer is caller-owned; "device" pointers are CUDA global memory of the
 * current device, "host" pointers are ordinary (preferably pinned) host memory.  The
 * library calls no allocator, and its scratch lives in a caller-provided workspace, with two
 * exceptions that keep state inside the library: cawn_phase_accumulate_fwd_host creates, on its
 * first large call per device, two copy streams and a handful of events that it keeps and
 * serialises behind a lock; cawn_phase_accumulate_fwd_static uses a 4 MiB __device__ array that
 * is part of the library image and shared by all calls on a device (serialise them).
 * Calls are asynchronous on the given CUDA stream
 * (a cudaStream_t passed as void*; NULL = the legacy default stream) unless stated.
 *
 * Shapes.  B batch, L time steps, H heads, F harmonics per head, C = H*F complex channels,
 * flat channel index j = h*F + k.  "complex64" = two consecutive floats (re, im).
 *   pushes / outputs / gradients   [B, L, C] complex64, C contiguous
 *   states                         [B, C]    complex64
 *   gamma, theta                   [C]       float   (retention, rotation in rad/step)
 *   gate mask                      [B, L, ceil(C/32)] uint32, bit (j%32) of word j/32
 * Arrays of shape [B,L,*] and the workspace must be 16-byte aligned, the others 8-byte.
 *
 * The operation (paper: Section "Causal Phase Accumulation and Positional Injection").
 *   z_t   = p_t if |p_t| >= gate_eps else 0               hard-threshold gate
 *   P_t   = z_t + gamma_j e^{i theta_j} P_{t-1}           Eq. (phase_accum_r), Eq. (phase_accum_i)
 *   P_-1  = state_in (0 when NULL)
 *   y_t   = clamp(P_t, +-clamp_abs) component-wise        Eq. (phase_clamp); output only
 *   state_out = P_{L-1}, never clamped                    O(1) state passing
 * All arithmetic is float32 on float32 data; per-channel coefficients are prepared in
 * double inside the kernels.
 *
 * Errors.  Every entry point returns a cawn_status.  Negative values mean the call was
 * rejected before anything was launched.  Conditions found on the device (a carry wait that
 * ran out) are recorded in the workspace and read with cawn_poll_status().  Nothing aborts,
 * traps or waits without a bound.
 */
#ifndef CAWN_H_
#define CAWN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define CAWN_API __attribute__((visibility("default")))
#else
#define CAWN_API
#endif

typedef enum cawn_status {
    CAWN_OK                       = 0,
    CAWN_ERR_INVALID_ARG          = -1,  /* bad struct_size, negative size, unknown op/flag     */
    CAWN_ERR_NULL_POINTER         = -2,  /* a required pointer is NULL                           */
    CAWN_ERR_MISALIGNED           = -3,  /* a pointer breaks the alignment rule above            */
    CAWN_ERR_UNSUPPORTED          = -4,  /* valid request this build has no kernel for           */
    CAWN_ERR_WORKSPACE_TOO_SMALL  = -5,
    CAWN_ERR_CUDA                 = -6,  /* a CUDA runtime call failed (launch, copy)            */
    CAWN_ERR_STATIC_TOO_LARGE     = -7,  /* cawn_phase_accumulate_fwd_static: the call needs more
                                            scratch than the library's built-in array holds      */
    CAWN_ERR_CARRY_TIMEOUT        = 1,   /* device: an inter-tile carry wait hit its bound;
                                            outputs of that call are incomplete                  */
    CAWN_STATUS_NONFINITE         = 2    /* device: an Inf or NaN was accumulated (an Inf input, a
                                            non-finite carried state, an overflow); outputs are
                                            complete but contain such values.  NaN pushes alone do
                                            not raise it: they fail the gate's comparison and are
                                            dropped.  The two device conditions are bits: a poll may
                                            return 3 when both occurred.                          */
} cawn_status;

enum {
    CAWN_FLAG_PRELUDE_CLAMP_SILU = 1u << 0, /* fused path: clamp conv output to +-50, then SiLU   */
    CAWN_FLAG_RETENTION_DYNAMIC  = 1u << 1, /* gamma_t = sigmoid(gamma_logit[b,t,h] + freq_bias[k]) */
    CAWN_FLAG_INPUT_INDEPENDENT  = 1u << 2, /* forward: the caller vouches that `input`, gamma, theta
                                               (and the conv weights) are not written by the call
                                               made just before this one on the same stream.  The
                                               kernels are launched so that a call may start while the
                                               previous one drains (programmatic dependent launch);
                                               with this flag the new call also fetches its input rows
                                               during that overlap.  States, masks, workspaces and all
                                               outputs are only touched once the previous call is
                                               complete, with or without the flag.                    */
    CAWN_FLAG_INPUT_BF16         = 1u << 3, /* forward: `input` is stored as bfloat16 (Cartesian: pairs
                                               (re, im) of bf16, 4 bytes per channel; fused path: one
                                               bf16 per channel) and widened, exactly, to float on load */
    CAWN_FLAG_OUTPUT_BF16        = 1u << 4  /* forward: `y` is stored as pairs (re, im) of bfloat16,
                                               each component rounded to nearest even from the fp32
                                               result.  With either flag the recurrence, the carried
                                               state, state_out and the conv history stay fp32 (the
                                               paper runs a bf16 network around an fp32 scan:
                                               Section "Mixed-Precision and Float32
                                               Stabilization").  With the time-varying retention or the
                                               Ear epilogue (the paper's own layer form) the two flags
                                               come together or not at all; the Ear's z_conv is then
                                               bfloat16 [B, L, 2, H, K].  Not available for the
                                               host-staged forward or any backward:
                                               CAWN_ERR_UNSUPPORTED.                                    */
};

/* Operation selector of cawn_workspace_bytes(). */
enum {
    CAWN_OP_FWD        = 0,  /* workspace of cawn_phase_accumulate_fwd                           */
    CAWN_OP_BWD_SAVED  = 1,  /* workspace of cawn_phase_accumulate_bwd with CAWN_SAVED_STATES    */
    CAWN_OP_BWD_PUSHES = 2,  /* ... with CAWN_SAVED_PUSHES (adds room for the recomputed states) */
    CAWN_OP_STATE      = 3,  /* size of one state blob                                           */
    CAWN_OP_FWD_HOST   = 4,  /* device staging + workspace of cawn_phase_accumulate_fwd_host     */
    CAWN_OP_MIXING_BWD = 5   /* workspace of cawn_mixing_bwd                                     */
};

/* What the backward was given to rebuild P_{t-1} from. */
enum {
    CAWN_SAVED_STATES = 0,   /* the forward's unclamped outputs P [B,L,C]                        */
    CAWN_SAVED_PUSHES = 1    /* the forward's input pushes p [B,L,C]; P is recomputed            */
};

/* Plain-data description of one call.  Fill struct_size with sizeof(cawn_params). */
typedef struct cawn_params {
    uint32_t struct_size;
    int32_t  B;              /* batch >= 1                                                       */
    int64_t  L;              /* time steps of this call, >= 0, any value (ragged is fine)        */
    int32_t  H, F;           /* C = H*F >= 1                                                     */
    float    gate_eps;       /* hard-gate threshold on |p| (fused path: on the magnitude m);
                                0 = always open                                                  */
    float    gate_tau;       /* fused path only: logit(gate_eps) rounded to float by the caller;
                                the gate is decided as conv_output >= gate_tau                   */
    float    clamp_abs;      /* output clamp bound (paper: 100); <= 0 disables                   */
    float    grad_clamp_abs; /* backward: clamp returned grad_p and grad_gamma (paper: 100);
                                <= 0 disables                                                    */
    int32_t  conv_k;         /* fused path: conv taps 1..4; 0 = input is Cartesian pushes        */
    uint32_t flags;          /* CAWN_FLAG_*                                                      */
} cawn_params;

/* State blob: P [B,C] complex64 (unclamped), then, at the next 16-byte boundary, the conv
 * history [B, conv_k-1, C] float (raw hidden rows; absent when conv_k <= 1).  This is the
 * fixed-size state the paper carries between chunks, micro-batches and decode steps
 * (Section "Theoretical Advantages", O(1) state passing; Section "Throughput and
 * Autoregressive Efficiency", the 2-step conv history).                                        */

CAWN_API const char *cawn_status_string(int status);

/* Host-only size query.  *bytes receives the size for `op` at these params. */
CAWN_API int cawn_workspace_bytes(const cawn_params *params, int op, size_t *bytes);

/* Zero a freshly allocated workspace (device).  Must run once before its first use; afterwards
 * the kernels keep it consistent themselves.  One workspace serves one call at a time: calls
 * that may overlap on the device need a workspace each.                                         */
CAWN_API int cawn_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Forward phase accumulation (Eq. (gated_push_r/i) gate, Eq. (phase_accum_r/i), Eq. (phase_clamp)).
 *
 * conv_k == 0:  `input` = pushes p [B,L,C] complex64 (device).  y may alias input.
 * conv_k >= 1:  fused Resonance mixing path.  `input` = hidden states h [B,L,C] float (device);
 *               u_t = bias + sum_k conv_w[c,k] h[t-(conv_k-1)+k]   (causal depthwise conv,
 *               Section "Temporal Syntax Cache"; rows left of t=0 from the state blob or zero),
 *               optional clamp+-50 and SiLU, magnitude m = sigmoid(x), phase = pi*tanh(x),
 *               gate, z = m (cos, sin)(phase).
 * gamma/theta:  [C] device.  With CAWN_FLAG_RETENTION_DYNAMIC gamma is ignored and
 *               gamma_logit [B,L,H], freq_bias [F] (device) define the retention
 *               (Section "Multi-Head Dynamic Parameter Projection", item 4); available for
 *               both input forms (with conv_k >= 1 this is the paper's own layer: Temporal
 *               Syntax Cache, gated push and per-token retention in one pass).
 * state_in:     state blob (device) or NULL for a zero state.
 * y:            [B,L,C] complex64 (device), clamped if clamp_abs > 0.
 * state_out:    state blob (device) or NULL.  May alias state_in.
 * gate_mask:    bit-packed mask (device) or NULL.
 * workspace:    device, >= cawn_workspace_bytes(CAWN_OP_FWD), initialised once.
 */
CAWN_API int cawn_phase_accumulate_fwd(const cawn_params *params,
                                       const void *input,
                                       const float *gamma, const float *theta,
                                       const float *conv_w, const float *conv_bias,
                                       const float *gamma_logit, const float *freq_bias,
                                       const void *state_in,
                                       void *y, void *state_out, uint32_t *gate_mask,
                                       void *workspace, size_t workspace_bytes,
                                       void *cuda_stream);

/*
 * Backward of the Cartesian forward (the reverse-time adjoint the paper's custom autograd
 * function computes, Section "Complex Domain Synthesis and Hardware Compilation").
 *   lam_t = grad_y_t + conj(a) lam_{t+1},  lam_{L-1} = grad_y_{L-1} + grad_state_out
 *   grad_p_t = lam_t at every position (straight-through gate; clamp passes gradient)
 *   grad_gamma_j = sum_{b,t} Re(conj(lam_t) e^{i theta_j} P_{t-1})
 *   grad_theta_j = sum_{b,t} Re(conj(lam_t) i a_j P_{t-1})
 *   grad_state_in = conj(a) lam_0
 * saved / saved_kind: CAWN_SAVED_STATES -> the forward's UNCLAMPED y; CAWN_SAVED_PUSHES -> the
 *               forward's pushes (re-gated and re-scanned into the workspace first).
 * grad_y:       [B,L,C] complex64 (device).  grad_p may alias it.
 * grad_state_out, state_in: [B,C] complex64 (device) or NULL (= 0).
 * grad_gamma, grad_theta: [C] float (device) or NULL.  grad_state_in: [B,C] complex64 or NULL.
 * Deterministic: partial sums are combined in a fixed order in double.
 * Static retention only (see cawn_phase_accumulate_bwd_dynamic for the other form).
 */
CAWN_API int cawn_phase_accumulate_bwd(const cawn_params *params,
                                       const void *saved, int saved_kind,
                                       const float *gamma, const float *theta,
                                       const void *state_in,
                                       const void *grad_y, const void *grad_state_out,
                                       void *grad_p, float *grad_gamma, float *grad_theta,
                                       void *grad_state_in,
                                       void *workspace, size_t workspace_bytes,
                                       void *cuda_stream);

/*
 * Backward with the paper's time-varying retention (Section "Multi-Head Dynamic Parameter
 * Projection", item 4: gamma_{t,h,k} = sigmoid(W_gamma x_t + b_k), the projection per head and a
 * static per-harmonic bias).  params->flags must carry CAWN_FLAG_RETENTION_DYNAMIC.
 *   a_t = gamma_t e^{i theta},  lam_t = grad_y_t + conj(a_{t+1}) lam_{t+1}
 *   d gamma_t(b,t,j) = Re(conj(lam_t) e^{i theta_j} P_{t-1}),  s = gamma_t (1 - gamma_t) d gamma_t
 *   grad_gamma_logit[b,t,h] = sum_k s      grad_freq_bias[k] = sum_{b,t,h} s
 *   grad_theta_j = sum_{b,t} Re(conj(lam_t) i a_t P_{t-1})      grad_state_in = conj(a_0) lam_0
 * gamma_logit [B,L,H], freq_bias [F] (device).  grad_gamma_logit [B,L,H] float, grad_freq_bias [F]
 * float, grad_theta [C] float: device or NULL.  Other arguments as cawn_phase_accumulate_bwd.
 * grad_gamma_logit: where a 64-channel group holds whole heads (F divides 64, or C <= 64) every entry
 * is the sum of one warp and is stored; otherwise the call zeroes the array and accumulates with
 * atomic adds, and when a head spans three or more groups (F > 128) its last bits may differ from
 * run to run.  Everything else is bitwise repeatable.
 */
CAWN_API int cawn_phase_accumulate_bwd_dynamic(const cawn_params *params,
                                               const void *saved, int saved_kind,
                                               const float *gamma_logit, const float *freq_bias,
                                               const float *theta, const void *state_in,
                                               const void *grad_y, const void *grad_state_out,
                                               void *grad_p, float *grad_gamma_logit,
                                               float *grad_freq_bias, float *grad_theta,
                                               void *grad_state_in,
                                               void *workspace, size_t workspace_bytes,
                                               void *cuda_stream);

/*
 * Backward of the fused Resonance mixing path (cawn_phase_accumulate_fwd with conv_k >= 1,
 * static retention): the reverse scan with the prelude's chain rule as its epilogue, one pass
 * over grad_y, the saved states and h.
 *   lam   = reverse scan of grad_y (as cawn_phase_accumulate_bwd); it is the gradient of the pushes
 *   magnitude m = sigmoid(x), phase ph = pi tanh(x), push z = m_used (cos ph, sin ph):
 *     d m  = Re(conj(lam) e^{i ph})                    straight-through: flows open or closed
 *     d ph = m_used (-lam_r sin ph + lam_i cos ph)     m_used = m if the gate is open else 0
 *   (the paper's hard-threshold gate with straight-through estimator, Section "Multi-Head Dynamic
 *   Parameter Projection"), through the optional clamp + SiLU and the causal depthwise conv
 *   (Section "Temporal Syntax Cache") to h, conv_w, conv_bias and the carried conv history.
 * h [B,L,C] float, conv_w [C,conv_k], conv_bias [C] or NULL, gamma/theta [C]: as in the forward.
 * saved_states: the forward's UNCLAMPED y [B,L,C] complex64; may be NULL when neither grad_gamma
 *               nor grad_theta is wanted.
 * state_in:     the forward's state blob (its conv history is read) or NULL.
 * grad_y [B,L,C] complex64; grad_state_out: gradient of the forward's state_out blob (state part
 *               and conv-history part, e.g. the next chunk's grad_state_in) or NULL.
 * grad_h [B,L,C] float; grad_conv_w [C,conv_k], grad_conv_bias [C], grad_gamma [C], grad_theta [C]
 *               float or NULL; grad_state_in: state blob of gradients or NULL.  All device.
 * workspace:    >= cawn_workspace_bytes(CAWN_OP_MIXING_BWD), initialised once (carry records, per-tile
 *               partial sums, and the few rows exchanged at tile seams; O(B*C*L/64)).
 * Deterministic (parameter sums: per-CTA partials combined in a fixed order in double).
 */
CAWN_API int cawn_mixing_bwd(const cawn_params *params,
                             const float *h, const float *conv_w, const float *conv_bias,
                             const float *gamma, const float *theta,
                             const void *saved_states, const void *state_in,
                             const void *grad_y, const void *grad_state_out,
                             float *grad_h, float *grad_conv_w, float *grad_conv_bias,
                             float *grad_gamma, float *grad_theta, void *grad_state_in,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * cawn_mixing_bwd with the paper's time-varying retention (the fused path run with
 * CAWN_FLAG_RETENTION_DYNAMIC, which params->flags must carry): the backward of the whole
 * Resonance mixing step as the paper defines it — Temporal Syntax Cache, gated push, per-token
 * per-head retention (Section "Multi-Head Dynamic Parameter Projection").  gamma_logit [B,L,H],
 * freq_bias [F] replace gamma; grad_gamma_logit [B,L,H] (as in cawn_phase_accumulate_bwd_dynamic)
 * and grad_freq_bias [F] replace grad_gamma; each may be NULL.  Everything
 * else as cawn_mixing_bwd, including the workspace size.
 */
CAWN_API int cawn_mixing_bwd_dynamic(const cawn_params *params,
                                     const float *h, const float *conv_w, const float *conv_bias,
                                     const float *gamma_logit, const float *freq_bias, const float *theta,
                                     const void *saved_states, const void *state_in,
                                     const void *grad_y, const void *grad_state_out,
                                     float *grad_h, float *grad_conv_w, float *grad_conv_bias,
                                     float *grad_gamma_logit, float *grad_freq_bias, float *grad_theta,
                                     void *grad_state_in,
                                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Forward with the front of the Convolutional SwiGLU Ear as the scan's epilogue (Eq. (wave_synth)
 * and Section "Projection to Hidden State: The Convolutional SwiGLU Ear", the depth-wise 1-D
 * convolution across the K harmonics).  Everything up to the clamped state y_t is
 * cawn_phase_accumulate_fwd (Cartesian or fused input, static or time-varying retention: with
 * conv_k >= 1 and CAWN_FLAG_RETENTION_DYNAMIC one kernel takes the hidden states through the
 * paper's whole Resonance mixing step up to the Ear's convolution); instead of storing y the
 * kernel writes
 *   Z_t = Concat(Re y_t, Im y_t)  viewed as 2H channels (real heads, then imaginary heads) x K
 *   z_conv[b,t,q,k] = ear_bias[q] + sum_j ear_w[q,j] Z_t[q, k + j - (ear_k-1)/2],  zero outside 0..K-1
 * The paper states neither the tap count nor the padding: taken as ear_k taps (1 or 3; other
 * values -> CAWN_ERR_UNSUPPORTED) with zero padding on both sides, cross-correlation order as in a
 * Conv1d layer.  ear_k = 1 with ear_w = 1 and no bias gives the planar Z itself.
 * ear_w:   [2H, ear_k] float (device).  ear_bias: [2H] float (device) or NULL.
 * z_conv:  [B, L, 2, H, K] float (device, 16-byte aligned), K = params->F; as many bytes as y.
 *          With CAWN_FLAG_INPUT_BF16 | CAWN_FLAG_OUTPUT_BF16 it holds bfloat16 instead (pass the pointer
 *          as it is).
 * state_out (if given) still receives the unclamped, unconvolved P_{L-1} (and the conv history).
 * Limits: K must divide 64 unless H*K <= 64 (a CTA owns 64 adjacent channels and does not read
 * its neighbours' harmonics).
 * Other arguments, ownership, stream order and status reporting as cawn_phase_accumulate_fwd.
 */
CAWN_API int cawn_phase_accumulate_fwd_ear(const cawn_params *params,
                                           const void *input,
                                           const float *gamma, const float *theta,
                                           const float *conv_w, const float *conv_bias,
                                           const float *gamma_logit, const float *freq_bias,
                                           const void *state_in,
                                           const float *ear_w, const float *ear_bias, int ear_k,
                                           float *z_conv, void *state_out, uint32_t *gate_mask,
                                           void *workspace, size_t workspace_bytes,
                                           void *cuda_stream);

/*
 * Associative combine of two segment summaries (static retention):
 *   state_out = a^n_steps * state_prev + state_local,   a_j = gamma_j e^{i theta_j}
 * where state_local is the end state of an n_steps-long segment run from a ZERO state.  This is
 * the O(1) state passing of the paper composed outside a call (prefill that skips outputs,
 * time sharding).  All states [B,C] complex64 (device); state_out may alias either input.
 * a^n is evaluated in double (pow, sincos), not by repeated multiplication.
 */
CAWN_API int cawn_state_carry(const cawn_params *params,
                              const void *state_prev, const void *state_local,
                              int64_t n_steps,
                              const float *gamma, const float *theta,
                              void *state_out, void *cuda_stream);

/* Synchronise `cuda_stream` and return the device-side status recorded in the workspace by
 * the calls so far (CAWN_OK, or the positive conditions CAWN_ERR_CARRY_TIMEOUT and
 * CAWN_STATUS_NONFINITE or-ed together); the record is then cleared.  This is the hook for the
 * paper's stability protocol (Section "Training Stability in the Complex Domain": skip the step
 * on NaN/Inf), without a pass over the outputs.                                                    */
CAWN_API int cawn_poll_status(void *workspace, void *cuda_stream);

/* Test hook for the bounded waits (no counterpart in the paper).  After this call, in every
 * kernel that uses `workspace`, tile number `withhold_tile` (0-based along time, in the kernel's
 * own tile size: 128 steps in the forward, 64 in the backward, 16 for calls of at most 32 steps)
 * of every (batch, channel group) keeps its summary to itself, and every carry wait gives up
 * after `poll_bound` polls (1..65535; 0 keeps the normal bound).  Tiles that depend on the silent
 * one then run into the bound, record CAWN_ERR_CARRY_TIMEOUT, skip their outputs and pass the
 * failure on; the kernel ends, nothing hangs or traps, and the workspace stays usable.
 * withhold_tile < 0 and poll_bound = 0 switch the hook off.  Stream-ordered.                   */
CAWN_API int cawn_workspace_set_wait_hook(void *workspace, int withhold_tile, unsigned poll_bound,
                                          void *cuda_stream);

/*
 * Host-buffer convenience for the Cartesian forward: copies pushes, gamma, theta (and
 * state_in) from HOST memory to the device staging area, runs the forward, copies y
 * (and state_out, gate_mask) back to HOST memory, all on `cuda_stream`, and returns without
 * synchronising.  `device_scratch` (device, >= cawn_workspace_bytes(CAWN_OP_FWD_HOST), zeroed
 * once with cawn_workspace_init) holds staging and workspace.  Static retention, conv_k == 0.
 * Calls of 8 MB and more are cut into up to 8 slices (batch rows, or for B = 1 stretches of time
 * with the state carried: the paper's chunked prefill) that go through two library-owned copy
 * streams, so that slice i is copied out while slice i+1 is copied in; both streams wait for
 * what precedes the call on `cuda_stream` and `cuda_stream` waits for both before anything
 * after it.  The host buffers should be page-locked for the copies to overlap.  The copy streams
 * and their events are created on the first such call per device (the only resources the
 * library ever creates) and calls that use them are serialised by a lock.
 */
CAWN_API int cawn_phase_accumulate_fwd_host(const cawn_params *params,
                                            const void *p_host,
                                            const float *gamma_host, const float *theta_host,
                                            const void *state_in_host,
                                            void *y_host, void *state_out_host,
                                            uint32_t *gate_mask_host,
                                            void *device_scratch, size_t device_scratch_bytes,
                                            void *cuda_stream);

/*
 * Forward phase accumulation for callers that cannot allocate device memory.  (The paper has
 * no counterpart: this is a packaging variant of cawn_phase_accumulate_fwd, same arithmetic.)
 *
 * Who needs it: code that runs where a cudaMalloc is not an option -- a plugin inside a serving
 * process whose device memory has all been handed to one framework-owned pool, a callback that
 * must not block on the allocator or synchronise the device, or a component that is given
 * input and output buffers and nothing else.  Such a caller cannot provide the carry workspace
 * the ordinary entry point asks for, so this one uses a scratch array compiled into the library
 * instead: a file-scope __device__ array of CAWN_STATIC_SCRATCH_BYTES (4 MiB), which every GPU
 * that loads the library holds until the process exits.
 *
 * Same operation and arguments as the Cartesian, static-retention cawn_phase_accumulate_fwd
 * (conv_k == 0, no CAWN_FLAG_RETENTION_DYNAMIC), without the workspace pair.
 * Anything else (conv_k != 0, CAWN_FLAG_RETENTION_DYNAMIC) is refused with CAWN_ERR_UNSUPPORTED;
 * all arguments are validated before anything is put on the stream.
 * device_status: device pointer to one uint32 or NULL.  When given, the device-side status of
 *               this call is copied there on the stream after the kernel: 0, or the bits
 *               CAWN_ERR_CARRY_TIMEOUT (1) and CAWN_STATUS_NONFINITE (2) or-ed together, as
 *               cawn_poll_status would return them; there is no separate poll call for the
 *               built-in scratch.
 *
 * Limits and rules.
 *  - The call is rejected with CAWN_ERR_STATIC_TOO_LARGE, before anything is launched, when
 *    cawn_workspace_bytes(params, CAWN_OP_FWD) exceeds CAWN_STATIC_SCRATCH_BYTES.  The need is
 *    256 + B * ceil(C/64) * (K + K/7 + 1) * 1024 bytes with K = ceil(L/128) tiles: 1.9 MB for
 *    B=8, L=2048, C=768; about 4,000 (batch x 64-channel group x tile) units in all.
 *  - It calls no cudaMalloc/cudaFree and no allocating library routine.
 *  - The first call on each device looks up the array's device address (one
 *    cudaGetSymbolAddress with that device current) and remembers it; make that first call
 *    outside any stream capture.
 *  - All calls on a device share the one array, and it keeps what the last call left in it.
 *    The kernel's epoch tags make stale records harmless and the status word is cleared at the
 *    start of every call, but two calls that overlap on the GPU (different streams, or
 *    different host threads) race on it: serialise them.
 */
#define CAWN_STATIC_SCRATCH_BYTES (4u << 20)
CAWN_API int cawn_phase_accumulate_fwd_static(const cawn_params *params,
                                              const void *input,
                                              const float *gamma, const float *theta,
                                              const void *state_in,
                                              void *y, void *state_out, uint32_t *gate_mask,
                                              uint32_t *device_status,
                                              void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* CAWN_H_ */
