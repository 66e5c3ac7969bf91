// libcawn: C-ABI entry points, argument validation, workspace layout and kernel launches.
#include "../../include/cawn.h"
#include "cawn_launch.cuh"
#include "cawn_small_kernels.cuh"

#include <math.h>
#include <string.h>

#include <mutex>

namespace {

using namespace cawn;

constexpr unsigned kPollLimit = 1u << 20;   // ~1 s of polling before a carry wait gives up

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Long calls use 128-step tiles (8 warps x 16 steps); short ones (decode, tiny chunks) use
// 16-step tiles so that a call is not one mostly empty CTA.
inline TileShape fwd_shape(int64_t L) { return L > 32 ? TileShape{16, 8} : TileShape{4, 4}; }
inline TileShape bwd_shape(int64_t L) { return L > 32 ? TileShape{8, 8} : TileShape{4, 4}; }

// C channels in G groups of 64; K tiles along time, of which every kWindow-th is a checkpoint
// (KP checkpoint slots per chain); MW mask words per row.  Records are 16 bytes per channel.
struct Geometry {
    int C, G, K, KP, MW;
    bool fits;                   // the tile count fits a grid dimension (K is clamped when it does not)
    size_t agg_bytes, pre_bytes, rec_bytes;
};
inline Geometry geometry(const cawn_params *p, TileShape ts)
{
    Geometry g;
    g.C = p->H * p->F;
    g.G = (g.C + 63) / 64;
    const int64_t tile = (int64_t)ts.T * ts.W;
    int64_t K64 = p->L / tile + (p->L % tile != 0 ? 1 : 0);     // no overflow for any L >= 0
    if (K64 < 1) K64 = 1;
    g.fits = K64 <= 65535;
    g.K = g.fits ? (int)K64 : 65535;
    g.KP = g.K / kWindow + 1;
    g.MW = (g.C + 31) / 32;
    g.agg_bytes = (size_t)p->B * g.G * g.K * 64 * sizeof(uint4);
    g.pre_bytes = (size_t)p->B * g.G * g.KP * 64 * sizeof(uint4);
    g.rec_bytes = g.agg_bytes + g.pre_bytes;
    return g;
}

// Carry-record area of a workspace: aggregates, then checkpoint carry-ins.
inline void set_records(ScanParams &sp, char *rec_base, const Geometry &g)
{
    sp.agg = reinterpret_cast<uint4 *>(rec_base);
    sp.pre = reinterpret_cast<uint4 *>(rec_base + g.agg_bytes);
    sp.G = g.G; sp.K = g.K; sp.KP = g.KP; sp.MW = g.MW; sp.C = g.C;
}

// fp32 screen of the gate.  The fp32 sum of squares is within 2^-22 (relative) of the exact
// one, so at a distance of more than 2^-20 eps^2 from fl(eps^2) it already decides the double
// comparison; inside that band the kernel falls back to double.
inline void set_gate(ScanParams &sp, float gate_eps)
{
    const double e2 = (double)gate_eps * (double)gate_eps;
    sp.eps2 = e2;
    if (e2 == 0.0) {                       // always open (NaN compares false in either form)
        sp.gate_mid = 0.f; sp.gate_hw = -1.f; sp.gate_keep = 0.f;
    } else if (e2 < 1e-27) {               // fp32 squares may be subnormal: keep everything in
        sp.gate_mid = 0.f; sp.gate_hw = 1e-24f;   // the first pass, decide small sums in double
        sp.gate_keep = 0.f;
    } else {
        sp.gate_mid = (float)e2;
        sp.gate_hw = nextafterf((float)(e2 / 1048576.0), INFINITY);
        sp.gate_keep = -sp.gate_hw;
    }
}

int check_params(const cawn_params *p)
{
    if (p == nullptr) return CAWN_ERR_NULL_POINTER;
    if (p->struct_size != sizeof(cawn_params)) return CAWN_ERR_INVALID_ARG;
    if (p->B < 1 || p->L < 0 || p->H < 1 || p->F < 1) return CAWN_ERR_INVALID_ARG;
    if ((int64_t)p->H * p->F > (1 << 24)) return CAWN_ERR_INVALID_ARG;
    if (p->conv_k < 0) return CAWN_ERR_INVALID_ARG;
    if (p->flags & ~(uint32_t)(CAWN_FLAG_PRELUDE_CLAMP_SILU | CAWN_FLAG_RETENTION_DYNAMIC | CAWN_FLAG_INPUT_INDEPENDENT |
                                 CAWN_FLAG_INPUT_BF16 | CAWN_FLAG_OUTPUT_BF16))
        return CAWN_ERR_INVALID_ARG;
    if (!(p->gate_eps >= 0.f)) return CAWN_ERR_INVALID_ARG;
    // every byte count derived from B*L*C (16 bytes per element at most, a few arrays) must fit 63 bits
    if ((double)p->B * (double)p->L * (double)p->H * (double)p->F > 1.0e17) return CAWN_ERR_UNSUPPORTED;
    return CAWN_OK;
}

size_t state_blob_bytes(const cawn_params *p)
{
    const size_t C = (size_t)p->H * p->F;
    size_t n = round_up((size_t)p->B * C * sizeof(float2), 16);
    if (p->conv_k > 1) n += round_up((size_t)p->B * (p->conv_k - 1) * C * sizeof(float), 16);
    return n;
}

// Grid size check: tiles are a (G, B, K) grid.
inline bool grid_ok(const cawn_params *p, const Geometry &g)
{
    return g.fits && p->B <= 65535 && g.K <= 65535 && (double)p->B * g.G * g.K < 4294967295.0;
}

// First-wave stagger of the static forward scan: about two thirds of the time one SM's share of
// HBM bandwidth needs for a tile's input and output.  Device numbers are read once per device.
void set_stagger(ScanParams &sp, TileShape ts, int bytes_per_element = 16)
{
    static int sms[64] = {}, cycles_per_byte_q20[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return;
    if (sms[dev] == 0) {
        int n = 0, mem_khz = 0, bus_bits = 0, sm_khz = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&mem_khz, cudaDevAttrMemoryClockRate, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&bus_bits, cudaDevAttrGlobalMemoryBusWidth, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_khz, cudaDevAttrClockRate, dev) != cudaSuccess ||
            n <= 0 || mem_khz <= 0 || bus_bits <= 0 || sm_khz <= 0)
            return;
        // achievable bandwidth taken as 0.8 of 2 x memory clock x bus width, split over the SMs
        const double bytes_per_s = 0.8 * 2.0 * (double)mem_khz * 1e3 * (double)bus_bits / 8.0 / (double)n;
        cycles_per_byte_q20[dev] = (int)((double)sm_khz * 1e3 / bytes_per_s * 1048576.0);
        sms[dev] = n;
    }
    const long long tile_bytes = (long long)ts.T * ts.W * 64 * bytes_per_element;   // input + output of one tile
    sp.stagger_cycles = (int)((tile_bytes * cycles_per_byte_q20[dev] * 2 / 3) >> 20);
    sp.stagger_group = sms[dev];
    sp.stagger_slots = 3;
}

// The backward's epilogue launch: the parameter sums that were asked for and, for the fused path,
// the rows at the tile seams.  Jobs that are not wanted get no blocks.
cudaError_t launch_epilogue(EpilogueParams ep, bool want_q, bool want_s, bool want_c, bool want_seams, cudaStream_t st)
{
    ep.nb_q = want_q ? (ep.C + kEpiCW - 1) / kEpiCW : 0;
    ep.nb_s = want_s ? (ep.F + kEpiFW - 1) / kEpiFW : 0;
    ep.nb_c = want_c ? (ep.C + kEpiCW - 1) / kEpiCW : 0;
    ep.nb_ex = (ep.C + kEpiWarps * 32 - 1) / (kEpiWarps * 32);
    const long long seams = want_seams ? (long long)ep.nb_ex * ((ep.K + kEpiSeams) / kEpiSeams) * ep.B : 0;
    const long long blocks = (long long)ep.nb_q + ep.nb_s + ep.nb_c + seams;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 2147483647ll) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, 1, 1);
    cfg.blockDim = dim3(kEpiWarps * 32, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, cawn_bwd_epilogue_kernel, ep);
}

// The logit gradient of a (row, head) is complete inside one 64-channel group when the group holds
// whole heads: it is then stored, not accumulated, and needs no zeroing first.
inline bool logit_grad_direct(const cawn_params *p)
{
    const long long C = (long long)p->H * p->F;
    return C <= 64 || (p->F <= 64 && 64 % p->F == 0);
}

constexpr uint32_t kBf16Flags = CAWN_FLAG_INPUT_BF16 | CAWN_FLAG_OUTPUT_BF16;
inline int io_of(const cawn_params *p)
{
    return ((p->flags & CAWN_FLAG_INPUT_BF16) ? IO_IN_BF16 : 0) | ((p->flags & CAWN_FLAG_OUTPUT_BF16) ? IO_OUT_BF16 : 0);
}

inline cudaError_t launch_fwd(TileShape ts, const ScanParams &sp, cudaStream_t st, bool dyn = false, int io = 0)
{
    if (io != 0 && (dyn || sp.ear_w != nullptr)) return launch_fwd_bf16_wide(ts, sp, st, dyn);
    if (io != 0) return launch_fwd_bf16(ts, sp, st, io);
    if (sp.ear_w != nullptr) return dyn ? launch_fwd_ear_dynamic(ts, sp, st) : launch_fwd_ear(ts, sp, st);
    return dyn ? launch_fwd_dynamic(ts, sp, st) : launch_fwd_static(ts, sp, st);
}
inline cudaError_t launch_fused(TileShape ts, const ScanParams &sp, cudaStream_t st, int io = 0, bool dyn = false)
{
    if (io != 0 && (dyn || sp.ear_w != nullptr)) return launch_fused_bf16_wide(ts, sp, st, dyn);
    if (dyn) return sp.ear_w != nullptr ? launch_fused_ear_dynamic(ts, sp, st) : launch_fused_dynamic(ts, sp, st);
    if (io != 0) return launch_fused_bf16(ts, sp, st, io);
    return sp.ear_w != nullptr ? launch_fused_ear(ts, sp, st) : launch_fused_plain(ts, sp, st);
}
inline cudaError_t launch_bwd(TileShape ts, const ScanParams &sp, cudaStream_t st, bool dyn = false)
{
    return dyn ? launch_bwd_dynamic(ts, sp, st) : launch_bwd_static(ts, sp, st);
}

// Workspace of cawn_mixing_bwd: header, carry records, per-tile sums for grad_gamma / grad_theta,
// du at the tile seams, per-tile sums for the conv gradients.
struct MixBwdLayout {
    size_t off_rec, off_qpart, off_spart, off_edge, off_cpart, total;
};
MixBwdLayout mix_bwd_layout(const cawn_params *p)
{
    const Geometry g = geometry(p, bwd_shape(p->L));
    const size_t tiles = (size_t)p->B * g.K;
    MixBwdLayout m;
    size_t o = sizeof(WsHeader);
    m.off_rec = o;    o += round_up(g.rec_bytes, 256);
    m.off_qpart = o;  o += round_up(tiles * g.C * sizeof(float2), 256);
    m.off_spart = o;  o += round_up(tiles * g.C * sizeof(float), 256);
    m.off_edge = o;   o += round_up(tiles * 6 * g.C * sizeof(float), 256);
    m.off_cpart = o;  o += round_up(tiles * g.C * 5 * sizeof(float), 256);
    m.total = o;
    return m;
}

// Host-staged forward: layout of the device scratch.
struct HostStage {
    size_t off_x, off_gamma, off_theta, off_state, off_mask, off_ws, total;
};
HostStage host_stage(const cawn_params *p)
{
    const Geometry g = geometry(p, fwd_shape(p->L));
    const size_t n = (size_t)p->B * (size_t)p->L * g.C;
    HostStage h;
    size_t o = 0;
    h.off_x = o;      o += round_up(n * sizeof(float2), 256);
    h.off_gamma = o;  o += round_up((size_t)g.C * sizeof(float), 256);
    h.off_theta = o;  o += round_up((size_t)g.C * sizeof(float), 256);
    h.off_state = o;  o += round_up((size_t)p->B * g.C * sizeof(float2), 256);
    h.off_mask = o;   o += round_up((size_t)p->B * (size_t)p->L * g.MW * sizeof(uint32_t), 256);
    h.off_ws = o;     o += sizeof(WsHeader) + g.rec_bytes;
    h.total = o;
    return h;
}

// Built-in scratch of cawn_phase_accumulate_fwd_static: lives in every GPU that loads the
// library.  In host code this name is only a handle; the device address comes from
// cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[CAWN_STATIC_SCRATCH_BYTES];

cudaError_t static_scratch_address(void **out)
{
    static void *address[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && address[dev] != nullptr) { *out = address[dev]; return cudaSuccess; }
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    if (dev >= 0 && dev < 64) address[dev] = p;
    *out = p;
    return cudaSuccess;
}

}  // namespace

extern "C" {

const char *cawn_status_string(int status)
{
    switch (status) {
    case CAWN_OK: return "ok";
    case CAWN_ERR_INVALID_ARG: return "invalid argument";
    case CAWN_ERR_NULL_POINTER: return "required pointer is NULL";
    case CAWN_ERR_MISALIGNED: return "pointer is not sufficiently aligned";
    case CAWN_ERR_UNSUPPORTED: return "request not supported by this build";
    case CAWN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CAWN_ERR_CUDA: return "CUDA runtime error";
    case CAWN_ERR_STATIC_TOO_LARGE: return "call needs more scratch than the built-in array holds";
    case CAWN_ERR_CARRY_TIMEOUT: return "device: inter-tile carry wait ran out";
    case CAWN_STATUS_NONFINITE: return "device: non-finite values seen";
    case CAWN_ERR_CARRY_TIMEOUT | CAWN_STATUS_NONFINITE: return "device: inter-tile carry wait ran out; non-finite values seen";
    default: return "unknown status";
    }
}

int cawn_workspace_bytes(const cawn_params *params, int op, size_t *bytes)
{
    int rc = check_params(params);
    if (rc != CAWN_OK) return rc;
    if (bytes == nullptr) return CAWN_ERR_NULL_POINTER;
    const size_t n = (size_t)params->B * (size_t)params->L * (size_t)params->H * params->F;
    switch (op) {
    case CAWN_OP_FWD: {
        const Geometry g = geometry(params, fwd_shape(params->L));
        *bytes = sizeof(WsHeader) + g.rec_bytes;
        return CAWN_OK;
    }
    case CAWN_OP_BWD_SAVED:
    case CAWN_OP_BWD_PUSHES: {
        const Geometry gb = geometry(params, bwd_shape(params->L));
        const Geometry gf = geometry(params, fwd_shape(params->L));
        size_t rec = gb.rec_bytes > gf.rec_bytes ? gb.rec_bytes : gf.rec_bytes;
        size_t total = sizeof(WsHeader) + round_up(rec, 256);
        total += round_up((size_t)params->B * gb.K * gb.C * sizeof(float2), 256);
        total += round_up((size_t)params->B * gb.K * gb.C * sizeof(float), 256);
        if (op == CAWN_OP_BWD_PUSHES) total += round_up(n * sizeof(float2), 256);
        *bytes = total;
        return CAWN_OK;
    }
    case CAWN_OP_MIXING_BWD:
        *bytes = mix_bwd_layout(params).total;
        return CAWN_OK;
    case CAWN_OP_STATE:
        *bytes = state_blob_bytes(params);
        return CAWN_OK;
    case CAWN_OP_FWD_HOST:
        *bytes = host_stage(params).total;
        return CAWN_OK;
    default:
        return CAWN_ERR_INVALID_ARG;
    }
}

int cawn_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (workspace == nullptr) return CAWN_ERR_NULL_POINTER;
    if (!aligned(workspace, 16)) return CAWN_ERR_MISALIGNED;
    if (workspace_bytes < sizeof(WsHeader)) return CAWN_ERR_WORKSPACE_TOO_SMALL;
    if (cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)cuda_stream) != cudaSuccess)
        return CAWN_ERR_CUDA;
    return CAWN_OK;
}

// Forward, with (ear_w != NULL) or without the Ear epilogue.
static int fwd_common(const cawn_params *params, const void *input,
                      const float *gamma, const float *theta,
                      const float *conv_w, const float *conv_bias,
                      const float *gamma_logit, const float *freq_bias,
                      const void *state_in, void *y, void *state_out,
                      uint32_t *gate_mask, void *workspace, size_t workspace_bytes,
                      void *cuda_stream, const float *ear_w, const float *ear_bias, int ear_k,
                      bool validate_only = false)
{
    int rc = check_params(params);
    if (rc != CAWN_OK) return rc;
    const bool dyn = (params->flags & CAWN_FLAG_RETENTION_DYNAMIC) != 0;
    const bool fused = params->conv_k != 0;
    const int io = io_of(params);
    // with time-varying retention or the Ear epilogue, bf16 storage is built for input and output together
    if (io != 0 && io != (IO_IN_BF16 | IO_OUT_BF16) && (dyn || ear_w != nullptr)) return CAWN_ERR_UNSUPPORTED;
    if (ear_w != nullptr) {
        if (ear_k != 1 && ear_k != 3) return CAWN_ERR_UNSUPPORTED;
        // a CTA owns 64 adjacent channels: a head's harmonics must not straddle two of them
        if ((long long)params->H * params->F > 64 && 64 % params->F != 0) return CAWN_ERR_UNSUPPORTED;
        if (!aligned(ear_w, 4) || !aligned(ear_bias, 4)) return CAWN_ERR_MISALIGNED;
    }
    if (dyn) {
        if (gamma_logit == nullptr || freq_bias == nullptr) return CAWN_ERR_NULL_POINTER;
        if (!aligned(gamma_logit, 4) || !aligned(freq_bias, 4)) return CAWN_ERR_MISALIGNED;
    }
    if (fused) {
        if (params->conv_k > 4) return CAWN_ERR_UNSUPPORTED;
        if (conv_w == nullptr) return CAWN_ERR_NULL_POINTER;
        // with clamp + SiLU the magnitude is at least 0.43: thresholds below that leave every gate
        // open, which is what the kernel assumes; higher ones are not provided for
        if ((params->flags & CAWN_FLAG_PRELUDE_CLAMP_SILU) && params->gate_eps > 0.4f) return CAWN_ERR_UNSUPPORTED;
        if (!aligned(conv_w, 4) || !aligned(conv_bias, 4)) return CAWN_ERR_MISALIGNED;
    }
    if ((gamma == nullptr && !dyn) || theta == nullptr || workspace == nullptr) return CAWN_ERR_NULL_POINTER;
    if (params->L > 0 && (input == nullptr || y == nullptr)) return CAWN_ERR_NULL_POINTER;
    if (!aligned(input, 16) || !aligned(y, 16) || !aligned(workspace, 16) ||
        !aligned(gate_mask, 4) || !aligned(state_in, 8) || !aligned(state_out, 8) ||
        !aligned(gamma, 4) || !aligned(theta, 4))
        return CAWN_ERR_MISALIGNED;
    const TileShape ts = fwd_shape(params->L);
    const Geometry g = geometry(params, ts);
    if (!grid_ok(params, g)) return CAWN_ERR_UNSUPPORTED;
    if (workspace_bytes < sizeof(WsHeader) + g.rec_bytes) return CAWN_ERR_WORKSPACE_TOO_SMALL;
    if (validate_only) return CAWN_OK;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    if (params->L == 0) {               // nothing to scan: the state (and conv history) passes through
        if (state_out != nullptr && state_out != state_in) {
            const size_t nb = fused ? state_blob_bytes(params) : (size_t)params->B * g.C * sizeof(float2);
            cudaError_t e = state_in ? cudaMemcpyAsync(state_out, state_in, nb, cudaMemcpyDeviceToDevice, st)
                                     : cudaMemsetAsync(state_out, 0, nb, st);
            if (e != cudaSuccess) return CAWN_ERR_CUDA;
        }
        return CAWN_OK;
    }

    ScanParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.in = input; sp.out = y;
    sp.gamma = gamma; sp.theta = theta;
    sp.state_in = reinterpret_cast<const float2 *>(state_in);
    sp.state_out = reinterpret_cast<float2 *>(state_out);
    sp.mask = gate_mask;
    sp.ws = reinterpret_cast<WsHeader *>(workspace);
    set_records(sp, reinterpret_cast<char *>(workspace) + sizeof(WsHeader), g);
    sp.L = params->L; sp.B = params->B;
    set_gate(sp, params->gate_eps);
    sp.clampv = params->clamp_abs > 0.f ? params->clamp_abs : 0.f;
    sp.poll_limit = kPollLimit;
    sp.ear_w = ear_w; sp.ear_bias = ear_bias; sp.ear_k = ear_k;
    sp.H = params->H; sp.F = params->F;
    if (fused) {
        // state blob: P [B,C] complex64, then (16-byte aligned) the conv history [B,conv_k-1,C]
        const size_t tail_off = round_up((size_t)params->B * g.C * sizeof(float2), 16);
        sp.conv_w = conv_w; sp.conv_bias = conv_bias;
        sp.conv_k = params->conv_k;
        sp.clamp_silu = (params->flags & CAWN_FLAG_PRELUDE_CLAMP_SILU) ? 1 : 0;
        sp.gate_tau = params->gate_tau;
        sp.early_loads = (params->flags & CAWN_FLAG_INPUT_INDEPENDENT) ? 1 : 0;
        if (params->conv_k > 1) {
            sp.tail_in = state_in ? reinterpret_cast<const float *>(reinterpret_cast<const char *>(state_in) + tail_off) : nullptr;
            sp.tail_out = state_out ? reinterpret_cast<float *>(reinterpret_cast<char *>(state_out) + tail_off) : nullptr;
        }
        sp.gamma_logit = gamma_logit; sp.freq_bias = freq_bias;
        if (launch_fused(ts, sp, st, io, dyn) != cudaSuccess) return CAWN_ERR_CUDA;
        return CAWN_OK;
    }
    sp.gamma_logit = gamma_logit; sp.freq_bias = freq_bias; sp.H = params->H; sp.F = params->F;
    sp.early_loads = (params->flags & CAWN_FLAG_INPUT_INDEPENDENT) ? 1 : 0;
    if (!dyn && ts.T == 16) set_stagger(sp, ts, ((io & IO_IN_BF16) ? 4 : 8) + ((io & IO_OUT_BF16) ? 4 : 8));
    if (launch_fwd(ts, sp, st, dyn, io) != cudaSuccess) return CAWN_ERR_CUDA;
    return CAWN_OK;
}

int cawn_phase_accumulate_fwd(const cawn_params *params, const void *input,
                              const float *gamma, const float *theta,
                              const float *conv_w, const float *conv_bias,
                              const float *gamma_logit, const float *freq_bias,
                              const void *state_in, void *y, void *state_out,
                              uint32_t *gate_mask, void *workspace, size_t workspace_bytes,
                              void *cuda_stream)
{
    return fwd_common(params, input, gamma, theta, conv_w, conv_bias, gamma_logit, freq_bias, state_in, y,
                      state_out, gate_mask, workspace, workspace_bytes, cuda_stream, nullptr, nullptr, 0);
}

int cawn_phase_accumulate_fwd_ear(const cawn_params *params, const void *input,
                                  const float *gamma, const float *theta,
                                  const float *conv_w, const float *conv_bias,
                                  const float *gamma_logit, const float *freq_bias,
                                  const void *state_in,
                                  const float *ear_w, const float *ear_bias, int ear_k,
                                  float *z_conv, void *state_out, uint32_t *gate_mask,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (ear_w == nullptr) return CAWN_ERR_NULL_POINTER;
    return fwd_common(params, input, gamma, theta, conv_w, conv_bias, gamma_logit, freq_bias, state_in, z_conv,
                      state_out, gate_mask, workspace, workspace_bytes, cuda_stream, ear_w, ear_bias, ear_k);
}

// Backward of the Cartesian forward, static (gamma) or time-varying (gamma_logit, freq_bias)
// retention.  Static: grad_gamma; time-varying: grad_logit [B,L,H], grad_fbias [F].
static int bwd_common(const cawn_params *params, bool dyn, const void *saved, int saved_kind,
                      const float *gamma, const float *gamma_logit, const float *freq_bias,
                      const float *theta, const void *state_in,
                      const void *grad_y, const void *grad_state_out,
                      void *grad_p, float *grad_gamma, float *grad_logit, float *grad_fbias,
                      float *grad_theta, void *grad_state_in, void *workspace, size_t workspace_bytes,
                      void *cuda_stream)
{
    int rc = check_params(params);
    if (rc != CAWN_OK) return rc;
    if (params->flags & kBf16Flags) return CAWN_ERR_UNSUPPORTED;   // fp32 storage only here
    if (params->conv_k != 0) return CAWN_ERR_UNSUPPORTED;
    if (saved_kind != CAWN_SAVED_STATES && saved_kind != CAWN_SAVED_PUSHES) return CAWN_ERR_INVALID_ARG;
    if (theta == nullptr || workspace == nullptr) return CAWN_ERR_NULL_POINTER;
    if (dyn ? (gamma_logit == nullptr || freq_bias == nullptr) : gamma == nullptr) return CAWN_ERR_NULL_POINTER;
    const bool want_param = (grad_gamma != nullptr || grad_theta != nullptr || grad_logit != nullptr ||
                             grad_fbias != nullptr);
    if (params->L > 0 && (grad_y == nullptr || grad_p == nullptr)) return CAWN_ERR_NULL_POINTER;
    if (params->L > 0 && want_param && saved == nullptr) return CAWN_ERR_NULL_POINTER;
    if (!aligned(saved, 16) || !aligned(grad_y, 16) || !aligned(grad_p, 16) || !aligned(workspace, 16) ||
        !aligned(state_in, 8) || !aligned(grad_state_out, 8) || !aligned(grad_state_in, 8))
        return CAWN_ERR_MISALIGNED;
    size_t need = 0;
    rc = cawn_workspace_bytes(params, saved_kind == CAWN_SAVED_PUSHES ? CAWN_OP_BWD_PUSHES : CAWN_OP_BWD_SAVED, &need);
    if (rc != CAWN_OK) return rc;
    if (workspace_bytes < need) return CAWN_ERR_WORKSPACE_TOO_SMALL;
    const TileShape tb = bwd_shape(params->L), tf = fwd_shape(params->L);
    const Geometry gb = geometry(params, tb), gf = geometry(params, tf);
    if (!grid_ok(params, gb) || !grid_ok(params, gf)) return CAWN_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int C = gb.C;

    if (params->L == 0) {
        const size_t nb = (size_t)params->B * C * sizeof(float2);
        if (grad_state_in != nullptr && grad_state_in != grad_state_out) {
            cudaError_t e = grad_state_out ? cudaMemcpyAsync(grad_state_in, grad_state_out, nb, cudaMemcpyDeviceToDevice, st)
                                           : cudaMemsetAsync(grad_state_in, 0, nb, st);
            if (e != cudaSuccess) return CAWN_ERR_CUDA;
        }
        if (grad_gamma && cudaMemsetAsync(grad_gamma, 0, C * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        if (grad_theta && cudaMemsetAsync(grad_theta, 0, C * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        if (grad_fbias && cudaMemsetAsync(grad_fbias, 0, params->F * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        return CAWN_OK;
    }
    // where the logit gradient is accumulated with atomic adds it starts from zero
    const bool direct = logit_grad_direct(params);
    if (grad_logit != nullptr && !direct &&
        cudaMemsetAsync(grad_logit, 0, (size_t)params->B * (size_t)params->L * params->H * sizeof(float), st) != cudaSuccess)
        return CAWN_ERR_CUDA;

    char *base = reinterpret_cast<char *>(workspace);
    const size_t rec = gb.rec_bytes > gf.rec_bytes ? gb.rec_bytes : gf.rec_bytes;
    size_t off = sizeof(WsHeader);
    char *recs = base + off;                                        off += round_up(rec, 256);
    float2 *qpart = reinterpret_cast<float2 *>(base + off);         off += round_up((size_t)params->B * gb.K * C * sizeof(float2), 256);
    float *spart = reinterpret_cast<float *>(base + off);           off += round_up((size_t)params->B * gb.K * C * sizeof(float), 256);
    float2 *Pbuf = reinterpret_cast<float2 *>(base + off);

    const void *states = saved;
    if (want_param && saved_kind == CAWN_SAVED_PUSHES) {
        // rebuild the unclamped forward states from the pushes (gate, then scan)
        ScanParams fp;
        memset(&fp, 0, sizeof(fp));
        fp.in = saved; fp.out = Pbuf;
        fp.gamma = gamma; fp.theta = theta;
        fp.state_in = reinterpret_cast<const float2 *>(state_in);
        fp.ws = reinterpret_cast<WsHeader *>(workspace);
        set_records(fp, recs, gf);
        fp.L = params->L; fp.B = params->B;
        set_gate(fp, params->gate_eps);
        fp.clampv = 0.f;
        fp.poll_limit = kPollLimit;
        fp.gamma_logit = gamma_logit; fp.freq_bias = freq_bias; fp.H = params->H; fp.F = params->F;
        if (launch_fwd(tf, fp, st, dyn) != cudaSuccess) return CAWN_ERR_CUDA;
        states = Pbuf;
    }

    ScanParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.in = grad_y; sp.out = grad_p;
    sp.aux = want_param ? states : nullptr;
    sp.gamma = gamma; sp.theta = theta;
    sp.state_in = reinterpret_cast<const float2 *>(state_in);
    sp.edge_in = reinterpret_cast<const float2 *>(grad_state_out);
    sp.state_out = reinterpret_cast<float2 *>(grad_state_in);
    sp.ws = reinterpret_cast<WsHeader *>(workspace);
    set_records(sp, recs, gb);
    sp.qpart = want_param ? qpart : nullptr;
    sp.L = params->L; sp.B = params->B;
    sp.clampv = params->grad_clamp_abs > 0.f ? params->grad_clamp_abs : 0.f;
    sp.poll_limit = kPollLimit;
    sp.gamma_logit = gamma_logit; sp.freq_bias = freq_bias; sp.H = params->H; sp.F = params->F;
    sp.grad_logit = (dyn && want_param) ? grad_logit : nullptr;
    sp.logit_direct = direct ? 1 : 0;
    sp.spart = (dyn && want_param && grad_fbias != nullptr) ? spart : nullptr;
    if (launch_bwd(tb, sp, st, dyn) != cudaSuccess) return CAWN_ERR_CUDA;

    if (want_param) {
        EpilogueParams ep;
        memset(&ep, 0, sizeof(ep));
        ep.nparts = params->B * gb.K; ep.C = C; ep.H = params->H; ep.F = params->F;
        ep.qpart = qpart; ep.gamma = dyn ? nullptr : gamma; ep.theta = theta;
        ep.grad_gamma = dyn ? nullptr : grad_gamma; ep.grad_theta = grad_theta; ep.clampv = sp.clampv;
        ep.spart = spart; ep.grad_fbias = grad_fbias;
        if (launch_epilogue(ep, true, dyn && grad_fbias != nullptr, false, false, st) != cudaSuccess) return CAWN_ERR_CUDA;
    }
    return CAWN_OK;
}

int cawn_phase_accumulate_bwd(const cawn_params *params, const void *saved, int saved_kind,
                              const float *gamma, const float *theta, const void *state_in,
                              const void *grad_y, const void *grad_state_out,
                              void *grad_p, float *grad_gamma, float *grad_theta,
                              void *grad_state_in, void *workspace, size_t workspace_bytes,
                              void *cuda_stream)
{
    if (params != nullptr && (params->flags & CAWN_FLAG_RETENTION_DYNAMIC)) return CAWN_ERR_UNSUPPORTED;
    return bwd_common(params, false, saved, saved_kind, gamma, nullptr, nullptr, theta, state_in, grad_y,
                      grad_state_out, grad_p, grad_gamma, nullptr, nullptr, grad_theta, grad_state_in,
                      workspace, workspace_bytes, cuda_stream);
}

int cawn_phase_accumulate_bwd_dynamic(const cawn_params *params, const void *saved, int saved_kind,
                                      const float *gamma_logit, const float *freq_bias,
                                      const float *theta, const void *state_in,
                                      const void *grad_y, const void *grad_state_out,
                                      void *grad_p, float *grad_gamma_logit, float *grad_freq_bias,
                                      float *grad_theta, void *grad_state_in,
                                      void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (params != nullptr && !(params->flags & CAWN_FLAG_RETENTION_DYNAMIC)) return CAWN_ERR_INVALID_ARG;
    return bwd_common(params, true, saved, saved_kind, nullptr, gamma_logit, freq_bias, theta, state_in, grad_y,
                      grad_state_out, grad_p, nullptr, grad_gamma_logit, grad_freq_bias, grad_theta,
                      grad_state_in, workspace, workspace_bytes, cuda_stream);
}

// Backward of the fused path, static (gamma) or time-varying (gamma_logit, freq_bias) retention.
static int mix_bwd_common(const cawn_params *params, bool dyn, const float *h, const float *conv_w, const float *conv_bias,
                          const float *gamma, const float *gamma_logit, const float *freq_bias,
                          const float *theta, const void *saved_states, const void *state_in,
                          const void *grad_y, const void *grad_state_out, float *grad_h, float *grad_conv_w,
                          float *grad_conv_bias, float *grad_gamma, float *grad_logit, float *grad_fbias,
                          float *grad_theta, void *grad_state_in,
                          void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    int rc = check_params(params);
    if (rc != CAWN_OK) return rc;
    if (params->flags & kBf16Flags) return CAWN_ERR_UNSUPPORTED;   // fp32 storage only here
    if (params->conv_k < 1 || params->conv_k > 4) return CAWN_ERR_UNSUPPORTED;
    if ((params->flags & CAWN_FLAG_PRELUDE_CLAMP_SILU) && params->gate_eps > 0.4f) return CAWN_ERR_UNSUPPORTED;
    if (conv_w == nullptr || theta == nullptr || workspace == nullptr) return CAWN_ERR_NULL_POINTER;
    if (dyn ? (gamma_logit == nullptr || freq_bias == nullptr) : gamma == nullptr) return CAWN_ERR_NULL_POINTER;
    if (params->L > 0 && (h == nullptr || grad_y == nullptr || grad_h == nullptr)) return CAWN_ERR_NULL_POINTER;
    if (!aligned(h, 16) || !aligned(grad_h, 16) || !aligned(workspace, 16) || !aligned(state_in, 16) ||
        !aligned(grad_state_out, 16) || !aligned(grad_state_in, 16))
        return CAWN_ERR_MISALIGNED;
    const MixBwdLayout lay = mix_bwd_layout(params);
    if (workspace_bytes < lay.total) return CAWN_ERR_WORKSPACE_TOO_SMALL;
    const TileShape ts = bwd_shape(params->L);
    const Geometry g = geometry(params, ts);
    if (!grid_ok(params, g) || g.K + 1 > 65535) return CAWN_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int C = g.C, Kc = params->conv_k, Kh = Kc - 1;
    const size_t tail_off = round_up((size_t)params->B * C * sizeof(float2), 16);
    const bool want_scan_param = grad_gamma != nullptr || grad_theta != nullptr || grad_logit != nullptr || grad_fbias != nullptr;
    const bool want_conv_param = grad_conv_w != nullptr || grad_conv_bias != nullptr;
    if (params->L > 0 && want_scan_param && saved_states == nullptr) return CAWN_ERR_NULL_POINTER;
    if (!aligned(saved_states, 16) || !aligned(grad_y, 16)) return CAWN_ERR_MISALIGNED;

    if (params->L == 0) {
        // nothing ran: the incoming state gradient passes through, the parameter gradients are zero
        if (grad_state_in != nullptr && grad_state_in != grad_state_out) {
            const size_t nb = state_blob_bytes(params);
            cudaError_t e = grad_state_out ? cudaMemcpyAsync(grad_state_in, grad_state_out, nb, cudaMemcpyDeviceToDevice, st)
                                           : cudaMemsetAsync(grad_state_in, 0, nb, st);
            if (e != cudaSuccess) return CAWN_ERR_CUDA;
        }
        if (grad_conv_w && cudaMemsetAsync(grad_conv_w, 0, (size_t)C * Kc * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        if (grad_conv_bias && cudaMemsetAsync(grad_conv_bias, 0, (size_t)C * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        if (grad_gamma && cudaMemsetAsync(grad_gamma, 0, (size_t)C * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        if (grad_theta && cudaMemsetAsync(grad_theta, 0, (size_t)C * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        if (grad_fbias && cudaMemsetAsync(grad_fbias, 0, (size_t)params->F * sizeof(float), st) != cudaSuccess) return CAWN_ERR_CUDA;
        return CAWN_OK;
    }
    // where the logit gradient is accumulated with atomic adds it starts from zero
    const bool direct = logit_grad_direct(params);
    if (grad_logit != nullptr && !direct &&
        cudaMemsetAsync(grad_logit, 0, (size_t)params->B * (size_t)params->L * params->H * sizeof(float), st) != cudaSuccess)
        return CAWN_ERR_CUDA;

    char *base = reinterpret_cast<char *>(workspace);
    float2 *qpart = reinterpret_cast<float2 *>(base + lay.off_qpart);
    float *spart = reinterpret_cast<float *>(base + lay.off_spart);
    float *edge = reinterpret_cast<float *>(base + lay.off_edge);
    float *cpart = reinterpret_cast<float *>(base + lay.off_cpart);
    const float *tail_in = nullptr, *dtail_out = nullptr;
    float *dtail_in = nullptr;
    if (Kh > 0) {
        if (state_in) tail_in = reinterpret_cast<const float *>(reinterpret_cast<const char *>(state_in) + tail_off);
        if (grad_state_out) dtail_out = reinterpret_cast<const float *>(reinterpret_cast<const char *>(grad_state_out) + tail_off);
        if (grad_state_in) dtail_in = reinterpret_cast<float *>(reinterpret_cast<char *>(grad_state_in) + tail_off);
    }

    // 1. reverse scan with the prelude's chain rule and the conv transpose as its epilogue
    ScanParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.in = grad_y; sp.out = grad_h;
    sp.aux = want_scan_param ? saved_states : nullptr;
    sp.gamma = gamma; sp.theta = theta;
    sp.state_in = reinterpret_cast<const float2 *>(state_in);
    sp.edge_in = reinterpret_cast<const float2 *>(grad_state_out);
    sp.state_out = reinterpret_cast<float2 *>(grad_state_in);
    sp.ws = reinterpret_cast<WsHeader *>(workspace);
    set_records(sp, base + lay.off_rec, g);
    sp.qpart = want_scan_param ? qpart : nullptr;
    sp.L = params->L; sp.B = params->B;
    sp.clampv = params->grad_clamp_abs > 0.f ? params->grad_clamp_abs : 0.f;
    sp.poll_limit = kPollLimit;
    sp.H = params->H; sp.F = params->F;
    sp.gamma_logit = gamma_logit; sp.freq_bias = freq_bias;
    sp.grad_logit = (dyn && want_scan_param) ? grad_logit : nullptr;
    sp.logit_direct = direct ? 1 : 0;
    sp.spart = (dyn && want_scan_param && grad_fbias != nullptr) ? spart : nullptr;
    sp.hid = h; sp.conv_w = conv_w; sp.conv_bias = conv_bias; sp.tail_in = tail_in;
    sp.conv_k = Kc;
    sp.clamp_silu = (params->flags & CAWN_FLAG_PRELUDE_CLAMP_SILU) ? 1 : 0;
    sp.gate_tau = params->gate_tau;
    sp.edge_du = edge;
    sp.cpart = want_conv_param ? cpart : nullptr;
    if ((dyn ? launch_mix_bwd_dynamic(ts, sp, st) : launch_mix_bwd(ts, sp, st)) != cudaSuccess) return CAWN_ERR_CUDA;

    // 2. one more launch: the rows at the tile seams, the gradient of the carried conv history, and
    //    the parameter gradients from the per-tile partial sums
    EpilogueParams ep;
    memset(&ep, 0, sizeof(ep));
    ep.nparts = params->B * g.K; ep.C = C; ep.H = params->H; ep.F = params->F; ep.Kc = Kc;
    ep.qpart = qpart; ep.gamma = dyn ? nullptr : gamma; ep.theta = theta;
    ep.grad_gamma = dyn ? nullptr : grad_gamma; ep.grad_theta = grad_theta; ep.clampv = sp.clampv;
    ep.spart = spart; ep.grad_fbias = grad_fbias;
    ep.cpart = cpart; ep.grad_w = grad_conv_w; ep.grad_bias = grad_conv_bias;
    ep.edge_du = edge; ep.conv_w = conv_w; ep.dtail_out = dtail_out; ep.grad_h = grad_h; ep.dtail_in = dtail_in;
    ep.L = params->L; ep.B = params->B; ep.K = g.K; ep.tile = ts.T * ts.W;
    if (launch_epilogue(ep, want_scan_param, dyn && want_scan_param && grad_fbias != nullptr, want_conv_param, true, st) != cudaSuccess)
        return CAWN_ERR_CUDA;
    return CAWN_OK;
}

int cawn_mixing_bwd(const cawn_params *params, const float *h, const float *conv_w, const float *conv_bias,
                    const float *gamma, const float *theta, const void *saved_states, const void *state_in,
                    const void *grad_y, const void *grad_state_out, float *grad_h, float *grad_conv_w,
                    float *grad_conv_bias, float *grad_gamma, float *grad_theta, void *grad_state_in,
                    void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (params != nullptr && (params->flags & CAWN_FLAG_RETENTION_DYNAMIC)) return CAWN_ERR_UNSUPPORTED;
    return mix_bwd_common(params, false, h, conv_w, conv_bias, gamma, nullptr, nullptr, theta, saved_states, state_in,
                          grad_y, grad_state_out, grad_h, grad_conv_w, grad_conv_bias, grad_gamma, nullptr, nullptr,
                          grad_theta, grad_state_in, workspace, workspace_bytes, cuda_stream);
}

int cawn_mixing_bwd_dynamic(const cawn_params *params, const float *h, const float *conv_w, const float *conv_bias,
                            const float *gamma_logit, const float *freq_bias, const float *theta,
                            const void *saved_states, const void *state_in,
                            const void *grad_y, const void *grad_state_out, float *grad_h, float *grad_conv_w,
                            float *grad_conv_bias, float *grad_gamma_logit, float *grad_freq_bias, float *grad_theta,
                            void *grad_state_in, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (params != nullptr && !(params->flags & CAWN_FLAG_RETENTION_DYNAMIC)) return CAWN_ERR_INVALID_ARG;
    return mix_bwd_common(params, true, h, conv_w, conv_bias, nullptr, gamma_logit, freq_bias, theta, saved_states, state_in,
                          grad_y, grad_state_out, grad_h, grad_conv_w, grad_conv_bias, nullptr, grad_gamma_logit,
                          grad_freq_bias, grad_theta, grad_state_in, workspace, workspace_bytes, cuda_stream);
}

int cawn_state_carry(const cawn_params *params, const void *state_prev, const void *state_local,
                     int64_t n_steps, const float *gamma, const float *theta,
                     void *state_out, void *cuda_stream)
{
    int rc = check_params(params);
    if (rc != CAWN_OK) return rc;
    if (n_steps < 0) return CAWN_ERR_INVALID_ARG;
    if (params->flags & CAWN_FLAG_RETENTION_DYNAMIC) return CAWN_ERR_UNSUPPORTED;
    if (!state_prev || !state_local || !gamma || !theta || !state_out) return CAWN_ERR_NULL_POINTER;
    if (!aligned(state_prev, 8) || !aligned(state_local, 8) || !aligned(state_out, 8))
        return CAWN_ERR_MISALIGNED;
    const int C = params->H * params->F;
    const long long n = (long long)params->B * C;
    cawn_state_carry_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)cuda_stream>>>(
        reinterpret_cast<const float2 *>(state_prev), reinterpret_cast<const float2 *>(state_local),
        reinterpret_cast<float2 *>(state_out), gamma, theta, n_steps, params->B, C);
    return cudaGetLastError() == cudaSuccess ? CAWN_OK : CAWN_ERR_CUDA;
}

int cawn_poll_status(void *workspace, void *cuda_stream)
{
    if (workspace == nullptr) return CAWN_ERR_NULL_POINTER;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    WsHeader *ws = reinterpret_cast<WsHeader *>(workspace);
    unsigned status = 0;
    if (cudaMemcpyAsync(&status, &ws->status, sizeof(status), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return CAWN_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CAWN_ERR_CUDA;
    if (status != 0) {
        if (cudaMemsetAsync(&ws->status, 0, sizeof(status), st) != cudaSuccess) return CAWN_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return CAWN_ERR_CUDA;
    }
    return (int)status;
}

int cawn_workspace_set_wait_hook(void *workspace, int withhold_tile, unsigned poll_bound, void *cuda_stream)
{
    if (workspace == nullptr) return CAWN_ERR_NULL_POINTER;
    if (withhold_tile >= 65535 || poll_bound > 65535u) return CAWN_ERR_INVALID_ARG;
    const unsigned word = (poll_bound << 16) | (withhold_tile < 0 ? 0u : (unsigned)withhold_tile + 1u);
    WsHeader *ws = reinterpret_cast<WsHeader *>(workspace);
    cawn_set_word_kernel<<<1, 1, 0, (cudaStream_t)cuda_stream>>>(&ws->hook, word);
    return cudaGetLastError() == cudaSuccess ? CAWN_OK : CAWN_ERR_CUDA;
}

// Copy pipes of the host-staged forward: one stream for host-to-device copies and kernels, one
// for device-to-host copies, so that the two directions of the bus work at the same time.  One
// set per device, created on first use and kept; calls that use them are serialised.
constexpr int kHostSlices = 8;
struct CopyPipes {
    cudaStream_t in, out;
    cudaEvent_t fork, in_done, out_done, slice[kHostSlices];
    bool ready;
};
static std::mutex g_pipes_mutex;
static CopyPipes g_pipes[64];

static cudaError_t get_pipes(CopyPipes **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    CopyPipes &p = g_pipes[dev];
    if (!p.ready) {
        if ((e = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking)) != cudaSuccess) return e;
        if ((e = cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking)) != cudaSuccess) return e;
        cudaEvent_t *ev[3] = {&p.fork, &p.in_done, &p.out_done};
        for (int i = 0; i < 3; ++i)
            if ((e = cudaEventCreateWithFlags(ev[i], cudaEventDisableTiming)) != cudaSuccess) return e;
        for (int i = 0; i < kHostSlices; ++i)
            if ((e = cudaEventCreateWithFlags(&p.slice[i], cudaEventDisableTiming)) != cudaSuccess) return e;
        p.ready = true;
    }
    *out = &p;
    return cudaSuccess;
}

int cawn_phase_accumulate_fwd_host(const cawn_params *params, const void *p_host,
                                   const float *gamma_host, const float *theta_host,
                                   const void *state_in_host, void *y_host, void *state_out_host,
                                   uint32_t *gate_mask_host, void *device_scratch,
                                   size_t device_scratch_bytes, void *cuda_stream)
{
    int rc = check_params(params);
    if (rc != CAWN_OK) return rc;
    if (params->flags & kBf16Flags) return CAWN_ERR_UNSUPPORTED;   // fp32 storage only here
    if (params->conv_k != 0 || (params->flags & CAWN_FLAG_RETENTION_DYNAMIC))
        return CAWN_ERR_UNSUPPORTED;
    if (!gamma_host || !theta_host || !device_scratch) return CAWN_ERR_NULL_POINTER;
    if (params->L > 0 && (!p_host || !y_host)) return CAWN_ERR_NULL_POINTER;
    if (!aligned(device_scratch, 256)) return CAWN_ERR_MISALIGNED;
    const HostStage h = host_stage(params);
    if (device_scratch_bytes < h.total) return CAWN_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *d = reinterpret_cast<char *>(device_scratch);
    const size_t C = (size_t)params->H * params->F, MW = (C + 31) / 32;
    const size_t n = (size_t)params->B * (size_t)params->L * C;
    const size_t state_bytes = (size_t)params->B * C * sizeof(float2);

    // Slices that can be copied in, scanned and copied out one after another: batch rows when
    // there are several (independent), else stretches of time with the state carried from one
    // to the next (chunked prefill inside the call).  Small calls are one slice.
    const bool by_batch = params->B >= 2;
    int S = 1;
    if (by_batch) {
        S = params->B < kHostSlices ? params->B : kHostSlices;
    } else {
        const size_t want = n * sizeof(float2) / ((size_t)4 << 20);
        S = want < 1 ? 1 : (want > (size_t)kHostSlices ? kHostSlices : (int)want);
    }
    if (n * sizeof(float2) < ((size_t)8 << 20)) S = 1;

    CopyPipes *pp = nullptr;
    std::unique_lock<std::mutex> lock(g_pipes_mutex, std::defer_lock);
    cudaStream_t s_in = st, s_out = st;
    bool ok = true;
    if (S > 1) {
        lock.lock();
        if (get_pipes(&pp) != cudaSuccess) return CAWN_ERR_CUDA;
        s_in = pp->in; s_out = pp->out;
        ok &= cudaEventRecord(pp->fork, st) == cudaSuccess;
        ok &= cudaStreamWaitEvent(s_in, pp->fork, 0) == cudaSuccess;
        ok &= cudaStreamWaitEvent(s_out, pp->fork, 0) == cudaSuccess;
    }
    ok &= cudaMemcpyAsync(d + h.off_gamma, gamma_host, C * sizeof(float), cudaMemcpyHostToDevice, s_in) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + h.off_theta, theta_host, C * sizeof(float), cudaMemcpyHostToDevice, s_in) == cudaSuccess;
    if (state_in_host)
        ok &= cudaMemcpyAsync(d + h.off_state, state_in_host, state_bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
    if (!ok) return CAWN_ERR_CUDA;

    const int64_t rows_total = by_batch ? params->B : params->L;       // what the slices divide
    int64_t per = (rows_total + S - 1) / S;
    if (!by_batch && S > 1) per = (per + 127) / 128 * 128;              // whole tiles per stretch of time
    int64_t r0 = 0;
    for (int i = 0; i < S && (r0 < rows_total || i == 0); ++i) {
        const int64_t r1 = (r0 + per < rows_total) ? r0 + per : rows_total;
        cawn_params q = *params;
        size_t x_off, m_off, s_off = 0;
        bool have_state = state_in_host != nullptr;
        if (by_batch) {
            q.B = (int32_t)(r1 - r0);
            x_off = (size_t)r0 * (size_t)params->L * C;
            m_off = (size_t)r0 * (size_t)params->L * MW;
            s_off = (size_t)r0 * C;
        } else {
            q.L = r1 - r0;
            x_off = (size_t)r0 * C;
            m_off = (size_t)r0 * MW;
            have_state = have_state || i > 0;                           // later stretches continue the first
        }
        const size_t nx = (size_t)q.B * (size_t)q.L * C;
        char *x_dev = d + h.off_x + x_off * sizeof(float2);
        char *state_dev = d + h.off_state + s_off * sizeof(float2);
        uint32_t *mask_dev = reinterpret_cast<uint32_t *>(d + h.off_mask) + m_off;
        const bool need_state_out = state_out_host != nullptr || (!by_batch && S > 1);
        if (nx)
            ok &= cudaMemcpyAsync(x_dev, reinterpret_cast<const char *>(p_host) + x_off * sizeof(float2), nx * sizeof(float2),
                                  cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        if (!ok) return CAWN_ERR_CUDA;
        rc = cawn_phase_accumulate_fwd(&q, x_dev,
                                       reinterpret_cast<const float *>(d + h.off_gamma),
                                       reinterpret_cast<const float *>(d + h.off_theta),
                                       nullptr, nullptr, nullptr, nullptr,
                                       have_state ? state_dev : nullptr,
                                       x_dev,                                  /* in place */
                                       need_state_out ? state_dev : nullptr,
                                       gate_mask_host ? mask_dev : nullptr,
                                       d + h.off_ws, h.total - h.off_ws, s_in);
        if (rc != CAWN_OK) return rc;
        if (S > 1) {
            ok &= cudaEventRecord(pp->slice[i], s_in) == cudaSuccess;
            ok &= cudaStreamWaitEvent(s_out, pp->slice[i], 0) == cudaSuccess;
        }
        if (nx)
            ok &= cudaMemcpyAsync(reinterpret_cast<char *>(y_host) + x_off * sizeof(float2), x_dev, nx * sizeof(float2),
                                  cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
        if (gate_mask_host && nx)
            ok &= cudaMemcpyAsync(gate_mask_host + m_off, mask_dev, (size_t)q.B * (size_t)q.L * MW * sizeof(uint32_t),
                                  cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
        if (!ok) return CAWN_ERR_CUDA;
        r0 = r1;
    }
    // the state leaves after the last slice (s_out has waited for it)
    if (state_out_host)
        ok &= cudaMemcpyAsync(state_out_host, d + h.off_state, state_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
    if (S > 1) {                                     // join both pipes back into the caller's stream
        ok &= cudaEventRecord(pp->in_done, s_in) == cudaSuccess;
        ok &= cudaEventRecord(pp->out_done, s_out) == cudaSuccess;
        ok &= cudaStreamWaitEvent(st, pp->in_done, 0) == cudaSuccess;
        ok &= cudaStreamWaitEvent(st, pp->out_done, 0) == cudaSuccess;
    }
    return ok ? CAWN_OK : CAWN_ERR_CUDA;
}

int cawn_phase_accumulate_fwd_static(const cawn_params *params, const void *input,
                                     const float *gamma, const float *theta, const void *state_in,
                                     void *y, void *state_out, uint32_t *gate_mask,
                                     uint32_t *device_status, void *cuda_stream)
{
    size_t need = 0;
    int rc = cawn_workspace_bytes(params, CAWN_OP_FWD, &need);
    if (rc != CAWN_OK) return rc;
    if (params->conv_k != 0 || (params->flags & CAWN_FLAG_RETENTION_DYNAMIC)) return CAWN_ERR_UNSUPPORTED;
    if (need > (size_t)CAWN_STATIC_SCRATCH_BYTES) return CAWN_ERR_STATIC_TOO_LARGE;
    if (!aligned(device_status, 4)) return CAWN_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // every argument is checked before anything is put on the stream (the workspace pointer of this
    // dry run only has to be non-NULL and aligned: nothing dereferences it)
    rc = fwd_common(params, input, gamma, theta, nullptr, nullptr, nullptr, nullptr, state_in, y, state_out, gate_mask,
                    reinterpret_cast<void *>((uintptr_t)256), (size_t)CAWN_STATIC_SCRATCH_BYTES, st, nullptr, nullptr, 0,
                    /*validate_only=*/true);
    if (rc != CAWN_OK) return rc;
    void *scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess) return CAWN_ERR_CUDA;
    WsHeader *ws = reinterpret_cast<WsHeader *>(scratch);
    // the array keeps the previous call's contents: only the sticky status has to start at zero
    if (cudaMemsetAsync(&ws->status, 0, sizeof(unsigned), st) != cudaSuccess) return CAWN_ERR_CUDA;
    rc = cawn_phase_accumulate_fwd(params, input, gamma, theta, nullptr, nullptr, nullptr, nullptr,
                                   state_in, y, state_out, gate_mask, scratch,
                                   (size_t)CAWN_STATIC_SCRATCH_BYTES, st);
    if (rc != CAWN_OK) return rc;
    if (device_status != nullptr &&
        cudaMemcpyAsync(device_status, &ws->status, sizeof(unsigned), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return CAWN_ERR_CUDA;
    return CAWN_OK;
}

}  // extern "C"
