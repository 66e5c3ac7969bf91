// The chunk-parallel phase-accumulation kernel.
//
// One CTA owns a tile of TILE = W*T consecutive time steps of one (batch, 64-channel group).
// Warp w owns T consecutive steps; lane l owns the adjacent channels 64g + 2l and 64g + 2l + 1,
// so a warp-wide access is one 512-byte row segment read or written as 32 float4.
// The tile is staged in shared memory between its single read from and its single write to
// global memory: the asynchronous copies hold no registers while they are in flight, which
// is what lets three 64 KB tiles per SM stay in flight next to the arithmetic.
//
//   0. every thread issues the asynchronous copies of its own T row pieces, in groups of a few
//      rows; meanwhile 64 threads prepare the per-channel coefficients a, a^T, a^TILE in
//      double                                                                    [barrier 1]
//   1. as its row groups land: gate (Cartesian forward; the gated value goes back to shared
//      memory), and each thread reduces its T steps from a zero start, leaving the end state
//      in shared memory                                                          [barrier 2]
//   2. warp 0 folds the W ends into the tile aggregate and publishes it; every warp fetches
//      its records of the carry window (below) into shared memory                [barrier 3]
//   3. every warp folds the window into the tile's carry-in, folds the earlier warps' ends on
//      top, re-runs its T steps as the plain recurrence from that state and stores them
//
// A warp only ever touches the tile rows it copied itself, so the tile needs no block barrier:
// complex64 rows are copied and used by the same thread; hidden rows and bf16 rows are copied a
// half-warp (or eight lanes) per row in 16-byte pieces, and the warp synchronises between waiting
// for a copy group and using it.  (Copies of 4 or 8 bytes per lane issue far more slowly.)
//
// Carry window.  With M = kWindow, the tiles k = M, 2M, ... of a chain are checkpoints: they also
// publish their carry-in X_k (the state before the tile).  Tile k reads the carry-in of the
// last checkpoint c < k (c = 0: the call's initial state) and the aggregates E_c .. E_{k-1},
// and evaluates X_k = A^(k-c) X_c + sum A^(k-1-i) E_i by Horner's rule, oldest first, A = a^TILE.
// What is read and the order it is combined in depend on k alone, never on timing, so results
// are bit-for-bit repeatable; aggregates are published before anything is waited for, so the
// only serial dependency runs from checkpoint to checkpoint.  A tile only ever waits for tiles
// with a smaller linear block index, which the hardware has dispatched before it.
//
// Each run of the fp32 recurrence is at most T steps long and everything that crosses a thread
// boundary is multiplied by a power of a_j rounded once from double: the rounding error of
// a_j does not build up with sequence length.
//
// The backward is the same operator run right-to-left with conj(a_j); it additionally
// accumulates sum conj(lam_t) P_{t-1} per channel for the retention and rotation gradients.
#pragma once
#include "cawn_device.cuh"
#include <cuda_bf16.h>
#include <type_traits>

namespace cawn {

// KIND_MIXBWD: the reverse scan of KIND_BWD whose push gradient is not stored but taken straight
// through the fused path's prelude (phasor map, straight-through gate, conv) to grad_h.
enum : int { KIND_FWD = 0, KIND_FUSED = 1, KIND_BWD = 2, KIND_MIXBWD = 3 };
__host__ __device__ constexpr bool kind_is_bwd(int kind) { return kind == KIND_BWD || kind == KIND_MIXBWD; }

// Storage type of the forward's input (pushes or hidden rows) and output; the arithmetic and the
// carried state are fp32 either way.
enum : int { IO_F32 = 0, IO_IN_BF16 = 1, IO_OUT_BF16 = 2 };

// A bf16 is the upper half of a float: widening is exact.
__device__ __forceinline__ float2 bf16x2_to_float2(unsigned u)
{
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}
__device__ __forceinline__ unsigned float2_to_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);       // round to nearest even
    return *reinterpret_cast<const unsigned *>(&v);
}

// Rows of hidden-state history in front of a tile that the fused conv prelude may read.
constexpr int kHalo = 3;

// Carry window: every kWindow-th tile of a chain is a checkpoint.
constexpr int kWindow = 7;

struct ScanParams {
    const void *in;              // FWD: pushes p;  BWD: grad_y              [B,L,C] complex64
                                 // FUSED: hidden states h                   [B,L,C] float
                                 // (IO_IN_BF16: pairs of bf16 / bf16; IO_OUT_BF16: y as pairs of bf16)
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
    float gate_mid, gate_hw;     // fp32 screen of the gate: fl(eps^2) and the half-width of the
                                 // band around it inside which only the double comparison decides
    float gate_keep;             // first pass keeps s - gate_mid >= gate_keep (normally -gate_hw)
    float clampv;                // output (FWD) or gradient (BWD) clamp; <= 0 off
    unsigned poll_limit;
    // fused conv prelude (KIND_FUSED)
    const float *conv_w;         // [C][conv_k]
    const float *conv_bias;      // [C] or NULL
    const float *tail_in;        // [B][conv_k-1][C] carried hidden rows or NULL (zeros)
    float *tail_out;             // [B][conv_k-1][C] or NULL
    int conv_k;                  // 1..4
    int clamp_silu;              // clamp the conv output to +-50, then SiLU
    float gate_tau;              // gate: conv output >= gate_tau (fp32 fmaf chain, tap order)
    // backward through the fused prelude (KIND_MIXBWD): out = grad_h [B,L,C] float
    const float *hid;            // hidden states h [B,L,C] float
    float *edge_du;              // [B*K][6][C]: du of a tile's three last rows in time (latest first), then of
                                 // its three first rows (earliest first); rows a tile does not have: 0
    float *cpart;                // [B*K][C][5] per-tile sums of du*h (four right-aligned taps) and du, or NULL
    // time-varying retention (DYN): gamma_t = sigmoid(gamma_logit[b,t,h] + freq_bias[k])
    const float *gamma_logit;    // [B][L][H]
    const float *freq_bias;      // [F]
    int H, F;
    float *grad_logit;           // BWD: [B][L][H]
    int first_wave;              // fused forward: CTAs the device holds at once (0: unknown), set at launch
    int logit_direct;            // every 64-channel group holds whole heads: the logit gradient of a (row, head)
                                 // is complete in one warp and is stored; otherwise it is added atomically
                                 // into an array zeroed before the launch
    float *spart;                // BWD: per-tile partial sums of the logit gradient [B*K][C]
    // First-wave stagger: the CTAs that land in the 2nd, 3rd, ... resident slot of an SM (linear
    // block index / stagger_group) start their copies stagger_cycles, 2 stagger_cycles, ... late,
    // so that the CTAs sharing an SM run out of phase and their load, arithmetic and store
    // phases overlap instead of alternating.  0 = off.
    int stagger_cycles, stagger_group, stagger_slots;
    // Ear epilogue (EAR): instead of interleaved complex y, the kernel writes the planar row
    // Z = (all real parts, all imaginary parts) [B,L,2,H,F] after a depthwise convolution along
    // the F harmonics of each head (ear_k taps, zero padding, one tap set per (part, head)).
    const float *ear_w;          // [2H][ear_k]
    const float *ear_bias;       // [2H] or NULL
    int ear_k;                   // 1 or 3
    int early_loads;             // the input rows may be fetched before the preceding launch on the
                                 // stream has finished (the caller vouches they are not its output)
};

// Shared memory of one CTA: the tile (two tiles in the backward: grad_y and P_{t-1}), then the
// small exchange areas.
template <int T, int W, int KIND, bool DYN = false>
struct ScanSmem {
    static constexpr int TILE = T * W;
    static constexpr int NT = kind_is_bwd(KIND) ? 2 : 1;
    float4 tile[NT][TILE][32];
    // MIXBWD: hidden rows in processing order (row R = physical row t_hi - R), then kHalo rows of history
    float hrev[KIND == KIND_MIXBWD ? TILE + kHalo : 1][KIND == KIND_MIXBWD ? 64 : 1];
    float4 sE[W][32];
    float4 sR[kWindow + 1][32];
    float sCoef[64][6];
    float2 sD[DYN ? W : 1][DYN ? 32 : 1];             // DYN: factor products of the warps' steps
    float2 sRD[DYN ? kWindow + 1 : 1][DYN ? 32 : 1];  // DYN: factor products of the window's tiles
    float2 sG[DYN ? TILE : 1][DYN ? 32 : 1];          // DYN: each row's own factor pair, kept from phase 1 for phase 3
    unsigned long long epoch;
    unsigned arrived;                                  // thread 0: this CTA's arrival count
    int err;
    unsigned hook;                                     // copy of the workspace's wait hook
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// Asynchronous global -> shared copies; the destination is a shared-space address plus a
// compile-time byte offset, so that an unrolled loop needs no address arithmetic for it.
template <int OFF>
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0+%2], [%1], 16;" :: "r"(dst), "l"(src), "n"(OFF) : "memory");
}
template <int OFF>
__device__ __forceinline__ void cp_async8(uint32_t dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0+%2], [%1], 8;" :: "r"(dst), "l"(src), "n"(OFF) : "memory");
}
template <int OFF>
__device__ __forceinline__ void cp_async4o(uint32_t dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0+%2], [%1], 4;" :: "r"(dst), "l"(src), "n"(OFF) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" :: "r"(dst), "l"(src) : "memory");
}
// Programmatic dependent launch: let the next launch on the stream start filling SMs as soon as
// every CTA of this one is running, and wait for the previous launch (and its memory) to be
// complete.  Both are no-ops for a launch made without the programmatic attribute.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_wait_previous() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// Wait until at most n of this thread's most recent copy groups are still in flight (n <= 4).
__device__ __forceinline__ void cp_async_wait_pending(int n)
{
    switch (n) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
    }
}

// base + i * step in one instruction (step fits 32 bits: a row is at most 2^27 bytes)
__device__ __forceinline__ const char *row_ptr(const char *base, int step, int i)
{
    long long r;
    asm("mad.wide.s32 %0, %1, %2, %3;" : "=l"(r) : "r"(step), "r"(i), "l"((long long)base));
    return reinterpret_cast<const char *>(r);
}

// Copy (asynchronously) or zero one row piece of this lane: two adjacent complex64 at byte
// offset OFF from the thread's first piece (`dst` generic, `dst_s` the same in shared space).
// HALF: the source holds two complex bf16 (8 bytes); they land in the first half of the piece and
// are widened in place by the thread that owns it.
template <bool VEC, int OFF, bool HALF = false>
__device__ __forceinline__ void fetch_piece(float4 *dst, uint32_t dst_s, const char *src, bool vA, bool vB)
{
    float4 *d4 = reinterpret_cast<float4 *>(reinterpret_cast<char *>(dst) + OFF);
    if constexpr (HALF) {
        unsigned *d = reinterpret_cast<unsigned *>(d4);
        if (VEC) {
            if (vA) cp_async8<OFF>(dst_s, src); else { d[0] = 0u; d[1] = 0u; }
        } else {
            if (vA) cp_async4o<OFF>(dst_s, src); else d[0] = 0u;
            if (vB) cp_async4o<OFF + 4>(dst_s, src + 4); else d[1] = 0u;
        }
    } else if (VEC) {
        if (vA) cp_async16<OFF>(dst_s, src); else *d4 = zero4();
    } else {
        float2 *d = reinterpret_cast<float2 *>(d4);
        if (vA) cp_async8<OFF>(dst_s, src); else d[0] = make_float2(0.f, 0.f);
        if (vB) cp_async8<OFF + 8>(dst_s, src + 8); else d[1] = make_float2(0.f, 0.f);
    }
}

// Unrolled helper: issue the T copies of one thread (rows i = 0..T-1, `step` bytes apart in
// global memory, 512 bytes apart in shared memory), committing one copy group per GR rows
// (GR = 0: the caller commits).  valid(i) says whether row i exists.
template <bool VEC, int T, int GR, int I = 0, bool HALF = false, typename F>
__device__ __forceinline__ void fetch_rows(float4 *dst, uint32_t dst_s, const char *src, int step,
                                           bool vA, bool vB, F valid)
{
    if constexpr (I < T) {
        const bool row = valid(I);
        fetch_piece<VEC, I * 512, HALF>(dst, dst_s, row_ptr(src, step, I), row && vA, row && vB);
        if constexpr (GR > 0) {
            if constexpr ((I + 1) % GR == 0) cp_async_commit();
        }
        fetch_rows<VEC, T, GR, I + 1, HALF>(dst, dst_s, src, step, vA, vB, valid);
    }
}

// Chain rule of the fused prelude for one channel at one step: from the push gradient
// (lr, li) = dLoss/d(Re z, Im z) and the conv output u to dLoss/du.  z = m_used (cos ph, sin ph)
// with m = sigmoid(x), ph = pi tanh(x), x = u (or SiLU(clamp(u)) with `act`), m_used = m where the
// gate is open, else 0.  Straight-through gate: the magnitude path ignores the gate
// (dm = lr cos ph + li sin ph), the phase path is scaled by the gated magnitude.
// As in the forward: q = e^-x, m = 1/(1+q), r = 1/(1+q^2), tanh x = 2r - 1, and
// (cos, sin)(ph) = -(cos, sin)(2 pi r); 1 - tanh^2 = 4 r (1 - r).  Where (1+q)(1+q^2) overflows
// m = r = 0, where q underflows m = r = 1, and every term stays finite.
template <bool PLAIN>
__device__ __forceinline__ float prelude_du(float u, float lr, float li, bool act, float tau)
{
    float x = u, dxdu = 1.f;
    if (!PLAIN && act) {
        const float v = fminf(fmaxf(u, -50.f), 50.f);
        const float sg = __fdividef(1.f, 1.f + __expf(-v));
        x = v * sg;
        dxdu = (u >= -50.f && u <= 50.f) ? sg * fmaf(v, 1.f - sg, 1.f) : 0.f;
    }
    const float q = ex2_ftz(fminf(x * -1.44269504088896f, 60.f));
    const float p1 = 1.f + q, p2 = fmaf(q, q, 1.f);
    const float rr = rcp_ftz(p1 * p2);
    const float m = p2 * rr, r = p1 * rr;
    float sn, cs;                                    // of 2 pi r: the negated sine and cosine of the phase
    sincos_ftz(r * 6.28318530717959f, sn, cs);
    const bool open = (!PLAIN && act) || u >= tau;           // with clamp + SiLU every gate is open (see the forward)
    const float dm = -fmaf(lr, cs, li * sn);
    const float dph = (open ? m : 0.f) * fmaf(lr, sn, -li * cs);
    // d ph / dx = pi (1 - tanh^2) = 4 pi r (1 - r);  d m / dx = m (1 - m)
    const float dx = fmaf(dm * m, 1.f - m, dph * (12.5663706143592f * r) * (1.f - r));
    return PLAIN ? dx : dx * dxdu;
}

// MASKED = false compiles the gate-mask output out (the caller then never passes a mask), which
// keeps its registers out of the plain forward.
template <int T, int W, int KIND, bool VEC, bool DYN, bool FULL, bool EAR = false, int IO = IO_F32, bool MASKED = true, bool LATE = false>
__device__ __forceinline__ void scan_tile(const ScanParams &prm, ScanSmem<T, W, KIND, DYN> &sm,
                                          const int g, const int b, const int k)
{
    static_assert(!(EAR && kind_is_bwd(KIND)), "the Ear epilogue belongs to the forward");
    static_assert(IO == IO_F32 || !kind_is_bwd(KIND), "bf16 storage is built for the forward");
    constexpr bool IN16 = (IO & IO_IN_BF16) != 0, OUT16 = (IO & IO_OUT_BF16) != 0;
    constexpr bool REV = kind_is_bwd(KIND);
    constexpr bool MIX = (KIND == KIND_MIXBWD);
    constexpr int TILE = T * W;
    constexpr int M = kWindow;
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
    const int rowbytes = (REV ? -C : C) * 8;
    const long long e0 = ((long long)b * L + t_first) * C + c0;    // only used when nvalid > 0
    float4 *const xs = &sm.tile[0][w * T][lane];                   // this thread's pieces, 32 float4 apart

    // ---- 0. asynchronous copies into shared memory -----------------------------------------
    // The rows go out as NG copy groups of GR rows each, so that phase 1 can start on the first
    // rows while the later ones are still in flight.  The backward's second tile (needed in
    // phase 3 only) is one more group behind them.
    constexpr int GR = T < 4 ? T : (T > 16 ? T / 4 : 4), NG = T / GR;
    static_assert(T % GR == 0 && NG <= 4, "copy groups");
    // Unless the caller vouched for the input rows, nothing is read before the previous launch
    // on the stream is complete.
    if (prm.stagger_cycles > 0) {
        const unsigned lin = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
        const unsigned slot = lin / (unsigned)prm.stagger_group;
        if (slot >= 1u && slot < (unsigned)prm.stagger_slots) {
            if (tid == 0) {
                const long long t0 = clock64(), target = (long long)slot * prm.stagger_cycles;
                for (int it = 0; it < 4096 && clock64() - t0 < target; ++it) __nanosleep(64);
            }
            __syncthreads();
        }
    }
    const bool early = !REV && prm.early_loads != 0;
    // LATE (static Cartesian forward without a mask, a call whose CTAs are all resident at once, the
    // input vouched for): the gate pass, which reads the input rows and writes shared memory only,
    // runs before the wait for the previous launch.
    static_assert(!LATE || (KIND == KIND_FWD && !DYN && !MASKED), "the late wait is built for the plain forward");
    const bool late_wait = LATE && early;
    // Fused forward: a CTA beyond the first wave starts in a slot that a CTA of this launch has
    // left, and that one had waited for the previous launch: its own wait returns at once, so it
    // waits (and asks for the epoch) before its copies instead of after them.
    const bool wait_first = KIND == KIND_FUSED && early && prm.first_wave > 0 &&
        (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x >= (unsigned)prm.first_wave;
    if (!early || wait_first) grid_wait_previous();
    // Reverse kinds (they have waited already) and the fused forward: the thread that later builds
    // channel tid's coefficients asks for its gamma and theta now, and thread 0 for the epoch (the
    // fused forward: once it has waited, below), so that the answers travel while the tile's
    // copies are issued and land.  (The plain forward is bound by memory, not by this chain.)
    constexpr bool PRE = REV || KIND == KIND_FUSED;
    float pre_gamma = 1.f, pre_theta = 0.f;
    if (PRE && tid < 64 && g * 64 + tid < C) {
        if (!DYN) pre_gamma = prm.gamma[g * 64 + tid];
        pre_theta = prm.theta[g * 64 + tid];
    }
    unsigned long long epoch0 = 0;
    unsigned hook0 = 0;
    if ((REV || wait_first) && tid == 0) ld_epoch_hook(prm.ws, epoch0, hook0);
    // Fused path: every warp stages its own T hidden rows (floats) behind kHalo rows of history in
    // the upper part of its own T x 512-byte slice of the tile, row r at byte 256 (T - 3) + 256 r
    // (r < kHalo: history).  The pushes the warp later writes into the same slice (row i at byte
    // 512 i) reach hidden row r only at step i >= (r + 12) / 2: the rows are read a copy group (GR)
    // at a time, rows i+3 .. i+GR+2 at step i = 0, GR, ..., and (r + 12) / 2 >= the step whose group
    // holds r; the warp synchronises between reading a group and writing its pushes.
    // No other warp touches the slice, so a warp starts as soon as its own first rows have landed.
    static_assert(KIND != KIND_FUSED || T == 16 || T == 4, "slice layout of the fused path is checked for 16 and 4 rows");
    float *const hstage = reinterpret_cast<float *>(&sm.tile[0][w * T][0]) + (T * 128 - (T + kHalo) * 64) + 2 * lane;
    bool in_packed = false;                             // bf16 pushes of this warp sit packed in the upper half of its slice
    bool packed16 = false;                              // bf16 hidden rows of this warp sit packed, history included
    bool fused_tail_group = false;                      // this thread committed one more group (carried history)
    if constexpr (KIND == KIND_FUSED) {
        const float *hin = reinterpret_cast<const float *>(prm.in);
        const unsigned short *hin16 = reinterpret_cast<const unsigned short *>(prm.in);
        const int Kh = prm.conv_k - 1;
        // a bf16 hidden value of a history row is kept as the float it widens to
        auto widen = [](unsigned short v) -> float { return __uint_as_float((unsigned)v << 16); };
        // float rows of whole 16-byte pieces: a half-warp copies one row's 256 bytes, a warp two
        // rows per instruction (copies of 4 and 8 bytes take the slower path through L1); the lanes
        // that read a row are then not the ones that brought it, so the warp synchronises after
        // each wait
        const bool wide = !IN16 && (C & 3) == 0 && (reinterpret_cast<uintptr_t>(prm.in) & 15) == 0;
        // bf16 rows of a whole tile with all four taps behind kHalo earlier rows of the call: a row is
        // 128 bytes, eight lanes copy it in 16-byte pieces, a warp four rows per instruction; every
        // row, history included, then sits packed in the first half of its 256-byte slot.  Copy group
        // gi ends with the instruction that holds the last row its steps read (row GR gi + GR + 2).
        packed16 = IN16 && FULL && Kh == kHalo && s0 >= kHalo && (C & 7) == 0 && (reinterpret_cast<uintptr_t>(prm.in) & 15) == 0;
        if (packed16) {
            static_assert(GR == 4 && kHalo == 3, "four rows to an instruction, one instruction to a copy group");
            const int p8 = (lane & 7) * 8, rr = lane >> 3;
            const unsigned short *src = hin16 + ((long long)b * L + s0 - kHalo + rr) * C + g * 64 + p8;
            const uint32_t d = smem_addr(hstage - 2 * lane + rr * 64 + (lane & 7) * 4);
#pragma unroll
            for (int m = 0; m < (T + kHalo + 3) / 4; ++m) {
                if (4 * m + rr < T + kHalo) cp_async16<0>(d + m * 1024, src);
                src += 4 * (long long)C;
                if (m >= 1) cp_async_commit();
            }
        } else if (wide) {
            const int q4 = (lane & 15) * 4, hh = lane >> 4;
            const bool cols = g * 64 + q4 < C;
            float *const hbase = hstage - 2 * lane + q4;
            auto history16 = [&](int j, bool on) {
                const long long t = s0 - kHalo + j;
                float *d = hbase + j * 64;
                if (!on) return;
                if (j >= kHalo - Kh && t >= 0 && t < L) {
                    if (cols) cp_async16<0>(smem_addr(d), hin + ((long long)b * L + t) * C + g * 64 + q4);
                    else *reinterpret_cast<float4 *>(d) = zero4();
                } else if (t >= 0 || prm.tail_in == nullptr || j < kHalo - Kh) {
                    *reinterpret_cast<float4 *>(d) = zero4();
                }
            };
            static_assert(kHalo == 3 && T % 2 == 0 && GR % 2 == 0, "rows go two to an instruction");
            if (FULL && Kh == kHalo && s0 >= kHalo) {
                // a whole tile with all four taps behind kHalo earlier rows of the call: all T + kHalo
                // rows exist and are whole, one pointer steps through them two rows at a time.  Copy
                // group gi ends with the pair that holds the last row its steps read (row GR gi + GR + 2).
                const float *src = hin + ((long long)b * L + s0 - kHalo + hh) * C + g * 64 + q4;
                const uint32_t d = smem_addr(hbase + hh * 64);
#pragma unroll
                for (int m = 0; m < (T + kHalo + 1) / 2; ++m) {
                    if (2 * m + 1 < T + kHalo || hh == 0) cp_async16<0>(d + m * 512, src);
                    src += 2 * (long long)C;
                    if (m >= GR / 2 + 1 && (m - (GR / 2 + 1)) % (GR / 2) == 0) cp_async_commit();
                }
            } else {
                history16(hh, true);
                history16(2, hh == 0);
                const float *r = hin + ((long long)b * L + s0 + hh) * C + g * 64 + q4;
#pragma unroll
                for (int i = 0; i < T; i += 2) {
                    const bool row = FULL || i + hh < nvalid;
                    float *d = hbase + (kHalo + i + hh) * 64;
                    if (row && cols) cp_async16<0>(smem_addr(d), r); else *reinterpret_cast<float4 *>(d) = zero4();
                    r += 2 * (long long)C;
                    if ((i + 2) % GR == 0) cp_async_commit();
                }
            }
        }
        if (!wide && !packed16) {
            // history rows that are earlier rows of h (they travel with the first group of own rows)
#pragma unroll
            for (int j = 0; j < kHalo; ++j) {
                const long long t = s0 - kHalo + j;
                float *d = hstage + j * 64;
                if (j >= kHalo - Kh && t >= 0 && t < L) {
                    if constexpr (IN16) {
                        const unsigned short *s16 = hin16 + ((long long)b * L + t) * C + c0;
                        d[0] = vA ? widen(s16[0]) : 0.f;
                        d[1] = vB ? widen(s16[1]) : 0.f;
                    } else {
                        const float *src = hin + ((long long)b * L + t) * C + c0;
                        if (vA) cp_async4(smem_addr(d), src); else d[0] = 0.f;
                        if (vB) cp_async4(smem_addr(d + 1), src + 1); else d[1] = 0.f;
                    }
                } else if (t >= 0 || prm.tail_in == nullptr || j < kHalo - Kh) {
                    d[0] = 0.f; d[1] = 0.f;                 // no such tap, or no carried history
                }
            }
            const float *r = hin + e0;
            const unsigned short *r16 = hin16 + e0;
#pragma unroll
            for (int i = 0; i < T; ++i) {
                const bool row = FULL || i < nvalid;
                float *d = hstage + (kHalo + i) * 64;
                if constexpr (IN16) {
                    // the pair of bf16 goes into the first word of the slot; phase 1 widens it
                    if (VEC) {
                        if (row && vA) cp_async4(smem_addr(d), r16); else d[0] = 0.f;
                    } else {
                        unsigned lo = 0u, hi = 0u;
                        if (row && vA) lo = r16[0];
                        if (row && vB) hi = r16[1];
                        reinterpret_cast<unsigned *>(d)[0] = lo | (hi << 16);
                    }
                    r16 += C;
                } else if (VEC) {
                    if (row && vA) cp_async8<0>(smem_addr(d), r); else *reinterpret_cast<float2 *>(d) = make_float2(0.f, 0.f);
                } else {
                    if (row && vA) cp_async4(smem_addr(d), r); else d[0] = 0.f;
                    if (row && vB) cp_async4(smem_addr(d + 1), r + 1); else d[1] = 0.f;
                }
                r += C;
                if ((i + 1) % GR == 0) cp_async_commit();
            }
        }
        // history rows before t = 0 come from the carried tail: the previous call's output, never
        // read before that call is complete
        if (early && !wait_first) grid_wait_previous();
        if (!wait_first && tid == 0) ld_epoch_hook(prm.ws, epoch0, hook0);
        if (s0 < kHalo && prm.tail_in != nullptr) {
#pragma unroll
            for (int j = 0; j < kHalo; ++j) {
                const long long t = s0 - kHalo + j;
                if (j >= kHalo - Kh && t < 0) {
                    float *d = hstage + j * 64;
                    const float *src = prm.tail_in + ((long long)b * Kh + (Kh + t)) * C + c0;
                    if (vA) cp_async4(smem_addr(d), src); else d[0] = 0.f;
                    if (vB) cp_async4(smem_addr(d + 1), src + 1); else d[1] = 0.f;
                }
            }
            cp_async_commit();
            fused_tail_group = true;
        }
    } else {
        if constexpr (IN16) {
            // Whole tiles of bf16 pushes whose rows are whole 16-byte pieces: a row is 256 bytes, a
            // half-warp copies it, a warp two rows per instruction.  The T packed rows fill the upper
            // half of the warp's T x 512-byte slice (row i at byte 256 T + 256 i); the gate pass widens
            // row i into its 512-byte slot at byte 512 i, which only reaches packed rows 2i - T and
            // 2i - T + 1 <= i: rows every lane has read by then (the warp synchronises after each read).
            in_packed = FULL && (C & 3) == 0 && (reinterpret_cast<uintptr_t>(prm.in) & 15) == 0;
            if (in_packed) {
                static_assert(T % 2 == 0 && GR % 2 == 0, "rows go two to an instruction");
                const int hh = lane >> 4;
                const char *src = reinterpret_cast<const char *>(prm.in) + (((long long)b * L + s0 + hh) * C + g * 64) * 4 + (lane & 15) * 16;
                const uint32_t d = smem_addr(&sm.tile[0][w * T][0]) + T * 256 + hh * 256 + (lane & 15) * 16;
#pragma unroll
                for (int m = 0; m < T / 2; ++m) {
                    cp_async16<0>(d + m * 512, src);
                    src += 8 * (long long)C;
                    if ((2 * m + 2) % GR == 0) cp_async_commit();
                }
            } else {
                fetch_rows<VEC, T, GR, 0, true>(xs, smem_addr(xs), reinterpret_cast<const char *>(prm.in) + e0 * 4, rowbytes / 2,
                                                vA, vB, [&](int i) { return FULL || i < nvalid; });
            }
        } else
            fetch_rows<VEC, T, GR>(xs, smem_addr(xs), reinterpret_cast<const char *>(prm.in) + e0 * 8, rowbytes, vA, vB,
                                   [&](int i) { return FULL || i < nvalid; });
    }
    if constexpr (MIX) {
        // hidden rows this tile's conv windows reach, in processing order: row R holds physical
        // row t_hi - R (t_hi = the tile's last row in time); before t = 0 comes the carried
        // history, before that zeros.  Each warp brings its own T rows, one warp the kHalo more.
        const int Kh = prm.conv_k - 1;
        const long long t_hi = L - 1 - (long long)k * TILE;
        auto stage_h = [&](int R) {
            const long long t = t_hi - R;
            float *d = &sm.hrev[R][2 * lane];
            const float *src = nullptr;
            if (t >= 0) src = prm.hid + ((long long)b * L + t) * C + c0;
            else if (t >= -Kh && prm.tail_in != nullptr) src = prm.tail_in + ((long long)b * Kh + (Kh + t)) * C + c0;
            if (VEC) {
                if (src != nullptr && vA) cp_async8<0>(smem_addr(d), src); else *reinterpret_cast<float2 *>(d) = make_float2(0.f, 0.f);
            } else {
                if (src != nullptr && vA) cp_async4(smem_addr(d), src); else d[0] = 0.f;
                if (src != nullptr && vB) cp_async4(smem_addr(d + 1), src + 1); else d[1] = 0.f;
            }
        };
        if ((C & 3) == 0 && ((reinterpret_cast<uintptr_t>(prm.hid) | reinterpret_cast<uintptr_t>(prm.tail_in)) & 15) == 0) {
            // rows of whole 16-byte pieces: a half-warp copies one row's 256 bytes, a warp two rows
            // per instruction (8-byte copies take the slower path through L1)
            const int q4 = (lane & 15) * 4, hh = lane >> 4;
            auto stage_h16 = [&](int R, bool on) {
                const long long t = t_hi - R;
                float *d = &sm.hrev[R][q4];
                const float *src = nullptr;
                if (t >= 0) src = prm.hid + ((long long)b * L + t) * C + g * 64 + q4;
                else if (t >= -Kh && prm.tail_in != nullptr) src = prm.tail_in + ((long long)b * Kh + (Kh + t)) * C + g * 64 + q4;
                if (on) {
                    if (src != nullptr && g * 64 + q4 < C) cp_async16<0>(smem_addr(d), src);
                    else *reinterpret_cast<float4 *>(d) = zero4();
                }
            };
            static_assert(T % 2 == 0 && kHalo == 3, "rows go two to an instruction");
            if (FULL) {
                // every own row exists and is whole: one pointer, stepped two rows at a time
                const float *src = prm.hid + ((long long)b * L + t_hi - (w * T + hh)) * C + g * 64 + q4;
                const uint32_t d = smem_addr(&sm.hrev[w * T + hh][q4]);
#pragma unroll
                for (int i = 0; i < T; i += 2) {
                    cp_async16<0>(d + i * 256, src);
                    src -= 2 * (long long)C;
                }
            } else {
#pragma unroll
                for (int i = 0; i < T; i += 2) stage_h16(w * T + i + hh, true);
            }
            if (w == W - 1) {
                stage_h16(TILE + hh, true);
                stage_h16(TILE + 2, hh == 0);
            }
        } else {
#pragma unroll
            for (int i = 0; i < T; ++i) stage_h(w * T + i);
            if (w == 0) {
#pragma unroll
                for (int j = 0; j < kHalo; ++j) stage_h(TILE + j);
            }
        }
    }
    if constexpr (REV) {
        float4 *const qs = &sm.tile[1][w * T][lane];
        const bool have = prm.aux != nullptr;
        if (FULL && have && t_first - (T - 1) >= 1)         // the common case: every row has a predecessor in the call
            fetch_rows<VEC, T, 0>(qs, smem_addr(qs), reinterpret_cast<const char *>(prm.aux) + (e0 - C) * 8, rowbytes,
                                  vA, vB, [](int) { return true; });
        else
            fetch_rows<VEC, T, 0>(qs, smem_addr(qs), reinterpret_cast<const char *>(prm.aux) + (e0 - C) * 8, rowbytes,
                                  vA, vB, [&](int i) { return have && (FULL || i < nvalid) && (t_first - i >= 1); });
        cp_async_commit();
    }

    // Fused path: this lane's conv taps (right-aligned: taps the conv does not have are zero) and
    // bias, requested here so that they arrive while the tile is still in flight.
    float wA[4] = {}, wB[4] = {}, bA = 0.f, bB = 0.f;
    if constexpr (KIND == KIND_FUSED) {
        const int Kc = prm.conv_k;
        if (FULL && Kc == 4 && (reinterpret_cast<uintptr_t>(prm.conv_w) & 15) == 0) {
            // four taps: the two channels' taps are two aligned 16-byte words
            const float4 *w4 = reinterpret_cast<const float4 *>(prm.conv_w) + c0;
            const float4 a4 = w4[0], b4 = w4[1];
            wA[0] = a4.x; wA[1] = a4.y; wA[2] = a4.z; wA[3] = a4.w;
            wB[0] = b4.x; wB[1] = b4.y; wB[2] = b4.z; wB[3] = b4.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int kk = j - (4 - Kc);
                if (kk >= 0 && vA) wA[j] = prm.conv_w[(long long)c0 * Kc + kk];
                if (kk >= 0 && vB) wB[j] = prm.conv_w[(long long)(c0 + 1) * Kc + kk];
            }
        }
        if (prm.conv_bias != nullptr) { if (vA) bA = prm.conv_bias[c0]; if (vB) bB = prm.conv_bias[c0 + 1]; }
    }

    // ---- per-channel coefficients, in double, rounded once --------------------------------
    // One thread per channel: a = gamma (cos theta, sin theta) from one sincos, then a^T and
    // a^TILE = (a^T)^W by square-and-multiply, all in double (a dozen complex products, each good to
    // 2^-52), each rounded to fp32 once.
    for (int cl = tid; cl < 64; cl += W * 32) {
        const int ch = g * 64 + cl;
        double c1r = 0.0, c1i = 0.0, cTr = 0.0, cTi = 0.0, cAr = 0.0, cAi = 0.0;
        if (ch < C) {
            const double gm = PRE ? (double)pre_gamma : DYN ? 1.0 : (double)prm.gamma[ch];
            double sn, cs;
            sincos(PRE ? (double)pre_theta : (double)prm.theta[ch], &sn, &cs);
            c1r = gm * cs;
            c1i = REV ? -(gm * sn) : gm * sn;
            auto cpow = [](double br, double bi, int n, double &rr, double &ri) {
                rr = 1.0; ri = 0.0;
                for (int m = n; m > 0; m >>= 1) {
                    if (m & 1) { const double t = rr * br - ri * bi; ri = rr * bi + ri * br; rr = t; }
                    const double t = br * br - bi * bi; bi = 2.0 * br * bi; br = t;
                }
            };
            cpow(c1r, c1i, T, cTr, cTi);
            cpow(cTr, cTi, W, cAr, cAi);
        }
        float *o = sm.sCoef[cl];
        o[0] = (float)c1r; o[1] = (float)c1i; o[2] = (float)cTr; o[3] = (float)cTi; o[4] = (float)cAr; o[5] = (float)cAi;
    }
    // everything below touches what the previous launch may have written (workspace, states)
    if (early && KIND != KIND_FUSED && !late_wait) grid_wait_previous();
    unsigned arrived = 0;
    auto read_epoch = [&]() {                            // thread 0 only
        if (!PRE) ld_epoch_hook(prm.ws, epoch0, hook0);
        sm.epoch = epoch0;
        sm.hook = hook0;
        // counted only once the epoch has been read (the increment depends on its value)
        arrived = atomicAdd(&prm.ws->done, 1u + (unsigned)(epoch0 >> 63));
    };
    if (tid == 0) {
        sm.err = 0;
        if (!late_wait) read_epoch();
    }
    __syncthreads();                                                           // barrier 1
    float4 a, aT;
    {
        // channel 2l: a, a^T, A at sCoef[2l][0..5]; channel 2l+1 follows: 12 contiguous floats
        const float4 *cp = reinterpret_cast<const float4 *>(&sm.sCoef[2 * lane][0]);
        const float4 u0 = cp[0], u1 = cp[1], u2 = cp[2];
        a = make_float4(u0.x, u0.y, u1.z, u1.w);
        aT = make_float4(u0.z, u0.w, u2.x, u2.y);
    }

    // Time-varying retention: this lane's heads and per-harmonic biases, and the factor pair of
    // one physical row t (0 outside the call, which only ever multiplies a zero carry).
    int hA = 0, hB = 0;
    float fbA = 0.f, fbB = 0.f;
    if constexpr (DYN) {
        hA = c0 / prm.F; hB = (c0 + 1) / prm.F;
        if (vA) fbA = prm.freq_bias[c0 % prm.F];
        if (vB) fbB = prm.freq_bias[(c0 + 1) % prm.F];
    }
    auto row_gamma = [&](long long t) -> float2 {
        float2 gm = make_float2(0.f, 0.f);
        if (t >= 0 && t < L) {
            const float *gl = prm.gamma_logit + ((long long)b * L + t) * prm.H;
            if (vA) gm.x = sigmoidf_fast(gl[hA] + fbA);
            if (vB) gm.y = sigmoidf_fast(gl[hB] + fbB);
        }
        return gm;
    };
    // Where every 64-channel group lies inside one head (F a multiple of 64) the T logits a warp
    // needs are one load: lane j fetches the logit of the warp's row j (lane T, for the reverse
    // kinds, that of the row processed just before the first), and shuffles hand them round.
    // (measured: a gain in the fused forward and the plain backward, a loss in the other two kinds)
    const bool onehead = DYN && (KIND == KIND_FUSED || KIND == KIND_BWD) && (prm.F & 63) == 0;
    float mylogit = 0.f;
    if constexpr (DYN) {
        if (onehead) {
            long long t = REV ? t_first - lane : s0 + lane;
            bool have = lane < T && (FULL || lane < nvalid);
            if (REV && lane == T) { t = t_first + 1; have = t < L; }
            if (have) mylogit = prm.gamma_logit[((long long)b * L + t) * prm.H + hA];
        }
    }
    // the logits of this lane's two channels at the warp's row i (physical row t); 0 where there is no such row
    auto row_logits = [&](int i, long long t) -> float2 {
        float2 lg = make_float2(0.f, 0.f);
        if (onehead) {
            lg.x = lg.y = __shfl_sync(0xffffffffu, mylogit, i);
        } else if (FULL || i < nvalid) {
            const float *gl = prm.gamma_logit + ((long long)b * L + t) * prm.H;
            if (vA) lg.x = gl[hA];
            if (vB) lg.y = gl[hB];
        }
        return lg;
    };
    float2 dprod = make_float2(1.f, 1.f);                // product of this thread's step factors
    float2 gfirst = make_float2(0.f, 0.f);               // DYN backward: factor of the row before this thread's first

    // Window of carry records this tile needs (see the header comment), and a first,
    // non-blocking reading of the record this warp is responsible for: it is usually there
    // already, and its latency then hides behind phase 1.
    const long long chain = (long long)b * G + g;
    const int cpt = k > 0 ? M * ((k - 1) / M) : 0;       // last checkpoint before this tile
    const int nrec = k - cpt;                            // aggregates in the window, 0..M
    const uint4 *early_ptr = nullptr;
    if (w < nrec) early_ptr = prm.agg + (chain * K + (k - 1 - w)) * 64;
    else if (w == M && cpt > 0) early_ptr = prm.pre + (chain * prm.KP + cpt / M) * 64;
    uint4 er0 = make_uint4(0u, 0u, 0u, 0u), er1 = er0;
    // The call's initial state is read before this tile publishes anything, so that state_out
    // may alias state_in: whoever writes state_out has waited for every tile's aggregate.
    float4 sinit = zero4();
    auto read_state_in = [&]() {
        if (!REV && cpt == 0 && w == M % W && prm.state_in != nullptr) {
            const float2 *sp = prm.state_in + (long long)b * C + c0;
            if (vA) { const float2 v = sp[0]; sinit.x = v.x; sinit.y = v.y; }
            if (vB) { const float2 v = sp[1]; sinit.z = v.x; sinit.w = v.y; }
        }
    };
    if (!late_wait) read_state_in();

    if constexpr (REV) {
        cp_async_wait_all();
        // the step at t = 0 multiplies the call's initial state; lam_{L-1} = G_{L-1} + grad_state_out
        if (nvalid > 0 && t_first - (nvalid - 1) == 0 && prm.aux != nullptr && prm.state_in != nullptr) {
            const float2 *r = prm.state_in + (long long)b * C + c0;
            float4 v = zero4();
            if (vA) { const float2 u = r[0]; v.x = u.x; v.y = u.y; }
            if (vB) { const float2 u = r[1]; v.z = u.x; v.w = u.y; }
            sm.tile[1][w * T + (nvalid - 1)][lane] = v;
        }
        if (prm.edge_in != nullptr && s0 == 0 && nvalid > 0) {
            const float2 *r = prm.edge_in + (long long)b * C + c0;
            float4 v = xs[0];
            if (vA) { const float2 u = r[0]; v.x += u.x; v.y += u.y; }
            if (vB) { const float2 u = r[1]; v.z += u.x; v.w += u.y; }
            xs[0] = v;
        }
    }

    // ---- 1. gate + local reduction from a zero start ---------------------------------------
    float4 e = zero4();
    if constexpr (KIND == KIND_FUSED) {
        // Temporal Syntax Cache prelude: causal depthwise conv over time (taps right-aligned on
        // the current token, fmaf chain in tap order from the bias), optional clamp + SiLU,
        // magnitude sigmoid(x), phase pi*tanh(x), gate on the conv output, push m (cos, sin).
        // hidden row r of this lane's channel pair (history rows are floats; own rows of a bf16
        // input are still packed pairs)
        auto hidden_row = [&](int r) -> float2 {
            const float *slot = hstage + r * 64;
            if (IN16 && packed16) return bf16x2_to_float2(reinterpret_cast<const unsigned *>(slot - 2 * lane)[lane]);
            if (IN16 && r >= kHalo) return bf16x2_to_float2(*reinterpret_cast<const unsigned *>(slot));
            return *reinterpret_cast<const float2 *>(slot);
        };
        if (early_ptr != nullptr) {
            er0 = ld_record(early_ptr + 2 * lane);
            er1 = ld_record(early_ptr + 2 * lane + 1);
        }
        const int Kc = prm.conv_k;
        // the first group of rows (and the history) has landed: the rolling window of the conv
        if (fused_tail_group) cp_async_wait_all(); else cp_async_wait_pending(NG - 1);
        __syncwarp();                                     // rows may have been brought by other lanes
        float2 hv0 = hidden_row(0), hv1 = hidden_row(1), hv2 = hidden_row(2), hq[GR];
        const bool act = prm.clamp_silu != 0;
        const float tau = prm.gate_tau;
        const bool want_mask = MASKED && prm.mask != nullptr;
        uint32_t *const mrow0 = prm.mask + ((long long)b * L + s0) * prm.MW + g * 2;
        static_assert(T <= 16, "one 32-bit word per lane holds the gate bits of its rows");
        unsigned mkeep = 0u;                              // bit pair i: this lane's gate bits of row i
        const bool second_word = g * 2 + 1 < prm.MW;
        const bool tap0 = Kc >= 4, tap1 = Kc >= 3, tap2 = Kc >= 2;
        // DYN: the rows' retention logits, all requested up front so that their latencies overlap
        float2 lgf[DYN ? T : 1];
        if constexpr (DYN) {
#pragma unroll
            for (int i = 0; i < T; ++i) lgf[i] = row_logits(i, s0 + i);
        }
        // One channel's push from its conv output u.  With q = e^-x: m = 1/(1+q) and
        // tanh x = 2/(1+q^2) - 1, so the phase is 2 pi r - pi with r = 1/(1+q^2), and
        // (cos, sin)(2 pi r - pi) = -(cos, sin)(2 pi r): z = -m (cos, sin)(2 pi r).  Both quotients
        // come from one reciprocal of (1+q)(1+q^2).  q is capped at 2^60 so that 1+q^2 stays finite;
        // where the product overflows its reciprocal is +0 and m = r = 0, a q that underflows gives
        // m = r = 1: the right limits.
        // `plain`: every tap present and no clamp + SiLU, the common case, compiled without the tests
        auto push = [&](auto plain, float u, bool valid, float &zr, float &zi) -> bool {
            constexpr bool PLAIN = decltype(plain)::value;
            float x = u;
            if (!PLAIN && act) {
                x = fminf(fmaxf(x, -50.f), 50.f);
                x = __fdividef(x, 1.f + __expf(-x));
            }
            const float q = ex2_ftz(fminf(x * -1.44269504088896f, 60.f));
            const float p1 = 1.f + q, p2 = fmaf(q, q, 1.f);
            const float rr = rcp_ftz(p1 * p2);               // one reciprocal serves both
            const float m = p2 * rr, r = p1 * rr;
            float sn, cs;
            sincos_ftz(r * 6.28318530717959f, sn, cs);
            // with clamp + SiLU the magnitude never falls below 0.43, and the host only admits
            // thresholds under that: every gate is open
            const bool open = valid && ((!PLAIN && act) || u >= tau);
            const float mn = open ? -m : 0.f;
            zr = mn * cs; zi = mn * sn;
            return open;
        };
        auto groups = [&](auto plain) {
            constexpr bool PLAIN = decltype(plain)::value;
#pragma unroll
            for (int gi = 0; gi < NG; ++gi) {
                // the group's GR new hidden rows come out of the slice together, then the warp
                // synchronises once: the pushes of these GR steps only reach rows read by now
                if (gi > 0 && !fused_tail_group) { cp_async_wait_pending(NG - 1 - gi); __syncwarp(); }
#pragma unroll
                for (int q = 0; q < GR; ++q) hq[q] = hidden_row(gi * GR + kHalo + q);
                __syncwarp();
#pragma unroll
                for (int q = 0; q < GR; ++q) {
                    const int i = gi * GR + q;
                    const float2 hv3 = hq[q];
                    float uA = bA, uB = bB;
                    if (PLAIN || tap0) { uA = fmaf(wA[0], hv0.x, uA); uB = fmaf(wB[0], hv0.y, uB); }     // fmaf per channel, tap order
                    if (PLAIN || tap1) { uA = fmaf(wA[1], hv1.x, uA); uB = fmaf(wB[1], hv1.y, uB); }
                    if (PLAIN || tap2) { uA = fmaf(wA[2], hv2.x, uA); uB = fmaf(wB[2], hv2.y, uB); }
                    uA = fmaf(wA[3], hv3.x, uA); uB = fmaf(wB[3], hv3.y, uB);
                    hv0 = hv1; hv1 = hv2; hv2 = hv3;
                    float4 z;
                    const bool oA = push(plain, uA, vA, z.x, z.y), oB = push(plain, uB, vB, z.z, z.w);
                    xs[i * 32] = z;
                    mkeep |= ((oA ? 1u : 0u) | (oB ? 2u : 0u)) << (2 * i);     // this lane's gate bits of row i
                    if (FULL || i < nvalid) {
                        if constexpr (DYN) {
                            // e <- gamma_t (a e) + z, the factor pair kept for phase 3
                            const float2 gm = make_float2(vA ? sigmoidf_fast(lgf[i].x + fbA) : 0.f,
                                                          vB ? sigmoidf_fast(lgf[i].y + fbB) : 0.f);
                            sm.sG[w * T + i][lane] = gm;
                            dprod.x *= gm.x; dprod.y *= gm.y;
                            e = scale_step2(a, e, gm, z);
                        } else {
                            e = cfma2(a, e, z);
                        }
                    }
                }
            }
        };
        if (Kc == 4 && !act) groups(std::true_type{}); else groups(std::false_type{});
        if (want_mask) {
            // the rows' mask words: lane r gets word 0 of row r, lane 16 + r word 1
            const unsigned word = transpose_pairs16(mkeep, lane);
            const int r = lane & 15;
            if (r < T && (FULL || r < nvalid) && (lane < 16 || second_word)) mrow0[(long long)r * prm.MW + (lane >> 4)] = word;
        }
    } else if constexpr (KIND == KIND_FWD) {
        // |p| >= eps decided as re^2 + im^2 >= eps^2 in double: both squares are exact there
        // and the sum rounds once, so the decision is reproducible bit for bit.  The fp32 sum
        // of squares s is within 2^-22 (relative) of the exact one, so d = s - mid, mid =
        // fl(eps^2), settles every case with |d| > hw = 2^-20 mid.  The first pass keeps
        // everything with d >= keep = -hw and remembers the smallest |d| it saw; if any lane of
        // the warp saw one inside the band, the warp redoes its rows with the double comparison
        // (shared memory still holds the original of every element the first pass kept).
        const float mid = prm.gate_mid, hw = prm.gate_hw, keep = prm.gate_keep;
        const bool want_mask = MASKED && prm.mask != nullptr;
        uint32_t *const mrow0 = prm.mask + ((long long)b * L + s0) * prm.MW + g * 2;
        const bool second_word = g * 2 + 1 < prm.MW;
        // DYN: the rows' retention logits, all requested up front so that their latencies overlap
        float2 lg[DYN ? T : 1];
        if constexpr (DYN) {
#pragma unroll
            for (int i = 0; i < T; ++i) {
                lg[i] = make_float2(0.f, 0.f);
                if (FULL || i < nvalid) {
                    const float *gl = prm.gamma_logit + ((long long)b * L + s0 + i) * prm.H;
                    if (vA) lg[i].x = gl[hA];
                    if (vB) lg[i].y = gl[hB];
                }
            }
        }
        auto pass = [&](auto exact_tag, auto mask_tag) -> float {
            constexpr bool EXACT = decltype(exact_tag)::value, MASK = decltype(mask_tag)::value;
            float nearest = INFINITY;
            static_assert(T <= 16, "one 32-bit word per lane holds the gate bits of its rows");
            unsigned mkeep = 0u;                          // bit pair i: this lane's gate bits of row i
            e = zero4();
            dprod = make_float2(1.f, 1.f);
#pragma unroll
            for (int i = 0; i < T; ++i) {
                if (!EXACT && i % GR == 0) {
                    cp_async_wait_pending(NG - 1 - i / GR);       // rows i .. i+GR-1 have landed
                    if (IN16 && in_packed) __syncwarp();          // (brought by other lanes)
                    if (i == 0 && early_ptr != nullptr && !late_wait) {
                        er0 = ld_record(early_ptr + 2 * lane);
                        er1 = ld_record(early_ptr + 2 * lane + 1);
                    }
                }
                float4 v;
                if (IN16 && !EXACT) {                     // first touch: widen the staged bf16 in place
                    uint2 u;
                    if (in_packed) {
                        u = *reinterpret_cast<const uint2 *>(reinterpret_cast<const char *>(&sm.tile[0][w * T][0]) + T * 256 + i * 256 + lane * 8);
                        __syncwarp();                     // every lane has read row i before any lane widens over it
                    } else {
                        u = *reinterpret_cast<const uint2 *>(&xs[i * 32]);
                    }
                    const float2 cA = bf16x2_to_float2(u.x), cB = bf16x2_to_float2(u.y);
                    v = make_float4(cA.x, cA.y, cB.x, cB.y);
                } else {
                    v = xs[i * 32];
                }
                bool oA, oB;
                if (EXACT) {
                    oA = ((double)v.x * (double)v.x + (double)v.y * (double)v.y >= prm.eps2);
                    oB = ((double)v.z * (double)v.z + (double)v.w * (double)v.w >= prm.eps2);
                } else {
                    const float dA = fmaf(v.x, v.x, v.y * v.y) - mid, dB = fmaf(v.z, v.z, v.w * v.w) - mid;
                    nearest = fminf(nearest, fminf(fabsf(dA), fabsf(dB)));
                    oA = dA >= keep; oB = dB >= keep;
                }
                if (!FULL) { oA = oA && vA; oB = oB && vB; }
                v.x = oA ? v.x : 0.f; v.y = oA ? v.y : 0.f;
                v.z = oB ? v.z : 0.f; v.w = oB ? v.w : 0.f;
                xs[i * 32] = v;                           // phase 3 reads the gated value
                if (MASK) mkeep |= ((oA ? 1u : 0u) | (oB ? 2u : 0u)) << (2 * i);   // this lane's gate bits of row i
                if (FULL || i < nvalid) {
                    if constexpr (DYN) {
                        const float2 gm = make_float2(vA ? sigmoidf_fast(lg[i].x + fbA) : 0.f,
                                                      vB ? sigmoidf_fast(lg[i].y + fbB) : 0.f);
                        sm.sG[w * T + i][lane] = gm;
                        e = scale_step2(a, e, gm, v);
                        dprod.x *= gm.x; dprod.y *= gm.y;
                    } else {
                        e = cfma2(a, e, v);
                    }
                }
            }
            if (MASK) {
                // the rows' mask words (lanes 0..15 hold channels 0..31 of the group, word 0; lanes
                // 16..31 word 1): lane r gets word 0 of row r, lane 16 + r word 1
                const unsigned word = transpose_pairs16(mkeep, lane);
                const int r = lane & 15;
                if (r < T && (FULL || r < nvalid) && (lane < 16 || second_word)) mrow0[(long long)r * prm.MW + (lane >> 4)] = word;
            }
            return nearest;
        };
        using yes = std::true_type;
        using no = std::false_type;
        float nearest;
        if constexpr (MASKED) nearest = want_mask ? pass(no{}, yes{}) : pass(no{}, no{});
        else nearest = pass(no{}, no{});
        if (__any_sync(0xffffffffu, nearest <= hw)) {
            if constexpr (MASKED) { if (want_mask) pass(yes{}, yes{}); else pass(yes{}, no{}); }
            else pass(yes{}, no{});
        }
    } else {
        if (early_ptr != nullptr) {
            er0 = ld_record(early_ptr + 2 * lane);
            er1 = ld_record(early_ptr + 2 * lane + 1);
        }
        if constexpr (DYN) {
            // moving from row t+1 to row t multiplies by gamma_{t+1} conj(R): the factor of the
            // row processed just before (row L does not exist: factor 0 on a zero carry)
            // (the rows' logits are requested up front so that their latencies overlap)
            float2 lgb[T];
#pragma unroll
            for (int i = 0; i < T; ++i) {
                if constexpr (KIND == KIND_BWD) {
                    lgb[i] = row_logits(i, t_first - i);
                } else {
                    lgb[i] = make_float2(0.f, 0.f);
                    if (FULL || i < nvalid) {
                        const float *gl = prm.gamma_logit + ((long long)b * L + (t_first - i)) * prm.H;
                        if (vA) lgb[i].x = gl[hA];
                        if (vB) lgb[i].y = gl[hB];
                    }
                }
            }
            float2 gm;
            if (KIND == KIND_BWD && onehead) {
                const float lgp = __shfl_sync(0xffffffffu, mylogit, T);
                const bool in = t_first + 1 < L;
                gm = make_float2(in && vA ? sigmoidf_fast(lgp + fbA) : 0.f, in && vB ? sigmoidf_fast(lgp + fbB) : 0.f);
            } else {
                gm = row_gamma(t_first + 1);
            }
            gfirst = gm;
#pragma unroll
            for (int i = 0; i < T; ++i) {
                if (FULL || i < nvalid) {
                    e = scale_step2(a, e, gm, xs[i * 32]);
                    dprod.x *= gm.x; dprod.y *= gm.y;
                    gm = make_float2(vA ? sigmoidf_fast(lgb[i].x + fbA) : 0.f, vB ? sigmoidf_fast(lgb[i].y + fbB) : 0.f);
                    sm.sG[w * T + i][lane] = gm;
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < T; ++i)
                if (FULL || i < nvalid) e = cfma2(a, e, xs[i * 32]);
        }
    }
    // MIXBWD: conv taps and bias for phase 3, requested here so that they arrive during the carry exchange
    float mwA[4] = {}, mwB[4] = {}, mbA = 0.f, mbB = 0.f;
    if constexpr (MIX) {
        const int Kc = prm.conv_k;
        if (FULL && Kc == 4 && (reinterpret_cast<uintptr_t>(prm.conv_w) & 15) == 0) {
            // four taps: the two channels' taps are two aligned 16-byte words
            const float4 *w4 = reinterpret_cast<const float4 *>(prm.conv_w) + c0;
            const float4 a4 = w4[0], b4 = w4[1];
            mwA[0] = a4.x; mwA[1] = a4.y; mwA[2] = a4.z; mwA[3] = a4.w;
            mwB[0] = b4.x; mwB[1] = b4.y; mwB[2] = b4.z; mwB[3] = b4.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int kk = j - (4 - Kc);
                if (kk >= 0 && vA) mwA[j] = prm.conv_w[(long long)c0 * Kc + kk];
                if (kk >= 0 && vB) mwB[j] = prm.conv_w[(long long)(c0 + 1) * Kc + kk];
            }
        }
        if (prm.conv_bias != nullptr) { if (vA) mbA = prm.conv_bias[c0]; if (vB) mbB = prm.conv_bias[c0 + 1]; }
    }
    sm.sE[w][lane] = e;
    if constexpr (DYN) sm.sD[w][lane] = dprod;
    if (late_wait) {
        // from here on the workspace, the carried state and the outputs are touched
        grid_wait_previous();
        if (tid == 0) read_epoch();
        read_state_in();
    }
    __syncthreads();                                                           // barrier 2
    const unsigned long long epoch = sm.epoch;

    // ---- 2. publish the aggregate, fetch the carry window ----------------------------------
    const unsigned hook = sm.hook;
    const unsigned poll_limit = (hook >> 16) != 0u ? (hook >> 16) : prm.poll_limit;
    const bool withheld = (hook & 0xffffu) == (unsigned)k + 1u;      // test hook: this tile stays silent
    if (w == 0 && k + 1 < K && !withheld) {
        float4 E = sm.sE[0][lane];
        if constexpr (DYN) {
            float2 D = sm.sD[0][lane];
#pragma unroll
            for (int i = 1; i < W; ++i) {
                const float2 di = sm.sD[i][lane];
                E = scale_step2(aT, E, di, sm.sE[i][lane]);
                D.x *= di.x; D.y *= di.y;
            }
            publish_pair_d(prm.agg + (chain * K + k) * 64, lane, E, D, epoch, REC_AGGREGATE);
        } else {
#pragma unroll
            for (int i = 1; i < W; ++i) E = cfma2(aT, E, sm.sE[i][lane]);
            publish_pair(prm.agg + (chain * K + k) * 64, lane, E, epoch, REC_AGGREGATE);
        }
    }
    // slot r < nrec of the window: aggregate of tile k-1-r; slot M: the carry-in the window starts from
    for (int slot = w; slot <= M; slot += W) {
        float4 r = zero4();
        bool ok = true;
        const uint4 none = make_uint4(0u, 0u, 0u, 0u);
        const bool mine = (slot == w);                   // the slot read ahead of phase 1
        float2 rd = make_float2(0.f, 0.f);
        if (slot < nrec) {
            const uint4 *rec = prm.agg + (chain * K + (k - 1 - slot)) * 64;
            if constexpr (DYN) ok = poll_pair_d(rec, lane, epoch, poll_limit, mine ? er0 : none, mine ? er1 : none, r, rd);
            else ok = poll_pair(rec, lane, epoch, poll_limit, mine ? er0 : none, mine ? er1 : none, r);
        } else if (slot == M) {
            if (cpt > 0) {
                const uint4 *rec = prm.pre + (chain * prm.KP + cpt / M) * 64;
                if constexpr (DYN) ok = poll_pair_d(rec, lane, epoch, poll_limit, mine ? er0 : none, mine ? er1 : none, r, rd);
                else ok = poll_pair(rec, lane, epoch, poll_limit, mine ? er0 : none, mine ? er1 : none, r);
            } else {
                r = sinit;
            }
        }
        sm.sR[slot][lane] = r;
        if constexpr (DYN) sm.sRD[slot][lane] = rd;
        if (!ok) {
            sm.err = 1;
            atomicOr(&prm.ws->status, STATUS_CARRY_TIMEOUT);
        }
    }
    __syncthreads();                                                           // barrier 3
    if (tid == 0) sm.arrived = arrived;              // (it has come back by now) wanted again at the very end

    // ---- 3. carry-in, the recurrence itself, stores -----------------------------------------
    const bool failed = (sm.err != 0);
    const bool checkpoint = (k > 0 && k % M == 0 && k + 1 < K);
    float4 qa = zero4();
    float2 sacc_out = make_float2(0.f, 0.f);
    if (!failed) {
        float4 P = sm.sR[M][lane];
        {
            const float4 *cp = reinterpret_cast<const float4 *>(&sm.sCoef[2 * lane][0]);
            const float4 u1 = cp[1], u2 = cp[2];
            const float4 AA = make_float4(u1.x, u1.y, u2.z, u2.w);
#pragma unroll 1
            for (int i = nrec - 1; i >= 0; --i) {
                if constexpr (DYN) P = scale_step2(AA, P, sm.sRD[i][lane], sm.sR[i][lane]);
                else P = cfma2(AA, P, sm.sR[i][lane]);
            }
        }
        if (checkpoint && w == 0) {
            if constexpr (DYN) publish_pair_d(prm.pre + (chain * prm.KP + k / M) * 64, lane, P, make_float2(0.f, 0.f), epoch, REC_PREFIX);
            else publish_pair(prm.pre + (chain * prm.KP + k / M) * 64, lane, P, epoch, REC_PREFIX);
        }
#pragma unroll 1
        for (int i = 0; i < w; ++i) {
            if constexpr (DYN) P = scale_step2(aT, P, sm.sD[i][lane], sm.sE[i][lane]);
            else P = cfma2(aT, P, sm.sE[i][lane]);
        }

        // EAR: a planar row is 2C floats, as long as an interleaved one; the real parts of this
        // lane's two channels sit c0 floats into it, the imaginary parts C floats further
        // (with bf16 output every one of these offsets halves)
        char *const rbase = reinterpret_cast<char *>(prm.out) +
                            (EAR ? ((e0 - c0) * 8 + c0 * 4) / (OUT16 ? 2 : 1) : (OUT16 ? e0 * 4 : e0 * 8));
        const int orow = OUT16 ? rowbytes / 2 : rowbytes;
        const float cl = prm.clampv;
        // Ear taps of this lane's two channels, real and imaginary part: (left, centre, right,
        // bias).  A tap whose source harmonic lies outside the head is zero (zero padding), so the
        // values the shuffles bring in from a neighbouring head never count.
        float ewr[2][4] = {}, ewi[2][4] = {};
        if constexpr (EAR) {
            const int Fh = prm.F, Ke = prm.ear_k, lead = (3 - Ke) / 2;
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                const int c = c0 + ch;
                if (c < C) {
                    const int hh = c / Fh, kk = c - hh * Fh;
#pragma unroll
                    for (int j = 0; j < 3; ++j) {
                        const int jj = j - lead, src = kk + j - 1;
                        if (jj >= 0 && jj < Ke && src >= 0 && src < Fh) {
                            ewr[ch][j] = prm.ear_w[hh * Ke + jj];
                            ewi[ch][j] = prm.ear_w[(prm.H + hh) * Ke + jj];
                        }
                    }
                    if (prm.ear_bias != nullptr) { ewr[ch][3] = prm.ear_bias[hh]; ewi[ch][3] = prm.ear_bias[prm.H + hh]; }
                }
            }
        }
        // one output row of this lane's channel pair; every lane of the warp takes part (the Ear
        // form exchanges edge channels with the neighbouring lanes)
        auto store_row = [&](int i, float4 o) {
            char *r = const_cast<char *>(row_ptr(rbase, orow, i));
            if constexpr (OUT16 && !EAR) {
                const unsigned pA = float2_to_bf16x2(o.x, o.y), pB = float2_to_bf16x2(o.z, o.w);
                if (VEC) {
                    if (vA) __stcs(reinterpret_cast<uint2 *>(r), make_uint2(pA, pB));
                } else {
                    if (vA) __stcs(reinterpret_cast<unsigned *>(r), pA);
                    if (vB) __stcs(reinterpret_cast<unsigned *>(r) + 1, pB);
                }
            } else if constexpr (EAR) {
                const float lre = __shfl_up_sync(0xffffffffu, o.z, 1), lim = __shfl_up_sync(0xffffffffu, o.w, 1);
                const float rre = __shfl_down_sync(0xffffffffu, o.x, 1), rim = __shfl_down_sync(0xffffffffu, o.y, 1);
                const float zrA = fmaf(ewr[0][0], lre, fmaf(ewr[0][1], o.x, fmaf(ewr[0][2], o.z, ewr[0][3])));
                const float zrB = fmaf(ewr[1][0], o.x, fmaf(ewr[1][1], o.z, fmaf(ewr[1][2], rre, ewr[1][3])));
                const float ziA = fmaf(ewi[0][0], lim, fmaf(ewi[0][1], o.y, fmaf(ewi[0][2], o.w, ewi[0][3])));
                const float ziB = fmaf(ewi[1][0], o.y, fmaf(ewi[1][1], o.w, fmaf(ewi[1][2], rim, ewi[1][3])));
                if constexpr (OUT16) {
                    // planar row of 2C bf16: real parts, then imaginary parts
                    unsigned short *zr = reinterpret_cast<unsigned short *>(r), *zi = zr + C;
                    const unsigned pr = float2_to_bf16x2(zrA, zrB), pi = float2_to_bf16x2(ziA, ziB);
                    if (VEC) {
                        if (vA) { __stcs(reinterpret_cast<unsigned *>(zr), pr); __stcs(reinterpret_cast<unsigned *>(zi), pi); }
                    } else {
                        if (vA) { zr[0] = (unsigned short)(pr & 0xffffu); zi[0] = (unsigned short)(pi & 0xffffu); }
                        if (vB) { zr[1] = (unsigned short)(pr >> 16); zi[1] = (unsigned short)(pi >> 16); }
                    }
                } else {
                    float *zr = reinterpret_cast<float *>(r), *zi = zr + C;
                    if (VEC) {
                        if (vA) { __stcs(reinterpret_cast<float2 *>(zr), make_float2(zrA, zrB)); __stcs(reinterpret_cast<float2 *>(zi), make_float2(ziA, ziB)); }
                    } else {
                        if (vA) { __stcs(zr, zrA); __stcs(zi, ziA); }
                        if (vB) { __stcs(zr + 1, zrB); __stcs(zi + 1, ziB); }
                    }
                }
            } else if (VEC) {
                // 16-byte rows go out as st.global.cg (kept in L2 until evicted: measured 0.5 us faster on
                // the training shape than the evict-first form, which stays the better one for the
                // narrower stores of the other output forms)
                if (vA) __stcg(reinterpret_cast<float4 *>(r), o);
            } else {
                float2 *r2 = reinterpret_cast<float2 *>(r);
                if (vA) __stcs(r2, make_float2(o.x, o.y));
                if (vB) __stcs(r2 + 1, make_float2(o.z, o.w));
            }
        };
        // DYN: factor of the step into row i (forward: the row's own; backward: the factor of
        // the row processed before it), and the running sum of the logit gradient
        float2 gstep = make_float2(0.f, 0.f), sacc = make_float2(0.f, 0.f);
        if constexpr (DYN && REV) gstep = gfirst;
        // DYN backward: the heads this 64-channel group touches
        int h_lo = 0, h_hi = 0;
        if constexpr (DYN && REV) {
            const int c_hi = g * 64 + 63 < C - 1 ? g * 64 + 63 : C - 1;
            h_lo = (g * 64) / prm.F;
            h_hi = c_hi / prm.F;
        }
        float rowsum[DYN && REV ? T : 1] = {};           // per row: this lane's share of the head's logit gradient
        // MIXBWD: conv taps (right-aligned: tap j multiplies the hidden row 3 - j steps back), the
        // rolling window of hidden rows, and the sums for the conv gradients
        float2 hwin[4] = {};                             // h(t), h(t-1), h(t-2), h(t-3) of the current row
        float caA[5] = {}, caB[5] = {};
        float2 dwin[3] = {};                             // du of the three rows processed before the current one
        float2 dfirst[3] = {};                           // du of this thread's first three rows (finished after the barrier)
        const bool mact = prm.clamp_silu != 0;
        const bool mtap0 = prm.conv_k >= 4, mtap1 = prm.conv_k >= 3, mtap2 = prm.conv_k >= 2;
        float *const gh = reinterpret_cast<float *>(prm.out);
        if constexpr (MIX) {
#pragma unroll
            for (int r = 0; r < 3; ++r) hwin[r + 1] = *reinterpret_cast<const float2 *>(&sm.hrev[w * T + r][2 * lane]);
        }
        // one row of the MIXBWD form: lam -> du, kept in the row's (spent) input slot for the
        // conv transpose that follows the loop
        auto mix_row = [&](auto plain, int i, float4 lam) {
            constexpr bool PLAIN = decltype(plain)::value;    // every tap present, no clamp + SiLU: no tests
            hwin[0] = hwin[1]; hwin[1] = hwin[2]; hwin[2] = hwin[3];
            hwin[3] = *reinterpret_cast<const float2 *>(&sm.hrev[w * T + i + 3][2 * lane]);
            float uA = mbA, uB = mbB;                    // the forward's fmaf chain, tap order
            if (PLAIN || mtap0) { uA = fmaf(mwA[0], hwin[3].x, uA); uB = fmaf(mwB[0], hwin[3].y, uB); }
            if (PLAIN || mtap1) { uA = fmaf(mwA[1], hwin[2].x, uA); uB = fmaf(mwB[1], hwin[2].y, uB); }
            if (PLAIN || mtap2) { uA = fmaf(mwA[2], hwin[1].x, uA); uB = fmaf(mwB[2], hwin[1].y, uB); }
            uA = fmaf(mwA[3], hwin[0].x, uA); uB = fmaf(mwB[3], hwin[0].y, uB);
            const float duA = vA ? prelude_du<PLAIN>(uA, lam.x, lam.y, mact, prm.gate_tau) : 0.f;
            const float duB = vB ? prelude_du<PLAIN>(uB, lam.z, lam.w, mact, prm.gate_tau) : 0.f;
            *reinterpret_cast<float2 *>(&xs[i * 32]) = make_float2(duA, duB);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                caA[j] = fmaf(duA, hwin[3 - j].x, caA[j]);
                caB[j] = fmaf(duB, hwin[3 - j].y, caB[j]);
            }
            caA[4] += duA; caB[4] += duB;
            // Transposed conv: grad_h(t) = sum_j w[j] du(t + 3 - j).  In processing order (row R is
            // time t_hi - R) that is du of rows R-3 .. R: from the fourth row of a thread on they are
            // all its own and still in registers; its first three rows wait for the barrier.
            if (i < 3) {
                dfirst[i] = make_float2(duA, duB);
            } else {
                const float gA = fmaf(mwA[3], duA, fmaf(mwA[2], dwin[0].x, fmaf(mwA[1], dwin[1].x, mwA[0] * dwin[2].x)));
                const float gB = fmaf(mwB[3], duB, fmaf(mwB[2], dwin[0].y, fmaf(mwB[1], dwin[1].y, mwB[0] * dwin[2].y)));
                float *o = gh + (e0 - (long long)i * C);
                if (VEC) { if (vA) __stcs(reinterpret_cast<float2 *>(o), make_float2(gA, gB)); }
                else { if (vA) __stcs(o, gA); if (vB) __stcs(o + 1, gB); }
            }
            dwin[2] = dwin[1]; dwin[1] = dwin[0]; dwin[0] = make_float2(duA, duB);
        };
        auto step_row = [&](auto plain, int i, bool clamped) {
            if (MIX && !(FULL || i < nvalid)) *reinterpret_cast<float2 *>(&xs[i * 32]) = make_float2(0.f, 0.f);      // no such row: its du is 0
            if (FULL || i < nvalid) {
                float2 gown = make_float2(0.f, 0.f);
                if constexpr (DYN) {
                    if (!REV) gstep = sm.sG[w * T + i][lane];
                    P = scale_step2(a, P, gstep, xs[i * 32]);
                    if (REV) { gown = sm.sG[w * T + i][lane]; gstep = gown; }
                } else {
                    P = cfma2(a, P, xs[i * 32]);
                }
                if constexpr (MIX) mix_row(plain, i, clamped ? clamp4(P, cl) : P);
                else store_row(i, clamped ? clamp4(P, cl) : P);
                if constexpr (REV) {
                    // conj(lam) * P_{t-1}
                    const float4 q = sm.tile[1][w * T + i][lane];
                    if constexpr (DYN) {
                        if (prm.aux != nullptr) {
                            // u = conj(lam_t) P_{t-1};  d gamma_t = Re(e^{i theta} u), chained through the
                            // sigmoid; the rotation gradient sums gamma_t u
                            const float uAx = fmaf(P.x, q.x, P.y * q.y), uAy = fmaf(P.x, q.y, -P.y * q.x);
                            const float uBx = fmaf(P.z, q.z, P.w * q.w), uBy = fmaf(P.z, q.w, -P.w * q.z);
                            qa.x = fmaf(gown.x, uAx, qa.x); qa.y = fmaf(gown.x, uAy, qa.y);
                            qa.z = fmaf(gown.y, uBx, qa.z); qa.w = fmaf(gown.y, uBy, qa.w);
                            // a holds conj(e^{i theta}) in the backward
                            const float sA = gown.x * (1.f - gown.x) * fmaf(a.x, uAx, a.y * uAy);
                            const float sB = gown.y * (1.f - gown.y) * fmaf(a.z, uBx, a.w * uBy);
                            sacc.x += sA; sacc.y += sB;
                            if (prm.grad_logit != nullptr && h_lo == h_hi) {
                                rowsum[i] = sA + sB;             // one head: all rows are reduced together below
                            } else if (prm.grad_logit != nullptr) {
                                // sum over the harmonics of each head present in this 64-channel group
                                for (int h = h_lo; h <= h_hi; ++h) {
                                    float v = (vA && hA == h ? sA : 0.f) + (vB && hB == h ? sB : 0.f);
#pragma unroll
                                    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                                    if (lane == 0) {
                                        float *gl = prm.grad_logit + ((long long)b * L + (t_first - i)) * prm.H + h;
                                        if (prm.logit_direct) *gl = v; else atomicAdd(gl, v);
                                    }
                                }
                            }
                        }
                    } else {
                        qa.x = fmaf(P.x, q.x, fmaf(P.y, q.y, qa.x));
                        qa.y = fmaf(P.x, q.y, fmaf(-P.y, q.x, qa.y));
                        qa.z = fmaf(P.z, q.z, fmaf(P.w, q.w, qa.z));
                        qa.w = fmaf(P.z, q.w, fmaf(-P.w, q.z, qa.w));
                    }
                }
            }
        };
        auto rows = [&](auto plain) {
            if (cl > 0.f) {
#pragma unroll
                for (int i = 0; i < T; ++i) step_row(plain, i, true);
            } else {
#pragma unroll
                for (int i = 0; i < T; ++i) step_row(plain, i, false);
            }
        };
        if constexpr (MIX) {
            if (prm.conv_k == 4 && !mact) rows(std::true_type{}); else rows(std::false_type{});
        } else {
            rows(std::false_type{});
        }
        sacc_out = sacc;
        if constexpr (DYN && REV) {
            if (prm.grad_logit != nullptr && prm.aux != nullptr && h_lo == h_hi) {
                // T row sums over the 32 lanes at once: each exchange halves the rows a lane still
                // carries, so that after log2(T) rounds lane (32/T) r holds row r's partial; then
                // plain butterflies among the 32/T lanes that share a row.  9 shuffles for 8 rows.
#pragma unroll
                for (int n = T / 2, off = 16; n >= 1; n >>= 1, off >>= 1) {
                    const bool upper = (lane & off) != 0;
#pragma unroll
                    for (int j = 0; j < n; ++j) {
                        const float send = upper ? rowsum[j] : rowsum[j + n];
                        const float keep = upper ? rowsum[j + n] : rowsum[j];
                        rowsum[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                    }
                }
#pragma unroll
                for (int off = 16 / T; off >= 1; off >>= 1) rowsum[0] += __shfl_xor_sync(0xffffffffu, rowsum[0], off);
                constexpr int LPR = 32 / T;              // lanes per row
                const int row = lane / LPR;
                if (lane % LPR == 0 && (FULL || row < nvalid)) {
                    float *gl = prm.grad_logit + ((long long)b * L + (t_first - row)) * prm.H + h_lo;
                    if (prm.logit_direct) *gl = rowsum[0]; else atomicAdd(gl, rowsum[0]);
                }
            }
        }
        // An Inf or NaN that entered anywhere (an input, the carried state, an overflow) is still
        // in the chain's last state: the recurrence never makes it finite again.  (A NaN push
        // itself fails the gate's comparison and is dropped like any closed gate.)
        if (nvalid > 0 && s0 + nvalid == L && nonfinite4(P)) atomicOr(&prm.ws->status, STATUS_NONFINITE);
        // the thread that owns the last step writes the carried state (never clamped)
        if (prm.state_out != nullptr && nvalid > 0 && s0 + nvalid == L) {
            if (REV) {                                   // grad_state_in = conj(a_0) lam_0
                P = cmul2(a, P);
                if constexpr (DYN) { P.x *= gstep.x; P.y *= gstep.x; P.z *= gstep.y; P.w *= gstep.y; }
            }
            float2 *s = prm.state_out + (long long)b * C + c0;
            if (vA) s[0] = make_float2(P.x, P.y);
            if (vB) s[1] = make_float2(P.z, P.w);
        }
        if constexpr (MIX) {
            // The first three rows of every thread need du of the warp before it; the tile's first
            // three rows would need the tile after it in time, so their du (and the du of its three
            // earliest rows, for the tile before it) go to the edge area and the epilogue launch
            // finishes those rows.
            // Every warp's partial sums go into its own rows of the saved-state tile, which only it
            // read and which it has spent: 320 floats of conv sums, then the rotation sums, then the
            // retention sums.  One barrier then serves the du rows and all the sums.
            static_assert(T * 512 >= 2048, "a warp's spent rows hold its partial sums");
            float *const part = reinterpret_cast<float *>(&sm.tile[1][w * T][0]);
            constexpr int PSTRIDE = T * 128;             // floats between the warps' areas
            if (prm.cpart != nullptr) {
#pragma unroll
                for (int j = 0; j < 5; ++j) { part[lane * 10 + j] = caA[j]; part[lane * 10 + 5 + j] = caB[j]; }
            }
            if (prm.qpart != nullptr) {
                reinterpret_cast<float4 *>(part + 320)[lane] = qa;
                if constexpr (DYN) reinterpret_cast<float2 *>(part + 448)[lane] = sacc_out;
            }
            __syncthreads();
            const float4 (*du)[32] = sm.tile[0];
#pragma unroll
            for (int i = 0; i < 3 && i < T; ++i) {
                const int R = w * T + i;
                if ((FULL || i < nvalid) && R >= 3) {
                    float dA = 0.f, dB = 0.f;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // rows of this thread are still in registers, earlier ones come from the tile
                        const float2 d = (i - 3 + j >= 0) ? dfirst[i - 3 + j >= 0 ? i - 3 + j : 0]
                                                          : *reinterpret_cast<const float2 *>(&du[R - 3 + j][lane]);
                        dA = fmaf(mwA[j], d.x, dA); dB = fmaf(mwB[j], d.y, dB);
                    }
                    float *o = gh + (e0 - (long long)i * C);
                    if (VEC) { if (vA) __stcs(reinterpret_cast<float2 *>(o), make_float2(dA, dB)); }
                    else { if (vA) __stcs(o, dA); if (vB) __stcs(o + 1, dB); }
                }
            }
            // the sums over the warps, each in a fixed order, shared out among the warps
            const float *const parts = reinterpret_cast<const float *>(&sm.tile[1][0][0]);
            if (w == W - 1) {
                const long long rem = L - (long long)k * TILE;
                const int nrows = rem >= TILE ? TILE : (int)rem;           // rows this tile has
                float *eg = prm.edge_du + (((long long)b * K + k) * 6) * C + c0;
#pragma unroll
                for (int r = 0; r < 3; ++r) {
                    const float2 hi = r < nrows ? *reinterpret_cast<const float2 *>(&du[r][lane]) : make_float2(0.f, 0.f);
                    const float2 lo = r < nrows ? *reinterpret_cast<const float2 *>(&du[nrows - 1 - r][lane]) : make_float2(0.f, 0.f);
                    if (vA) { eg[(long long)r * C] = hi.x; eg[(long long)(3 + r) * C] = lo.x; }
                    if (vB) { eg[(long long)r * C + 1] = hi.y; eg[(long long)(3 + r) * C + 1] = lo.y; }
                }
            }
            if (prm.cpart != nullptr) {
                float *o = prm.cpart + (((long long)b * K + k) * C + c0) * 5;
                for (int j = w; j < 10; j += W) {
                    float acc = 0.f;
#pragma unroll
                    for (int i = 0; i < W; ++i) acc += parts[i * PSTRIDE + lane * 10 + j];
                    if (j < 5 ? vA : vB) o[j] = acc;
                }
            }
            if (prm.qpart != nullptr) {
                if (w == 2 % W) {
                    float4 acc = reinterpret_cast<const float4 *>(parts + 320)[lane];
#pragma unroll
                    for (int i = 1; i < W; ++i) {
                        const float4 v = reinterpret_cast<const float4 *>(parts + i * PSTRIDE + 320)[lane];
                        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                    }
                    float2 *qp = prm.qpart + ((long long)b * K + k) * C + c0;
                    if (vA) qp[0] = make_float2(acc.x, acc.y);
                    if (vB) qp[1] = make_float2(acc.z, acc.w);
                }
                if constexpr (DYN) {
                    if (prm.spart != nullptr && w == 3 % W) {
                        float2 acc = reinterpret_cast<const float2 *>(parts + 448)[lane];
#pragma unroll
                        for (int i = 1; i < W; ++i) {
                            const float2 v = reinterpret_cast<const float2 *>(parts + i * PSTRIDE + 448)[lane];
                            acc.x += v.x; acc.y += v.y;
                        }
                        float *sp = prm.spart + ((long long)b * K + k) * C + c0;
                        if (vA) sp[0] = acc.x;
                        if (vB) sp[1] = acc.y;
                    }
                }
            }
        }
    } else if (checkpoint && w == 0) {
        if constexpr (DYN) publish_pair_d(prm.pre + (chain * prm.KP + k / M) * 64, lane, zero4(), make_float2(0.f, 0.f), epoch, REC_POISON);
        else publish_pair(prm.pre + (chain * prm.KP + k / M) * 64, lane, zero4(), epoch, REC_POISON);
    }
    if constexpr (KIND == KIND_FUSED) {
        // the call's last conv_k-1 hidden rows (reaching back into the carried tail when the
        // call is shorter than that) become the next call's history
        const int Kh = prm.conv_k - 1;
        if (prm.tail_out != nullptr && k == K - 1 && w == 0 && !failed) {
            const float *hin = reinterpret_cast<const float *>(prm.in);
            for (int r = 0; r < Kh; ++r) {
                const long long t = L - Kh + r;
                float vA_ = 0.f, vB_ = 0.f;
                if (t >= 0 && IN16) {
                    const unsigned short *src = reinterpret_cast<const unsigned short *>(prm.in) + ((long long)b * L + t) * C + c0;
                    if (vA) vA_ = __uint_as_float((unsigned)src[0] << 16);
                    if (vB) vB_ = __uint_as_float((unsigned)src[1] << 16);
                } else if (t >= 0) {
                    const float *src = hin + ((long long)b * L + t) * C + c0;
                    if (vA) vA_ = src[0];
                    if (vB) vB_ = src[1];
                } else if (prm.tail_in != nullptr) {
                    const float *src = prm.tail_in + ((long long)b * Kh + (Kh + t)) * C + c0;
                    if (vA) vA_ = src[0];
                    if (vB) vB_ = src[1];
                }
                float *dst = prm.tail_out + ((long long)b * Kh + r) * C + c0;
                if (vA) dst[0] = vA_;
                if (vB) dst[1] = vB_;
            }
        }
    }
    if constexpr (REV && !MIX) {
        if (prm.qpart != nullptr) {
            __syncthreads();
            sm.sE[w][lane] = qa;
            __syncthreads();
            if (w == 0) {
                float4 acc = sm.sE[0][lane];
#pragma unroll
                for (int i = 1; i < W; ++i) {
                    const float4 v = sm.sE[i][lane];
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                float2 *qp = prm.qpart + ((long long)b * K + k) * C + c0;
                if (vA) qp[0] = make_float2(acc.x, acc.y);
                if (vB) qp[1] = make_float2(acc.z, acc.w);
            }
            if constexpr (DYN) {
                if (prm.spart != nullptr) {
                    sm.sD[w][lane] = sacc_out;
                    __syncthreads();
                    if (w == 0) {
                        float2 acc = sm.sD[0][lane];
#pragma unroll
                        for (int i = 1; i < W; ++i) { const float2 v = sm.sD[i][lane]; acc.x += v.x; acc.y += v.y; }
                        float *sp = prm.spart + ((long long)b * K + k) * C + c0;
                        if (vA) sp[0] = acc.x;
                        if (vB) sp[1] = acc.y;
                    }
                }
            }
        }
    }
    if (tid == 0 && sm.arrived == gridDim.x * gridDim.y * gridDim.z - 1) {
        // every CTA of this launch has read the epoch: open the next one (the launch after this
        // one reads it only when this one is complete)
        st_volatile_u32(&prm.ws->done, 0u);
        st_volatile_u64(&prm.ws->epoch, sm.epoch + 1ull);
    }
}

template <int T, int W, int KIND, bool VEC, int MINB, bool DYN = false, bool EAR = false, int IO = IO_F32, bool MASKED = true, bool LATE = false>
__global__ void __launch_bounds__(W * 32, MINB) cawn_scan_kernel(const ScanParams prm)
{
    constexpr int TILE = T * W;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    ScanSmem<T, W, KIND, DYN> &sm = *reinterpret_cast<ScanSmem<T, W, KIND, DYN> *>(smem_raw);

    // grid = (G, B, K): blocks are dispatched x fastest, so a tile's predecessors along time
    // (smaller k) always have smaller linear block indices
    const int g = blockIdx.x, b = blockIdx.y;
    const int k = blockIdx.z;                         // tile index along (logical) time
    grid_launch_dependents();
    const bool full = ((long long)(k + 1) * TILE <= prm.L) && (g * 64 + 64 <= prm.C);
    if (full) scan_tile<T, W, KIND, VEC, DYN, true, EAR, IO, MASKED, LATE>(prm, sm, g, b, k);
    else      scan_tile<T, W, KIND, VEC, DYN, false, EAR, IO, MASKED, LATE>(prm, sm, g, b, k);
}

}  // namespace cawn
