// Device-side helpers shared by the libcawn kernels: complex float arithmetic, the
// workspace header, and the 16-byte tagged records the inter-tile carry protocol uses.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace cawn {

// ---------------------------------------------------------------------------------------
// Workspace layout: [WsHeader (256 B)] [carry records] [op-specific areas]
// epoch  : generation number of the current launch; records tagged with another epoch are
//          stale, so nothing ever needs clearing between launches.  The last CTA of a launch
//          bumps it.
// done   : CTAs of the current launch that have finished (reset by the last one).
// status : sticky device-side error (cawn_status > 0), cleared by cawn_poll_status.
struct __align__(16) WsHeader {
    unsigned long long epoch;
    unsigned int done;
    unsigned int status;
    unsigned int reserved[60];
};
static_assert(sizeof(WsHeader) == 256, "workspace header is 256 bytes");

enum : unsigned { REC_AGGREGATE = 1u, REC_PREFIX = 2u, REC_POISON = 3u };

// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float2 cmul(float2 a, float2 b)
{
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
// a * b + c
__device__ __forceinline__ float2 cfma(float2 a, float2 b, float2 c)
{
    float2 r;
    r.x = fmaf(a.x, b.x, fmaf(-a.y, b.y, c.x));
    r.y = fmaf(a.x, b.y, fmaf(a.y, b.x, c.y));
    return r;
}
__device__ __forceinline__ float clampf(float v, float c) { return fminf(fmaxf(v, -c), c); }

// Integer power of a complex double by square-and-multiply (N is a compile-time constant).
template <int N>
__device__ __forceinline__ void cpow_int(double ar, double ai, double &rr, double &ri)
{
    double br = ar, bi = ai;
    rr = 1.0; ri = 0.0;
#pragma unroll
    for (int n = N; n > 0; n >>= 1) {
        if (n & 1) { const double t = rr * br - ri * bi; ri = rr * bi + ri * br; rr = t; }
        const double t = br * br - bi * bi; bi = 2.0 * br * bi; br = t;
    }
}

// ---------------------------------------------------------------------------------------
// Carry records: {re, im, tag} in one aligned 16-byte word, written and read with single
// 128-bit accesses so value and tag are always seen together.
// tag = epoch * 4 + kind.
__device__ __forceinline__ void st_record(uint4 *p, float2 v, unsigned long long tag)
{
    asm volatile("st.volatile.global.v4.u32 [%0], {%1, %2, %3, %4};"
                 :: "l"(p), "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)),
                    "r"((unsigned)(tag & 0xffffffffull)), "r"((unsigned)(tag >> 32))
                 : "memory");
}
__device__ __forceinline__ uint4 ld_record(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_volatile_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_volatile_u64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.volatile.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// One lane's look-back over the tiles before tile k of its chain, for its two channels.
// Tile 0 of a chain always publishes a PREFIX, so the walk ends there at the latest.
// `chain` points at the records of tile 0 (64 per tile: lane and lane+32).
// Returns false when a wait ran out of polls or a predecessor published POISON.
__device__ __forceinline__ bool carry_lookback(const uint4 *chain, int k, int lane,
                                               bool v0, bool v1, unsigned long long epoch,
                                               float2 aW0, float2 aW1, unsigned poll_limit,
                                               float2 &S0, float2 &S1)
{
    int i0 = k - 1, i1 = k - 1;
    bool d0 = !v0, d1 = !v1, ok = true;
    float2 w0 = make_float2(1.f, 0.f), w1 = w0;
    S0 = make_float2(0.f, 0.f);
    S1 = S0;
    unsigned polls = 0;
    while (!(d0 && d1)) {
        uint4 r0 = make_uint4(0, 0, 0, 0), r1 = r0;
        if (!d0) r0 = ld_record(chain + (long long)i0 * 64 + lane);
        if (!d1) r1 = ld_record(chain + (long long)i1 * 64 + lane + 32);
        bool progressed = false;
        if (!d0) {
            const unsigned long long tag = ((unsigned long long)r0.w << 32) | r0.z;
            const unsigned kind = (unsigned)(tag & 3ull);
            if ((tag >> 2) == epoch && kind != 0u) {       // kind 0: never written (zeroed workspace)
                progressed = true;
                if (kind == REC_POISON || (kind != REC_PREFIX && i0 == 0)) { ok = false; d0 = true; }
                else {
                    S0 = cfma(w0, make_float2(__uint_as_float(r0.x), __uint_as_float(r0.y)), S0);
                    if (kind == REC_PREFIX) d0 = true;
                    else { w0 = cmul(w0, aW0); --i0; }
                }
            }
        }
        if (!d1) {
            const unsigned long long tag = ((unsigned long long)r1.w << 32) | r1.z;
            const unsigned kind = (unsigned)(tag & 3ull);
            if ((tag >> 2) == epoch && kind != 0u) {
                progressed = true;
                if (kind == REC_POISON || (kind != REC_PREFIX && i1 == 0)) { ok = false; d1 = true; }
                else {
                    S1 = cfma(w1, make_float2(__uint_as_float(r1.x), __uint_as_float(r1.y)), S1);
                    if (kind == REC_PREFIX) d1 = true;
                    else { w1 = cmul(w1, aW1); --i1; }
                }
            }
        }
        if (!progressed) {
            if (++polls > poll_limit) { ok = false; break; }
            if (polls > 8) __nanosleep(polls > 64 ? 200 : 40);
        }
    }
    return ok;
}

}  // namespace cawn
