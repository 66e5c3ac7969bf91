// Device-side helpers shared by the libcawn kernels: paired complex float arithmetic, the
// workspace header, and the 16-byte tagged records the inter-tile carry protocol uses.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace cawn {

// ---------------------------------------------------------------------------------------
// Workspace layout: [WsHeader (256 B)] [aggregate records] [prefix records] [op-specific areas]
// epoch  : generation number of the current launch.  Records carry the epoch they were
//          written in; a record of another epoch is stale, so nothing is cleared between
//          launches (and a launch replayed from a CUDA graph still sees a fresh epoch).
// done   : CTAs of the current launch that have read the epoch.  The last one to arrive
//          resets the count and opens the next epoch; by then nobody reads `epoch` any more.
// status : sticky device-side conditions (bits: STATUS_CARRY_TIMEOUT, STATUS_NONFINITE), cleared by
//          cawn_poll_status.
// hook   : test hook for the bounded waits, 0 = off: low 16 bits = 1 + index of the tile (of every
//          chain) that does not publish its aggregate, high 16 bits = poll bound to use instead
//          of the normal one.  Only cawn_workspace_set_wait_hook writes it.
struct __align__(16) WsHeader {
    unsigned long long epoch;
    unsigned int hook;           // next to the epoch: a CTA reads both with one 16-byte load
    unsigned int done;
    unsigned int status;
    unsigned int reserved[59];
};
static_assert(sizeof(WsHeader) == 256, "workspace header is 256 bytes");

enum : unsigned { REC_AGGREGATE = 1u, REC_PREFIX = 2u, REC_POISON = 3u };
enum : unsigned { STATUS_CARRY_TIMEOUT = 1u, STATUS_NONFINITE = 2u };

// true unless all four components are finite (their sum is then finite too, short of overflow,
// which is reported just the same)
__device__ __forceinline__ bool nonfinite4(float4 v)
{
    return !(fabsf((v.x + v.y) + (v.z + v.w)) < INFINITY);
}

// ---------------------------------------------------------------------------------------
// Every lane works on two adjacent channels at once; a float4 holds (re0, im0, re1, im1).
// a * b + c on both channels of a pair
__device__ __forceinline__ float4 cfma2(float4 a, float4 b, float4 c)
{
    float4 r;
    r.x = fmaf(a.x, b.x, fmaf(-a.y, b.y, c.x));
    r.y = fmaf(a.x, b.y, fmaf(a.y, b.x, c.y));
    r.z = fmaf(a.z, b.z, fmaf(-a.w, b.w, c.z));
    r.w = fmaf(a.z, b.w, fmaf(a.w, b.z, c.w));
    return r;
}
__device__ __forceinline__ float4 cmul2(float4 a, float4 b)
{
    float4 r;
    r.x = fmaf(a.x, b.x, -a.y * b.y);
    r.y = fmaf(a.x, b.y, a.y * b.x);
    r.z = fmaf(a.z, b.z, -a.w * b.w);
    r.w = fmaf(a.z, b.w, a.w * b.z);
    return r;
}
__device__ __forceinline__ float clampf(float v, float c) { return fminf(fmaxf(v, -c), c); }
__device__ __forceinline__ float4 clamp4(float4 v, float c)
{
    return make_float4(clampf(v.x, c), clampf(v.y, c), clampf(v.z, c), clampf(v.w, c));
}
__device__ __forceinline__ float4 zero4() { return make_float4(0.f, 0.f, 0.f, 0.f); }

// ---------------------------------------------------------------------------------------
// Carry records: {re, im, tag} in one aligned 16-byte word, written and read with single
// 128-bit accesses at GPU scope so value and tag are always seen together.
// tag = epoch * 4 + kind; kind 0 never occurs in a written record.
__device__ __forceinline__ void st_record(uint4 *p, float re, float im, unsigned long long tag)
{
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};"
                 :: "l"(p), "r"(__float_as_uint(re)), "r"(__float_as_uint(im)),
                    "r"((unsigned)(tag & 0xffffffffull)), "r"((unsigned)(tag >> 32))
                 : "memory");
}
__device__ __forceinline__ uint4 ld_record(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
// epoch and hook of a workspace header in one access
__device__ __forceinline__ void ld_epoch_hook(const void *hdr, unsigned long long &epoch, unsigned &hook)
{
    unsigned x, y, z;
    [[maybe_unused]] unsigned w;                         // the arrival count: not used here
    asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "l"(hdr) : "memory");
    epoch = ((unsigned long long)y << 32) | x;
    hook = z;
}
__device__ __forceinline__ void st_volatile_u64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.volatile.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_volatile_u32(unsigned *p, unsigned v)
{
    asm volatile("st.volatile.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// 0 = not written in this epoch yet, else the record's kind.
__device__ __forceinline__ unsigned record_kind(uint4 r, unsigned long long epoch)
{
    const unsigned long long tag = ((unsigned long long)r.w << 32) | r.z;
    return (tag >> 2) == epoch ? (unsigned)(tag & 3ull) : 0u;
}

// Publish the two records of this lane's channel pair (lane l owns records 2l and 2l+1 of the
// 64 that belong to one tile).
__device__ __forceinline__ void publish_pair(uint4 *tile_recs, int lane, float4 v,
                                             unsigned long long epoch, unsigned kind)
{
    const unsigned long long tag = epoch * 4ull + kind;
    st_record(tile_recs + 2 * lane, v.x, v.y, tag);
    st_record(tile_recs + 2 * lane + 1, v.z, v.w, tag);
}

// Wait (with a bound) until both records of this lane's pair carry `epoch`.  (r0, r1) are a
// first reading taken earlier (zeros if none was taken): if it is already valid no further load
// is issued.  Returns false when the wait ran out or the writer published POISON.
__device__ __forceinline__ bool poll_pair(const uint4 *tile_recs, int lane, unsigned long long epoch,
                                          unsigned poll_limit, uint4 r0, uint4 r1, float4 &v)
{
    const uint4 *p = tile_recs + 2 * lane;
    unsigned polls = 0;
    for (;;) {
        const unsigned k0 = record_kind(r0, epoch), k1 = record_kind(r1, epoch);
        if (k0 != 0u && k1 != 0u) {
            v = make_float4(__uint_as_float(r0.x), __uint_as_float(r0.y),
                            __uint_as_float(r1.x), __uint_as_float(r1.y));
            return k0 != REC_POISON && k1 != REC_POISON;
        }
        if (++polls > poll_limit) { v = zero4(); return false; }
        if (polls > 4) __nanosleep(polls > 64 ? 256 : 32);
        r0 = ld_record(p);
        r1 = ld_record(p + 1);
    }
}

// Gate-mask words from per-lane bits.  Lane l of a half-warp holds in bit pair i of `m` the two gate
// bits (its two channels) of row i, i < 16.  Returns, in lane r of the same half-warp, the word
// whose bit pair l holds what lane l had for row r: the mask word of row r for the half-warp's 32
// channels.  A 16 x 16 transpose of 2-bit entries over 16 lanes: four butterfly exchanges.
__device__ __forceinline__ unsigned transpose_pairs16(unsigned m, int lane)
{
#pragma unroll
    for (int d = 8; d >= 1; d >>= 1) {
        // the bit pairs whose index has bit d clear
        const unsigned m0 = d == 8 ? 0x0000ffffu : d == 4 ? 0x00ff00ffu : d == 2 ? 0x0f0f0f0fu : 0x33333333u;
        const unsigned y = __shfl_xor_sync(0xffffffffu, m, d);
        m = (lane & d) ? ((m & ~m0) | ((y & ~m0) >> (2 * d))) : ((m & m0) | ((y & m0) << (2 * d)));
    }
    return m;
}

// ---------------------------------------------------------------------------------------
// Time-varying retention: one step is  P <- g (a P) + x  with a real per-step factor g per
// channel on top of the fixed rotation a; a segment is summarised by its end state and the
// product of its factors.
__device__ __forceinline__ float4 scale_step2(float4 a, float4 P, float2 g, float4 x)
{
    const float4 t = cmul2(a, P);
    return make_float4(fmaf(g.x, t.x, x.x), fmaf(g.x, t.y, x.y), fmaf(g.y, t.z, x.z), fmaf(g.y, t.w, x.w));
}
// Single-instruction special functions in their flush-to-zero forms (no subnormal fix-up code
// around them).  What the callers rely on: ex2 of a large argument is +inf and of a very negative
// one +0, the reciprocal of +inf is +0 and of 1 is 1 (the limits of the sigmoid and tanh forms
// built from them); sines and cosines are taken of angles in [0, 2 pi] or [-pi, pi], where the
// approximation's absolute error (about 2^-21) is far below the tolerance, and only feed sums.
__device__ __forceinline__ float ex2_ftz(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_ftz(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void sincos_ftz(float x, float &sn, float &cs)
{
    asm("sin.approx.ftz.f32 %0, %1;" : "=f"(sn) : "f"(x));
    asm("cos.approx.ftz.f32 %0, %1;" : "=f"(cs) : "f"(x));
}
__device__ __forceinline__ float sigmoidf_fast(float s) { return rcp_ftz(1.f + ex2_ftz(s * -1.44269504088896f)); }

// Records of the time-varying form: {re, im, factor product, tag} with a 32-bit tag
// (epoch mod 2^30) * 4 + kind.
__device__ __forceinline__ unsigned record_kind32(uint4 r, unsigned long long epoch)
{
    return (r.w >> 2) == (unsigned)(epoch & 0x3fffffffull) ? (r.w & 3u) : 0u;
}
__device__ __forceinline__ void publish_pair_d(uint4 *tile_recs, int lane, float4 v, float2 d,
                                               unsigned long long epoch, unsigned kind)
{
    const unsigned tag = (unsigned)(epoch & 0x3fffffffull) * 4u + kind;
    uint4 *p = tile_recs + 2 * lane;
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};"
                 :: "l"(p), "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)), "r"(__float_as_uint(d.x)), "r"(tag) : "memory");
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};"
                 :: "l"(p + 1), "r"(__float_as_uint(v.z)), "r"(__float_as_uint(v.w)), "r"(__float_as_uint(d.y)), "r"(tag) : "memory");
}
__device__ __forceinline__ bool poll_pair_d(const uint4 *tile_recs, int lane, unsigned long long epoch,
                                            unsigned poll_limit, uint4 r0, uint4 r1, float4 &v, float2 &d)
{
    const uint4 *p = tile_recs + 2 * lane;
    unsigned polls = 0;
    for (;;) {
        const unsigned k0 = record_kind32(r0, epoch), k1 = record_kind32(r1, epoch);
        if (k0 != 0u && k1 != 0u) {
            v = make_float4(__uint_as_float(r0.x), __uint_as_float(r0.y),
                            __uint_as_float(r1.x), __uint_as_float(r1.y));
            d = make_float2(__uint_as_float(r0.z), __uint_as_float(r1.z));
            return k0 != REC_POISON && k1 != REC_POISON;
        }
        if (++polls > poll_limit) { v = zero4(); d = make_float2(0.f, 0.f); return false; }
        if (polls > 4) __nanosleep(polls > 64 ? 256 : 32);
        r0 = ld_record(p);
        r1 = ld_record(p + 1);
    }
}

}  // namespace cawn
