// Launch templates shared by the cawn_launch_*.cu translation units.
#pragma once
#include "cawn_launch.cuh"

namespace cawn {

// The float4 path needs every row segment on a 16-byte boundary: C even (the arrays
// themselves are checked to be 16-byte aligned).  The tile is staged in dynamic shared memory;
// MINB is the number of CTAs per SM the register allocation leaves room for.
template <int T, int W, int KIND, bool VEC, int MINB, bool DYN, bool EAR = false, int IO = IO_F32, bool MASKED = true, bool LATE = false>
cudaError_t launch_scan_inst(const ScanParams &sp, cudaStream_t st)
{
    constexpr size_t smem = sizeof(ScanSmem<T, W, KIND, DYN>);
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(cawn_scan_kernel<T, W, KIND, VEC, MINB, DYN, EAR, IO, MASKED, LATE>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    // Launched with programmatic stream serialisation: when the launch before it on the stream
    // is one of these kernels, this one may start occupying SMs while that one drains; the
    // kernel itself waits for its predecessor before touching anything that one may have written.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)sp.G, (unsigned)sp.B, (unsigned)sp.K);
    cfg.blockDim = dim3(W * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if constexpr (KIND == KIND_FUSED) {
        // how many of these CTAs the device holds at once (asked once per device)
        static int slots[64] = {};
        ScanParams spf = sp;
        if (dev >= 0 && dev < 64) {
            if (slots[dev] == 0) {
                int per_sm = 0, sms = 0;
                if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, cawn_scan_kernel<T, W, KIND, VEC, MINB, DYN, EAR, IO, MASKED, LATE>,
                                                                  W * 32, smem) == cudaSuccess &&
                    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && per_sm > 0 && sms > 0)
                    slots[dev] = per_sm * sms;
                else
                    slots[dev] = -1;
            }
            spf.first_wave = slots[dev] > 0 ? slots[dev] : 0;
        }
        return cudaLaunchKernelEx(&cfg, cawn_scan_kernel<T, W, KIND, VEC, MINB, DYN, EAR, IO, MASKED, LATE>, spf);
    }
    return cudaLaunchKernelEx(&cfg, cawn_scan_kernel<T, W, KIND, VEC, MINB, DYN, EAR, IO, MASKED, LATE>, sp);
}
template <int T, int W, int KIND, int MINB, bool DYN = false, bool EAR = false, int IO = IO_F32, bool MASKED = true, bool LATE = false>
cudaError_t launch_scan(const ScanParams &sp, cudaStream_t st)
{
    return sp.C % 2 == 0 ? launch_scan_inst<T, W, KIND, true, MINB, DYN, EAR, IO, MASKED, LATE>(sp, st)
                         : launch_scan_inst<T, W, KIND, false, MINB, DYN, EAR, IO, MASKED, LATE>(sp, st);
}
// The bf16 storage forms of the static forward (io = IO_IN_BF16, IO_OUT_BF16 or both).
template <int KIND, int IO>
cudaError_t launch_scan_io(TileShape ts, const ScanParams &sp, cudaStream_t st)
{
    // (the Cartesian long-call shape exists with and without the gate-mask output compiled in)
    if (KIND == KIND_FWD && ts.T == 16 && sp.mask == nullptr) return launch_scan<16, 8, KIND, 3, false, false, IO, false>(sp, st);
    if (ts.T == 16) return launch_scan<16, 8, KIND, 3, false, false, IO>(sp, st);
    return launch_scan<4, 4, KIND, 8, false, false, IO>(sp, st);
}

}  // namespace cawn
