#include "cawn_launch_impl.cuh"

namespace cawn {

// bf16 storage of input and output together with the time-varying retention and / or the Ear
// epilogue: the forms of the paper's own layer (a bf16 network around the fp32 scan).
constexpr int IO_BOTH = IO_IN_BF16 | IO_OUT_BF16;

template <int KIND>
static cudaError_t launch_wide(TileShape ts, const ScanParams &sp, cudaStream_t st, bool dyn)
{
    const bool ear = sp.ear_w != nullptr;
    if (ts.T == 16) {
        if (dyn && ear) return launch_scan<16, 8, KIND, 2, true, true, IO_BOTH>(sp, st);
        if (dyn) return launch_scan<16, 8, KIND, 2, true, false, IO_BOTH>(sp, st);
        return launch_scan<16, 8, KIND, 3, false, true, IO_BOTH>(sp, st);
    }
    if (dyn && ear) return launch_scan<4, 4, KIND, 8, true, true, IO_BOTH>(sp, st);
    if (dyn) return launch_scan<4, 4, KIND, 8, true, false, IO_BOTH>(sp, st);
    return launch_scan<4, 4, KIND, 8, false, true, IO_BOTH>(sp, st);
}

cudaError_t launch_fwd_bf16_wide(TileShape ts, const ScanParams &sp, cudaStream_t st, bool dyn)
{
    return launch_wide<KIND_FWD>(ts, sp, st, dyn);
}

cudaError_t launch_fused_bf16_wide(TileShape ts, const ScanParams &sp, cudaStream_t st, bool dyn)
{
    return launch_wide<KIND_FUSED>(ts, sp, st, dyn);
}

}  // namespace cawn
