#include "cawn_launch_impl.cuh"

namespace cawn {

cudaError_t launch_fwd_ear_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st)
{
    if (ts.T == 16) return launch_scan<16, 8, KIND_FWD, 2, true, true>(sp, st);
    return launch_scan<4, 4, KIND_FWD, 8, true, true>(sp, st);
}

cudaError_t launch_fused_ear_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st)
{
    if (ts.T == 16) return launch_scan<16, 8, KIND_FUSED, 2, true, true>(sp, st);
    return launch_scan<4, 4, KIND_FUSED, 8, true, true>(sp, st);
}

}  // namespace cawn
