#include "cawn_launch_impl.cuh"

namespace cawn {

cudaError_t launch_fused_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st)
{
    if (ts.T == 16) return launch_scan<16, 8, KIND_FUSED, 2, true>(sp, st);
    return launch_scan<4, 4, KIND_FUSED, 8, true>(sp, st);
}

}  // namespace cawn
