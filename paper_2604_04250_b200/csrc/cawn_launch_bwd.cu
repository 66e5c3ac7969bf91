#include "cawn_launch_impl.cuh"

namespace cawn {

cudaError_t launch_bwd_static(TileShape ts, const ScanParams &sp, cudaStream_t st)
{
    if (ts.T == 8) return launch_scan<8, 8, KIND_BWD, 3>(sp, st);
    return launch_scan<4, 4, KIND_BWD, 8>(sp, st);
}

}  // namespace cawn
