#include "cawn_launch_impl.cuh"

namespace cawn {

cudaError_t launch_mix_bwd_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st)
{
    if (ts.T == 8) return launch_scan<8, 8, KIND_MIXBWD, 2, true>(sp, st);
    return launch_scan<4, 4, KIND_MIXBWD, 8, true>(sp, st);
}

}  // namespace cawn
