#include "cawn_launch_impl.cuh"

namespace cawn {

cudaError_t launch_fwd_static(TileShape ts, const ScanParams &sp, cudaStream_t st)
{
    // A call whose CTAs are all resident at once (three per SM), with the input vouched for and no
    // mask: the form that runs its gate pass before it waits for the previous launch.
    if (ts.T == 16 && sp.mask == nullptr && sp.early_loads != 0 && sp.stagger_group > 0 &&
        (long long)sp.G * sp.B * sp.K <= (long long)sp.stagger_group * sp.stagger_slots)
        return launch_scan<16, 8, KIND_FWD, 3, false, false, IO_F32, false, true>(sp, st);
    // the long-call shape exists with and without the gate-mask output compiled in
    if (ts.T == 16 && sp.mask == nullptr) return launch_scan<16, 8, KIND_FWD, 3, false, false, IO_F32, false>(sp, st);
    if (ts.T == 16) return launch_scan<16, 8, KIND_FWD, 3>(sp, st);
    return launch_scan<4, 4, KIND_FWD, 8>(sp, st);
}

}  // namespace cawn
