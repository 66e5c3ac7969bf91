#include "cawn_launch_impl.cuh"

namespace cawn {

cudaError_t launch_fused_bf16(TileShape ts, const ScanParams &sp, cudaStream_t st, int io)
{
    switch (io) {
    case IO_IN_BF16: return launch_scan_io<KIND_FUSED, IO_IN_BF16>(ts, sp, st);
    case IO_OUT_BF16: return launch_scan_io<KIND_FUSED, IO_OUT_BF16>(ts, sp, st);
    case IO_IN_BF16 | IO_OUT_BF16: return launch_scan_io<KIND_FUSED, IO_IN_BF16 | IO_OUT_BF16>(ts, sp, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace cawn
