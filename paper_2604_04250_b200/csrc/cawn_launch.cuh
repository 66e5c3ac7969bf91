// Kernel launchers of libcawn.  The scan kernel's instantiations are spread over several
// translation units (cawn_launch_*.cu) so that they compile side by side; this header declares
// one launcher per family.  Each takes the tile shape the host picked and the filled parameters.
#pragma once
#include "cawn_scan.cuh"

namespace cawn {

// Tile shape of the scan kernels: T steps per warp, W warps.
struct TileShape { int T, W; };

cudaError_t launch_fwd_static(TileShape ts, const ScanParams &sp, cudaStream_t st);    // Cartesian forward
cudaError_t launch_fwd_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st);   // time-varying retention
cudaError_t launch_fwd_ear(TileShape ts, const ScanParams &sp, cudaStream_t st);       // Ear epilogue
cudaError_t launch_fused_plain(TileShape ts, const ScanParams &sp, cudaStream_t st);   // fused mixing path
cudaError_t launch_fused_ear(TileShape ts, const ScanParams &sp, cudaStream_t st);
cudaError_t launch_fwd_ear_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st);   // Ear epilogue + time-varying retention
cudaError_t launch_fused_ear_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st);
cudaError_t launch_fused_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st); // fused path, time-varying retention
// bf16 storage of the input (io & IO_IN_BF16) and / or the output (io & IO_OUT_BF16); io != 0
cudaError_t launch_fwd_bf16(TileShape ts, const ScanParams &sp, cudaStream_t st, int io);
cudaError_t launch_fused_bf16(TileShape ts, const ScanParams &sp, cudaStream_t st, int io);
// bf16 input and output together with time-varying retention (dyn) and / or the Ear epilogue (sp.ear_w)
cudaError_t launch_fwd_bf16_wide(TileShape ts, const ScanParams &sp, cudaStream_t st, bool dyn);
cudaError_t launch_fused_bf16_wide(TileShape ts, const ScanParams &sp, cudaStream_t st, bool dyn);
cudaError_t launch_bwd_static(TileShape ts, const ScanParams &sp, cudaStream_t st);    // reverse scan
cudaError_t launch_bwd_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st);
cudaError_t launch_mix_bwd(TileShape ts, const ScanParams &sp, cudaStream_t st);       // reverse scan + prelude backward
cudaError_t launch_mix_bwd_dynamic(TileShape ts, const ScanParams &sp, cudaStream_t st);

}  // namespace cawn
