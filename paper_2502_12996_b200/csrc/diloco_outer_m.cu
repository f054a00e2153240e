// The direct outer-step kernels of ONE translation unit, compiled once per -DDILOCO_M=<id>, in
// parallel, and linked into libdiloco.so.  id = a replica count with kernels of its own
// (1, 2, 3, 4, 8) or a run-time form (0 two sweeps, 1000 warp split, 1001 warp per replica).
#include "diloco_outer_launch.cuh"

#ifndef DILOCO_M
#error "compile with -DDILOCO_M=<translation unit id>"
#endif

namespace diloco {
template int launch_outer_shape<DILOCO_M, false>(int, int, bool, const OuterArgs &, cudaStream_t);
template int launch_outer_shape<DILOCO_M, true>(int, int, bool, const OuterArgs &, cudaStream_t);
} // namespace diloco
