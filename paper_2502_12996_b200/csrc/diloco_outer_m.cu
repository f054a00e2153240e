// The direct outer-step kernels of ONE translation unit, compiled once per -DDILOCO_M=<id>, in
// parallel, and linked into libdiloco.so.  id = a replica count with kernels of its own
// (1, 2, 3, 4, 8), a warp-split form (1000: four replicas per warp, 1002: two) or
// 0, the recording-only first steps.
#include "diloco_outer_launch.cuh"

#ifndef DILOCO_M
#error "compile with -DDILOCO_M=<translation unit id>"
#endif

namespace diloco {
template int launch_outer_shape<DILOCO_M, false>(int, int, const OuterArgs &, cudaStream_t);
template int launch_outer_shape<DILOCO_M, true>(int, int, const OuterArgs &, cudaStream_t);
} // namespace diloco
