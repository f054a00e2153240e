// The direct outer-step kernels of ONE replica count: compiled once per -DDILOCO_M=<M>
// (0 = the runtime-M kernel), in parallel, and linked into libdiloco.so.
#include "diloco_outer_launch.cuh"

#ifndef DILOCO_M
#error "compile with -DDILOCO_M=<replica count>"
#endif

namespace diloco {
template int launch_outer_shape<DILOCO_M, false>(int, int, bool, const OuterArgs &, cudaStream_t);
template int launch_outer_shape<DILOCO_M, true>(int, int, bool, const OuterArgs &, cudaStream_t);
} // namespace diloco
