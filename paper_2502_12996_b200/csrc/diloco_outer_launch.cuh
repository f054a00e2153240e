// Launching the direct (register-resident) outer-step kernels: grid computation, the
// (variant, storage, first-step) dispatch and the launch shape chosen for each replica count.
// One translation unit per replica count instantiates launch_outer_shape<M, Q> (the kernels
// are many; compiling them side by side keeps the build short); the host code only calls it.
#pragma once
#include "../../include/diloco.h"
#include "diloco_kernels.cuh"

namespace diloco {

// defined next to the C ABI: record the failing cudaError_t / count a successful launch
int cuda_fail(cudaError_t e);
void count_launch();

template <int M, int G, int VAR, int TK, bool BOOT, int V, int NT, int MINB, bool Q>
int launch_outer_t(const OuterArgs &a, cudaStream_t s) {
  constexpr int CW = 32 / G;
  const long long nvec = a.P / V;
  const long long warps = (nvec + CW - 1) / CW;
  long long blocks = (warps * 32 + NT - 1) / NT;
  if (blocks < 1) blocks = 1; // the last block also handles the P % V tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  outer_step_kernel<M, G, VAR, TK, BOOT, V, NT, MINB, Q><<<(unsigned)blocks, NT, 0, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  count_launch();
  return DILOCO_OK;
}

template <bool Q, int M, int G, int V, int NT, int MINB>
int launch_outer_m(int var, int tk, bool boot, const OuterArgs &a, cudaStream_t s) {
#define DILOCO_CASE(VAR_, TK_)                                                                           \
  if (var == VAR_ && tk == TK_) {                                                                        \
    if constexpr (VAR_ != VAR_STANDARD) {                                                                \
      if (boot) return launch_outer_t<M, G, VAR_, TK_, true, V, NT, MINB, Q>(a, s);                      \
    }                                                                                                    \
    return launch_outer_t<M, G, VAR_, TK_, false, V, NT, MINB, Q>(a, s);                                  \
  }
  DILOCO_CASE(VAR_STANDARD, TK_F32)
  DILOCO_CASE(VAR_STANDARD, TK_BF16)
  DILOCO_CASE(VAR_STANDARD, TK_MASTER_BF16)
  DILOCO_CASE(VAR_DELAYED, TK_F32)
  DILOCO_CASE(VAR_DELAYED, TK_BF16)
  DILOCO_CASE(VAR_DELAYED, TK_MASTER_BF16)
  DILOCO_CASE(VAR_EAGER, TK_F32)
  DILOCO_CASE(VAR_EAGER, TK_BF16)
  DILOCO_CASE(VAR_EAGER, TK_MASTER_BF16)
#undef DILOCO_CASE
  return DILOCO_ERR_INVALID_ARG;
}

// Launch shapes per M (lane groups G, vector width V, threads NT, min resident blocks MINB),
// chosen by measurement on B200 under two rules: no register spills, and every warp-level
// access covers at least 128 contiguous bytes of a row (64-byte runs halved the bandwidth).
// M <= 3: one thread per column.  M = 4, 8, 16: the replica axis is split over G lanes.
// (M = 4: 6.70 TB/s, M = 8: 6.77, M = 16: 6.45, M = 2: 6.65 in the microbenchmark.)
// warp-split form (one warp per 4 replicas): blocks of 8 M threads, 32 columns each
template <int VAR, int TK, bool BOOT, bool Q>
int launch_outer_cta_t(const OuterArgs &a, cudaStream_t s) {
  constexpr int V = 2; // 64-bit accesses, 64 registers per thread, 1024 threads per SM
  long long blocks = (a.P / V + 31) / 32;
  if (blocks < 1) blocks = 1; // the last block also handles the P % V tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  const size_t smem = (size_t)a.M * V * 32 * sizeof(float);
  outer_step_cta_kernel<VAR, TK, BOOT, Q, V><<<(unsigned)blocks, 8 * a.M, smem, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  count_launch();
  return DILOCO_OK;
}

// one warp per replica, any M <= 32 at run time
template <int VAR, int TK, bool BOOT, bool Q>
int launch_outer_wpr_t(const OuterArgs &a, cudaStream_t s) {
  constexpr int V = 4;
  long long blocks = (a.P / V + 31) / 32;
  if (blocks < 1) blocks = 1; // the last block also handles the P % V tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  const size_t smem = (size_t)a.M * V * 32 * sizeof(float);
  outer_step_warp_per_replica_kernel<VAR, TK, BOOT, Q, V><<<(unsigned)blocks, 32 * a.M, smem, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  count_launch();
  return DILOCO_OK;
}

template <bool Q>
int launch_outer_wpr(int var, int tk, bool boot, const OuterArgs &a, cudaStream_t s) {
#define DILOCO_CASE(VAR_, TK_)                                                              \
  if (var == VAR_ && tk == TK_) {                                                           \
    if constexpr (VAR_ != VAR_STANDARD) {                                                   \
      if (boot) return launch_outer_wpr_t<VAR_, TK_, true, Q>(a, s);                        \
    }                                                                                       \
    return launch_outer_wpr_t<VAR_, TK_, false, Q>(a, s);                                   \
  }
  DILOCO_CASE(VAR_STANDARD, TK_F32)
  DILOCO_CASE(VAR_STANDARD, TK_BF16)
  DILOCO_CASE(VAR_STANDARD, TK_MASTER_BF16)
  DILOCO_CASE(VAR_DELAYED, TK_F32)
  DILOCO_CASE(VAR_DELAYED, TK_BF16)
  DILOCO_CASE(VAR_DELAYED, TK_MASTER_BF16)
  DILOCO_CASE(VAR_EAGER, TK_F32)
  DILOCO_CASE(VAR_EAGER, TK_BF16)
  DILOCO_CASE(VAR_EAGER, TK_MASTER_BF16)
#undef DILOCO_CASE
  return DILOCO_ERR_INVALID_ARG;
}

template <bool Q>
int launch_outer_cta(int var, int tk, bool boot, const OuterArgs &a, cudaStream_t s) {
#define DILOCO_CASE(VAR_, TK_)                                                              \
  if (var == VAR_ && tk == TK_) {                                                           \
    if constexpr (VAR_ != VAR_STANDARD) {                                                   \
      if (boot) return launch_outer_cta_t<VAR_, TK_, true, Q>(a, s);                        \
    }                                                                                       \
    return launch_outer_cta_t<VAR_, TK_, false, Q>(a, s);                                   \
  }
  DILOCO_CASE(VAR_STANDARD, TK_F32)
  DILOCO_CASE(VAR_STANDARD, TK_BF16)
  DILOCO_CASE(VAR_STANDARD, TK_MASTER_BF16)
  DILOCO_CASE(VAR_DELAYED, TK_F32)
  DILOCO_CASE(VAR_DELAYED, TK_BF16)
  DILOCO_CASE(VAR_DELAYED, TK_MASTER_BF16)
  DILOCO_CASE(VAR_EAGER, TK_F32)
  DILOCO_CASE(VAR_EAGER, TK_BF16)
  DILOCO_CASE(VAR_EAGER, TK_MASTER_BF16)
#undef DILOCO_CASE
  return DILOCO_ERR_INVALID_ARG;
}

// Launch shapes, chosen by measurement on B200 under two rules: no register spills, and
// every warp-level access covers at least 128 contiguous bytes of a row.
//   M <= 3          one thread per column, 128-bit accesses
//   M = 4, 8        replica axis split over 2 lanes of a warp (running sum passed by shuffle)
//   M = 12, 16 .. 64 (multiples of 4): replica axis split over the warps of a block (through
//                   shared memory), 64-bit accesses, 64 registers, 1024 threads per SM:
//                   6.5 TB/s at M = 12, 16, 24, 32, 64 against 6.32 / 6.35 / 5.19 at M = 16 /
//                   32 / 64 for a 4-lane split or the two-sweep form
//   M = 5, 6, 7     one warp per replica: 6.57 / 6.44 / 6.11 TB/s against 6.02 / 5.96 / 5.84
//   any other M     two sweeps over the replicas in one thread
// The template argument names a translation unit: a replica count with its own kernels, or
// one of the three run-time forms.
enum { SHAPE_TWO_SWEEP = 0, SHAPE_WARP_SPLIT = 1000, SHAPE_WARP_PER_REPLICA = 1001 };

template <int M, bool Q>
int launch_outer_shape(int var, int tk, bool boot, const OuterArgs &a, cudaStream_t s) {
  if constexpr (M == 1) return launch_outer_m<Q, 1, 1, 4, 128, 8>(var, tk, boot, a, s);
  else if constexpr (M == 2) return launch_outer_m<Q, 2, 1, 4, 128, 6>(var, tk, boot, a, s);
  else if constexpr (M == 3) return launch_outer_m<Q, 3, 1, 4, 128, 4>(var, tk, boot, a, s);
  else if constexpr (M == 4) return launch_outer_m<Q, 4, 2, 4, 256, 4>(var, tk, boot, a, s);
  // M = 8: 5 resident blocks (96 registers) measured 4 % faster than 4; the quantised eager
  // form needs ~100 registers and would spill under that cap
  else if constexpr (M == 8) return launch_outer_m<Q, 8, 2, 4, 128, Q ? 4 : 5>(var, tk, boot, a, s);
  else if constexpr (M == SHAPE_WARP_SPLIT) return launch_outer_cta<Q>(var, tk, boot, a, s);
  else if constexpr (M == SHAPE_WARP_PER_REPLICA) return launch_outer_wpr<Q>(var, tk, boot, a, s);
  else return launch_outer_m<Q, 0, 1, 4, 128, 4>(var, tk, boot, a, s);
}

// the translation units
#define DILOCO_FOR_EACH_M(X) X(0) X(1) X(2) X(3) X(4) X(8) X(1000) X(1001)

} // namespace diloco
