// Launching the direct (register-resident) outer-step kernels: grid computation, the
// (variant, storage) dispatch and the launch shape chosen for each replica count.
// One translation unit per shape instantiates launch_outer_shape<ID, Q> (the kernels are many;
// compiling them side by side keeps the build short); the host code only calls it.
#pragma once
#include <type_traits>

#include "../../include/diloco.h"
#include "diloco_kernels.cuh"

namespace diloco {

// defined next to the C ABI: record the failing cudaError_t / count a successful launch
int cuda_fail(cudaError_t e);
void count_launch();

// The one (variant, theta storage) -> template-argument ladder: f is called with two
// std::integral_constant tags.
template <class F>
int dispatch_variant_storage(int var, int tk, F &&f) {
#define DILOCO_CASE(VAR_, TK_) \
  if (var == VAR_ && tk == TK_) return f(std::integral_constant<int, VAR_>{}, std::integral_constant<int, TK_>{});
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

inline int finish_launch() {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  count_launch();
  return DILOCO_OK;
}

// compile-time M: one column per thread (G = 1) or per G lanes of a warp
template <bool Q, int M, int G, int V, int NT, int MINB>
int launch_outer_m(int var, int tk, const OuterArgs &a, cudaStream_t s) {
  constexpr int CW = 32 / G;
  const long long warps = (a.P / V + CW - 1) / CW;
  long long blocks = (warps * 32 + NT - 1) / NT;
  if (blocks < 1) blocks = 1; // the last block also handles the P % V tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  return dispatch_variant_storage(var, tk, [&](auto var_, auto tk_) {
    outer_step_kernel<M, G, decltype(var_)::value, decltype(tk_)::value, V, NT, MINB, Q><<<(unsigned)blocks, NT, 0, s>>>(a);
    return finish_launch();
  });
}

// run-time M, replica axis over the warps of a block: R replicas per warp, V indices per column,
// two groups of columns per block where they fit 512 threads
template <bool Q, int V, int R>
int launch_outer_split(int var, int tk, const OuterArgs &a, cudaStream_t s) {
  const int warps = (a.M + R - 1) / R;
  if (warps > (R <= 4 ? 16 : 8)) return DILOCO_ERR_UNSUPPORTED;
  // 2 x 6 or 2 x 7 warps leave a quarter of the SM's thread slots empty; R = 8 blocks are register-bound
  const int groups = (R <= 4 && (warps <= 5 || warps == 8)) ? 2 : 1;
  long long blocks = ((a.P / V + 31) / 32 + groups - 1) / groups;
  if (blocks < 1) blocks = 1; // the last block also handles the P % V tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  const size_t smem = (size_t)groups * a.M * V * 32 * sizeof(float);
  OuterArgs b = a;
  b.groups = groups;
  b.wpg = warps;
  return dispatch_variant_storage(var, tk, [&](auto var_, auto tk_) {
    outer_step_split_kernel<decltype(var_)::value, decltype(tk_)::value, Q, V, R><<<(unsigned)blocks, 32 * warps * groups, smem, s>>>(b);
    return finish_launch();
  });
}

// M = 8 W as a chain of W warps per 16 columns
template <bool Q, int W, int NT, int MINB>
int launch_outer_chain(int var, int tk, const OuterArgs &a, cudaStream_t s) {
  constexpr int GROUPS = NT / (32 * W);
  const long long groups = (a.P / 4 + 15) / 16;
  long long blocks = (groups + GROUPS - 1) / GROUPS;
  if (blocks < 1) blocks = 1; // the last block also handles the P % 4 tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  return dispatch_variant_storage(var, tk, [&](auto var_, auto tk_) {
    outer_step_chain_kernel<W, decltype(var_)::value, decltype(tk_)::value, NT, MINB, Q><<<(unsigned)blocks, NT, 0, s>>>(a);
    return finish_launch();
  });
}

// the recording-only first outer steps of a delayed / eager run, any M
template <bool Q>
int launch_outer_first_steps(int var, int tk, const OuterArgs &a, cudaStream_t s) {
  constexpr int V = 4, NT = 128;
  long long blocks = (a.P / V + NT - 1) / NT;
  if (blocks < 1) blocks = 1;
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  if (var == VAR_STANDARD) return DILOCO_ERR_INVALID_ARG; // the standard step has no such phase
  return dispatch_variant_storage(var, tk, [&](auto var_, auto tk_) {
    constexpr int VAR = decltype(var_)::value == VAR_STANDARD ? VAR_DELAYED : decltype(var_)::value;
    outer_first_steps_kernel<VAR, decltype(tk_)::value, V, NT, Q><<<(unsigned)blocks, NT, 0, s>>>(a);
    return finish_launch();
  });
}

// Launch shapes, chosen by measurement on B200 under two rules: no register spills, and
// every warp-level access covers at least 128 contiguous bytes of a row (64-byte runs halved
// the bandwidth).
//   M <= 3          one thread per column, 128-bit accesses
// and a third found later: a block should touch at least 1 KB of every row it touches (512
// bytes per row and block cost 3 %: the DRAM pages it opens are used less fully).
//   M = 4, 8        replica axis split over 2 lanes of a warp (running sum passed by shuffle)
//   M = 16          two such warps chained (the running sum handed on through shared memory)
//   every other M   replica axis split over the warps of a block (through shared memory), 64
//                   registers: SPLIT_R2 two replicas per warp with 128-bit accesses up to M = 20
//                   (6.55-6.8 TB/s at M = 5 .. 20; one replica per warp measured 5.8-6.2 at
//                   M = 5, 6, 7 and 4.4-5.6 beyond), SPLIT_R4 four per warp with 64-bit accesses
//                   above (6.5 TB/s at M = 24, 32 against 6.1-6.3 for R2: blocks of more than 10
//                   warps wait too long at the barrier), SPLIT_R6 six per warp for M = 41 .. 48
//                   and SPLIT_R8 eight per warp above (blocks of at most 8 warps: M = 44 6.50
//                   against 5.85 TB/s, M = 64 6.44 against 5.9; seven per warp for M = 49 .. 56
//                   measured no better than eight: 6.0-6.3); two column
//                   groups per block where that keeps the SM's thread slots filled
// The ID names a translation unit: a replica count with its own kernels (1, 2, 3, 4, 8, 16), one
// of the split forms, or the first-steps form.
enum { SHAPE_FIRST_STEPS = 0, SHAPE_SPLIT_R4 = 1000, SHAPE_SPLIT_R2 = 1002, SHAPE_SPLIT_R8 = 1003, SHAPE_SPLIT_R6 = 1004 };

template <int ID, bool Q>
int launch_outer_shape(int var, int tk, const OuterArgs &a, cudaStream_t s) {
  if constexpr (ID == 1) return launch_outer_m<Q, 1, 1, 4, 128, 8>(var, tk, a, s);
  else if constexpr (ID == 2) return launch_outer_m<Q, 2, 1, 4, 128, 6>(var, tk, a, s);
  else if constexpr (ID == 3) return launch_outer_m<Q, 3, 1, 4, 128, 4>(var, tk, a, s);
  else if constexpr (ID == 4) return launch_outer_m<Q, 4, 2, 4, 256, 4>(var, tk, a, s);
  // M = 8: blocks of 256 threads (2 KB of every row per block) measured 0.7 % faster than 128
  else if constexpr (ID == 8) return launch_outer_m<Q, 8, 2, 4, 256, 2>(var, tk, a, s);
  // M = 16: two M = 8 warps chained per 16 columns, 4 such groups per block (1 KB of every row)
  else if constexpr (ID == 16) return launch_outer_chain<Q, 2, 256, 2>(var, tk, a, s);
  else if constexpr (ID == SHAPE_SPLIT_R4) return launch_outer_split<Q, 2, 4>(var, tk, a, s);
  else if constexpr (ID == SHAPE_SPLIT_R2) return launch_outer_split<Q, 4, 2>(var, tk, a, s);
  else if constexpr (ID == SHAPE_SPLIT_R8) return launch_outer_split<Q, 2, 8>(var, tk, a, s);
  else if constexpr (ID == SHAPE_SPLIT_R6) return launch_outer_split<Q, 2, 6>(var, tk, a, s);
  else return launch_outer_first_steps<Q>(var, tk, a, s);
}

// the translation units
#define DILOCO_FOR_EACH_SHAPE(X) X(0) X(1) X(2) X(3) X(4) X(8) X(1000) X(1002) X(1003) X(1004) X(16)

} // namespace diloco
