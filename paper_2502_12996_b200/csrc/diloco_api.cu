// Host side of libdiloco: the C ABI declared in include/diloco.h.  Validates arguments,
// keeps the per-state bookkeeping (counters, have_prev) and launches the kernels of
// diloco_kernels.cuh / diloco_bulk.cuh on the caller's stream.  No device allocation, no
// device synchronisation (except diloco_check_device_status), no CPU fallback.
#include "../../include/diloco.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "diloco_bulk.cuh"
#include "diloco_kernels.cuh"
#include "diloco_outer_launch.cuh"
#include "diloco_tensor.cuh"
#include "diloco_worker.cuh"

using namespace diloco;

// launch_outer_shape<ID, Q> is instantiated in diloco_outer_m.cu, once per shape
#define DILOCO_EXTERN(ID_)                                                                                 \
  extern template int diloco::launch_outer_shape<ID_, false>(int, int, const OuterArgs &, cudaStream_t); \
  extern template int diloco::launch_outer_shape<ID_, true>(int, int, const OuterArgs &, cudaStream_t);
DILOCO_FOR_EACH_SHAPE(DILOCO_EXTERN)
#undef DILOCO_EXTERN

// One fragment of the parameter axis with its own outer-step schedule (Streaming DiLoCo applies
// the outer step to different parts of the model at different times, Section 3).
struct Fragment {
  int64_t offset, len;
  int64_t outer_step; // outer steps this fragment has taken: selects its slot of the generation ring
  int32_t have_prev;  // generations of its recorded gradients that are valid, 0 .. overlap_steps
};

struct diloco_state {
  diloco_config_t cfg;
  diloco_buffers_t buf;
  int device;
  int sm_count;
  int64_t inner_step;
  int64_t outer_step;
  int32_t have_prev;
  std::vector<Fragment> frags;
  const void *checked[8]; // per-call buffers already seen to be memory of this device (H calls per phase
  int checked_next;       // pass the same gradient / send / receive buffers again and again)
  uint64_t wait_limit_ns;  // bound of every device-side wait of the bulk form
  uint32_t test_extra_tx;  // bytes its barriers over-expect: 0 except in the give-up test
  std::vector<cudaEvent_t> events; // host-path chunk events, created on first use
  cudaEvent_t last_d2h;
};

// Scratch of diloco_outer_quantized_static: part of the library image, so every GPU that loads
// the library holds these 64 words (256 bytes) until the process exits.
constexpr uint64_t kDefaultWaitLimitNs = 1000000000ull; // 1 s per device-side wait
constexpr int kStaticScratchWords = DILOCO_MAX_M;
static __device__ __align__(256) unsigned g_static_scratch[kStaticScratchWords];

namespace {
std::atomic<int64_t> g_launches{0};
std::atomic<int32_t> g_last_cuda_error{0};
} // namespace

int diloco::cuda_fail(cudaError_t e) {
  g_last_cuda_error.store((int32_t)e);
  return DILOCO_ERR_CUDA;
}
void diloco::count_launch() { g_launches.fetch_add(1); }

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t theta_elt(int32_t kind) { return kind == DILOCO_THETA_F32 ? 4 : 2; }

int validate_config(const diloco_config_t *c) {
  if (!c) return DILOCO_ERR_INVALID_ARG;
  if (c->M < 1 || c->P < 1 || c->stride < c->P || c->H < 0) return DILOCO_ERR_INVALID_ARG;
  if (c->M > DILOCO_MAX_M) return DILOCO_ERR_UNSUPPORTED;
  if (c->theta_kind < DILOCO_THETA_F32 || c->theta_kind > DILOCO_THETA_MASTER_BF16) return DILOCO_ERR_INVALID_ARG;
  if (c->grad_kind < DILOCO_GRAD_F32 || c->grad_kind > DILOCO_GRAD_BF16) return DILOCO_ERR_INVALID_ARG;
  if (c->impl < DILOCO_IMPL_AUTO || c->impl > DILOCO_IMPL_TENSOR_T64) return DILOCO_ERR_INVALID_ARG;
  if (!(c->outer_momentum >= 0.f && c->outer_momentum < 1.f)) return DILOCO_ERR_INVALID_ARG;
  if (!std::isfinite(c->outer_lr)) return DILOCO_ERR_INVALID_ARG;
  if (!(c->beta1 >= 0.f && c->beta1 < 1.f) || !(c->beta2 >= 0.f && c->beta2 < 1.f)) return DILOCO_ERR_INVALID_ARG;
  if (!(c->eps >= 0.f) || !(c->weight_decay >= 0.f)) return DILOCO_ERR_INVALID_ARG;
  if (c->overlap_steps < 1) return DILOCO_ERR_INVALID_ARG;
  if (c->overlap_steps > DILOCO_MAX_OVERLAP) return DILOCO_ERR_UNSUPPORTED;
  if (c->have_prev < 0 || c->have_prev > c->overlap_steps) return DILOCO_ERR_INVALID_ARG;
  if (c->shared_outer_state != 0 && c->shared_outer_state != 1) return DILOCO_ERR_INVALID_ARG;
  // 128-byte rows for every dtype in use
  if ((c->stride * 4) % 128 != 0) return DILOCO_ERR_MISALIGNED;
  if (c->theta_kind != DILOCO_THETA_F32 && (c->stride * 2) % 128 != 0) return DILOCO_ERR_MISALIGNED;
  return DILOCO_OK;
}

// A pointer the kernels will dereference must be device (or managed) memory of `device`;
// a host pointer here would otherwise surface as an illegal-address fault inside a kernel.
int check_device_pointer(const void *p, int device) {
  cudaPointerAttributes at;
  cudaError_t e = cudaPointerGetAttributes(&at, p);
  if (e != cudaSuccess) {
    cudaGetLastError(); // clear the sticky-less error state of the query
    return DILOCO_ERR_INVALID_ARG;
  }
  if (at.type == cudaMemoryTypeManaged) return DILOCO_OK;
  if (at.type != cudaMemoryTypeDevice || at.device != device) return DILOCO_ERR_INVALID_ARG;
  return DILOCO_OK;
}

// Per-call buffers (gradients, send / receive buffers) are checked once per address and state:
// a training loop passes the same few buffers at every step, and the attribute query is a
// driver call on the launch path.
int check_call_pointer(diloco_state *st, const void *p) {
  for (const void *q : st->checked)
    if (q == p) return DILOCO_OK;
  const int rc = check_device_pointer(p, st->device);
  if (rc != DILOCO_OK) return rc;
  st->checked[st->checked_next] = p;
  st->checked_next = (st->checked_next + 1) % 8;
  return DILOCO_OK;
}

int validate_buffers(const diloco_config_t *c, const diloco_buffers_t *b) {
  if (!b) return DILOCO_ERR_INVALID_ARG;
  if (!b->theta || !b->start || !b->outer_mom) return DILOCO_ERR_INVALID_ARG;
  if (c->theta_kind == DILOCO_THETA_MASTER_BF16 && !b->master) return DILOCO_ERR_INVALID_ARG;
  if ((b->adam_m == nullptr) != (b->adam_v == nullptr)) return DILOCO_ERR_INVALID_ARG;
  const void *all[] = {b->theta, b->master, b->start, b->delta_prev_local, b->delta_prev_avg,
                       b->outer_mom, b->adam_m, b->adam_v};
  for (const void *p : all)
    if (p && !aligned16(p)) return DILOCO_ERR_MISALIGNED;
  if (b->device_status && (reinterpret_cast<uintptr_t>(b->device_status) & 3u)) return DILOCO_ERR_MISALIGNED;
  if (b->comm_scratch && (reinterpret_cast<uintptr_t>(b->comm_scratch) & 3u)) return DILOCO_ERR_MISALIGNED;
  return DILOCO_OK;
}

// Which warp-split form serves a replica count that has no compile-time shape (see
// diloco_outer_launch.cuh); `forced` (a state's impl field, for measurements) overrides it.
int split_shape_for(int M, int forced) {
  if (forced == DILOCO_IMPL_SPLIT_R2 && M <= 32) return SHAPE_SPLIT_R2; // 16 warps per block at most
  if (forced == DILOCO_IMPL_SPLIT_R4) return SHAPE_SPLIT_R4;
  if (M <= 20) return SHAPE_SPLIT_R2;
  if (M <= 40) return SHAPE_SPLIT_R4;
  return M <= 48 ? SHAPE_SPLIT_R6 : SHAPE_SPLIT_R8; // blocks of at most 8 warps beyond M = 40
}

template <bool Q>
int launch_outer_direct(const diloco_state *st, int var, bool boot, const OuterArgs &a, cudaStream_t s) {
  const int tk = st->cfg.theta_kind, M = st->cfg.M, impl = st->cfg.impl;
  if (boot) return launch_outer_shape<SHAPE_FIRST_STEPS, Q>(var, tk, a, s);
  const bool forced_split = impl == DILOCO_IMPL_SPLIT_R2 || impl == DILOCO_IMPL_SPLIT_R4;
  if (!forced_split) {
    switch (M) {
      case 1: return launch_outer_shape<1, Q>(var, tk, a, s);
      case 2: return launch_outer_shape<2, Q>(var, tk, a, s);
      case 3: return launch_outer_shape<3, Q>(var, tk, a, s);
      case 4: return launch_outer_shape<4, Q>(var, tk, a, s);
      case 8: return launch_outer_shape<8, Q>(var, tk, a, s);
      case 16: return launch_outer_shape<16, Q>(var, tk, a, s);
      default: break;
    }
  }
  switch (split_shape_for(M, impl)) {
    case SHAPE_SPLIT_R2: return launch_outer_shape<SHAPE_SPLIT_R2, Q>(var, tk, a, s);
    case SHAPE_SPLIT_R8: return launch_outer_shape<SHAPE_SPLIT_R8, Q>(var, tk, a, s);
    case SHAPE_SPLIT_R6: return launch_outer_shape<SHAPE_SPLIT_R6, Q>(var, tk, a, s);
    default: return launch_outer_shape<SHAPE_SPLIT_R4, Q>(var, tk, a, s);
  }
}

// Delayed and eager steps consume the gradients recorded overlap_steps outer steps ago: the
// state keeps that many generations in a ring, slot = outer-step counter mod overlap_steps,
// and the step that reads a slot overwrites it with the new generation.  Until every slot
// has been written once (have_prev < overlap_steps) there is nothing to receive yet.
inline int ring_slot(const diloco_state *st) { return (int)(st->outer_step % st->cfg.overlap_steps); }
inline bool is_first_steps(const diloco_state *st, int var) {
  return var != VAR_STANDARD && st->have_prev < st->cfg.overlap_steps;
}
inline void advance(diloco_state *st, int var) {
  if (var != VAR_STANDARD && st->have_prev < st->cfg.overlap_steps) st->have_prev += 1;
  st->outer_step += 1;
}

// The buffers live on the device that was current at diloco_state_init; launching from
// another current device would run the kernel where those pointers mean nothing.
int check_device(const diloco_state *st) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  return dev == st->device ? DILOCO_OK : DILOCO_ERR_BAD_STATE;
}

// variant-specific buffer requirements, and the state's device must be current
int check_variant(const diloco_state *st, int var) {
  if (var < VAR_STANDARD || var > VAR_EAGER) return DILOCO_ERR_INVALID_ARG;
  int rc = check_device(st);
  if (rc != DILOCO_OK) return rc;
  // one shared copy of s and b exists only for the standard step: the others let the replicas' copies differ
  if (st->cfg.shared_outer_state && var != VAR_STANDARD) return DILOCO_ERR_BAD_STATE;
  if (var != VAR_STANDARD && !st->buf.delta_prev_avg) return DILOCO_ERR_BAD_STATE;
  if (var == VAR_EAGER && !st->buf.delta_prev_local) return DILOCO_ERR_BAD_STATE;
  return DILOCO_OK;
}

OuterArgs outer_args(const diloco_state *st, int64_t offset, int64_t len, int ring = -1) {
  OuterArgs a;
  const diloco_buffers_t &b = st->buf;
  a.theta = b.theta ? static_cast<char *>(b.theta) + (size_t)offset * theta_elt(st->cfg.theta_kind) : nullptr;
  a.master = b.master ? b.master + offset : nullptr;
  a.start = b.start + offset;
  const size_t slot = (size_t)(ring < 0 ? ring_slot(st) : ring);
  a.dpl = b.delta_prev_local ? b.delta_prev_local + slot * (size_t)st->cfg.M * (size_t)st->cfg.stride + offset : nullptr;
  a.dpa = b.delta_prev_avg ? b.delta_prev_avg + slot * (size_t)st->cfg.stride + offset : nullptr;
  a.mom = b.outer_mom + offset;
  a.P = len;
  a.stride = st->cfg.stride;
  a.eta = st->cfg.outer_lr;
  a.mu = st->cfg.outer_momentum;
  a.fM = (float)st->cfg.M;
  a.M = st->cfg.M;
  a.groups = 1;
  a.wpg = 0;
  a.amax = nullptr;
  a.fmt_max = 0.f;
  a.comm = COMM_F32;
  a.man_bits = a.emin = a.bias = 0;
  return a;
}

template <int TK>
int launch_amax_t(const diloco_state *st, const OuterArgs &a, unsigned *amax, cudaStream_t s) {
  constexpr int NT = 256, U = 4;
  const long long nvec = a.P / 4;
  long long blocks = (nvec + (long long)NT * U - 1) / ((long long)NT * U);
  const long long cap = (long long)st->sm_count * 8; // grid-stride: few atomics, every SM busy
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  dim3 grid((unsigned)blocks, (unsigned)st->cfg.M);
  delta_amax_kernel<TK, NT, U><<<grid, NT, 0, s>>>(a, amax);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1);
  return DILOCO_OK;
}

// One quantised outer step on indices [0, P): (EXMY only) zero the per-replica maxima and
// reduce max |Delta_m| into `scratch`, then the fused step with the wire rounding in line 8.
int launch_outer_quantized(diloco_state *st, int var, bool boot, int comm, int X, int Y, unsigned *scratch,
                           cudaStream_t s, int64_t offset = 0, int64_t len = -1, int ring = -1) {
  OuterArgs a = outer_args(st, offset, len < 0 ? st->cfg.P : len, ring);
  a.comm = comm;
  if (comm == COMM_EXMY) {
    a.bias = (1 << (X - 1)) - 1;
    a.emin = 1 - a.bias;
    a.man_bits = Y;
    a.fmt_max = std::ldexp(2.0f - std::ldexp(1.0f, -Y), (1 << X) - 1 - a.bias);
    a.amax = scratch;
    cudaError_t e = cudaMemsetAsync(scratch, 0, sizeof(unsigned) * (size_t)st->cfg.M, s);
    if (e != cudaSuccess) return cuda_fail(e);
    int rc;
    switch (st->cfg.theta_kind) {
      case TK_F32: rc = launch_amax_t<TK_F32>(st, a, scratch, s); break;
      case TK_BF16: rc = launch_amax_t<TK_BF16>(st, a, scratch, s); break;
      default: rc = launch_amax_t<TK_MASTER_BF16>(st, a, scratch, s); break;
    }
    if (rc != DILOCO_OK) return rc;
  }
  return launch_outer_direct<true>(st, var, boot, a, s);
}

// Bulk (TMA-staged) form: one CTA ring per SM slot, grid capped by the tile count.
template <int M, int VAR, int TK, int T, int S, int NT>
int launch_bulk_t(const diloco_state *st, const OuterArgs &a, cudaStream_t s) {
  auto k = outer_step_bulk_kernel<M, VAR, TK, T, S, NT>;
  constexpr int smem = S * BulkStage<M, VAR, TK, T>::kBytes;
  static_assert(smem <= 227 * 1024, "stage ring exceeds the shared memory of one SM");
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, NT, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  if (per_sm < 1) per_sm = 1;
  long long grid = (long long)per_sm * st->sm_count;
  const long long ntiles = a.P / T;
  if (grid > ntiles) grid = ntiles;
  k<<<(unsigned)grid, NT, smem, s>>>(a, st->buf.device_status, (unsigned long long)st->wait_limit_ns, st->test_extra_tx);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1);
  return DILOCO_OK;
}

template <int M, int T, int S, int NT>
int launch_bulk_m(const diloco_state *st, int var, int tk, const OuterArgs &a, cudaStream_t s) {
  return dispatch_variant_storage(var, tk, [&](auto var_, auto tk_) {
    return launch_bulk_t<M, decltype(var_)::value, decltype(tk_)::value, T, S, NT>(st, a, s);
  });
}

// ---- tensor (2-D TMA) form ---------------------------------------------------------------------
// cuTensorMapEncodeTiled is a driver entry point; it is looked up through the runtime so that the
// library needs no link-time dependency on the driver library.
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  });
  return fn;
}

// fp32 tensor [rows, cols] with row pitch `pitch` elements, boxes of [rows, T]
int encode_rows(CUtensorMap *map, float *base, int64_t cols, int rows, int64_t pitch, int T) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return DILOCO_ERR_UNSUPPORTED;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)T, (cuuint32_t)rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? DILOCO_OK : DILOCO_ERR_CUDA;
}

template <int VAR, int T>
int launch_tensor_t(const diloco_state *st, const OuterArgs &whole, cudaStream_t s) {
  constexpr int NT = 256;
  auto k = outer_step_tensor_kernel<VAR, T, NT>;
  const int M = st->cfg.M;
  const size_t stage = (size_t)tensor_rows_per_stage<VAR>(M) * T * sizeof(float);
  const size_t budget = 227 * 1024 - 1024; // dynamic shared memory of one CTA, static part left out
  int stages = (int)(budget / stage);
  if (stages > kTensorMaxStages) stages = kTensorMaxStages;
  if (stages < 3) return DILOCO_ERR_UNSUPPORTED;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(stage * stages));
  if (e != cudaSuccess) return cuda_fail(e);
  // TMA coordinates are 32-bit: segments of at most 2^30 columns, each with tensor maps of its own
  const long long seg = 1ll << 30;
  for (long long off = 0; off < whole.P; off += seg) {
    OuterArgs a = whole;
    a.P = whole.P - off < seg ? whole.P - off : seg;
    a.theta = reinterpret_cast<float *>(whole.theta) + off;
    a.start = whole.start + off;
    a.mom = whole.mom + off;
    a.dpl = whole.dpl ? whole.dpl + off : nullptr;
    a.dpa = whole.dpa ? whole.dpa + off : nullptr;
    // the tensors end at a multiple of 4 columns (16 bytes: the unit in which stores are clipped);
    // the kernel's last CTA does the remaining P % 4 indices itself
    const long long cols = a.P & ~3ll;
    TensorMaps maps;
    int rc = DILOCO_OK;
    if (cols > 0) {
      rc = encode_rows(&maps.theta, reinterpret_cast<float *>(a.theta), cols, M, a.stride, T);
      if (rc == DILOCO_OK) rc = encode_rows(&maps.start, a.start, cols, M, a.stride, T);
      if (rc == DILOCO_OK) rc = encode_rows(&maps.mom, a.mom, cols, M, a.stride, T);
      if (rc == DILOCO_OK && VAR == VAR_EAGER) rc = encode_rows(&maps.dpl, a.dpl, cols, M, a.stride, T);
      if (rc == DILOCO_OK && VAR != VAR_STANDARD) rc = encode_rows(&maps.dpa, a.dpa, cols, 1, a.stride, T);
    } else {
      std::memset(&maps, 0, sizeof(maps)); // fewer than 4 indices: no tile, the maps are never used
    }
    if (rc != DILOCO_OK) return rc;
    long long grid = st->sm_count;
    const long long ntiles = (cols + T - 1) / T;
    if (grid > ntiles) grid = ntiles;
    if (grid < 1) grid = 1;
    k<<<(unsigned)grid, NT, stage * stages, s>>>(maps, a, st->buf.device_status, stages, (unsigned long long)st->wait_limit_ns,
                                                 st->test_extra_tx);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    g_launches.fetch_add(1);
  }
  return DILOCO_OK;
}

template <int T>
int launch_tensor(const diloco_state *st, int var, const OuterArgs &a, cudaStream_t s) {
  if (var == VAR_STANDARD) return launch_tensor_t<VAR_STANDARD, T>(st, a, s);
  if (var == VAR_DELAYED) return launch_tensor_t<VAR_DELAYED, T>(st, a, s);
  return launch_tensor_t<VAR_EAGER, T>(st, a, s);
}

template <int TK, int U>
int launch_standard_shared_u(const OuterArgs &a, cudaStream_t s) {
  constexpr int NT = 256;
  long long blocks = (a.P / 4 + (long long)NT * U - 1) / ((long long)NT * U);
  if (blocks < 1) blocks = 1; // the last block also handles the P % 4 tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  outer_standard_shared_kernel<TK, NT, U><<<(unsigned)blocks, NT, 0, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1);
  return DILOCO_OK;
}

template <int TK>
int launch_standard_shared_t(const OuterArgs &a, cudaStream_t s) {
  return a.M <= 4 ? launch_standard_shared_u<TK, 2>(a, s) : launch_standard_shared_u<TK, 1>(a, s);
}

int launch_outer(diloco_state *st, int var, bool boot, int64_t offset, int64_t len, cudaStream_t s, int ring = -1) {
  OuterArgs a = outer_args(st, offset, len, ring);
  if (st->cfg.shared_outer_state) { // check_variant has let only the standard step through
    switch (st->cfg.theta_kind) {
      case TK_F32: return launch_standard_shared_t<TK_F32>(a, s);
      case TK_BF16: return launch_standard_shared_t<TK_BF16>(a, s);
      default: return launch_standard_shared_t<TK_MASTER_BF16>(a, s);
    }
  }
  // The tensor form: fp32 theta, needs the status word for its bounded waits; falls back to the
  // direct form where a stage ring of three tiles does not fit shared memory.
  if (st->cfg.impl >= DILOCO_IMPL_TENSOR_T256 && st->cfg.impl <= DILOCO_IMPL_TENSOR_T64 && !boot &&
      st->buf.device_status && st->cfg.theta_kind == DILOCO_THETA_F32) {
    int rc = DILOCO_ERR_UNSUPPORTED;
    switch (st->cfg.impl) {
      case DILOCO_IMPL_TENSOR_T256: rc = launch_tensor<256>(st, var, a, s); break;
      case DILOCO_IMPL_TENSOR_T128: rc = launch_tensor<128>(st, var, a, s); break;
      default: rc = launch_tensor<64>(st, var, a, s); break;
    }
    if (rc != DILOCO_ERR_UNSUPPORTED) return rc;
  }
  // The bulk form exists for M = 2 and M = 4 only, needs the status word for its bounded
  // waits and at least one full tile; everything else (and AUTO) takes the direct form,
  // which measured faster at every M.
  if (st->cfg.impl == DILOCO_IMPL_BULK && !boot && st->buf.device_status) {
    if (st->cfg.M == 2 && len >= 1024) return launch_bulk_m<2, 1024, 3, 256>(st, var, st->cfg.theta_kind, a, s);
    if (st->cfg.M == 4 && len >= 512) return launch_bulk_m<4, 512, 3, 128>(st, var, st->cfg.theta_kind, a, s);
  }
  return launch_outer_direct<false>(st, var, boot, a, s);
}

int outer_whole(diloco_state *st, int var, void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  int rc = check_variant(st, var);
  if (rc != DILOCO_OK) return rc;
  rc = launch_outer(st, var, is_first_steps(st, var), 0, st->cfg.P, static_cast<cudaStream_t>(stream));
  if (rc != DILOCO_OK) return rc;
  advance(st, var);
  return DILOCO_OK;
}

template <int TK, int GK>
int launch_adamw_t(const diloco_state *st, const AdamArgs &a, cudaStream_t s) {
  constexpr int V = 4, U = 1, NT = 256, MINB = 4;
  const long long nvec = a.P / V;
  long long blocks = (nvec + (long long)NT * U - 1) / ((long long)NT * U);
  if (blocks < 1) blocks = 1;
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  dim3 grid((unsigned)blocks, (unsigned)st->cfg.M);
  adamw_kernel<TK, GK, V, U, NT, MINB><<<grid, NT, 0, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1);
  return DILOCO_OK;
}

template <int MODE, int VAR, int TK>
int launch_worker_t(const WorkerArgs &a, cudaStream_t s) {
  constexpr int V = 4, NT = 256;
  long long blocks = (a.P / V + NT - 1) / NT;
  if (blocks < 1) blocks = 1; // the last block also handles the P % V tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  worker_outer_kernel<MODE, VAR, TK, V, NT><<<(unsigned)blocks, NT, 0, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1);
  return DILOCO_OK;
}

template <int MODE, int VAR>
int launch_worker(int tk, const WorkerArgs &a, cudaStream_t s) {
  switch (tk) {
    case TK_F32: return launch_worker_t<MODE, VAR, TK_F32>(a, s);
    case TK_BF16: return launch_worker_t<MODE, VAR, TK_BF16>(a, s);
    default: return launch_worker_t<MODE, VAR, TK_MASTER_BF16>(a, s);
  }
}

WorkerArgs worker_args(const diloco_state *st, int32_t world_replicas, const float *recv, float *send) {
  WorkerArgs a;
  const diloco_buffers_t &b = st->buf;
  a.theta = b.theta;
  a.master = b.master;
  a.start = b.start;
  a.dpl = b.delta_prev_local ? b.delta_prev_local + (size_t)ring_slot(st) * (size_t)st->cfg.stride : nullptr;
  a.mom = b.outer_mom;
  a.recv = recv;
  a.send = send;
  a.P = st->cfg.P;
  a.eta = st->cfg.outer_lr;
  a.mu = st->cfg.outer_momentum;
  a.fM = (float)world_replicas;
  return a;
}

template <int MODE, int VAR, int TK>
int launch_worker_q_t(const WorkerQArgs &q, cudaStream_t s) {
  constexpr int NT = 256;
  long long blocks = (q.w.P / 4 + NT - 1) / NT;
  if (blocks < 1) blocks = 1; // the last block also handles the P % 4 tail
  if (blocks > 0x7fffffffLL) return DILOCO_ERR_UNSUPPORTED;
  worker_quantized_kernel<MODE, VAR, TK, NT><<<(unsigned)blocks, NT, 0, s>>>(q);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1);
  return DILOCO_OK;
}

template <int MODE, int VAR>
int launch_worker_q(int tk, const WorkerQArgs &q, cudaStream_t s) {
  switch (tk) {
    case TK_F32: return launch_worker_q_t<MODE, VAR, TK_F32>(q, s);
    case TK_BF16: return launch_worker_q_t<MODE, VAR, TK_BF16>(q, s);
    default: return launch_worker_q_t<MODE, VAR, TK_MASTER_BF16>(q, s);
  }
}

bool valid_exmy(int X, int Y) { return X >= 1 && X <= 5 && Y >= 0 && X + Y <= 7; }

WorkerQArgs worker_q_args(const diloco_state *st, int world, int X, int Y) {
  WorkerQArgs q;
  q.w = worker_args(st, world, nullptr, nullptr);
  q.precv = nullptr;
  q.amax_recv = nullptr;
  q.pstride = 0;
  q.psend = nullptr;
  q.amax_send = nullptr;
  q.world = world;
  q.man_bits = Y;
  q.bias = (1 << (X - 1)) - 1;
  q.emin = 1 - q.bias;
  q.code_bits = X + Y;
  q.fmt_max = std::ldexp(2.0f - std::ldexp(1.0f, -Y), (1 << X) - 1 - q.bias);
  q.packed = (X + Y + 1 <= 4) ? 1 : 0;
  return q;
}

// max |Delta_m| of this worker's replica into *amax (zeroed first), on stream s
int launch_worker_amax(diloco_state *st, unsigned *amax, cudaStream_t s) {
  cudaError_t e = cudaMemsetAsync(amax, 0, sizeof(unsigned), s);
  if (e != cudaSuccess) return cuda_fail(e);
  OuterArgs a = outer_args(st, 0, st->cfg.P);
  switch (st->cfg.theta_kind) {
    case TK_F32: return launch_amax_t<TK_F32>(st, a, amax, s);
    case TK_BF16: return launch_amax_t<TK_BF16>(st, a, amax, s);
    default: return launch_amax_t<TK_MASTER_BF16>(st, a, amax, s);
  }
}

// ---- per-device address of the scratch inside the library image ----------------------------
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned *g_static_ptr[kMaxDevices] = {}; // device address of g_static_scratch, per device ordinal

// `g_static_scratch` in host code is only a handle for the runtime, not a device address:
// ask the runtime for the address on the device that is current, once per device.
int static_scratch_for_current_device(int device, unsigned **out) {
  if (device < 0 || device >= kMaxDevices) return DILOCO_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[device]) {
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return cuda_fail(e);
    g_static_ptr[device] = static_cast<unsigned *>(p);
  }
  *out = g_static_ptr[device];
  return DILOCO_OK;
}

} // namespace

extern "C" {

int diloco_state_init(const diloco_config_t *config, const diloco_buffers_t *buffers, diloco_state_t **out) {
  if (!out) return DILOCO_ERR_INVALID_ARG;
  int rc = validate_config(config);
  if (rc != DILOCO_OK) return rc;
  rc = validate_buffers(config, buffers);
  if (rc != DILOCO_OK) return rc;
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return cuda_fail(e);
  {
    const void *all[] = {buffers->theta, buffers->master, buffers->start, buffers->delta_prev_local,
                         buffers->delta_prev_avg, buffers->outer_mom, buffers->adam_m, buffers->adam_v,
                         buffers->device_status, buffers->comm_scratch};
    for (const void *p : all)
      if (p && check_device_pointer(p, dev) != DILOCO_OK) return DILOCO_ERR_INVALID_ARG;
  }
  diloco_state *st = new (std::nothrow) diloco_state();
  if (!st) return DILOCO_ERR_INVALID_ARG;
  st->cfg = *config;
  st->buf = *buffers;
  st->device = dev;
  st->sm_count = sms;
  st->inner_step = 0;
  st->outer_step = 0;
  st->have_prev = config->have_prev;
  for (const void *&q : st->checked) q = nullptr;
  st->checked_next = 0;
  st->wait_limit_ns = kDefaultWaitLimitNs;
  st->test_extra_tx = 0;
  st->last_d2h = nullptr;
  *out = st;
  return DILOCO_OK;
}

int diloco_state_free(diloco_state_t *st) {
  if (!st) return DILOCO_OK;
  for (cudaEvent_t ev : st->events) cudaEventDestroy(ev);
  if (st->last_d2h) cudaEventDestroy(st->last_d2h);
  delete st;
  return DILOCO_OK;
}

int diloco_inner_adamw(diloco_state_t *st, const void *grads, int64_t grad_stride, float lr, void *stream) {
  if (!st || !grads) return DILOCO_ERR_INVALID_ARG;
  if (!st->buf.adam_m || !st->buf.adam_v) return DILOCO_ERR_BAD_STATE;
  if (grad_stride < st->cfg.P || !std::isfinite(lr)) return DILOCO_ERR_INVALID_ARG;
  {
    int rc = check_device(st);
    if (rc != DILOCO_OK) return rc;
  }
  const size_t gelt = st->cfg.grad_kind == DILOCO_GRAD_F32 ? 4 : 2;
  if (!aligned16(grads) || (grad_stride * (int64_t)gelt) % 128 != 0) return DILOCO_ERR_MISALIGNED;
  if (check_call_pointer(st, grads) != DILOCO_OK) return DILOCO_ERR_INVALID_ARG;
  const int64_t k = st->inner_step + 1;
  AdamArgs a;
  a.theta = st->buf.theta;
  a.master = st->buf.master;
  a.grads = grads;
  a.m = st->buf.adam_m;
  a.v = st->buf.adam_v;
  a.P = st->cfg.P;
  a.stride = st->cfg.stride;
  a.gstride = grad_stride;
  a.lr = lr;
  a.beta1 = st->cfg.beta1;
  a.beta2 = st->cfg.beta2;
  a.omb1 = 1.0f - st->cfg.beta1;
  a.omb2 = 1.0f - st->cfg.beta2;
  // bias corrections 1 - beta^k: in double, then one rounding to fp32
  a.c1 = (float)(1.0 - std::pow((double)st->cfg.beta1, (double)k));
  a.c2 = (float)(1.0 - std::pow((double)st->cfg.beta2, (double)k));
  a.eps = st->cfg.eps;
  a.wd = st->cfg.weight_decay;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = DILOCO_ERR_INVALID_ARG;
  const int tk = st->cfg.theta_kind, gk = st->cfg.grad_kind;
#define DILOCO_ADAM(TK_, GK_) \
  if (tk == TK_ && gk == GK_) rc = launch_adamw_t<TK_, GK_>(st, a, s);
  DILOCO_ADAM(TK_F32, GK_F32)
  DILOCO_ADAM(TK_F32, GK_BF16)
  DILOCO_ADAM(TK_BF16, GK_F32)
  DILOCO_ADAM(TK_BF16, GK_BF16)
  DILOCO_ADAM(TK_MASTER_BF16, GK_F32)
  DILOCO_ADAM(TK_MASTER_BF16, GK_BF16)
#undef DILOCO_ADAM
  if (rc != DILOCO_OK) return rc;
  st->inner_step = k;
  return DILOCO_OK;
}

int diloco_outer_standard(diloco_state_t *st, void *stream) { return outer_whole(st, VAR_STANDARD, stream); }
int diloco_outer_delayed(diloco_state_t *st, void *stream) { return outer_whole(st, VAR_DELAYED, stream); }
int diloco_outer_eager(diloco_state_t *st, void *stream) { return outer_whole(st, VAR_EAGER, stream); }

int diloco_outer_quantized(diloco_state_t *st, int32_t variant, int32_t comm_format, int32_t exp_bits, int32_t man_bits,
                           void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  int rc = check_variant(st, variant);
  if (rc != DILOCO_OK) return rc;
  if (comm_format == DILOCO_COMM_F32) return outer_whole(st, variant, stream);
  if (comm_format != DILOCO_COMM_BF16 && comm_format != DILOCO_COMM_EXMY) return DILOCO_ERR_INVALID_ARG;
  if (st->cfg.shared_outer_state) return DILOCO_ERR_BAD_STATE; // the wire formats have per-replica kernels only
  if (comm_format == DILOCO_COMM_EXMY) {
    if (exp_bits < 1 || exp_bits > 5 || man_bits < 0 || exp_bits + man_bits > 7) return DILOCO_ERR_INVALID_ARG;
    if (!st->buf.comm_scratch) return DILOCO_ERR_BAD_STATE;
  }
  rc = launch_outer_quantized(st, variant, is_first_steps(st, variant), comm_format, exp_bits, man_bits,
                              st->buf.comm_scratch, static_cast<cudaStream_t>(stream));
  if (rc != DILOCO_OK) return rc;
  advance(st, variant);
  return DILOCO_OK;
}

int diloco_outer_quantized_static(diloco_state_t *st, int32_t variant, int32_t comm_format, int32_t exp_bits,
                                  int32_t man_bits, void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  int rc = check_variant(st, variant);
  if (rc != DILOCO_OK) return rc;
  if (comm_format < DILOCO_COMM_F32 || comm_format > DILOCO_COMM_EXMY) return DILOCO_ERR_INVALID_ARG;
  if (comm_format == DILOCO_COMM_EXMY &&
      (exp_bits < 1 || exp_bits > 5 || man_bits < 0 || exp_bits + man_bits > 7))
    return DILOCO_ERR_INVALID_ARG;
  // one word of scratch per replica; today no state can have more replicas than the array has
  // words, the check keeps that true if the state limit is ever raised
  if (st->cfg.M > kStaticScratchWords) return DILOCO_ERR_UNSUPPORTED;
  if (comm_format == DILOCO_COMM_F32) return outer_whole(st, variant, stream);
  if (st->cfg.shared_outer_state) return DILOCO_ERR_BAD_STATE;
  unsigned *scratch = nullptr; // only the EXMY formats reduce maxima; the others never touch the array
  if (comm_format == DILOCO_COMM_EXMY) {
    // check_variant has verified that the state's GPU is the current one
    rc = static_scratch_for_current_device(st->device, &scratch);
    if (rc != DILOCO_OK) return rc;
  }
  // launch_outer_quantized zeroes the M words it reduces into before every use
  rc = launch_outer_quantized(st, variant, is_first_steps(st, variant), comm_format, exp_bits, man_bits, scratch,
                              static_cast<cudaStream_t>(stream));
  if (rc != DILOCO_OK) return rc;
  advance(st, variant);
  return DILOCO_OK;
}

int diloco_worker_outer_send(diloco_state_t *st, float *delta_send, void *stream) {
  if (!st || !delta_send) return DILOCO_ERR_INVALID_ARG;
  if (st->cfg.M != 1) return DILOCO_ERR_BAD_STATE;
  if (!aligned16(delta_send)) return DILOCO_ERR_MISALIGNED;
  int rc = check_device(st);
  if (rc != DILOCO_OK) return rc;
  if (check_call_pointer(st, delta_send) != DILOCO_OK) return DILOCO_ERR_INVALID_ARG;
  WorkerArgs a = worker_args(st, 1, nullptr, delta_send);
  return launch_worker<WMODE_SEND_ONLY, VAR_STANDARD>(st->cfg.theta_kind, a, static_cast<cudaStream_t>(stream));
}

int diloco_worker_outer_apply(diloco_state_t *st, int32_t variant, int32_t world_replicas, const float *delta_sum_recv,
                              float *delta_send, void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  if (variant < VAR_STANDARD || variant > VAR_EAGER) return DILOCO_ERR_INVALID_ARG;
  if (world_replicas < 1 || world_replicas > (1 << 24)) return DILOCO_ERR_INVALID_ARG; // exact as a float
  if (st->cfg.M != 1) return DILOCO_ERR_BAD_STATE;
  if (variant == VAR_EAGER && !st->buf.delta_prev_local) return DILOCO_ERR_BAD_STATE;
  const bool first = is_first_steps(st, variant);
  if (variant != VAR_STANDARD && !delta_send) return DILOCO_ERR_INVALID_ARG;
  if (!first && !delta_sum_recv) return DILOCO_ERR_INVALID_ARG;
  if ((delta_send && !aligned16(delta_send)) || (delta_sum_recv && !aligned16(delta_sum_recv))) return DILOCO_ERR_MISALIGNED;
  int rc = check_device(st);
  if (rc != DILOCO_OK) return rc;
  if (delta_send && check_call_pointer(st, delta_send) != DILOCO_OK) return DILOCO_ERR_INVALID_ARG;
  if (!first && check_call_pointer(st, delta_sum_recv) != DILOCO_OK) return DILOCO_ERR_INVALID_ARG;
  WorkerArgs a = worker_args(st, world_replicas, delta_sum_recv, delta_send);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int tk = st->cfg.theta_kind;
  if (variant == VAR_STANDARD) rc = launch_worker<WMODE_APPLY, VAR_STANDARD>(tk, a, s);
  else if (variant == VAR_DELAYED) rc = first ? launch_worker<WMODE_RECORD, VAR_DELAYED>(tk, a, s)
                                              : launch_worker<WMODE_APPLY_SEND, VAR_DELAYED>(tk, a, s);
  else rc = first ? launch_worker<WMODE_RECORD, VAR_EAGER>(tk, a, s) : launch_worker<WMODE_APPLY_SEND, VAR_EAGER>(tk, a, s);
  if (rc != DILOCO_OK) return rc;
  advance(st, variant);
  return DILOCO_OK;
}

int64_t diloco_wire_payload_bytes(int64_t P, int32_t exp_bits, int32_t man_bits) {
  if (P < 0 || !valid_exmy(exp_bits, man_bits)) return DILOCO_ERR_INVALID_ARG;
  return (exp_bits + man_bits + 1 <= 4) ? (P + 1) / 2 : P;
}

int diloco_worker_quantized_send(diloco_state_t *st, int32_t exp_bits, int32_t man_bits, uint8_t *payload_send,
                                 uint32_t *amax_send, void *stream) {
  if (!st || !payload_send || !amax_send || !valid_exmy(exp_bits, man_bits)) return DILOCO_ERR_INVALID_ARG;
  if (st->cfg.M != 1) return DILOCO_ERR_BAD_STATE;
  if ((reinterpret_cast<uintptr_t>(payload_send) & 3u) || (reinterpret_cast<uintptr_t>(amax_send) & 3u)) return DILOCO_ERR_MISALIGNED;
  int rc = check_device(st);
  if (rc != DILOCO_OK) return rc;
  if (check_call_pointer(st, payload_send) != DILOCO_OK || check_call_pointer(st, amax_send) != DILOCO_OK)
    return DILOCO_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  rc = launch_worker_amax(st, amax_send, s);
  if (rc != DILOCO_OK) return rc;
  WorkerQArgs q = worker_q_args(st, 1, exp_bits, man_bits);
  q.psend = payload_send;
  q.amax_send = amax_send;
  return launch_worker_q<WMODE_SEND_ONLY, VAR_STANDARD>(st->cfg.theta_kind, q, s);
}

int diloco_worker_quantized_apply(diloco_state_t *st, int32_t variant, int32_t world_replicas, int32_t exp_bits,
                                  int32_t man_bits, const uint8_t *payloads_recv, int64_t payload_stride,
                                  const uint32_t *amaxes_recv, uint8_t *payload_send, uint32_t *amax_send, void *stream) {
  if (!st || !valid_exmy(exp_bits, man_bits)) return DILOCO_ERR_INVALID_ARG;
  if (variant < VAR_STANDARD || variant > VAR_EAGER) return DILOCO_ERR_INVALID_ARG;
  if (world_replicas < 1) return DILOCO_ERR_INVALID_ARG;
  if (world_replicas > DILOCO_WORKER_MAX_WORLD) return DILOCO_ERR_UNSUPPORTED;
  if (st->cfg.M != 1) return DILOCO_ERR_BAD_STATE;
  if (variant == VAR_EAGER && !st->buf.delta_prev_local) return DILOCO_ERR_BAD_STATE;
  const bool first = is_first_steps(st, variant);
  const bool sends = variant != VAR_STANDARD;
  if (sends && (!payload_send || !amax_send)) return DILOCO_ERR_INVALID_ARG;
  if (!first) {
    if (!payloads_recv || !amaxes_recv) return DILOCO_ERR_INVALID_ARG;
    if (payload_stride < diloco_wire_payload_bytes(st->cfg.P, exp_bits, man_bits) || payload_stride % 4 != 0)
      return DILOCO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(payloads_recv) & 3u) || (reinterpret_cast<uintptr_t>(amaxes_recv) & 3u)) return DILOCO_ERR_MISALIGNED;
  }
  if (sends && ((reinterpret_cast<uintptr_t>(payload_send) & 3u) || (reinterpret_cast<uintptr_t>(amax_send) & 3u))) return DILOCO_ERR_MISALIGNED;
  int rc = check_device(st);
  if (rc != DILOCO_OK) return rc;
  if (!first && (check_call_pointer(st, payloads_recv) != DILOCO_OK ||
                 check_call_pointer(st, amaxes_recv) != DILOCO_OK))
    return DILOCO_ERR_INVALID_ARG;
  if (sends && (check_call_pointer(st, payload_send) != DILOCO_OK ||
                check_call_pointer(st, amax_send) != DILOCO_OK))
    return DILOCO_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (sends) {
    rc = launch_worker_amax(st, amax_send, s);
    if (rc != DILOCO_OK) return rc;
  }
  WorkerQArgs q = worker_q_args(st, world_replicas, exp_bits, man_bits);
  q.precv = payloads_recv;
  q.amax_recv = amaxes_recv;
  q.pstride = payload_stride;
  q.psend = payload_send;
  q.amax_send = amax_send;
  const int tk = st->cfg.theta_kind;
  if (variant == VAR_STANDARD) rc = launch_worker_q<WMODE_APPLY, VAR_STANDARD>(tk, q, s);
  else if (variant == VAR_DELAYED) rc = first ? launch_worker_q<WMODE_RECORD, VAR_DELAYED>(tk, q, s)
                                              : launch_worker_q<WMODE_APPLY_SEND, VAR_DELAYED>(tk, q, s);
  else rc = first ? launch_worker_q<WMODE_RECORD, VAR_EAGER>(tk, q, s) : launch_worker_q<WMODE_APPLY_SEND, VAR_EAGER>(tk, q, s);
  if (rc != DILOCO_OK) return rc;
  advance(st, variant);
  return DILOCO_OK;
}

int diloco_outer_fragment(diloco_state_t *st, int32_t variant, int32_t bootstrap, int64_t offset, int64_t len,
                          void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  int rc = check_variant(st, variant);
  if (rc != DILOCO_OK) return rc;
  if (variant == VAR_STANDARD && bootstrap) return DILOCO_ERR_INVALID_ARG;
  if (offset < 0 || len < 1 || offset > st->cfg.P - len) return DILOCO_ERR_INVALID_ARG;
  const int64_t q = st->cfg.theta_kind == DILOCO_THETA_F32 ? 32 : 64;
  if (offset % q != 0) return DILOCO_ERR_MISALIGNED;
  return launch_outer(st, variant, bootstrap != 0, offset, len, static_cast<cudaStream_t>(stream));
}

int diloco_fragments_set(diloco_state_t *st, int32_t n, const int64_t *offsets, const int64_t *lens) {
  if (!st || n < 0 || (n > 0 && (!offsets || !lens))) return DILOCO_ERR_INVALID_ARG;
  if (n > DILOCO_MAX_FRAGMENTS) return DILOCO_ERR_UNSUPPORTED;
  const int64_t q = st->cfg.theta_kind == DILOCO_THETA_F32 ? 32 : 64;
  std::vector<Fragment> f((size_t)n);
  for (int32_t i = 0; i < n; ++i) {
    if (offsets[i] < 0 || lens[i] < 1 || offsets[i] > st->cfg.P - lens[i]) return DILOCO_ERR_INVALID_ARG;
    if (offsets[i] % q != 0) return DILOCO_ERR_MISALIGNED;
    f[(size_t)i] = Fragment{offsets[i], lens[i], st->outer_step, st->have_prev};
  }
  // fragments must not overlap: two schedules writing one index would make its history meaningless
  std::vector<std::pair<int64_t, int64_t>> spans;
  for (const Fragment &x : f) spans.emplace_back(x.offset, x.offset + x.len);
  std::sort(spans.begin(), spans.end());
  for (size_t i = 1; i < spans.size(); ++i)
    if (spans[i].first < spans[i - 1].second) return DILOCO_ERR_INVALID_ARG;
  st->frags.swap(f);
  return DILOCO_OK;
}

int diloco_outer_fragment_step(diloco_state_t *st, int32_t variant, int32_t fragment_id, void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  int rc = check_variant(st, variant);
  if (rc != DILOCO_OK) return rc;
  if (fragment_id < 0 || (size_t)fragment_id >= st->frags.size()) return DILOCO_ERR_INVALID_ARG;
  Fragment &f = st->frags[(size_t)fragment_id];
  const bool boot = variant != VAR_STANDARD && f.have_prev < st->cfg.overlap_steps;
  const int ring = (int)(f.outer_step % st->cfg.overlap_steps);
  rc = launch_outer(st, variant, boot, f.offset, f.len, static_cast<cudaStream_t>(stream), ring);
  if (rc != DILOCO_OK) return rc;
  if (boot) f.have_prev += 1;
  f.outer_step += 1;
  return DILOCO_OK;
}

int diloco_outer_fragment_step_quantized(diloco_state_t *st, int32_t variant, int32_t fragment_id, int32_t comm_format,
                                         int32_t exp_bits, int32_t man_bits, void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  if (comm_format == DILOCO_COMM_F32) return diloco_outer_fragment_step(st, variant, fragment_id, stream);
  int rc = check_variant(st, variant);
  if (rc != DILOCO_OK) return rc;
  if (fragment_id < 0 || (size_t)fragment_id >= st->frags.size()) return DILOCO_ERR_INVALID_ARG;
  if (comm_format != DILOCO_COMM_BF16 && comm_format != DILOCO_COMM_EXMY) return DILOCO_ERR_INVALID_ARG;
  if (st->cfg.shared_outer_state) return DILOCO_ERR_BAD_STATE;
  if (comm_format == DILOCO_COMM_EXMY) {
    if (!valid_exmy(exp_bits, man_bits)) return DILOCO_ERR_INVALID_ARG;
    if (!st->buf.comm_scratch) return DILOCO_ERR_BAD_STATE;
  }
  Fragment &f = st->frags[(size_t)fragment_id];
  const bool boot = variant != VAR_STANDARD && f.have_prev < st->cfg.overlap_steps;
  const int ring = (int)(f.outer_step % st->cfg.overlap_steps);
  rc = launch_outer_quantized(st, variant, boot, comm_format, exp_bits, man_bits, st->buf.comm_scratch,
                              static_cast<cudaStream_t>(stream), f.offset, f.len, ring);
  if (rc != DILOCO_OK) return rc;
  if (boot) f.have_prev += 1;
  f.outer_step += 1;
  return DILOCO_OK;
}

int diloco_fragment_get_counters(const diloco_state_t *st, int32_t fragment_id, int64_t *outer_step, int32_t *have_prev) {
  if (!st || fragment_id < 0 || (size_t)fragment_id >= st->frags.size()) return DILOCO_ERR_INVALID_ARG;
  if (outer_step) *outer_step = st->frags[(size_t)fragment_id].outer_step;
  if (have_prev) *have_prev = st->frags[(size_t)fragment_id].have_prev;
  return DILOCO_OK;
}

int diloco_fragment_set_counters(diloco_state_t *st, int32_t fragment_id, int64_t outer_step, int32_t have_prev) {
  if (!st || fragment_id < 0 || (size_t)fragment_id >= st->frags.size()) return DILOCO_ERR_INVALID_ARG;
  if (outer_step < 0 || have_prev < 0 || have_prev > st->cfg.overlap_steps) return DILOCO_ERR_INVALID_ARG;
  st->frags[(size_t)fragment_id].outer_step = outer_step;
  st->frags[(size_t)fragment_id].have_prev = have_prev;
  return DILOCO_OK;
}

int diloco_outer_step_host(diloco_state_t *st, int32_t variant, const diloco_buffers_t *host, void *const streams[3],
                           int64_t chunk) {
  if (!st || !host || !streams) return DILOCO_ERR_INVALID_ARG;
  int rc = check_variant(st, variant);
  if (rc != DILOCO_OK) return rc;
  if (chunk < 64 || chunk % 64 != 0) return DILOCO_ERR_INVALID_ARG;
  if (st->cfg.shared_outer_state) return DILOCO_ERR_BAD_STATE; // the copy plan below assumes one row per replica
  cudaStream_t s_in = static_cast<cudaStream_t>(streams[0]);
  cudaStream_t s_k = static_cast<cudaStream_t>(streams[1]);
  cudaStream_t s_out = static_cast<cudaStream_t>(streams[2]);
  if (s_in == s_k || s_k == s_out || s_in == s_out) return DILOCO_ERR_INVALID_ARG;
  const diloco_buffers_t &d = st->buf;
  const bool boot = is_first_steps(st, variant);
  const int tk = st->cfg.theta_kind;
  const size_t slot = (size_t)ring_slot(st);
  const size_t slot_rows = slot * (size_t)st->cfg.M * (size_t)st->cfg.stride; // this step's generation
  const size_t slot_row = slot * (size_t)st->cfg.stride;
  // which buffers the variant reads (in) and writes (out); rows = M, or 1 for delta_prev_avg
  struct Leg { void *dev; void *hst; size_t elt; int rows; bool in, out; };
  const bool master = tk == DILOCO_THETA_MASTER_BF16;
  Leg legs[6] = {
      {d.theta, host->theta, theta_elt(tk), st->cfg.M, !master, !boot},
      {d.master, host->master, 4, st->cfg.M, master, master && !boot},
      {d.start, host->start, 4, st->cfg.M, true, true},
      {d.delta_prev_local ? d.delta_prev_local + slot_rows : nullptr,
       host->delta_prev_local ? host->delta_prev_local + slot_rows : nullptr, 4, st->cfg.M,
       variant == VAR_EAGER && !boot, variant == VAR_EAGER},
      {d.delta_prev_avg ? d.delta_prev_avg + slot_row : nullptr,
       host->delta_prev_avg ? host->delta_prev_avg + slot_row : nullptr, 4, 1,
       variant != VAR_STANDARD && !boot, variant != VAR_STANDARD},
      {d.outer_mom, host->outer_mom, 4, st->cfg.M, !boot, !boot},
  };
  for (const Leg &l : legs)
    if ((l.in || l.out) && !l.dev) return DILOCO_ERR_INVALID_ARG;
  if (!host->theta && !host->master) return DILOCO_ERR_INVALID_ARG; // something must come from the host
  // a host buffer that is really device memory would turn the copies below into silent
  // device-to-device copies of the wrong data: refuse it (unregistered host memory is accepted,
  // the copies are then synchronous with respect to the host)
  for (const Leg &l : legs) {
    if (!l.hst || !(l.in || l.out)) continue;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, l.hst) != cudaSuccess) {
      cudaGetLastError();
      continue; // older drivers report plain malloc memory as an error: that is host memory
    }
    if (at.type == cudaMemoryTypeDevice) return DILOCO_ERR_INVALID_ARG;
  }
  const int64_t P = st->cfg.P;
  const size_t nchunks = (size_t)((P + chunk - 1) / chunk);
  cudaError_t e;
  // everything that can fail without touching a stream comes first
  while (st->events.size() < 2 * nchunks) {
    cudaEvent_t ev;
    e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(e);
    st->events.push_back(ev);
  }
  if (!st->last_d2h) {
    e = cudaEventCreateWithFlags(&st->last_d2h, cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(e);
  } else {
    // the staging area is reused: do not overwrite it before the previous call has drained
    e = cudaStreamWaitEvent(s_in, st->last_d2h, 0);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  const size_t row = (size_t)st->cfg.stride;
  // One plain copy per row and chunk (rows of 2^29 fp32 elements and more exceed the pitch
  // limit of the 2-D copy routines; chunks are megabytes, so the copies stay few and large).
  auto copy_rows = [&](const Leg &l, int64_t off, int64_t len, bool to_device, cudaStream_t s) -> cudaError_t {
    for (int r = 0; r < l.rows; ++r) {
      const size_t at = ((size_t)r * row + (size_t)off) * l.elt;
      char *dv = static_cast<char *>(l.dev) + at;
      char *hs = static_cast<char *>(l.hst) + at;
      cudaError_t ce = to_device ? cudaMemcpyAsync(dv, hs, (size_t)len * l.elt, cudaMemcpyHostToDevice, s)
                                 : cudaMemcpyAsync(hs, dv, (size_t)len * l.elt, cudaMemcpyDeviceToHost, s);
      if (ce != cudaSuccess) return ce;
    }
    return cudaSuccess;
  };
  for (size_t c = 0; c < nchunks; ++c) {
    const int64_t off = (int64_t)c * chunk;
    const int64_t len = (off + chunk <= P) ? chunk : (P - off);
    for (const Leg &l : legs) {
      if (!l.in || !l.hst) continue; // a NULL host pointer: that buffer is resident on the device
      e = copy_rows(l, off, len, true, s_in);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    e = cudaEventRecord(st->events[2 * c], s_in);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamWaitEvent(s_k, st->events[2 * c], 0);
    if (e != cudaSuccess) return cuda_fail(e);
    rc = launch_outer(st, variant, boot, off, len, s_k);
    if (rc != DILOCO_OK) return rc;
    e = cudaEventRecord(st->events[2 * c + 1], s_k);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamWaitEvent(s_out, st->events[2 * c + 1], 0);
    if (e != cudaSuccess) return cuda_fail(e);
    for (const Leg &l : legs) {
      if (!l.out || !l.hst) continue;
      e = copy_rows(l, off, len, false, s_out);
      if (e != cudaSuccess) return cuda_fail(e);
    }
  }
  e = cudaEventRecord(st->last_d2h, s_out);
  if (e != cudaSuccess) return cuda_fail(e);
  advance(st, variant);
  return DILOCO_OK;
}

int diloco_state_get_counters(const diloco_state_t *st, int64_t *inner_step, int64_t *outer_step, int32_t *have_prev) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  if (inner_step) *inner_step = st->inner_step;
  if (outer_step) *outer_step = st->outer_step;
  if (have_prev) *have_prev = st->have_prev;
  return DILOCO_OK;
}

int diloco_state_set_counters(diloco_state_t *st, int64_t inner_step, int64_t outer_step, int32_t have_prev) {
  if (!st || inner_step < 0 || outer_step < 0 || have_prev < 0 || have_prev > st->cfg.overlap_steps)
    return DILOCO_ERR_INVALID_ARG;
  st->inner_step = inner_step;
  st->outer_step = outer_step;
  st->have_prev = have_prev;
  return DILOCO_OK;
}

int diloco_set_outer_hparams(diloco_state_t *st, float outer_lr, float outer_momentum) {
  if (!st || !std::isfinite(outer_lr) || !(outer_momentum >= 0.f && outer_momentum < 1.f)) return DILOCO_ERR_INVALID_ARG;
  st->cfg.outer_lr = outer_lr;
  st->cfg.outer_momentum = outer_momentum;
  return DILOCO_OK;
}

int diloco_set_impl(diloco_state_t *st, int32_t impl) {
  if (!st || impl < DILOCO_IMPL_AUTO || impl > DILOCO_IMPL_TENSOR_T64) return DILOCO_ERR_INVALID_ARG;
  st->cfg.impl = impl;
  return DILOCO_OK;
}

int diloco_set_wait_limit(diloco_state_t *st, uint64_t limit_ns, uint32_t test_extra_expect_bytes) {
  if (!st || test_extra_expect_bytes % 16 != 0 || test_extra_expect_bytes > 1024) return DILOCO_ERR_INVALID_ARG;
  st->wait_limit_ns = limit_ns ? limit_ns : kDefaultWaitLimitNs;
  st->test_extra_tx = test_extra_expect_bytes;
  return DILOCO_OK;
}

int diloco_check_device_status(diloco_state_t *st, void *stream) {
  if (!st) return DILOCO_ERR_INVALID_ARG;
  if (!st->buf.device_status) return DILOCO_OK;
  uint32_t word = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(&word, st->buf.device_status, sizeof(word), cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(e);
  return word == 0 ? DILOCO_OK : DILOCO_ERR_DEVICE_TIMEOUT;
}

int64_t diloco_launch_count(void) { return g_launches.load(); }
int32_t diloco_last_cuda_error(void) { return g_last_cuda_error.load(); }

const char *diloco_status_string(int status) {
  switch (status) {
    case DILOCO_OK: return "ok";
    case DILOCO_ERR_INVALID_ARG: return "invalid argument";
    case DILOCO_ERR_MISALIGNED: return "misaligned pointer, stride or offset";
    case DILOCO_ERR_BAD_STATE: return "state lacks a buffer this call needs";
    case DILOCO_ERR_CUDA: return "CUDA runtime error";
    case DILOCO_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case DILOCO_ERR_UNSUPPORTED: return "unsupported size";
    default: return "unknown status";
  }
}

} // extern "C"
