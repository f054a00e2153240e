// Fused outer step, "tensor" form: every state buffer is described to the TMA unit as a 2-D
// tensor [M rows x P columns] (row pitch = the replica stride), and one box copy moves the
// tile [all M replicas x T consecutive indices] of a buffer between global and shared memory.
// A tile therefore costs 5 loads and 5 stores (theta, start, outer_mom, delta_prev_local,
// delta_prev_avg) whatever M is, where the row-by-row form of diloco_bulk.cuh needs 4 M + 1 of
// each - the per-copy cost of the copy engine was what limited that form.  The tensor maps cover
// this GPU's own memory only and no copy uses cluster multicast.  The tensors cover the columns
// [0, P4), P4 = P rounded down to a multiple of 4: the hardware zero-fills a box's columns
// beyond that on load and clips them on store, but it clips in units of 16 bytes, so a tensor
// that ended inside a 16-byte unit would have its padding overwritten.  The last P % 4 indices
// are done with plain loads and stores by the last CTA.
//
// Per CTA (one per SM, tiles taken round-robin), ring of S stages:
//   thread 0:  arm full[s] with the tile's byte count, issue the box loads (complete_tx)
//   all:       wait full[s] (bounded in time); pass 1: one index per thread, the ordered sum
//              m = 0 .. M-1 of Delta_m = s_m - theta_m and its mean into the stage; barrier;
//              pass 2: one (replica, 4 indices) item per thread, the update in place;
//              fence.proxy.async; barrier
//   thread 0:  issue the box stores as one bulk group; before a stage is refilled, wait until
//              the group that drained it has finished reading shared memory
// Same arithmetic, same order, same bits as the direct form.  fp32 theta, M at run time.
// Measured (eager fp32, GB/s; direct form in brackets): T = 256: M = 2 2548 [6760], M = 4 4401
// [6773], M = 8 6163-6573 [6755], M = 16 6250 [6737], M = 32 falls back.  One CTA per SM works
// through its tiles one after the other, so below M = 8 the per-tile latency of the two passes
// (about 1 us) is not hidden by anything, and at M = 16 only three 68 KB stages fit, i.e. one
// tile of loads in flight.  A hybrid with TMA loads and ordinary stores from registers (half the
// box copies, one more stage for loads) measured the same or lower (M = 8 6380, M = 16 5903) and
// was dropped.  The form is kept as a tested alternative; AUTO never selects it.
#pragma once
#include <cuda.h>

#include "diloco_bulk.cuh"

namespace diloco {

constexpr int kTensorMaxStages = 16;

struct TensorMaps {
  CUtensorMap theta, start, mom, dpl; // [M, P] boxes of [M, T]
  CUtensorMap dpa;                    // [1, P] boxes of [1, T]
};

__device__ __forceinline__ void tensor_load_2d(void *dst_smem, const CUtensorMap *map, int x, int y,
                                               unsigned long long *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst_smem)),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tensor_store_2d(const CUtensorMap *map, int x, int y, const void *src_smem) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                   reinterpret_cast<unsigned long long>(map)),
               "r"(x), "r"(y), "r"(smem_u32(src_smem))
               : "memory");
}

// floats per stage: theta, start, mom [M][T] each, dpl [M][T] (eager), dpa [T] (delayed, eager), mean [T]
template <int VAR> __host__ __device__ constexpr int tensor_rows_per_stage(int M) {
  return (VAR == VAR_EAGER ? 4 : 3) * M + (VAR != VAR_STANDARD ? 1 : 0) + 1;
}

template <int VAR, int T, int NT>
__global__ void __launch_bounds__(NT, 1)
    outer_step_tensor_kernel(const __grid_constant__ TensorMaps maps, const OuterArgs a, unsigned *status, int stages,
                             unsigned long long limit_ns, unsigned extra_tx) {
  static_assert(T % 32 == 0 && T <= 256, "a box is at most 256 elements wide; stage buffers stay 128-byte aligned");
  extern __shared__ __align__(128) float smem_f[];
  __shared__ unsigned long long full[kTensorMaxStages];
  __shared__ volatile unsigned s_abort;

  const int M = a.M, S = stages, tid = threadIdx.x;
  const int rows = tensor_rows_per_stage<VAR>(M);
  const long long P4 = a.P & ~3ll;                 // columns the tensor maps cover
  const long long ntiles = (P4 + T - 1) / T;
  const long long mine = ntiles > blockIdx.x ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const int LOOK = S - 2; // tiles in flight ahead of the one being computed; one more stage is draining
  // stage layout, in floats
  const int oX = 0, oS = M * T, oB = 2 * M * T, oPL = 3 * M * T;
  const int oPA = (VAR == VAR_EAGER ? 4 : 3) * M * T;
  const int oMEAN = oPA + (VAR != VAR_STANDARD ? T : 0);
  const unsigned load_bytes = (unsigned)((rows - 1) * T * 4) + extra_tx;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) mbar_init(&full[s], 1);
    s_abort = 0;
    fence_mbar_init();
  }
  __syncthreads();

  auto issue_loads = [&](long long j) {
    float *st = smem_f + (size_t)(j % S) * rows * T;
    unsigned long long *bar = &full[j % S];
    const int x = (int)((blockIdx.x + j * gridDim.x) * T);
    mbar_expect_tx(bar, load_bytes);
    tensor_load_2d(st + oX, &maps.theta, x, 0, bar);
    tensor_load_2d(st + oS, &maps.start, x, 0, bar);
    tensor_load_2d(st + oB, &maps.mom, x, 0, bar);
    if (VAR == VAR_EAGER) tensor_load_2d(st + oPL, &maps.dpl, x, 0, bar);
    if (VAR != VAR_STANDARD) tensor_load_2d(st + oPA, &maps.dpa, x, 0, bar);
  };
  auto issue_stores = [&](long long j) {
    const float *st = smem_f + (size_t)(j % S) * rows * T;
    const int x = (int)((blockIdx.x + j * gridDim.x) * T);
    tensor_store_2d(&maps.theta, x, 0, st + oX);
    tensor_store_2d(&maps.start, x, 0, st + oS);
    tensor_store_2d(&maps.mom, x, 0, st + oB);
    if (VAR == VAR_EAGER) tensor_store_2d(&maps.dpl, x, 0, st + oPL);
    if (VAR != VAR_STANDARD) tensor_store_2d(&maps.dpa, x, 0, st + oMEAN);
    bulk_commit();
  };

  if (tid == 0)
    for (long long j = 0; j < LOOK && j < mine; ++j) issue_loads(j);

  bool aborted = false;
  for (long long j = 0; j < mine; ++j) {
    if (tid == 0 && j + LOOK < mine) {
      bulk_wait_read<1>(); // the group that drained stage (j + LOOK) % S is tile j-2's
      issue_loads(j + LOOK);
    }
    const bool ok = mbar_wait_bounded(&full[j % S], (unsigned)((j / S) & 1), limit_ns, &s_abort);
    if (!ok) s_abort = 1;
    float *st = smem_f + (size_t)(j % S) * rows * T;
    if (ok) {
      // pass 1, Alg. 1-3 lines 7-8: Delta = (1/M) sum_m (s_m - theta_m), m in order, one index per thread
      for (int i = tid; i < T; i += NT) {
        float acc = st[oS + i] - st[oX + i];
        for (int m = 1; m < M; ++m) {
          const float d = st[oS + m * T + i] - st[oX + m * T + i];
          acc = acc + d;
        }
        st[oMEAN + i] = acc / a.fM;
      }
    }
    __syncthreads();
    if (ok && !s_abort) {
      // pass 2, lines 10-12: item = (replica m, column of 4 indices), updated in place
      const int items = M * (T / 4);
      for (int it = tid; it < items; it += NT) {
        const int m = it / (T / 4), c = (it % (T / 4)) * 4;
        const float4 x4 = *reinterpret_cast<const float4 *>(st + oX + m * T + c);
        const float4 s4 = *reinterpret_cast<const float4 *>(st + oS + m * T + c);
        const float4 b4 = *reinterpret_cast<const float4 *>(st + oB + m * T + c);
        float s[4] = {s4.x, s4.y, s4.z, s4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
        const float x[4] = {x4.x, x4.y, x4.z, x4.w};
        float d[4], pl[4] = {0.f, 0.f, 0.f, 0.f}, pa[4] = {0.f, 0.f, 0.f, 0.f}, mean[4];
        if (VAR == VAR_EAGER) {
          const float4 t = *reinterpret_cast<const float4 *>(st + oPL + m * T + c);
          pl[0] = t.x; pl[1] = t.y; pl[2] = t.z; pl[3] = t.w;
        }
        if (VAR != VAR_STANDARD) {
          const float4 t = *reinterpret_cast<const float4 *>(st + oPA + c);
          pa[0] = t.x; pa[1] = t.y; pa[2] = t.z; pa[3] = t.w;
        }
        if (VAR == VAR_STANDARD) {
          const float4 t = *reinterpret_cast<const float4 *>(st + oMEAN + c);
          mean[0] = t.x; mean[1] = t.y; mean[2] = t.z; mean[3] = t.w;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          d[e] = s[e] - x[e];                       // line 7 again: same operands, same bits
          float g;
          if (VAR == VAR_STANDARD) g = mean[e];     // Alg. 1 line 10
          else if (VAR == VAR_DELAYED) g = pa[e];   // Alg. 2 line 11
          else {
            float t = d[e] - pl[e];                 // Alg. 3 line 11
            t = t / a.fM;
            g = t + pa[e];
          }
          nesterov(g, a.eta, a.mu, b[e], s[e]);
        }
        const float4 ns = make_float4(s[0], s[1], s[2], s[3]);
        *reinterpret_cast<float4 *>(st + oS + m * T + c) = ns;
        *reinterpret_cast<float4 *>(st + oX + m * T + c) = ns;
        *reinterpret_cast<float4 *>(st + oB + m * T + c) = make_float4(b[0], b[1], b[2], b[3]);
        if (VAR == VAR_EAGER) *reinterpret_cast<float4 *>(st + oPL + m * T + c) = make_float4(d[0], d[1], d[2], d[3]);
      }
    }
    fence_async_smem(); // generic-proxy writes above -> visible to the store's async proxy
    aborted = __syncthreads_or(s_abort != 0) != 0; // one decision for the whole CTA
    if (aborted) {
      if (tid == 0) {
        // give the loads still in flight a bounded chance to land before shared memory is released
        for (long long q = j; q < mine && q <= j + LOOK; ++q)
          mbar_wait_bounded(&full[q % S], (unsigned)((q / S) & 1), limit_ns, nullptr);
      }
      break;
    }
    if (tid == 0) issue_stores(j);
  }
  if (tid == 0) {
    bulk_wait_all();
    if (aborted && status) atomicExch(status, kStatusTimeout);
  }
  // ragged remainder (P % 4 indices): plain loads and stores, one index per thread
  if (blockIdx.x == gridDim.x - 1 && !aborted) {
    const long long i = P4 + tid;
    if (i < a.P) outer_column_rt<VAR, TK_F32, false, 1>(a, i);
  }
}

} // namespace diloco
