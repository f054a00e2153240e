// Fused outer step, "bulk" form: replica tiles are staged through shared memory by the TMA
// unit (1-D cp.async.bulk, no tensor map, no multicast), updated in place there and written
// back by bulk stores.  Same arithmetic, same order, same bits as the direct form; what
// changes is who moves the bytes: one elected thread issues (4M+1) asynchronous row copies
// per tile and direction, so the bytes in flight per SM are set by the stage count, not by
// registers, which is what lets M = 8 and M = 16 stream as well as M = 2.
//
// Per CTA (persistent, tiles taken round-robin so that all SMs walk memory together):
//   stage ring of S buffers, each holding one tile = T consecutive indices of every row
//   thread 0:  arm full[s] with the tile's byte count, issue the row loads (complete_tx)
//   all:       wait full[s] (bounded), update the tile in place, fence.proxy.async, barrier
//   thread 0:  issue the row stores as one bulk group; before a stage is refilled, wait
//              until the group that drained it has finished reading shared memory
// Every wait is bounded in TIME: a thread that has polled a barrier for longer than the
// launch's wait limit (nanoseconds of %globaltimer; 1 s unless the caller set another) raises
// the CTA's abort flag, the CTA stops taking tiles, gives its loads in flight one more limit
// to land, drains its own stores and reports through the device status word (host:
// DILOCO_ERR_DEVICE_TIMEOUT).  Worst case a CTA therefore returns after (ring depth + 1) wait
// limits.  A hard poll count backs the clock up.
#pragma once
#include "diloco_kernels.cuh"

namespace diloco {

constexpr unsigned kSpinLimit = 1u << 26; // hard cap on polls of mbarrier.try_wait, whatever the clock says
constexpr unsigned kStatusTimeout = 0x7101u;

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// global -> shared, completion signalled on an mbarrier of this CTA
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, unsigned bytes, unsigned long long *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// shared -> global, tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void bulk_store(void *dst_gmem, const void *src_smem, unsigned bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_gmem), "r"(smem_u32(src_smem)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// Shared-memory layout of one stage for (M, VAR, TK) with tile length T (elements).
template <int M, int VAR, int TK, int T> struct BulkStage {
  static constexpr int kThetaBytes = (TK == TK_BF16 ? 2 : 4) * T; // row of theta (bf16) or of theta/master (fp32)
  static constexpr int kRow = 4 * T;
  static constexpr int offX = 0;                                  // M rows: theta or master
  static constexpr int offS = offX + M * kThetaBytes;             // M rows: start
  static constexpr int offB = offS + M * kRow;                    // M rows: outer_mom
  static constexpr int offPL = offB + M * kRow;                   // M rows: delta_prev_local (eager)
  static constexpr int offPA = offPL + (VAR == VAR_EAGER ? M * kRow : 0); // 1 row: delta_prev_avg
  static constexpr int offC = offPA + (VAR != VAR_STANDARD ? kRow : 0);   // M rows bf16: working copy (master mode)
  static constexpr int kBytes = offC + (TK == TK_MASTER_BF16 ? M * 2 * T : 0);
  static constexpr unsigned kLoadBytes = (unsigned)offC; // everything before the bf16 copy is loaded
};

// Poll `bar` for the given phase until it completes, `limit_ns` has passed, the poll cap is hit
// or (if `abort` is given) another thread of the CTA has given up.  Returns whether it completed.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long *bar, unsigned parity, unsigned long long limit_ns,
                                                  const volatile unsigned *abort) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (unsigned spins = 0; spins < kSpinLimit; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if (abort && *abort) return false;
    if (global_ns() - t0 > limit_ns) return false;
  }
  return false;
}

// limit_ns: how long one wait may last.  extra_tx: bytes added to what every tile's barrier
// expects, 0 in production; a test sets it to make the waits run out (every copy still lands,
// the barrier just never completes) and so exercise the give-up path without any fault.
template <int M, int VAR, int TK, int T, int S, int NT>
__global__ void __launch_bounds__(NT, 1) outer_step_bulk_kernel(const OuterArgs a, unsigned *status,
                                                                unsigned long long limit_ns, unsigned extra_tx) {
  using L = BulkStage<M, VAR, TK, T>;
  static_assert(T % 8 == 0 && L::kBytes % 16 == 0, "rows must be multiples of 16 bytes");
  static_assert(S >= 3, "ring needs a current, a loading and a draining stage");
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ unsigned long long full[S];
  __shared__ volatile unsigned s_abort;

  const long long ntiles = a.P / T;
  const int tid = threadIdx.x;
  // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
  const long long mine = ntiles > blockIdx.x ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  constexpr int LOOK = S - 2;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) mbar_init(&full[s], 1);
    s_abort = 0;
    fence_mbar_init();
  }
  __syncthreads();

  const unsigned short *theta16 = reinterpret_cast<const unsigned short *>(a.theta);
  const float *theta32 = reinterpret_cast<const float *>(a.theta);

  auto issue_loads = [&](long long j) {
    unsigned char *st = smem + (size_t)(j % S) * L::kBytes;
    unsigned long long *bar = &full[j % S];
    const long long i0 = (blockIdx.x + j * gridDim.x) * T;
    mbar_expect_tx(bar, L::kLoadBytes + extra_tx);
#pragma unroll
    for (int m = 0; m < M; ++m) {
      const long long at = m * a.stride + i0;
      if (TK == TK_F32) bulk_load(st + L::offX + m * L::kThetaBytes, theta32 + at, L::kThetaBytes, bar);
      else if (TK == TK_BF16) bulk_load(st + L::offX + m * L::kThetaBytes, theta16 + at, L::kThetaBytes, bar);
      else bulk_load(st + L::offX + m * L::kThetaBytes, a.master + at, L::kThetaBytes, bar);
      bulk_load(st + L::offS + m * L::kRow, a.start + at, L::kRow, bar);
      bulk_load(st + L::offB + m * L::kRow, a.mom + at, L::kRow, bar);
      if (VAR == VAR_EAGER) bulk_load(st + L::offPL + m * L::kRow, a.dpl + at, L::kRow, bar);
    }
    if (VAR != VAR_STANDARD) bulk_load(st + L::offPA, a.dpa + i0, L::kRow, bar);
  };
  auto issue_stores = [&](long long j) {
    unsigned char *st = smem + (size_t)(j % S) * L::kBytes;
    const long long i0 = (blockIdx.x + j * gridDim.x) * T;
#pragma unroll
    for (int m = 0; m < M; ++m) {
      const long long at = m * a.stride + i0;
      if (TK == TK_F32) bulk_store(reinterpret_cast<float *>(a.theta) + at, st + L::offX + m * L::kThetaBytes, L::kThetaBytes);
      else if (TK == TK_BF16) bulk_store(reinterpret_cast<unsigned short *>(a.theta) + at, st + L::offX + m * L::kThetaBytes, L::kThetaBytes);
      else {
        bulk_store(a.master + at, st + L::offX + m * L::kThetaBytes, L::kThetaBytes);
        bulk_store(reinterpret_cast<unsigned short *>(a.theta) + at, st + L::offC + m * 2 * T, 2 * T);
      }
      bulk_store(a.start + at, st + L::offS + m * L::kRow, L::kRow);
      bulk_store(a.mom + at, st + L::offB + m * L::kRow, L::kRow);
      if (VAR == VAR_EAGER) bulk_store(a.dpl + at, st + L::offPL + m * L::kRow, L::kRow);
    }
    if (VAR != VAR_STANDARD) bulk_store(a.dpa + i0, st + L::offPA, L::kRow);
    bulk_commit();
  };

  if (tid == 0) {
    for (long long j = 0; j < LOOK && j < mine; ++j) issue_loads(j);
  }

  bool aborted = false;
  for (long long j = 0; j < mine; ++j) {
    if (tid == 0 && j + LOOK < mine) {
      bulk_wait_read<1>(); // the group that drained stage (j + LOOK) % S is tile j-2's
      issue_loads(j + LOOK);
    }
    // wait for this tile's rows, bounded
    {
      const bool ok = mbar_wait_bounded(&full[j % S], (unsigned)((j / S) & 1), limit_ns, &s_abort);
      if (!ok) s_abort = 1;
      else {
        unsigned char *st = smem + (size_t)(j % S) * L::kBytes;
        // in-place update of the tile: thread t owns columns t, t + NT, ... of 4 indices each
        for (int c = tid; c < T / 4; c += NT) {
          float s[M][4], d[M][4], b[M][4], pl[M][4], pa[4], mean[4];
#pragma unroll
          for (int m = 0; m < M; ++m) {
            if (TK == TK_BF16) {
              uint2 t2 = *reinterpret_cast<const uint2 *>(st + L::offX + m * L::kThetaBytes + c * 8);
              d[m][0] = bf16_bits_to_f32(t2.x & 0xffffu); d[m][1] = bf16_bits_to_f32(t2.x >> 16);
              d[m][2] = bf16_bits_to_f32(t2.y & 0xffffu); d[m][3] = bf16_bits_to_f32(t2.y >> 16);
            } else {
              float4 t4 = *reinterpret_cast<const float4 *>(st + L::offX + m * L::kThetaBytes + c * 16);
              d[m][0] = t4.x; d[m][1] = t4.y; d[m][2] = t4.z; d[m][3] = t4.w;
            }
            float4 t4 = *reinterpret_cast<const float4 *>(st + L::offS + m * L::kRow + c * 16);
            s[m][0] = t4.x; s[m][1] = t4.y; s[m][2] = t4.z; s[m][3] = t4.w;
            t4 = *reinterpret_cast<const float4 *>(st + L::offB + m * L::kRow + c * 16);
            b[m][0] = t4.x; b[m][1] = t4.y; b[m][2] = t4.z; b[m][3] = t4.w;
            if (VAR == VAR_EAGER) {
              t4 = *reinterpret_cast<const float4 *>(st + L::offPL + m * L::kRow + c * 16);
              pl[m][0] = t4.x; pl[m][1] = t4.y; pl[m][2] = t4.z; pl[m][3] = t4.w;
            }
          }
          if (VAR != VAR_STANDARD) {
            float4 t4 = *reinterpret_cast<const float4 *>(st + L::offPA + c * 16);
            pa[0] = t4.x; pa[1] = t4.y; pa[2] = t4.z; pa[3] = t4.w;
          }
          // Alg. 1-3 lines 7-8
#pragma unroll
          for (int m = 0; m < M; ++m) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              d[m][e] = s[m][e] - d[m][e];
              mean[e] = (m == 0) ? d[m][e] : mean[e] + d[m][e];
            }
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) mean[e] = mean[e] / a.fM;
#pragma unroll
          for (int m = 0; m < M; ++m) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float g;
              if (VAR == VAR_STANDARD) g = mean[e];
              else if (VAR == VAR_DELAYED) g = pa[e];
              else {
                float t = d[m][e] - pl[m][e]; // Alg. 3 line 11
                t = t / a.fM;
                g = t + pa[e];
              }
              nesterov(g, a.eta, a.mu, b[m][e], s[m][e]);
            }
            *reinterpret_cast<float4 *>(st + L::offS + m * L::kRow + c * 16) = make_float4(s[m][0], s[m][1], s[m][2], s[m][3]);
            *reinterpret_cast<float4 *>(st + L::offB + m * L::kRow + c * 16) = make_float4(b[m][0], b[m][1], b[m][2], b[m][3]);
            if (VAR == VAR_EAGER)
              *reinterpret_cast<float4 *>(st + L::offPL + m * L::kRow + c * 16) = make_float4(d[m][0], d[m][1], d[m][2], d[m][3]);
            if (TK != TK_BF16)
              *reinterpret_cast<float4 *>(st + L::offX + m * L::kThetaBytes + c * 16) = make_float4(s[m][0], s[m][1], s[m][2], s[m][3]);
            if (TK != TK_F32) {
              uint2 o;
              o.x = (unsigned)f32_to_bf16_bits(s[m][0]) | ((unsigned)f32_to_bf16_bits(s[m][1]) << 16);
              o.y = (unsigned)f32_to_bf16_bits(s[m][2]) | ((unsigned)f32_to_bf16_bits(s[m][3]) << 16);
              unsigned char *dst = (TK == TK_BF16) ? st + L::offX + m * L::kThetaBytes + c * 8 : st + L::offC + m * 2 * T + c * 8;
              *reinterpret_cast<uint2 *>(dst) = o;
            }
          }
          if (VAR != VAR_STANDARD) *reinterpret_cast<float4 *>(st + L::offPA + c * 16) = make_float4(mean[0], mean[1], mean[2], mean[3]);
        }
      }
    }
    fence_async_smem(); // generic-proxy writes above -> visible to the bulk store's async proxy
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
  // ragged remainder (fewer than T indices): plain loads and stores by the last CTA
  if (blockIdx.x == gridDim.x - 1 && !aborted) {
    const long long done = ntiles * T;
    const long long nvec = (a.P - done) / 4;
    for (long long j = tid; j < nvec; j += NT) outer_column<M, 1, VAR, TK, 4>(a, done + j * 4, 0, true);
    for (long long i = done + nvec * 4 + tid; i < a.P; i += NT) outer_column_rt<VAR, TK, false, 1>(a, i);
  }
}

} // namespace diloco
