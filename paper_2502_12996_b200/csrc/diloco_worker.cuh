// One worker's share of the outer step, for deployments where the M replicas of Algorithms
// 1-3 live on M different GPUs (one process per GPU) and line 8's mean really is an
// all-reduce.  The worker holds one replica; what crosses the network is its local outer
// gradient Delta_m (`send`) and, D outer steps later, the element-wise SUM over all workers
// (`recv`), which the kernel divides by M itself so that the arithmetic is the fused
// kernel's: Delta = (sum_m Delta_m) / M, then lines 10-12.  With the sum formed in the order
// m = 0 .. M-1 the results are bit-identical to the M-replica kernel (for M = 2 any order
// is that order).  Same rules as diloco_kernels.cuh: one column per thread, all loads first,
// no FMA contraction.
#pragma once
#include "diloco_kernels.cuh"

namespace diloco {

enum {
  WMODE_SEND_ONLY = 0,  // standard, before the blocking all-reduce: send = Delta_m, state untouched
  WMODE_RECORD = 1,     // delayed / eager while nothing has arrived yet: send, restart from theta
  WMODE_APPLY = 2,      // standard, after the all-reduce: OuterOpt with Delta = recv / M
  WMODE_APPLY_SEND = 3  // delayed / eager: OuterOpt with the sum that arrived, send the new Delta_m
};

struct WorkerArgs {
  void *theta;       // [stride] fp32 or bf16
  float *master;     // [stride] or nullptr
  float *start;      // [stride] s_m
  float *dpl;        // [stride] Delta_m^(t-DH) of this worker (eager), current ring slot
  float *mom;        // [stride] b_m
  const float *recv; // [stride] sum over workers of the Delta_m sent D outer steps ago
  float *send;       // [stride] out: this worker's Delta_m of this step
  long long P;
  float eta, mu, fM; // fM = number of workers M
};

template <int TK, int V>
__device__ __forceinline__ void worker_load_theta(const WorkerArgs &a, long long i, float (&x)[V]) {
  if (TK == TK_F32) F32Vec<V>::load(reinterpret_cast<const float *>(a.theta) + i, x);
  else if (TK == TK_BF16) BF16Vec<V>::load(reinterpret_cast<const unsigned short *>(a.theta) + i, x);
  else F32Vec<V>::load(a.master + i, x);
}
template <int TK, int V>
__device__ __forceinline__ void worker_store_theta(const WorkerArgs &a, long long i, const float (&n)[V]) {
  if (TK == TK_F32) {
    F32Vec<V>::store(reinterpret_cast<float *>(a.theta) + i, n);
  } else if (TK == TK_BF16) {
    BF16Vec<V>::store(reinterpret_cast<unsigned short *>(a.theta) + i, n);
  } else {
    F32Vec<V>::store(a.master + i, n);
    BF16Vec<V>::store(reinterpret_cast<unsigned short *>(a.theta) + i, n);
  }
}

template <int MODE, int VAR, int TK, int V>
__device__ __forceinline__ void worker_column(const WorkerArgs &a, long long i) {
  constexpr bool kApply = MODE == WMODE_APPLY || MODE == WMODE_APPLY_SEND;
  constexpr bool kSend = MODE != WMODE_APPLY;
  float s[V], x[V], b[V], pl[V], sum[V], d[V];
  F32Vec<V>::load(a.start + i, s);
  if (kSend) worker_load_theta<TK, V>(a, i, x);
  if (kApply) {
    F32Vec<V>::load(a.mom + i, b);
    F32Vec<V>::load(a.recv + i, sum);
    if (MODE == WMODE_APPLY_SEND && VAR == VAR_EAGER) F32Vec<V>::load(a.dpl + i, pl);
  }
  if (kSend) {
#pragma unroll
    for (int e = 0; e < V; ++e) d[e] = s[e] - x[e]; // Alg. 1-3 line 7
    F32Vec<V>::store(a.send + i, d);               // line 8: what this worker contributes
  }
  if (MODE == WMODE_RECORD) {
    F32Vec<V>::store(a.start + i, x);              // t <= DH: nothing to apply, restart from theta_m
    if (VAR == VAR_EAGER) F32Vec<V>::store(a.dpl + i, d);
  }
  if (kApply) {
#pragma unroll
    for (int e = 0; e < V; ++e) {
      const float mean = sum[e] / a.fM;            // the all-reduce delivered the sum
      float g;
      if (VAR == VAR_EAGER && MODE == WMODE_APPLY_SEND) {
        float t = d[e] - pl[e];                    // Alg. 3 line 11
        t = t / a.fM;
        g = t + mean;
      } else {
        g = mean;                                  // Alg. 1 line 10 / Alg. 2 line 11
      }
      nesterov(g, a.eta, a.mu, b[e], s[e]);
    }
    F32Vec<V>::store(a.mom + i, b);
    F32Vec<V>::store(a.start + i, s);
    worker_store_theta<TK, V>(a, i, s);
    if (MODE == WMODE_APPLY_SEND && VAR == VAR_EAGER) F32Vec<V>::store(a.dpl + i, d);
  }
}

template <int MODE, int VAR, int TK, int V, int NT>
__global__ void __launch_bounds__(NT, 4) worker_outer_kernel(const WorkerArgs a) {
  const long long nvec = a.P / V;
  const long long j = (long long)blockIdx.x * NT + threadIdx.x;
  if (j < nvec) worker_column<MODE, VAR, TK, V>(a, j * V);
  if (blockIdx.x == gridDim.x - 1) {
    const long long i = nvec * V + threadIdx.x;
    if (i < a.P) worker_column<MODE, VAR, TK, 1>(a, i);
  }
}

} // namespace diloco
