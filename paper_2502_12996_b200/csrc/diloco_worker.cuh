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

#ifndef DILOCO_WORKER_MAX_WORLD
#define DILOCO_WORKER_MAX_WORLD 64 // workers whose payloads one quantised apply can gather
#endif

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

// ---------------------------------------------------------------- quantised wire, worker form
// What crosses the network is each worker's Delta_m as EXMY codes plus one fp32 word (its
// max |Delta_m|); every worker gathers all M payloads and forms the mean itself:
//   Delta = ( sum_{m = 0 .. M-1, in order} scale_m * value(code_m) ) / M
// which is the fused quantised kernel's line 8 exactly, for any M (a gather keeps the order).
// Code of an element: sign << (X+Y) | exponent field << Y | mantissa; codes of at most 4 bits
// are packed two per byte (element 2j in bits 0-3), wider codes take one byte.
namespace diloco {

struct WorkerQArgs {
  WorkerArgs w;                 // state pointers, P, eta, mu, fM (recv / send unused)
  const unsigned char *precv;   // [world, pstride] gathered payloads of the step that is due
  const unsigned *amax_recv;    // [world] their max |Delta_m| words
  long long pstride;            // bytes between payload rows
  unsigned char *psend;         // out: this worker's payload
  const unsigned *amax_send;    // this worker's max |Delta_m| (reduced by delta_amax_kernel before)
  int world;                    // M
  int man_bits, emin, bias, code_bits; // Y, 1 - bias, bias, X + Y (sign excluded)
  float fmt_max;
  int packed;                   // 1: two codes per byte
};

// EXMY code (without sign) and sign of y; same rounding as exmy_round
__device__ __forceinline__ unsigned exmy_encode(float y, const WorkerQArgs &a) {
  const unsigned sign = (__float_as_uint(y) >> 31) << a.code_bits;
  const unsigned top = (1u << a.code_bits) - 1u; // all exponent and mantissa bits set
  const float ay = fabsf(y);
  if (ay == 0.f) return sign;
  if (!(ay > 0.f)) return 0u;                    // NaN has no code; it arises only when this worker's scale is NaN
                                                 // or infinite, and code 0 (+0) times that scale decodes to NaN
  const float ac = fminf(ay, a.fmt_max);         // saturating
  int E = (int)((__float_as_uint(ac) >> 23) & 0xffu) - 127;
  E = max(E, a.emin);
  const int qe = E - a.man_bits;
  const float n = ac * __uint_as_float((unsigned)(127 - qe) << 23);
  float r = rintf(n);
  if (a.man_bits == 0 && n == 1.5f) r = ((E + a.bias) & 1) ? 2.f : 1.f;
  const float q = r * __uint_as_float((unsigned)(127 + qe) << 23);
  if (q >= a.fmt_max) return sign | top;
  const unsigned ri = (unsigned)r;
  const unsigned one = 1u << a.man_bits;
  unsigned code;
  if (ri < one) code = ri;                                        // subnormal: exponent field 0 (E == emin here)
  else if (ri == 2u * one) code = (unsigned)(E + a.bias + 1) << a.man_bits; // rounded up into the next binade
  else code = ((unsigned)(E + a.bias) << a.man_bits) | (ri - one);
  return sign | code;
}

__device__ __forceinline__ float exmy_decode(unsigned code, const WorkerQArgs &a) {
  const unsigned e = (code >> a.man_bits) & ((1u << (a.code_bits - a.man_bits)) - 1u);
  const unsigned m = code & ((1u << a.man_bits) - 1u);
  const int ex = e == 0 ? a.emin - a.man_bits : (int)e - a.bias - a.man_bits;
  const float v = (float)(e == 0 ? m : m + (1u << a.man_bits)) * __uint_as_float((unsigned)(127 + ex) << 23);
  return (code >> a.code_bits) & 1u ? -v : v;
}

__device__ __forceinline__ float amax_to_scale(unsigned bits, float fmt_max) {
  return amax_bits_to_scale(bits, fmt_max); // zero or underflowing scale -> 1; NaN and infinity propagate
}

// N consecutive elements starting at index i (N = 4 with i % 4 == 0, or N = 1): the codes of row m
template <int N>
__device__ __forceinline__ void load_codes(const unsigned char *row, long long i, int packed, unsigned (&c)[N]) {
  if (N == 4) {
    if (packed) {
      const unsigned t = *reinterpret_cast<const unsigned short *>(row + i / 2);
#pragma unroll
      for (int e = 0; e < N; ++e) c[e] = (t >> (4 * e)) & 15u;
    } else {
      const unsigned t = *reinterpret_cast<const unsigned *>(row + i);
#pragma unroll
      for (int e = 0; e < N; ++e) c[e] = (t >> (8 * e)) & 255u;
    }
  } else {
    c[0] = packed ? (row[i / 2] >> (4 * (i & 1))) & 15u : row[i];
  }
}

// One column of N elements.  scales: shared array of the world's scales; my_scale: this worker's.
template <int MODE, int VAR, int TK, int N>
__device__ __forceinline__ void worker_q_column(const WorkerQArgs &q, long long i, const float *scales, float my_scale,
                                                unsigned (&codes_out)[N]) {
  const WorkerArgs &a = q.w;
  constexpr bool kApply = MODE == WMODE_APPLY || MODE == WMODE_APPLY_SEND;
  constexpr bool kSend = MODE != WMODE_APPLY;
  float s[N], x[N], b[N], pl[N], sum[N], d[N];
  F32Vec<N>::load(a.start + i, s);
  if (kSend) worker_load_theta<TK, N>(a, i, x);
  if (kApply) {
    F32Vec<N>::load(a.mom + i, b);
    if (MODE == WMODE_APPLY_SEND && VAR == VAR_EAGER) F32Vec<N>::load(a.dpl + i, pl);
    for (int m = 0; m < q.world; ++m) { // line 8 from the gathered payloads, worker order
      unsigned c[N];
      load_codes<N>(q.precv + m * q.pstride, i, q.packed, c);
#pragma unroll
      for (int e = 0; e < N; ++e) {
        const float w = exmy_decode(c[e], q) * scales[m];
        sum[e] = (m == 0) ? w : sum[e] + w;
      }
    }
  }
  if (kSend) {
#pragma unroll
    for (int e = 0; e < N; ++e) {
      d[e] = s[e] - x[e];                          // Alg. 1-3 line 7
      codes_out[e] = exmy_encode(d[e] / my_scale, q);
    }
  }
  if (MODE == WMODE_RECORD) {
    F32Vec<N>::store(a.start + i, x);
    if (VAR == VAR_EAGER) F32Vec<N>::store(a.dpl + i, d);
  }
  if (kApply) {
#pragma unroll
    for (int e = 0; e < N; ++e) {
      const float mean = sum[e] / a.fM;
      float g;
      if (VAR == VAR_EAGER && MODE == WMODE_APPLY_SEND) {
        float t = d[e] - pl[e];                    // Alg. 3 line 11: local terms in full precision
        t = t / a.fM;
        g = t + mean;
      } else {
        g = mean;
      }
      nesterov(g, a.eta, a.mu, b[e], s[e]);
    }
    F32Vec<N>::store(a.mom + i, b);
    F32Vec<N>::store(a.start + i, s);
    worker_store_theta<TK, N>(a, i, s);
    if (MODE == WMODE_APPLY_SEND && VAR == VAR_EAGER) F32Vec<N>::store(a.dpl + i, d);
  }
}

template <int MODE, int VAR, int TK, int NT>
__global__ void __launch_bounds__(NT, 4) worker_quantized_kernel(const WorkerQArgs q) {
  constexpr bool kApply = MODE == WMODE_APPLY || MODE == WMODE_APPLY_SEND;
  constexpr bool kSend = MODE != WMODE_APPLY;
  __shared__ float scales[DILOCO_WORKER_MAX_WORLD];
  if (kApply) {
    for (int m = threadIdx.x; m < q.world; m += NT) scales[m] = amax_to_scale(q.amax_recv[m], q.fmt_max);
    __syncthreads();
  }
  const float my_scale = kSend ? amax_to_scale(*q.amax_send, q.fmt_max) : 1.f;
  const long long nvec = q.w.P / 4;
  const long long j = (long long)blockIdx.x * NT + threadIdx.x;
  if (j < nvec) {
    unsigned c[4];
    worker_q_column<MODE, VAR, TK, 4>(q, j * 4, scales, my_scale, c);
    if (kSend) {
      if (q.packed) *reinterpret_cast<unsigned short *>(q.psend + j * 2) = (unsigned short)(c[0] | (c[1] << 4) | (c[2] << 8) | (c[3] << 12));
      else *reinterpret_cast<unsigned *>(q.psend + j * 4) = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24);
    }
  }
  // ragged tail (P % 4 elements): one thread, so that two nibbles of a byte have one writer
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
    unsigned pending = 0;
    for (long long i = nvec * 4; i < q.w.P; ++i) {
      unsigned c[1];
      worker_q_column<MODE, VAR, TK, 1>(q, i, scales, my_scale, c);
      if (kSend) {
        if (!q.packed) q.psend[i] = (unsigned char)c[0];
        else if (i & 1) q.psend[i / 2] = (unsigned char)(pending | (c[0] << 4));
        else {
          pending = c[0];
          if (i == q.w.P - 1) q.psend[i / 2] = (unsigned char)pending; // odd P: high nibble zero
        }
      }
    }
  }
}

} // namespace diloco
