// Device code of libdiloco: the fused outer step (Algorithms 1-3, lines 7-12) and the inner
// AdamW step, register-resident "direct" form.  Compiled for sm_100a only, with
// -fmad=false: every fp32 operation below is one IEEE round-to-nearest operation, written
// in the order the algorithms state it, so results are bit-identical for any launch shape.
//
// Memory behaviour is the whole design (the path is < 1 flop/byte): each state word is read
// once and written once, with 64- or 128-bit accesses that a warp issues as 256 or 512
// contiguous bytes per row, all loads of a column issued before its first dependent use so
// that one thread keeps up to 17 vectors in flight, no register spills (a spilling variant
// measured 30 % slower), and streaming cache hints since nothing is reused.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace diloco {

enum { VAR_STANDARD = 0, VAR_DELAYED = 1, VAR_EAGER = 2 };
enum { TK_F32 = 0, TK_BF16 = 1, TK_MASTER_BF16 = 2 };
enum { GK_F32 = 0, GK_BF16 = 1 };


struct OuterArgs {
  void *theta;     // [M, stride] fp32 or bf16
  float *master;   // [M, stride] or nullptr
  float *start;    // [M, stride]
  float *dpl;      // [M, stride] Delta_m^(t-H) (eager)
  float *dpa;      // [stride]    Delta^(t-H)   (delayed, eager)
  float *mom;      // [M, stride] b_m
  long long P;      // indices [0, P) are processed (pointers already offset for fragments)
  long long stride; // elements between replicas
  float eta, mu, fM;
  int M;            // used by the runtime-M kernels only
  int groups, wpg;  // warp-split kernel: column groups per block (1 or 2) and warps per group, set by its launcher
  // quantised communication of the outer gradients (Q kernels only)
  const unsigned *amax; // [M] bit patterns of max_i |Delta_m[i]|, written by delta_amax_kernel
  float fmt_max;        // largest EXMY value
  int comm;             // COMM_BF16 or COMM_EXMY
  int man_bits;         // Y
  int emin;             // 1 - bias: exponent of the smallest normal
  int bias;             // 2^(X-1) - 1
};

enum { COMM_F32 = 0, COMM_BF16 = 1, COMM_EXMY = 2 };

struct AdamArgs {
  void *theta;
  float *master;
  const void *grads;
  float *m, *v;
  long long P, stride, gstride;
  float lr, beta1, beta2, omb1, omb2, c1, c2, eps, wd;
};

// ---------------------------------------------------------------- vector access helpers
// V consecutive elements starting at an index that is a multiple of V.
// Cache policy of the streaming accesses.  Default (no hint) measured 2-3 % faster than
// ld.global.cs / st.global.cs and than ld.global.nc here: each line is written back ~1 us after
// it was read, and leaving it in L2 until then lets the store hit it (L2 hit rate ~50 %).
#ifndef DILOCO_LDG
#define DILOCO_LDG(p) (*(p))
#endif
#ifndef DILOCO_STG
#define DILOCO_STG(p, v) (*(p) = (v))
#endif
template <int V> struct F32Vec;
template <> struct F32Vec<4> {
  static __device__ __forceinline__ void load(const float *p, float (&r)[4]) {
    float4 t = DILOCO_LDG(reinterpret_cast<const float4 *>(p));
    r[0] = t.x; r[1] = t.y; r[2] = t.z; r[3] = t.w;
  }
  static __device__ __forceinline__ void load_cached(const float *p, float (&r)[4]) {
    float4 t = *reinterpret_cast<const float4 *>(p);
    r[0] = t.x; r[1] = t.y; r[2] = t.z; r[3] = t.w;
  }
  static __device__ __forceinline__ void store(float *p, const float (&r)[4]) {
    DILOCO_STG(reinterpret_cast<float4 *>(p), make_float4(r[0], r[1], r[2], r[3]));
  }
};
// 256-bit accesses (sm_100: ld/st.global.v8.f32), 32-byte aligned
template <> struct F32Vec<8> {
  static __device__ __forceinline__ void load(const float *p, float (&r)[8]) {
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
                 : "l"(p));
  }
  static __device__ __forceinline__ void load_cached(const float *p, float (&r)[8]) {
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
                 : "l"(p));
  }
  static __device__ __forceinline__ void store(float *p, const float (&r)[8]) {
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(r[0]), "f"(r[1]), "f"(r[2]),
                 "f"(r[3]), "f"(r[4]), "f"(r[5]), "f"(r[6]), "f"(r[7])
                 : "memory");
  }
};
template <> struct F32Vec<2> {
  static __device__ __forceinline__ void load(const float *p, float (&r)[2]) {
    float2 t = DILOCO_LDG(reinterpret_cast<const float2 *>(p));
    r[0] = t.x; r[1] = t.y;
  }
  static __device__ __forceinline__ void load_cached(const float *p, float (&r)[2]) {
    float2 t = *reinterpret_cast<const float2 *>(p);
    r[0] = t.x; r[1] = t.y;
  }
  static __device__ __forceinline__ void store(float *p, const float (&r)[2]) {
    DILOCO_STG(reinterpret_cast<float2 *>(p), make_float2(r[0], r[1]));
  }
};
template <> struct F32Vec<1> {
  static __device__ __forceinline__ void load(const float *p, float (&r)[1]) { r[0] = DILOCO_LDG(p); }
  static __device__ __forceinline__ void load_cached(const float *p, float (&r)[1]) { r[0] = *p; }
  static __device__ __forceinline__ void store(float *p, const float (&r)[1]) { DILOCO_STG(p, r[0]); }
};

__device__ __forceinline__ float bf16_bits_to_f32(unsigned short h) { return __uint_as_float(((unsigned)h) << 16); }
__device__ __forceinline__ unsigned short f32_to_bf16_bits(float f) {
  return __bfloat16_as_ushort(__float2bfloat16_rn(f)); // round-to-nearest-even
}
// two values in one conversion instruction: lo in bits 0-15, hi in bits 16-31 (same rounding)
__device__ __forceinline__ unsigned f32x2_to_bf16x2_bits(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const unsigned *>(&t);
}

template <int V> struct BF16Vec;
template <> struct BF16Vec<8> {
  static __device__ __forceinline__ void load(const unsigned short *p, float (&r)[8], bool cached = false) {
    uint4 t = cached ? *reinterpret_cast<const uint4 *>(p) : DILOCO_LDG(reinterpret_cast<const uint4 *>(p));
    const unsigned w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      r[2 * k] = bf16_bits_to_f32(w[k] & 0xffffu);
      r[2 * k + 1] = bf16_bits_to_f32(w[k] >> 16);
    }
  }
  static __device__ __forceinline__ void store(unsigned short *p, const float (&r)[8]) {
    unsigned w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) w[k] = f32x2_to_bf16x2_bits(r[2 * k], r[2 * k + 1]);
    DILOCO_STG(reinterpret_cast<uint4 *>(p), make_uint4(w[0], w[1], w[2], w[3]));
  }
};
template <> struct BF16Vec<4> {
  static __device__ __forceinline__ void load(const unsigned short *p, float (&r)[4], bool cached = false) {
    uint2 t = cached ? *reinterpret_cast<const uint2 *>(p) : DILOCO_LDG(reinterpret_cast<const uint2 *>(p));
    r[0] = bf16_bits_to_f32(t.x & 0xffffu); r[1] = bf16_bits_to_f32(t.x >> 16);
    r[2] = bf16_bits_to_f32(t.y & 0xffffu); r[3] = bf16_bits_to_f32(t.y >> 16);
  }
  static __device__ __forceinline__ void store(unsigned short *p, const float (&r)[4]) {
    uint2 t;
    t.x = f32x2_to_bf16x2_bits(r[0], r[1]);
    t.y = f32x2_to_bf16x2_bits(r[2], r[3]);
    DILOCO_STG(reinterpret_cast<uint2 *>(p), t);
  }
};
template <> struct BF16Vec<2> {
  static __device__ __forceinline__ void load(const unsigned short *p, float (&r)[2], bool cached = false) {
    unsigned t = cached ? *reinterpret_cast<const unsigned *>(p) : DILOCO_LDG(reinterpret_cast<const unsigned *>(p));
    r[0] = bf16_bits_to_f32(t & 0xffffu); r[1] = bf16_bits_to_f32(t >> 16);
  }
  static __device__ __forceinline__ void store(unsigned short *p, const float (&r)[2]) {
    DILOCO_STG(reinterpret_cast<unsigned *>(p), f32x2_to_bf16x2_bits(r[0], r[1]));
  }
};
template <> struct BF16Vec<1> {
  static __device__ __forceinline__ void load(const unsigned short *p, float (&r)[1], bool cached = false) {
    unsigned short t = cached ? *p : DILOCO_LDG(p);
    r[0] = bf16_bits_to_f32(t);
  }
  static __device__ __forceinline__ void store(unsigned short *p, const float (&r)[1]) { DILOCO_STG(p, f32_to_bf16_bits(r[0])); }
};

// theta_m^(t) as the fp32 value the algorithms operate on
template <int TK, int V>
__device__ __forceinline__ void load_theta(const OuterArgs &a, long long at, float (&x)[V], bool cached = false) {
  if (TK == TK_F32) {
    if (cached) F32Vec<V>::load_cached(reinterpret_cast<const float *>(a.theta) + at, x);
    else F32Vec<V>::load(reinterpret_cast<const float *>(a.theta) + at, x);
  } else if (TK == TK_BF16) {
    BF16Vec<V>::load(reinterpret_cast<const unsigned short *>(a.theta) + at, x, cached);
  } else {
    if (cached) F32Vec<V>::load_cached(a.master + at, x);
    else F32Vec<V>::load(a.master + at, x);
  }
}
template <int TK, int V>
__device__ __forceinline__ void store_theta(const OuterArgs &a, long long at, const float (&n)[V]) {
  if (TK == TK_F32) {
    F32Vec<V>::store(reinterpret_cast<float *>(a.theta) + at, n);
  } else if (TK == TK_BF16) {
    BF16Vec<V>::store(reinterpret_cast<unsigned short *>(a.theta) + at, n);
  } else {
    F32Vec<V>::store(a.master + at, n);
    BF16Vec<V>::store(reinterpret_cast<unsigned short *>(a.theta) + at, n);
  }
}

// OuterOpt(theta^(t-H), g): SGD with Nesterov momentum.  b <- mu b + g ; s <- s - eta (g + mu b)
__device__ __forceinline__ void nesterov(float g, float eta, float mu, float &b, float &s) {
  float nb = mu * b;
  nb = nb + g;
  float u = mu * nb;
  u = g + u;
  u = eta * u;
  s = s - u;
  b = nb;
}

// ---------------------------------------------------------------- wire formats of Delta_m
// Section 3, "Quantized Communication": the all-reduce operand is rounded to bfloat16 or to
// an EXMY float (1 sign, X exponent, Y mantissa bits, bias 2^(X-1)-1, subnormals, every code
// finite, round to nearest with ties to the even code, saturating) after scaling each
// replica's vector so that its largest magnitude lands on the format's largest value.
// All scalings below are by powers of two and therefore exact in fp32.
__device__ __forceinline__ float exmy_round(float y, const OuterArgs &a) {
  const float ay = fabsf(y);
  if (!(ay > 0.f)) return y;                                // zero keeps its sign, NaN stays NaN
  const float ac = fminf(ay, a.fmt_max);                    // saturating: the largest value is a fixed point of
                                                            // the rounding, and infinity never reaches the exponent
  int E = (int)((__float_as_uint(ac) >> 23) & 0xffu) - 127; // binade of |y| (fp32 subnormals: clamped next)
  E = max(E, a.emin);                                       // below the smallest normal the spacing is fixed
  const int qe = E - a.man_bits;                            // spacing = 2^qe
  const float n = ac * __uint_as_float((unsigned)(127 - qe) << 23); // |y| / spacing, exact
  float r = rintf(n);                                       // halves go to the even integer = even code ...
  if (a.man_bits == 0 && n == 1.5f) r = ((E + a.bias) & 1) ? 2.f : 1.f; // ... except with no mantissa bits,
                                                            // where the code's parity is the exponent field's
  const float q = r * __uint_as_float((unsigned)(127 + qe) << 23);
  return copysignf(q, y);
}

// The per-replica scale: max |Delta_m| maps to the format's largest value; a scale of zero
// (the replica did not move, or so little that the quotient underflows) is replaced by 1.  The
// maximum propagates NaN, so a replica whose outer gradient holds a NaN or an infinity gets a
// NaN or infinite scale and everything it sends decodes to NaN (x / NaN, 0 * inf).
__device__ __forceinline__ float amax_bits_to_scale(unsigned bits, float fmt_max) {
  const float scale = __uint_as_float(bits) / fmt_max;
  return scale == 0.f ? 1.f : scale;
}
__device__ __forceinline__ float comm_scale(const OuterArgs &a, int m) {
  if (a.comm != COMM_EXMY) return 1.f;
  return amax_bits_to_scale(a.amax[m], a.fmt_max);
}

// what replica m puts on the wire for one element of its outer gradient
__device__ __forceinline__ float comm_round(float d, float scale, const OuterArgs &a) {
  if (a.comm == COMM_BF16) return bf16_bits_to_f32(f32_to_bf16_bits(d));
  const float y = d / scale;
  return exmy_round(y, a) * scale;
}

// Pass 1 of a quantised step: amax[m] = max_i |s_m[i] - theta_m[i]| (fp32, exact: max is
// order-free).  grid = (blocks, M).  The maximum is taken over the BIT PATTERNS of |Delta|:
// non-negative floats order like their bit patterns, infinity sits above every finite value
// and every NaN pattern above infinity, so one NaN element makes the result NaN.
template <int TK, int NT, int U>
__global__ void __launch_bounds__(NT) delta_amax_kernel(const OuterArgs a, unsigned *amax) {
  const int m = blockIdx.y;
  const long long nvec = a.P / 4;
  unsigned best = 0u;
  for (long long j0 = (long long)blockIdx.x * (NT * U) + threadIdx.x; j0 < nvec; j0 += (long long)gridDim.x * (NT * U)) {
    float s[U][4], x[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long j = j0 + (long long)u * NT;
      if (j < nvec) {
        F32Vec<4>::load(a.start + m * a.stride + j * 4, s[u]);
        load_theta<TK, 4>(a, m * a.stride + j * 4, x[u]);
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[u][e] = x[u][e] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int e = 0; e < 4; ++e) best = max(best, __float_as_uint(fabsf(s[u][e] - x[u][e])));
  }
  if (blockIdx.x == 0) {
    for (long long i = nvec * 4 + threadIdx.x; i < a.P; i += NT) {
      float s[1], x[1];
      F32Vec<1>::load(a.start + m * a.stride + i, s);
      load_theta<TK, 1>(a, m * a.stride + i, x);
      best = max(best, __float_as_uint(fabsf(s[0] - x[0])));
    }
  }
  best = __reduce_max_sync(0xffffffffu, best);
  __shared__ unsigned warp_best[NT / 32];
  if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < NT / 32; ++w) best = max(best, warp_best[w]);
    atomicMax(amax + m, best);
  }
}

// ---------------------------------------------------------------- outer step, compile-time M
// One column = V consecutive parameter indices.  A thread owns R = M / G replicas
// (m0 .. m0+R-1) of its column; with G > 1 the G lanes that share a column sit CW = 32 / G
// lanes apart in one warp and pass the running sum of the local outer gradients from group
// to group with shuffles, so the mean is still the left-to-right sum m = 0 .. M-1 and every
// lane divides the same total (identical bits in all G lanes).  Splitting the replica axis
// keeps the per-thread register count of M = 8 at that of M = 4.
// (The first outer steps of a delayed / eager run, which only record, go through
// outer_column_rt<BOOT = true> for every M: they happen once per run.)
template <int R, int G, int VAR, int TK, int V, bool Q = false>
__device__ __forceinline__ void outer_column(const OuterArgs &a, long long i, int m0, bool active) {
  constexpr int CW = 32 / G;
  float s[R][V], d[R][V], b[R][V], pl[R][V], pa[V], mean[V];
  float w[R][V]; // what replica m0+r sends into the all-reduce: Delta_m, or its wire-format rounding
  if (active) {
    // Alg. 1-3 line 7 operands: theta_m^(t-H) and theta_m^(t)
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const long long at = (m0 + r) * a.stride + i;
      F32Vec<V>::load(a.start + at, s[r]);
      load_theta<TK, V>(a, at, d[r]);
      F32Vec<V>::load(a.mom + at, b[r]);
      if (VAR == VAR_EAGER) F32Vec<V>::load(a.dpl + at, pl[r]);
    }
    if (VAR != VAR_STANDARD) F32Vec<V>::load(a.dpa + i, pa);
  } else {
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int e = 0; e < V; ++e) s[r][e] = d[r][e] = 0.f;
  }
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int e = 0; e < V; ++e) d[r][e] = s[r][e] - d[r][e]; // line 7: Delta_m
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const float scale = Q ? comm_scale(a, m0 + r) : 1.f;
#pragma unroll
    for (int e = 0; e < V; ++e) w[r][e] = Q ? comm_round(d[r][e], scale, a) : d[r][e];
  }
  // line 8: Delta = (1/M) sum_m Delta_m, m in order (stands in for the all-reduce)
  if (G == 1) {
#pragma unroll
    for (int e = 0; e < V; ++e) {
      mean[e] = w[0][e];
#pragma unroll
      for (int r = 1; r < R; ++r) mean[e] = mean[e] + w[r][e];
    }
  } else {
    const int g = (threadIdx.x & 31) / CW;
#pragma unroll
    for (int e = 0; e < V; ++e) mean[e] = 0.f;
#pragma unroll
    for (int gg = 0; gg < G; ++gg) {
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const float prev = __shfl_up_sync(0xffffffffu, mean[e], CW); // running sum of groups < gg
        if (g == gg) {
          float acc = (gg == 0) ? w[0][e] : prev + w[0][e];
#pragma unroll
          for (int r = 1; r < R; ++r) acc = acc + w[r][e];
          mean[e] = acc;
        }
      }
    }
#pragma unroll
    for (int e = 0; e < V; ++e) mean[e] = __shfl_sync(0xffffffffu, mean[e], (G - 1) * CW + ((threadIdx.x & 31) % CW));
  }
#pragma unroll
  for (int e = 0; e < V; ++e) mean[e] = mean[e] / a.fM;
  if (!active) return;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const long long at = (m0 + r) * a.stride + i;
#pragma unroll
    for (int e = 0; e < V; ++e) {
      float g;
      if (VAR == VAR_STANDARD) {
        g = mean[e];                      // Alg. 1 line 10
      } else if (VAR == VAR_DELAYED) {
        g = pa[e];                        // Alg. 2 line 11
      } else {
        float t = d[r][e] - pl[r][e];     // Alg. 3 line 11
        t = t / a.fM;
        g = t + pa[e];
      }
      nesterov(g, a.eta, a.mu, b[r][e], s[r][e]);
    }
    F32Vec<V>::store(a.mom + at, b[r]);
    F32Vec<V>::store(a.start + at, s[r]);
    store_theta<TK, V>(a, at, s[r]);
    if (VAR == VAR_EAGER) F32Vec<V>::store(a.dpl + at, d[r]);
  }
  if (VAR != VAR_STANDARD && m0 == 0) F32Vec<V>::store(a.dpa + i, mean);
}

// ---------------------------------------------------------------- outer step, runtime M, one thread per column
// Two sweeps over the replicas: the first forms the mean, the second re-reads s_m and
// theta_m (L1/L2 hits: the same thread read them a few hundred cycles earlier) and updates.
// Serves the recording-only first steps (BOOT) of every M and the ragged last P % V indices of
// every kernel; the steady-state steps have the faster forms above and below.
template <int VAR, int TK, bool BOOT, int V, bool Q = false>
__device__ __forceinline__ void outer_column_rt(const OuterArgs &a, long long i) {
  float mean[V];
  for (int m = 0; m < a.M; ++m) {
    float s[V], x[V];
    F32Vec<V>::load_cached(a.start + m * a.stride + i, s);
    load_theta<TK, V>(a, m * a.stride + i, x, true);
    const float scale = Q ? comm_scale(a, m) : 1.f;
#pragma unroll
    for (int e = 0; e < V; ++e) {
      float dm = s[e] - x[e];
      if (Q) dm = comm_round(dm, scale, a);
      mean[e] = (m == 0) ? dm : mean[e] + dm;
    }
  }
#pragma unroll
  for (int e = 0; e < V; ++e) mean[e] = mean[e] / a.fM;
  float pa[V];
  if (!BOOT && VAR != VAR_STANDARD) F32Vec<V>::load(a.dpa + i, pa);
  for (int m = 0; m < a.M; ++m) {
    float s[V], x[V], d[V];
    F32Vec<V>::load_cached(a.start + m * a.stride + i, s);
    load_theta<TK, V>(a, m * a.stride + i, x, true);
#pragma unroll
    for (int e = 0; e < V; ++e) d[e] = s[e] - x[e];
    if (BOOT) {
      F32Vec<V>::store(a.start + m * a.stride + i, x);
      if (VAR == VAR_EAGER) F32Vec<V>::store(a.dpl + m * a.stride + i, d);
      continue;
    }
    float b[V], pl[V];
    F32Vec<V>::load(a.mom + m * a.stride + i, b);
    if (VAR == VAR_EAGER) F32Vec<V>::load(a.dpl + m * a.stride + i, pl);
#pragma unroll
    for (int e = 0; e < V; ++e) {
      float g;
      if (VAR == VAR_STANDARD) {
        g = mean[e];
      } else if (VAR == VAR_DELAYED) {
        g = pa[e];
      } else {
        float t = d[e] - pl[e];
        t = t / a.fM;
        g = t + pa[e];
      }
      nesterov(g, a.eta, a.mu, b[e], s[e]);
    }
    F32Vec<V>::store(a.mom + m * a.stride + i, b);
    F32Vec<V>::store(a.start + m * a.stride + i, s);
    store_theta<TK, V>(a, m * a.stride + i, s);
    if (VAR == VAR_EAGER) F32Vec<V>::store(a.dpl + m * a.stride + i, d);
  }
  if (VAR != VAR_STANDARD) F32Vec<V>::store(a.dpa + i, mean);
}

// One column per thread (per G lanes), one launch wave after the other: the hardware block
// scheduler refills an SM as soon as a CTA retires, which measured ~10 % faster than a
// persistent grid-stride loop.
// Grid: ceil(ceil(nvec / CW) * 32 / NT) blocks, nvec = P / V, CW = 32 / G.  The ragged tail
// (P % V indices) is done one index per thread by the last block with the runtime-M code.
template <int M, int G, int VAR, int TK, int V, int NT, int MINB, bool Q = false>
__global__ void __launch_bounds__(NT, MINB) outer_step_kernel(const OuterArgs a) {
  static_assert(M >= 1 && M % G == 0, "replicas must divide evenly over the lane groups");
  constexpr int CW = 32 / G;
  constexpr int R = M / G;
  const long long nvec = a.P / V;
  const long long t = (long long)blockIdx.x * NT + threadIdx.x;
  const int lane = threadIdx.x & 31;
  const long long j = (t >> 5) * CW + (lane % CW);
  const bool active = j < nvec;
  if (G > 1 || active) outer_column<R, G, VAR, TK, V, Q>(a, j * V, (lane / CW) * R, active);
  if (blockIdx.x == gridDim.x - 1) {
    const long long i = nvec * V + threadIdx.x;
    if (i < a.P) outer_column_rt<VAR, TK, false, 1, Q>(a, i);
  }
}

// The first outer steps of a delayed / eager run (t <= D H: record the gradients, restart from
// the current parameters, apply nothing), any M at run time, one column per thread.  They run
// once per training run, so one plain form serves every replica count.
template <int VAR, int TK, int V, int NT, bool Q = false>
__global__ void __launch_bounds__(NT, 4) outer_first_steps_kernel(const OuterArgs a) {
  const long long nvec = a.P / V;
  const long long j = (long long)blockIdx.x * NT + threadIdx.x;
  if (j < nvec) outer_column_rt<VAR, TK, true, V, Q>(a, j * V);
  if (blockIdx.x == gridDim.x - 1) {
    const long long i = nvec * V + threadIdx.x;
    if (i < a.P) outer_column_rt<VAR, TK, true, 1, Q>(a, i);
  }
}

// ---------------------------------------------------------------- standard step, one shared copy of s and b
// Algorithm 1 with the outer parameters and the momentum stored once instead of once per replica
// (under the standard step the M copies are bit-identical for ever: same start, same gradient).
// Per index: reads s, b and the M theta_m, writes s, b and the M theta_m: 8 M + 16 bytes instead
// of 24 M.  M at run time; the theta_m are loaded four at a time, all loads of a batch before
// the first use, and summed in the order m = 0 .. M-1.
template <int TK, int V, int U>
__device__ __forceinline__ void standard_shared_columns(const OuterArgs &a, const long long (&idx)[U]) {
  float s[U][V], b[U][V], acc[U][V];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    F32Vec<V>::load(a.start + idx[u], s[u]);
    F32Vec<V>::load(a.mom + idx[u], b[u]);
  }
  for (int m0 = 0; m0 < a.M; m0 += 4) {
    float x[4][U][V];
#pragma unroll
    for (int r = 0; r < 4; ++r)
      if (m0 + r < a.M) {
#pragma unroll
        for (int u = 0; u < U; ++u) load_theta<TK, V>(a, (m0 + r) * a.stride + idx[u], x[r][u]);
      }
#pragma unroll
    for (int r = 0; r < 4; ++r)
      if (m0 + r < a.M) {
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
          for (int e = 0; e < V; ++e) {
            const float d = s[u][e] - x[r][u][e];                     // Alg. 1 line 7
            acc[u][e] = (m0 + r == 0) ? d : acc[u][e] + d;            // line 8, replica order
          }
      }
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
#pragma unroll
    for (int e = 0; e < V; ++e) {
      const float mean = acc[u][e] / a.fM;
      nesterov(mean, a.eta, a.mu, b[u][e], s[u][e]);                  // line 10, once for all replicas
    }
    F32Vec<V>::store(a.mom + idx[u], b[u]);
    F32Vec<V>::store(a.start + idx[u], s[u]);
  }
  for (int m = 0; m < a.M; ++m)
#pragma unroll
    for (int u = 0; u < U; ++u) store_theta<TK, V>(a, m * a.stride + idx[u], s[u]);
}

// U columns per thread (columns j, j + NT, ...): with few replicas one column is only 2 + M
// vectors in flight per thread, too few to keep the memory system busy (M = 2: 6.2 TB/s).
template <int TK, int NT, int U>
__global__ void __launch_bounds__(NT, U == 1 ? 4 : 3) outer_standard_shared_kernel(const OuterArgs a) {
  constexpr int V = 4;
  const long long nvec = a.P / V;
  const long long j0 = (long long)blockIdx.x * (NT * U) + threadIdx.x;
  if (j0 + (long long)(U - 1) * NT < nvec) {
    long long idx[U];
#pragma unroll
    for (int u = 0; u < U; ++u) idx[u] = (j0 + (long long)u * NT) * V;
    standard_shared_columns<TK, V, U>(a, idx);
  } else {
    for (int u = 0; u < U; ++u) {
      const long long j = j0 + (long long)u * NT;
      if (j < nvec) {
        const long long one[1] = {j * V};
        standard_shared_columns<TK, V, 1>(a, one);
      }
    }
  }
  if (blockIdx.x == gridDim.x - 1) {
    const long long i = nvec * V + threadIdx.x;
    if (i < a.P) {
      const long long one[1] = {i};
      standard_shared_columns<TK, 1, 1>(a, one);
    }
  }
}

// ---------------------------------------------------------------- outer step, M = 8 W: a chain of W warps
// The lane-split shape of M = 8 (two half-warps of 16 columns, 4 replicas per lane, 128-bit
// accesses, no shared-memory exchange of the contributions) extended to M = 16, 24, 32: W warps
// form a group that shares 16 columns, warp k owning replicas 8k .. 8k+7.  The ordered sum runs
// down the chain: warp k adds its 8 gradients (lower half-warp first, handed to the upper one by
// shuffle) to the running sum that warp k-1 left in shared memory, leaves the new running sum
// there, and a barrier of the group's 32 W threads (a named barrier: groups do not wait for one
// another) releases the next warp.  After W steps the total is there for everybody.  Only one
// float per index travels through shared memory per step instead of all M contributions.
template <int W, int VAR, int TK, int NT, int MINB, bool Q>
__global__ void __launch_bounds__(NT, MINB) outer_step_chain_kernel(const OuterArgs a) {
  constexpr int R = 4, V = 4, CW = 16;
  constexpr int GROUPS = NT / (32 * W);           // groups of W warps per block
  static_assert(NT % (32 * W) == 0 && GROUPS >= 1 && GROUPS <= 15, "whole groups, one named barrier each");
  __shared__ float running[GROUPS][CW][V];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = warp / W, k = warp % W, half = lane / CW, col = lane % CW;
  const int m0 = k * 8 + half * R;
  const long long nvec = a.P / V;
  const long long j = ((long long)blockIdx.x * GROUPS + grp) * CW + col;
  const bool active = j < nvec;
  const long long i = j * V;
  float s[R][V], d[R][V], b[R][V], pl[R][V], pa[V], mean[V], w[R][V];
  if (active) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const long long at = (m0 + r) * a.stride + i;
      F32Vec<V>::load(a.start + at, s[r]);
      load_theta<TK, V>(a, at, d[r]);
      F32Vec<V>::load(a.mom + at, b[r]);
      if (VAR == VAR_EAGER) F32Vec<V>::load(a.dpl + at, pl[r]);
    }
    if (VAR != VAR_STANDARD) F32Vec<V>::load(a.dpa + i, pa);
  } else {
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int e = 0; e < V; ++e) s[r][e] = d[r][e] = 0.f;
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const float scale = Q ? comm_scale(a, m0 + r) : 1.f;
#pragma unroll
    for (int e = 0; e < V; ++e) {
      d[r][e] = s[r][e] - d[r][e];                                   // Alg. 1-3 line 7
      w[r][e] = Q ? comm_round(d[r][e], scale, a) : d[r][e];
    }
  }
  // line 8: the ordered sum m = 0 .. M-1, handed down the chain of warps
#pragma unroll
  for (int step = 0; step < W; ++step) {
    if (k == step) {
#pragma unroll
      for (int e = 0; e < V; ++e) {
        float acc = (step == 0) ? w[0][e] : running[grp][col][e] + w[0][e];
#pragma unroll
        for (int r = 1; r < R; ++r) acc = acc + w[r][e];
        const float lower = __shfl_up_sync(0xffffffffu, acc, CW);     // the lower half-warp's running sum
        if (half == 1) {
          acc = lower + w[0][e];
#pragma unroll
          for (int r = 1; r < R; ++r) acc = acc + w[r][e];
          running[grp][col][e] = acc;
        }
      }
    }
    asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "r"(32 * W) : "memory");
  }
#pragma unroll
  for (int e = 0; e < V; ++e) mean[e] = running[grp][col][e] / a.fM;
  if (active) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const long long at = (m0 + r) * a.stride + i;
#pragma unroll
      for (int e = 0; e < V; ++e) {
        float g;
        if (VAR == VAR_STANDARD) g = mean[e];
        else if (VAR == VAR_DELAYED) g = pa[e];
        else {
          float t = d[r][e] - pl[r][e];                              // Alg. 3 line 11
          t = t / a.fM;
          g = t + pa[e];
        }
        nesterov(g, a.eta, a.mu, b[r][e], s[r][e]);
      }
      F32Vec<V>::store(a.mom + at, b[r]);
      F32Vec<V>::store(a.start + at, s[r]);
      store_theta<TK, V>(a, at, s[r]);
      if (VAR == VAR_EAGER) F32Vec<V>::store(a.dpl + at, d[r]);
    }
    if (VAR != VAR_STANDARD && m0 == 0) F32Vec<V>::store(a.dpa + i, mean);
  }
  if (blockIdx.x == gridDim.x - 1) { // ragged tail, one index per thread
    const long long t = nvec * V + threadIdx.x;
    if (t < a.P) outer_column_rt<VAR, TK, false, 1, Q>(a, t);
  }
}

// ---------------------------------------------------------------- outer step, replica axis over warps
// Replica counts that have no compile-time shape (5, 6, 7 and everything from 9 to 64; M is a
// run-time argument).  A lane split would leave runs of 64 bytes or less per row and access
// here; instead the replica axis is split across the WARPS of a block: warp w owns replicas
// w R .. w R + R - 1 (the last warp possibly fewer) of 32 columns of V indices, so every row is
// still read and written 32 V elements at a time.  Every warp leaves what its replicas send
// (Delta_m, or its wire rounding) in shared memory, and after one barrier every thread sums
// all M contributions of its own V indices in the order m = 0 .. M-1: the same left-to-right
// sum as everywhere else.  A block holds GROUPS such groups of ceil(M / R) warps on adjacent
// columns (each with a barrier of its own), so that a block touches GROUPS x 32 V consecutive
// elements of every row: at least 1 KB per row and block measured 3 % faster than 512 bytes
// (the DRAM pages a block opens are used more fully).  Shared memory GROUPS x M x V x 32 floats.
template <int VAR, int TK, bool Q, int V, int R>
__global__ void __launch_bounds__(R <= 4 ? 512 : 256, R == 6 ? 3 : 2) outer_step_split_kernel(const OuterArgs a) {
  extern __shared__ float sent_all[];  // [groups][M][V][32]
  const int wpg = a.wpg;               // warps per group: one group = all M replicas of 32 columns
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int grp = wid >= wpg ? 1 : 0;  // at most two groups per block
  const int warp = wid - grp * wpg;
  float *sent_dyn = sent_all + grp * (a.M * V * 32);
  const int m0 = warp * R;
  const int mine = min(R, a.M - m0);   // replicas of this warp: R, fewer in the last warp
  const long long nvec = a.P / V;
  const long long j = ((long long)blockIdx.x * a.groups + grp) * 32 + lane;
  const bool active = j < nvec;
  const long long i = j * V;
  float s[R][V], d[R][V], b[R][V], pl[R][V], pa[V], mean[V];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    if (active && r < mine) {
      const long long at = (m0 + r) * a.stride + i;
      F32Vec<V>::load(a.start + at, s[r]);
      load_theta<TK, V>(a, at, d[r]);
      F32Vec<V>::load(a.mom + at, b[r]);
      if (VAR == VAR_EAGER) F32Vec<V>::load(a.dpl + at, pl[r]);
    } else {
#pragma unroll
      for (int e = 0; e < V; ++e) s[r][e] = d[r][e] = b[r][e] = pl[r][e] = 0.f;
    }
  }
  if (VAR != VAR_STANDARD) {
    if (active) F32Vec<V>::load(a.dpa + i, pa);
    else {
#pragma unroll
      for (int e = 0; e < V; ++e) pa[e] = 0.f;
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
    if (r < mine) {
      const float scale = Q ? comm_scale(a, m0 + r) : 1.f;
#pragma unroll
      for (int e = 0; e < V; ++e) {
        d[r][e] = s[r][e] - d[r][e];                                  // Alg. 1-3 line 7
        sent_dyn[((m0 + r) * V + e) * 32 + lane] = Q ? comm_round(d[r][e], scale, a) : d[r][e];
      }
    }
  }
  // the warps of one group wait for one another only (a named barrier per group)
  if (a.groups == 1) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "r"(32 * wpg) : "memory");
  // line 8: Delta = (1/M) sum_m (what replica m sent), m in order
#pragma unroll 4
  for (int m = 0; m < a.M; ++m) {
#pragma unroll
    for (int e = 0; e < V; ++e) {
      const float w = sent_dyn[(m * V + e) * 32 + lane];
      mean[e] = (m == 0) ? w : mean[e] + w;
    }
  }
#pragma unroll
  for (int e = 0; e < V; ++e) mean[e] = mean[e] / a.fM;
  if (active) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (r < mine) {
        const long long at = (m0 + r) * a.stride + i;
#pragma unroll
        for (int e = 0; e < V; ++e) {
          float g;
          if (VAR == VAR_STANDARD) g = mean[e];
          else if (VAR == VAR_DELAYED) g = pa[e];
          else {
            float t = d[r][e] - pl[r][e];                            // Alg. 3 line 11
            t = t / a.fM;
            g = t + pa[e];
          }
          nesterov(g, a.eta, a.mu, b[r][e], s[r][e]);
        }
        F32Vec<V>::store(a.mom + at, b[r]);
        F32Vec<V>::store(a.start + at, s[r]);
        store_theta<TK, V>(a, at, s[r]);
        if (VAR == VAR_EAGER) F32Vec<V>::store(a.dpl + at, d[r]);
      }
    }
    if (VAR != VAR_STANDARD && warp == 0) F32Vec<V>::store(a.dpa + i, mean);
  }
  if (blockIdx.x == gridDim.x - 1) { // ragged tail, one index per thread
    const long long t = nvec * V + threadIdx.x;
    if (t < a.P) outer_column_rt<VAR, TK, false, 1, Q>(a, t);
  }
}

// ---------------------------------------------------------------- inner AdamW
// U columns of one thread: all loads of all U columns are issued before the first use, so a
// thread keeps U x (theta, g, m, v) vectors in flight.
template <int TK, int GK, int V, int U>
__device__ __forceinline__ void adamw_columns(const AdamArgs &a, int m, const long long (&idx)[U]) {
  float g[U][V], x[U][V], m1[U][V], v1[U][V];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const long long at = m * a.stride + idx[u];
    const long long gat = m * a.gstride + idx[u];
    if (GK == GK_F32) F32Vec<V>::load(reinterpret_cast<const float *>(a.grads) + gat, g[u]);
    else BF16Vec<V>::load(reinterpret_cast<const unsigned short *>(a.grads) + gat, g[u]);
    if (TK == TK_F32) F32Vec<V>::load(reinterpret_cast<const float *>(a.theta) + at, x[u]);
    else if (TK == TK_BF16) BF16Vec<V>::load(reinterpret_cast<const unsigned short *>(a.theta) + at, x[u]);
    else F32Vec<V>::load(a.master + at, x[u]);
    F32Vec<V>::load(a.m + at, m1[u]);
    F32Vec<V>::load(a.v + at, v1[u]);
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
#pragma unroll
    for (int e = 0; e < V; ++e) {
      float t1 = a.beta1 * m1[u][e];
      float t2 = a.omb1 * g[u][e];
      m1[u][e] = t1 + t2;
      float t3 = a.beta2 * v1[u][e];
      float t4 = a.omb2 * g[u][e];
      t4 = t4 * g[u][e];
      v1[u][e] = t3 + t4;
      float mh = m1[u][e] / a.c1;
      float vh = v1[u][e] / a.c2;
      float den = sqrtf(vh) + a.eps;
      float r = mh / den;
      float w = a.wd * x[u][e];
      float upd = r + w;
      upd = a.lr * upd;
      x[u][e] = x[u][e] - upd;
    }
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const long long at = m * a.stride + idx[u];
    F32Vec<V>::store(a.m + at, m1[u]);
    F32Vec<V>::store(a.v + at, v1[u]);
    if (TK == TK_F32) {
      F32Vec<V>::store(reinterpret_cast<float *>(a.theta) + at, x[u]);
    } else if (TK == TK_BF16) {
      BF16Vec<V>::store(reinterpret_cast<unsigned short *>(a.theta) + at, x[u]);
    } else {
      F32Vec<V>::store(a.master + at, x[u]);
      BF16Vec<V>::store(reinterpret_cast<unsigned short *>(a.theta) + at, x[u]);
    }
  }
}

// grid = (ceil(nvec / (NT * U)), M): thread t of block x owns columns x*NT*U + u*NT + t
template <int TK, int GK, int V, int U, int NT, int MINB>
__global__ void __launch_bounds__(NT, MINB) adamw_kernel(const AdamArgs a) {
  const int m = blockIdx.y;
  const long long nvec = a.P / V;
  const long long j0 = (long long)blockIdx.x * (NT * U) + threadIdx.x;
  if (j0 + (long long)(U - 1) * NT < nvec) {
    long long idx[U];
#pragma unroll
    for (int u = 0; u < U; ++u) idx[u] = (j0 + (long long)u * NT) * V;
    adamw_columns<TK, GK, V, U>(a, m, idx);
  } else {
    for (int u = 0; u < U; ++u) {
      const long long j = j0 + (long long)u * NT;
      if (j < nvec) {
        long long idx[1] = {j * V};
        adamw_columns<TK, GK, V, 1>(a, m, idx);
      }
    }
  }
  if (blockIdx.x == gridDim.x - 1) {
    const long long i = nvec * V + threadIdx.x;
    if (i < a.P) {
      long long idx[1] = {i};
      adamw_columns<TK, GK, 1, 1>(a, m, idx);
    }
  }
}

} // namespace diloco
