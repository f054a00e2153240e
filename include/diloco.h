/*
 * libdiloco - the DiLoCo outer-optimisation step (standard, naive delayed, eager) and the
 * inner AdamW step as fused sm_100a CUDA kernels, behind a plain C ABI.
 *
 * Method: "Eager Updates For Overlapped Communication and Computation in DiLoCo",
 * Section 2, Algorithms 1-3.  M workers are simulated as M replica parameter buffers on ONE
 * GPU; the cross-worker all-reduce of the outer gradients (line 8 of each algorithm) is
 * replaced by a fixed-order reduction over the replica axis inside the kernel, and the
 * one-phase delay of its result ("async-send" / "block-receive") by a state buffer that is
 * written at outer step k and read at outer step k+1.
 *
 * Notation (the paper's): M replicas, H inner steps per outer step, theta_m the current
 * parameters of replica m, s_m = theta_m^(t-H) its start-of-phase ("outer") parameters,
 * Delta_m = s_m - theta_m the local outer gradient, Delta = (1/M) sum_m Delta_m the
 * all-reduced one, b_m the momentum buffer of OuterOpt (SGD with Nesterov momentum),
 * eta / mu the outer learning rate / momentum.  InnerOpt is AdamW.
 *
 * General rules of this ABI
 *   - every pointer inside diloco_buffers_t is a DEVICE pointer on the device that is
 *     current when diloco_state_init is called; the memory is BORROWED: the caller
 *     allocates it, keeps it alive while the state exists and frees it afterwards.  The
 *     library never allocates or frees device memory.
 *   - every other pointer (config, buffers struct, out-parameters) is a HOST pointer.
 *   - layout: every [M, stride] buffer is replica-major, element (m, i) at m*stride + i,
 *     0 <= i < P <= stride.  Elements with i >= P are padding: never read, never written.
 *     stride * sizeof(element) must be a multiple of 128 bytes for every buffer (so stride
 *     is a multiple of 64 when any buffer is bf16, else of 32), base pointers 16-byte
 *     aligned.  grads use their own stride with the same rule.  (Performance, not
 *     correctness: rows that start on 4 KB boundaries, i.e. a stride that is a multiple of
 *     1024 elements, measured 1-2 % faster on B200.)
 *   - all kernels are launched asynchronously on the stream the caller passes
 *     (a cudaStream_t cast to void*; NULL = the legacy default stream).  No call
 *     synchronises the device.  All buffers are updated in place.
 *   - every call returns a status (0 = DILOCO_OK, negative = error); nothing throws or
 *     aborts.  On error nothing has been launched and the state is unchanged (one exception,
 *     stated there: a runtime failure in the middle of diloco_outer_step_host).
 *   - the device that was current at diloco_state_init must be current at every launching
 *     call on that state (DILOCO_ERR_BAD_STATE otherwise).
 *   - arithmetic: fp32, one IEEE round-to-nearest-even per operation, no FMA contraction,
 *     IEEE division and square root; the sum over replicas runs m = 0 .. M-1 in order; 1/M
 *     is a division by (float)M.  bf16 is a storage type only (round-to-nearest-even).
 *   - a state is not thread-safe: one caller at a time.
 *   - CUDA graphs: a steady-state diloco_outer_standard / _delayed / _eager call (have_prev =
 *     overlap_steps = 1, direct kernels) is one launch whose arguments do not change from step to
 *     step and may be captured and replayed; the counters advance when the call is captured, not
 *     when the graph runs.  Do not capture diloco_inner_adamw (its bias corrections are launch
 *     arguments computed from the step count), steps with overlap_steps > 1 (the ring slot is a
 *     launch argument) or first steps.  Nothing is said here about the other entry points.
 */
#ifndef DILOCO_H_
#define DILOCO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DILOCO_MAX_M 64
#define DILOCO_MAX_OVERLAP 4
#define DILOCO_MAX_FRAGMENTS 4096

enum {
  DILOCO_OK = 0,
  DILOCO_ERR_INVALID_ARG = -1,    /* null pointer, M < 1, P < 1, stride < P, bad dtype, bad hyper-parameter */
  DILOCO_ERR_MISALIGNED = -2,     /* base pointer not 16-byte aligned or stride bytes not a multiple of 128 */
  DILOCO_ERR_BAD_STATE = -3,      /* the state lacks a buffer this call needs */
  DILOCO_ERR_CUDA = -4,           /* a CUDA runtime call failed; see diloco_last_cuda_error */
  DILOCO_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait ran out (see diloco_check_device_status) */
  DILOCO_ERR_UNSUPPORTED = -6     /* M > DILOCO_MAX_M or a size beyond a fixed limit */
};

/* storage of theta */
enum {
  DILOCO_THETA_F32 = 0,        /* theta is fp32 */
  DILOCO_THETA_BF16 = 1,       /* theta is bf16; Delta_m is formed from the stored (rounded) value */
  DILOCO_THETA_MASTER_BF16 = 2 /* fp32 master (the value) + bf16 working copy written alongside */
};
enum { DILOCO_GRAD_F32 = 0, DILOCO_GRAD_BF16 = 1 };

/* wire format of the outer gradients in diloco_outer_quantized */
enum {
  DILOCO_COMM_F32 = 0,  /* full precision: the algorithms as printed */
  DILOCO_COMM_BF16 = 1, /* bfloat16, round to nearest even, no scaling */
  DILOCO_COMM_EXMY = 2  /* 1 sign + exp_bits + man_bits float, scaled per replica (see the call) */
};

/* kernel implementation selector (performance only; results are bit-identical) */
enum {
  DILOCO_IMPL_AUTO = 0,
  DILOCO_IMPL_DIRECT = 1, /* register-resident columns, 128-bit global loads and stores */
  DILOCO_IMPL_BULK = 2,   /* replica tiles staged through shared memory by the TMA unit (1-D bulk copies) */
  /* force one of the warp-split forms (replica axis over the warps of a block) whatever M is,
     for measurements; AUTO picks among them and the per-M shapes by M */
  DILOCO_IMPL_SPLIT_R2 = 3, /* two replicas per warp, 128-bit accesses (M <= 32, else as AUTO) */
  DILOCO_IMPL_SPLIT_R4 = 4, /* four replicas per warp, 64-bit accesses                          */
  /* tiles [M replicas x T indices] of every buffer moved by 2-D TMA box copies (tensor maps over
     this GPU's memory, no multicast), updated in shared memory; fp32 theta only, needs
     device_status; other states and first steps take the direct form */
  DILOCO_IMPL_TENSOR_T256 = 5,
  DILOCO_IMPL_TENSOR_T128 = 6,
  DILOCO_IMPL_TENSOR_T64 = 7
};

typedef struct {
  int32_t M;            /* number of replicas (Alg. 1-3 "Require M replicas") */
  int32_t H;            /* inner steps per outer step (Alg. 1-3 "Synchronization frequency H"); bookkeeping only */
  int64_t P;            /* flat parameters per replica */
  int64_t stride;       /* elements between consecutive replicas in every [M, stride] state buffer */
  float outer_lr;       /* eta  of OuterOpt (Section 3: tuned to 0.4 in the paper) */
  float outer_momentum; /* mu   of OuterOpt, in [0, 1) */
  float beta1, beta2;   /* AdamW, each in [0, 1) */
  float eps;            /* AdamW, >= 0, added after the square root */
  float weight_decay;   /* AdamW, decoupled, >= 0 */
  int32_t theta_kind;   /* DILOCO_THETA_* */
  int32_t grad_kind;    /* DILOCO_GRAD_* : dtype of the grads argument of diloco_inner_adamw */
  int32_t have_prev;    /* how many generations of delta_prev_local / delta_prev_avg already hold recorded
                           gradients, 0 .. overlap_steps.  overlap_steps: every delayed / eager call applies
                           (t > H); 0: the next overlap_steps such calls only record (t <= overlap_steps H) */
  int32_t impl;         /* DILOCO_IMPL_* */
  int32_t overlap_steps;/* D >= 1: outer steps by which the all-reduce result is delayed.  1 is the paper's
                           Algorithms 2-3 ("1-outer-step" overlap); 2 is the "two-outer-steps" overlap of
                           Section 3, for which the paper prints no formula: this library reads it as
                           line 11 with t-H replaced by t-DH,
                             g_m = (Delta_m^(t) - Delta_m^(t-DH)) / M + Delta^(t-DH).
                           At most DILOCO_MAX_OVERLAP. */
  int32_t shared_outer_state; /* 0: start and outer_mom are [M, stride], one copy per replica (every call works).
                           1: standard DiLoCo only: under Algorithm 1 every replica's OuterOpt sees the same
                           start point and the same gradient, so the M copies of s_m and b_m stay bit-identical
                           for ever; with this flag the state keeps ONE copy, start and outer_mom are [stride],
                           and the standard step moves 8 M + 16 bytes per index instead of 24 M (same bits in
                           theta).  diloco_outer_standard, diloco_outer_fragment(_step) with variant 0 and
                           diloco_inner_adamw work; every other outer call returns DILOCO_ERR_BAD_STATE (the
                           delayed and eager steps let the replicas' start points differ). */
} diloco_config_t;

typedef struct {
  void *theta;             /* [M, stride] fp32 or bf16 per theta_kind: theta_m^(t)                      */
  float *master;           /* [M, stride] fp32, only for DILOCO_THETA_MASTER_BF16, else NULL            */
  float *start;            /* [M, stride] fp32: s_m = theta_m^(t-H)                 (Alg. 1-3 line 7);
                              [stride] with shared_outer_state                                            */
  float *delta_prev_local; /* [D, M, stride] fp32, D = overlap_steps: Delta_m of the last D outer steps, a
                              ring indexed by (outer-step counter mod D): the step that reads a generation
                              overwrites it.  Eager only, else may be NULL              (Alg. 3 l.11)    */
  float *delta_prev_avg;   /* [D, stride] fp32: the means of those steps, i.e. the all-reduces in flight;
                              delayed and eager, may be NULL if only the standard step is used
                                                                                    (Alg. 2-3 line 10)  */
  float *outer_mom;        /* [M, stride] fp32: b_m, Nesterov buffer of OuterOpt; [stride] with
                              shared_outer_state                                                          */
  float *adam_m;           /* [M, stride] fp32 first moment;  NULL if diloco_inner_adamw is not used    */
  float *adam_v;           /* [M, stride] fp32 second moment; NULL if diloco_inner_adamw is not used    */
  uint32_t *device_status; /* 1 word, zero-initialised by the caller; needed only by DILOCO_IMPL_BULK,
                              whose bounded mbarrier waits record a give-up here; else may be NULL      */
  uint32_t *comm_scratch;  /* [DILOCO_MAX_M] words of scratch, contents irrelevant on entry; needed only by
                              diloco_outer_quantized with DILOCO_COMM_EXMY (per-replica max |Delta_m|),
                              else may be NULL                                                            */
} diloco_buffers_t;

typedef struct diloco_state diloco_state_t; /* opaque, host memory, owned by the library */

/*
 * Create a state handle: validates config and buffers (ranges, alignment, and that every
 * buffer pointer is device or managed memory of the current device: a host pointer is
 * rejected here rather than faulting in a kernel later; sizes cannot be checked), records
 * the current device and its SM count.  *out is set only on success.  Launches nothing.
 * Errors: INVALID_ARG, MISALIGNED, UNSUPPORTED, CUDA (no usable device).
 */
int diloco_state_init(const diloco_config_t *config, const diloco_buffers_t *buffers, diloco_state_t **out);

/* Free the host handle.  Device buffers are the caller's and are not touched.  NULL is OK. */
int diloco_state_free(diloco_state_t *state);

/*
 * Inner optimisation step, Alg. 1-3 line 5 with InnerOpt = AdamW, for all M replicas in one
 * launch: with k = the state's inner-step counter + 1,
 *     m <- beta1 m + (1-beta1) g,  v <- beta2 v + ((1-beta2) g) g,
 *     theta <- theta - lr * ( (m/(1-beta1^k)) / (sqrt(v/(1-beta2^k)) + eps) + weight_decay * theta ).
 * grads: device pointer, [M, grad_stride] of config.grad_kind, read only.  lr: this step's
 * inner learning rate (the schedule is the caller's).  The bias corrections are computed on
 * the host in double and rounded to fp32.  Increments the inner-step counter on success.
 * Errors: INVALID_ARG, MISALIGNED, BAD_STATE (no Adam moments), CUDA.
 */
int diloco_inner_adamw(diloco_state_t *state, const void *grads, int64_t grad_stride, float lr, void *cuda_stream);

/*
 * Outer step of standard DiLoCo, Algorithm 1 lines 7-10, one fused pass:
 *     Delta_m = s_m - theta_m;  Delta = (1/M) sum_m Delta_m;
 *     b_m <- mu b_m + Delta;  s_m <- s_m - eta (Delta + mu b_m);  theta_m <- s_m.
 * Touches theta (master), start, outer_mom only.
 */
int diloco_outer_standard(diloco_state_t *state, void *cuda_stream);

/*
 * Outer step with naive delayed outer gradients, Algorithm 2 lines 7-11: as above but
 * OuterOpt consumes delta_prev_avg (the mean formed at the previous outer step), and the new
 * mean replaces it afterwards.  While have_prev < overlap_steps (t = H with the paper's
 * overlap of one outer step) nothing is applied: the mean is recorded, s_m <- theta_m, theta
 * and outer_mom are unchanged, have_prev grows by one.  With overlap_steps = D > 1 the mean
 * consumed is the one recorded D outer steps ago (generation ring, see diloco_buffers_t).
 * Errors additionally: BAD_STATE (delta_prev_avg missing).
 */
int diloco_outer_delayed(diloco_state_t *state, void *cuda_stream);

/*
 * Outer step with eager updates, Algorithm 3 lines 7-12, one fused pass:
 *     Delta_m = s_m - theta_m;  Delta = (1/M) sum_m Delta_m;
 *     g_m = (Delta_m - delta_prev_local_m) / M + delta_prev_avg          (line 11)
 *     b_m <- mu b_m + g_m;  s_m <- s_m - eta (g_m + mu b_m);  theta_m <- s_m  (line 12)
 *     delta_prev_local_m <- Delta_m;  delta_prev_avg <- Delta.
 * have_prev < overlap_steps: first outer step(s), as for diloco_outer_delayed, also recording
 * Delta_m; overlap_steps = D > 1: delta_prev_local / delta_prev_avg of D outer steps ago.
 * Errors additionally: BAD_STATE (delta_prev_local or delta_prev_avg missing).
 */
int diloco_outer_eager(diloco_state_t *state, void *cuda_stream);

/*
 * Any of the three outer steps with QUANTISED COMMUNICATION of the outer gradients (Section 3,
 * "Quantized Communication": float32, bfloat16, float8 and float4 "using EXMY").  Only the
 * operand of the all-reduce is rounded: line 8 becomes Delta = (1/M) sum_m Q_m(Delta_m), while
 * every local use of Delta_m (line 11's fresh and stale terms, delta_prev_local) keeps fp32.
 *   DILOCO_COMM_BF16: Q = round to bfloat16 (nearest even).
 *   DILOCO_COMM_EXMY: Q_m(x) = scale_m * R(x / scale_m), R = nearest number of the float with
 *     1 sign, exp_bits exponent and man_bits mantissa bits (bias 2^(exp_bits-1) - 1, subnormals,
 *     every code finite, ties to the even code, saturating), scale_m = max_i |Delta_m[i]| /
 *     (largest value of the format), or 1 if the replica did not move.  1 <= exp_bits <= 5,
 *     man_bits >= 0, exp_bits + man_bits <= 7 (E4M3, E5M2: 8 bits; E2M1, E3M0: 4 bits).
 *     Two kernels: a reduction of max |Delta_m| into comm_scratch (zeroed by the call, so calls
 *     on one state must not overlap), then the fused step.
 * variant: 0 standard, 1 delayed, 2 eager; have_prev and the counters advance as in the plain
 * calls.  DILOCO_COMM_F32 is the plain call.  The paper fixes no bit layout or scaling: the
 * above is this library's reading.
 * Errors additionally: INVALID_ARG (format), BAD_STATE (comm_scratch missing for EXMY).
 */
int diloco_outer_quantized(diloco_state_t *state, int32_t variant, int32_t comm_format, int32_t exp_bits,
                           int32_t man_bits, void *cuda_stream);

/*
 * diloco_outer_quantized for callers that cannot provide comm_scratch.  (The paper has no
 * counterpart: this is a packaging variant of the call above, same arithmetic, same results.)
 *
 * Who needs it: code that gets handed the state tensors and nothing else and has no way to
 * obtain one more device buffer - for instance an extension running inside a trainer whose
 * memory pool already owns all of the GPU's memory, so that a raw cudaMalloc fails, or a
 * callback that must not allocate because allocation may synchronise the device.  For them
 * the per-replica maxima are reduced into an array that is part of the library image
 * instead: DILOCO_MAX_M (64) words = 256 bytes of device memory, present on every GPU that
 * loads the library for as long as the process lives.  The state's comm_scratch is ignored
 * and may be NULL.  The call allocates and frees nothing, on the host side of CUDA or on the
 * device.
 *
 * Limits and rules:
 *   - M <= DILOCO_MAX_M (64), else DILOCO_ERR_UNSUPPORTED: one word of scratch per replica
 *     (diloco_state_init has the same limit today, so no existing state can exceed it).
 *   - the device's ordinal must be below 64 (the library keeps one looked-up address per
 *     ordinal), else DILOCO_ERR_UNSUPPORTED.
 *   - the state's device must be the current device, else DILOCO_ERR_BAD_STATE.
 *   - the first DILOCO_COMM_EXMY call on each device looks up the array's device address
 *     (cudaGetSymbolAddress) and keeps it; make that first call outside any stream capture.
 *     The bf16 and fp32 formats reduce no maxima and never touch the array.
 *   - all states and all calls on a device share the one array.  The call clears the words
 *     it uses before reducing into them, so stale contents never matter, but two calls whose
 *     kernels can overlap on the GPU (different streams, no ordering between them) race on
 *     it: order such calls yourself.
 * Otherwise identical to diloco_outer_quantized, including errors, have_prev and counters.
 */
int diloco_outer_quantized_static(diloco_state_t *state, int32_t variant, int32_t comm_format, int32_t exp_bits,
                                  int32_t man_bits, void *cuda_stream);

/*
 * WORKER FORM of the outer step, for deployments where the M replicas live on M GPUs (one
 * process per GPU) and line 8's mean is a real all-reduce between them (Section 2.1; the
 * paper's implementation: an all-reduce without parameter server, Section 3).  The state
 * holds ONE replica (config M = 1, every [M, stride] buffer is [stride], delta_prev_avg is
 * not used); the M of the algorithm is world_replicas.  The caller owns the communication:
 *   delta_send      [>= P] fp32 device buffer the kernel fills with this worker's Delta_m
 *                   (Alg. 1-3 line 7); all-reduce it with SUM over the workers;
 *   delta_sum_recv  [>= P] fp32 device buffer holding that element-wise SUM for the outer
 *                   step whose result is due now; the kernel divides by world_replicas itself,
 *                   so the arithmetic is Delta = (sum_m Delta_m) / M exactly as in the fused
 *                   M-replica calls (bit-identical to them when the sum was formed in the
 *                   order m = 0 .. M-1; for M = 2 every order is that order).
 * Both 16-byte aligned; nothing else is communicated.
 *
 * diloco_worker_outer_send: standard DiLoCo (Algorithm 1) only, lines 7-8: delta_send =
 *   s - theta, state untouched.  All-reduce it (blocking, line 9), then call
 *   diloco_worker_outer_apply(variant 0) with the sum: line 10.
 * diloco_worker_outer_apply, variant 1 (naive delayed) or 2 (eager): one kernel per outer
 *   step.  It applies OuterOpt with the sum that was sent overlap_steps outer steps ago
 *   (Algorithm 2 line 11 / Algorithm 3 lines 11-12) and fills delta_send with the new
 *   Delta_m, whose all-reduce the caller starts asynchronously and lets run during the next
 *   inner phase.  While have_prev < overlap_steps nothing has arrived yet: delta_sum_recv is
 *   ignored (may be NULL), the step only records (s <- theta, own Delta_m kept for line 11).
 *   The worker's own stale gradients live in the state's delta_prev_local ring as usual.
 * Counters and have_prev advance as in the fused calls.
 * Errors: INVALID_ARG, MISALIGNED, BAD_STATE (M != 1, delta_prev_local missing for eager,
 * wrong current device), CUDA.
 */
int diloco_worker_outer_send(diloco_state_t *state, float *delta_send, void *cuda_stream);
int diloco_worker_outer_apply(diloco_state_t *state, int32_t variant, int32_t world_replicas,
                              const float *delta_sum_recv, float *delta_send, void *cuda_stream);

/*
 * WORKER FORM WITH A QUANTISED WIRE (Section 3, "Quantized Communication", between real
 * workers): what a worker sends is its Delta_m as EXMY codes plus one fp32 word, its
 * max |Delta_m|; the workers exchange these with an ALL-GATHER (a sum of codes means nothing)
 * and each forms the mean itself,
 *     Delta = ( sum over m = 0 .. M-1, in order, of scale_m * value(code_m) ) / M,
 *     scale_m = amax_m / (largest value of the format), or 1 if amax_m = 0,
 * which is line 8 of diloco_outer_quantized exactly, for any M.  Format as there
 * (1 <= exp_bits <= 5, exp_bits + man_bits <= 7).  Wire layout: code of an element =
 * sign << (exp_bits + man_bits) | exponent field << man_bits | mantissa; codes of at most
 * 4 bits are packed two per byte (element 2j in bits 0-3, element 2j+1 in bits 4-7), wider
 * codes take one byte each: diloco_wire_payload_bytes(P, ...) bytes per worker, i.e. a quarter
 * or an eighth of the fp32 gradient.
 *
 * diloco_worker_quantized_send: standard DiLoCo, lines 7-8: payload_send and amax_send from
 *   this worker's Delta_m, state untouched (two kernels: the maximum, then the codes).
 * diloco_worker_quantized_apply: as diloco_worker_outer_apply.  payloads_recv [world_replicas,
 *   payload_stride bytes] and amaxes_recv [world_replicas] are the gathered payloads and
 *   maxima, in worker order, of the outer step whose result is due (ignored while have_prev <
 *   overlap_steps); for variants 1 and 2 the call also fills payload_send / amax_send with the
 *   new Delta_m for the gather that runs during the next inner phase.  world_replicas <= 64.
 * All four buffers: device memory, 4-byte aligned; payload_stride a multiple of 4.
 */
int64_t diloco_wire_payload_bytes(int64_t P, int32_t exp_bits, int32_t man_bits);
int diloco_worker_quantized_send(diloco_state_t *state, int32_t exp_bits, int32_t man_bits, uint8_t *payload_send,
                                 uint32_t *amax_send, void *cuda_stream);
int diloco_worker_quantized_apply(diloco_state_t *state, int32_t variant, int32_t world_replicas, int32_t exp_bits,
                                  int32_t man_bits, const uint8_t *payloads_recv, int64_t payload_stride,
                                  const uint32_t *amaxes_recv, uint8_t *payload_send, uint32_t *amax_send,
                                  void *cuda_stream);

/*
 * The same three steps restricted to parameter indices [offset, offset + len) of every
 * replica, with NO bookkeeping: the low-level form under diloco_outer_fragment_step (below),
 * for callers that keep their own schedule state.  variant: 0 standard, 1 delayed, 2 eager.  bootstrap
 * != 0 performs the first-outer-step form for this fragment; the state's have_prev count is
 * NOT consulted and neither it nor the outer-step counter is changed: per-fragment
 * bookkeeping is the caller's (with overlap_steps > 1 the generation used is the one the
 * outer-step counter currently selects; move it with diloco_state_set_counters).
 * offset must be a multiple of 32 elements (64 if theta is bf16); len >= 1; offset + len <= P.
 */
int diloco_outer_fragment(diloco_state_t *state, int32_t variant, int32_t bootstrap,
                          int64_t offset, int64_t len, void *cuda_stream);

/*
 * FRAGMENT SCHEDULES.  Streaming DiLoCo (Section 3, Experiments: the outer step is applied
 * "to different parts of the models on different schedules"; appendix Table 4: fragments of
 * three layers) gives every fragment of the parameter axis its own outer-step times.  Every
 * index is independent of every other, so a fragment is just a range; what makes a schedule is
 * that each fragment must remember on its own how many outer steps it has taken (which slot of
 * the generation ring it reads and overwrites) and how many generations of its recorded
 * gradients are valid (whether a delayed / eager step still only records, the t = H case).
 *
 * diloco_fragments_set: install a table of n fragments, fragment i = indices
 *   [offsets[i], offsets[i] + lens[i]) of every replica; offsets multiples of 32 elements (64 if
 *   theta is bf16), lens >= 1, inside [0, P), pairwise disjoint (they need not cover P).
 *   offsets / lens are host arrays, copied.  Every fragment starts from the state's current
 *   counters (outer-step counter and have_prev at the time of the call).  n = 0 removes the
 *   table.  Errors: INVALID_ARG, MISALIGNED, UNSUPPORTED (n > DILOCO_MAX_FRAGMENTS).
 * diloco_outer_fragment_step: one outer step (variant 0 standard, 1 delayed, 2 eager) of
 *   fragment fragment_id, same kernel and arithmetic as the whole-vector calls.  Uses and
 *   advances that fragment's counters only: while its have_prev < overlap_steps a delayed /
 *   eager step records without applying, and with overlap_steps = D > 1 it consumes what this
 *   fragment recorded D of ITS OWN outer steps ago.  The state's global counters are untouched.
 * diloco_outer_fragment_step_quantized: the same with the fragment's outer gradients rounded to
 *   a wire format before the mean (the paper's bandwidth figures are for streaming fragments with
 *   4-bit communication, Table 4): formats, arguments and rounding as diloco_outer_quantized; the
 *   per-replica scale is the maximum over THIS FRAGMENT's indices, since a fragment is what one
 *   exchange carries.  DILOCO_COMM_F32 is diloco_outer_fragment_step.  Needs comm_scratch for
 *   DILOCO_COMM_EXMY; calls on one state must not overlap.
 * diloco_fragment_get_counters / _set_counters: per-fragment checkpoint / resume.
 * Whole-vector calls and diloco_outer_fragment (below) ignore the table.
 */
int diloco_fragments_set(diloco_state_t *state, int32_t n, const int64_t *offsets, const int64_t *lens);
int diloco_outer_fragment_step(diloco_state_t *state, int32_t variant, int32_t fragment_id, void *cuda_stream);
int diloco_outer_fragment_step_quantized(diloco_state_t *state, int32_t variant, int32_t fragment_id, int32_t comm_format,
                                         int32_t exp_bits, int32_t man_bits, void *cuda_stream);
int diloco_fragment_get_counters(const diloco_state_t *state, int32_t fragment_id, int64_t *outer_step, int32_t *have_prev);
int diloco_fragment_set_counters(diloco_state_t *state, int32_t fragment_id, int64_t outer_step, int32_t have_prev);

/*
 * End-to-end form of the three outer steps for callers whose state lives in HOST memory:
 * copies every state buffer the variant reads from the host_* buffers (same layout and
 * dtypes as `state`'s device buffers, which serve as the staging area) to the device,
 * runs the step, and copies every buffer it writes back, chunked along P so that
 * copies and kernels of different chunks overlap on the three streams given.  host: a
 * diloco_buffers_t whose pointers are HOST pointers (pinned memory for full copy speed); a
 * NULL entry means that buffer is resident on the device and is neither copied in nor out
 * (e.g. only theta travels and the optimiser state stays on the GPU); theta or master must
 * be given;
 * streams: three distinct cudaStream_t cast to void* (h2d, compute, d2h); chunk: elements
 * per chunk, a multiple of 64.  Returns after enqueueing; the caller synchronises streams[2].
 * Advances have_prev / outer-step counter like the device forms.
 * Rows are moved one cudaMemcpyAsync per row and chunk, so rows of any length work.  Host
 * memory that is not pinned is accepted but makes the copies synchronous with the host; a
 * host_* pointer that is in fact device memory is refused (INVALID_ARG).
 * Errors: arguments, buffers and everything else that can fail without touching a stream are
 * checked before the first copy is enqueued, and such an error leaves the state unchanged.  If
 * the CUDA runtime itself fails later, while chunks are being enqueued (DILOCO_ERR_CUDA from a
 * copy, an event or a launch), earlier chunks are already in flight: the call returns at once,
 * the counters are NOT advanced, and the state buffers on both sides are then a mixture of
 * stepped and unstepped chunks - synchronise the three streams and restore from a checkpoint.
 */
int diloco_outer_step_host(diloco_state_t *state, int32_t variant, const diloco_buffers_t *host,
                           void *const streams[3], int64_t chunk);

/* Counters and flags, e.g. for checkpoint / resume (buffers are the caller's to save). */
int diloco_state_get_counters(const diloco_state_t *state, int64_t *inner_step, int64_t *outer_step, int32_t *have_prev);
int diloco_state_set_counters(diloco_state_t *state, int64_t inner_step, int64_t outer_step, int32_t have_prev);
int diloco_set_outer_hparams(diloco_state_t *state, float outer_lr, float outer_momentum);
int diloco_set_impl(diloco_state_t *state, int32_t impl);

/*
 * Bound of the device-side waits.  Only DILOCO_IMPL_BULK waits on anything (an mbarrier that
 * the TMA unit completes when a tile's rows have landed in shared memory); every such wait
 * gives up after limit_ns nanoseconds of the GPU's global timer (0 selects the default, 1 s),
 * the CTA then stops, gives its copies in flight one more limit to land, and the kernel
 * reports through device_status (diloco_check_device_status -> DILOCO_ERR_DEVICE_TIMEOUT).  A
 * kernel in which every wait runs out returns after about (ring depth 3 + 1) x limit_ns.
 * After a time-out the step's results are invalid: the buffers hold a mixture of stepped and
 * unstepped tiles, while have_prev and the outer-step counter have advanced as for a
 * successful call; restore both from a checkpoint.
 * test_extra_expect_bytes: 0 in production.  A multiple of 16, at most 1024: every tile's
 * barrier is told to expect that many bytes more than the copies deliver, so every copy still
 * lands but no wait ever completes.  It exists so that a test can drive the give-up path
 * without faulting or hanging anything; with it set no tile is stepped and no state buffer is
 * written.
 */
int diloco_set_wait_limit(diloco_state_t *state, uint64_t limit_ns, uint32_t test_extra_expect_bytes);

/*
 * Read the state's device_status word (synchronises the given stream first).  Returns
 * DILOCO_OK if it is zero or absent, DILOCO_ERR_DEVICE_TIMEOUT if a kernel gave up a bounded
 * wait (its results are then invalid), DILOCO_ERR_CUDA on a runtime error.
 */
int diloco_check_device_status(diloco_state_t *state, void *cuda_stream);

/*
 * COMPUTE-UTILISATION CALCULATOR (host only, no GPU work).  Section 3.1 and Table 2: a worker
 * spends H * step_time_s computing per outer round and must move its outer gradient through its
 * link once per round; with the all-reduce overlapped with the next D inner phases (D = 1:
 * Algorithms 2-3, D = 2: "two-outer-steps" overlap) communication is free as long as it takes
 * no longer than the TOLERATED LATENCY D * H * step_time_s (Table 2: 30 x 0.08 s = 2.4 s, and
 * 4.8 s for D = 2; overlapping one inner step instead tolerates 0.08 s; blocking tolerates 0).
 * Whatever exceeds it is idle time:
 *     comm_time      = wire_bits / bandwidth_bit_s
 *     exposed        = max(0, comm_time - tolerated_latency)
 *     utilization    = compute_time / (compute_time + exposed)          (1 = never idle)
 * wire_bits = P * bits_per_param, times 2 (M-1)/M if ring != 0 (what one worker sends in a ring
 * all-reduce).  bits_per_param: 32, 16, or 8 * diloco_wire_payload_bytes(P, X, Y) / P for an EXMY
 * wire.  This is the closed form the paper states in words; the figures of its Table 4 and
 * Figure 4 come from a DAG simulator specified in another paper, which is NOT reproduced, so do
 * not expect those numbers from this function.
 * diloco_bandwidth_for_utilization inverts it: the smallest bandwidth (bit/s) that reaches the
 * target utilisation in (0, 1] (bandwidth_bit_s of the input is ignored); INFINITY if none
 * does (target 1 with nothing overlapped); a negative status cast to double on bad arguments.
 * Errors: INVALID_ARG (null, P/M/H < 1, non-positive times, widths or bandwidth, negative
 * overlaps, overlap_inner_steps > H or combined with overlap_outer_steps > 0).
 */
typedef struct {
  int64_t P;                   /* parameters whose outer gradient is exchanged per outer step             */
  double bits_per_param;       /* width of one outer-gradient element on the wire                         */
  int32_t M;                   /* workers (matters only with ring != 0)                                   */
  int32_t H;                   /* inner steps per outer step                                              */
  double step_time_s;          /* pure compute time of one inner step                                     */
  double bandwidth_bit_s;      /* link bandwidth per worker, bits per second (may be INFINITY)            */
  int32_t overlap_outer_steps; /* D: 0 blocking (Algorithm 1), 1 Algorithms 2-3, 2 two-outer-steps, ...   */
  int32_t overlap_inner_steps; /* with D = 0: inner steps the exchange is overlapped with (0 .. H)        */
  int32_t ring;                /* 0: wire_bits = P * bits_per_param; 1: ring all-reduce factor 2 (M-1)/M  */
} diloco_cu_input_t;
typedef struct {
  double wire_bits, comm_time_s, tolerated_latency_s, exposed_comm_time_s, compute_time_s, compute_utilization;
} diloco_cu_output_t;
int diloco_compute_utilization(const diloco_cu_input_t *in, diloco_cu_output_t *out);
double diloco_bandwidth_for_utilization(const diloco_cu_input_t *in, double target_utilization);

/* Number of kernels this library has launched in this process so far. */
int64_t diloco_launch_count(void);
/* The raw cudaError_t of the last failed runtime call made by the library (0 if none). */
int32_t diloco_last_cuda_error(void);
/* Static, never NULL. */
const char *diloco_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* DILOCO_H_ */
