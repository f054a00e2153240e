// Host-only part of libdiloco: a closed-form compute-utilisation calculator for one DiLoCo
// outer round (Section 3.1 "Compute utilization simulation"; Table 2's "tolerated latency"
// column).  No device code.  The paper's own figures come from a DAG simulator that is
// specified in another paper and is NOT reproduced here; this is only the arithmetic that the
// paper states in words: an all-reduce that is given D whole inner phases to finish costs
// nothing as long as it takes at most D * H * (step time), and whatever exceeds that is time
// the workers sit idle.
#include "../../include/diloco.h"

#include <cmath>

namespace {

bool valid(const diloco_cu_input_t *in) {
  if (!in) return false;
  if (in->P < 1 || in->M < 1 || in->H < 1) return false;
  if (!(in->bits_per_param > 0.0) || !(in->step_time_s > 0.0) || !(in->bandwidth_bit_s > 0.0)) return false;
  if (!std::isfinite(in->bits_per_param) || !std::isfinite(in->step_time_s) || std::isnan(in->bandwidth_bit_s)) return false;
  if (in->overlap_outer_steps < 0 || in->overlap_inner_steps < 0 || in->overlap_inner_steps > in->H) return false;
  if (in->overlap_outer_steps > 0 && in->overlap_inner_steps != 0) return false;
  if (in->ring != 0 && in->ring != 1) return false;
  return true;
}

// bits one worker must push through its link per outer step
double wire_bits(const diloco_cu_input_t *in) {
  double bits = (double)in->P * in->bits_per_param;
  if (in->ring) bits *= 2.0 * (double)(in->M - 1) / (double)in->M; // reduce-scatter + all-gather of a ring
  return bits;
}

double tolerated(const diloco_cu_input_t *in) {
  // D outer steps of overlap hide D * H inner steps; without it, the inner steps overlapped directly
  const double steps = in->overlap_outer_steps > 0 ? (double)in->overlap_outer_steps * (double)in->H
                                                   : (double)in->overlap_inner_steps;
  return steps * in->step_time_s;
}

} // namespace

extern "C" {

int diloco_compute_utilization(const diloco_cu_input_t *in, diloco_cu_output_t *out) {
  if (!valid(in) || !out) return DILOCO_ERR_INVALID_ARG;
  const double compute = (double)in->H * in->step_time_s;
  const double bits = wire_bits(in);
  out->wire_bits = bits;
  out->comm_time_s = bits / in->bandwidth_bit_s;
  out->tolerated_latency_s = tolerated(in);
  out->exposed_comm_time_s = out->comm_time_s > out->tolerated_latency_s ? out->comm_time_s - out->tolerated_latency_s : 0.0;
  out->compute_time_s = compute;
  out->compute_utilization = compute / (compute + out->exposed_comm_time_s);
  return DILOCO_OK;
}

double diloco_bandwidth_for_utilization(const diloco_cu_input_t *in, double target_utilization) {
  diloco_cu_input_t probe;
  if (!in) return (double)DILOCO_ERR_INVALID_ARG;
  probe = *in;
  probe.bandwidth_bit_s = 1.0; // not used by what follows, only validated
  if (!valid(&probe) || !(target_utilization > 0.0 && target_utilization <= 1.0)) return (double)DILOCO_ERR_INVALID_ARG;
  const double compute = (double)in->H * in->step_time_s;
  // utilisation u needs exposed <= compute (1/u - 1), i.e. comm <= tolerated + compute (1/u - 1)
  const double budget = tolerated(in) + compute * (1.0 / target_utilization - 1.0);
  if (!(budget > 0.0)) return INFINITY; // full utilisation with nothing overlapped: no finite bandwidth does it
  return wire_bits(in) / budget;
}

} // extern "C"
