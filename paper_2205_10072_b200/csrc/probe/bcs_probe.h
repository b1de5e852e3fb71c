/*
 * bcs_probe.h -- measurement helper of the benchmark, not part of the schedule construction
 * (the paper has no counterpart): the integer instruction rate of the GPU, which is the
 * denominator of the roofline of the schedule kernels.
 */
#ifndef BCS_PROBE_H_
#define BCS_PROBE_H_

#include <stdint.h>

#include "bcs.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Runs, on the current device and the given stream, a kernel of 148 * 8 CTAs of 256 threads in
 * which every thread executes `iters` rounds of 32 independent 32-bit integer instructions, and
 * synchronises the stream.
 *   mix 0: three-input logic operations only (these issue on the integer ALU pipe alone);
 *   mix 1: logic operations and multiply-adds alternating (the latter issue on the FMA pipe:
 *          the best case of two pipes fed in parallel);
 *   mix 2: logic operations and three-input additions alternating (the compiler is free to
 *          place additions on either pipe).
 * ops_out (host): thread-level instructions of the measured loop body that were executed,
 * ms_out (host): their device time by CUDA events.  sink_dev: device word that receives a
 * value depending on all results (so that nothing can be optimised away), may not be NULL. */
bcs_status bcs_probe_int_rate(int mix, uint32_t iters, uint32_t *sink_dev, double *ops_out,
                              float *ms_out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BCS_PROBE_H_ */
