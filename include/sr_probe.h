/*
 * sr_probe.h -- measurement helpers shipped with the sr_gate library.
 *
 * The gate kernels are bound by the SM's 32-bit integer ALUs, a rate that no
 * vendor tool reports directly.  sr_probe_int32 launches a register-only kernel
 * of independent integer dependency chains on every SM so that the caller can time
 * it (CUDA events on `stream`) and obtain the achievable int32 lane-operations per
 * second of the device it runs on.  It has no counterpart in the paper.
 */
#ifndef SR_PROBE_H_
#define SR_PROBE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SR_PROBE_LOGIC 0   /* three-input logic operations only */
#define SR_PROBE_ADD 1     /* 32-bit adds only */
#define SR_PROBE_MIX 2     /* 8 logic : 2 add, the mix of the bit-vector recurrence */

/* Enqueue the probe: `blocks` x `threads` threads, each running 8 independent chains
 * of `iters` x 16 operations.  `sink` is a DEVICE buffer of blocks*threads uint32
 * that receives one word per thread (keeps the chains live).  Returns SR_OK or a
 * negative error code as in sr_gate.h. */
int sr_probe_int32(int32_t variant, int32_t iters, int32_t blocks, int32_t threads,
                   uint32_t* sink, void* stream);

/* Host-only, pure: lane-operations one such launch executes. */
uint64_t sr_probe_int32_ops(int32_t iters, int32_t blocks, int32_t threads);

/*
 * sr_gate_stages -- sr_gate (same arguments, same results) that also records five
 * caller-created CUDA events on `stream`, so that a benchmark can time the stages of
 * the multi-word pipeline separately: events[0] before the first launch, [1] after
 * the match-stream preparation, [2] after the ordering of the pairs, [3] after the
 * bit-vector kernel, [4] after the per-group reduction.  With K <= 32 there is one
 * kernel: events[0] precedes it and events[1..4] follow it.  `events` is a HOST
 * array of 5 cudaEvent_t.  Measurement aid; no counterpart in the paper.
 */
int sr_gate_stages(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                   int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                   int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                   int32_t* status, void* workspace, size_t workspace_bytes, void* stream,
                   void* const* events);

#ifdef __cplusplus
}
#endif
#endif /* SR_PROBE_H_ */
