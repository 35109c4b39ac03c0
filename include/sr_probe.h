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

#ifdef __cplusplus
}
#endif
#endif /* SR_PROBE_H_ */
