/*
 * Measurement and self-test helpers shipped with libnbos.so. They are not part of the placement
 * path; the benchmark and the tests use them. The paper has no counterpart for either.
 */
#ifndef NBOS_PROBE_H_
#define NBOS_PROBE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NBOS_PROBE_MIX_ALU 0  /* xor / min / max chains: the integer ALU pipe only            */
#define NBOS_PROBE_MIX_IMAD 1 /* 32-bit multiply-add chains: the multiply pipe only           */
#define NBOS_PROBE_MIX_BOTH 2 /* the two interleaved one to one                               */

/*
 * Integer issue-rate probe. Launches `blocks` x `threads` threads that each run `iters`
 * iterations over 8 independent dependency chains of 32-bit integer instructions, times the
 * launch with CUDA events on `cuda_stream` and synchronises it.
 *   out_thread_ops  thread-level integer instructions the kernel was written to execute
 *                   (iters * 8 chains * 4 instructions * threads * blocks)
 *   out_ms          duration of the launch
 * Returns NBOS_OK or a negative NBOS_ERR_* code (see nbos.h).
 */
int nbos_probe_int32_issue(int mix, int iters, int blocks, int threads, void *cuda_stream,
                           double *out_thread_ops, float *out_ms);

/*
 * Bounded-wait self-test: one thread block waits on a shared-memory barrier that nothing ever
 * completes, with the same bounded wait the placement kernel uses, limited to `limit_ns`
 * nanoseconds (clamped to 1 ms .. 5 s). The block must give up, record it and exit normally.
 *   out_gave_up  1 if the kernel reported that its wait ran out, else 0
 *   out_ms       duration of the launch
 * The CUDA context stays usable afterwards.
 */
int nbos_probe_wait_timeout(uint64_t limit_ns, void *cuda_stream, int *out_gave_up, float *out_ms);

#ifdef __cplusplus
}
#endif
#endif /* NBOS_PROBE_H_ */
