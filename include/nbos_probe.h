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
 * Bounded-wait self-test: the two warps of one thread block wait on a shared-memory barrier that
 * nothing ever completes, through the very wait function the placement kernel uses (the limit,
 * 2 s there, is `limit_ns` here, clamped to 1 ms .. 5 s). The warp whose wait runs out raises the
 * block's abort flag, the other leaves through it; both record it and exit normally.
 *   out_gave_up  0 if no wait ran out, else a mask of the warps that came back empty-handed
 *                (bit 0 = warp 0, bit 1 = warp 1; 3 = both, as it must be)
 *   out_ms       duration of the launch
 * The CUDA context stays usable afterwards.
 */
int nbos_probe_wait_timeout(uint64_t limit_ns, void *cuda_stream, int *out_gave_up, float *out_ms);

/*
 * The same self-test reporting where the placement kernel reports: in the status word of `snap`.
 * Afterwards nbos_snapshot_status(snap) returns NBOS_ERR_DEVICE_TIMEOUT, and keeps doing so across
 * nbos_snapshot_update, until the snapshot is destroyed -- which is how a caller learns that some
 * placement on this snapshot gave up on a wait. Synchronises `cuda_stream`.
 */
struct nbos_snapshot;
int nbos_probe_wait_timeout_on_snapshot(struct nbos_snapshot *snap, uint64_t limit_ns, void *cuda_stream,
                                        float *out_ms);

#ifdef __cplusplus
}
#endif
#endif /* NBOS_PROBE_H_ */
