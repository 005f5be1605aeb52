/*
 * efqat_aux.h -- measurement and self-test aids of the EfQAT library.  Nothing here is part of
 * the method (the paper has no counterpart to any of these calls) and no compute call depends
 * on them; they exist for benchmarks and for the test of the library's error reporting.  All
 * of their state lives in the efqat_ctx they are given.
 */
#ifndef EFQAT_AUX_H_
#define EFQAT_AUX_H_

#include "efqat.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Per-kernel timing for benchmarks.  While enabled, each of the three tensor-core
 * launches (which = 0 forward GEMM, 1 grad-input GEMM, 2 weight-gradient GEMM) made through
 * `ctx` is bracketed by a pair of CUDA events on the caller's stream.  The events are created
 * by the enabling call (never on the hot path); at most 8192 launches per kind are kept
 * between two reads, later ones are not recorded. */
int efqat_profile_enable(efqat_ctx* ctx, int enable);
/* Synchronises the context's device (which must be current), returns the summed duration
 * (ms) and number of recorded launches of kernel `which` since the previous read, and clears
 * the record. */
int efqat_profile_read(efqat_ctx* ctx, int which, float* ms_total, int* launches);
/* Number of kernels launched through `ctx` since it was created (0 for NULL). */
int64_t efqat_launch_count(efqat_ctx* ctx);

/* Self-test of the bounded in-kernel wait behind EFQAT_DEV_WAIT_TIMEOUT.  Launches one warp
 * that waits, with the library's own wait routine and a limit of limit_ns nanoseconds
 * (1 us .. 1 s, else EFQAT_ERR_SHAPE), on a shared-memory barrier that nothing ever signals;
 * no copy is in flight and no tensor memory is held.  The wait runs out, the kernel records
 * EFQAT_DEV_WAIT_TIMEOUT in the context's status word and returns; the context stays usable.
 * Read the result with efqat_device_status. */
int efqat_selftest_bounded_wait(efqat_ctx* ctx, uint64_t limit_ns, efqat_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* EFQAT_AUX_H_ */
