/*
 * koala_debug.h -- diagnostic exports of libkoala that are not part of its interface: kernel
 * tuning for A/B runs, a launch counter, a self-test of the bounded-wait error path and a check
 * of the guard words between workspace buffers.  Used by the test-suite and the measurement
 * scripts; nothing here is needed to run the draft-then-verify step.
 */
#ifndef KOALA_DEBUG_H_
#define KOALA_DEBUG_H_

#include "../../include/koala.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Process-wide tuning of the tensor-core matrix multiply (the defaults are chosen for B200):
 * key 1 = shared-memory pipeline stages per CTA (0 = as many as fit, at most 8); key 2 = upper
 * bound on the automatic split-K factor (0 = default); key 3 = 1 switches stream-K off (every CTA
 * stays inside one weight tile); key 5 = weight tiles prefetched into L2 ahead of the pipeline
 * (< 0 = default 0); key 6 = 1 delays the weight stream until the previous kernel has finished;
 * key 7 = divisor of the split-K partial-sum traffic bound (default 8); key 8 = how many pipeline
 * stages request their weight tile before that wait (< 0 = all, the default); key 9 = fewest query
 * rows per sequence for which the tcgen05 attention kernel is used (default 16); key 10 = 1 keeps
 * the one-wave split-K factor when a launch has several token tiles (more than 128 rows);
 * key 11 = 1 keeps 128 weight rows per CTA also for the widest token tiles (MMA N = 256);
 * key 12 = key chunks per (sequence, head) of the tcgen05 attention kernel (0 = chosen from the shape);
 * key 13 = 1 runs pairs of more than 128 tokens as 128-token tiles with the residual rows as extra
 * accumulator columns (the form used up to 128 tokens) instead of 256-token tiles with two accumulating
 * MMAs; key 14 = weight tiles requested into L2 ahead of the ring in the 256-token form (default 0);
 * keys 15 (256-row weight tiles) and 16 (128-row tiles) = 1, 2 or 4: that many epilogue warps per
 * 32 accumulator lanes instead of the default; key 17 = 1: no CTA-pair GEMM kernel, 2: not up to 128
 * rows; key 18 = fewest rows for it (default 113); key 19 = K/V tiles the
 * tcgen05 attention requests into L2 ahead of its ring (default 0); key 20 = 0: no dry pass over its
 * tile loop before the dependency wait; key 21 = 0: no dry pass of the GEMM epilogue warps; key 22 =
 * key chunks of the mma.sync attention kernel (0 = by rule). */
void koala_set_tuning(int key, int value);

/* Kernels launched by the library in this process so far (all contexts). */
uint64_t koala_launch_count(void);

/* Exercises the path a bounded device-side wait takes when it runs out, without anything else in
 * flight: a one-thread kernel on the context's stream initialises an mbarrier that nothing ever
 * arrives at, waits for it for `limit_cycles` SM clock cycles (1 .. 10^8), and on expiry records
 * KOALA_E_TIMEOUT in the context's device status word exactly as the matrix-multiply and
 * attention kernels do.  koala_poll() then reports it.  The status word keeps the code: use a
 * context made for this purpose. */
int koala_selftest_timeout(koala_ctx *ctx, int limit_cycles);

/* Every buffer carved from the workspace is followed by a 256-byte guard that koala_init fills
 * with a fixed pattern and nothing ever writes.  Waits for the context's stream, reads the guards
 * back and counts those that changed (a write past the end of the buffer before it).  n_guards /
 * n_damaged: host ints. */
int koala_debug_check_guards(koala_ctx *ctx, int *n_guards, int *n_damaged);

#ifdef __cplusplus
}
#endif
#endif /* KOALA_DEBUG_H_ */
