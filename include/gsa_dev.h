/*
 * libgsa -- development aids (no counterpart in the paper).  Not part of the layer's interface:
 * self-tests of the tensor-core building blocks and of the bounded device-side wait, and the
 * per-kernel timing hooks that the benchmark uses.  Production code includes gsa.h only.
 */
#ifndef GSA_DEV_H_
#define GSA_DEV_H_

#include "gsa.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Self-test of the tensor-core building blocks (no counterpart in the paper): computes one
 * 128-row bf16 product per operand layout the chunk kernels use, from two 128 x 128
 * row-major bf16 device matrices X, Y into D (fp32, row-major):
 *   mode 0: D[128x128] = X Y^T        mode 1: D[128x128] = X Y
 *   mode 2: D[128x64]  = X^T Y[:64]^T mode 3: D[128x64]  = X Y[:, :64]
 *   mode 4: D[128x128] = X Y^T        mode 5: D[128x128] = X Y      (A operand in tensor memory)
 * dev_status (nullable) receives GSA_ERR_TIMEOUT if a bounded wait expired.
 */
GSA_API gsa_status_t gsa_tc_selftest(int32_t mode, const void* X, const void* Y, float* D,
                                     void* stream, int32_t* dev_status);

/*
 * Per-kernel timing for benchmarks (no counterpart in the paper).  Between
 * gsa_timing_begin(capacity) and gsa_timing_end() on the same HOST thread, every kernel
 * that this thread's gsa_* calls enqueue is bracketed by a pair of CUDA events on its
 * stream (up to `capacity` kernels).  gsa_timing_end waits for the last one, writes the
 * duration in milliseconds and a static label of each timed kernel, in launch order, to
 * ms[0..n) / labels[0..n), and returns n (-1 on error or if timing was not active).  These
 * two calls create and destroy events and synchronise with the host: keep them out of
 * production paths.
 */
GSA_API gsa_status_t gsa_timing_begin(int32_t capacity);
GSA_API int32_t gsa_timing_end(float* ms, const char** labels, int32_t capacity);

/*
 * Self-test of the bounded device-side wait (no counterpart in the paper).  One CTA waits, with
 * a limit of limit_us microseconds (1 .. 100000), on an mbarrier that nothing ever signals --
 * the situation the chunk kernels guard against -- gives up, writes GSA_ERR_TIMEOUT to
 * *dev_status (required) and the time it waited to *waited_us (nullable), frees its tensor
 * memory and returns.  Nothing traps or spins without limit; the context stays usable.
 */
GSA_API gsa_status_t gsa_wait_selftest(uint32_t limit_us, void* stream, int32_t* dev_status, uint32_t* waited_us);

/*
 * Development switch (no counterpart in the paper).  The backward's four time-reversed scans share
 * their states in pairs (dv with dI^v, dk with dI^k; App. B) and by default run as two kernels that
 * compute a pair each.  enable == 0 makes later gsa_bwd calls of this process run four single scans
 * instead (same results up to the rounding order of a few fp32 additions); non-zero restores the
 * default.  Returns the previous setting.  Process-wide; takes effect at the next call.
 */
GSA_API int32_t gsa_dev_pair_scans(int32_t enable);

#ifdef __cplusplus
}
#endif
#endif /* GSA_DEV_H_ */
