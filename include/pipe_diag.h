/*
 * pipe_diag.h -- diagnostic and test-only entry points of libpipe.
 *
 * Nothing here belongs to the method of the paper (arXiv 2311.15806) and no production caller needs it:
 * these calls exist so that tests can force a GEMM back end, so that the benchmark can measure the
 * integer tensor-core issue rate that its roofline fractions are quoted against, and so that the
 * bounded-wait path of the kernels (PIPE_ERR_TIMEOUT) can be exercised without withholding a signal
 * inside a production kernel.  Conventions are those of pipe.h.
 */
#ifndef PIPE_DIAG_H_
#define PIPE_DIAG_H_

#include "pipe.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Which GEMM kernel the forward calls use from now on, for the whole process (so only for tests and
 * measurements; concurrent users of the library would all see the change):
 * 0 = automatic, 1 = CUDA-core kernel, 2 = one-SM tcgen05 kernel, 3 = small-token weight-streaming kernel,
 * 4 = SM-pair tcgen05 kernel (clusters of two CTAs), 5 = small-token tcgen05 kernel.  A forced kernel that cannot run a request makes the
 * forward call return PIPE_ERR_UNSUPPORTED. */
pipe_status pipe_diag_select_kernel(int32_t which);

/* Issue-bound rate of tcgen05.mma kind::i8 on this device: one CTA per SM issues `mma_per_cta`
 * instructions of shape M = 128, N = n_cols (16..256, a multiple of 16), K = 32 on operands that stay in
 * shared memory (no loads, no epilogue), alternating between two accumulators.  cta_pairs != 0: the CTAs
 * run as clusters of two and the first CTA of each pair issues `mma_per_cta` instructions of the two-SM
 * form (cta_group::2, M = 256, each CTA holding half of the n_cols rows of B).  The work is queued on
 * `stream`; the caller times it (CUDA events) and divides *h_ops_per_launch -- the integer operations
 * (2 per multiply-accumulate) of the whole launch -- by the duration.  Allocates nothing. */
pipe_status pipe_diag_mma_i8_rate(int32_t n_cols, int64_t mma_per_cta, int32_t cta_pairs, double* h_ops_per_launch,
                                  void* stream);

/* Exercises the bounded wait of the kernels: one CTA initialises an mbarrier on which nobody ever arrives and
 * waits on it with the library's own wait routine, limited to `limit_cycles` SM cycles (1..2^31).  The wait
 * runs out, the kernel records PIPE_ERR_TIMEOUT in the device status word (read it with pipe_poll_status) and
 * returns normally; the device stays usable. */
pipe_status pipe_diag_bounded_wait(int64_t limit_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PIPE_DIAG_H_ */
