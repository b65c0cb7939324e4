/*
 * Self-test hook of the B200 residual-VQ library: not part of the quantizer's
 * interface (include/rvq.h), exported so that the error path of the encoder can
 * be exercised on a healthy GPU.
 */
#ifndef RVQ_SELFTEST_H
#define RVQ_SELFTEST_H

#include "rvq.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * rvq_encode with a fault made on purpose on the host side of the kernel's
 * protocol (the paper has no counterpart).  Every wait inside the tensor-core
 * encode kernel is bounded: a wait that runs out raises a flag, all roles of the
 * CTA stop at their next check, the CTA frees its tensor memory and returns, and
 * status->wait_timeouts counts it.  Normally no wait runs out.  Here one MMA
 * issuer per CTA leaves out the last chain it would issue (the one no other work
 * follows, so nothing asynchronous is in flight when the CTA gives up), and the
 * epilogue's wait for that chain gives up after `wait_polls` polls (>= 1024)
 * instead of the regular four million.
 *   arguments as rvq_encode (tensor-core shapes only: group_dim 32); status must
 *   not be NULL.  Returns RVQ_OK after queueing; once the stream has drained
 *   status->wait_timeouts >= 1 and codes / std_f16 are unspecified.  The
 *   context stays usable: a regular rvq_encode afterwards is correct.
 */
int rvq_selftest_encode_timeout(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
                                const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
                                uint32_t wait_polls, rvq_status *status, void *stream /* cudaStream_t */);

#ifdef __cplusplus
}
#endif

#endif
