/*
 * adaspark_attn_debug.h - diagnostic entry points of libadaspark_attn (not part of the AdaS-Attn
 * path; the paper has no counterpart).  They exercise hardware building blocks in isolation so
 * that a failure of the attention kernel can be told apart from a failure of its primitives.
 */
#ifndef ADASPARK_ATTN_DEBUG_H_
#define ADASPARK_ATTN_DEBUG_H_

#include <stdint.h>

#include "adaspark_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* One 128x128x128 problem through the tcgen05 path on the current device:
 *   d_out = A * B^T (fp32 [128,128]),  e_out = bf16(d_out / 64) * C^T (fp32 [128,128]),
 * with A, B, C bf16 row-major [128,128] device buffers (16-byte aligned).  `status` is a device
 * int32 the kernel sets to ADASPARK_ERR_TIMEOUT if a bounded wait expired (caller zeroes it).
 * Returns ERR_CUDA if the tensor maps cannot be encoded or the launch fails. */
adaspark_status_t adaspark_attn_debug_umma_selftest(const void *a, const void *b, const void *c,
                                                    float *d_out, float *e_out, int32_t *status,
                                                    void *cuda_stream);

/* One 128x128x128 product through the int8 tcgen05 path: d_out = A * B^T (int32 [128,128]) with A, B
 * signed 8-bit row-major [128,128] device buffers (16-byte aligned).  `status` as above. */
adaspark_status_t adaspark_attn_debug_imma_selftest(const void *a, const void *b, int32_t *d_out,
                                                    int32_t *status, void *cuda_stream);

/* Host only: n / d computed by the multiply-shift routine the kernels use for their index
 * arithmetic (0 <= n < 2^31, 1 <= d < 2^31); -1 for arguments outside that range. */
int32_t adaspark_attn_debug_fastdiv(int32_t n, int32_t d);

/* Exercises the give-up path of the kernels' bounded waits without disturbing a real kernel: one
 * small CTA waits on a barrier at which nothing ever arrives.  After `limit_ns` nanoseconds
 * (1000 <= limit_ns <= 100 000 000, else ERR_INVALID_ARG) the wait expires, the kernel stores
 * ADASPARK_ERR_TIMEOUT in status[0], 1 in status[1] (a second waiting thread was released through
 * the shared abort flag) and the time it waited in *waited_ns, and returns normally; the context
 * stays usable.  `status` is a device int32[2] and `waited_ns` a device uint64, both zeroed by the
 * caller. */
adaspark_status_t adaspark_attn_debug_wait_timeout(uint64_t limit_ns, int32_t *status,
                                                   uint64_t *waited_ns, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ADASPARK_ATTN_DEBUG_H_ */
