/*
 * Test-only C ABI of libmdn_probe.so: bring-up probes for the sm_100a building blocks the
 * tensor-core kernels of libmdn are made of (TMA tiles, tcgen05 products, tensor-memory layouts,
 * bounded waits).  Not part of the product library; built by tests/probe/build_probe.py.
 */
#ifndef MDN_PROBE_H_
#define MDN_PROBE_H_

#include "mdn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Runs one small tcgen05 / TMA case on one CTA (the operand configurations the
 * tensor-core chain kernel uses) so that each can be checked against a host matmul.
 *   mode 0: TMA 128-byte-swizzled load of a [64 x 128] bf16 matrix `a`; out = the raw 16 KB of shared memory
 *   mode 1: out[128 x 64]  = a[128 x 128] * b[64 x 128]^T     (A and B from shared memory, K-major)
 *   mode 2: out[128 x 64]  = a[128 x 64]  * b[64 x 64]^T      (A from tensor memory)
 *   mode 3: out[128 x 128] = 1 - a[128 x 64] * b[64 x 128]    (A from tensor memory, negated; B MN-major via TMA;
 *                                                              accumulating onto a preloaded D)
 *   mode 4: M = 64: a[64 x 128] * b[128 x 128]^T from shared memory into tensor memory pre-filled with -777;
 *           out[128 x 128] = all 128 lanes x 128 columns (shows which lanes the 64 rows of the result occupy)
 *   mode 5: M = 64 with an MN-major B: out[64 x 128] = a[64 x 128] * b[128 x 128], b laid out in shared memory as
 *           mdn_chunk_fwd_keep_states keeps a chunk state (value index x key index, two swizzled blocks)
 * a, b: bf16 row-major device buffers; out: float32 device buffer; status: device int32 (0 = ok).
 */
mdn_status mdn_selftest_umma(int32_t mode, const void* a, const void* b, float* out, int32_t* status,
                             void* cuda_stream);

/*
 * kind::tf32 probes (fp32 operands; row-major device buffers; out float32; status device int32[4], 0 = ok):
 *   mode 0: out[128 x 64]  = a[128 x 128] * b[64 x 128]^T     (A from tensor memory, B K-major fp32 blocks)
 *   mode 1: out[128 x 128] = a[128 x 64]  * b[64 x 128]       (B read MN-major from the same block layout)
 *   mode 2: out[128 x 64]  = (a * b^T) * c[64 x 64]^T, the second product issued right behind the first, whose
 *           accumulator it reads as its A operand;  mode 3: the same with a commit + wait in between
 *   mode 9: out[128 x 64] = a * b^T while a second product, issued right behind the first, overwrites the columns the
 *           first one reads its A operand from (write-after-read through the pipe)
 *   mode 8: stamps of the issuing thread around commits, waits and fences (out[0..19], cycles)
 *   mode 4..7: timings, out[0] = cycles from first issue to completion, out[1] = products issued
 *           (4: tf32 N = 64 A in tensor memory; 5: tf32 N = 128 MN-major B; 6: bf16 N = 64 A in shared memory;
 *            7: as 4 with a commit + wait after every 16 products)
 */
mdn_status mdn_probe_tf32(int32_t mode, const float* a, const float* b, const float* c, float* out, int32_t* status,
                          void* cuda_stream);

/*
 * Cost of one tcgen05 product as a function of its shape: a stream of 4 * reps products D[m x n] += A[m x K] *
 * B[n x K]^T (K = 16 bf16 or 8 tf32 elements), A from tensor memory (a_tmem = 1; a_tmem = 2: bf16 with B read MN-major, n = 128; a_tmem = 3: tf32, sixteen k-steps over 128 columns of A and 64 KB of B, n = 128) or from shared memory, issued by one
 * thread; out[0] = cycles from the first issue to completion, out[1] = products issued.  n in {32, 64, 128, 256},
 * m in {64, 128}.
 */
mdn_status mdn_probe_mma_timing(int32_t tf32, int32_t a_tmem, int32_t n, int32_t m, int32_t reps, float* out,
                                int32_t* status, void* cuda_stream);

/*
 * One CTA waits on an mbarrier nothing arrives at, with the poll limit given (1 .. 2^20): the wait runs out,
 * status[0] becomes the device-timeout code (2), status[1] = 1 (a second thread left its wait on the first one's
 * abort flag), and the kernel returns normally.  No trap, no fault, no unbounded wait.
 */
mdn_status mdn_probe_bounded_wait(uint32_t spin_limit, int32_t* status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MDN_PROBE_H_ */
