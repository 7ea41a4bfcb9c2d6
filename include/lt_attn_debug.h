/*
 * lt_attn_debug.h -- test-support entry points of the attention library.
 *
 * These are not part of the product interface (lt_attn.h): the tests use them to pin the
 * tensor-core operand conventions and to exercise the give-up path of the bounded device-side
 * waits without hanging or faulting a GPU.  None has a counterpart in the paper.  Conventions
 * (device pointers, status codes, the 256-byte status block read with lt_attn_check_status) are
 * those of lt_attn.h.
 */
#ifndef LT_ATTN_DEBUG_H_
#define LT_ATTN_DEBUG_H_

#include "lt_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Bring-up check of one tensor-core tile product, used by the tests to pin the
 * shared-memory / tensor-memory operand conventions the attention kernels rely on
 * (no counterpart in the paper; its analogue is the GEMM primitive inside Attention BP,
 * Section 4.1).  Computes C[128,128] (fp32, row-major, device) from fp16 device
 * matrices, each 128 x 128 row-major:
 *   mode 0: C = A  B^T   (A rows = M, B rows = N; both contraction-contiguous)
 *   mode 1: C = A  B     (B rows = contraction index)
 *   mode 2: C = A^T B    (A and B rows = contraction index)
 *   mode 3: C = A  B     (A staged through tensor memory instead of shared memory)
 *   mode 4: as mode 0, with the accumulator read back in the 16-lane x 256-bit
 *           arrangement that the dQ reduction uses
 *   mode 5: C = A B^T + 1000 * B[n][0] added to column n through one extra, unswizzled
 *           contraction step (the way the kernels subtract LSE and delta)
 *   mode 6: no product is read back: the first 96 columns of C receive 1000 * row + column, written
 *           to tensor memory with the two 16-lane store arrangements (64 columns as 32-bit values,
 *           32 columns in the arrangement used for packed 16-bit pairs) and read back with the
 *           32-lane arrangement; checks the register-to-element maps the forward relies on */
int lt_dbg_tile_gemm(const lt_half *A, const lt_half *B, float *C, int mode,
                     void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* Failure-path check used by the tests (no counterpart in the paper): launches one small
 * kernel whose threads wait on a barrier that nothing ever completes.  The wait is bounded
 * (about 10 ms of cycles), after which the kernel records a code in the status block of
 * `workspace` and returns normally; lt_attn_check_status then reports
 * LT_ERR_DEVICE_TIMEOUT and the CUDA context stays usable.  This is the same give-up path
 * every wait inside the attention kernels takes. */
int lt_dbg_wait_timeout(void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* Development builds only (not exported by the product library, hence described, not declared):
 *   -DLT_BWD_TIMELINE=<cta>: `int lt_dbg_bwd_timeline(long long *out)` copies 20 x 256 clock stamps to the
 *     host buffer `out` ([event][tile pair] of that CTA's first 256 tile pairs in the last backward call;
 *     paper_2606_10415_b200/timeline.py names the events and prints them); out == NULL clears the stamps.
 *   -DLT_BWD_TRACE: `int lt_dbg_bwd_trace(unsigned long long *out, int reset)` copies 80 per-role cycle
 *     totals (slot = 16 * role + wait code - 200; 64.. = per-CTA totals) summed over all CTAs. */

#ifdef __cplusplus
}
#endif
#endif /* LT_ATTN_DEBUG_H_ */
