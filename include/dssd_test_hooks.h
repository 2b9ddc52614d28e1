/*
 * dssd_test_hooks.h - entry points for the library's own tests.  NOT part of the product API:
 * they exist so that the bounded waits inside the kernels can be made to run out on purpose,
 * in a way that cannot hang or fault a GPU, and their outcome be checked.  (The paper has no
 * counterpart: its link model of Section 2.2 has no loss or failure term.)
 *
 * Every wait in the kernels - for a partial sum that another CTA stores, for a chunk sum, for a
 * stage of the shared-memory ring - polls a bounded number of times; when the polls run out the
 * waiting code gives up, reports it per sequence (DSSD_EDGE_FLAG_TIMEOUT with accept_len = -1,
 * DSSD_RS_FLAG_TIMEOUT | DSSD_RS_FLAG_INVALID with token = -1) and the kernel ends normally.  The
 * two calls below provoke exactly that by withholding ONE store that a wait depends on and by
 * giving that wait a small poll limit; nothing else about the launch changes, no address is
 * wrong and no wait is unbounded.
 */
#ifndef DSSD_TEST_HOOKS_H
#define DSSD_TEST_HOOKS_H

#include "dssd.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * dssd_edge_verify (always through the streaming kernel) in which the partial sum of target row
 * `drop_row` (0 <= drop_row < B * (gamma + 1)) is computed and counted but never stored, and the
 * fold of a sequence polls at most `poll_limit` times for a missing partial sum.  The sequence
 * that owns the row ends with accept_len = -1 and DSSD_EDGE_FLAG_TIMEOUT and its p_row is not
 * written; every other sequence is verified as usual.  Arguments otherwise as dssd_edge_verify.
 */
dssd_status dssd_test_edge_verify_wait_runs_out(const void *target_logits, dssd_dtype dtype,
                                                int64_t row_stride, const int32_t *draft_tokens,
                                                const float *draft_q_tok, const float *uniforms,
                                                float temperature, int B, int gamma, int V,
                                                int32_t *accept_len, float *p_row, uint32_t *flags,
                                                void *workspace, size_t workspace_bytes,
                                                long long drop_row, unsigned poll_limit,
                                                void *cuda_stream);

/*
 * dssd_device_resample in which the chunk sums of sequence `drop_seq` (0 <= drop_seq < B) are
 * computed but never stored, and a draw polls at most `poll_limit` times for a missing chunk sum.
 * That sequence ends with token = -1 and DSSD_RS_FLAG_TIMEOUT | DSSD_RS_FLAG_INVALID; every other
 * sequence is drawn for as usual.  Arguments otherwise as dssd_device_resample.
 */
dssd_status dssd_test_device_resample_wait_runs_out(const float *p_row, const float *draft_q,
                                                    const int32_t *accept_len,
                                                    const float *uniforms, int B, int gamma, int V,
                                                    int32_t *token, uint32_t *flags,
                                                    void *workspace, size_t workspace_bytes,
                                                    int drop_seq, unsigned poll_limit,
                                                    void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DSSD_TEST_HOOKS_H */
