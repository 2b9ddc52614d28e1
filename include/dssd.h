/*
 * dssd.h - C ABI of the split speculative verification library for NVIDIA B200 (sm_100a).
 *
 * One verification round of Distributed Split Speculative Decoding (DSSD, Algorithm 2 of the
 * paper) for B independent sequences:
 *
 *   dssd_edge_verify      the edge (base-station) half: "Verification Process" and the
 *                         payload of "Downlink Transmission" (Section 3, Algorithm 2);
 *   dssd_device_resample  the device half: "Resample" (Section 3, Algorithm 2), plus the
 *                         bonus draw x_{gamma+1} ~ P_{gamma+1} that Algorithm 2 performs when
 *                         every draft token was accepted;
 *   dssd_round_host       both halves on host buffers, with the copies to and from the GPU;
 *   dssd_edge_verify_topk, dssd_device_resample_topk, dssd_round_host_topk
 *                         the same round on distributions truncated to their k most likely
 *                         tokens, the sampler of the paper's experiments (Section 4);
 *   dssd_edge_verify_p16, dssd_device_resample_p16
 *                         the round with the downlink row in 16 bits per value (Section 2.2);
 *   dssd_dsd_verify       the fused verification of Algorithm 1 (no row is transmitted);
 *   dssd_edge_partial, dssd_edge_combine, dssd_edge_emit_shard, dssd_resample_shard_mass,
 *   dssd_resample_shard_draw
 *                         the round for an edge whose vocabulary is sharded over several GPUs.
 *
 * Notation follows the paper: gamma draft tokens x_1..x_gamma with draft probabilities
 * q_i(x_i), target distributions P_1..P_{gamma+1} over a vocabulary of V entries, uniforms
 * r_i.  Indices here are 0-based: accept_len n = j - 1, where j is the paper's 1-based position
 * of the first rejected token (j = gamma + 1, n = gamma, when all drafts were accepted).
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - The caller owns every buffer.  The library allocates no memory, enqueues its work on the
 *     given CUDA stream and returns without synchronising.  It keeps no state between calls except
 *     per-device launch constants (SM count, resident CTAs per kernel), which are looked up on the
 *     first call made with a device current and cached, and the built-in scratch of
 *     dssd_device_resample_static.
 *   - The streaming kernels are launched cooperatively (every CTA resident at once): two calls
 *     issued to different streams run one after the other on the GPU, not side by side.
 *   - Every call with device pointers only can be recorded in a CUDA graph by stream capture
 *     (it enqueues kernels and nothing else), provided one call of the same entry point was made
 *     on that device before the capture began (the first call looks the launch constants up).
 *     dssd_round_host synchronises the stream in the middle and cannot be captured.
 *   - Buffers need only their natural alignment; 16-byte aligned rows take the fast path.
 *   - A status other than DSSD_OK means nothing was enqueued (except DSSD_ERR_CUDA, after
 *     which the outputs are undefined).  Data-dependent anomalies never fault or trap: they
 *     are reported per sequence in the flags outputs.
 *   - Calls that share a workspace must not overlap on the GPU.
 */
#ifndef DSSD_H
#define DSSD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DSSD_OK = 0,
    DSSD_ERR_INVALID_ARG = 1, /* NULL required pointer, B < 1, gamma < 0, V < 1, T <= 0 or not finite, row_stride < V */
    DSSD_ERR_UNSUPPORTED = 2, /* a size beyond DSSD_MAX_* or an unknown dtype */
    DSSD_ERR_WORKSPACE = 3,   /* workspace NULL, misaligned (256 bytes) or too small */
    DSSD_ERR_CUDA = 4         /* a CUDA call failed; see dssd_last_cuda_error() */
} dssd_status;

typedef enum {
    DSSD_F32 = 0, /* IEEE binary32 logits  */
    DSSD_BF16 = 1 /* bfloat16 logits       */
} dssd_dtype;

#define DSSD_MAX_V (1 << 30)
#define DSSD_MAX_ROWS 0x7fffffff /* B * (gamma + 1) */

/* flags written by dssd_edge_verify, one word per sequence */
#define DSSD_EDGE_FLAG_BAD_TOKEN 1u /* some x_i outside [0, V): that position is rejected        */
#define DSSD_EDGE_FLAG_NONFINITE 2u /* some row of the sequence has no finite log-sum-exp (NaN,  \
                                       +inf, or all -inf): that position is rejected, its row is NaN */
#define DSSD_EDGE_FLAG_TIMEOUT 4u   /* internal wait ran out; p_row of this sequence was not written */

/* flags written by dssd_device_resample, one word per sequence */
#define DSSD_RS_FLAG_BONUS 1u    /* n == gamma: token drawn from P_{gamma+1}                       */
#define DSSD_RS_FLAG_FALLBACK 2u /* residual mass sum max(0, p - q) <= 0: token drawn from p instead */
#define DSSD_RS_FLAG_INVALID 4u  /* no positive mass at all, or n outside [0, gamma]: token = -1    */
#define DSSD_RS_FLAG_TIMEOUT 8u  /* internal wait ran out: token = -1 (set together with INVALID)    */

/* Human-readable name of a status (static storage, never NULL). */
const char *dssd_status_string(int status);

/* Library version, major * 10000 + minor * 100 + patch. */
int dssd_version(void);

/* CUDA error code (cudaError_t as int) behind the calling thread's last DSSD_ERR_CUDA, else 0. */
int dssd_last_cuda_error(void);

/*
 * Bytes of scratch that dssd_edge_verify needs for these sizes (0 if the sizes are invalid).
 * Depends on the sizes only, not on the GPU.
 */
size_t dssd_edge_verify_workspace_bytes(int B, int gamma, int V);

/*
 * Edge half of one round (Algorithm 2, "Verification Process" at the edge and the payload of
 * "Downlink Transmission"; Section 3).
 *
 * For every sequence b and position i = 0..gamma the target distribution is
 *   P_i(v) = softmax(l_{b,i,v} / T)                      (temperature: Section 4)
 * computed through the row's log-sum-exp.  Draft token x_i is accepted iff
 *   u_i < min(1, p_i(x_i) / q_i(x_i))
 * (Algorithm 2 prints the ratio upside down; this direction is the one consistent with the
 * residual max(0, P - Q) of the "Resample" step).  n is the first position that fails, or gamma.
 * The single row P_n(.) - the rejected position's target distribution, or the bonus position's
 * when n == gamma - is written in float32: it is the downlink payload of Section 3.1
 * (b_prob = 32).  Unlike the paper, the row is also written when n == gamma, so that
 * dssd_device_resample can draw the bonus token; a caller that wants the paper's byte saving
 * simply does not transmit it.
 *
 * Arithmetic: with c1 = float32(log2(e) / T), every term 2^(l_v * c1 - ref) is formed in float32
 * (one fused multiply-add, one ex2 of relative error 2^-22) and added up in float32 per lane, at
 * most a few hundred terms per accumulator; the per-lane sums are combined in float64 by exact
 * power-of-two scaling.  p_i(x_i) = 2^(l_x * c1 - ref) / S and the test u * q < p are evaluated in
 * float64.  The result is within about 1e-6 relative of the exact softmax as long as
 * |l| * log2(e) / T stays well inside the float32 range (the rounding of c1 alone contributes
 * 6e-8 * |l_v / T - E_p[l / T]| to ln p); rows whose scaled logits overflow float32 are flagged
 * DSSD_EDGE_FLAG_NONFINITE.  u == 1 never accepts; q <= 0 accepts iff p > 0; a NaN q or an
 * out-of-range token rejects.
 *
 * target_logits  [B, gamma+1, V] of `dtype`, unit stride along V, `row_stride` elements between
 *                consecutive rows (>= V); row (b, i) starts at element (b*(gamma+1)+i)*row_stride
 * draft_tokens   [B, gamma] int32      x_i          (may be NULL iff gamma == 0)
 * draft_q_tok    [B, gamma] float32    q_i(x_i)     (may be NULL iff gamma == 0)
 * uniforms       [B, gamma] float32    u_i in [0,1) (may be NULL iff gamma == 0)
 * temperature    T > 0, finite
 * accept_len     [B] int32     out: n in [0, gamma]; -1 (with DSSD_EDGE_FLAG_TIMEOUT) if an internal wait ran out
 * p_row          [B, V] float32 out: P_n(.)
 * p_tok          [B, gamma] float32   out, optional (NULL ok): p_i(x_i)
 * lse            [B, gamma+1] float32 out, optional (NULL ok): ln sum_v exp(l_v / T)
 * flags          [B] uint32    out, optional (NULL ok): DSSD_EDGE_FLAG_*
 * workspace      >= dssd_edge_verify_workspace_bytes(B, gamma, V) bytes, 256-byte aligned;
 *                contents need not be initialised and are garbage afterwards
 * cuda_stream    cudaStream_t (NULL = the legacy default stream)
 */
dssd_status dssd_edge_verify(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                             const int32_t *draft_tokens, const float *draft_q_tok,
                             const float *uniforms, float temperature, int B, int gamma, int V,
                             int32_t *accept_len, float *p_row, float *p_tok, float *lse,
                             uint32_t *flags, void *workspace, size_t workspace_bytes,
                             void *cuda_stream);

/* Bytes of scratch that dssd_device_resample needs (0 if the sizes are invalid). */
size_t dssd_device_resample_workspace_bytes(int B, int gamma, int V);

/*
 * Device half of one round (Algorithm 2, "Resample"; Section 3 "Verification Process (on
 * Device)"), and the bonus draw of Algorithm 2's "Sample x_{gamma+1} ~ P_{gamma+1}".
 *
 * For a rejected sequence (n < gamma):  r_v = max(0, p_v - q_{n,v}),  Z = sum_v r_v,
 *   token = min{k : sum_{v<=k} r_v > u' * Z}      (inverse CDF in index order, float64 sums);
 * for n == gamma the same draw with r = p.  If rounding leaves no such k the last index with
 * r_v > 0 is returned.  If Z <= 0 (p == q) the draw falls back to r = p and sets
 * DSSD_RS_FLAG_FALLBACK.
 *
 * p_row       [B, V] float32        the row produced by dssd_edge_verify (the downlink payload)
 * draft_q     [B, gamma, V] float32 the device's own Q_i(.); only row n of each sequence is read
 *                                   (may be NULL iff gamma == 0)
 * accept_len  [B] int32             n
 * uniforms    [B] float32           u' in [0,1)
 * token       [B] int32   out
 * flags       [B] uint32  out, optional (NULL ok): DSSD_RS_FLAG_*
 * workspace   >= dssd_device_resample_workspace_bytes(B, gamma, V) bytes, 256-byte aligned
 */
dssd_status dssd_device_resample(const float *p_row, const float *draft_q,
                                 const int32_t *accept_len, const float *uniforms, int B,
                                 int gamma, int V, int32_t *token, uint32_t *flags,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * dssd_device_resample without a caller-provided workspace.  (The paper has no counterpart: this
 * entry point exists for the library's users, not for the method.)
 *
 * Some callers cannot allocate device memory at the point where they sample: code running inside
 * a serving loop whose memory pool is frozen after start-up, a plugin that is handed input and
 * output buffers by its host framework and nothing else, or a process whose allocator must not be
 * touched while other work is in flight.  For them the scratch lives inside the library: a fixed
 * array of DSSD_STATIC_SCRATCH_BYTES bytes in the library's device image, which every GPU that
 * loads the library holds until the process exits.  The call itself allocates nothing and frees
 * nothing.
 *
 * Same inputs, outputs and results as dssd_device_resample (the two share the kernel).
 *   - Sizes whose scratch need (dssd_device_resample_workspace_bytes: 256 bytes of counters plus
 *     8 bytes per 4096 vocabulary entries per sequence) exceeds DSSD_STATIC_SCRATCH_BYTES, i.e.
 *     B * ceil(V / 4096) > 131 040, are refused with DSSD_ERR_UNSUPPORTED before anything is
 *     enqueued; use dssd_device_resample for those.
 *   - The first call made with a given device current looks up the array's device address (once
 *     per device ordinal, for the context current at that moment: a process that creates a second
 *     context on the same device must not use this entry point from it).  Make that first call
 *     during set-up, before any stream capture is begun.
 *   - Every call on a device uses the same array.  Each call clears the counters it needs and
 *     overwrites the rest before reading it, so calls that follow one another on a stream are
 *     independent; two calls that run on the GPU at the same time (different streams, or
 *     different host threads without ordering) race on the array and give undefined results.
 */
#define DSSD_STATIC_SCRATCH_BYTES (1 << 20)
dssd_status dssd_device_resample_static(const float *p_row, const float *draft_q,
                                        const int32_t *accept_len, const float *uniforms, int B,
                                        int gamma, int V, int32_t *token, uint32_t *flags,
                                        void *cuda_stream);

/* Bytes of device memory that dssd_round_host needs as its arena (0 if the sizes are invalid). */
size_t dssd_round_host_arena_bytes(int B, int gamma, int V, dssd_dtype dtype);

/*
 * Both halves of Algorithm 2's verification on HOST buffers: copies the inputs to the GPU,
 * runs dssd_edge_verify and dssd_device_resample, and copies the results back, all enqueued on
 * `cuda_stream`.  The host buffers must stay valid until the stream has finished; use pinned
 * memory for the copies to be asynchronous.
 *
 * Of the draft distributions only the rows the device half reads cross the bus: the call waits
 * on the host for the accepted lengths (one cudaStreamSynchronize in the middle; accept_len is
 * final when the call returns) and then uploads row Q_n of every sequence with a rejection,
 * B * V * 4 bytes at most instead of B * gamma * V * 4.  Because of that wait the call cannot be
 * made while the stream is being captured (DSSD_ERR_CUDA then).
 *
 * host inputs:  target_logits [B, gamma+1, V] contiguous, draft_tokens, draft_q_tok, uniforms
 *               [B, gamma], draft_q [B, gamma, V], uniforms_rs [B]
 * host outputs: accept_len [B], token [B], edge_flags [B] (NULL ok), rs_flags [B] (NULL ok),
 *               p_row [B, V] (NULL ok: the row then stays on the GPU)
 * device_arena  device memory, >= dssd_round_host_arena_bytes(...) bytes, 256-byte aligned
 */
dssd_status dssd_round_host(const void *target_logits, dssd_dtype dtype,
                            const int32_t *draft_tokens, const float *draft_q_tok,
                            const float *uniforms, const float *draft_q, const float *uniforms_rs,
                            float temperature, int B, int gamma, int V, int32_t *accept_len,
                            int32_t *token, uint32_t *edge_flags, uint32_t *rs_flags,
                            float *p_row, void *device_arena, size_t arena_bytes,
                            void *cuda_stream);

/*
 * ---------------------------------------------------------------------------------------------
 * Truncated-support round (Section 4: the experiments sample with top-k, k = 10, T = 1).
 *
 * Reading of "top-k sampling": a model's distribution is restricted to its k most likely tokens
 * and renormalised over them.  The support of a target row is its k largest logits; equal logits
 * are ordered by vocabulary index, lower index first, so the support is unique.  Inside it
 *   P(v) = exp(l_v / T - m) / sum_{w in support} exp(l_w / T - m),   m = max_w l_w / T,
 * outside it P(v) = 0.  The draft side truncates its own distributions the same way before it
 * samples.  Algorithm 2 then runs unchanged on the truncated P and Q; the downlink payload of
 * Section 3.1 shrinks from |V| values to k (index, value) pairs.
 * ---------------------------------------------------------------------------------------------
 */
#define DSSD_TOPK_MAX 32

/* Bytes of scratch that dssd_edge_verify_topk needs (0 if the sizes are invalid). */
size_t dssd_edge_verify_topk_workspace_bytes(int B, int gamma, int V, int k);

/*
 * Edge half of one round on truncated target distributions (Algorithm 2, "Verification Process"
 * and the payload of "Downlink Transmission", with the sampler of Section 4).
 *
 * Inputs as dssd_edge_verify; draft_q_tok holds the draft's truncated q_i(x_i).  A drafted token
 * outside the target row's support has p_i(x_i) = 0 and is rejected.  All probabilities and the
 * acceptance test are evaluated in float64; the logits are read exactly once.
 *
 * k           1 <= k <= min(V, DSSD_TOPK_MAX)
 * accept_len  [B] int32        out: n in [0, gamma]
 * p_idx       [B, k] int32     out: support of row n, most likely first (equal logits: lower
 *                              index first); -1 everywhere for a row flagged NONFINITE
 * p_val       [B, k] float32   out: its probabilities, same order (NaN for a NONFINITE row)
 * p_tok       [B, gamma] float32 out, optional (NULL ok): p_i(x_i)
 * flags       [B] uint32       out, optional (NULL ok): DSSD_EDGE_FLAG_BAD_TOKEN / _NONFINITE
 *                              (a row holding NaN or +inf, or nothing above -inf)
 * workspace   >= dssd_edge_verify_topk_workspace_bytes(B, gamma, V, k) bytes, 256-byte aligned;
 *             contents need not be initialised and are garbage afterwards
 */
dssd_status dssd_edge_verify_topk(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                                  const int32_t *draft_tokens, const float *draft_q_tok,
                                  const float *uniforms, float temperature, int B, int gamma,
                                  int V, int k, int32_t *accept_len, int32_t *p_idx, float *p_val,
                                  float *p_tok, uint32_t *flags, void *workspace,
                                  size_t workspace_bytes, void *cuda_stream);

/*
 * Device half on truncated distributions (Algorithm 2, "Resample", and the bonus draw).
 *
 * The residual max(0, P_n - Q_n) lives on P_n's support, so the draw walks P_n's k entries in
 * increasing vocabulary index - the order dssd_device_resample walks the vocabulary in - with
 * Q_n looked up by index (0 where Q_n has no such entry; the first listed if an index occurs
 * twice):  r_e = max(0, p_e - q_n(idx_e)),  Z = sum r_e,  token = idx of the first entry whose
 * running sum exceeds u' * Z; for n == gamma the same with r = p.  Fallback and flags as in
 * dssd_device_resample.  Sums run sequentially in float64, so results are reproducible bit for bit.
 *
 * p_idx, p_val  [B, k]         the pairs dssd_edge_verify_topk wrote; the indices of a sequence
 *                              must be distinct; a negative index marks a sequence without a row
 *                              (token = -1, DSSD_RS_FLAG_INVALID)
 * q_idx, q_val  [B, gamma, k]  the draft's truncated Q_i; only row n is read (may be NULL iff
 *                              gamma == 0)
 * accept_len    [B] int32;  uniforms [B] float32 u' in [0,1)
 * token         [B] int32 out;  flags [B] uint32 out, optional (NULL ok): DSSD_RS_FLAG_*
 * Needs no workspace.
 */
dssd_status dssd_device_resample_topk(const int32_t *p_idx, const float *p_val,
                                      const int32_t *q_idx, const float *q_val,
                                      const int32_t *accept_len, const float *uniforms, int B,
                                      int gamma, int k, int32_t *token, uint32_t *flags,
                                      void *cuda_stream);

/* Bytes of device memory that dssd_round_host_topk needs as its arena (0 if the sizes are invalid). */
size_t dssd_round_host_topk_arena_bytes(int B, int gamma, int V, int k, dssd_dtype dtype);

/*
 * Both halves of the truncated-support round on HOST buffers: copies the inputs to the GPU, runs
 * dssd_edge_verify_topk and dssd_device_resample_topk, and copies the results back, all enqueued
 * on `cuda_stream` (the draft side's lists are k pairs per position, so all of them are
 * uploaded and nothing is waited for: unlike dssd_round_host the call returns without
 * synchronising and can be captured).  The host buffers must stay valid until the stream has
 * finished; use pinned memory for the copies to be asynchronous.
 *
 * host inputs:  target_logits [B, gamma+1, V] contiguous, draft_tokens, draft_q_tok, uniforms
 *               [B, gamma], q_idx, q_val [B, gamma, k], uniforms_rs [B]
 * host outputs: accept_len [B], token [B], edge_flags [B] (NULL ok), rs_flags [B] (NULL ok),
 *               p_idx, p_val [B, k] (NULL ok: the downlink pairs then stay on the GPU)
 * device_arena  device memory, >= dssd_round_host_topk_arena_bytes(...) bytes, 256-byte aligned
 * Errors as for dssd_edge_verify_topk; DSSD_ERR_WORKSPACE for a missing, misaligned or short arena.
 */
dssd_status dssd_round_host_topk(const void *target_logits, dssd_dtype dtype,
                                 const int32_t *draft_tokens, const float *draft_q_tok,
                                 const float *uniforms, const int32_t *q_idx, const float *q_val,
                                 const float *uniforms_rs, float temperature, int B, int gamma, int V,
                                 int k, int32_t *accept_len, int32_t *token, uint32_t *edge_flags,
                                 uint32_t *rs_flags, int32_t *p_idx, float *p_val, void *device_arena,
                                 size_t arena_bytes, void *cuda_stream);

/*
 * ---------------------------------------------------------------------------------------------
 * 16-bit downlink payload (Section 2.2: a probability value takes b_prob = 32 or 16 bits; the
 * payload |V| * b_prob of Section 3.1 halves).
 *
 * Reading of "16 bits": IEEE binary16, each probability rounded once to nearest-even.  Values
 * below 2^-25 become 0 and those below 2^-14 are subnormal, so the far tail of a row loses its
 * mass; the relative error of a normal value is at most 2^-11.
 * ---------------------------------------------------------------------------------------------
 */

/*
 * dssd_edge_verify with the row P_n(.) written as binary16 bit patterns.  Everything else -
 * inputs, decisions, accept_len, p_tok, lse, flags, workspace - is as in dssd_edge_verify; the
 * kernel writes half the bytes.  The probabilities are computed in float32 as there and rounded
 * once more, so a value may differ from the float64 value's rounding by one unit in the last
 * place of binary16.
 *
 * p_row16  [B, V] uint16 out: binary16 bit patterns of P_n(.), 2-byte aligned (8-byte aligned rows
 *          take the fast path)
 */
dssd_status dssd_edge_verify_p16(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                                 const int32_t *draft_tokens, const float *draft_q_tok,
                                 const float *uniforms, float temperature, int B, int gamma, int V,
                                 int32_t *accept_len, uint16_t *p_row16, float *p_tok, float *lse,
                                 uint32_t *flags, void *workspace, size_t workspace_bytes,
                                 void *cuda_stream);

/*
 * dssd_device_resample on a binary16 row: every p_v is widened exactly to float32 and the draw
 * is the one of dssd_device_resample (same sums in float64, same flags, same workspace size).
 */
dssd_status dssd_device_resample_p16(const uint16_t *p_row16, const float *draft_q,
                                     const int32_t *accept_len, const float *uniforms, int B,
                                     int gamma, int V, int32_t *token, uint32_t *flags,
                                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * ---------------------------------------------------------------------------------------------
 * Fused verification of Algorithm 1 (DSD, the scheme the paper's split round is measured against):
 * the edge holds the uploaded draft rows Q_i(.), so it tests every position with q_i(x_i) read
 * from the row and draws the corrected token from norm(max(0, P_n - Q_n)), or the bonus token from
 * P_{gamma+1}, itself.  No row P_n is written or read back: the draw forms p_v from row n's
 * logits on the fly with the log-sum-exp the first pass left behind.
 * ---------------------------------------------------------------------------------------------
 */

/* Bytes of scratch that dssd_dsd_verify needs (0 if the sizes are invalid). */
size_t dssd_dsd_verify_workspace_bytes(int B, int gamma, int V);

/*
 * Acceptance rule, first-rejection scan, flags: as dssd_edge_verify.  Draw: as dssd_device_resample,
 * with p_v = the float32 value dssd_edge_verify would have emitted, so that the token equals the one
 * the two split calls give on the same inputs.
 *
 * target_logits [B, gamma+1, V] as in dssd_edge_verify;  draft_q [B, gamma, V] float32, contiguous
 * draft_tokens, uniforms [B, gamma];  uniforms_rs [B]      (draft_* and uniforms may be NULL iff gamma == 0)
 * accept_len [B] int32 out;  token [B] int32 out
 * edge_flags [B] uint32 out, optional: DSSD_EDGE_FLAG_*;  rs_flags [B] uint32 out, optional: DSSD_RS_FLAG_*
 * workspace  >= dssd_dsd_verify_workspace_bytes(B, gamma, V) bytes, 256-byte aligned
 */
dssd_status dssd_dsd_verify(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                            const float *draft_q, const int32_t *draft_tokens, const float *uniforms,
                            const float *uniforms_rs, float temperature, int B, int gamma, int V,
                            int32_t *accept_len, int32_t *token, uint32_t *edge_flags,
                            uint32_t *rs_flags, void *workspace, size_t workspace_bytes,
                            void *cuda_stream);

/*
 * ---------------------------------------------------------------------------------------------
 * The bonus token drawn at the edge (Algorithm 2, "if j = gamma + 1: sample x_{gamma+1} ~
 * P_{gamma+1}" inside the edge's verification loop; Section 3, "Downlink Transmission": after a
 * round without rejection the downlink carries a token, not a row, which is the a = 0 term of the
 * latency model of Section 3.1).  dssd_edge_verify hands the bonus row to the device instead; the
 * two calls below follow the printed algorithm: a row P_n(.) is emitted only for sequences with a
 * rejection, and a fully accepted sequence gets its token at the edge, drawn straight from row
 * gamma's logits (no row is written for it, none is read back).
 * ---------------------------------------------------------------------------------------------
 */

/* Bytes of scratch that dssd_edge_verify_bonus needs (0 if the sizes are invalid). */
size_t dssd_edge_verify_bonus_workspace_bytes(int B, int gamma, int V);

/*
 * dssd_edge_verify plus the bonus draw.  Decisions, accept_len, p_tok, lse, flags as there.
 *
 * uniforms_bonus [B] float32  u' in [0,1): read for fully accepted sequences only
 * p_row          [B, V] float32 out: row b is written iff accept_len[b] < gamma; the rows of
 *                fully accepted sequences keep their previous contents
 * token          [B] int32 out: the bonus token min{k : sum_{v<=k} p_v > u' * sum_v p_v} where
 *                accept_len[b] == gamma (p_v the float32 value dssd_edge_verify would have
 *                emitted, sums in float64), -1 elsewhere
 * token_flags    [B] uint32 out, optional (NULL ok): DSSD_RS_FLAG_BONUS (| _INVALID for a row
 *                without mass) where accept_len[b] == gamma, 0 elsewhere
 * workspace      >= dssd_edge_verify_bonus_workspace_bytes(B, gamma, V) bytes, 256-byte aligned;
 *                contents need not be initialised and are garbage afterwards
 * Passing `token` and `token_flags` on to dssd_device_resample_rejected completes the round.
 */
dssd_status dssd_edge_verify_bonus(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                                   const int32_t *draft_tokens, const float *draft_q_tok,
                                   const float *uniforms, const float *uniforms_bonus,
                                   float temperature, int B, int gamma, int V, int32_t *accept_len,
                                   float *p_row, int32_t *token, float *p_tok, float *lse,
                                   uint32_t *flags, uint32_t *token_flags, void *workspace,
                                   size_t workspace_bytes, void *cuda_stream);

/*
 * dssd_device_resample for the rejected sequences only (Algorithm 2, "Resample"): where
 * accept_len[b] < gamma the residual draw is made and token[b], flags[b] are written; where
 * accept_len[b] == gamma nothing is read of row b and token[b], flags[b] are left as they are
 * (the bonus token arrived with the downlink).  accept_len outside [0, gamma]: token -1,
 * DSSD_RS_FLAG_INVALID.  Arguments and workspace size as dssd_device_resample.
 */
dssd_status dssd_device_resample_rejected(const float *p_row, const float *draft_q,
                                          const int32_t *accept_len, const float *uniforms, int B,
                                          int gamma, int V, int32_t *token, uint32_t *flags,
                                          void *workspace, size_t workspace_bytes,
                                          void *cuda_stream);

/*
 * ---------------------------------------------------------------------------------------------
 * Vocabulary-sharded round.  (The paper runs the target model on one GPU; this is Algorithm 2,
 * "Verification Process" / "Downlink Transmission" / "Resample" of Section 3, unchanged, for an
 * edge whose LM head is tensor-parallel: GPU g of G holds entries [v_g, v_{g+1}) of every logit
 * row.  Only the sums over the vocabulary are formed shard by shard.)
 *
 *   1. every shard: dssd_edge_partial          per row, its slice's share of sum_v exp(l_v / T)
 *   2. exchange:    all-gather of part_ref, part_sum [B, gamma+1] and tok_logit [B, gamma]
 *                   (a few bytes per row; the caller's collective, e.g. NCCL)
 *   3. every shard: dssd_edge_combine          log-sum-exp, acceptance test, first rejection n:
 *                                              identical inputs give identical results everywhere
 *   4. every shard: dssd_edge_emit_shard       its slice of the downlink row P_n
 *   5. every shard: dssd_resample_shard_mass   its slice's residual mass and plain mass
 *   6. exchange:    all-gather of mass [B, 2]
 *   7. every shard: dssd_resample_shard_draw   the shard that holds u' Z returns the token, the
 *                                              others -1 (a max over shards completes the round)
 * Steps 5-7 are the device half for a device that holds the rows sharded the same way; a device
 * that receives whole rows calls dssd_device_resample on the assembled row instead.
 * The library makes no collective call itself and never reads another GPU's memory.
 * ---------------------------------------------------------------------------------------------
 */

/* Bytes of scratch that dssd_edge_partial needs (0 if the sizes are invalid). */
size_t dssd_edge_partial_workspace_bytes(int B, int gamma, int V_shard);

/*
 * One shard's share of every row's log-sum-exp (Section 3, "Verification Process").
 *
 * logits_shard  this shard's slice of the target logits: row (b, i) starts at element
 *               (b*(gamma+1)+i)*row_stride and holds V_shard entries, vocabulary ids
 *               v_begin .. v_begin + V_shard - 1 (a view into whole rows works: row_stride >= V_shard)
 * draft_tokens  [B, gamma] int32  x_i, ids in the whole vocabulary (may be NULL iff gamma == 0)
 * part_ref      [B, gamma+1] float32 out, integer-valued, and
 * part_sum      [B, gamma+1] float64 out:  sum_{v in slice} 2^(l_v * c1) = part_sum * 2^part_ref with
 *               c1 = float32(log2(e) / T); (0, 0) for a slice of -inf only; part_sum is NaN for a
 *               slice that holds a NaN or +inf
 * tok_logit     [B, gamma] float32 out: l_{x_i} where v_begin <= x_i < v_begin + V_shard, NaN
 *               elsewhere (may be NULL iff gamma == 0)
 * workspace     >= dssd_edge_partial_workspace_bytes(B, gamma, V_shard) bytes, 256-byte aligned;
 *               contents need not be initialised and are garbage afterwards
 */
dssd_status dssd_edge_partial(const void *logits_shard, dssd_dtype dtype, int64_t row_stride,
                              const int32_t *draft_tokens, int v_begin, float temperature, int B,
                              int gamma, int V_shard, float *part_ref, double *part_sum,
                              float *tok_logit, void *workspace, size_t workspace_bytes,
                              void *cuda_stream);

/*
 * The shards' partial sums -> log-sum-exp of every row, p_i(x_i), the acceptance test
 * u_i < min(1, p_i(x_i) / q_i(x_i)) and the first rejection n (Algorithm 2, "Verification
 * Process"), evaluated exactly as dssd_edge_verify evaluates them.
 *
 * part_ref, part_sum  [G, B, gamma+1], tok_logit [G, B, gamma]: the outputs of the G calls of
 *               dssd_edge_partial, shard-major (the layout an all-gather leaves)
 * temperature   the T the partial sums were formed with
 * V             size of the whole vocabulary (ids outside [0, V) are rejected and flagged)
 * accept_len    [B] int32 out;  p_tok [B, gamma], lse [B, gamma+1], flags [B] out, optional
 * row_scale     [B, 2] float32 out: row n's reference exponent and 1 / sum, which
 *               dssd_edge_emit_shard turns logits into probabilities with
 */
dssd_status dssd_edge_combine(const float *part_ref, const double *part_sum, const float *tok_logit,
                              int G, const int32_t *draft_tokens, const float *draft_q_tok,
                              const float *uniforms, float temperature, int B, int gamma, int V,
                              int32_t *accept_len, float *row_scale, float *p_tok, float *lse,
                              uint32_t *flags, void *cuda_stream);

/*
 * This shard's slice of the downlink row (Section 3, "Downlink Transmission"; b_prob = 32):
 * p_row_shard[b, v] = P_n(v_begin + v) for the slice's V_shard entries, the float32 values that
 * dssd_edge_verify would have written there.  p_stride: elements between consecutive rows of
 * p_row_shard (>= V_shard; the slices of all shards may interleave into whole rows).  Rows of
 * sequences with accept_len outside [0, gamma] are left untouched.
 */
dssd_status dssd_edge_emit_shard(const void *logits_shard, dssd_dtype dtype, int64_t row_stride,
                                 const int32_t *accept_len, const float *row_scale,
                                 float temperature, int B, int gamma, int V_shard,
                                 float *p_row_shard, int64_t p_stride, void *cuda_stream);

/* Bytes of scratch shared by dssd_resample_shard_mass and dssd_resample_shard_draw. */
size_t dssd_resample_shard_workspace_bytes(int B, int gamma, int V_shard);

/*
 * One shard's masses for the draw (Section 3, "Resample"): mass[b, 0] = sum over the slice of
 * max(0, p_v - q_{n,v}) (of p_v when n == gamma: the bonus draw), mass[b, 1] = sum over the slice
 * of p_v (what the draw falls back to when no shard has residual mass); float64, NaN for a
 * sequence with n outside [0, gamma].
 *
 * p_row_shard   [B, V_shard] float32, p_stride elements between rows
 * draft_q_shard [B, gamma, V_shard] float32: row (b, i) starts at element (b*gamma+i)*q_stride
 *               (may be NULL iff gamma == 0); only row n of each sequence is read
 * mass          [B, 2] float64 out
 * workspace     >= dssd_resample_shard_workspace_bytes(...) bytes, 256-byte aligned; it keeps the
 *               per-chunk sums that dssd_resample_shard_draw needs: pass the same, untouched
 *               buffer to that call
 */
dssd_status dssd_resample_shard_mass(const float *p_row_shard, int64_t p_stride,
                                     const float *draft_q_shard, int64_t q_stride,
                                     const int32_t *accept_len, int B, int gamma, int V_shard,
                                     double *mass, void *workspace, size_t workspace_bytes,
                                     void *cuda_stream);

/*
 * The draw as shard g sees it.  masses [G, B, 2] are the G outputs of dssd_resample_shard_mass,
 * shard-major.  Z = sum_g masses[g, b, 0] (in shard order); if Z <= 0 for a rejected sequence the
 * draw falls back to the plain masses (DSSD_RS_FLAG_FALLBACK); t = u' * Z; the owner is the first
 * shard whose running total exceeds t (the last shard with mass if rounding leaves none).  On the
 * owner token[b] = v_begin + min{k : c_k > t - (mass before the shard)} over its slice, as in
 * dssd_device_resample; on every other shard token[b] = -1.  flags[b] are the sequence's
 * DSSD_RS_FLAG_* and are the same on every shard.  The other arguments as for the mass call,
 * with the same rows and the workspace that call left.
 */
dssd_status dssd_resample_shard_draw(const double *masses, int G, int g, int v_begin,
                                     const float *p_row_shard, int64_t p_stride,
                                     const float *draft_q_shard, int64_t q_stride,
                                     const int32_t *accept_len, const float *uniforms, int B,
                                     int gamma, int V_shard, int32_t *token, uint32_t *flags,
                                     const void *workspace, size_t workspace_bytes,
                                     void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DSSD_H */
